/*
 * ffsplit.h -- C ABI of the split feed-forward network library (FFSplit, arXiv 2401.04044).
 *
 * The library follows the paper's statement of the problem, per FFN layer:
 *   weights U = W1 [d, m], V = W2 [m, d]  (Section 2: FFN(X) = sigma(X U) V)
 *   -> calibration scores per neuron                      (Eq. 3, Section 4.2)
 *   -> heavy-hitter index set h2 = top-k neurons          (Sections 4.1, 5.1.1)
 *   -> split weights U1 = U[:, h2], V1 = V[h2, :] kept dense, the remaining
 *      U2, V2 replaced by rank-r factors                  (Figure 3 caption, Section 5.1.1)
 *   -> forward FFN(X) = FFN_1(X) + FFN_2(X)               (Eq. 2)
 *
 * Conventions for every entry point
 *   - All tensors are row-major and dense.  "dev" pointers are CUDA device
 *     memory owned by the caller; the library never allocates, frees or keeps
 *     a tensor pointer past the call (the workspace is kept until replaced;
 *     a packed blob's address is remembered as the key under which its header
 *     is registered, see ffsplit_blob_open()).
 *   - Storage dtype (ffsplit_dtype) applies to X, Y, weights, biases and
 *     factors alike: FFSPLIT_BF16 computes with bf16 tensor-core products and
 *     fp32 accumulation; FFSPLIT_F32 computes in plain fp32 (no TF32).
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).  Calls
 *     enqueue work and return; argument errors are returned synchronously and
 *     launch nothing.  Conditions only the device can see (non-finite score,
 *     unsorted index list, a blob whose bytes changed after registration, a
 *     wait that ran out) are recorded in a status word inside the workspace
 *     and returned by ffsplit_poll().
 *   - Device pointers must be 16-byte aligned (FFSPLIT_ERR_ALIGN otherwise).
 *     For FFSPLIT_BF16, d must be a multiple of 8 (rows of X start 16-byte aligned).
 *   - Same inputs give bitwise the same outputs on every call.
 *   - Functions return FFSPLIT_OK (0) or an error code; ffsplit_last_error()
 *     gives the text for the last failing call on that context.
 *   - A context is bound to one device and is not thread-safe.
 */
#ifndef FFSPLIT_H_
#define FFSPLIT_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  FFSPLIT_OK = 0,
  FFSPLIT_ERR_INVALID_ARG = 1,
  FFSPLIT_ERR_SHAPE = 2,
  FFSPLIT_ERR_ALIGN = 3,
  FFSPLIT_ERR_DTYPE = 4,
  FFSPLIT_ERR_BUFFER_TOO_SMALL = 5,
  FFSPLIT_ERR_NONFINITE = 6,
  FFSPLIT_ERR_BAD_BLOB = 7,
  FFSPLIT_ERR_ARCH = 8,
  FFSPLIT_ERR_CUDA = 9,
  FFSPLIT_ERR_TIMEOUT = 10,
  FFSPLIT_ERR_BAD_INDEX = 11
} ffsplit_status;

typedef enum { FFSPLIT_F32 = 0, FFSPLIT_BF16 = 1 } ffsplit_dtype;

/* sigma of Section 2.  GELU_ERF is x*Phi(x); GELU_TANH the tanh form; SWIGLU is
 * SiLU(X W1) * (X W1u) with no bias (named in Section 2 as the other dominant family). */
typedef enum { FFSPLIT_GELU_ERF = 0, FFSPLIT_GELU_TANH = 1, FFSPLIT_SWIGLU = 2 } ffsplit_act;

/* Which reading of the importance score is accumulated (see ffsplit_score). */
typedef enum { FFSPLIT_SCORE_EQ3 = 0, FFSPLIT_SCORE_ACT_ONLY = 1, FFSPLIT_SCORE_SUM_NORM = 2 } ffsplit_score_mode;

typedef struct {
  int32_t d;       /* hidden width (columns of X)                */
  int32_t m;       /* d_ff, number of FFN neurons                */
  int32_t act;     /* ffsplit_act                                */
  int32_t dtype;   /* ffsplit_dtype of every tensor of the layer */
} ffsplit_shape;

/* One dense FFN layer.  All dev pointers in the storage dtype. */
typedef struct {
  const void* W1;   /* dev [d, m]   U (GELU) or the gate projection (SwiGLU) */
  const void* W1u;  /* dev [d, m]   SwiGLU up projection, else NULL           */
  const void* b1;   /* dev [m]      first-layer bias, NULL = zeros (must be NULL for SwiGLU) */
  const void* W2;   /* dev [m, d]   V                                          */
  const void* b2;   /* dev [d]      output bias, NULL = zeros                  */
} ffsplit_weights;

/* Rank-r factors of the light slices, light neurons in ascending index order
 * (Section 5.1.1: SVD on U2 and V2 only).  U2 ~ A1 B1, V2 ~ A2 B2. */
typedef struct {
  const void* A1;   /* dev [d, r]        */
  const void* B1;   /* dev [r, m-k]      */
  const void* A1u;  /* dev [d, r]        SwiGLU up slice, else NULL */
  const void* B1u;  /* dev [r, m-k]      SwiGLU up slice, else NULL */
  const void* A2;   /* dev [m-k, r]      */
  const void* B2;   /* dev [r, d]        */
  int32_t r;
} ffsplit_factors;

typedef struct ffsplit_ctx ffsplit_ctx;

/* Create / destroy a context on CUDA device `device` (host memory only; no
 * device allocation).  Fails with FFSPLIT_ERR_ARCH unless the device is
 * compute capability 10.x, FFSPLIT_ERR_CUDA if the runtime reports an error. */
ffsplit_status ffsplit_create(ffsplit_ctx** out, int device);
ffsplit_status ffsplit_destroy(ffsplit_ctx* ctx);

/* Bytes of caller-provided scratch needed for ffsplit_forward() with up to
 * T_fwd tokens and ffsplit_score() with up to T_cal tokens per call on a layer
 * of this shape split with (k, r).  Pass 0 for a phase that is not used.
 * Always >= 65536 (the control block: device status word and kernel tickets). */
ffsplit_status ffsplit_workspace_size(const ffsplit_shape* shape, int64_t T_fwd, int64_t T_cal,
                                      int32_t k, int32_t r, size_t* bytes);

/* Give the context its scratch memory (dev, 256-byte aligned, >= 65536 bytes).  The
 * first 65536 bytes hold the device status word and kernel tickets and are cleared
 * here, synchronously.
 * The workspace must outlive every call that uses the context, and calls that
 * share a workspace must not overlap on the GPU. */
ffsplit_status ffsplit_set_workspace(ffsplit_ctx* ctx, void* dev_ptr, size_t bytes);

/* Heavy-hitter scoring over one batch of calibration tokens (Eq. 3; Section
 * 4.2: the calibration pass over a small token set).
 *   X       dev [T, d] calibration tokens, T >= 1
 *   energy  dev float[m], caller-owned accumulator: e_j = sum_t H[t,j]^2 with
 *           H = sigma(X W1 + b1) (sum_t |H[t,j]| for SCORE_SUM_NORM).
 *           accumulate = 0 overwrites it, 1 adds this batch to it.
 *   scores  dev float[m] or NULL.  When given: s_j = e_j * w_j (EQ3),
 *           e_j (ACT_ONLY) or e_j * sqrt(w_j) (SUM_NORM), w_j = sum_c W2[j,c]^2,
 *           formed from the accumulated energy after this batch.
 * The T x m activation matrix is never written to memory.  Uses the workspace.
 * With accumulate = 1, the transposed weights a previous batch left in the workspace
 * are reused when the weight pointers and the shape are the same and no other call
 * has used the workspace in between: do not change the weights during an accumulation. */
ffsplit_status ffsplit_score(ffsplit_ctx* ctx, const ffsplit_shape* shape, const ffsplit_weights* weights,
                             const void* X, int64_t T, int32_t mode, int32_t accumulate,
                             float* energy, float* scores, void* stream);

/* ffsplit_score() with the calibration tokens in HOST memory (Eq. 3; Section 4.2): X_host [T, d] is
 * copied to the device in chunks that pass through the workspace (pinned host memory makes the copies
 * asynchronous), each chunk is scored and added to `energy`; `scores` is formed after the last one.
 * Weights, energy and scores are device memory as for ffsplit_score().  The workspace must hold the
 * scoring buffers plus at least 128 staged tokens (ffsplit_workspace_size(shape, 0, T_cal, 0, 0) plus
 * T_cal * d * sizeof(dtype) stages all of a T_cal-token batch at once); FFSPLIT_ERR_BUFFER_TOO_SMALL
 * otherwise.  Copies and kernels are all enqueued on `stream`. */
ffsplit_status ffsplit_score_host(ffsplit_ctx* ctx, const ffsplit_shape* shape, const ffsplit_weights* weights,
                                  const void* X_host, int64_t T, int32_t mode, int32_t accumulate,
                                  float* energy, float* scores, void* stream);

/* Scores from an energy vector that is already complete (Eq. 3: s_j = e_j * ||V_j||^2, or the other
 * modes of ffsplit_score): for calibration runs whose energy was accumulated elsewhere -- over several
 * calls with scores = NULL, or summed over the ranks of a token-sharded calibration (Section 4.2; every
 * rank then forms bitwise the same scores from the same summed energy).
 *   W2      dev [m, d]; may be NULL for SCORE_ACT_ONLY
 *   energy  dev float[m], read (and left unchanged); scores dev float[m], written
 * Workspace: 65536 + 4 m bytes. */
ffsplit_status ffsplit_score_finalize(ffsplit_ctx* ctx, const ffsplit_shape* shape, const void* W2, int32_t mode,
                                      float* energy, float* scores, void* stream);

/* Eq. 3 from a stored activation matrix: the same energy, scores and modes as ffsplit_score, for a
 * caller that already holds H = sigma(X U) [T, m] in device memory (kept from a forward pass, say), so
 * that scoring is one streaming read of H instead of a product: e_j (+)= sum_t H[t,j]^2 (SUM_NORM:
 * sum_t |H[t,j]|), then s_j as in ffsplit_score.  For SwiGLU, H is SiLU(X Wg) * (X Wu).
 *   H          dev [T, m] row-major, shape->dtype, 16-byte aligned
 *   W2         dev [m, d]; may be NULL when scores is NULL or mode is ACT_ONLY
 *   energy, scores, accumulate, mode: as for ffsplit_score
 * Workspace: what ffsplit_workspace_size(shape, 0, T, 0, 0) reports is enough.  Partial sums are added
 * in a fixed order: results are bitwise reproducible.  Rounding differs from ffsplit_score, which
 * squares the un-rounded fp32 activations: here H has already been rounded to its storage type. */
ffsplit_status ffsplit_score_activations(ffsplit_ctx* ctx, const ffsplit_shape* shape, const void* H, int64_t T,
                                         const void* W2, int32_t mode, int32_t accumulate, float* energy,
                                         float* scores, void* stream);

/* Deterministic top-k (Section 4.1: the neurons with the highest output norm
 * are the heavy hitters).  Equal scores go to the lower index.
 *   scores     dev float[m], finite (a NaN/Inf sets FFSPLIT_ERR_NONFINITE in the status block)
 *   heavy_idx  dev int32[k], ascending           (may be NULL when k == 0)
 *   light_idx  dev int32[m-k], ascending, or NULL if not wanted
 * 0 <= k <= m. */
ffsplit_status ffsplit_select(ffsplit_ctx* ctx, const float* scores, int32_t m, int32_t k,
                              int32_t* heavy_idx, int32_t* light_idx, void* stream);

/* Size of the packed layer: `padded_bytes` is what ffsplit_pack() writes (tile
 * padding and header included), `logical_bytes` counts the split model's
 * weights and biases only: sizeof(dtype) * ((n_in+1) * (d k + r (d + m - k)) + m + d). */
ffsplit_status ffsplit_pack_size(const ffsplit_shape* shape, int32_t k, int32_t r,
                                 size_t* padded_bytes, size_t* logical_bytes);

/* Build the split layer (Figure 3 caption: U1 = U[:, h2], V1 = V[h2, :], kept
 * unchanged; the light slices are given as factors).
 *   heavy_idx  dev int32[k], strictly ascending, each in [0, m)  (else
 *              FFSPLIT_ERR_BAD_INDEX in the status block)
 *   factors    NULL (or r == 0) drops the light part: required when k == m;
 *              with k < m it yields FFN_1 alone
 *   blob       dev, 256-byte aligned, blob_bytes >= padded_bytes; position
 *              independent (may be copied or saved and reloaded as bytes)
 * The heavy slices in the blob are bit-exact copies of the inputs. */
ffsplit_status ffsplit_pack(ffsplit_ctx* ctx, const ffsplit_shape* shape, const ffsplit_weights* weights,
                            const int32_t* heavy_idx, int32_t k, const ffsplit_factors* factors,
                            void* blob, size_t blob_bytes, void* stream);

/* Register a blob that reached device memory by other means than ffsplit_pack() on this context (a
 * copy, a reload, a pack on another context).  The forward calls accept only blobs that were packed or
 * opened on the context they are called on (FFSPLIT_ERR_BAD_BLOB otherwise; nothing is opened
 * implicitly).  The 256-byte header is copied to the host on `stream`, which is then synchronised, and
 * validated against blob_bytes, the size of the caller's buffer: FFSPLIT_ERR_BAD_BLOB if it is not a
 * blob or claims more than blob_bytes.  The bytes of the blob must be complete in `stream`'s order
 * (pass the stream that produced them, or synchronise first).
 * A registration is keyed by the blob's address and describes the bytes that were there at the time:
 * after overwriting a registered buffer with another blob, or before reusing its address for something
 * else, call ffsplit_blob_open() again or ffsplit_blob_close().  As a safeguard the first kernel of
 * every forward compares the header in device memory with the registered one and reports a mismatch
 * as FFSPLIT_ERR_BAD_BLOB through ffsplit_poll(); the output of such a call is undefined. */
ffsplit_status ffsplit_blob_open(ffsplit_ctx* ctx, const void* blob, size_t blob_bytes, void* stream);

/* Forget a blob (packed or opened on this context).  FFSPLIT_ERR_BAD_BLOB if it is not known. */
ffsplit_status ffsplit_blob_close(ffsplit_ctx* ctx, const void* blob);

/* Where one matrix of the blob lives, for inspection and tests.
 * which: 0 heavy U1^T [k_pad, d] (1: SwiGLU up), 2 A1^T [r_pad, d] (3: up),
 *        4 B1^T [mL_pad, r_pad] (5: up), 6 A2^T [r_pad, mL_pad],
 *        7 [V1 ; B2]^T [d, k_pad + r_pad], 8 b1[h2] f32, 9 b1[light] f32, 10 b2 f32.
 * Returns byte offset, rows, cols and leading dimension (elements). */
ffsplit_status ffsplit_blob_section(ffsplit_ctx* ctx, const void* blob, int32_t which,
                                    size_t* offset, int64_t* rows, int64_t* cols, int64_t* ld);

/* Split forward (Eq. 2): Y = sigma(X U1 + b1[h2]) V1 + sigma((X A1) B1 + b1[light]) (A2 B2) + b2.
 *   X dev [T, d], Y dev [T, d], T >= 1, both in the blob's dtype.  Uses the workspace.
 * A blob packed with k == m is the dense FFN through the same kernels. */
ffsplit_status ffsplit_forward(ffsplit_ctx* ctx, const void* blob, const void* X, int64_t T,
                               void* Y, void* stream);

/* Dense (unsplit) FFN straight from the row-major weights: Y = act(X W1 + b1) W2 + b2, the first
 * equation of Section 2 (SwiGLU: Y = (SiLU(X W1) * (X W1u)) W2).  It is the split forward with every
 * neuron heavy (h2 = all, no light part: Eq. 2 with FFN_2 empty), run by the same kernels: on every call
 * the weights are first brought into the packed form inside the workspace, so the result is bit for bit
 * that of ffsplit_pack with heavy_idx = 0 .. m-1, k = m followed by ffsplit_forward.  Meant as the
 * comparator of the split forward; for repeated use pack once with k = m and call ffsplit_forward.
 *   shape, wt   as for ffsplit_pack (dev pointers, row-major, 16-byte aligned, not retained)
 *   X, Y        dev [T, d], 16-byte aligned
 * Workspace needed: ffsplit_workspace_size(shape, T, 0, m, 0), rounded up to 256, plus the padded size
 * ffsplit_pack_size(shape, m, 0) reports; FFSPLIT_ERR_BUFFER_TOO_SMALL otherwise, nothing launched. */
ffsplit_status ffsplit_forward_dense(ffsplit_ctx* ctx, const ffsplit_shape* shape, const ffsplit_weights* wt,
                                     const void* X, int64_t T, void* Y, void* stream);

/* Same computation with HOST buffers: X_host [T, d] is copied to the device,
 * the forward runs, Y is copied back to Y_host [T, d]; all three on `stream`
 * (pinned host memory makes the copies asynchronous).  The workspace must have
 * been sized for T_fwd >= T. */
ffsplit_status ffsplit_forward_host(ffsplit_ctx* ctx, const void* blob, const void* X_host, int64_t T,
                                    void* Y_host, void* stream);

/* A stack of split layers (Eq. 2 applied layer after layer, the per-stack figure of the throughput
 * reports): layer l reads what layer l-1 wrote, Y = FFN_{n-1}( ... FFN_0(X)).  Nothing sits between the
 * layers (no residual, no normalisation).  All blobs must be known to the context and share d and dtype.
 *   blobs   host array of n_layers dev pointers
 *   X, Y    dev [T, d] (ffsplit_forward_stack) or host [T, d] (ffsplit_forward_stack_host: copied in
 *           and out on `stream`, like ffsplit_forward_host)
 * Workspace: ffsplit_stack_workspace_size() (the largest per-layer need plus two [T, d] buffers). */
ffsplit_status ffsplit_stack_workspace_size(ffsplit_ctx* ctx, const void* const* blobs, int32_t n_layers, int64_t T,
                                            size_t* bytes);
ffsplit_status ffsplit_forward_stack(ffsplit_ctx* ctx, const void* const* blobs, int32_t n_layers, const void* X,
                                     int64_t T, void* Y, void* stream);
ffsplit_status ffsplit_forward_stack_host(ffsplit_ctx* ctx, const void* const* blobs, int32_t n_layers,
                                          const void* X_host, int64_t T, void* Y_host, void* stream);

/* The split forward of ffsplit_forward() for callers that cannot allocate device memory.
 * (The paper has no counterpart to this entry point; it exists for deployment.)
 *
 * Who needs it: code that runs the per-token decode step inside a host application that owns
 * all of the GPU's memory -- an inference server that has handed every free byte to its KV-cache
 * arena, a plug-in called from inside another runtime's execution step -- where cudaMalloc would
 * fail, or would stall the device, and where no workspace was set aside for this library.  This
 * call needs no ffsplit_set_workspace(): its intermediates, K-split partials and counters live in
 * a 4.06 MiB array built into the library (held by every GPU that loads the library, from load
 * until the process exits).  It calls no allocator of any kind.
 *
 *   blob  dev  a bf16 layer packed by ffsplit_pack() (GELU or SwiGLU)
 *   X     dev  [T, d], Y dev [T, d], 1 <= T <= 8
 * Limits, rejected with an error and nothing launched: T > 8 (FFSPLIT_ERR_SHAPE), fp32 layers
 * (FFSPLIT_ERR_DTYPE), layers whose intermediates T*(k_pad + (n_in+1)*r_pad + mL_pad)*2 bytes
 * exceed 2 MiB (FFSPLIT_ERR_BUFFER_TOO_SMALL).
 * The first call on a device looks up the array's device address and sets kernel attributes;
 * make that first call outside any stream capture.
 * All calls on a device share the one array and it keeps the previous call's contents: the call
 * clears the counters it needs at zero itself, but two calls that overlap on the GPU (different
 * streams, no ordering between them) race on it.  Results equal those of ffsplit_forward() where that call runs the same weight-streaming
 * kernels (it takes large GELU layers through its tensor-core path instead: equal within rounding there).
 * Like ffsplit_forward() it accepts only blobs packed or opened on `ctx`.  A device-side condition of
 * this call (a wait that ran out, a changed blob) is kept in the array's own status words until
 * ffsplit_poll() on any context of that device reports it; ffsplit_poll() needs no workspace for that. */
ffsplit_status ffsplit_forward_noalloc(ffsplit_ctx* ctx, const void* blob, const void* X, int64_t T,
                                       void* Y, void* stream);

/* ---- On-device factors of the light slices (Section 5.1.1: the low-rank decomposition is applied to U2
 * and V2 only; Section 5.1.1 fixes the rank, not the algorithm) --------------------------------------------
 * The step between ffsplit_select() and ffsplit_pack() without leaving the GPU.  For W = U2 = W1[:, light]
 * (d x (m-k)), for the SwiGLU up slice likewise, and for W = V2^T with V2 = W2[light, :], an orthonormal basis
 * Q [d, r] of the dominant left singular subspace is found by `iters` rounds of block power iteration
 * (Y = W W^T Q on the tensor cores in bf16 with fp32 accumulation, Q = orth(Y) by Cholesky QR in fp32) from
 * the starting basis the caller supplies, and the factors of the projection Q Q^T W are returned:
 *     U2 ~ A1 B1,  A1 = Q, B1 = Q^T U2            V2 ~ A2 B2,  A2 = V2 Q, B2 = Q^T
 * As span(Q) converges to the leading singular subspace, A B converges to the truncated SVD's product, the
 * best rank-r approximation (Eckart-Young); the factors themselves differ from U_r S_r^(1/2), S_r^(1/2) V_r^T
 * by an invertible r x r mixing, which the forward does not see.  With a random starting basis, 6 rounds bring
 * the Frobenius error within about 1 % of the optimum on the layers the tests use (tests/test_gpu_factor.py).
 *   light_idx  dev int32[m-k], ascending (ffsplit_select's output); an index outside [0, m) reads as a zero neuron
 *   start      dev bf16 [n][r, d], n = 2 (GELU: bases for U2, V2) or 3 (SwiGLU: gate, V2, up); full row rank
 *              (draw it from a normal distribution: the library draws no random numbers)
 *   A1 [d, r], B1 [r, m-k], A2 [m-k, r], B2 [r, d] (and A1u, B1u for SwiGLU, else NULL): dev bf16, written;
 *              the layouts ffsplit_factors takes
 * bf16 layers, 1 <= r <= min(d, m-k, 2048), 0 <= iters <= 64.  Uses the workspace (ffsplit_factor_workspace_size).
 * A Gram matrix that is not positive definite (a rank-deficient start or slice) is reported as
 * FFSPLIT_ERR_NONFINITE through ffsplit_poll(); the factors are then finite but meaningless. */
ffsplit_status ffsplit_factor_workspace_size(const ffsplit_shape* shape, int32_t k, int32_t r, size_t* bytes);
ffsplit_status ffsplit_factor_light(ffsplit_ctx* ctx, const ffsplit_shape* shape, const ffsplit_weights* weights,
                                    const int32_t* light_idx, int32_t k, int32_t r, int32_t iters, const void* start,
                                    void* A1, void* B1, void* A2, void* B2, void* A1u, void* B1u, void* stream);

/* ---- The transformer block around the FFN (Section 5.1.2, Table 2: the paper times whole BERT-base models) --
 * One post-LayerNorm encoder layer, so that the split FFN can be timed in its context:
 *     A  = MultiHeadAttention(X)          Q, K, V = X Wq, X Wk, X Wv (+ biases), heads of width 64,
 *                                         softmax(Q K^T / 8) V per head and sequence, heads concatenated, times Wo (+ bo)
 *     X1 = LayerNorm(X + A)               over the d features, with gain and bias
 *     Y  = LayerNorm(X1 + FFN(X1))        FFN = the packed layer `ffn_blob`, split or dense (Eq. 2)
 * Scope: bf16, d = heads * 64 <= 1024, sequences of `seq` <= 128 tokens attended whole (no padding mask),
 * T = batch * seq tokens stored sequence after sequence.  The projection weights are given K-major (row j of
 * Wqkv_t holds the d input weights of output feature j; features 0..d-1 are Q, d..2d-1 K, 2d..3d-1 V, head h
 * owning columns 64 h .. 64 h + 63 of each), the way every right operand of this library is stored. */
typedef struct {
  int32_t batch, seq, heads;
  const void* Wqkv_t;      /* dev bf16 [3 d, d]  */
  const float* bqkv;       /* dev float [3 d]    */
  const void* Wo_t;        /* dev bf16 [d, d]    */
  const float* bo;         /* dev float [d]      */
  const float* ln1_gamma;  /* dev float [d]      */
  const float* ln1_beta;
  const float* ln2_gamma;
  const float* ln2_beta;
  float ln_eps;            /* added to the variance (BERT: 1e-12) */
  const void* ffn_blob;    /* packed FFN of width d, packed or opened on the context */
} ffsplit_encoder_layer;

/* Workspace ffsplit_encoder_forward() needs for this layer (the FFN's own forward buffers included). */
ffsplit_status ffsplit_encoder_workspace_size(ffsplit_ctx* ctx, const ffsplit_encoder_layer* layer, size_t* bytes);
/* X, Y dev bf16 [batch * seq, d], 16-byte aligned; X and Y may not overlap.  Uses the workspace. */
ffsplit_status ffsplit_encoder_forward(ffsplit_ctx* ctx, const ffsplit_encoder_layer* layer, const void* X, void* Y,
                                       void* stream);

/* ---- Quantised split (Section 5.2, Table 3: round-to-nearest, group size 128, 8 bits for the heavy-hitter
 * neurons, 3 bits for everything else) ------------------------------------------------------------------
 * The second way the paper compresses the light part: instead of rank-r factors, U2 and V2 are kept whole at
 * 3 bits and U1, V1 at 8 bits.  Reading taken where the paper is silent: each of the four matrices is quantised
 * on its own, per output channel, in groups of 128 consecutive weights along its input dimension (along d for a
 * neuron's column of U; along the part's neurons, in ascending index order, for a column of V; a last group may
 * be shorter); asymmetric min/max grid, weight = lo + code * scale with lo = min, scale = (max - min) / (2^b - 1),
 * code = round-half-even((w - lo) / scale), all decided in float32; scale and lo are stored as float32; biases
 * are not quantised.  bf16 layers only (GELU or SwiGLU). */

/* Size of the quantised packed layer.  logical_bytes = the codes at their bit width + 8 bytes per group
 * + 4 (m + d) bytes of float32 biases. */
ffsplit_status ffsplit_quant_pack_size(const ffsplit_shape* shape, int32_t k, size_t* padded_bytes, size_t* logical_bytes);

/* Workspace ffsplit_quant_forward() needs for a layer of this shape and split (any token count). */
ffsplit_status ffsplit_quant_workspace_size(const ffsplit_shape* shape, int32_t k, size_t* bytes);

/* Quantise and pack a layer.  heavy_idx dev int32[k] and light_idx dev int32[m-k] are the two ascending
 * lists ffsplit_select() writes (heavy_idx is validated like in ffsplit_pack(); light_idx must be its
 * complement).  blob dev, 256-byte aligned, >= padded_bytes.  Needs a workspace (status word only). */
ffsplit_status ffsplit_quant_pack(ffsplit_ctx* ctx, const ffsplit_shape* shape, const ffsplit_weights* weights,
                                  const int32_t* heavy_idx, int32_t k, const int32_t* light_idx, void* blob,
                                  size_t blob_bytes, void* stream);

/* Register a quantised blob that was not packed on this context (see ffsplit_blob_open()). */
ffsplit_status ffsplit_quant_blob_open(ffsplit_ctx* ctx, const void* blob, size_t blob_bytes, void* stream);

/* Expand one matrix of a quantised blob, for inspection and tests.
 * which: 0 U1 [k, d]   1 U2 [m-k, d]   2 / 3 the SwiGLU up projections likewise   4 V1 [d, k]   5 V2 [d, m-k]
 * (rows = output channels, columns = the grouped input axis).
 *   codes dev uint8 [rows, cols]; scale, lo dev float [rows, ceil(cols / 128)] */
ffsplit_status ffsplit_quant_unpack(ffsplit_ctx* ctx, const void* blob, int32_t which, uint8_t* codes, float* scale,
                                    float* lo, void* stream);

/* Eq. 2 on the quantised weights: Y = sigma(X U1~ + b1[h2]) V1~ + sigma(X U2~ + b1[light]) V2~ + b2, with
 * w~ = lo + code * scale applied inside the weight-streaming kernel (the few-token path: the tokens are taken
 * eight at a time, one launch each; meant for decode, T <= 8).  X, Y dev bf16 [T, d].  Uses the workspace. */
ffsplit_status ffsplit_quant_forward(ffsplit_ctx* ctx, const void* blob, const void* X, int64_t T, void* Y, void* stream);

/* Synchronise `stream`, then return and clear the first device-side condition found in the workspace's
 * status word or in that of the built-in scratch of ffsplit_forward_noalloc() on the context's device
 * (FFSPLIT_OK if no kernel recorded one).  Works on a context without a workspace. */
ffsplit_status ffsplit_poll(ffsplit_ctx* ctx, void* stream);

/* Self-test of the bounded waits (every wait inside the library's kernels gives up after a limit
 * instead of spinning forever): launches a one-CTA kernel whose wait on a barrier that nothing signals
 * is limited to `limit_cycles` SM clocks (1 .. 1e8).  The wait runs out, the kernel returns normally,
 * and the next ffsplit_poll() reports FFSPLIT_ERR_TIMEOUT; the context stays usable.  (The paper has no
 * counterpart; this is a diagnostic.)  Needs a workspace (for the status word). */
ffsplit_status ffsplit_debug_wait_timeout(ffsplit_ctx* ctx, int64_t limit_cycles, void* stream);

/* Per-launch device timing of the library's main kernels, for roofline reports.
 * Between ffsplit_profile_begin() and ffsplit_profile_end() every launch of a
 * kernel class is bracketed by CUDA events on its stream.  profile_end
 * synchronises `stream` and returns, for `kernel_class` (0 tensor-core GEMM,
 * 1 fp32 GEMM, 2 few-token streaming forward): the number of launches, the sum
 * of their durations in milliseconds and the sum of their algorithmic work
 * (FLOPs for the GEMMs, bytes for the streaming kernel; unpadded sizes).
 * Profiling adds event overhead between kernels: never time a step with it on. */
ffsplit_status ffsplit_profile_begin(ffsplit_ctx* ctx);
ffsplit_status ffsplit_profile_end(ffsplit_ctx* ctx, void* stream, int32_t kernel_class, int32_t* launches,
                                   double* total_ms, double* total_work);

/* Number of kernels this context has launched so far. */
int64_t ffsplit_launch_count(const ffsplit_ctx* ctx);

/* Text for the last error returned on this context ("" if none).  Valid until
 * the next call on the context.  ctx may be NULL (returns a static string). */
const char* ffsplit_last_error(const ffsplit_ctx* ctx);

/* Library version, major*10000 + minor*100 + patch. */
int32_t ffsplit_version(void);

#ifdef __cplusplus
}
#endif
#endif /* FFSPLIT_H_ */
