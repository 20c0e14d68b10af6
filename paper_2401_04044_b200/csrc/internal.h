// Internal declarations shared by the translation units of libffsplit.
// Nothing here is part of the public ABI (see include/ffsplit.h).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <string>
#include <unordered_map>
#include <vector>

#include "ffsplit.h"

#include <utility>

namespace ffsp {

// ----------------------------------------------------------------------------
// Device status block: the first 256 bytes of the workspace.
// word 0: first ffsplit_status recorded by a kernel (0 = none)
// word 1: detail (an index, a CTA id ...), word 2: kernel id
// ----------------------------------------------------------------------------
constexpr size_t kStatusBytes = 256;
// Control block at the start of the workspace: the status block, then the ticket
// counters of the fused light-chain kernel (zero between launches).  Cleared when
// the workspace is installed and whenever ffsplit_poll() reports a device condition.
constexpr size_t kCtrlBytes = 65536;
constexpr long long kMaxTicketTiles = (kCtrlBytes - kStatusBytes) / 4;

enum KernelId : int {
  KID_SELECT = 1, KID_PACK = 2, KID_GEMM_TC = 3, KID_GEMM_SIMT = 4, KID_SCORE = 5, KID_DECODE = 6, KID_FUSED = 7, KID_PROBE = 8, KID_QUANT = 9, KID_FACTOR = 10, KID_ENCODER = 11, KID_GEMM_AR = 12
};

__device__ __forceinline__ void record_status(int* status, int code, int detail, int kid) {
  if (atomicCAS(status, 0, code) == 0) {
    status[1] = detail;
    status[2] = kid;
  }
}

// ----------------------------------------------------------------------------
// Epilogue description shared by the tensor-core and the SIMT GEMM.
// The GEMM computes acc[row, n] = sum_k A[row, k] * B[n, k]  (both operands
// K-major).  Per output column n:
//   v = acc + (n < n_bias ? bias[n] : 0)
//   if (n < n_act) v = act(v)            (gated: v = silu(acc0) * acc1)
//   n <  n_split : C0[row * ld0 + n]            = v
//   n >= n_split : C1[row * ld1 + (n - n_split)] = v
// Score mode (col_partial != nullptr): nothing is stored; instead one partial
// per row group g and column: col_partial[g * N + n] = sum over the group's valid
// rows of act(v)^2 (or |act(v)|).  Row groups are 32 rows (tensor-core kernel)
// or 64 rows (SIMT kernel).
// ----------------------------------------------------------------------------
struct Epilogue {
  void* C0;
  void* C1;
  long long ld0;
  long long ld1;
  const float* bias;
  float* col_partial;
  int n_split;
  int n_act;
  int n_bias;
  int act;        // ffsplit_act
  int score_abs;  // 1: accumulate |v| instead of v^2
  int c0_f32;     // tensor-core kernel only: C0 is float (the Gram matrices of the on-device factorisation)
  // Blob guard (first kernel of a forward only, else nullptr): the 256-byte header at `guard` must still
  // hash to `guard_hash`, the value taken when the blob was packed or opened on this context; a blob whose
  // bytes were replaced behind the library's back is reported as FFSPLIT_ERR_BAD_BLOB through the status block.
  const unsigned long long* guard;
  unsigned long long guard_hash;
};

// Hash of a 256-byte blob header (32 words of 8 bytes), the same on host and device.
__host__ __device__ __forceinline__ unsigned long long header_word_mix(unsigned long long w, int i) {
  unsigned long long v = (w + static_cast<unsigned long long>(i) + 1ull) * 0x9E3779B97F4A7C15ull;
  return v ^ (v >> 29);
}
inline unsigned long long header_hash_host(const void* hdr256) {
  const unsigned long long* w = static_cast<const unsigned long long*>(hdr256);
  unsigned long long h = 0;
  for (int i = 0; i < 32; ++i) h ^= header_word_mix(w[i], i);
  return h;
}
#ifdef __CUDACC__
// Called by one whole warp.
__device__ __forceinline__ void check_blob_guard(const Epilogue& e, int* status, int kid) {
  if (e.guard == nullptr) return;
  const int lane = threadIdx.x & 31;
  unsigned long long h = header_word_mix(e.guard[lane], lane);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) h ^= __shfl_xor_sync(0xffffffffu, h, o);
  if (lane == 0 && h != e.guard_hash) record_status(status, FFSPLIT_ERR_BAD_BLOB, 0, kid);
}
#endif

struct GemmArgs {
  const void* A0;   // [M, K], leading dimension lda0
  const void* B0;   // [N, K], leading dimension ldb0
  const void* A1;   // gated GEMM: second operand pair (acc1), else nullptr
  const void* B1;
  long long lda0, ldb0, lda1, ldb1;
  long long M;
  int N;
  int K;
  double algo_flops;  // unpadded FLOPs of this product, for profiling reports
  // Few tokens (M <= 64) on the tensor cores: the product is run with the operands exchanged (weights as the rows of
  // the accumulator, tokens as its columns), cut along K into enough work units to fill the SMs, and finished by a
  // small kernel that adds the fp32 partials, applies this epilogue and stores the transpose.  Needs scratch.
  void* few; size_t few_bytes;
  int force_split;    // internal: K ranges of the exchanged product (set by the few-token path)
  int trans_tokens;   // internal: > 0 with force_split == 1: the exchanged product finishes its own output -- bias, activation
                      // and the transposed bf16 store of this many token rows -- instead of leaving an fp32 partial
  int weights_stable; // the weights (B0 / B1) are not written by the kernel before this launch in the stream (set for every
                      // product of a forward but its first): the few-token path then loads them under that kernel's tail
  int early_rows;     // internal: the row operand A0 may be loaded before the programmatic-launch wait
  void* splitk;       // optional scratch for fp32 partials: lets a thin product with a long contraction (bf16, no bias,
  size_t splitk_bytes; // no activation, one output) be cut along K over the SMs; nullptr = never
  Epilogue epi;
};

// ----------------------------------------------------------------------------
// Packed-layer header: the first 256 bytes of a blob.
// ----------------------------------------------------------------------------
constexpr uint32_t kBlobMagic = 0x46465350u;  // "FFSP"
constexpr uint32_t kBlobVersion = 1;
constexpr int kNumSections = 11;

struct BlobHeader {
  uint32_t magic, version;
  int32_t d, m, act, dtype;
  int32_t k, r, n_in;
  int32_t k_pad, r_pad, ml_pad, ml;     // ml = m - k
  int32_t reserved0;
  uint64_t total_bytes, logical_bytes;
  uint64_t off[kNumSections];           // byte offsets from the blob start
  uint8_t pad[256 - 4 * 14 - 8 * 2 - 8 * kNumSections];
};
static_assert(sizeof(BlobHeader) == 256, "blob header is 256 bytes");

enum Section : int {
  SEC_U1T = 0, SEC_U1UT = 1, SEC_A1T = 2, SEC_A1UT = 3, SEC_B1T = 4, SEC_B1UT = 5,
  SEC_A2T = 6, SEC_V1B2T = 7, SEC_B1H = 8, SEC_B1L = 9, SEC_B2 = 10
};

// ----------------------------------------------------------------------------
// Batched preparation jobs (see kernels_misc.cu)
// ----------------------------------------------------------------------------
constexpr int kMaxPrepJobs = 12;
struct PrepJob {
  int kind;
  int rows, cols, rows_pad, cols_pad, idx_limit;
  int tiles_x, block_begin;
  long long ldi, ldo;
  const void* in; const void* in2;
  void* out; void* out2; void* out3;
  const int* idx;
};
struct PrepBatch {
  PrepJob job[kMaxPrepJobs];
  int n;
};

// ----------------------------------------------------------------------------
// Host context
// ----------------------------------------------------------------------------
struct TmapKey {
  const void* ptr; long long rows, cols, ld; int box_rows; int box_cols;
  bool operator==(const TmapKey& o) const {
    return ptr == o.ptr && rows == o.rows && cols == o.cols && ld == o.ld && box_rows == o.box_rows &&
           box_cols == o.box_cols;
  }
};
struct TmapKeyHash {
  size_t operator()(const TmapKey& k) const {
    size_t h = reinterpret_cast<size_t>(k.ptr);
    auto mix = [&h](size_t v) { h ^= v + 0x9e3779b97f4a7c15ull + (h << 6) + (h >> 2); };
    mix((size_t)k.rows); mix((size_t)k.cols); mix((size_t)k.ld); mix((size_t)k.box_rows); mix((size_t)k.box_cols);
    return h;
  }
};

}  // namespace ffsp

constexpr int kFewTensorAuto = -2;

struct ffsplit_ctx {
  int device = 0;
  int num_sms = 0;
  int cc_major = 0, cc_minor = 0;
  char* ws = nullptr;
  size_t ws_bytes = 0;
  long long launches = 0;
  std::string err;
  struct BlobEntry { ffsp::BlobHeader h; size_t bytes; unsigned long long hash; };
  std::unordered_map<const void*, BlobEntry> blobs;   // blobs packed or opened on this context, by address
  struct QuantEntry { unsigned char header[256]; size_t bytes; unsigned long long hash; };
  std::unordered_map<const void*, QuantEntry> qblobs; // quantised blobs (Section 5.2), likewise
  std::unordered_map<ffsp::TmapKey, CUtensorMap, ffsp::TmapKeyHash> tmaps;
  void* encode_fn = nullptr;  // cuTensorMapEncodeTiled
  struct ProfRec { int cls; cudaEvent_t a, b; double work; };
  bool profiling = false;
  std::vector<ProfRec> prof;
  ffsp::PrepBatch prep{};
  int prep_blocks = 0;
  bool prep_active = false;
  bool attr_tc_set = false;
  bool attr_fused_set = false;
  bool attr_ares_set = false;
  bool attr_layer_set = false;
  bool attr_att_set = false;
  int* status() const { return reinterpret_cast<int*>(ws); }
  int* tickets() const { return reinterpret_cast<int*>(ws + ffsp::kStatusBytes); }
  int gemm_two_m = 1;          // tensor-core GEMM: 256-row tiles where they pay (FFSPLIT_GEMM_TWO_M=0: never, 2: wherever allowed)
  int few_tensor_min = kFewTensorAuto;   // few-token forward (up to 64 tokens): token counts above this take the
                               // tensor-core path with exchanged operands, the others the weight-streaming kernels
                               // (FFSPLIT_FEW_TENSOR_MIN; -1 = always the tensor path, 64 = never).  Unset: chosen per
                               // layer from its size and activation, see decode_path_applies()
  int gemm_ares = 1;           // short contractions (K <= 512) with the row operand resident in tensor memory (FFSPLIT_GEMM_ARES=0: never)
  int gemm_split_k = 1;        // tensor-core GEMM: cut thin products with a long contraction along K (FFSPLIT_GEMM_SPLIT_K=0: never)
  int gemm_panel = 0;          // tensor-core GEMM: tile rows per panel of the tile walk (0: chosen per launch; FFSPLIT_GEMM_PANEL)
  int decode_one_launch = 0;   // few-token forward: 1 = all products in one cooperative launch (FFSPLIT_DECODE_LAYER=1), 0 = one launch per product
  int decode_stream = 1;       // few tokens: 1 = the single-launch streaming kernel where it is the faster one, 2 = for every T <= 8, 0 = never (FFSPLIT_DECODE_STREAM)
  int use_fused = -1;  // -1: not decided yet (environment FFSPLIT_NO_FUSED=1 turns the fused kernel off)
  int use_layer_kernel = 1;    // small hidden widths at prefill: the whole split layer in one cluster launch (FFSPLIT_LAYER_KERNEL=0: off)
  // What the scoring region of the workspace holds from the last ffsplit_score() call: U^T, the fp32 bias
  // and ||V_j||^2 of these weights.  A later batch of the same accumulation (accumulate = 1, same pointers
  // and shape) reuses them; any other call that writes the workspace clears `valid`.
  struct ScorePrep {
    bool valid = false, has_w = false;
    const void *W1 = nullptr, *W1u = nullptr, *b1 = nullptr, *W2 = nullptr;
    int d = 0, m = 0, act = 0, dtype = 0;
  } score_prep;
};

namespace ffsp {

ffsplit_status fail(ffsplit_ctx* ctx, ffsplit_status code, const std::string& msg);
ffsplit_status check_cuda(ffsplit_ctx* ctx, cudaError_t e, const char* what);

inline int round_up(int v, int q) { return (v + q - 1) / q * q; }
inline long long round_up_ll(long long v, long long q) { return (v + q - 1) / q * q; }
inline size_t elem_size(int dtype) { return dtype == FFSPLIT_BF16 ? 2 : 4; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// ----------------------------------------------------------------------------
// Few-token forward (T <= 64): the products of one layer, run by one persistent kernel
// (decode_layer.cu).  C[t, n] = epi(sum_k X[t, k] W[n, k]); W1 != nullptr: gated pair.
// ----------------------------------------------------------------------------
struct DecodeProduct {
  const void* X0; const void* X1; long long ldx;   // [T, K] bf16; X1 for the gated pair
  const void* W0; const void* W1; long long ldw;   // [N, K] bf16
  int N, K;
  int tiles, steps;   // row tiles (128 rows, gated 64) and k steps of 256
  Epilogue epi;
};
constexpr int kMaxDecodeProducts = 5;
struct DecodeLayerPlan {
  DecodeProduct prod[kMaxDecodeProducts];
  int n = 0;
  double algo_bytes = 0.0;
};
bool decode_layer_applies(long long T);
size_t decode_layer_scratch_bytes(int num_sms, long long T);
ffsplit_status decode_layer_add(ffsplit_ctx* ctx, DecodeLayerPlan* plan, const void* X0, const void* X1, long long ldx,
                                const void* W0, const void* W1, long long ldw, int N, int K, const Epilogue& epi,
                                double algo_bytes);
ffsplit_status decode_layer_launch(ffsplit_ctx* ctx, const DecodeLayerPlan* plan, int T, float* partial, int* ctrl,
                                   cudaStream_t st);

// Launch with programmatic stream serialisation: the kernel may be scheduled while the kernel before it in
// the stream is still running.  Every kernel launched this way executes `griddepcontrol.wait` before its
// first global-memory access (pdl_wait() below), so only its launch latency overlaps.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                              Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}
#ifdef __CUDACC__
// Wait for the kernel before this one (complete, writes visible), then let the one after start launching.
__device__ __forceinline__ void pdl_wait() {
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
#endif

// Profiling brackets: no-ops unless ffsplit_profile_begin() is active.
enum ProfClass : int { PROF_GEMM_TC = 0, PROF_GEMM_SIMT = 1, PROF_DECODE = 2, PROF_ENERGY = 3 };
int prof_open(ffsplit_ctx* ctx, int cls, double work, cudaStream_t st);
void prof_close(ffsplit_ctx* ctx, int handle, cudaStream_t st);

// preparation jobs recorded between these two calls run as one launch
void prep_begin(ffsplit_ctx* ctx);
ffsplit_status prep_flush(ffsplit_ctx* ctx, int dtype, cudaStream_t st);

// launchers (each returns a CUDA error state through check_cuda)
ffsplit_status launch_gemm(ffsplit_ctx* ctx, int dtype, const GemmArgs& g, cudaStream_t st);
ffsplit_status launch_select(ffsplit_ctx* ctx, const float* scores, int m, int k, int* heavy, int* light,
                             cudaStream_t st);
ffsplit_status launch_row_energy(ffsplit_ctx* ctx, int dtype, const void* W2, int m, int d, float* w, cudaStream_t st);
ffsplit_status launch_transpose(ffsplit_ctx* ctx, int dtype, const void* in, long long ldi, int rows, int cols,
                                void* out, long long ldo, int rows_pad_out, int cols_pad_out, const int* row_idx,
                                int idx_limit, cudaStream_t st);
ffsplit_status launch_gather_cols_t(ffsplit_ctx* ctx, int dtype, const void* in, long long ldi, int rows,
                                    const int* col_idx, int ncols, int idx_limit, void* out, long long ldo,
                                    int rows_out_pad, cudaStream_t st);
ffsplit_status launch_pack_bias(ffsplit_ctx* ctx, int dtype, const void* b1, const void* b2, const int* heavy, int m,
                                int k, int d, float* b1h, int k_pad, float* b1l, int ml_pad, float* b2o,
                                cudaStream_t st);
int column_energy_groups(long long rows);
ffsplit_status launch_column_energy(ffsplit_ctx* ctx, int dtype, const void* H, long long ldh, long long rows, int m,
                                    float* partial, int use_abs, cudaStream_t st);
ffsplit_status launch_score_finalize(ffsplit_ctx* ctx, const float* partial, int groups, int m, const float* w,
                                     float* energy, float* scores, int mode, int accumulate, cudaStream_t st);
bool fused_light_applies(int dtype, int act, int r_pad, int ml_pad);
size_t fused_light_scratch_bytes(long long T, int r_pad);
ffsplit_status launch_fused_light(ffsplit_ctx* ctx, const void* Q, long long ldq, long long T, const void* B1T,
                                  const void* A2T, const float* b1l, int r_pad, int ml_pad, int act, void* P,
                                  long long ldp, char* scratch, int* tickets, double algo_flops,
                                  cudaStream_t st);
bool fused_layer_applies(int dtype, int act, int d, int k, int k_pad, int r_pad, int ml_pad, long long T, int num_sms);
size_t fused_layer_scratch_bytes(long long T, int r_pad);
ffsplit_status launch_fused_layer(ffsplit_ctx* ctx, const BlobHeader& h, const char* blob, const void* X, long long T,
                                  char* scratch, void* H, long long ldh, void* Y, unsigned long long guard_hash,
                                  cudaStream_t st);
// forward of one packed FFN layer (split or dense) inside another entry point; defined in api.cu
ffsplit_status run_ffn_forward(ffsplit_ctx* ctx, const void* blob, const void* X, long long T, void* Y, cudaStream_t st);
size_t ffn_forward_workspace_end(ffsplit_ctx* ctx, const void* blob, long long T, ffsplit_status* status, int* d, int* dtype);
ffsplit_status launch_wait_timeout_probe(ffsplit_ctx* ctx, long long limit_cycles, cudaStream_t st);
ffsplit_status launch_to_f32(ffsplit_ctx* ctx, int dtype, const void* in, int n, float* out, cudaStream_t st);

}  // namespace ffsp
