// Few-token (decode) split forward for bf16 layers, T <= 64 tokens: the host side.
//
// With a handful of tokens every stage of Eq. 2 is a skinny product
//     C[t, n] = epi( sum_k X[t, k] * W[n, k] )        W: [N, K] K-major weights from the packed blob
// whose cost is reading W once from HBM.  This file lists the products of one layer -- stage 1
// [A_H | Q] = X [U1 | A1], the light chain H_L = act(Q B1 + b1_L), P = H_L A2, and stage 3
// Y = [A_H | P] [V1; B2] + b2 -- and hands them to the persistent weight-streaming kernel of
// decode_layer.cu.  It also holds the entry point that runs the same path out of a built-in scratch
// array, for callers that cannot allocate.
#include <cstring>
#include <mutex>

#include "decode_stream.h"
#include "epilogue.cuh"
#include "internal.h"

namespace ffsp {

constexpr long long kDecodeScratchBytes = 16ll << 20;   // fp32 partials of the row tiles that several CTAs share
constexpr long long kFewScratchBytes = 64ll << 20;      // the region's size: also the fp32 partials of the tensor-core few-token path

// ---- 1..8 tokens: the phases of one layer for decode_stream_kernel ---------------------------------------
// Every phase writes raw fp32 sums (one slice per k range); the phase that reads them adds the slices, the
// bias and the activation.  Returns FFSPLIT_ERR_BUFFER_TOO_SMALL without launching when `scratch_bytes`
// cannot hold the slices (the caller then takes the other few-token kernel).
// k ranges for a contraction of length K over `rows` output rows: at least as many as the activation operand's
// capacity demands.  One k range lets the phase finish its outputs itself (bias, activation, bf16), so more are
// taken only when the row shares would come out badly uneven over the CTAs of a phase that is big enough for
// that to matter.
static int stream_splits(int K, long long rows, int kx_max, int ncta) {
  const int k32 = (K + 31) / 32, cap = kx_max / 32;
  const int s_min = k32 <= cap ? 1 : (k32 + cap - 1) / cap;
  auto waste = [&](int s) {
    const long long U = rows * s;
    return static_cast<double>((U + ncta - 1) / ncta) * ncta / static_cast<double>(U > 0 ? U : 1);
  };
  const double bytes_per_cta = 2.0 * static_cast<double>(rows) * K / ncta;
  if (bytes_per_cta < 49152.0 || waste(s_min) <= 1.08) return s_min;
  int best = s_min;
  double best_waste = waste(s_min);
  for (int s = s_min + 1; s < s_min + 4 && s <= k32; ++s) {
    if ((k32 + s - 1) / s > cap) continue;
    const double w = waste(s);
    if (w < best_waste - 1e-9) { best_waste = w; best = s; }
    if (w <= 1.03) break;
  }
  return best;
}

static ffsplit_status stream_forward(ffsplit_ctx* ctx, const BlobHeader& h, const char* blob, const void* X, int T,
                                     void* Y, char* scratch, long long scratch_bytes, int* ctrl, cudaStream_t st,
                                     unsigned long long guard_hash, bool* launched) {
  *launched = false;
  const int d = h.d, k_pad = h.k_pad, r_pad = h.r_pad, ml_pad = h.ml_pad, kp_rp = h.k_pad + h.r_pad;
  const bool gated = h.act == FFSPLIT_SWIGLU;
  const bool light = r_pad > 0 && h.ml > 0;
  const int g2 = gated ? 2 : 1;
  auto W = [&](int sec) { return reinterpret_cast<const __nv_bfloat16*>(blob + h.off[sec]); };
  auto F = [&](int sec) { return reinterpret_cast<const float*>(blob + h.off[sec]); };
  const int x_rows = stream_x_rows(T), kx = stream_kx_max(x_rows), G = ctx->num_sms;
  const long long N1 = static_cast<long long>(g2) * (k_pad + (light ? r_pad : 0));
  const long long N2a = static_cast<long long>(g2) * ml_pad;
  const int K3 = light ? kp_rp : k_pad;
  const int S1 = stream_splits(d, N1, kx, G), S2a = stream_splits(r_pad, N2a, kx, G);
  const int S2b = stream_splits(ml_pad, r_pad, kx, G);
  // the layer output is written by the stage-3 phase itself when its contraction fits one k range
  const int S3 = (K3 + 31) / 32 <= kx / 32 ? 1 : stream_splits(K3, d, kx, G);
  // A phase with one k range whose outputs are not gated pairs finishes them itself (bf16); the others leave
  // raw fp32 slices for their readers.
  const bool fin1 = S1 == 1 && !gated, fin2a = S2a == 1 && !gated, fin2b = S2b == 1;
  // the unit arithmetic of the kernel is 32-bit
  for (long long u : {S1 * N1, S2a * N2a, static_cast<long long>(S2b) * r_pad, static_cast<long long>(S3) * d})
    if (u * (G + 1) >= 2147483648ll) return FFSPLIT_ERR_BUFFER_TOO_SMALL;
  // slices and finished vectors in the scratch area (256-byte aligned pieces)
  long long off = 0;
  auto take = [&](long long bytes) { const long long o = off; off += (bytes + 255) / 256 * 256; return o; };
  const long long o_p1 = take(fin1 ? 8 * N1 * 2 : S1 * 8 * N1 * 4);
  const long long o_2a = light ? take(fin2a ? 8 * N2a * 2 : S2a * 8 * N2a * 4) : 0;
  const long long o_2b = light ? take(fin2b ? 8ll * r_pad * 2 : static_cast<long long>(S2b) * 8 * r_pad * 4) : 0;
  const long long o_y = S3 > 1 ? take(static_cast<long long>(S3) * 8 * d * 4) : 0;
  if (off > scratch_bytes) return FFSPLIT_ERR_BUFFER_TOO_SMALL;
  auto FS = [&](long long o) { return reinterpret_cast<float*>(scratch + o); };
  auto BS = [&](long long o) { return reinterpret_cast<__nv_bfloat16*>(scratch + o); };

  StreamParams p;
  std::memset(&p, 0, sizeof(p));
  p.T = T; p.act = h.act; p.ctrl = ctrl;
  p.x_rows = x_rows; p.x_pitch = 2 * kx + 64;
  p.guard = guard_hash ? reinterpret_cast<const unsigned long long*>(blob) : nullptr;
  p.guard_hash = guard_hash;
  auto add_seg = [](StreamPhase& ph, const __nv_bfloat16* Wp, long long ldw, int rows, int x_off, int out_col,
                    int fin_kind = STREAM_IN_LINEAR, const float* fin_bias = nullptr) {
    if (rows <= 0) return;
    StreamSegment& s = ph.seg[ph.nseg++];
    s.W = Wp; s.ldw = ldw; s.rows = rows; s.x_off = x_off; s.out_col = out_col;
    s.fin_kind = fin_kind; s.fin_bias = fin_bias;
    ph.Nall += rows;
  };
  // columns [c0, c1) of a phase's activation matrix from what an earlier phase left: finished bf16 values
  // (`fin`) or `nsl` raw slices to be added, biased and activated as `kind` says
  auto feed = [](StreamPhase& ph, int c0, int c1, bool fin, int kind, const void* src, int nsl, long long ld,
                 int src_col, int gate_off, const float* bias) {
    if (c1 <= c0) return;
    StreamInPart& in = ph.in[ph.nin++];
    in.col_begin = c0; in.col_end = c1; in.kind = fin ? STREAM_IN_BF16 : kind; in.nslices = fin ? 1 : nsl;
    in.src = src; in.ld = ld; in.slice_stride = 8 * ld; in.src_col = src_col; in.gate_off = gate_off;
    in.bias = fin ? nullptr : bias;
  };
  auto set_out = [&](StreamPhase& ph, bool fin, long long o, long long ld) {
    if (fin) ph.outb = BS(o); else ph.out = FS(o);
    ph.out_ld = ld;
  };
  // ---- stage 1: z_H = X U1 (+ b1[h2], sigma when finished here) and Q = X A1 (SwiGLU: gate and up of each)
  {
    StreamPhase& ph = p.ph[p.nph++];
    ph.K = d; ph.S = S1;
    if (!gated) {
      add_seg(ph, W(SEC_U1T), d, k_pad, 0, 0, STREAM_IN_ACT, F(SEC_B1H));
      if (light) add_seg(ph, W(SEC_A1T), d, r_pad, 0, k_pad);
    } else {
      add_seg(ph, W(SEC_U1T), d, k_pad, 0, 0);
      add_seg(ph, W(SEC_U1UT), d, k_pad, 0, k_pad);
      if (light) add_seg(ph, W(SEC_A1T), d, 2 * r_pad, 0, 2 * k_pad);   // [A1 | A1u]^T
    }
    StreamInPart& in = ph.in[ph.nin++];
    in.col_begin = 0; in.col_end = d; in.kind = STREAM_IN_BF16; in.src = X; in.ld = d;
    set_out(ph, fin1, o_p1, N1);
  }
  const int q_col = g2 * k_pad;   // where Q starts among stage 1's output columns
  const void* p1 = scratch + o_p1;
  if (light) {
    // ---- stage 2a: z_L = Q B1 (+ b1[light], sigma when finished here)
    StreamPhase& a = p.ph[p.nph++];
    a.K = r_pad; a.S = S2a;
    add_seg(a, W(SEC_B1T), r_pad, ml_pad, 0, 0, STREAM_IN_ACT, gated ? nullptr : F(SEC_B1L));
    if (gated) add_seg(a, W(SEC_B1UT), r_pad, ml_pad, r_pad, ml_pad);
    feed(a, 0, g2 * r_pad, fin1, STREAM_IN_LINEAR, p1, S1, N1, q_col, 0, nullptr);
    set_out(a, fin2a, o_2a, N2a);
    // ---- stage 2b: P = sigma(z_L + b1[light]) A2
    StreamPhase& b = p.ph[p.nph++];
    b.K = ml_pad; b.S = S2b;
    add_seg(b, W(SEC_A2T), ml_pad, r_pad, 0, 0);
    feed(b, 0, ml_pad, fin2a, gated ? STREAM_IN_GATED : STREAM_IN_ACT, scratch + o_2a, S2a, N2a, 0, ml_pad,
         gated ? nullptr : F(SEC_B1L));
    set_out(b, fin2b, o_2b, r_pad);
  }
  // ---- stage 3: Y = [sigma(z_H + b1[h2]) | P] [V1 ; B2] + b2
  {
    StreamPhase& ph = p.ph[p.nph++];
    ph.K = K3; ph.S = S3;
    add_seg(ph, W(SEC_V1B2T), kp_rp, d, 0, 0);
    feed(ph, 0, k_pad, fin1, gated ? STREAM_IN_GATED : STREAM_IN_ACT, p1, S1, N1, 0, k_pad, gated ? nullptr : F(SEC_B1H));
    if (light) feed(ph, k_pad, kp_rp, fin2b, STREAM_IN_LINEAR, scratch + o_2b, S2b, r_pad, 0, 0, nullptr);
    if (S3 == 1) {
      ph.y = static_cast<__nv_bfloat16*>(Y); ph.y_ld = d; ph.y_bias = F(SEC_B2); ph.y_cols = d;
    } else {
      ph.out = FS(o_y); ph.out_ld = d;
      StreamPhase& rd = p.ph[p.nph++];
      rd.kind = 1;
      feed(rd, 0, d, false, STREAM_IN_LINEAR, scratch + o_y, S3, d, 0, 0, nullptr);
      rd.y = static_cast<__nv_bfloat16*>(Y); rd.y_ld = d; rd.y_bias = F(SEC_B2); rd.y_cols = d;
    }
  }
  const double n_in = h.n_in;
  const double algo_bytes = 2.0 * ((n_in + 1) * (static_cast<double>(d) * h.k + static_cast<double>(h.r) * (d + h.ml))) +
                            4.0 * (h.m + d) + 2.0 * T * d * 2;
  *launched = true;
  return decode_stream_launch(ctx, p, algo_bytes, st);
}

// Up to 64 tokens of a bf16 layer: true = the weight-streaming kernels of this file, false = the forward runs its
// stage GEMMs on the tensor cores with the operands exchanged (GemmArgs::few).
bool decode_path_applies(const ffsplit_ctx* ctx, const BlobHeader& h, long long T) {
  // Measured per layer (graph replays over distinct weight copies), tensor path vs streaming kernels, split / dense:
  //   OPT-13B shape (5 % heavy, r = 512; 71 / 419 MB): the tensor path at every token count -- 33 vs 42 us at 1 token,
  //     34 vs 44 at 4, 35 vs 57 at 16, 46 vs 151 at 64; dense 81 vs 90 at 1 token, 83 vs 91 at 16, 99 vs 187 at 64 --
  //     except the dense layer at 2 to 4 tokens (83 vs 80 us); the same shape at 1 % heavy, r = 256 (15 MB): 27.5 vs
  //     34 us at 1 token, 29.5 vs 50 at 16;
  //   gated (SwiGLU) layers, Llama-2-7B shape: the streaming kernels at one token (48.5 vs 49.4 us split, 53 vs 60.5
  //     dense), the tensor path above (split 50.4 vs 53.5 us at 4 tokens, 50.5 vs 53 at 8, 51 vs 61 at 9; dense 60 vs
  //     66 at 4, 60 vs 64.6 at 8);
  //   split layers under 10 MB and dense ones under 32 MB: the streaming kernels up to 8 tokens (GPT-2-medium shape,
  //     6 / 17 MB, 1 token: 17.6 vs 20.4 us split, 11 vs 15 dense; BERT-base shape 16.9 vs 19.0 us), the tensor path
  //     from 9 on (16 tokens: 21.6 vs 26.5 us, 19.9 vs 25.6 us).
  // FFSPLIT_FEW_TENSOR_MIN = t replaces all of this by "streaming kernels up to t tokens": 64 keeps every count on
  // them, -1 sends every count to the tensor path.
  if (h.dtype != FFSPLIT_BF16 || T < 1 || T > 64) return false;
  if (ctx->few_tensor_min != kFewTensorAuto) return T <= ctx->few_tensor_min;
  const double layer_bytes = 2.0 * (h.n_in + 1) * (static_cast<double>(h.d) * h.k + static_cast<double>(h.r) * (h.d + h.ml));
  const bool no_light = h.r == 0 || h.ml == 0;
  if (no_light ? layer_bytes < 32e6 : layer_bytes < 10e6) return T <= 8;
  if (h.act == FFSPLIT_SWIGLU) return no_light ? T <= 2 : T == 1;
  return no_light && T >= 2 && T <= 4;
}

// fp32 partials of one product.
size_t decode_scratch_bytes(int dtype, long long T) {
  if (dtype != FFSPLIT_BF16 || T > 64 || T < 1) return 0;
  return static_cast<size_t>(kFewScratchBytes);
}

static ffsplit_status decode_forward_impl(ffsplit_ctx* ctx, const BlobHeader& h, const char* blob, const void* X,
                                          long long T64, void* Y, char* AP, char* Q, char* HL, char* scratch,
                                          cudaStream_t st, int* tickets, long long scratch_bytes,
                                          unsigned long long guard_hash) {
  const int T = static_cast<int>(T64);
  // Which of the two few-token kernels (measured per layer, CUDA-graph replays over distinct weight copies).  The
  // single-launch streaming kernel wins on layers without a light part, whose two products are tens of megabytes
  // each: dense Llama-2-7B shape 53 vs 62 us at one token, dense GPT-2-medium shape 11 vs 13.5 us.  On split layers
  // (four or five dependent products) the two are within 1.5 us of each other at one token where the streaming
  // kernel is ahead (OPT-13B shape, 5 % heavy, r = 512: 40.7 vs 41.7 us) and the per-product kernel is up to 10 us
  // ahead elsewhere (1 % heavy or r = 1280: 51.7 vs 61.8 us) and at every point with more than one token (36-56 vs
  // 48-79 us at four tokens); only the gated (SwiGLU) split layer at one token keeps the streaming kernel (48.6 vs
  // 51.2 us).  FFSPLIT_DECODE_STREAM=2 forces the streaming kernel for every T <= 8, 0 turns it off.
  const double layer_bytes = 2.0 * (h.n_in + 1) * (static_cast<double>(h.d) * h.k + static_cast<double>(h.r) * (h.d + h.ml));
  const bool no_light = h.r == 0 || h.ml == 0;
  const bool gated_one = h.act == FFSPLIT_SWIGLU && T == 1;
  const bool stream = ctx->decode_stream == 2 ||
                      (ctx->decode_stream == 1 && T <= 4 && layer_bytes >= 16e6 && (no_light || gated_one));
  if (T <= 8 && stream) {
    // one persistent launch whose weight stream runs ahead of the stage dependencies; its slices take the whole
    // scratch area (the [A_H | P], Q and H_L buffers of the other kernel are not used)
    bool launched = false;
    const ffsplit_status ss = stream_forward(ctx, h, blob, X, T, Y, scratch, scratch_bytes, tickets ? tickets : ctx->status(),
                                             st, guard_hash, &launched);
    if (launched || ss != FFSPLIT_ERR_BUFFER_TOO_SMALL) return ss;
  }
  const int d = h.d, k_pad = h.k_pad, r_pad = h.r_pad, ml_pad = h.ml_pad, kp_rp = h.k_pad + h.r_pad;
  const bool gated = h.act == FFSPLIT_SWIGLU;
  const bool light = r_pad > 0 && h.ml > 0;
  const float* b1h = reinterpret_cast<const float*>(blob + h.off[SEC_B1H]);
  const float* b1l = reinterpret_cast<const float*>(blob + h.off[SEC_B1L]);
  const float* b2 = reinterpret_cast<const float*>(blob + h.off[SEC_B2]);
  float* part = reinterpret_cast<float*>(scratch);
  const double xy = 2.0 * T * d * 2;   // X read once, Y written once: charged to the first and last product
  ffsplit_status s;
  Epilogue e;
  // the products are collected and run by one persistent kernel (one launch each, or one for all)
  DecodeLayerPlan plan;
  auto emit = [&](const void* X0, const void* X1, long long ldx, const void* W0, const void* W1, long long ldw, int,
                  int N, int K, const Epilogue& epi, float*, double algo_bytes) -> ffsplit_status {
    return decode_layer_add(ctx, &plan, X0, X1, ldx, W0, W1, ldw, N, K, epi, algo_bytes);
  };
  bool guard_pending = guard_hash != 0;   // the first product checks the blob header
  auto clear = [&]() {
    std::memset(&e, 0, sizeof(e));
    e.act = h.act;
    if (guard_pending) {
      e.guard = reinterpret_cast<const unsigned long long*>(blob);
      e.guard_hash = guard_hash;
      guard_pending = false;
    }
  };
  // ---- stage 1
  if (!gated) {
    clear();
    e.C0 = AP; e.ld0 = kp_rp; e.C1 = Q; e.ld1 = r_pad;
    e.n_split = k_pad; e.n_act = k_pad; e.n_bias = k_pad; e.bias = b1h;
    if ((s = emit(X, nullptr, d, blob + h.off[SEC_U1T], nullptr, d, T, kp_rp, d, e, part,
                         2.0 * d * (h.k + h.r) + 4.0 * h.k + xy / 2)) != FFSPLIT_OK) return s;
  } else {
    clear();
    e.C0 = AP; e.ld0 = kp_rp; e.n_split = k_pad;
    if ((s = emit(X, X, d, blob + h.off[SEC_U1T], blob + h.off[SEC_U1UT], d, T, k_pad, d, e, part,
                         4.0 * d * h.k + xy / 2)) != FFSPLIT_OK) return s;
    if (light) {
      clear();
      e.C0 = Q; e.ld0 = 2 * r_pad; e.n_split = 2 * r_pad;
      if ((s = emit(X, nullptr, d, blob + h.off[SEC_A1T], nullptr, d, T, 2 * r_pad, d, e, part,
                           4.0 * d * h.r)) != FFSPLIT_OK) return s;
    }
  }
  // ---- stage 2
  if (light) {
    clear();
    e.C0 = HL; e.ld0 = ml_pad; e.n_split = ml_pad;
    if (!gated) { e.n_act = ml_pad; e.n_bias = ml_pad; e.bias = b1l; }
    const long long ldq = static_cast<long long>(h.n_in) * r_pad;
    if ((s = emit(Q, gated ? Q + static_cast<size_t>(r_pad) * 2 : nullptr, ldq, blob + h.off[SEC_B1T],
                         gated ? blob + h.off[SEC_B1UT] : nullptr, r_pad, T, ml_pad, r_pad, e, part,
                         2.0 * h.n_in * h.r * h.ml + (gated ? 0.0 : 4.0 * h.ml))) != FFSPLIT_OK) return s;
    clear();
    e.C0 = AP + static_cast<size_t>(k_pad) * 2; e.ld0 = kp_rp; e.n_split = r_pad;
    if ((s = emit(HL, nullptr, ml_pad, blob + h.off[SEC_A2T], nullptr, ml_pad, T, r_pad, ml_pad, e, part,
                         2.0 * h.r * h.ml)) != FFSPLIT_OK) return s;
  }
  // ---- stage 3
  clear();
  e.C0 = Y; e.ld0 = d; e.n_split = d; e.n_bias = d; e.bias = b2;
  if ((s = emit(AP, nullptr, kp_rp, blob + h.off[SEC_V1B2T], nullptr, kp_rp, T, d, light ? kp_rp : k_pad, e,
                     part, 2.0 * d * (h.k + (light ? h.r : 0)) + 4.0 * d + xy / 2)) != FFSPLIT_OK) return s;
  if (static_cast<long long>(decode_layer_scratch_bytes(ctx->num_sms, T)) > scratch_bytes)
    return fail(ctx, FFSPLIT_ERR_BUFFER_TOO_SMALL, "few-token forward: scratch smaller than two partials per SM");
  // control block: the caller's (status and barrier words, then the tickets), else the workspace's
  int* ctrl = tickets ? tickets : ctx->status();
  return decode_layer_launch(ctx, &plan, T, part, ctrl, st);
}

// Scratch from the caller's workspace, ticket counters from its control block.
ffsplit_status launch_decode_forward(ffsplit_ctx* ctx, const BlobHeader& h, const char* blob, const void* X,
                                     long long T, void* Y, char* AP, char* Q, char* HL, char* scratch,
                                     cudaStream_t st, unsigned long long guard_hash) {
  return decode_forward_impl(ctx, h, blob, X, T, Y, AP, Q, HL, scratch, st, nullptr, kDecodeScratchBytes, guard_hash);
}

}  // namespace ffsp

// =====================================================================================
// Few-token forward that needs no memory from its caller beyond inputs and outputs.
// =====================================================================================
namespace {

constexpr int kNoAllocMaxTokens = 8;
constexpr size_t kNoAllocTicketBytes = ffsp::kCtrlBytes;                 // ticket counters of the K-split reduction
constexpr size_t kNoAllocPartialBytes = 2u << 20;                       // fp32 partials of the K-split reduction
constexpr size_t kNoAllocStageBytes = 2u << 20;                         // A_H | P, Q and the light activations
constexpr size_t kNoAllocBytes = kNoAllocTicketBytes + kNoAllocPartialBytes + kNoAllocStageBytes;   // 4.06 MiB

// Scratch of ffsplit_forward_noalloc.  Lives in every GPU context that loads the library, from
// load to exit.  In host code this name is only a handle for cudaGetSymbolAddress -- it is not a
// device address and must never be handed to a kernel as a pointer.
static __device__ __align__(256) unsigned char g_noalloc_scratch[kNoAllocBytes];

// Device address of the array on each device, resolved on first use.  Contexts are independent and may be
// driven from different host threads: the table is read and written under a lock.
constexpr int kMaxDevices = 64;
std::mutex g_noalloc_mutex;
char* g_noalloc_ptr[kMaxDevices] = {nullptr};

}  // namespace

namespace ffsp {
char* noalloc_control_block(int device) {
  if (device < 0 || device >= kMaxDevices) return nullptr;
  std::lock_guard<std::mutex> lock(g_noalloc_mutex);
  return g_noalloc_ptr[device];
}
}  // namespace ffsp

extern "C" ffsplit_status ffsplit_forward_noalloc(ffsplit_ctx* ctx, const void* blob, const void* X, int64_t T,
                                                  void* Y, void* stream) {
  using namespace ffsp;
  if (!ctx) return FFSPLIT_ERR_INVALID_ARG;
  ctx->err.clear();
  int dev = -1;
  cudaError_t ce = cudaGetDevice(&dev);
  if (ce != cudaSuccess) return check_cuda(ctx, ce, "cudaGetDevice");
  if (dev != ctx->device || dev < 0 || dev >= kMaxDevices)
    return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "the context's device is not the current device");
  if (!blob || !X || !Y) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "NULL tensor");
  if (!aligned16(X) || !aligned16(Y)) return fail(ctx, FFSPLIT_ERR_ALIGN, "X and Y must be 16-byte aligned");
  if (T < 1 || T > kNoAllocMaxTokens)
    return fail(ctx, FFSPLIT_ERR_SHAPE, "ffsplit_forward_noalloc handles 1..8 tokens per call");
  auto it = ctx->blobs.find(blob);
  if (it == ctx->blobs.end())
    return fail(ctx, FFSPLIT_ERR_BAD_BLOB,
                "blob not known to this context: pack it here or register it with ffsplit_blob_open()");
  const BlobHeader& h = it->second.h;
  if (h.dtype != FFSPLIT_BF16) return fail(ctx, FFSPLIT_ERR_DTYPE, "ffsplit_forward_noalloc handles bf16 layers only");
  // intermediates of one call: [A_H | P], Q, light activations, each 256-byte aligned
  auto up = [](size_t v) { return (v + 255) / 256 * 256; };
  const size_t ap_b = up(static_cast<size_t>(T) * (h.k_pad + h.r_pad) * 2);
  const size_t q_b = up(static_cast<size_t>(T) * h.n_in * h.r_pad * 2);
  const size_t hl_b = up(static_cast<size_t>(T) * h.ml_pad * 2);
  if (ap_b + q_b + hl_b > kNoAllocStageBytes)
    return fail(ctx, FFSPLIT_ERR_BUFFER_TOO_SMALL,
                "layer too wide for the built-in scratch of ffsplit_forward_noalloc (2 MiB of intermediates)");
  // one-time set-up per device: the device address of the built-in scratch
  char* base = nullptr;
  {
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!g_noalloc_ptr[dev]) {
      void* ptr = nullptr;
      ce = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);
      if (ce != cudaSuccess || !ptr) return check_cuda(ctx, ce != cudaSuccess ? ce : cudaErrorInvalidSymbol, "cudaGetSymbolAddress(scratch)");
      ce = cudaMemset(ptr, 0, kNoAllocTicketBytes);   // first use on this device: status words, barrier words and tickets start at zero
      if (ce != cudaSuccess) return check_cuda(ctx, ce, "cudaMemset(built-in control block)");
      g_noalloc_ptr[dev] = static_cast<char*>(ptr);
    }
    base = g_noalloc_ptr[dev];
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // The barrier and ticket words must read zero when the kernels start (a call that gave up may have left
  // them mid-way); the status words in front of them stay as they are until ffsplit_poll() has reported them.
  constexpr size_t kStatusWordsBytes = 64;   // words 0..15; the barrier words start at word 16
  ce = cudaMemsetAsync(base + kStatusWordsBytes, 0, kNoAllocTicketBytes - kStatusWordsBytes, st);
  if (ce != cudaSuccess) return check_cuda(ctx, ce, "cudaMemsetAsync(tickets)");
  char* part = base + kNoAllocTicketBytes;
  char* AP = part + kNoAllocPartialBytes;
  char* Q = AP + ap_b;
  char* HL = Q + q_b;
  return decode_forward_impl(ctx, h, static_cast<const char*>(blob), X, T, Y, AP, Q, HL, part, st,
                             reinterpret_cast<int*>(base), static_cast<long long>(kNoAllocPartialBytes),
                             it->second.hash);
}
