// Few-token (decode) split forward for bf16 layers: T <= 64 tokens.
//
// With a handful of tokens every stage of Eq. 2 is a skinny product
//     C[t, n] = epi( sum_k X[t, k] * W[n, k] )        W: [N, K] K-major weights from the packed blob
// whose cost is reading W once from HBM.  The kernel streams W with 128-bit loads that bypass L1
// (each warp-wide load covers 8 rows x 64 contiguous bytes, whole sectors), keeps the few X rows in
// L1, and feeds warp-level tensor-core MMAs (m16n8k16, weights as the 16-row operand, tokens as the
// 8-wide one) straight from registers: because a contraction does not care in which order k is
// visited, each thread's 16-byte load is used as-is for two MMAs and X is loaded with the same
// pattern, so no shuffle or shared-memory staging of operands is needed.  At these sizes the tensor
// pipe is idle most of the time; what matters is bytes in flight per SM.
//
// Work split: a CTA of 8 warps owns 16*RT weight rows and one K range; its warps take disjoint
// sub-ranges of K and add their accumulators through shared memory in warp order.  When there are
// few rows the K range is also split across CTAs (`splits`): each CTA writes an fp32 partial and the
// last one to arrive (atomic ticket) adds the partials in split order, so results are bitwise
// reproducible.  The epilogue (bias, GELU / SiLU gating, the [A_H | Q] column split) runs once per
// output element, after the reduction.
#include <cstring>

#include "decode_common.cuh"
#include "epilogue.cuh"
#include "internal.h"

namespace ffsp {
namespace dec {

struct Params {
  const __nv_bfloat16* X0; const __nv_bfloat16* X1; long long ldx;   // [T, K]; X1 for the gated pair
  const __nv_bfloat16* W0; const __nv_bfloat16* W1; long long ldw;   // [N, K]
  int T, N, K;
  int splits, steps_total;
  int wk;           // warps along K inside a CTA; WR = warps / wk groups of 16 rows
  Epilogue epi;
  float* partial;   // [splits][row groups][WR][16 TILES][8 NT] fp32
  int* tickets;     // [row groups], zero before and after the launch
};

// NT token tiles of 8.  DUAL: two tiles of the same 16 rows, (X0, W0) and (X1, W1); output
// row n = silu(acc0[n]) * acc1[n].  WARPS warps per CTA (8 plain, 4 gated: shared memory).
template <int NT, bool DUAL>
__global__ void __launch_bounds__(DUAL ? 128 : 256, 1) decode_gemm_kernel(const Params p) {
  constexpr int WARPS = DUAL ? 4 : 8;
  constexpr int THREADS = WARPS * 32;
  constexpr int TILES = DUAL ? 2 : 1;
  constexpr int TP = 8 * NT;
  constexpr int WARP_BYTES = STAGES * TILES * TILE_BYTES;
  constexpr int ELEMS = 16 * TILES * TP;     // accumulator values of one warp
  extern __shared__ __align__(16) unsigned char smem[];
  __shared__ int s_last;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, c = lane & 3;
  const int WK = p.wk, WR = WARPS / WK;
  const int wr = warp / WK, wk = warp - wr * WK;
  const int rg = blockIdx.x, split = blockIdx.y;
  const int row0 = (rg * WR + wr) * 16;

  // This CTA's range of k steps; its WK warps take the steps round robin, so that at any time the
  // warps of a row group read neighbouring 512-byte pieces of the same rows (long runs in DRAM).
  const int cta_lo = static_cast<int>(static_cast<long long>(p.steps_total) * split / p.splits);
  const int cta_hi = static_cast<int>(static_cast<long long>(p.steps_total) * (split + 1) / p.splits);
  const int my_steps = (cta_hi - cta_lo - wk + WK - 1) / WK;   // steps cta_lo + wk + i * WK

  float acc[TILES][NT][4];
#pragma unroll
  for (int i = 0; i < TILES; ++i)
#pragma unroll
    for (int j = 0; j < NT; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[i][j][e] = 0.f;

  const uint32_t my_smem = static_cast<uint32_t>(__cvta_generic_to_shared(smem)) + warp * WARP_BYTES;
  // one stage: 16 rows (x TILES) of 512 contiguous bytes each, one row per warp-wide copy
  auto issue = [&](int i) {
    const int step = cta_lo + wk + i * WK;
    const uint32_t dst0 = my_smem + (i & 1) * (TILES * TILE_BYTES) + lane * 16;
    const int k = step * KSTEP + lane * 8;
    const bool kin = k < p.K;   // K is a multiple of 8
#pragma unroll
    for (int i = 0; i < TILES; ++i) {
      const __nv_bfloat16* W = i ? p.W1 : p.W0;
#pragma unroll
      for (int r = 0; r < 16; ++r) {
        const int n = row0 + r;
        const bool ok = kin && n < p.N;
        cp_async16(dst0 + i * TILE_BYTES + r * ROW_PITCH, W + static_cast<long long>(ok ? n : 0) * p.ldw + (ok ? k : 0), ok);
      }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  auto compute = [&](int i) {
    const int step = cta_lo + wk + i * WK;
    const uint32_t src0 = my_smem + (i & 1) * (TILES * TILE_BYTES) + g * ROW_PITCH + c * 16;
#pragma unroll(NT >= 4 ? 2 : 8)
    for (int it = 0; it < 8; ++it) {
      const int k = step * KSTEP + (it * 4 + c) * 8;
      const bool kin = k < p.K;
      uint4 xb[TILES][NT];
#pragma unroll
      for (int i = 0; i < TILES; ++i) {
        const __nv_bfloat16* X = i ? p.X1 : p.X0;
#pragma unroll
        for (int j = 0; j < NT; ++j) {
          const int t = 8 * j + g;
          xb[i][j] = (kin && t < p.T) ? __ldg(reinterpret_cast<const uint4*>(X + static_cast<long long>(t) * p.ldx + k))
                                      : make_uint4(0u, 0u, 0u, 0u);
        }
      }
#pragma unroll
      for (int i = 0; i < TILES; ++i) {
        // rows g and g + 8 of the tile, the same 16 bytes of k: used as they are for two MMAs (the
        // order in which a contraction visits k is free as long as both operands agree on it)
        const uint4 lo = lds128(src0 + i * TILE_BYTES + it * 64);
        const uint4 hi = lds128(src0 + i * TILE_BYTES + 8 * ROW_PITCH + it * 64);
#pragma unroll
        for (int j = 0; j < NT; ++j) {
          mma_bf16(acc[i][j], lo.x, hi.x, lo.y, hi.y, xb[i][j].x, xb[i][j].y);
          mma_bf16(acc[i][j], lo.z, hi.z, lo.w, hi.w, xb[i][j].z, xb[i][j].w);
        }
      }
    }
  };

  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the next product may start its own prologue
  if (my_steps > 0) issue(0);
  if (my_steps > 1) issue(1);
  // everything below reads or writes what the previous kernel of the stream produced or still reads
  asm volatile("griddepcontrol.wait;" ::: "memory");
  for (int i = 0; i < my_steps; ++i) {
    if (i + 1 < my_steps) asm volatile("cp.async.wait_group 1;" ::: "memory");
    else asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncwarp();
    compute(i);
    __syncwarp();
    if (i + 2 < my_steps) issue(i + 2);
  }

  // ---- the WK accumulators of each row group are added in warp order (staging buffers are free now)
  __syncthreads();
  float* red = reinterpret_cast<float*>(smem);   // [WARPS][16 TILES][TP]
  float* mine = red + warp * ELEMS;
#pragma unroll
  for (int i = 0; i < TILES; ++i)
#pragma unroll
    for (int j = 0; j < NT; ++j) {
      const int t = 8 * j + 2 * c;
      mine[(16 * i + g) * TP + t] = acc[i][j][0];
      mine[(16 * i + g) * TP + t + 1] = acc[i][j][1];
      mine[(16 * i + g + 8) * TP + t] = acc[i][j][2];
      mine[(16 * i + g + 8) * TP + t + 1] = acc[i][j][3];
    }
  __syncthreads();
  const int cta_elems = WR * ELEMS;
  float* mypart = p.partial + (static_cast<long long>(split) * gridDim.x + rg) * (WARPS * ELEMS);
  for (int idx = threadIdx.x; idx < cta_elems; idx += THREADS) {
    const int r = idx / ELEMS, rem = idx - r * ELEMS;
    float v = 0.f;
    for (int w = 0; w < WK; ++w) v += red[(r * WK + w) * ELEMS + rem];
    if (p.splits > 1) mypart[idx] = v;
    else red[(r * WK) * ELEMS + rem] = v;   // read and written by this thread only
  }
  // ---- across CTAs: partials + ticket, the last CTA of the row group adds them in split order
  if (p.splits > 1) {
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
      const int t = atomicAdd(p.tickets + rg, 1);
      s_last = (t == p.splits - 1) ? 1 : 0;
      __threadfence();
    }
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    for (int idx = threadIdx.x; idx < cta_elems; idx += THREADS) {
      const int r = idx / ELEMS, rem = idx - r * ELEMS;
      float v = 0.f;
      for (int sp = 0; sp < p.splits; ++sp)
        v += __ldcg(p.partial + (static_cast<long long>(sp) * gridDim.x + rg) * (WARPS * ELEMS) + idx);
      red[(r * WK) * ELEMS + rem] = v;
    }
    if (threadIdx.x == 0) p.tickets[rg] = 0;
  }
  __syncthreads();
  // ---- epilogue, n fastest across threads
  const Epilogue& ep = p.epi;
  const GeluCoef gc = gelu_coef(ep.act);
  const int out_cta = WR * 16;
  for (int idx = threadIdx.x; idx < out_cta * TP; idx += THREADS) {
    const int t = idx / out_cta, nc = idx - t * out_cta;
    const int r = nc >> 4, nl = nc & 15;
    const int n = rg * out_cta + nc;
    if (t >= p.T || n >= p.N) continue;
    const float* src = red + (r * WK) * ELEMS;
    float v;
    if (DUAL) {
      v = silu_fast(src[nl * TP + t]) * src[(nl + 16) * TP + t];
    } else {
      v = src[nl * TP + t];
      if (n < ep.n_bias) v += __ldg(ep.bias + n);
      if (n < ep.n_act) v = gelu_fast(v, gc);
    }
    if (n < ep.n_split) reinterpret_cast<__nv_bfloat16*>(ep.C0)[static_cast<long long>(t) * ep.ld0 + n] = __float2bfloat16_rn(v);
    else reinterpret_cast<__nv_bfloat16*>(ep.C1)[static_cast<long long>(t) * ep.ld1 + (n - ep.n_split)] = __float2bfloat16_rn(v);
  }
}

template <int NT, bool DUAL>
cudaError_t launch_one(const Params& p, int row_groups, cudaStream_t st) {
  constexpr int WARPS = DUAL ? 4 : 8;
  constexpr int TILES = DUAL ? 2 : 1;
  const int smem = WARPS * STAGES * TILES * TILE_BYTES;   // also holds [WARPS][16 TILES][8 NT] floats afterwards
  static bool attr_done = false;
  if (!attr_done) {
    cudaError_t e = cudaFuncSetAttribute(decode_gemm_kernel<NT, DUAL>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem);
    if (e != cudaSuccess) return e;
    attr_done = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(row_groups, p.splits);
  cfg.blockDim = dim3(WARPS * 32);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, decode_gemm_kernel<NT, DUAL>, p);
}

}  // namespace dec

constexpr long long kDecodeScratchBytes = 16ll << 20;   // fp32 partials of one product

// One skinny product.  dual: (X0, W0) and (X1, W1) on the same rows, gated.
static ffsplit_status decode_gemm(ffsplit_ctx* ctx, const void* X0, const void* X1, long long ldx, const void* W0,
                                  const void* W1, long long ldw, int T, int N, int K, const Epilogue& epi,
                                  float* partial, double algo_bytes, cudaStream_t st, int* tickets = nullptr,
                                  long long scratch_bytes = kDecodeScratchBytes) {
  if (N <= 0 || K <= 0) return FFSPLIT_OK;
  const bool dual = W1 != nullptr;
  dec::Params p;
  p.X0 = static_cast<const __nv_bfloat16*>(X0); p.X1 = static_cast<const __nv_bfloat16*>(X1); p.ldx = ldx;
  p.W0 = static_cast<const __nv_bfloat16*>(W0); p.W1 = static_cast<const __nv_bfloat16*>(W1); p.ldw = ldw;
  p.T = T; p.N = N; p.K = K;
  p.steps_total = (K + dec::KSTEP - 1) / dec::KSTEP;
  p.epi = epi;
  p.partial = partial;
  p.tickets = tickets ? tickets : ctx->tickets();
  const int nt = T <= 8 ? 1 : T <= 16 ? 2 : T <= 32 ? 4 : 8;
  const int warps = dual ? 4 : 8, tiles = dual ? 2 : 1;
  // Plan: wk warps of a CTA share 16 rows and split the CTA's K range; `splits` CTAs share a row group.
  // Wanted: at least one CTA per SM, every warp with a few steps (of 256 k) to pipeline, and fp32
  // partials (written and read once) small beside the weights.
  int best_wk = 1, best_splits = 1;
  double best = -1.0;
  for (int wk = warps; wk >= 1; wk >>= 1) {
    const int wr = warps / wk;
    const long long rgs = (N + 16ll * wr - 1) / (16ll * wr);
    if (rgs > kMaxTicketTiles) continue;
    for (int sp = 1; sp <= 16; ++sp) {
      const double steps_per_warp = static_cast<double>(p.steps_total) / (wk * sp);
      if ((sp > 1 || wk > 1) && steps_per_warp < 1.0) break;
      const double part_bytes = sp > 1 ? 2.0 * sp * rgs * warps * 16.0 * tiles * 8 * nt * 4 : 0.0;
      if (sp > 1 && (sp * rgs * warps * 16ll * tiles * 8 * nt * 4 > scratch_bytes || part_bytes > 0.12 * 2.0 * N * K)) break;
      const double fill = static_cast<double>(rgs) * sp / ctx->num_sms;
      const double score = (fill < 1.0 ? fill : 1.0) * (steps_per_warp < 3.0 ? steps_per_warp / 3.0 : 1.0) - 0.002 * sp -
                           0.001 * wk;
      if (score > best) { best = score; best_wk = wk; best_splits = sp; }
    }
  }
  p.wk = best_wk;
  p.splits = best_splits;
  const int wr = warps / p.wk;
  const int row_groups = static_cast<int>((N + 16ll * wr - 1) / (16ll * wr));
  const int ph = prof_open(ctx, PROF_DECODE, algo_bytes, st);
  cudaError_t e;
#define FFS_DEC(NT_) (dual ? dec::launch_one<NT_, true>(p, row_groups, st) : dec::launch_one<NT_, false>(p, row_groups, st))
  if (nt == 1) e = FFS_DEC(1);
  else if (nt == 2) e = FFS_DEC(2);
  else if (nt == 4) e = FFS_DEC(4);
  else e = FFS_DEC(8);
#undef FFS_DEC
  prof_close(ctx, ph, st);
  ctx->launches++;
  return check_cuda(ctx, e, "decode_gemm_kernel launch");
}

bool decode_path_applies(const ffsplit_ctx* ctx, const BlobHeader& h, long long T) {
  (void)ctx;
  return h.dtype == FFSPLIT_BF16 && T >= 1 && T <= 64;
}

// fp32 partials of one product.
size_t decode_scratch_bytes(int dtype, long long T) {
  if (dtype != FFSPLIT_BF16 || T > 64 || T < 1) return 0;
  return static_cast<size_t>(kDecodeScratchBytes);
}

static ffsplit_status decode_forward_impl(ffsplit_ctx* ctx, const BlobHeader& h, const char* blob, const void* X,
                                          long long T64, void* Y, char* AP, char* Q, char* HL, char* scratch,
                                          cudaStream_t st, int* tickets, long long scratch_bytes) {
  const int T = static_cast<int>(T64);
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
  // T <= 32: the products are collected and run by one persistent kernel; above that, one launch each
  const bool one_kernel = decode_layer_applies(T);
  DecodeLayerPlan plan;
  auto emit = [&](const void* X0, const void* X1, long long ldx, const void* W0, const void* W1, long long ldw, int T_,
                  int N, int K, const Epilogue& epi, float* partial, double algo_bytes) -> ffsplit_status {
    if (one_kernel) return decode_layer_add(ctx, &plan, X0, X1, ldx, W0, W1, ldw, N, K, epi, algo_bytes);
    return decode_gemm(ctx, X0, X1, ldx, W0, W1, ldw, T_, N, K, epi, partial, algo_bytes, st, tickets, scratch_bytes);
  };
  auto clear = [&]() { std::memset(&e, 0, sizeof(e)); e.act = h.act; };
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
  if (!one_kernel) return FFSPLIT_OK;
  if (static_cast<long long>(decode_layer_scratch_bytes(ctx->num_sms, T)) > scratch_bytes)
    return fail(ctx, FFSPLIT_ERR_BUFFER_TOO_SMALL, "few-token forward: scratch smaller than two partials per SM");
  // control block: the caller's (status and barrier words, then the tickets), else the workspace's
  int* ctrl = tickets ? tickets : ctx->status();
  return decode_layer_launch(ctx, &plan, T, part, ctrl, st);
}

// Scratch from the caller's workspace, ticket counters from its control block.
ffsplit_status launch_decode_forward(ffsplit_ctx* ctx, const BlobHeader& h, const char* blob, const void* X,
                                     long long T, void* Y, char* AP, char* Q, char* HL, char* scratch,
                                     cudaStream_t st) {
  return decode_forward_impl(ctx, h, blob, X, T, Y, AP, Q, HL, scratch, st, nullptr, kDecodeScratchBytes);
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

constexpr int kMaxDevices = 64;
char* g_noalloc_ptr[kMaxDevices] = {nullptr};

}  // namespace

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
  if (it == ctx->blobs.end()) {
    const ffsplit_status s = ffsplit_blob_open(ctx, blob, 0);
    if (s != FFSPLIT_OK) return s;
    it = ctx->blobs.find(blob);
  }
  const BlobHeader& h = it->second;
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
  if (!g_noalloc_ptr[dev]) {
    void* ptr = nullptr;
    ce = cudaGetSymbolAddress(&ptr, g_noalloc_scratch);
    if (ce != cudaSuccess || !ptr) return check_cuda(ctx, ce != cudaSuccess ? ce : cudaErrorInvalidSymbol, "cudaGetSymbolAddress(scratch)");
    g_noalloc_ptr[dev] = static_cast<char*>(ptr);
  }
  char* base = g_noalloc_ptr[dev];
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  // the ticket counters must read zero when the kernels start; the rest is overwritten before it is read
  ce = cudaMemsetAsync(base, 0, kNoAllocTicketBytes, st);
  if (ce != cudaSuccess) return check_cuda(ctx, ce, "cudaMemsetAsync(tickets)");
  char* part = base + kNoAllocTicketBytes;
  char* AP = part + kNoAllocPartialBytes;
  char* Q = AP + ap_b;
  char* HL = Q + q_b;
  return decode_forward_impl(ctx, h, static_cast<const char*>(blob), X, T, Y, AP, Q, HL, part, st,
                             reinterpret_cast<int*>(base), static_cast<long long>(kNoAllocPartialBytes));
}
