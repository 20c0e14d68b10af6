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

#include "epilogue.cuh"
#include "internal.h"

namespace ffsp {
namespace dec {

constexpr int WARPS = 8;
constexpr int THREADS = WARPS * 32;
constexpr int KSTEP = 32;   // k elements per warp step: one 16-byte load per thread and row

struct Params {
  const __nv_bfloat16* X0; const __nv_bfloat16* X1; long long ldx;   // [T, K]; X1 for the gated pair
  const __nv_bfloat16* W0; const __nv_bfloat16* W1; long long ldw;   // [N, K]
  int T, N, K;
  int splits, steps_total;
  Epilogue epi;
  float* partial;   // [splits][row groups][16 RT][8 NT] fp32
  int* tickets;     // [row groups], zero before and after the launch
};

__device__ __forceinline__ uint4 ldg_stream(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ void mma_bf16(float* c, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                         uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
               "{%0, %1, %2, %3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// RT row tiles of 16 weight rows per CTA, NT token tiles of 8.  DUAL: the first RT/2 tiles come from
// (X0, W0), the others from (X1, W1) on the same rows; output row n = silu(acc0[n]) * acc1[n].
template <int RT, int NT, bool DUAL>
__global__ void __launch_bounds__(THREADS, 1) decode_gemm_kernel(const Params p) {
  extern __shared__ float red[];   // [WARPS][16 RT][8 NT]
  __shared__ int s_last;
  constexpr int ROWS = 16 * RT;          // weight-row slots per CTA
  constexpr int TP = 8 * NT;
  constexpr int OUT_ROWS = DUAL ? ROWS / 2 : ROWS;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, c = lane & 3;
  const int rg = blockIdx.x, split = blockIdx.y;
  const int row0 = rg * OUT_ROWS;

  // this warp's range of k steps
  const int cta_lo = static_cast<int>(static_cast<long long>(p.steps_total) * split / p.splits);
  const int cta_hi = static_cast<int>(static_cast<long long>(p.steps_total) * (split + 1) / p.splits);
  const int n_cta = cta_hi - cta_lo;
  const int s_lo = cta_lo + static_cast<int>(static_cast<long long>(n_cta) * warp / WARPS);
  const int s_hi = cta_lo + static_cast<int>(static_cast<long long>(n_cta) * (warp + 1) / WARPS);

  float acc[RT][NT][4];
#pragma unroll
  for (int i = 0; i < RT; ++i)
#pragma unroll
    for (int j = 0; j < NT; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[i][j][e] = 0.f;

  // row pointers of this thread: tile i, rows g and g + 8
  const __nv_bfloat16* wrow[RT][2];
  bool wok[RT][2];
#pragma unroll
  for (int i = 0; i < RT; ++i) {
    const bool second = DUAL && i >= RT / 2;
    const int tile = second ? i - RT / 2 : i;
    const __nv_bfloat16* W = second ? p.W1 : p.W0;
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int n = row0 + tile * 16 + g + 8 * h;
      wok[i][h] = n < p.N;
      wrow[i][h] = W + static_cast<long long>(wok[i][h] ? n : 0) * p.ldw + c * 8;
    }
  }
  const uint4 zero4 = make_uint4(0u, 0u, 0u, 0u);
  auto load_w = [&](uint4 (&w)[RT][2], int step) {
    const int k = step * KSTEP;
    const bool kin = k + c * 8 < p.K;   // K is a multiple of 8
#pragma unroll
    for (int i = 0; i < RT; ++i)
#pragma unroll
      for (int h = 0; h < 2; ++h) w[i][h] = (kin && wok[i][h]) ? ldg_stream(wrow[i][h] + k) : zero4;
  };
  auto compute = [&](const uint4 (&w)[RT][2], int step) {
    const int k = step * KSTEP + c * 8;
    const bool kin = k < p.K;
    uint4 xb[DUAL ? 2 : 1][NT];
#pragma unroll
    for (int s = 0; s < (DUAL ? 2 : 1); ++s) {
      const __nv_bfloat16* X = s ? p.X1 : p.X0;
#pragma unroll
      for (int j = 0; j < NT; ++j) {
        const int t = 8 * j + g;
        xb[s][j] = (kin && t < p.T) ? __ldg(reinterpret_cast<const uint4*>(X + static_cast<long long>(t) * p.ldx + k))
                                    : zero4;
      }
    }
#pragma unroll
    for (int i = 0; i < RT; ++i) {
      const int s = (DUAL && i >= RT / 2) ? 1 : 0;
#pragma unroll
      for (int j = 0; j < NT; ++j) {
        mma_bf16(acc[i][j], w[i][0].x, w[i][1].x, w[i][0].y, w[i][1].y, xb[s][j].x, xb[s][j].y);
        mma_bf16(acc[i][j], w[i][0].z, w[i][1].z, w[i][0].w, w[i][1].w, xb[s][j].z, xb[s][j].w);
      }
    }
  };

  // two steps of weights in flight per warp
  uint4 wa[RT][2], wb[RT][2];
  int s = s_lo;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // the next product may start its own prologue
  if (s < s_hi) load_w(wa, s);
  // everything below reads or writes what the previous kernel of the stream produced or still reads
  asm volatile("griddepcontrol.wait;" ::: "memory");
  while (s < s_hi) {
    if (s + 1 < s_hi) load_w(wb, s + 1);
    compute(wa, s);
    ++s;
    if (s >= s_hi) break;
    if (s + 1 < s_hi) load_w(wa, s + 1);
    compute(wb, s);
    ++s;
  }

  // ---- add the warps' accumulators in warp order
  float* mine = red + warp * ROWS * TP;
#pragma unroll
  for (int i = 0; i < RT; ++i)
#pragma unroll
    for (int j = 0; j < NT; ++j) {
      const int t = 8 * j + 2 * c;
      mine[(16 * i + g) * TP + t] = acc[i][j][0];
      mine[(16 * i + g) * TP + t + 1] = acc[i][j][1];
      mine[(16 * i + g + 8) * TP + t] = acc[i][j][2];
      mine[(16 * i + g + 8) * TP + t + 1] = acc[i][j][3];
    }
  __syncthreads();
  constexpr int ELEMS = ROWS * TP;
  constexpr int PER = (ELEMS + THREADS - 1) / THREADS;
  float tot[PER];
#pragma unroll
  for (int e = 0; e < PER; ++e) {
    const int idx = threadIdx.x + e * THREADS;
    float v = 0.f;
    if (idx < ELEMS) {
#pragma unroll
      for (int w = 0; w < WARPS; ++w) v += red[w * ROWS * TP + idx];
    }
    tot[e] = v;
  }
  __syncthreads();
  // ---- across CTAs: partials + ticket, the last CTA of the row group adds them in split order
  if (p.splits > 1) {
    float* mypart = p.partial + (static_cast<long long>(split) * gridDim.x + rg) * ELEMS;
#pragma unroll
    for (int e = 0; e < PER; ++e) {
      const int idx = threadIdx.x + e * THREADS;
      if (idx < ELEMS) mypart[idx] = tot[e];
    }
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
#pragma unroll
    for (int e = 0; e < PER; ++e) {
      const int idx = threadIdx.x + e * THREADS;
      float v = 0.f;
      if (idx < ELEMS) {
        for (int sp = 0; sp < p.splits; ++sp)
          v += (sp == split) ? tot[e] : __ldcg(p.partial + (static_cast<long long>(sp) * gridDim.x + rg) * ELEMS + idx);
      }
      tot[e] = v;
    }
    if (threadIdx.x == 0) p.tickets[rg] = 0;
  }
  // ---- totals back to shared memory as [row][t], then the epilogue with n fastest across threads
#pragma unroll
  for (int e = 0; e < PER; ++e) {
    const int idx = threadIdx.x + e * THREADS;
    if (idx < ELEMS) red[idx] = tot[e];
  }
  __syncthreads();
  const Epilogue& ep = p.epi;
  const GeluCoef gc = gelu_coef(ep.act);
  for (int idx = threadIdx.x; idx < OUT_ROWS * TP; idx += THREADS) {
    const int t = idx / OUT_ROWS, nl = idx - t * OUT_ROWS;
    const int n = row0 + nl;
    if (t >= p.T || n >= p.N) continue;
    float v;
    if (DUAL) {
      v = silu_fast(red[nl * TP + t]) * red[(nl + OUT_ROWS) * TP + t];
    } else {
      v = red[nl * TP + t];
      if (n < ep.n_bias) v += __ldg(ep.bias + n);
      if (n < ep.n_act) v = gelu_fast(v, gc);
    }
    if (n < ep.n_split) reinterpret_cast<__nv_bfloat16*>(ep.C0)[static_cast<long long>(t) * ep.ld0 + n] = __float2bfloat16_rn(v);
    else reinterpret_cast<__nv_bfloat16*>(ep.C1)[static_cast<long long>(t) * ep.ld1 + (n - ep.n_split)] = __float2bfloat16_rn(v);
  }
}

template <int RT, int NT, bool DUAL>
cudaError_t launch_one(const Params& p, int row_groups, cudaStream_t st) {
  const int smem = WARPS * 16 * RT * 8 * NT * 4;
  static bool attr_done = false;
  if (!attr_done) {
    cudaError_t e = cudaFuncSetAttribute(decode_gemm_kernel<RT, NT, DUAL>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         smem);
    if (e != cudaSuccess) return e;
    attr_done = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(row_groups, p.splits);
  cfg.blockDim = dim3(THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, decode_gemm_kernel<RT, NT, DUAL>, p);
}

}  // namespace dec

constexpr long long kDecodeMaxPartialRows = 65536;

// One skinny product.  dual: (X0, W0) and (X1, W1) on the same rows, gated.
static ffsplit_status decode_gemm(ffsplit_ctx* ctx, const void* X0, const void* X1, long long ldx, const void* W0,
                                  const void* W1, long long ldw, int T, int N, int K, const Epilogue& epi,
                                  float* partial, double algo_bytes, cudaStream_t st, int* tickets = nullptr) {
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
  const int rt = nt == 8 ? 2 : 4;
  const int out_rows = dual ? 8 * rt : 16 * rt;
  const int row_groups = (N + out_rows - 1) / out_rows;
  if (row_groups > kMaxTicketTiles) return fail(ctx, FFSPLIT_ERR_SHAPE, "decode: too many row groups");
  // Several waves of small CTAs (less loss in the last, partly filled wave), each warp keeping at
  // least two k steps, the fp32 partials (written and read once) at most ~12 % of the weight bytes.
  int splits = (ctx->decode_ctas_per_sm_target * ctx->num_sms + row_groups - 1) / row_groups;
  const int max_by_k = p.steps_total / (2 * dec::WARPS);
  if (splits > max_by_k) splits = max_by_k;
  const int max_by_traffic = static_cast<int>(0.03 * K / (8 * nt));
  if (splits > max_by_traffic) splits = max_by_traffic;
  if (splits > 16) splits = 16;
  const long long rows_slots = static_cast<long long>(row_groups) * 16 * rt;
  if (splits > 1 && splits * rows_slots > kDecodeMaxPartialRows) splits = static_cast<int>(kDecodeMaxPartialRows / rows_slots);
  if (splits < 1) splits = 1;
  p.splits = splits;
  const int ph = prof_open(ctx, PROF_DECODE, algo_bytes, st);
  cudaError_t e;
#define FFS_DEC(RT_, NT_) (dual ? dec::launch_one<RT_, NT_, true>(p, row_groups, st) : dec::launch_one<RT_, NT_, false>(p, row_groups, st))
  if (nt == 1) e = FFS_DEC(4, 1);
  else if (nt == 2) e = FFS_DEC(4, 2);
  else if (nt == 4) e = FFS_DEC(4, 4);
  else e = FFS_DEC(2, 8);
#undef FFS_DEC
  prof_close(ctx, ph, st);
  ctx->launches++;
  return check_cuda(ctx, e, "decode_gemm_kernel launch");
}

bool decode_path_applies(const ffsplit_ctx* ctx, const BlobHeader& h, long long T) {
  (void)ctx;
  return h.dtype == FFSPLIT_BF16 && T >= 1 && T <= 64;
}

// fp32 partials of one product: at most kDecodeMaxPartialRows row slots of 64 tokens.
size_t decode_scratch_bytes(int dtype, long long T) {
  if (dtype != FFSPLIT_BF16 || T > 64 || T < 1) return 0;
  return static_cast<size_t>(kDecodeMaxPartialRows) * 64 * 4;
}

static ffsplit_status decode_forward_impl(ffsplit_ctx* ctx, const BlobHeader& h, const char* blob, const void* X,
                                          long long T64, void* Y, char* AP, char* Q, char* HL, char* scratch,
                                          cudaStream_t st, int* tickets) {
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
  auto clear = [&]() { std::memset(&e, 0, sizeof(e)); e.act = h.act; };
  // ---- stage 1
  if (!gated) {
    clear();
    e.C0 = AP; e.ld0 = kp_rp; e.C1 = Q; e.ld1 = r_pad;
    e.n_split = k_pad; e.n_act = k_pad; e.n_bias = k_pad; e.bias = b1h;
    if ((s = decode_gemm(ctx, X, nullptr, d, blob + h.off[SEC_U1T], nullptr, d, T, kp_rp, d, e, part,
                         2.0 * d * (h.k + h.r) + 4.0 * h.k + xy / 2, st, tickets)) != FFSPLIT_OK) return s;
  } else {
    clear();
    e.C0 = AP; e.ld0 = kp_rp; e.n_split = k_pad;
    if ((s = decode_gemm(ctx, X, X, d, blob + h.off[SEC_U1T], blob + h.off[SEC_U1UT], d, T, k_pad, d, e, part,
                         4.0 * d * h.k + xy / 2, st, tickets)) != FFSPLIT_OK) return s;
    if (light) {
      clear();
      e.C0 = Q; e.ld0 = 2 * r_pad; e.n_split = 2 * r_pad;
      if ((s = decode_gemm(ctx, X, nullptr, d, blob + h.off[SEC_A1T], nullptr, d, T, 2 * r_pad, d, e, part,
                           4.0 * d * h.r, st, tickets)) != FFSPLIT_OK) return s;
    }
  }
  // ---- stage 2
  if (light) {
    clear();
    e.C0 = HL; e.ld0 = ml_pad; e.n_split = ml_pad;
    if (!gated) { e.n_act = ml_pad; e.n_bias = ml_pad; e.bias = b1l; }
    const long long ldq = static_cast<long long>(h.n_in) * r_pad;
    if ((s = decode_gemm(ctx, Q, gated ? Q + static_cast<size_t>(r_pad) * 2 : nullptr, ldq, blob + h.off[SEC_B1T],
                         gated ? blob + h.off[SEC_B1UT] : nullptr, r_pad, T, ml_pad, r_pad, e, part,
                         2.0 * h.n_in * h.r * h.ml + (gated ? 0.0 : 4.0 * h.ml), st, tickets)) != FFSPLIT_OK) return s;
    clear();
    e.C0 = AP + static_cast<size_t>(k_pad) * 2; e.ld0 = kp_rp; e.n_split = r_pad;
    if ((s = decode_gemm(ctx, HL, nullptr, ml_pad, blob + h.off[SEC_A2T], nullptr, ml_pad, T, r_pad, ml_pad, e, part,
                         2.0 * h.r * h.ml, st, tickets)) != FFSPLIT_OK) return s;
  }
  // ---- stage 3
  clear();
  e.C0 = Y; e.ld0 = d; e.n_split = d; e.n_bias = d; e.bias = b2;
  return decode_gemm(ctx, AP, nullptr, kp_rp, blob + h.off[SEC_V1B2T], nullptr, kp_rp, T, d, light ? kp_rp : k_pad, e,
                     part, 2.0 * d * (h.k + (light ? h.r : 0)) + 4.0 * d + xy / 2, st, tickets);
}

// Scratch from the caller's workspace, ticket counters from its control block.
ffsplit_status launch_decode_forward(ffsplit_ctx* ctx, const BlobHeader& h, const char* blob, const void* X,
                                     long long T, void* Y, char* AP, char* Q, char* HL, char* scratch,
                                     cudaStream_t st) {
  return decode_forward_impl(ctx, h, blob, X, T, Y, AP, Q, HL, scratch, st, nullptr);
}

}  // namespace ffsp

// =====================================================================================
// Few-token forward that needs no memory from its caller beyond inputs and outputs.
// =====================================================================================
namespace {

constexpr int kNoAllocMaxTokens = 8;
constexpr size_t kNoAllocTicketBytes = ffsp::kCtrlBytes;                 // ticket counters of the K-split reduction
constexpr size_t kNoAllocPartialBytes = static_cast<size_t>(ffsp::kDecodeMaxPartialRows) * 8 * 4;   // fp32 partials, 8 tokens
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
                             reinterpret_cast<int*>(base));
}
