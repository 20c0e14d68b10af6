// Few-token (decode) split forward, T <= 32 tokens: every product of Eq. 2 in one persistent kernel.
//
// With a handful of tokens each stage of Eq. 2 is a skinny product
//     C[t, n] = epi( sum_k X[t, k] * W[n, k] )        W: [N, K] K-major weights from the packed blob
// whose cost is reading W once from HBM, and a split layer is four or five such products of a few
// megabytes each: what is left to lose is time in which an SM has no loads in flight.  So:
//
//  * One CTA per SM stays resident for the whole layer.  A product is cut into units of
//    128 weight rows x 256 k (64 KB of W); the units, in row-tile-major order, are dealt to the CTAs in
//    equal contiguous shares (a tile's K range may straddle two or more CTAs), and a CTA walks its share
//    with a two-stage cp.async pipeline that does not drain at tile boundaries.
//  * A tile finished inside one CTA goes through the epilogue straight from the accumulator registers.
//    A tile shared by several CTAs: each writes an fp32 partial (at most two per CTA and product: the
//    tile its share starts in and the tile it ends in), takes an atomic ticket, and the last to arrive
//    adds the partials in CTA order -- the result does not depend on who arrives when.
//  * Each warp-wide copy moves 512 contiguous bytes of one weight row; the token rows of the same k
//    range are staged beside the weights, once per CTA.  Fragments for the warp-level MMA (m16n8k16,
//    weights as the 16-row operand, tokens as the 8-wide one) are read from shared memory with
//    128-bit loads; since a contraction does not care in which order k is visited, a thread's 16
//    bytes feed two MMAs as they are, and the token operand is read with the same pattern.
//  * Products are separated by a grid-wide barrier (cooperative launch: all CTAs are resident), before
//    which each CTA has already issued the first weight copies of the next product.
//  * The code is kept small (one call site per building block, short unrolls): the weights stream
//    through L2 and push the kernel's instructions out of it between launches, so every launch
//    fetches its code from DRAM again and straight-line code is paid for in fetch latency.
//
// Launched one product at a time (no barrier; programmatic dependent launch hides the launch gap)
// when a cooperative launch is not available.
#include <cstring>

#include "decode_common.cuh"
#include "epilogue.cuh"
#include "internal.h"

namespace ffsp {
namespace dsk {

using namespace dec;

constexpr int WARPS = 8, THREADS = WARPS * 32;
constexpr int W_STAGE = WARPS * TILE_BYTES;     // eight 16-row tiles: 128 rows, or 64 rows of a gated pair
constexpr int W_BYTES = STAGES * W_STAGE;
constexpr int kBarCount = 16, kBarGen = 17;     // words of the control block used by the grid barrier
constexpr int kTicketWord0 = static_cast<int>(kStatusBytes / 4);   // tickets follow the status block
constexpr int kSlotTable = 256;                 // partial slots looked up per pass when a tile's partials are added
constexpr long long kWaitLimit = 2000000000ll;  // clock cycles (about a second) before a barrier wait gives up

using Product = DecodeProduct;

struct Params {
  Product prod[kMaxDecodeProducts];
  int nprod;
  int T;
  float* partial;   // [2 * gridDim.x] slots of 128 * 8 NT floats
  int* ctrl;        // control block: status words, barrier words, then one ticket per row tile (zero between launches)
};

template <int NT>
constexpr int smem_bytes() { return W_BYTES + STAGES * 2 * (8 * NT) * ROW_PITCH; }

// Shares of the `ge` CTAs that have one: CTA c owns units [c U / ge, (c + 1) U / ge).  U * (ge + 1) fits
// in 32 bits (checked when the product is planned).
__device__ __forceinline__ int share_lo(unsigned c, unsigned U, unsigned ge) { return static_cast<int>(c * U / ge); }
// the CTA whose share holds unit u
__device__ __forceinline__ int cta_of(unsigned u, unsigned U, unsigned ge) {
  return static_cast<int>(((u + 1) * ge - 1) / U);
}

// ---- copies of one unit ---------------------------------------------------------------------------
// weights: warp w stages rows [16 w, 16 w + 16) of the tile (gated: warps 0..3, both matrices)
template <bool DUAL>
__device__ __forceinline__ void issue_w(const Product& pr, int u, int buf, uint32_t smem0, int warp, int lane) {
  constexpr int AW = DUAL ? 4 : 8;
  if (warp >= AW) return;
  const int tile = u / pr.steps, step = u - tile * pr.steps;
  const int row0 = tile * (AW * 16) + warp * 16;
  const int k = step * KSTEP + lane * 8;
  const bool kin = k < pr.K;   // K is a multiple of 8
#pragma unroll
  for (int ti = 0; ti < (DUAL ? 2 : 1); ++ti) {
    const __nv_bfloat16* W = static_cast<const __nv_bfloat16*>(ti ? pr.W1 : pr.W0) + k;
    const uint32_t dst = smem0 + buf * W_STAGE + (DUAL ? 2 * warp + ti : warp) * TILE_BYTES + lane * 16;
#pragma unroll 4
    for (int r = 0; r < 16; ++r) {
      const int n = row0 + r;
      const bool ok = kin && n < pr.N;
      cp_async16(dst + r * ROW_PITCH, ok ? W + static_cast<long long>(n) * pr.ldw : W - k, ok);
    }
  }
}
// tokens: T rows of 512 bytes (twice that for a gated pair with two inputs), dealt to the eight warps;
// rows T .. 8 NT - 1 of a slab are never written and only feed accumulator columns that nobody reads
template <int NT>
__device__ __forceinline__ void issue_x(const Product& pr, int T, int u, int buf, uint32_t xs0, int warp, int lane) {
  constexpr int TP = 8 * NT;
  const int step = u % pr.steps;
  const int slabs = (pr.W1 != nullptr && pr.X1 != pr.X0) ? 2 : 1;
  const int k = step * KSTEP + lane * 8;
  const bool ok = k < pr.K;
  for (int q = warp; q < slabs * T; q += WARPS) {
    const int xi = q >= T ? 1 : 0, t = q - xi * T;
    const __nv_bfloat16* X = static_cast<const __nv_bfloat16*>(xi ? pr.X1 : pr.X0);
    cp_async16(xs0 + buf * (2 * TP * ROW_PITCH) + (xi * TP + t) * ROW_PITCH + lane * 16,
               X + (ok ? static_cast<long long>(t) * pr.ldx + k : 0), ok);
  }
}

template <int NT, bool DUAL>
__device__ __forceinline__ void compute(float (&acc)[DUAL ? 2 : 1][NT][4], bool two_slabs, int buf, uint32_t smem0,
                                        uint32_t xs0, int warp, int lane) {
  constexpr int AW = DUAL ? 4 : 8, TILES = DUAL ? 2 : 1, TP = 8 * NT;
  if (warp >= AW) return;
  const int g = lane >> 2, c = lane & 3;
  const uint32_t src0 = smem0 + buf * W_STAGE + (DUAL ? 2 * warp : warp) * TILE_BYTES + g * ROW_PITCH + c * 16;
  const uint32_t xsrc = xs0 + buf * (2 * TP * ROW_PITCH) + g * ROW_PITCH + c * 16;
  const uint32_t x1off = two_slabs ? TP * ROW_PITCH : 0;
#pragma unroll 2
  for (int it = 0; it < 8; ++it) {
    // rows g and g + 8 of the tile, the same 16 bytes of k: used as they are for two MMAs
    uint4 lo[TILES], hi[TILES];
#pragma unroll
    for (int ti = 0; ti < TILES; ++ti) {
      lo[ti] = lds128(src0 + ti * TILE_BYTES + it * 64);
      hi[ti] = lds128(src0 + ti * TILE_BYTES + 8 * ROW_PITCH + it * 64);
    }
#pragma unroll
    for (int j = 0; j < NT; ++j) {
      const uint4 xb = lds128(xsrc + 8 * j * ROW_PITCH + it * 64);
      mma_bf16(acc[0][j], lo[0].x, hi[0].x, lo[0].y, hi[0].y, xb.x, xb.y);
      mma_bf16(acc[0][j], lo[0].z, hi[0].z, lo[0].w, hi[0].w, xb.z, xb.w);
      if (DUAL) {
        const uint4 xu = two_slabs ? lds128(xsrc + x1off + 8 * j * ROW_PITCH + it * 64) : xb;
        mma_bf16(acc[TILES - 1][j], lo[TILES - 1].x, hi[TILES - 1].x, lo[TILES - 1].y, hi[TILES - 1].y, xu.x, xu.y);
        mma_bf16(acc[TILES - 1][j], lo[TILES - 1].z, hi[TILES - 1].z, lo[TILES - 1].w, hi[TILES - 1].w, xu.z, xu.w);
      }
    }
  }
}

// bias, activation and the [C0 | C1] column split for one output value (gated values arrive finished)
template <bool DUAL>
__device__ __forceinline__ void store_out(const Epilogue& ep, const GeluCoef& gc, int n, int t, float v) {
  if (!DUAL) {
    if (n < ep.n_bias) v += __ldg(ep.bias + n);
    if (n < ep.n_act) v = gelu_fast(v, gc);
  }
  const __nv_bfloat16 o = __float2bfloat16_rn(v);
  if (n < ep.n_split) reinterpret_cast<__nv_bfloat16*>(ep.C0)[static_cast<long long>(t) * ep.ld0 + n] = o;
  else reinterpret_cast<__nv_bfloat16*>(ep.C1)[static_cast<long long>(t) * ep.ld1 + (n - ep.n_split)] = o;
}

// All CTAs are resident (cooperative launch).  Count in, the last one opens the next generation.
// Returns false when the wait ran out; the caller then leaves the kernel.
__device__ __noinline__ bool grid_barrier(int* ctrl, int* s_flag) {
  __syncthreads();
  if (threadIdx.x == 0) {
    unsigned* count = reinterpret_cast<unsigned*>(ctrl + kBarCount);
    unsigned* genp = reinterpret_cast<unsigned*>(ctrl + kBarGen);
    unsigned gen;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(gen) : "l"(genp) : "memory");
    __threadfence();
    int ok = 1;
    if (atomicAdd(count, 1u) == gridDim.x - 1) {
      atomicExch(count, 0u);
      __threadfence();
      asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(genp), "r"(gen + 1) : "memory");
    } else {
      const long long t0 = clock64();
      unsigned now = gen;
      while (now == gen) {
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(now) : "l"(genp) : "memory");
        if (now == gen && clock64() - t0 > kWaitLimit) { ok = 0; break; }
      }
      if (!ok) record_status(ctrl, FFSPLIT_ERR_TIMEOUT, static_cast<int>(blockIdx.x), KID_DECODE);
    }
    __threadfence();
    *s_flag = ok;
  }
  __syncthreads();
  return *s_flag != 0;
}

// ---- one product -------------------------------------------------------------------------------
// `first`: the product opens the kernel (its inputs come from the launch before: wait for that one);
// otherwise its inputs come from the product before (grid barrier).  Either wait sits behind the
// first two weight copies.  Returns false if the barrier gave up.
template <int NT, bool DUAL>
__device__ __forceinline__ bool run_product(const Product& pr, const Params& p, bool first, uint32_t smem0,
                                            uint32_t xs0, int* s_flag, int* s_slot) {
  constexpr int AW = DUAL ? 4 : 8, TR = AW * 16, TILES = DUAL ? 2 : 1, TP = 8 * NT;
  constexpr int SLOT = 128 * TP;   // floats of one partial: [TILES][TR][TP]
  constexpr int EPT = TR * TP / (4 * THREADS) > 0 ? TR * TP / (4 * THREADS) : 1;   // float4 sums per thread when partials are added
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, c = lane & 3;
  const unsigned U = static_cast<unsigned>(pr.tiles) * pr.steps;
  const unsigned ge = U < gridDim.x ? U : gridDim.x;   // CTAs with a share
  const int cta = blockIdx.x;
  const bool mine = cta < static_cast<int>(ge);
  const int u0 = mine ? share_lo(cta, U, ge) : 0, u1 = mine ? share_lo(cta + 1, U, ge) : 0;
  const int n = u1 - u0;
  const bool two_slabs = DUAL && pr.X1 != pr.X0;
  const GeluCoef gc = gelu_coef(pr.epi.act);

  float acc[TILES][NT][4];
#pragma unroll
  for (int i = 0; i < TILES; ++i)
#pragma unroll
    for (int j = 0; j < NT; ++j)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[i][j][e] = 0.f;

  const int first_tile = u0 / pr.steps;
  int tile = first_tile, step = u0 - first_tile * pr.steps;
  int seg_lo = step;
  // q = -2, -1: the weights of units 0 and 1 go out ahead of the wait; from q = 0 on the pipeline runs
  for (int q = -2; q < n || q <= 0; ++q) {
    if (q == 0) {
      if (first) asm volatile("griddepcontrol.wait;" ::: "memory");
      else if (!grid_barrier(p.ctrl, s_flag)) return false;
      if (n > 0) { issue_x<NT>(pr, p.T, u0, 0, xs0, warp, lane); asm volatile("cp.async.commit_group;" ::: "memory"); }
      if (n > 1) { issue_x<NT>(pr, p.T, u0 + 1, 1, xs0, warp, lane); asm volatile("cp.async.commit_group;" ::: "memory"); }
      if (n == 0) break;
    }
    if (q >= 0) {
      if (q + 1 < n) asm volatile("cp.async.wait_group 1;" ::: "memory");
      else asm volatile("cp.async.wait_group 0;" ::: "memory");
      __syncthreads();   // unit q of every warp has landed: the token rows are shared
      compute<NT, DUAL>(acc, two_slabs, q & 1, smem0, xs0, warp, lane);
      __syncthreads();   // its stage is free again
    }
    if (q + 2 < n) {
      issue_w<DUAL>(pr, u0 + q + 2, q & 1, smem0, warp, lane);
      if (q >= 0) {
        issue_x<NT>(pr, p.T, u0 + q + 2, q & 1, xs0, warp, lane);
        asm volatile("cp.async.commit_group;" ::: "memory");
      }
    }
    if (q < 0) continue;
    if (step == pr.steps - 1 || q == n - 1) {
      // ---- end of this CTA's part of the tile
      if (seg_lo == 0 && step == pr.steps - 1) {
        if (warp < AW) {
          const int n0 = tile * TR + warp * 16 + g;
#pragma unroll
          for (int j = 0; j < NT; ++j)
#pragma unroll
            for (int e = 0; e < 4; ++e) {
              const int nn = n0 + (e >= 2 ? 8 : 0), t = 8 * j + 2 * c + (e & 1);
              const float v = DUAL ? silu_fast(acc[0][j][e]) * acc[TILES - 1][j][e] : acc[0][j][e];
              if (nn < pr.N && t < p.T) store_out<DUAL>(pr.epi, gc, nn, t, v);
            }
        }
      } else {
        float* dst = p.partial + static_cast<long long>(2 * cta + (tile == first_tile ? 0 : 1)) * SLOT;
        if (warp < AW) {
#pragma unroll
          for (int i = 0; i < TILES; ++i)
#pragma unroll
            for (int j = 0; j < NT; ++j) {
              float* d0 = dst + (i * TR + warp * 16 + g) * TP + 8 * j + 2 * c;
              *reinterpret_cast<float2*>(d0) = make_float2(acc[i][j][0], acc[i][j][1]);
              *reinterpret_cast<float2*>(d0 + 8 * TP) = make_float2(acc[i][j][2], acc[i][j][3]);
            }
        }
        const unsigned t_lo = static_cast<unsigned>(tile) * pr.steps;
        const int c_first = cta_of(t_lo, U, ge), c_last = cta_of(t_lo + pr.steps - 1, U, ge);
        __threadfence();
        __syncthreads();
        if (threadIdx.x == 0) {
          int* ticket = p.ctrl + kTicketWord0 + tile;
          const int arrived = atomicAdd(ticket, 1);
          const int last = arrived == c_last - c_first;
          if (last) *ticket = 0;   // nobody else comes for this tile; the next product starts behind a barrier
          *s_flag = last;
          __threadfence();
        }
        __syncthreads();
        if (*s_flag) {
          // The partials of the tile, added in CTA order.  Which of its two slots a CTA used is worked
          // out once per CTA; then every thread sums four neighbouring values, with many loads in flight.
          const int ncon = c_last - c_first + 1;
          float4 sum0[EPT], sum1[EPT];
#pragma unroll
          for (int e = 0; e < EPT; ++e) sum0[e] = sum1[e] = make_float4(0.f, 0.f, 0.f, 0.f);
          for (int i0 = 0; i0 < ncon; i0 += kSlotTable) {
            const int nc = ncon - i0 < kSlotTable ? ncon - i0 : kSlotTable;
            __syncthreads();
            for (int i = threadIdx.x; i < nc; i += THREADS) {
              const int cc = c_first + i0 + i;
              s_slot[i] = 2 * cc + (share_lo(cc, U, ge) / pr.steps == tile ? 0 : 1);
            }
            __syncthreads();
#pragma unroll
            for (int e = 0; e < EPT; ++e) {
              const int idx = 4 * (threadIdx.x + e * THREADS);
              if (idx >= TR * TP) break;
#pragma unroll 8
              for (int i = 0; i < nc; ++i) {
                const float* src = p.partial + static_cast<long long>(s_slot[i]) * SLOT + idx;
                const float4 a = __ldcg(reinterpret_cast<const float4*>(src));
                sum0[e].x += a.x; sum0[e].y += a.y; sum0[e].z += a.z; sum0[e].w += a.w;
                if (DUAL) {
                  const float4 b = __ldcg(reinterpret_cast<const float4*>(src + TR * TP));
                  sum1[e].x += b.x; sum1[e].y += b.y; sum1[e].z += b.z; sum1[e].w += b.w;
                }
              }
            }
          }
#pragma unroll
          for (int e = 0; e < EPT; ++e) {
            const int idx = 4 * (threadIdx.x + e * THREADS);
            if (idx >= TR * TP) break;
            const int r = idx / TP, t = idx - r * TP;
            const int nn = tile * TR + r;
            const float a[4] = {sum0[e].x, sum0[e].y, sum0[e].z, sum0[e].w};
            const float b[4] = {sum1[e].x, sum1[e].y, sum1[e].z, sum1[e].w};
#pragma unroll
            for (int x = 0; x < 4; ++x)
              if (nn < pr.N && t + x < p.T) store_out<DUAL>(pr.epi, gc, nn, t + x, DUAL ? silu_fast(a[x]) * b[x] : a[x]);
          }
        }
      }
#pragma unroll
      for (int i = 0; i < TILES; ++i)
#pragma unroll
        for (int j = 0; j < NT; ++j)
#pragma unroll
          for (int e = 0; e < 4; ++e) acc[i][j][e] = 0.f;
      seg_lo = 0;
    }
    if (++step == pr.steps) { step = 0; ++tile; }
  }
  return true;
}

// GATED: the layer has gated pairs (then both kinds of product occur); otherwise only plain products.
template <int NT, bool GATED>
__global__ void __launch_bounds__(THREADS, 1) decode_layer_kernel(const __grid_constant__ Params p) {
  extern __shared__ __align__(16) unsigned char smem[];
  __shared__ int s_flag;
  __shared__ int s_slot[kSlotTable];
  const uint32_t smem0 = static_cast<uint32_t>(__cvta_generic_to_shared(smem));
  const uint32_t xs0 = smem0 + W_BYTES;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // a dependent launch may start its own first copies
  for (int pi = 0; pi < p.nprod; ++pi) {
    const Product& pr = p.prod[pi];
    bool ok;
    if (GATED && pr.W1) ok = run_product<NT, true>(pr, p, pi == 0, smem0, xs0, &s_flag, s_slot);
    else ok = run_product<NT, false>(pr, p, pi == 0, smem0, xs0, &s_flag, s_slot);
    if (!ok) {
      asm volatile("cp.async.wait_all;" ::: "memory");
      return;
    }
    __syncthreads();   // every warp is done with the staging buffers
  }
}

template <int NT, bool GATED>
cudaError_t launch_nt(const Params& p, int grid, bool cooperative, cudaStream_t st) {
  static bool attr_done = false;
  if (!attr_done) {
    cudaError_t e = cudaFuncSetAttribute(decode_layer_kernel<NT, GATED>, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes<NT>());
    if (e != cudaSuccess) return e;
    attr_done = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(THREADS);
  cfg.dynamicSmemBytes = smem_bytes<NT>();
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  if (cooperative) {
    attr[0].id = cudaLaunchAttributeCooperative;
    attr[0].val.cooperative = 1;
  } else {
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
  }
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, decode_layer_kernel<NT, GATED>, p);
}

cudaError_t launch_any(int nt, bool gated, const Params& p, int grid, bool cooperative, cudaStream_t st) {
#define FFS_DL(NT_) (gated ? launch_nt<NT_, true>(p, grid, cooperative, st) : launch_nt<NT_, false>(p, grid, cooperative, st))
  if (nt == 1) return FFS_DL(1);
  if (nt == 2) return FFS_DL(2);
  return FFS_DL(4);
#undef FFS_DL
}

}  // namespace dsk

// ---- host side ---------------------------------------------------------------------------------
bool decode_layer_applies(long long T) { return T >= 1 && T <= 32; }

// fp32 partials: two slots per CTA
size_t decode_layer_scratch_bytes(int num_sms, long long T) {
  const int nt = T <= 8 ? 1 : T <= 16 ? 2 : 4;
  return static_cast<size_t>(2) * num_sms * 128 * 8 * nt * 4;
}

ffsplit_status decode_layer_add(ffsplit_ctx* ctx, DecodeLayerPlan* plan, const void* X0, const void* X1, long long ldx,
                                const void* W0, const void* W1, long long ldw, int N, int K, const Epilogue& epi,
                                double algo_bytes) {
  if (N <= 0 || K <= 0) return FFSPLIT_OK;
  if (plan->n >= kMaxDecodeProducts) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "few-token forward: too many products");
  DecodeProduct pr;
  pr.X0 = X0; pr.X1 = X1; pr.ldx = ldx;
  pr.W0 = W0; pr.W1 = W1; pr.ldw = ldw;
  pr.N = N; pr.K = K;
  const int tr = W1 ? 64 : 128;
  pr.tiles = (N + tr - 1) / tr;
  pr.steps = (K + dec::KSTEP - 1) / dec::KSTEP;
  pr.epi = epi;
  if (pr.tiles > kMaxTicketTiles) return fail(ctx, FFSPLIT_ERR_SHAPE, "few-token forward: more row tiles than ticket counters");
  if (static_cast<double>(pr.tiles) * pr.steps * (ctx->num_sms + 1) >= 2147483648.0)
    return fail(ctx, FFSPLIT_ERR_SHAPE, "few-token forward: product too large for the unit arithmetic");
  plan->prod[plan->n++] = pr;
  plan->algo_bytes += algo_bytes;
  return FFSPLIT_OK;
}

// ctrl: the control block (status and barrier words, then the tickets); partial: decode_layer_scratch_bytes.
ffsplit_status decode_layer_launch(ffsplit_ctx* ctx, const DecodeLayerPlan* plan, int T, float* partial, int* ctrl,
                                   cudaStream_t st) {
  if (plan->n == 0) return FFSPLIT_OK;
  const int nt = T <= 8 ? 1 : T <= 16 ? 2 : 4;
  bool gated = false;
  for (int i = 0; i < plan->n; ++i) gated = gated || plan->prod[i].W1 != nullptr;
  // cooperative launch: supported, and one CTA per SM fits
  static int coop_ok[64] = {0};   // per device: 0 unknown, 1 yes, -1 no
  const int dev = ctx->device;
  if (dev >= 0 && dev < 64 && coop_ok[dev] == 0) {
    int v = 0;
    coop_ok[dev] = (cudaDeviceGetAttribute(&v, cudaDevAttrCooperativeLaunch, dev) == cudaSuccess && v) ? 1 : -1;
  }
  const bool coop = ctx->decode_one_launch && dev >= 0 && dev < 64 && coop_ok[dev] == 1 && plan->n > 1;
  dsk::Params p;
  std::memset(&p, 0, sizeof(p));
  p.T = T; p.partial = partial; p.ctrl = ctrl;
  const int ph = prof_open(ctx, PROF_DECODE, plan->algo_bytes, st);
  cudaError_t e = cudaSuccess;
  if (coop) {
    for (int i = 0; i < plan->n; ++i) p.prod[i] = plan->prod[i];
    p.nprod = plan->n;
    e = dsk::launch_any(nt, gated, p, ctx->num_sms, true, st);
    ctx->launches++;
  } else {
    for (int i = 0; i < plan->n && e == cudaSuccess; ++i) {
      p.prod[0] = plan->prod[i];
      p.nprod = 1;
      e = dsk::launch_any(nt, gated, p, ctx->num_sms, false, st);
      ctx->launches++;
    }
  }
  prof_close(ctx, ph, st);
  return check_cuda(ctx, e, "decode_layer_kernel launch");
}

}  // namespace ffsp
