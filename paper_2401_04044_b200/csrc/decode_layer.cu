// Few-token (decode) split forward, T <= 64 tokens: every product of Eq. 2 in one persistent kernel.
//
// With a handful of tokens each stage of Eq. 2 is a skinny product
//     C[t, n] = epi( sum_k X[t, k] * W[n, k] )        W: [N, K] K-major weights from the packed blob
// whose cost is reading W once from HBM, and a split layer is four or five such products of a few
// megabytes each: what is left to lose is time in which an SM has no loads in flight.  So:
//
//  * One CTA per SM stays resident for the whole layer.  A product is cut into units of
//    128 weight rows x 256 k (64 KB of W); the units, in row-tile-major order, are dealt to the CTAs in
//    equal contiguous shares (a tile's K range may straddle two or more CTAs).
//  * The warps of a CTA walk its share side by side -- each owns 16 rows of every tile -- and never wait
//    for one another's weights: each has its own two-stage cp.async ring, so a late DRAM reply holds up
//    one warp, not the SM, and the ring does not drain at tile boundaries.
//  * Each warp-wide copy moves 512 contiguous bytes of one weight row.  The token rows of a unit's k
//    range are staged once per CTA, a few units ahead, in a ring of slabs guarded by mbarriers (loading
//    them at the point of use costs a quarter of the bandwidth: they queue behind the weight stream).
//    Fragments for the warp-level MMA (m16n8k16, weights as the 16-row operand, tokens as the 8-wide
//    one) are read from shared memory with 128-bit loads; since a contraction does not care in which
//    order k is visited, a thread's 16 bytes feed two MMAs as they are, and the token operand is read
//    with the same pattern.
//  * Rows finished inside one CTA go through the epilogue straight from the accumulator registers.
//    Rows shared by several CTAs: each warp writes an fp32 partial (at most two per CTA and product:
//    the tile its share starts in and the tile it ends in), takes an atomic ticket, and the last to
//    arrive adds the partials in CTA order -- the result does not depend on who arrives when.
//  * Products are separated by a grid-wide barrier (cooperative launch: all CTAs are resident), before
//    which each warp has already issued the first weight copies of the next product.
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
#include "ptx.cuh"

namespace ffsp {
namespace dsk {

using namespace dec;

constexpr int WARPS = 8, THREADS = WARPS * 32;
constexpr int SMEM_BYTES = 3 * 8 * TILE_BYTES;   // the same for every shape below
constexpr int RING_BYTES = 2 * 8 * TILE_BYTES;   // weight rings of the warps; the rest holds token rows
constexpr int XCAP_BYTES = SMEM_BYTES - RING_BYTES;   // shared token slabs (more than 8 tokens)
constexpr int kMaxSlots = 8;                     // slabs in the shared ring, at most
constexpr int kBarCount = 16, kBarGen = 17;     // words of the control block used by the grid barrier
constexpr int kTicketWord0 = static_cast<int>(kStatusBytes / 4);   // tickets follow the status block
constexpr long long kWaitLimit = 2000000000ll;  // clock cycles (about a second) before a barrier wait gives up

using Product = DecodeProduct;

struct Params {
  Product prod[kMaxDecodeProducts];
  int nprod;
  int T;
  float* partial;   // [2 * gridDim.x] slots of 128 * 8 NT floats
  int* ctrl;        // control block: status words, barrier words, then eight tickets per row tile (zero between launches)
};

// A CTA tile is 128 weight rows (64 rows of each matrix for a gated pair); warp w owns 16 of them and
// has a two-stage ring for them.  The token rows of a unit's k range (a slab) are staged once per CTA, in
// a ring of slabs beside the weight rings: all warps load a share of each slab, a few units ahead of its
// use, and meet only through two mbarriers per slot -- `full` (the slab has landed: every thread's copies,
// tracked by cp.async.mbarrier.arrive) and `empty` (every warp is done reading it).  No warp waits for
// another's weights.  (Measured alternatives, OPT-13B dense layer, 1 / 8 tokens: every warp copying the
// token rows for itself 87 / 103 us; this ring 88 / 87 us.)
template <int NT, bool DUAL>
struct Shape {
  static constexpr int NST = 2;                      // stages of a warp's weight ring
  static constexpr int TILES = DUAL ? 2 : 1;
  static constexpr int AW = DUAL ? 4 : 8;            // working warps
  static constexpr int TR = AW * 16;                 // rows of a CTA tile
  static constexpr int TP = 8 * NT;                  // token rows, padded
  static constexpr int W_BYTES = TILES * TILE_BYTES;
  static constexpr int STAGE = W_BYTES;
  static_assert(AW * NST * STAGE == RING_BYTES, "shared memory plan");
  static_assert(TILES * TP * ROW_PITCH <= XCAP_BYTES, "one slab must fit");
};

// Shares of the `ge` CTAs that have one: CTA c owns units [c U / ge, (c + 1) U / ge).  U * (ge + 1) fits
// in 32 bits (checked when the product is planned).
__device__ __forceinline__ int share_lo(unsigned c, unsigned U, unsigned ge) { return static_cast<int>(c * U / ge); }
// the CTA whose share holds unit u
__device__ __forceinline__ int cta_of(unsigned u, unsigned U, unsigned ge) {
  return static_cast<int>(((u + 1) * ge - 1) / U);
}

// weights of one unit: the warp's 16 rows (gated: of both matrices), 512 bytes each, one row per warp-wide copy
template <int NT, bool DUAL>
__device__ __forceinline__ void issue_w(const Product& pr, int tile, int step, uint32_t stage_smem, int warp, int lane) {
  using S = Shape<NT, DUAL>;
  const int row0 = tile * S::TR + warp * 16;
  const int k = step * KSTEP + lane * 8;
  const bool inside = row0 + 16 <= pr.N && (step + 1) * KSTEP <= pr.K;   // the same for the whole warp
#pragma unroll
  for (int ti = 0; ti < S::TILES; ++ti) {
    const __nv_bfloat16* W = static_cast<const __nv_bfloat16*>(ti ? pr.W1 : pr.W0);
    const __nv_bfloat16* src = W + static_cast<long long>(row0) * pr.ldw + k;
    uint32_t dst = stage_smem + ti * TILE_BYTES + lane * 16;
    if (inside) {
#pragma unroll 8
      for (int r = 0; r < 16; ++r, src += pr.ldw, dst += ROW_PITCH) cp_async16_full(dst, src);
    } else {
      const bool kin = k < pr.K;   // K is a multiple of 8
#pragma unroll 4
      for (int r = 0; r < 16; ++r, src += pr.ldw, dst += ROW_PITCH) {
        const bool ok = kin && row0 + r < pr.N;
        cp_async16(dst, ok ? src : W, ok);
      }
    }
  }
}
// One unit: the warp's 16 rows x 256 k against the token rows at xsmem (a second input, if there
// is one, follows 8 NT rows later).
template <int NT, bool DUAL>
__device__ __forceinline__ void compute(float (&acc)[DUAL ? 2 : 1][NT][4], bool two, uint32_t stage_smem,
                                        uint32_t xsmem, int lane) {
  using S = Shape<NT, DUAL>;
  const int g = lane >> 2, c = lane & 3;
  const uint32_t wsrc = stage_smem + g * ROW_PITCH + c * 16;
  const uint32_t xsrc = xsmem + g * ROW_PITCH + c * 16;
#pragma unroll 2
  for (int it = 0; it < 8; ++it) {
#pragma unroll
    for (int ti = 0; ti < S::TILES; ++ti) {
      uint4 xb[NT];
      const uint32_t xs = xsrc + ((ti && two) ? S::TP * ROW_PITCH : 0) + it * 64;
#pragma unroll
      for (int j = 0; j < NT; ++j) xb[j] = lds128(xs + 8 * j * ROW_PITCH);
      // rows g and g + 8 of the tile, the same 16 bytes of k: used as they are for two MMAs (the order
      // in which a contraction visits k is free as long as both operands agree on it)
      const uint32_t ws = wsrc + ti * TILE_BYTES + it * 64;
      const uint4 lo = lds128(ws), hi = lds128(ws + 8 * ROW_PITCH);
      // all token tiles with the first half of k, then all with the second: two MMAs into the same
      // accumulator are NT instructions apart instead of back to back
#pragma unroll
      for (int j = 0; j < NT; ++j) mma_bf16(acc[ti][j], lo.x, hi.x, lo.y, hi.y, xb[j].x, xb[j].y);
#pragma unroll
      for (int j = 0; j < NT; ++j) mma_bf16(acc[ti][j], lo.z, hi.z, lo.w, hi.w, xb[j].z, xb[j].w);
    }
  }
}

// This warp's share of a shared slab: token rows warp, warp + 8, ... of each input; then every lane
// tells the slot's `full` barrier to count it in once its copies have landed.
__device__ __forceinline__ void issue_slab(const Product& pr, int T, int TP, int slabs, int step, uint32_t slab_smem,
                                               uint64_t* full, int warp, int lane) {
  const int k = step * KSTEP + lane * 8;
  const bool ok = k < pr.K;
  for (int xi = 0; xi < slabs; ++xi) {
    const __nv_bfloat16* X = static_cast<const __nv_bfloat16*>(xi ? pr.X1 : pr.X0) + (ok ? k : 0);
    const uint32_t dst = slab_smem + xi * (TP * ROW_PITCH) + lane * 16;
    for (int t = warp; t < T; t += WARPS) cp_async16(dst + t * ROW_PITCH, ok ? X + static_cast<long long>(t) * pr.ldx : X, ok);
  }
  asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(ptx::smem_u32(full)) : "memory");
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
// The working warps of a CTA walk the CTA's share side by side: each has its own ring of weight
// stages, its own accumulators, and finishes its rows of a tile by itself (ticket per tile and warp).
// `first`: the product opens the kernel (its inputs come from the launch before: wait for that one);
// otherwise its inputs come from the product before (grid barrier).  Either wait sits behind the
// first weight copies.  Returns false if a wait gave up.
template <int NT, bool DUAL>
__device__ __forceinline__ bool run_product(const Product& pr, const Params& p, bool first, uint32_t smem0,
                                            int* s_flag, uint64_t* full, uint64_t* empty, volatile int* s_abort) {
  using S = Shape<NT, DUAL>;
  constexpr int TILES = S::TILES, TR = S::TR, TP = S::TP, NST = S::NST;
  constexpr int SLOT = 128 * TP;              // floats of one CTA partial: [TILES][TR][TP]
  constexpr int ROWV = 16 * TP / 4;           // float4 values of the warp's rows (one matrix)
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 2, c = lane & 3;
  const unsigned U = static_cast<unsigned>(pr.tiles) * pr.steps;
  const unsigned ge = U < gridDim.x ? U : gridDim.x;   // CTAs with a share
  const int cta = blockIdx.x;
  const bool has = cta < static_cast<int>(ge);
  const bool worker = warp < S::AW;            // the other warps only help with shared slabs
  const int u0 = has ? share_lo(cta, U, ge) : 0, u1 = has ? share_lo(cta + 1, U, ge) : 0;
  const int n = u1 - u0;
  const bool two = DUAL && pr.X1 != pr.X0;
  const GeluCoef gc = gelu_coef(pr.epi.act);
  const uint32_t my_smem = smem0 + warp * (NST * S::STAGE);
  // shared slabs: as many slots as fit, filled LOOK units ahead of their use
  const int slabs = two ? 2 : 1;
  const int slab_bytes = slabs * TP * ROW_PITCH;
  const int R = XCAP_BYTES / slab_bytes < kMaxSlots ? XCAP_BYTES / slab_bytes : kMaxSlots;
  const int LOOK = R > 1 ? R / 2 : 0;   // slabs in flight ahead of their use; the other slots let the warps drift apart
  const uint32_t xring = smem0 + RING_BYTES;

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
  int tile_a = tile, step_a = step;   // the next unit whose weights go out
  int step_x = step;                  // the k step of the next shared slab
  // q < 0: the weights of the first units go out ahead of the wait; from q = 0 on the pipeline runs.
  // A worker commits one copy group per unit (its slab copies ride in whichever group comes next).
  for (int q = -NST; q < n || q <= 0; ++q) {
    if (q == 0) {
      if (first) asm volatile("griddepcontrol.wait;" ::: "memory");
      else if (!grid_barrier(p.ctrl, s_flag)) return false;
      if (cta == 0 && warp == 0) check_blob_guard(pr.epi, p.ctrl, KID_DECODE);
      if (n == 0) break;
      for (int j = 0; j < LOOK && j < n; ++j) {
        issue_slab(pr, p.T, TP, slabs, step_x, xring + j * slab_bytes, full + j, warp, lane);
        if (++step_x == pr.steps) step_x = 0;
      }
    }
    const uint32_t stage_smem = my_smem + ((q + NST) % NST) * S::STAGE;
    if (q >= 0) {
      // the slab LOOK units ahead goes into the slot that unit q - 1 used: wait until every warp has read it
      const int j = q + LOOK;
      if (j < n) {
        const int slot = j % R, use = j / R;
        if (use > 0 && !ptx::mbar_wait(empty + slot, (use - 1) & 1, s_abort)) return false;
        issue_slab(pr, p.T, TP, slabs, step_x, xring + slot * slab_bytes, full + slot, warp, lane);
        if (++step_x == pr.steps) step_x = 0;
      }
      const uint32_t xsmem = xring + (q % R) * slab_bytes;
      if (worker) {
        if (n - 1 - q >= 1) asm volatile("cp.async.wait_group 1;" ::: "memory");
        else asm volatile("cp.async.wait_group 0;" ::: "memory");
      }
      if (!ptx::mbar_wait(full + q % R, (q / R) & 1, s_abort)) return false;
      __syncwarp();
      if (worker) compute<NT, DUAL>(acc, two, stage_smem, xsmem, lane);
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(empty + q % R);
    }
    if (worker && q + NST < n) {
      issue_w<NT, DUAL>(pr, tile_a, step_a, stage_smem, warp, lane);
      if (++step_a == pr.steps) { step_a = 0; ++tile_a; }
      asm volatile("cp.async.commit_group;" ::: "memory");
    }
    if (q < 0) continue;
    if (!worker) {
      if (++step == pr.steps) { step = 0; ++tile; }
      continue;
    }
    if (step == pr.steps - 1 || q == n - 1) {
      // ---- end of this warp's part of the tile
      const int wrow = warp * 16;   // the warp's first row inside the tile
      if (seg_lo == 0 && step == pr.steps - 1) {
#pragma unroll
        for (int j = 0; j < NT; ++j)
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const int nn = tile * TR + wrow + g + (e >= 2 ? 8 : 0), t = 8 * j + 2 * c + (e & 1);
            const float v = DUAL ? silu_fast(acc[0][j][e]) * acc[TILES - 1][j][e] : acc[0][j][e];
            if (nn < pr.N && t < p.T) store_out<DUAL>(pr.epi, gc, nn, t, v);
          }
      } else {
        float* dst = p.partial + static_cast<long long>(2 * cta + (tile == first_tile ? 0 : 1)) * SLOT;
#pragma unroll
        for (int i = 0; i < TILES; ++i)
#pragma unroll
          for (int j = 0; j < NT; ++j) {
            float* d0 = dst + (i * TR + wrow + g) * TP + 8 * j + 2 * c;
            *reinterpret_cast<float2*>(d0) = make_float2(acc[i][j][0], acc[i][j][1]);
            *reinterpret_cast<float2*>(d0 + 8 * TP) = make_float2(acc[i][j][2], acc[i][j][3]);
          }
        const unsigned t_lo = static_cast<unsigned>(tile) * pr.steps;
        const int c_first = cta_of(t_lo, U, ge), c_last = cta_of(t_lo + pr.steps - 1, U, ge);
        __threadfence();
        __syncwarp();
        int last = 0;
        if (lane == 0) {
          int* ticket = p.ctrl + kTicketWord0 + tile * WARPS + warp;
          last = atomicAdd(ticket, 1) == c_last - c_first;
          if (last) *ticket = 0;   // nobody else comes for these rows; the next product starts behind a barrier
          __threadfence();
        }
        last = __shfl_sync(0xffffffffu, last, 0);
        if (last) {
          // The partials of these rows, added in CTA order.  Which of its two slots a CTA used is worked
          // out by one lane per CTA and handed round; each lane sums four neighbouring values at a time.
          const int ncon = c_last - c_first + 1;
          const float* base = p.partial + wrow * TP;
          for (int v4 = lane; v4 < ROWV; v4 += 32) {
            float4 s0 = make_float4(0.f, 0.f, 0.f, 0.f), s1 = s0;
            for (int i0 = 0; i0 < ncon; i0 += 32) {
              const int nc = ncon - i0 < 32 ? ncon - i0 : 32;
              const int cc = c_first + i0 + (lane < nc ? lane : 0);
              const int my_slot = 2 * cc + (share_lo(cc, U, ge) / pr.steps == tile ? 0 : 1);
#pragma unroll 8
              for (int i = 0; i < nc; ++i) {
                const float* src = base + static_cast<long long>(__shfl_sync(0xffffffffu, my_slot, i)) * SLOT;
                const float4 a = __ldcg(reinterpret_cast<const float4*>(src) + v4);
                s0.x += a.x; s0.y += a.y; s0.z += a.z; s0.w += a.w;
                if (DUAL) {
                  const float4 b = __ldcg(reinterpret_cast<const float4*>(src + TR * TP) + v4);
                  s1.x += b.x; s1.y += b.y; s1.z += b.z; s1.w += b.w;
                }
              }
            }
            const int r = (4 * v4) / TP, t = 4 * v4 - r * TP;
            const int nn = tile * TR + wrow + r;
            const float a[4] = {s0.x, s0.y, s0.z, s0.w};
            const float b[4] = {s1.x, s1.y, s1.z, s1.w};
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
  __shared__ int s_abort;
  __shared__ __align__(8) uint64_t s_full[kMaxSlots], s_empty[kMaxSlots];
  const uint32_t smem0 = static_cast<uint32_t>(__cvta_generic_to_shared(smem));
  if (threadIdx.x == 0) s_abort = 0;
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");   // a dependent launch may start its own first copies
  for (int pi = 0; pi < p.nprod; ++pi) {
    const Product& pr = p.prod[pi];
    {
      // slab barriers start every product in phase 0: `full` counts every thread, `empty` every warp
      if (threadIdx.x == 0) {
        for (int i = 0; i < kMaxSlots; ++i) { ptx::mbar_init(s_full + i, THREADS); ptx::mbar_init(s_empty + i, WARPS); }
        ptx::mbar_fence_init();
      }
      __syncthreads();
    }
    bool ok;
    if (GATED && pr.W1) ok = run_product<NT, true>(pr, p, pi == 0, smem0, &s_flag, s_full, s_empty, &s_abort);
    else ok = run_product<NT, false>(pr, p, pi == 0, smem0, &s_flag, s_full, s_empty, &s_abort);
    if (!ok) {
      // a wait ran out: say so, let the copies in flight land, leave
      if ((threadIdx.x & 31) == 0) record_status(p.ctrl, FFSPLIT_ERR_TIMEOUT, static_cast<int>(blockIdx.x), KID_DECODE);
      asm volatile("cp.async.wait_all;" ::: "memory");
      return;
    }
    __syncthreads();   // every warp is done with the staging buffers
  }
}

template <int NT, bool GATED>
cudaError_t launch_nt(const Params& p, int grid, bool cooperative, cudaStream_t st) {
  // the shared-memory allowance is a per-device property of the function: set once on every device used
  static bool attr_done[64] = {false};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= 64 || !attr_done[dev]) {
    e = cudaFuncSetAttribute(decode_layer_kernel<NT, GATED>, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < 64) attr_done[dev] = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(THREADS);
  cfg.dynamicSmemBytes = SMEM_BYTES;
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
  if (nt == 4) return FFS_DL(4);
  return FFS_DL(8);
#undef FFS_DL
}

}  // namespace dsk

// ---- host side ---------------------------------------------------------------------------------
bool decode_layer_applies(long long T) { return T >= 1 && T <= 64; }

// fp32 partials: two slots per CTA
size_t decode_layer_scratch_bytes(int num_sms, long long T) {
  const int nt = T <= 8 ? 1 : T <= 16 ? 2 : T <= 32 ? 4 : 8;
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
  if (static_cast<long long>(pr.tiles) * 8 > kMaxTicketTiles) return fail(ctx, FFSPLIT_ERR_SHAPE, "few-token forward: more row tiles than ticket counters");
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
  const int nt = T <= 8 ? 1 : T <= 16 ? 2 : T <= 32 ? 4 : 8;
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
