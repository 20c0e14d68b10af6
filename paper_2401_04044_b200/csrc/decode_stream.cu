// Few-token (decode) split forward for 1..8 tokens: ONE persistent kernel per layer whose weight stream never
// waits for the dependencies between the stages of Eq. 2.
//
// With a handful of tokens every stage of Eq. 2 is a skinny product C[t, n] = sum_k A[t, k] W[n, k] whose
// cost is reading W once, and a split layer is a chain of four of them (stage 1, the two halves of the light
// chain, stage 3) of a few megabytes each.  What bounds such a layer is not bandwidth but the hand-over
// between dependent products.  This kernel is built around two facts:
//
//  * The weights do not depend on the activations.  One warp per CTA (the producer) walks the CTA's share of
//    ALL phases of the layer and copies it into a ring of shared-memory stages with bulk asynchronous copies
//    (cp.async.bulk, one 512-byte row segment per lane and instruction, completion counted on an mbarrier).
//    It never waits for a grid barrier: while the consumers wait for the previous phase to finish everywhere,
//    the next phase's weights are already landing, and HBM stays busy as long as the ring has a free stage.
//  * Eq. 1: output rows (neurons, or output columns of V) are independent.  Every phase's rows -- times a
//    small number S of k ranges when K is long -- are dealt to the CTAs in equal contiguous shares with
//    single-row granularity, so the load balance does not depend on tile shapes.  Inside a CTA the eight
//    consumer warps split the k range of every stage between them (each takes 64 bytes of every row: two
//    m16n8k16 MMAs per 16 rows) and are added through shared memory in warp order at the end of a block of
//    32 rows.  No CTA ever waits for another one's partial sums inside a phase: what a phase writes is raw
//    fp32 sums, one slice per k range, and whoever reads them in the next phase adds the S slices, adds the
//    bias, applies the activation and rounds to bf16 while staging its activation operand.  All sums are
//    taken in a fixed order: results are bitwise reproducible.
//
// Phases are separated by a grid-wide barrier (cooperative launch: all CTAs are resident).  Every wait --
// mbarrier or grid barrier -- is bounded; when one runs out the CTA raises a flag, every later wait returns
// at once, the control flow runs to its end (so that no warp is left behind at a CTA barrier), copies in
// flight are given a bounded time to land, and FFSPLIT_ERR_TIMEOUT is recorded in the status block.
#include <cstring>

#include "decode_common.cuh"
#include "decode_stream.h"
#include "epilogue.cuh"
#include "internal.h"
#include "ptx.cuh"

namespace ffsp {
namespace dst {

using namespace dec;

constexpr int CWARPS = 8;                                // consumer warps
constexpr int CTHREADS = 32 * CWARPS;
constexpr int THREADS = CTHREADS + 32;                   // + the producer warp
constexpr int BLOCK_ROWS = 32;                           // weight rows per stage: one bulk copy per lane
constexpr int KC = 256;                                  // k elements per stage: 512 contiguous bytes per row
constexpr int STAGE_BYTES = BLOCK_ROWS * ROW_PITCH;      // 18432
constexpr int NSTAGE = 9;
constexpr int X_PITCH = kStreamKxMax * 2 + 64;           // bytes between token rows of the activation operand
constexpr int X_BYTES = 8 * X_PITCH;
constexpr int RED_TOK = 36;                              // floats between token rows of a warp's partial block
constexpr int RED_WARP = 8 * RED_TOK;
constexpr int RED_BYTES = 2 * CWARPS * RED_WARP * 4;     // two buffers, used alternately
constexpr int OFF_X = NSTAGE * STAGE_BYTES;
constexpr int OFF_RED = OFF_X + X_BYTES;
constexpr int OFF_BAR = OFF_RED + RED_BYTES;
constexpr int SMEM_BYTES = OFF_BAR + 256;
static_assert(X_PITCH % 128 == 64 && ROW_PITCH % 128 == 64, "conflict-free 128-bit fragment reads");
static_assert(SMEM_BYTES <= 232448, "shared memory plan");
constexpr int kBarCount = 16, kBarGen = 17;              // words of the control block used by the grid barrier
constexpr long long kWaitLimit = 2000000000ll;           // SM clocks (about a second)

__device__ __forceinline__ void cbar() { asm volatile("bar.sync 1, %0;" ::"n"(CTHREADS) : "memory"); }

// ---- the walk over a CTA's share of one phase, taken identically by the producer and the consumers -----
struct Pass {
  int seg, s;          // segment, k range
  int row0, rows;      // rows [row0, row0 + rows) of the segment
  int kbeg, klen;      // k range in elements
};
struct Share { long long lo, hi; };   // units [lo, hi) of the phase: unit = s * Nall + row

__device__ __forceinline__ Share share_of(const StreamPhase& ph, int cta, int ncta) {
  const long long U = static_cast<long long>(ph.S) * ph.Nall;
  Share sh;
  sh.lo = U * cta / ncta;
  sh.hi = U * (cta + 1) / ncta;
  return sh;
}
// the pass that starts at unit u (u < hi)
__device__ __forceinline__ Pass pass_at(const StreamPhase& ph, long long u, long long hi) {
  Pass p;
  p.s = static_cast<int>(u / ph.Nall);
  const int row = static_cast<int>(u - static_cast<long long>(p.s) * ph.Nall);
  int j = 0, start = 0;
  while (j + 1 < ph.nseg && row >= start + ph.seg[j].rows) { start += ph.seg[j].rows; ++j; }
  p.seg = j;
  p.row0 = row - start;
  long long end = static_cast<long long>(p.s) * ph.Nall + start + ph.seg[j].rows;   // end of the segment in this k range
  if (end > hi) end = hi;
  p.rows = static_cast<int>(end - u);
  const int k32 = (ph.K + 31) / 32;
  p.kbeg = 32 * static_cast<int>(static_cast<long long>(p.s) * k32 / ph.S);
  const int kend = p.s + 1 == ph.S ? ph.K : 32 * static_cast<int>(static_cast<long long>(p.s + 1) * k32 / ph.S);
  p.klen = kend - p.kbeg;
  return p;
}
// rows of a pass are cut into blocks of at most 32 rows of nearly equal size
__device__ __forceinline__ int blocks_of(int rows) { return (rows + BLOCK_ROWS - 1) / BLOCK_ROWS; }
__device__ __forceinline__ int block_lo(int rows, int nb, int b) { return static_cast<int>(static_cast<long long>(rows) * b / nb); }

// ---- producer ---------------------------------------------------------------------------------------
__device__ void producer(const StreamParams& p, uint32_t ring, uint64_t* full, uint64_t* empty, volatile int* s_abort) {
  const int lane = threadIdx.x & 31;
  uint32_t it = 0;
  bool ok = true;
  for (int pi = 0; pi < p.nph && ok; ++pi) {
    const StreamPhase& ph = p.ph[pi];
    if (ph.kind != 0) continue;
    const Share sh = share_of(ph, blockIdx.x, gridDim.x);
    for (long long u = sh.lo; u < sh.hi && ok;) {
      const Pass ps = pass_at(ph, u, sh.hi);
      const StreamSegment& sg = ph.seg[ps.seg];
      const int nb = blocks_of(ps.rows);
      const int nch = (ps.klen + KC - 1) / KC;
      for (int b = 0; b < nb && ok; ++b) {
        const int r_lo = block_lo(ps.rows, nb, b), r_hi = block_lo(ps.rows, nb, b + 1);
        const char* src = reinterpret_cast<const char*>(sg.W) +
                          (static_cast<long long>(ps.row0 + r_lo + lane) * sg.ldw + ps.kbeg) * 2;
        for (int ch = 0; ch < nch; ++ch, ++it) {
          const int slot = it % NSTAGE;
          // every lane waits; lane 0's verdict is taken by all, so that the warp stays together
          const bool got = ptx::mbar_wait_limit(&empty[slot], ((it / NSTAGE) & 1) ^ 1, s_abort, kWaitLimit);
          if (__shfl_sync(0xffffffffu, got ? 1 : 0, 0) == 0) { ok = false; break; }
          const int bytes = 2 * (ps.klen - ch * KC < KC ? ps.klen - ch * KC : KC);
          if (lane == 0) ptx::mbar_expect_tx(&full[slot], static_cast<uint32_t>((r_hi - r_lo) * bytes));
          __syncwarp();
          if (lane < r_hi - r_lo) {
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                             ring + slot * STAGE_BYTES + lane * ROW_PITCH),
                         "l"(src + ch * (KC * 2)), "r"(bytes), "r"(ptx::smem_u32(&full[slot]))
                         : "memory");
          }
        }
      }
      u += ps.rows;
    }
  }
  if (!ok) {
    // give the copies already issued a bounded chance to land before the CTA exits
    const uint32_t first = it > NSTAGE ? it - NSTAGE : 0;
    for (uint32_t j = first; j < it; ++j) {
      const long long t0 = clock64();
      while (!ptx::mbar_try_wait(&full[j % NSTAGE], (j / NSTAGE) & 1) && clock64() - t0 < kWaitLimit / 8) {}
    }
  }
}

// ---- consumers ----------------------------------------------------------------------------------------
// One value of a phase's activation matrix from its source: the layer input as it is, or the raw sums of an
// earlier phase with their slices added in order, bias, activation.
__device__ __forceinline__ float4 load_sum4(const StreamInPart& in, int t, long long col) {
  const float* base = static_cast<const float*>(in.src) + static_cast<long long>(t) * in.ld + col;
  float4 a = __ldcg(reinterpret_cast<const float4*>(base));
  for (int s = 1; s < in.nslices; ++s) {
    const float4 b = __ldcg(reinterpret_cast<const float4*>(base + s * in.slice_stride));
    a.x += b.x; a.y += b.y; a.z += b.z; a.w += b.w;
  }
  return a;
}

// Activation operand of a pass: columns [c0, c0 + klen) of the phase's activation matrix for tokens 0..7
// (rows beyond T are zero), bf16, token rows X_PITCH bytes apart.  Four columns per thread and step.
__device__ void build_x(const StreamPhase& ph, int T, int act, int c0, int klen, unsigned char* xbuf) {
  const GeluCoef gc = gelu_coef(act);
  const int tid = threadIdx.x;
  const int groups = (klen + 3) >> 2;          // klen is a multiple of 8
  for (int e = tid; e < 8 * groups; e += CTHREADS) {
    const int t = e / groups, q = e - t * groups;
    const int col = c0 + 4 * q;
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (t < T) {
      const StreamInPart& in = (ph.nin > 1 && col >= ph.in[1].col_begin) ? ph.in[1] : ph.in[0];
      const long long sc = in.src_col + (col - in.col_begin);
      if (in.kind == STREAM_IN_BF16) {
        const uint2 raw = __ldg(reinterpret_cast<const uint2*>(static_cast<const __nv_bfloat16*>(in.src) +
                                                               static_cast<long long>(t) * in.ld + sc));
        *reinterpret_cast<uint2*>(xbuf + t * X_PITCH + 8 * q) = raw;
        continue;
      }
      v = load_sum4(in, t, sc);
      if (in.kind == STREAM_IN_GATED) {
        const float4 u = load_sum4(in, t, sc + in.gate_off);
        v.x = silu_fast(v.x) * u.x; v.y = silu_fast(v.y) * u.y; v.z = silu_fast(v.z) * u.z; v.w = silu_fast(v.w) * u.w;
      } else {
        if (in.bias) {
          const float4 b = __ldg(reinterpret_cast<const float4*>(in.bias + (col - in.col_begin)));
          v.x += b.x; v.y += b.y; v.z += b.z; v.w += b.w;
        }
        if (in.kind == STREAM_IN_ACT) {
          v.x = gelu_fast(v.x, gc); v.y = gelu_fast(v.y, gc); v.z = gelu_fast(v.z, gc); v.w = gelu_fast(v.w, gc);
        }
      }
    }
    uint2 o;
    o.x = pack_bf16x2(v.x, v.y);
    o.y = pack_bf16x2(v.z, v.w);
    *reinterpret_cast<uint2*>(xbuf + t * X_PITCH + 8 * q) = o;
  }
}

// All CTAs are resident (cooperative launch).  Called by the consumer threads; count in, the last one opens
// the next generation.  Always arrives; gives up waiting after the limit or when the CTA has already given up.
__device__ void grid_barrier(int* ctrl, volatile int* s_abort) {
  __threadfence();
  cbar();
  if (threadIdx.x == 0) {
    unsigned* count = reinterpret_cast<unsigned*>(ctrl + kBarCount);
    unsigned* genp = reinterpret_cast<unsigned*>(ctrl + kBarGen);
    unsigned gen;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(gen) : "l"(genp) : "memory");
    __threadfence();
    if (atomicAdd(count, 1u) == gridDim.x - 1) {
      atomicExch(count, 0u);
      __threadfence();
      asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(genp), "r"(gen + 1) : "memory");
    } else {
      const long long t0 = clock64();
      unsigned now = gen;
      while (now == gen && !*s_abort) {
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(now) : "l"(genp) : "memory");
        if (now == gen && clock64() - t0 > kWaitLimit) *s_abort = 1;
      }
    }
    __threadfence();
  }
  cbar();
}

__device__ void consumers(const StreamParams& p, unsigned char* smem, uint32_t ring, uint64_t* full, uint64_t* empty,
                          volatile int* s_abort) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, c = lane & 3;
  unsigned char* xbuf = smem + OFF_X;
  const uint32_t xs = ring + OFF_X;
  float* red = reinterpret_cast<float*>(smem + OFF_RED);
  const int kb = warp * 64 + c * 16;     // this lane's 16 bytes inside a 512-byte row segment
  uint32_t it = 0;
  unsigned flushes = 0;
  if (blockIdx.x == 0 && warp == 0) {
    Epilogue e;
    e.guard = p.guard;
    e.guard_hash = p.guard_hash;
    check_blob_guard(e, p.ctrl, KID_DECODE);
  }
  for (int pi = 0; pi < p.nph; ++pi) {
    const StreamPhase& ph = p.ph[pi];
    if (pi > 0) grid_barrier(p.ctrl, s_abort);
    if (ph.kind != 0) {
      // ---- closing reduction: y[t, n] = sum of the slices + bias, for a share of the columns
      const StreamInPart& in = ph.in[0];
      const int q4 = ph.y_cols >> 2;
      const long long total = static_cast<long long>(p.T) * q4;
      for (long long e = static_cast<long long>(blockIdx.x) * CTHREADS + tid; e < total;
           e += static_cast<long long>(gridDim.x) * CTHREADS) {
        const int t = static_cast<int>(e / q4), n = 4 * static_cast<int>(e - static_cast<long long>(t) * q4);
        float4 v = load_sum4(in, t, n);
        if (ph.y_bias) {
          const float4 b = __ldg(reinterpret_cast<const float4*>(ph.y_bias + n));
          v.x += b.x; v.y += b.y; v.z += b.z; v.w += b.w;
        }
        uint2 o;
        o.x = pack_bf16x2(v.x, v.y);
        o.y = pack_bf16x2(v.z, v.w);
        *reinterpret_cast<uint2*>(ph.y + static_cast<long long>(t) * ph.y_ld + n) = o;
      }
      continue;
    }
    const Share sh = share_of(ph, blockIdx.x, gridDim.x);
    int x_c0 = -1, x_len = -1;
    for (long long u = sh.lo; u < sh.hi;) {
      const Pass ps = pass_at(ph, u, sh.hi);
      const StreamSegment& sg = ph.seg[ps.seg];
      // ---- the activation operand of this pass, unless the pass before left exactly it in place
      const int c0 = sg.x_off + ps.kbeg;
      if (c0 != x_c0 || ps.klen != x_len) {
        if (x_c0 >= 0) cbar();               // everyone is done with the operand of the pass before
        build_x(ph, p.T, p.act, c0, ps.klen, xbuf);
        cbar();
        x_c0 = c0; x_len = ps.klen;
      }
      const int nb = blocks_of(ps.rows);
      const int nch = (ps.klen + KC - 1) / KC;
      for (int b = 0; b < nb; ++b) {
        const int r_lo = block_lo(ps.rows, nb, b), r_hi = block_lo(ps.rows, nb, b + 1);
        float acc[2][4];
#pragma unroll
        for (int i = 0; i < 2; ++i)
#pragma unroll
          for (int e = 0; e < 4; ++e) acc[i][e] = 0.f;
        const bool second = r_hi - r_lo > 16;   // the block has rows in its second group of 16
        for (int ch = 0; ch < nch; ++ch, ++it) {
          const int slot = it % NSTAGE;
          const int bytes = 2 * (ps.klen - ch * KC < KC ? ps.klen - ch * KC : KC);
          ptx::mbar_wait_limit(&full[slot], (it / NSTAGE) & 1, s_abort, kWaitLimit);
          if (warp * 64 < bytes) {               // the same for the whole warp (the MMAs need all 32 lanes)
            const uint32_t ws = ring + slot * STAGE_BYTES + g * ROW_PITCH + kb;
            uint4 xb = lds128(xs + g * X_PITCH + ch * (KC * 2) + kb);
            uint4 lo = lds128(ws), hi = lds128(ws + 8 * ROW_PITCH);
            const bool tail = kb >= bytes;       // a row segment ends inside this warp's 64 bytes: nothing was copied
            if (tail) {                          // here, and what the buffers hold must not reach the sums
              xb = make_uint4(0u, 0u, 0u, 0u);
              lo = xb; hi = xb;
            }
            // the same 16 bytes of k from rows g and g + 8 and from token g feed two MMAs as they are: the order
            // in which a contraction visits k is free as long as both operands agree on it
            mma_bf16(acc[0], lo.x, hi.x, lo.y, hi.y, xb.x, xb.y);
            mma_bf16(acc[0], lo.z, hi.z, lo.w, hi.w, xb.z, xb.w);
            if (second) {
              uint4 lo2 = lds128(ws + 16 * ROW_PITCH), hi2 = lds128(ws + 24 * ROW_PITCH);
              if (tail) { lo2 = xb; hi2 = xb; }
              mma_bf16(acc[1], lo2.x, hi2.x, lo2.y, hi2.y, xb.x, xb.y);
              mma_bf16(acc[1], lo2.z, hi2.z, lo2.w, hi2.w, xb.z, xb.w);
            }
          }
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(&empty[slot]);
        }
        // ---- the eight warps' sums over their parts of k, added in warp order
        float* rb = red + (flushes & 1) * (CWARPS * RED_WARP) + warp * RED_WARP;
        ++flushes;
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          rb[(2 * c) * RED_TOK + 16 * i + g] = acc[i][0];
          rb[(2 * c + 1) * RED_TOK + 16 * i + g] = acc[i][1];
          rb[(2 * c) * RED_TOK + 16 * i + g + 8] = acc[i][2];
          rb[(2 * c + 1) * RED_TOK + 16 * i + g + 8] = acc[i][3];
        }
        cbar();
        {
          const int t = tid >> 5, r = tid & 31;
          const float* src = red + ((flushes - 1) & 1) * (CWARPS * RED_WARP) + t * RED_TOK + r;
          float v = 0.f;
#pragma unroll
          for (int w = 0; w < CWARPS; ++w) v += src[w * RED_WARP];
          if (r < r_hi - r_lo && t < p.T) {
            const int n = sg.out_col + ps.row0 + r_lo + r;
            if (ph.out) {
              ph.out[(static_cast<long long>(ps.s) * 8 + t) * ph.out_ld + n] = v;
            } else {
              if (ph.y_bias) v += __ldg(ph.y_bias + n);
              ph.y[static_cast<long long>(t) * ph.y_ld + n] = __float2bfloat16_rn(v);
            }
          }
        }
      }
      u += ps.rows;
    }
  }
}

__global__ void __launch_bounds__(THREADS, 1) decode_stream_kernel(const __grid_constant__ StreamParams p) {
  extern __shared__ __align__(128) unsigned char smem[];
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + OFF_BAR);
  uint64_t* empty = full + NSTAGE;
  volatile int* s_abort = reinterpret_cast<volatile int*>(empty + NSTAGE);
  const uint32_t ring = static_cast<uint32_t>(__cvta_generic_to_shared(smem));
  if (threadIdx.x == 0) {
    for (int i = 0; i < NSTAGE; ++i) {
      ptx::mbar_init(&full[i], 1);
      ptx::mbar_init(&empty[i], CWARPS);
    }
    *s_abort = 0;
    ptx::mbar_fence_init();
  }
  __syncthreads();
  if (threadIdx.x >= CTHREADS) producer(p, ring, full, empty, s_abort);
  else consumers(p, smem, ring, full, empty, s_abort);
  __syncthreads();
  if (threadIdx.x == 0 && *s_abort) record_status(p.ctrl, FFSPLIT_ERR_TIMEOUT, static_cast<int>(blockIdx.x), KID_DECODE);
}

}  // namespace dst

// ---- host side ---------------------------------------------------------------------------------------
ffsplit_status decode_stream_launch(ffsplit_ctx* ctx, const StreamParams& p, double algo_bytes, cudaStream_t st) {
  static bool attr_done[64] = {false};
  static int coop_ok[64] = {0};   // per device: 0 unknown, 1 yes, -1 no
  const int dev = ctx->device;
  if (dev < 0 || dev >= 64) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "device index out of range");
  if (coop_ok[dev] == 0) {
    int v = 0;
    coop_ok[dev] = (cudaDeviceGetAttribute(&v, cudaDevAttrCooperativeLaunch, dev) == cudaSuccess && v) ? 1 : -1;
  }
  if (coop_ok[dev] != 1) return fail(ctx, FFSPLIT_ERR_ARCH, "the device does not support cooperative launches");
  if (!attr_done[dev]) {
    cudaError_t e = cudaFuncSetAttribute(dst::decode_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         dst::SMEM_BYTES);
    if (e != cudaSuccess) return check_cuda(ctx, e, "cudaFuncSetAttribute(decode_stream_kernel)");
    attr_done[dev] = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(ctx->num_sms);
  cfg.blockDim = dim3(dst::THREADS);
  cfg.dynamicSmemBytes = dst::SMEM_BYTES;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;
  attr[0].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const int ph = prof_open(ctx, PROF_DECODE, algo_bytes, st);
  const cudaError_t e = cudaLaunchKernelEx(&cfg, dst::decode_stream_kernel, p);
  prof_close(ctx, ph, st);
  ctx->launches++;
  return check_cuda(ctx, e, "decode_stream_kernel launch");
}

}  // namespace ffsp
