// Few-token (decode) split forward for 1..8 tokens: ONE persistent kernel per layer whose weight stream never
// waits for the dependencies between the stages of Eq. 2.
//
// With a handful of tokens every stage of Eq. 2 is a skinny product C[t, n] = sum_k A[t, k] W[n, k] whose
// cost is reading W once, and a split layer is a chain of four of them (stage 1, the two halves of the light
// chain, stage 3) of a few megabytes each.  What bounds such a layer is not bandwidth but the hand-over
// between dependent products.  This kernel is built around two facts:
//
//  * The weights do not depend on the activations.  Producer warps walk the CTA's share of ALL phases of the
//    layer and copy it into a ring of shared-memory stages with asynchronous copies (cp.async, 16 bytes per
//    lane: one warp-wide instruction moves 512 contiguous bytes of one weight row; completion is counted on
//    the stage's mbarrier).  They never wait for a grid barrier: while the consumers wait for the previous
//    phase to finish everywhere, the next phase's weights are already landing, and HBM stays busy as long as
//    the ring has a free stage.  (Bulk copies, cp.async.bulk, of one 512-byte row segment each measured
//    1.9 TB/s on this path: about 77 clocks per copy whatever its size.)
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

#include "decode_stream.h"
#include "epilogue.cuh"
#include "stream_common.cuh"

namespace ffsp {
namespace dst {

static_assert(STAGE_BYTES == kStreamStageBytes && X_BYTES == kStreamXBytes, "the host's plan and the kernel agree");

// ---- producers -------------------------------------------------------------------------------------
__device__ void producer(const StreamParams& p, uint32_t ring, uint64_t* full, uint64_t* empty, volatile int* s_abort,
                         int pw) {
  const int lane = threadIdx.x & 31;
  if (pw == 0 && blockIdx.x == 0) {
    Epilogue e;
    e.guard = p.guard;
    e.guard_hash = p.guard_hash;
    check_blob_guard(e, p.ctrl, KID_DECODE);
  }
  uint32_t it = 0;
  bool ok = true;
  for (int pi = 0; pi < p.nph && ok; ++pi) {
    const StreamPhase& ph = p.ph[pi];
    if (ph.kind != 0) continue;
    const Share sh = share_of(ph, blockIdx.x, gridDim.x);
    for (unsigned u = sh.lo; u < sh.hi && ok;) {
      const Pass ps = pass_at(ph, u, sh.hi);
      const StreamSegment& sg = ph.seg[ps.seg];
      const int nb = blocks_of(ps.rows);
      const long long pitch = sg.ldw * 2;
      for (int b = 0; b < nb && ok; ++b) {
        const int r_lo = block_lo(ps.rows, nb, b), r_hi = block_lo(ps.rows, nb, b + 1);
        const int sub = stream_stage_sub(r_hi - r_lo);
        const int chunk = 512 * sub, row_pitch = chunk + 64;
        const int nch = (2 * ps.klen + chunk - 1) / chunk;
        const char* base = reinterpret_cast<const char*>(sg.W) +
                           (static_cast<long long>(ps.row0 + r_lo) * sg.ldw + ps.kbeg) * 2 + lane * 16;
        for (int ch = 0; ch < nch; ++ch, ++it) {
          if (static_cast<int>(it % PWARPS) != pw) continue;
          const int slot = it % NSTAGE;
          // every lane waits; lane 0's verdict is taken by all, so that the warp stays together
          const bool got = ptx::mbar_wait_limit(&empty[slot], ((it / NSTAGE) & 1) ^ 1, s_abort, kWaitLimit);
          if (__shfl_sync(0xffffffffu, got ? 1 : 0, 0) == 0) { ok = false; break; }
          const int bytes = 2 * ps.klen - ch * chunk < chunk ? 2 * ps.klen - ch * chunk : chunk;   // multiple of 16
          const char* src0 = base + static_cast<long long>(ch) * chunk;
          const uint32_t dst0 = ring + slot * STAGE_BYTES + lane * 16;
          for (int j = 0; j < sub && j * 512 < bytes; ++j) {
            // one 512-byte piece of every row of the block: a warp-wide copy per row, four rows per turn
            const bool valid = j * 512 + lane * 16 < bytes;
            issue_rows(dst0 + j * 512, row_pitch, valid ? src0 + j * 512 : reinterpret_cast<const char*>(sg.W),
                       valid ? pitch : 0, r_hi - r_lo, valid);
          }
          asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(ptx::smem_u32(&full[slot])) : "memory");
        }
      }
      u += ps.rows;
    }
  }
  // on every way out: this thread's copies have landed before the CTA may exit
  asm volatile("cp.async.wait_all;" ::: "memory");
}

// ---- consumers ----------------------------------------------------------------------------------------
// Activation operand of a pass: columns [c0, c0 + klen) of the phase's activation matrix for tokens
// 0 .. x_rows - 1 (rows beyond T are zero), bf16, token rows X_PITCH bytes apart.  Four columns per thread and
// element.  Values that an earlier phase finished (or the layer input) are copied asynchronously as they are;
// raw sums are added slice by slice, biased, activated and rounded here.  A thread takes eight elements per turn:
// the loads of a turn are all issued before the first is used, and the loop body has no branch that depends on
// the element (an element with nothing to load reads a valid address and is masked afterwards) -- with branches
// between them the loads went out one latency at a time.
// One part of the operand: columns [a0, a1) of the activation matrix, all of one kind.
template <int KIND>
__device__ __forceinline__ void build_part(const StreamInPart& in, int T, const GeluCoef& gc, int c0, int a0, int a1,
                                           unsigned char* xbuf, uint32_t xs0, int x_rows, int X_PITCH) {
  const int tid = threadIdx.x;
  const int groups = (a1 - a0) >> 2;           // part boundaries and k ranges are multiples of 8 columns
  const int total = x_rows * groups;
  const int qoff = (a0 - c0) >> 2;             // where the part starts inside the operand, in 4-column elements
  if (KIND == STREAM_IN_BF16) {
    for (int e = tid; e < total; e += CTHREADS) {
      const int t = e / groups, q = e - t * groups;
      if (t < T) {
        const __nv_bfloat16* src = static_cast<const __nv_bfloat16*>(in.src) + static_cast<long long>(t) * in.ld +
                                   in.src_col + (a0 - in.col_begin) + 4 * q;
        asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(xs0 + t * X_PITCH + 8 * (qoff + q)), "l"(src) : "memory");
      } else {
        *reinterpret_cast<uint2*>(xbuf + t * X_PITCH + 8 * (qoff + q)) = make_uint2(0u, 0u);
      }
    }
    return;
  }
  constexpr int B = 8;
  for (int e0 = tid; e0 < total; e0 += B * CTHREADS) {
    float4 v[B], u[B];
    bool live[B];
#pragma unroll
    for (int j = 0; j < B; ++j) {
      const int e = e0 + j * CTHREADS;
      const int ee = e < total ? e : tid % total;   // a valid element to read in any case
      const int t = ee / groups, q = ee - t * groups;
      live[j] = e < total && t < T;
      const long long at = static_cast<long long>(live[j] ? t : 0) * in.ld + in.src_col + (a0 - in.col_begin) + 4 * q;
      const float* base = static_cast<const float*>(in.src) + at;
      v[j] = __ldcg(reinterpret_cast<const float4*>(base));
      if (KIND == STREAM_IN_GATED) u[j] = __ldcg(reinterpret_cast<const float4*>(base + in.gate_off));
      else u[j] = in.bias ? __ldg(reinterpret_cast<const float4*>(in.bias + (a0 - in.col_begin) + 4 * q))
                          : make_float4(0.f, 0.f, 0.f, 0.f);
    }
    // further k ranges of the phase before: slice by slice, the eight elements' loads together
    for (int s = 1; s < in.nslices; ++s) {
      float4 b[B], bu[B];
#pragma unroll
      for (int j = 0; j < B; ++j) {
        const int e = e0 + j * CTHREADS;
        const int ee = e < total ? e : tid % total;
        const int t = ee / groups, q = ee - t * groups;
        const long long at = static_cast<long long>(live[j] ? t : 0) * in.ld + in.src_col + (a0 - in.col_begin) + 4 * q;
        const float* base = static_cast<const float*>(in.src) + s * in.slice_stride + at;
        b[j] = __ldcg(reinterpret_cast<const float4*>(base));
        if (KIND == STREAM_IN_GATED) bu[j] = __ldcg(reinterpret_cast<const float4*>(base + in.gate_off));
      }
#pragma unroll
      for (int j = 0; j < B; ++j) {
        v[j].x += b[j].x; v[j].y += b[j].y; v[j].z += b[j].z; v[j].w += b[j].w;
        if (KIND == STREAM_IN_GATED) { u[j].x += bu[j].x; u[j].y += bu[j].y; u[j].z += bu[j].z; u[j].w += bu[j].w; }
      }
    }
#pragma unroll
    for (int j = 0; j < B; ++j) {
      const int e = e0 + j * CTHREADS;
      if (e >= total) continue;
      const int t = e / groups, q = e - t * groups;
      float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
      if (live[j]) {
        if (KIND == STREAM_IN_GATED) {
          a.x = silu_fast(v[j].x) * u[j].x; a.y = silu_fast(v[j].y) * u[j].y;
          a.z = silu_fast(v[j].z) * u[j].z; a.w = silu_fast(v[j].w) * u[j].w;
        } else {
          a.x = v[j].x + u[j].x; a.y = v[j].y + u[j].y; a.z = v[j].z + u[j].z; a.w = v[j].w + u[j].w;
          if (KIND == STREAM_IN_ACT) {
            a.x = gelu_fast(a.x, gc); a.y = gelu_fast(a.y, gc); a.z = gelu_fast(a.z, gc); a.w = gelu_fast(a.w, gc);
          }
        }
      }
      uint2 o;
      o.x = pack_bf16x2(a.x, a.y);
      o.y = pack_bf16x2(a.z, a.w);
      *reinterpret_cast<uint2*>(xbuf + t * X_PITCH + 8 * (qoff + q)) = o;
    }
  }
}

__device__ void build_x(const StreamPhase& ph, int T, int act, int c0, int klen, unsigned char* xbuf, uint32_t xs0,
                        int x_rows, int X_PITCH) {
  const GeluCoef gc = gelu_coef(act);
  for (int pi = 0; pi < ph.nin; ++pi) {
    const StreamInPart& in = ph.in[pi];
    const int a0 = in.col_begin > c0 ? in.col_begin : c0;
    const int a1 = in.col_end < c0 + klen ? in.col_end : c0 + klen;
    if (a1 <= a0) continue;
    if (in.kind == STREAM_IN_BF16) build_part<STREAM_IN_BF16>(in, T, gc, c0, a0, a1, xbuf, xs0, x_rows, X_PITCH);
    else if (in.kind == STREAM_IN_GATED) build_part<STREAM_IN_GATED>(in, T, gc, c0, a0, a1, xbuf, xs0, x_rows, X_PITCH);
    else if (in.kind == STREAM_IN_ACT) build_part<STREAM_IN_ACT>(in, T, gc, c0, a0, a1, xbuf, xs0, x_rows, X_PITCH);
    else build_part<STREAM_IN_LINEAR>(in, T, gc, c0, a0, a1, xbuf, xs0, x_rows, X_PITCH);
  }
  asm volatile("cp.async.wait_all;" ::: "memory");
}

__device__ void consumers(const StreamParams& p, unsigned char* smem, uint32_t ring, uint64_t* full, uint64_t* empty,
                          volatile int* s_abort) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, c = lane & 3;
  unsigned char* xbuf = smem + OFF_X;
  const int X_PITCH = p.x_pitch;
  const bool my_token = g < p.x_rows;      // token rows beyond the operand's are zero
  const uint32_t xs = ring + OFF_X + (my_token ? g * X_PITCH : 0);
  float* red = reinterpret_cast<float*>(smem + OFF_RED);
  const int kb = warp * 64 + c * 16;     // this lane's 16 bytes inside a 512-byte row segment
  const GeluCoef gc = gelu_coef(p.act);
  uint32_t it = 0;
  unsigned flushes = 0;
  for (int pi = 0; pi < p.nph; ++pi) {
    const StreamPhase& ph = p.ph[pi];
    // this CTA's share and its first pass: arithmetic only, done before the wait for the phase before
    Share sh;
    sh.lo = sh.hi = 0;
    Pass ps;
    if (ph.kind == 0) {
      sh = share_of(ph, blockIdx.x, gridDim.x);
      if (sh.lo < sh.hi) ps = pass_at(ph, sh.lo, sh.hi);
    }
    if (pi > 0) grid_barrier(p.ctrl, s_abort);
    if (ph.kind != 0) {
      // ---- closing reduction: y[t, n] = sum of the slices + bias, for a share of the columns
      const StreamInPart& in = ph.in[0];
      const int q4 = ph.y_cols >> 2;
      const int total = p.T * q4;
      for (int e = blockIdx.x * CTHREADS + tid; e < total; e += gridDim.x * CTHREADS) {
        const int t = e / q4, n = 4 * (e - t * q4);
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
    int x_c0 = -1, x_len = -1;
    for (unsigned u = sh.lo; u < sh.hi;) {
      const StreamSegment& sg = ph.seg[ps.seg];
      // ---- the activation operand of this pass, unless the pass before left exactly it in place
      const int c0 = sg.x_off + ps.kbeg;
      if (c0 != x_c0 || ps.klen != x_len) {
        if (x_c0 >= 0) cbar();               // everyone is done with the operand of the pass before
        build_x(ph, p.T, p.act, c0, ps.klen, xbuf, ring + OFF_X, p.x_rows, X_PITCH);
        cbar();
        x_c0 = c0; x_len = ps.klen;
      }
      const int nb = blocks_of(ps.rows);
      for (int b = 0; b < nb; ++b) {
        const int r_lo = block_lo(ps.rows, nb, b), r_hi = block_lo(ps.rows, nb, b + 1);
        const int sub = stream_stage_sub(r_hi - r_lo);
        const int chunk = 512 * sub, row_pitch = chunk + 64;
        const int nch = (2 * ps.klen + chunk - 1) / chunk;
        // Four accumulator sets per group of 16 rows, used in turn: a chain of MMAs into one accumulator runs at
        // the instruction's latency (about a hundred clocks each), and a stage of few rows and long chunks is a
        // chain of up to sixteen.
        float acc[2][4][4];
#pragma unroll
        for (int i = 0; i < 2; ++i)
#pragma unroll
          for (int a = 0; a < 4; ++a)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[i][a][e] = 0.f;
        const bool second = r_hi - r_lo > 16;   // the block has rows in its second group of 16
        // what the flush of this block will add to this thread's output value: on its way while the weights stream
        float fbias = 0.f;
        {
          const int t = tid >> 5, r = tid & 31;
          if (r < r_hi - r_lo && t < p.T && !ph.out) {
            const int nl = ps.row0 + r_lo + r;
            if (ph.outb) { if (sg.fin_bias) fbias = __ldg(sg.fin_bias + nl); }
            else if (ph.y_bias) fbias = __ldg(ph.y_bias + sg.out_col + nl);
          }
        }
        for (int ch = 0; ch < nch; ++ch, ++it) {
          const int slot = it % NSTAGE;
          const int bytes = 2 * ps.klen - ch * chunk < chunk ? 2 * ps.klen - ch * chunk : chunk;
          ptx::mbar_wait_limit(&full[slot], (it / NSTAGE) & 1, s_abort, kWaitLimit);
          // rows beyond the block's last one were not copied: read row 0 instead (their sums are never stored)
          const int nr = r_hi - r_lo;
          const uint32_t st0 = ring + slot * STAGE_BYTES + kb;
          const uint32_t ws0 = st0 + (g < nr ? g : 0) * row_pitch, ws1 = st0 + (g + 8 < nr ? g + 8 : 0) * row_pitch;
          const uint32_t ws2 = st0 + (g + 16 < nr ? g + 16 : 0) * row_pitch, ws3 = st0 + (g + 24 < nr ? g + 24 : 0) * row_pitch;
          const uint32_t xs0 = xs + ch * chunk + kb;
#pragma unroll 2
          for (int j = 0; j < sub; ++j) {
            if (j * 512 + warp * 64 >= bytes) break;     // the same for the whole warp (the MMAs need all 32 lanes)
            uint4 xb = lds128(xs0 + j * 512);
            uint4 lo = lds128(ws0 + j * 512), hi = lds128(ws1 + j * 512);
            const bool tail = j * 512 + kb >= bytes;     // a row segment ends inside this warp's 64 bytes: nothing was
            if (tail || !my_token) xb = make_uint4(0u, 0u, 0u, 0u);   // copied here, and what the buffers hold must not
            if (tail) {                                               // reach the sums
              lo = make_uint4(0u, 0u, 0u, 0u);
              hi = lo;
            }
            // the same 16 bytes of k from rows g and g + 8 and from token g feed two MMAs as they are: the order
            // in which a contraction visits k is free as long as both operands agree on it
            float* a0 = acc[0][(2 * j) & 3];
            float* a1 = acc[0][(2 * j + 1) & 3];
            mma_bf16(a0, lo.x, hi.x, lo.y, hi.y, xb.x, xb.y);
            mma_bf16(a1, lo.z, hi.z, lo.w, hi.w, xb.z, xb.w);
            if (second) {
              uint4 lo2 = lds128(ws2 + j * 512), hi2 = lds128(ws3 + j * 512);
              if (tail) { lo2 = lo; hi2 = lo; }
              mma_bf16(acc[1][(2 * j) & 3], lo2.x, hi2.x, lo2.y, hi2.y, xb.x, xb.y);
              mma_bf16(acc[1][(2 * j + 1) & 3], lo2.z, hi2.z, lo2.w, hi2.w, xb.z, xb.w);
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
          float v4[4];
#pragma unroll
          for (int e = 0; e < 4; ++e) v4[e] = (acc[i][0][e] + acc[i][1][e]) + (acc[i][2][e] + acc[i][3][e]);
          rb[(2 * c) * RED_TOK + 16 * i + g] = v4[0];
          rb[(2 * c + 1) * RED_TOK + 16 * i + g] = v4[1];
          rb[(2 * c) * RED_TOK + 16 * i + g + 8] = v4[2];
          rb[(2 * c + 1) * RED_TOK + 16 * i + g + 8] = v4[3];
        }
        cbar();
        {
          const int t = tid >> 5, r = tid & 31;
          const float* src = red + ((flushes - 1) & 1) * (CWARPS * RED_WARP) + t * RED_TOK + r;
          float v = 0.f;
#pragma unroll
          for (int w = 0; w < CWARPS; ++w) v += src[w * RED_WARP];
          if (r < r_hi - r_lo && t < p.T) {
            const int nl = ps.row0 + r_lo + r;             // row inside the segment
            const int n = sg.out_col + nl;
            if (ph.out) {
              ph.out[(static_cast<long long>(ps.s) * 8 + t) * ph.out_ld + n] = v;
            } else if (ph.outb) {
              v += fbias;
              if (sg.fin_kind == STREAM_IN_ACT) v = gelu_fast(v, gc);
              ph.outb[static_cast<long long>(t) * ph.out_ld + n] = __float2bfloat16_rn(v);
            } else {
              ph.y[static_cast<long long>(t) * ph.y_ld + n] = __float2bfloat16_rn(v + fbias);
            }
          }
        }
      }
      u += ps.rows;
      if (u < sh.hi) ps = pass_at(ph, u, sh.hi);
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
      ptx::mbar_init(&full[i], 32);          // every lane of the warp that fills the stage
      ptx::mbar_init(&empty[i], CWARPS);
    }
    *s_abort = 0;
    ptx::mbar_fence_init();
  }
  __syncthreads();
  if (threadIdx.x >= CTHREADS) producer(p, ring, full, empty, s_abort, (threadIdx.x - CTHREADS) >> 5);
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
