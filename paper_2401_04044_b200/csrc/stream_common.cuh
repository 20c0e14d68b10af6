// Pieces shared by the persistent few-token kernels (decode_stream.cu: bf16 weights; decode_quant.cu: 8- and
// 3-bit weights): the CTA's shape, the walk over a CTA's share of a phase, the producers' row copies and the
// grid-wide barrier.
#pragma once

#include "decode_common.cuh"
#include "decode_stream.h"
#include "internal.h"
#include "ptx.cuh"

namespace ffsp {
namespace dst {

using namespace dec;

constexpr int CWARPS = 8;                                // consumer warps
constexpr int CTHREADS = 32 * CWARPS;
constexpr int PWARPS = 4;                                // producer warps: stage i is filled by warp i mod 4
constexpr int THREADS = CTHREADS + 32 * PWARPS;
constexpr int BLOCK_ROWS = 32;                           // weight rows per stage, at most
constexpr int STAGE_BYTES = 32 * 576;                    // 18432 (kStreamStageBytes of the bf16 plan)
constexpr int NSTAGE = 9;
constexpr int X_BYTES = 41472;                           // activation operand of a pass (kStreamXBytes of the bf16 plan)
constexpr int RED_TOK = 36;                              // floats between token rows of a warp's partial block
constexpr int RED_WARP = 8 * RED_TOK;
constexpr int RED_BYTES = 2 * CWARPS * RED_WARP * 4;     // two buffers, used alternately
constexpr int OFF_X = NSTAGE * STAGE_BYTES;
constexpr int OFF_RED = OFF_X + X_BYTES;
constexpr int OFF_BAR = OFF_RED + RED_BYTES;
constexpr int SMEM_BYTES = OFF_BAR + 256;
static_assert(SMEM_BYTES <= 232448, "shared memory plan");
constexpr int kBarTicket = 18;                           // words 18-19 of the control block: the grid barrier's 64-bit ticket counter
constexpr long long kWaitLimit = 2000000000ll;           // SM clocks (about a second)

__device__ __forceinline__ void cbar() { asm volatile("bar.sync 1, %0;" ::"n"(CTHREADS) : "memory"); }

// ---- the walk over a CTA's share of one phase, taken identically by the producers and the consumers -----
// (32-bit arithmetic: the host checks S * Nall * (grid + 1) < 2^31 when it plans a phase)
struct Pass {
  int seg, s;          // segment, k range
  int row0, rows;      // rows [row0, row0 + rows) of the segment
  int kbeg, klen;      // k range in elements
};
struct Share { unsigned lo, hi; };   // units [lo, hi) of the phase: unit = s * Nall + row

template <class PH>
__device__ __forceinline__ Share share_of(const PH& ph, unsigned cta, unsigned ncta) {
  const unsigned U = static_cast<unsigned>(ph.S) * ph.Nall;
  Share sh;
  sh.lo = U * cta / ncta;
  sh.hi = U * (cta + 1) / ncta;
  return sh;
}
// the pass that starts at unit u (u < hi)
// K is cut into S ranges on multiples of PH::kQuantum elements (32 for bf16 rows, a group of 128 for quantised ones)
template <class PH>
__device__ __forceinline__ Pass pass_at(const PH& ph, unsigned u, unsigned hi) {
  Pass p;
  const unsigned nall = ph.Nall;
  p.s = static_cast<int>(u / nall);
  const int row = static_cast<int>(u - p.s * nall);
  int j = 0, start = 0;
  while (j + 1 < ph.nseg && row >= start + ph.seg[j].rows) { start += ph.seg[j].rows; ++j; }
  p.seg = j;
  p.row0 = row - start;
  unsigned end = p.s * nall + start + ph.seg[j].rows;   // end of the segment in this k range
  if (end > hi) end = hi;
  p.rows = static_cast<int>(end - u);
  constexpr unsigned Q = PH::kQuantum;
  const unsigned kq = (ph.K + Q - 1) / Q;
  p.kbeg = static_cast<int>(Q * (p.s * kq / ph.S));
  const int kend = p.s + 1 == ph.S ? ph.K : static_cast<int>(Q * ((p.s + 1) * kq / ph.S));
  p.klen = kend - p.kbeg;
  return p;
}
// rows of a pass are cut into blocks of at most 32 rows of nearly equal size
__device__ __forceinline__ int blocks_of(int rows) { return (rows + BLOCK_ROWS - 1) / BLOCK_ROWS; }
__device__ __forceinline__ int block_lo(int rows, int nb, int b) { return rows * b / nb; }

// 16 bytes per lane of each of `nr` rows (src_step bytes apart; a lane outside the k range copies nothing and its
// 16 bytes are zero filled)
__device__ __forceinline__ void issue_rows(uint32_t dst, int dst_pitch, const char* src, long long src_step, int nr,
                                           bool valid) {
  int r = 0;
#pragma unroll 1
  for (; r + 4 <= nr; r += 4) {
    cp_async16(dst, src, valid);
    cp_async16(dst + dst_pitch, src + src_step, valid);
    cp_async16(dst + 2 * dst_pitch, src + 2 * src_step, valid);
    cp_async16(dst + 3 * dst_pitch, src + 3 * src_step, valid);
    dst += 4 * dst_pitch;
    src += 4 * src_step;
  }
  for (; r < nr; ++r, dst += dst_pitch, src += src_step) cp_async16(dst, src, valid);
}

// All CTAs are resident (cooperative launch).  Called by the consumer threads.  One 64-bit counter that only
// ever grows: an arrival takes a ticket v, and the barrier it belongs to is complete when the counter reaches
// the next multiple of the grid size above v (every barrier receives exactly one arrival per CTA, so the
// counter stays aligned from launch to launch; a run that gave up leaves it misaligned, and ffsplit_poll()
// clears the control block when it reports that).  The arrival is a release at GPU scope, ordered after the
// whole CTA's writes by the CTA barrier before it, and the wait ends with an acquire: no separate fences, one
// atomic round trip on the critical path.  Always arrives; gives up waiting after the limit or when the CTA has
// already given up.
__device__ __forceinline__ void grid_barrier(int* ctrl, volatile int* s_abort) {
  cbar();
  if (threadIdx.x == 0) {
    unsigned long long* ctr = reinterpret_cast<unsigned long long*>(ctrl + kBarTicket);
    unsigned long long v;
    asm volatile("atom.add.acq_rel.gpu.global.u64 %0, [%1], 1;" : "=l"(v) : "l"(ctr) : "memory");
    const unsigned long long target = (v / gridDim.x + 1ull) * gridDim.x;
    if (v + 1ull != target) {
      const long long t0 = clock64();
      while (!*s_abort) {
        unsigned long long now;
        asm volatile("ld.acquire.gpu.global.u64 %0, [%1];" : "=l"(now) : "l"(ctr) : "memory");
        if (now >= target) break;
        if (clock64() - t0 > kWaitLimit) *s_abort = 1;
      }
    }
  }
  cbar();
}

// Four columns of a phase's activation matrix from raw sums of an earlier phase: the slices added in order.
// The loads of up to four slices are in flight together.
__device__ __forceinline__ float4 load_sum4(const StreamInPart& in, int t, long long col) {
  const float* base = static_cast<const float*>(in.src) + static_cast<long long>(t) * in.ld + col;
  float4 a = __ldcg(reinterpret_cast<const float4*>(base));
  for (int s0 = 1; s0 < in.nslices; s0 += 4) {
    float4 b[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      b[j] = make_float4(0.f, 0.f, 0.f, 0.f);
      if (s0 + j < in.nslices) b[j] = __ldcg(reinterpret_cast<const float4*>(base + (s0 + j) * in.slice_stride));
    }
#pragma unroll
    for (int j = 0; j < 4; ++j)
      if (s0 + j < in.nslices) { a.x += b[j].x; a.y += b[j].y; a.z += b[j].z; a.w += b[j].w; }
  }
  return a;
}

}  // namespace dst
}  // namespace ffsp
