// Few-token forward of the QUANTISED split layer (Section 5.2: heavy-hitter neurons 8 bits, everything else
// 3 bits, group size 128): Y = sigma(X U1~ + b1[h2]) V1~ + sigma(X U2~ + b1[light]) V2~ + b2 for 1..8 tokens, the
// weights dequantised in registers inside the weight-streaming kernel.
//
// Same machinery as decode_stream.cu -- one persistent cooperative kernel per layer, producer warps that copy
// every phase's packed rows into a ring of shared-memory stages ahead of the dependency between the phases,
// consumer warps that split the k range of a stage between them -- with three differences:
//
//  * A weight row is a run of groups, each 128 codes followed by its (scale, lo) pair (quant.h); a stage holds
//    an even number of whole groups of up to 32 rows, and a consumer warp takes whole groups.
//  * Codes never become weights.  A code q goes into the low mantissa bits of the fp16 value 1024 + q (one
//    shift and one mask per pair of 3-bit codes, one byte permute per pair of 8-bit codes), the tensor-core MMA
//    multiplies those exact small integers with the fp16 activations, and the group's affine map is applied to
//    the group's sum:  sum_k (lo + q_k scale) x_k = scale * (sum_k (1024 + q_k) x_k) + (lo - 1024 scale) * sum_k x_k.
//    The activation sums sum_k x_k per token and group are taken once when the activation operand is staged.
//  * Rows of the 8-bit and the 3-bit part have different lengths in bytes, so a phase's rows are dealt to the
//    CTAs by weight: a row counts as many units as its group has 8-byte words (17 or 7), and a row belongs to
//    the CTA whose share holds its first unit.
//
// Phases: (1) z = X [U1~ | U2~] (SwiGLU: gate and up) raw; (2a) the heavy part a_H V1~ and (2b), without a
// barrier in between, the light part a_L V2~, each as raw slices per k range; (3) the closing reduction adds all
// slices and b2.  Activations are applied by whoever reads the raw sums.  All sums are taken in a fixed order.
#include <cstring>

#include <cuda_fp16.h>

#include "decode_stream.h"
#include "epilogue.cuh"
#include "quant.h"
#include "quant_plan.h"
#include "stream_common.cuh"

namespace ffsp {
namespace dqt {

using namespace dst;

constexpr int XSUM_BYTES = 160 * 8 * 4;                  // activation sums: up to 160 groups x 8 tokens
constexpr int OFF_XSUM = OFF_X + X_BYTES;
constexpr int OFF_RED_Q = OFF_XSUM + XSUM_BYTES;
constexpr int OFF_BAR_Q = OFF_RED_Q + RED_BYTES;
constexpr int SMEM_BYTES_Q = OFF_BAR_Q + 256;
static_assert(SMEM_BYTES_Q <= 232448, "shared memory plan");
static_assert(X_BYTES == kQuantXBytes, "the host's plan and the kernel agree");

// ---- the weighted walk over a CTA's share of a phase ----------------------------------------------------
struct QPass {
  int seg, s;
  int row0, rows;
  int gbeg, glen;      // group range of this k range
};
__device__ __forceinline__ unsigned seg_weight(const QSegment& sg) { return sg.bits == 8 ? 17u : 7u; }
// units of one k range
__device__ __forceinline__ unsigned units_per_split(const QPhase& ph) {
  unsigned u = 0;
  for (int j = 0; j < ph.nseg; ++j) u += static_cast<unsigned>(ph.seg[j].rows) * seg_weight(ph.seg[j]);
  return u;
}
// The pass that starts at unit u: rows of one segment in one k range whose first unit lies in [u, hi).  `next`
// receives the unit where the following pass starts.  A pass may come out empty (rows == 0).
__device__ __forceinline__ QPass qpass_at(const QPhase& ph, unsigned uw, unsigned u, unsigned hi, unsigned* next) {
  QPass p;
  p.s = static_cast<int>(u / uw);
  const unsigned v = u - p.s * uw;
  int j = 0;
  unsigned start = 0;
  while (j + 1 < ph.nseg && v >= start + static_cast<unsigned>(ph.seg[j].rows) * seg_weight(ph.seg[j])) {
    start += static_cast<unsigned>(ph.seg[j].rows) * seg_weight(ph.seg[j]);
    ++j;
  }
  const unsigned w = seg_weight(ph.seg[j]);
  unsigned end = p.s * uw + start + static_cast<unsigned>(ph.seg[j].rows) * w;   // end of the segment in this k range
  if (end > hi) end = hi;
  const unsigned r0 = (v - start + w - 1) / w, r1 = (end - p.s * uw - start + w - 1) / w;
  p.seg = j;
  p.row0 = static_cast<int>(r0);
  p.rows = r1 > r0 ? static_cast<int>(r1 - r0) : 0;
  const unsigned g2 = static_cast<unsigned>(ph.G) / 2;     // k ranges start on even group numbers
  p.gbeg = 2 * static_cast<int>(p.s * g2 / ph.S);
  const int gend = p.s + 1 == ph.S ? ph.G : 2 * static_cast<int>((p.s + 1) * g2 / ph.S);
  p.glen = gend - p.gbeg;
  *next = end;
  return p;
}
// groups per stage for a block of `rows` rows: even, as many as fit; and the bytes between the rows of a stage,
// chosen so that the lanes' code loads spread over the banks (3 bits: pitch = 48 mod 128; 8 bits: 16 mod 128)
__device__ __forceinline__ void stage_shape(int rows, int bits, int* gch, int* pitch) {
  const int gb = bits == 8 ? qnt::kGroupBytes8 : qnt::kGroupBytes3;
  const int want = bits == 8 ? 16 : 48;   // (the pitch must stay a multiple of 16 for the copies: the 8-bit rows keep a two-way conflict)
  int g = (STAGE_BYTES / rows - 127) / gb;
  g = g / 2 * 2;
  if (g < 2) g = 2;
  if (g > 40) g = 40;
  int p = g * gb;
  p += ((want - p) % 128 + 128) % 128;
  *gch = g;
  *pitch = p;
}

// ---- producers -------------------------------------------------------------------------------------
__device__ void producer(const QParams& p, uint32_t ring, uint64_t* full, uint64_t* empty, volatile int* s_abort, int pw) {
  const int lane = threadIdx.x & 31;
  if (pw == 0 && blockIdx.x == 0) {
    Epilogue e;
    e.guard = p.guard;
    e.guard_hash = p.guard_hash;
    check_blob_guard(e, p.ctrl, KID_QUANT);
  }
  uint32_t it = 0;
  bool ok = true;
  for (int pi = 0; pi < p.nph && ok; ++pi) {
    const QPhase& ph = p.ph[pi];
    if (ph.kind != 0) continue;
    const unsigned uw = units_per_split(ph), U = uw * ph.S;
    const unsigned lo = U * blockIdx.x / gridDim.x, hi = U * (blockIdx.x + 1) / gridDim.x;
    for (unsigned u = lo; u < hi && ok;) {
      unsigned next;
      const QPass ps = qpass_at(ph, uw, u, hi, &next);
      u = next;
      if (ps.rows == 0) continue;
      const QSegment& sg = ph.seg[ps.seg];
      const int gb = sg.bits == 8 ? qnt::kGroupBytes8 : qnt::kGroupBytes3;
      const int nb = blocks_of(ps.rows);
      for (int b = 0; b < nb && ok; ++b) {
        const int r_lo = block_lo(ps.rows, nb, b), r_hi = block_lo(ps.rows, nb, b + 1);
        int gch, row_pitch;
        stage_shape(r_hi - r_lo, sg.bits, &gch, &row_pitch);
        const int nch = (ps.glen + gch - 1) / gch;
        const char* base = reinterpret_cast<const char*>(sg.W) + static_cast<long long>(ps.row0 + r_lo) * sg.row_bytes +
                           static_cast<long long>(ps.gbeg) * gb + lane * 16;
        for (int ch = 0; ch < nch; ++ch, ++it) {
          if (static_cast<int>(it % PWARPS) != pw) continue;
          const int slot = it % NSTAGE;
          const bool got = ptx::mbar_wait_limit(&empty[slot], ((it / NSTAGE) & 1) ^ 1, s_abort, kWaitLimit);
          if (__shfl_sync(0xffffffffu, got ? 1 : 0, 0) == 0) { ok = false; break; }
          const int gcnt = ps.glen - ch * gch < gch ? ps.glen - ch * gch : gch;     // even
          const int bytes = gcnt * gb;                                             // a multiple of 16
          const char* src0 = base + static_cast<long long>(ch) * gch * gb;
          const uint32_t dst0 = ring + slot * STAGE_BYTES + lane * 16;
          // a lane past the end of the row's groups copies nothing at all: the rows of a stage lie closer together
          // than the next multiple of 512 bytes, and a zero fill there would land in the next row
          for (int j = 0; j * 512 < bytes; ++j)
            if (j * 512 + lane * 16 < bytes) issue_rows(dst0 + j * 512, row_pitch, src0 + j * 512, sg.row_bytes, r_hi - r_lo, true);
          asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(ptx::smem_u32(&full[slot])) : "memory");
        }
      }
    }
  }
  asm volatile("cp.async.wait_all;" ::: "memory");
}

// ---- consumers ----------------------------------------------------------------------------------------
// Byte offset, inside a token row of the activation operand, of the 8 bytes that hold columns e .. e+3 (e a
// multiple of 4) of group `grp`: a group is four runs of 64 bytes (one per lane c of the MMA fragment), and the
// four 16-byte chunks of a run are stored rotated by the run's number so that the lanes' 128-bit loads of chunk j
// fall on different banks.
__device__ __forceinline__ int x_offset(int grp, int e) {
  const int c = e >> 5, j = (e >> 3) & 3, half = (e >> 2) & 1;
  return grp * 256 + c * 64 + ((j + c) & 3) * 16 + half * 8;
}

__device__ __forceinline__ uint32_t pack_f16x2(float lo, float hi) {
  const __half2 h = __floats2half2_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&h);
}

// Activation operand of a pass: columns [c0, c0 + 128 glen) of the phase's activation matrix for tokens
// 0 .. x_rows - 1 as fp16 (zero beyond the last token and beyond the part's last real column), then the sum of
// every token's values per group, from the rounded values, in a fixed order.
// A thread takes eight elements of four columns per turn.  The loads of a turn are all issued before the first
// is used and the loop body has no branch that depends on the element (an element with nothing to load reads a
// valid address and is masked afterwards): with branches between them the loads went out one latency at a time
// (23 us for one 19456-column operand).
template <int KIND>
__device__ __forceinline__ void build_x_kind(const StreamInPart& in, int T, const GeluCoef& gc, int c0, int glen,
                                             unsigned char* xbuf, int x_rows, int X_PITCH) {
  const int tid = threadIdx.x;
  const int groups = glen * 32;                // 4-column elements per token row
  constexpr int B = 8;
  const int total = x_rows * groups;
  for (int e0 = tid; e0 < total; e0 += B * CTHREADS) {
    float4 v[B], u[B];
    uint2 raw[B];
    bool live[B];
#pragma unroll
    for (int j = 0; j < B; ++j) {
      const int e = e0 + j * CTHREADS;
      const int ee = e < total ? e : tid;      // a valid element to read in any case
      const int t = ee / groups, q = ee - t * groups;
      const int col = c0 + 4 * q;
      live[j] = e < total && t < T && col < in.col_end;
      const int tt = live[j] ? t : 0;
      const long long sc = in.src_col + (live[j] ? col - in.col_begin : 0);
      if (KIND == STREAM_IN_BF16) {
        raw[j] = __ldg(reinterpret_cast<const uint2*>(static_cast<const __nv_bfloat16*>(in.src) +
                                                      static_cast<long long>(tt) * in.ld + sc));
      } else {
        const float* base = static_cast<const float*>(in.src) + static_cast<long long>(tt) * in.ld + sc;
        v[j] = __ldcg(reinterpret_cast<const float4*>(base));
        if (KIND == STREAM_IN_GATED) u[j] = __ldcg(reinterpret_cast<const float4*>(base + in.gate_off));
        else u[j] = in.bias ? __ldg(reinterpret_cast<const float4*>(in.bias + (live[j] ? col - in.col_begin : 0)))
                            : make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
    if (KIND != STREAM_IN_BF16) {
      // further k ranges of the phase before: slice by slice, the eight elements' loads together
      for (int s = 1; s < in.nslices; ++s) {
        float4 b[B], bu[B];
#pragma unroll
        for (int j = 0; j < B; ++j) {
          const int e = e0 + j * CTHREADS;
          const int ee = e < total ? e : tid;
          const int t = ee / groups, q = ee - t * groups;
          const int col = c0 + 4 * q;
          const int tt = live[j] ? t : 0;
          const long long sc = in.src_col + (live[j] ? col - in.col_begin : 0);
          const float* base = static_cast<const float*>(in.src) + s * in.slice_stride + static_cast<long long>(tt) * in.ld + sc;
          b[j] = __ldcg(reinterpret_cast<const float4*>(base));
          if (KIND == STREAM_IN_GATED) bu[j] = __ldcg(reinterpret_cast<const float4*>(base + in.gate_off));
        }
#pragma unroll
        for (int j = 0; j < B; ++j) {
          v[j].x += b[j].x; v[j].y += b[j].y; v[j].z += b[j].z; v[j].w += b[j].w;
          if (KIND == STREAM_IN_GATED) { u[j].x += bu[j].x; u[j].y += bu[j].y; u[j].z += bu[j].z; u[j].w += bu[j].w; }
        }
      }
    }
#pragma unroll
    for (int j = 0; j < B; ++j) {
      const int e = e0 + j * CTHREADS;
      if (e >= total) continue;
      const int t = e / groups, q = e - t * groups;
      float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
      if (live[j]) {
        if (KIND == STREAM_IN_BF16) {
          const __nv_bfloat162 p0 = *reinterpret_cast<const __nv_bfloat162*>(&raw[j].x);
          const __nv_bfloat162 p1 = *reinterpret_cast<const __nv_bfloat162*>(&raw[j].y);
          a = make_float4(__low2float(p0), __high2float(p0), __low2float(p1), __high2float(p1));
        } else if (KIND == STREAM_IN_GATED) {
          a.x = silu_fast(v[j].x) * u[j].x; a.y = silu_fast(v[j].y) * u[j].y;
          a.z = silu_fast(v[j].z) * u[j].z; a.w = silu_fast(v[j].w) * u[j].w;
        } else {
          a.x = v[j].x + u[j].x; a.y = v[j].y + u[j].y; a.z = v[j].z + u[j].z; a.w = v[j].w + u[j].w;
          if (KIND == STREAM_IN_ACT) {
            a.x = gelu_fast(a.x, gc); a.y = gelu_fast(a.y, gc); a.z = gelu_fast(a.z, gc); a.w = gelu_fast(a.w, gc);
          }
        }
        // columns past the part's last real one multiply the zero codes of a group whose lo is not zero: they
        // must be exactly zero
        const int col = c0 + 4 * q;
        if (col + 1 >= in.col_end) a.y = 0.f;
        if (col + 2 >= in.col_end) a.z = 0.f;
        if (col + 3 >= in.col_end) a.w = 0.f;
      }
      uint2 o;
      o.x = pack_f16x2(a.x, a.y);
      o.y = pack_f16x2(a.z, a.w);
      *reinterpret_cast<uint2*>(xbuf + t * X_PITCH + x_offset(q >> 5, 4 * (q & 31))) = o;
    }
  }
}

__device__ void build_x(const QPhase& ph, int T, int act, int c0, int glen, unsigned char* xbuf, float* xsum, int x_rows,
                        int X_PITCH) {
  const GeluCoef gc = gelu_coef(act);
  const StreamInPart& in = ph.in[0];
  if (in.kind == STREAM_IN_BF16) build_x_kind<STREAM_IN_BF16>(in, T, gc, c0, glen, xbuf, x_rows, X_PITCH);
  else if (in.kind == STREAM_IN_GATED) build_x_kind<STREAM_IN_GATED>(in, T, gc, c0, glen, xbuf, x_rows, X_PITCH);
  else if (in.kind == STREAM_IN_ACT) build_x_kind<STREAM_IN_ACT>(in, T, gc, c0, glen, xbuf, x_rows, X_PITCH);
  else build_x_kind<STREAM_IN_LINEAR>(in, T, gc, c0, glen, xbuf, x_rows, X_PITCH);
  cbar();
  // sums per (group, token): one warp per pair, lane l adds the 4 values in bytes [8l, 8l+8) of the group, then
  // a fixed shuffle tree
  const int tid = threadIdx.x;
  const int warp = tid >> 5, lane = tid & 31;
  for (int task = warp; task < glen * x_rows; task += CWARPS) {
    const int grp = task / x_rows, t = task - grp * x_rows;
    const uint2 w = *reinterpret_cast<const uint2*>(xbuf + t * X_PITCH + grp * 256 + 8 * lane);
    const float2 a = __half22float2(*reinterpret_cast<const __half2*>(&w.x));
    const float2 b = __half22float2(*reinterpret_cast<const __half2*>(&w.y));
    float s = (a.x + a.y) + (b.x + b.y);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (lane == 0) xsum[grp * 8 + t] = s;
  }
  if (x_rows < 8) {
    for (int i = tid; i < glen * 8; i += CTHREADS)
      if ((i & 7) >= x_rows) xsum[i] = 0.f;
  }
}

__device__ __forceinline__ void mma_f16(float* c, uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0,
                                        uint32_t b1) {
  asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
               "{%0, %1, %2, %3};"
               : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
               : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t lds32(uint32_t addr) {
  uint32_t v;
  asm volatile("ld.shared.u32 %0, [%1];" : "=r"(v) : "r"(addr));
  return v;
}
__device__ __forceinline__ uint2 lds64(uint32_t addr) {
  uint2 v;
  asm volatile("ld.shared.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "r"(addr));
  return v;
}
// pair q (0..15) of a run of 32 three-bit codes as the fp16 pair (1024 + even code, 1024 + odd code)
template <int Q>
__device__ __forceinline__ uint32_t pair3(const uint32_t (&w)[3]) {
  if (Q < 15) return ((w[Q / 5] >> (3 * (Q % 5))) & 0x00070007u) | 0x64006400u;
  return ((w[0] >> 15) & 0x00010001u) | ((w[1] >> 14) & 0x00020002u) | ((w[2] >> 13) & 0x00040004u) | 0x64006400u;
}
__device__ __forceinline__ uint32_t prmt(uint32_t a, uint32_t b, uint32_t sel) {
  uint32_t r;
  asm("prmt.b32 %0, %1, %2, %3;" : "=r"(r) : "r"(a), "r"(b), "r"(sel));
  return r;
}

// One group (128 k) of up to 32 rows against the tokens.  ga, gb: the group's bytes in rows g and g + 8; gc, gd:
// in rows g + 16 and g + 24 (SECOND).  acc[i] receives sum_k (1024 + q_k) x_k for (row g + 16 i, tokens 2c, 2c+1)
// and (row g + 8 + 16 i, tokens 2c, 2c+1).  The eight MMAs of a 16-row block alternate between two accumulators
// (and the two blocks are interleaved): a chain of MMAs into one accumulator runs at the instruction's latency.
template <int BITS, bool SECOND>
__device__ __forceinline__ void group_mma(float (&acc)[2][4], uint32_t ga, uint32_t gb_, uint32_t gc_, uint32_t gd_, int c,
                                          const uint32_t (&xr)[16]) {
  float a0[2][4], a1[2][4];
#pragma unroll
  for (int i = 0; i < 2; ++i)
#pragma unroll
    for (int e = 0; e < 4; ++e) { a0[i][e] = 0.f; a1[i][e] = 0.f; }
  if (BITS == 3) {
    uint32_t wa[3], wb[3], wc[3], wd[3];
#pragma unroll
    for (int i = 0; i < 3; ++i) {
      wa[i] = lds32(ga + 12 * c + 4 * i); wb[i] = lds32(gb_ + 12 * c + 4 * i);
      if (SECOND) { wc[i] = lds32(gc_ + 12 * c + 4 * i); wd[i] = lds32(gd_ + 12 * c + 4 * i); }
    }
#define FFS_Q3(I)                                                                                                              \
    mma_f16(a0[(I) & 1], pair3<2 * (I)>(wa), pair3<2 * (I)>(wb), pair3<2 * (I) + 1>(wa), pair3<2 * (I) + 1>(wb), xr[2 * (I)],  \
            xr[2 * (I) + 1]);                                                                                                  \
    if (SECOND)                                                                                                                \
      mma_f16(a1[(I) & 1], pair3<2 * (I)>(wc), pair3<2 * (I)>(wd), pair3<2 * (I) + 1>(wc), pair3<2 * (I) + 1>(wd), xr[2 * (I)], \
              xr[2 * (I) + 1]);
    FFS_Q3(0) FFS_Q3(1) FFS_Q3(2) FFS_Q3(3) FFS_Q3(4) FFS_Q3(5) FFS_Q3(6) FFS_Q3(7)
#undef FFS_Q3
  } else {
    uint32_t wa[8], wb[8], wc[8], wd[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const uint2 a = lds64(ga + 32 * c + 8 * i), b = lds64(gb_ + 32 * c + 8 * i);
      wa[2 * i] = a.x; wa[2 * i + 1] = a.y; wb[2 * i] = b.x; wb[2 * i + 1] = b.y;
      if (SECOND) {
        const uint2 cc = lds64(gc_ + 32 * c + 8 * i), dd = lds64(gd_ + 32 * c + 8 * i);
        wc[2 * i] = cc.x; wc[2 * i + 1] = cc.y; wd[2 * i] = dd.x; wd[2 * i + 1] = dd.y;
      }
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      mma_f16(a0[i & 1], prmt(wa[i], 0x64646464u, 0x4140u), prmt(wb[i], 0x64646464u, 0x4140u), prmt(wa[i], 0x64646464u, 0x4342u),
              prmt(wb[i], 0x64646464u, 0x4342u), xr[2 * i], xr[2 * i + 1]);
      if (SECOND)
        mma_f16(a1[i & 1], prmt(wc[i], 0x64646464u, 0x4140u), prmt(wd[i], 0x64646464u, 0x4140u), prmt(wc[i], 0x64646464u, 0x4342u),
                prmt(wd[i], 0x64646464u, 0x4342u), xr[2 * i], xr[2 * i + 1]);
    }
  }
#pragma unroll
  for (int e = 0; e < 4; ++e) {
    acc[0][e] = a0[0][e] + a0[1][e];
    acc[1][e] = SECOND ? a1[0][e] + a1[1][e] : 0.f;
  }
}

template <int BITS, bool SECOND>
__device__ __forceinline__ void consume_stage(float (&tot)[2][4], uint32_t stage, int row_pitch, int nr, int gcnt,
                                              int g_first, uint32_t xs, bool my_token, const float* xsum, int warp, int g,
                                              int c) {
  constexpr int GB = BITS == 8 ? qnt::kGroupBytes8 : qnt::kGroupBytes3;
  constexpr int PAR = BITS == 8 ? 128 : 48;
  const uint32_t r0 = stage + (g < nr ? g : 0) * row_pitch, r1 = stage + (g + 8 < nr ? g + 8 : 0) * row_pitch;
  const uint32_t r2 = stage + (g + 16 < nr ? g + 16 : 0) * row_pitch, r3 = stage + (g + 24 < nr ? g + 24 : 0) * row_pitch;
  // whole groups to the warps in turn, by the group's number inside the k range, so that the turn goes on across stages
  int gi = (warp - (g_first & 7)) & 7;
  for (; gi < gcnt; gi += CWARPS) {
    const int grp = g_first + gi;               // group inside the pass's k range: indexes the activation operand
    uint32_t xr[16];
    if (my_token) {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const uint4 t = lds128(xs + grp * 256 + c * 64 + ((j + c) & 3) * 16);
        xr[4 * j] = t.x; xr[4 * j + 1] = t.y; xr[4 * j + 2] = t.z; xr[4 * j + 3] = t.w;
      }
    } else {
#pragma unroll
      for (int j = 0; j < 16; ++j) xr[j] = 0u;
    }
    const float2 sx = *reinterpret_cast<const float2*>(xsum + grp * 8 + 2 * c);    // tokens 2c, 2c + 1
    const uint2 pa = lds64(r0 + gi * GB + PAR), pb = lds64(r1 + gi * GB + PAR);
    float acc[2][4];
    group_mma<BITS, SECOND>(acc, r0 + gi * GB, r1 + gi * GB, r2 + gi * GB, r3 + gi * GB, c, xr);
    {
      const float sa = __uint_as_float(pa.x), la = __uint_as_float(pa.y) - 1024.f * sa;
      const float sb = __uint_as_float(pb.x), lb = __uint_as_float(pb.y) - 1024.f * sb;
      tot[0][0] += fmaf(sa, acc[0][0], la * sx.x); tot[0][1] += fmaf(sa, acc[0][1], la * sx.y);
      tot[0][2] += fmaf(sb, acc[0][2], lb * sx.x); tot[0][3] += fmaf(sb, acc[0][3], lb * sx.y);
    }
    if (SECOND) {
      const uint2 pc = lds64(r2 + gi * GB + PAR), pd = lds64(r3 + gi * GB + PAR);
      const float sa = __uint_as_float(pc.x), la = __uint_as_float(pc.y) - 1024.f * sa;
      const float sb = __uint_as_float(pd.x), lb = __uint_as_float(pd.y) - 1024.f * sb;
      tot[1][0] += fmaf(sa, acc[1][0], la * sx.x); tot[1][1] += fmaf(sa, acc[1][1], la * sx.y);
      tot[1][2] += fmaf(sb, acc[1][2], lb * sx.x); tot[1][3] += fmaf(sb, acc[1][3], lb * sx.y);
    }
  }
}

__device__ void consumers(const QParams& p, unsigned char* smem, uint32_t ring, uint64_t* full, uint64_t* empty,
                          volatile int* s_abort) {
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, c = lane & 3;
  unsigned char* xbuf = smem + OFF_X;
  float* xsum = reinterpret_cast<float*>(smem + OFF_XSUM);
  const int X_PITCH = p.x_pitch;
  const bool my_token = g < p.x_rows;
  const uint32_t xs = ring + OFF_X + (my_token ? g * X_PITCH : 0);
  float* red = reinterpret_cast<float*>(smem + OFF_RED_Q);
  uint32_t it = 0;
  unsigned flushes = 0;
  for (int pi = 0; pi < p.nph; ++pi) {
    const QPhase& ph = p.ph[pi];
    unsigned uw = 0, lo = 0, hi = 0;
    if (ph.kind == 0) {
      uw = units_per_split(ph);
      const unsigned U = uw * ph.S;
      lo = U * blockIdx.x / gridDim.x;
      hi = U * (blockIdx.x + 1) / gridDim.x;
    }
    if (pi > 0 && ph.sync_before) grid_barrier(p.ctrl, s_abort);
    if (ph.kind != 0) {
      // ---- closing reduction: y[t, n] = sum of all slices + bias, for a share of the columns
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
    for (unsigned u = lo; u < hi;) {
      unsigned next;
      const QPass ps = qpass_at(ph, uw, u, hi, &next);
      u = next;
      if (ps.rows == 0) continue;
      const QSegment& sg = ph.seg[ps.seg];
      const int c0 = sg.x_off + ps.gbeg * qnt::kGroup;
      if (c0 != x_c0 || ps.glen != x_len) {
        if (x_c0 >= 0) cbar();
        build_x(ph, p.T, p.act, c0, ps.glen, xbuf, xsum, p.x_rows, X_PITCH);
        cbar();
        x_c0 = c0; x_len = ps.glen;
      }
      const int nb = blocks_of(ps.rows);
      for (int b = 0; b < nb; ++b) {
        const int r_lo = block_lo(ps.rows, nb, b), r_hi = block_lo(ps.rows, nb, b + 1);
        int gch, row_pitch;
        stage_shape(r_hi - r_lo, sg.bits, &gch, &row_pitch);
        const int nch = (ps.glen + gch - 1) / gch;
        float tot[2][4];
#pragma unroll
        for (int i = 0; i < 2; ++i)
#pragma unroll
          for (int e = 0; e < 4; ++e) tot[i][e] = 0.f;
        const bool second = r_hi - r_lo > 16;
        for (int ch = 0; ch < nch; ++ch, ++it) {
          const int slot = it % NSTAGE;
          const int gcnt = ps.glen - ch * gch < gch ? ps.glen - ch * gch : gch;
          ptx::mbar_wait_limit(&full[slot], (it / NSTAGE) & 1, s_abort, kWaitLimit);
          const uint32_t stage = ring + slot * STAGE_BYTES;
          const int nr = r_hi - r_lo;
          if (sg.bits == 8) {
            if (second) consume_stage<8, true>(tot, stage, row_pitch, nr, gcnt, ch * gch, xs, my_token, xsum, warp, g, c);
            else consume_stage<8, false>(tot, stage, row_pitch, nr, gcnt, ch * gch, xs, my_token, xsum, warp, g, c);
          } else {
            if (second) consume_stage<3, true>(tot, stage, row_pitch, nr, gcnt, ch * gch, xs, my_token, xsum, warp, g, c);
            else consume_stage<3, false>(tot, stage, row_pitch, nr, gcnt, ch * gch, xs, my_token, xsum, warp, g, c);
          }
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(&empty[slot]);
        }
        // ---- the eight warps' sums over their groups, added in warp order
        float* rb = red + (flushes & 1) * (CWARPS * RED_WARP) + warp * RED_WARP;
        ++flushes;
#pragma unroll
        for (int i = 0; i < 2; ++i) {
          rb[(2 * c) * RED_TOK + 16 * i + g] = tot[i][0];
          rb[(2 * c + 1) * RED_TOK + 16 * i + g] = tot[i][1];
          rb[(2 * c) * RED_TOK + 16 * i + g + 8] = tot[i][2];
          rb[(2 * c + 1) * RED_TOK + 16 * i + g + 8] = tot[i][3];
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
            ph.out[(static_cast<long long>(ph.slice0 + ps.s) * 8 + t) * ph.out_ld + n] = v;
          }
        }
      }
    }
  }
}

__global__ void __launch_bounds__(THREADS, 1) decode_quant_kernel(const __grid_constant__ QParams p) {
  extern __shared__ __align__(128) unsigned char smem[];
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + OFF_BAR_Q);
  uint64_t* empty = full + NSTAGE;
  volatile int* s_abort = reinterpret_cast<volatile int*>(empty + NSTAGE);
  const uint32_t ring = static_cast<uint32_t>(__cvta_generic_to_shared(smem));
  if (threadIdx.x == 0) {
    for (int i = 0; i < NSTAGE; ++i) {
      ptx::mbar_init(&full[i], 32);
      ptx::mbar_init(&empty[i], CWARPS);
    }
    *s_abort = 0;
    ptx::mbar_fence_init();
  }
  __syncthreads();
  if (threadIdx.x >= CTHREADS) producer(p, ring, full, empty, s_abort, (threadIdx.x - CTHREADS) >> 5);
  else consumers(p, smem, ring, full, empty, s_abort);
  __syncthreads();
  if (threadIdx.x == 0 && *s_abort) record_status(p.ctrl, FFSPLIT_ERR_TIMEOUT, static_cast<int>(blockIdx.x), KID_QUANT);
}

}  // namespace dqt

ffsplit_status decode_quant_launch(ffsplit_ctx* ctx, const QParams& p, double algo_bytes, cudaStream_t st) {
  static bool attr_done[64] = {false};
  const int dev = ctx->device;
  if (dev < 0 || dev >= 64) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "device index out of range");
  int coop = 0;
  if (cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, dev) != cudaSuccess || !coop)
    return fail(ctx, FFSPLIT_ERR_ARCH, "the device does not support cooperative launches");
  if (!attr_done[dev]) {
    cudaError_t e = cudaFuncSetAttribute(dqt::decode_quant_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         dqt::SMEM_BYTES_Q);
    if (e != cudaSuccess) return check_cuda(ctx, e, "cudaFuncSetAttribute(decode_quant_kernel)");
    attr_done[dev] = true;
  }
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(ctx->num_sms);
  cfg.blockDim = dim3(dst::THREADS);
  cfg.dynamicSmemBytes = dqt::SMEM_BYTES_Q;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;
  attr[0].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const int ph = prof_open(ctx, PROF_DECODE, algo_bytes, st);
  const cudaError_t e = cudaLaunchKernelEx(&cfg, dqt::decode_quant_kernel, p);
  prof_close(ctx, ph, st);
  ctx->launches++;
  return check_cuda(ctx, e, "decode_quant_kernel launch");
}

}  // namespace ffsp
