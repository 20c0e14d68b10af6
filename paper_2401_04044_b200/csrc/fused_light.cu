// Fused light chain of the split forward (FFN_2 of Eq. 2 with rank-r factors):
//
//     P = sigma(Q B1 + b1[light]) A2          Q: [T, r], B1: [r, mL], A2: [mL, r]
//
// for GELU layers in bf16 with r_pad <= 256.  The T x mL activation matrix never
// leaves the SM: per 128-token tile and 128-neuron chunk
//   GEMM-a   S = Q_tile B1[:, chunk]        tcgen05.mma, operands in shared memory, S in
//                                           tensor memory (TMEM), two S buffers
//   epilogue H = GELU(S + b1) -> bf16, written back into the first half of the TMEM
//            columns it was read from (two bf16 per 32-bit cell)
//   GEMM-b   Pacc += H A2[chunk, :]         tcgen05.mma with the A operand read from TMEM;
//                                           Pacc stays in TMEM for the whole tile
// Chains of dependent small-N MMAs are latency bound on the tensor pipe, hence the
// 128-wide chunks (N = 128 for GEMM-a, K = 128 for GEMM-b).
// Warp roles: warp 0 TMA producer of the Q tile, the B1 ring and the bias ring,
// warp 1 MMA issuer, warps 2-17 epilogue (four warps per TMEM lane quarter, 32
// columns each), warp 18 TMA producer of the A2 ring.  Both weight rings work at the
// granularity of one 64-deep k-block so that shared memory holds the Q tile plus
// about two chunks of each operand.
// The chunks of one token tile are spread over `splits` CTAs so that the grid covers
// the SMs; each CTA writes its fp32 partial of P and the last CTA to finish a token
// tile (atomic ticket) adds the partials in split order -- a fixed order, so the
// result does not depend on which CTA is last -- and stores bf16 P.
// Every wait is bounded (see gemm_tc.cu).
#include "epilogue.cuh"
#include "internal.h"
#include "ptx.cuh"

namespace ffsp {

ffsplit_status get_tmap_bf16(ffsplit_ctx* ctx, const void* ptr, long long rows, long long cols, long long ld,
                             int box_rows, CUtensorMap* out);

namespace fl {

constexpr int BLOCK_M = 128;
constexpr int CHUNK = 128;         // light neurons per chunk (N of GEMM-a, K of GEMM-b)
constexpr int KB = 64;             // K elements per shared-memory k-block (one 128-byte swizzle row)
constexpr int EPI_WARPS = 16;
constexpr int NUM_THREADS = 32 * (EPI_WARPS + 3);
constexpr int EPI_THREADS = 32 * EPI_WARPS;
constexpr int A2_WARP = EPI_WARPS + 2;
constexpr int MAX_B1_SLOTS = 8;
constexpr int MAX_A2_SLOTS = 6;
constexpr int BIAS_SLOTS = 8;
constexpr int TMEM_COLS = 512;
constexpr int TMEM_S0 = 256;       // S buffers at columns 256 and 384; P accumulator at 0..255
constexpr int QKB_BYTES = BLOCK_M * KB * 2;
constexpr int B1KB_BYTES = CHUNK * KB * 2;
constexpr int BIAS_BYTES = BIAS_SLOTS * CHUNK * 4;
constexpr int BAR_BYTES = 1024;
constexpr int MAX_SMEM = 232448;

struct Params {
  long long T;
  int r_pad, ml_pad, kbq;           // kbq = ceil(r_pad / 64): k-blocks of Q and of a B1 chunk
  int n_chunks, splits;
  int b1_slots, a2_slots;           // ring depths, in k-blocks
  int a2_slot_bytes;                // r_pad * 128
  int bias_off;                     // byte offset of the bias ring (after the rings and after the staging area)
  const float* b1l;
  __nv_bfloat16* P; long long ldp;  // output, bf16
  float* partial;                   // [splits][tiles_m * 128][r_pad] fp32 (splits > 1)
  int* tickets;                     // [tiles_m], zero before the launch, zero again after it
  int act;
  int* status;
};

// Position in a ring of n slots: slot index and the parity of the number of completed rounds (no divisions on the
// producers' and the MMA issuer's paths: they share their schedulers with the epilogue warps).
struct Cursor {
  int slot = 0;
  uint32_t phase = 0;
  __device__ __forceinline__ void next(int n) {
    if (++slot == n) { slot = 0; phase ^= 1u; }
  }
};

// D[tmem] (+)= A[tmem] * B[smem desc]: A is a 128 x 16 bf16 slab held as 8 TMEM columns.
__device__ __forceinline__ void umma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t idesc,
                                             uint32_t accumulate) {
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "setp.ne.b32 p, %4, 0;\n"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n"
      "}\n" ::"r"(d_tmem),
      "r"(a_tmem), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void tmem_st16(uint32_t taddr, const uint32_t* r) {
  asm volatile(
      "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
      "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};" ::"r"(taddr),
      "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]), "r"(r[9]),
      "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
      : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }
// Untiled bulk copy global -> shared with completion on an mbarrier (16-byte aligned, size % 16 == 0).
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   ptx::smem_u32(smem_dst)),
               "l"(gsrc), "r"(bytes), "r"(ptx::smem_u32(bar))
               : "memory");
}

__global__ void __launch_bounds__(NUM_THREADS, 1)
fused_light_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmB1,
                   const __grid_constant__ CUtensorMap tmA2, const Params p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* smem_q = smem;
  uint8_t* smem_b1 = smem_q + p.kbq * QKB_BYTES;
  uint8_t* smem_a2 = smem_b1 + p.b1_slots * B1KB_BYTES;
  float* smem_bias = reinterpret_cast<float*>(smem + p.bias_off);
  uint64_t* bars = reinterpret_cast<uint64_t*>(reinterpret_cast<uint8_t*>(smem_bias) + BIAS_BYTES);
  uint64_t* b1full = bars;                       // [MAX_B1_SLOTS] TMA -> MMA (one k-block of a B1 chunk)
  uint64_t* b1empty = b1full + MAX_B1_SLOTS;     // [MAX_B1_SLOTS] MMA -> TMA
  uint64_t* a2full = b1empty + MAX_B1_SLOTS;     // [MAX_A2_SLOTS] TMA -> MMA (one k-block of an A2 chunk)
  uint64_t* a2empty = a2full + MAX_A2_SLOTS;     // [MAX_A2_SLOTS] MMA -> TMA
  uint64_t* biasfull = a2empty + MAX_A2_SLOTS;   // [BIAS_SLOTS] TMA -> epilogue
  uint64_t* sfull = biasfull + BIAS_SLOTS;       // [2] GEMM-a done -> epilogue
  uint64_t* hfull = sfull + 2;                   // [2] epilogue wrote H -> MMA
  uint64_t* qfull = hfull + 2;                   // [1]
  uint64_t* pfull = qfull + 1;                   // [1] all GEMM-b done -> epilogue
  uint64_t* redbar = pfull + 1;                  // [1] epilogue warps rendezvous
  uint64_t* drain = redbar + 1;                  // [1]
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(drain + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);
  volatile int* last_flag = abort_flag + 1;

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int split = blockIdx.x;
  const int m_blk = blockIdx.y;
  // chunk range of this CTA
  const int c_begin = static_cast<int>(static_cast<long long>(p.n_chunks) * split / p.splits);
  const int c_end = static_cast<int>(static_cast<long long>(p.n_chunks) * (split + 1) / p.splits);
  const int my_chunks = c_end - c_begin;

  if (threadIdx.x == 0) {
    for (int s = 0; s < MAX_B1_SLOTS; ++s) { ptx::mbar_init(&b1full[s], 1); ptx::mbar_init(&b1empty[s], 1); }
    for (int s = 0; s < MAX_A2_SLOTS; ++s) { ptx::mbar_init(&a2full[s], 1); ptx::mbar_init(&a2empty[s], 1); }
    for (int s = 0; s < BIAS_SLOTS; ++s) ptx::mbar_init(&biasfull[s], 1);
    for (int a = 0; a < 2; ++a) { ptx::mbar_init(&sfull[a], 1); ptx::mbar_init(&hfull[a], EPI_WARPS); }
    ptx::mbar_init(qfull, 1);
    ptx::mbar_init(pfull, 1);
    ptx::mbar_init(redbar, EPI_WARPS);
    ptx::mbar_init(drain, 1);
    *abort_flag = 0;
    *last_flag = 0;
    ptx::mbar_fence_init();
    ptx::prefetch_tmap(&tmQ);
    ptx::prefetch_tmap(&tmB1);
    ptx::prefetch_tmap(&tmA2);
  }
  if (warp == 1) {
    ptx::tmem_alloc(tmem_holder, TMEM_COLS);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_holder;
  // Launched with programmatic stream serialisation: everything above (barriers, tensor maps, tensor
  // memory) overlapped the tail of the kernel before; nothing below may start until that kernel is
  // complete and its writes are visible.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  // Only now may the kernel after this one begin its set-up: it will block in its tensor-memory allocation
  // until this CTA frees its columns, which is safe because this CTA already holds its own (a dependent
  // that got the columns first would wait for this kernel, and this kernel for the columns).
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  if (warp == 0) {
    if (ptx::elect_one()) {
      // ------------------------------------------------------------ TMA producer: Q tile, bias ring, B1 ring
      bool ok = true;
      ptx::mbar_expect_tx(qfull, p.kbq * QKB_BYTES);
      for (int kb = 0; kb < p.kbq; ++kb) ptx::tma_load_2d(&tmQ, smem_q + kb * QKB_BYTES, qfull, kb * KB, m_blk * BLOCK_M);
      int g = 0;
      Cursor cur;
      for (int i = 0; i < my_chunks && ok; ++i) {
        const int chunk = c_begin + i;
        for (int kb = 0; kb < p.kbq; ++kb, ++g, cur.next(p.b1_slots)) {
          const int slot = cur.slot;
          if (!ptx::mbar_wait(&b1empty[slot], cur.phase ^ 1u, abort_flag)) { ok = false; break; }
          if (kb == 0) {
            // b1[light] of this chunk; a bias slot is reused 8 chunks later, by when its readers are long done
            const int n0 = chunk * CHUNK;
            const int cnt = p.ml_pad - n0 < CHUNK ? p.ml_pad - n0 : CHUNK;
            ptx::mbar_expect_tx(&biasfull[i % BIAS_SLOTS], cnt * 4);
            bulk_load(smem_bias + (i % BIAS_SLOTS) * CHUNK, p.b1l + n0, cnt * 4, &biasfull[i % BIAS_SLOTS]);
          }
          ptx::mbar_expect_tx(&b1full[slot], B1KB_BYTES);
          ptx::tma_load_2d(&tmB1, smem_b1 + slot * B1KB_BYTES, &b1full[slot], kb * KB, chunk * CHUNK);
        }
      }
      if (!ok) {
        const long long t0 = clock64();
        while (!ptx::mbar_try_wait(qfull, 0) && clock64() - t0 < ptx::kWaitLimitCycles / 8) {}
        const int first = g > p.b1_slots ? g - p.b1_slots : 0;
        for (int j = first; j < g; ++j) {
          const long long t1 = clock64();
          while (!ptx::mbar_try_wait(&b1full[j % p.b1_slots], (j / p.b1_slots) & 1) &&
                 clock64() - t1 < ptx::kWaitLimitCycles / 8) {}
        }
      }
    }
    __syncwarp();
  } else if (warp == A2_WARP) {
    if (ptx::elect_one()) {
      // ------------------------------------------------------------ TMA producer: A2 ring
      bool ok = true;
      int g = 0;
      Cursor cur;
      for (int i = 0; i < my_chunks && ok; ++i) {
        for (int kb = 0; kb < CHUNK / KB; ++kb, ++g, cur.next(p.a2_slots)) {
          const int slot = cur.slot;
          if (!ptx::mbar_wait(&a2empty[slot], cur.phase ^ 1u, abort_flag)) { ok = false; break; }
          ptx::mbar_expect_tx(&a2full[slot], p.a2_slot_bytes);
          ptx::tma_load_2d(&tmA2, smem_a2 + slot * p.a2_slot_bytes, &a2full[slot], (c_begin + i) * CHUNK + kb * KB, 0);
        }
      }
      if (!ok) {
        const int first = g > p.a2_slots ? g - p.a2_slots : 0;
        for (int j = first; j < g; ++j) {
          const long long t1 = clock64();
          while (!ptx::mbar_try_wait(&a2full[j % p.a2_slots], (j / p.a2_slots) & 1) &&
                 clock64() - t1 < ptx::kWaitLimitCycles / 8) {}
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    if (ptx::elect_one()) {
      // ------------------------------------------------------------ MMA issuer
      const uint32_t idesc_a = ptx::umma_idesc_bf16(BLOCK_M, CHUNK);
      const uint32_t idesc_b = ptx::umma_idesc_bf16(BLOCK_M, p.r_pad);
      bool ok = ptx::mbar_wait(qfull, 0, abort_flag);
      // GEMM-b of chunk j: Pacc += H(j) * A2 tile of chunk j.  H(j) sits in the S buffer j & 1: the
      // 32 fp32 columns [32 c, 32 c + 32) of S became the 16 packed columns [32 c, 32 c + 16).
      Cursor ca2, cb1;   // gemm_b is called for j = 0, 1, 2, ... in order
      const uint64_t q_desc0 = ptx::umma_desc_k128(ptx::smem_u32(smem_q));
      const uint64_t b1_desc0 = ptx::umma_desc_k128(ptx::smem_u32(smem_b1));
      const uint64_t a2_desc0 = ptx::umma_desc_k128(ptx::smem_u32(smem_a2));
      const uint32_t a2_step = static_cast<uint32_t>(p.a2_slot_bytes) >> 4;   // descriptor addresses count 16 bytes
      auto gemm_b = [&](int j) -> bool {
        if (!ptx::mbar_wait(&hfull[j & 1], (j >> 1) & 1, abort_flag)) return false;
        ptx::tc_fence_after();
        const uint32_t h_tmem = tmem_base + TMEM_S0 + (j & 1) * CHUNK;
#pragma unroll
        for (int kb = 0; kb < CHUNK / KB; ++kb, ca2.next(p.a2_slots)) {
          const int slot = ca2.slot;
          if (!ptx::mbar_wait(&a2full[slot], ca2.phase, abort_flag)) return false;
          ptx::tc_fence_after();
          const uint64_t b_desc = a2_desc0 + static_cast<uint32_t>(slot) * a2_step;
#pragma unroll
          for (int k = 0; k < KB / 16; ++k) {
            const int jj = kb * (KB / 16) + k;   // 16-element slab of this chunk's K range
            umma_bf16_ts(tmem_base, h_tmem + 32 * (jj >> 1) + 8 * (jj & 1), b_desc + 2 * k, idesc_b,
                         (j | jj) != 0 ? 1u : 0u);
          }
          ptx::umma_commit(&a2empty[slot]);
        }
        return true;
      };
      for (int i = 0; i < my_chunks && ok; ++i) {
        // S buffer i & 1 is free: GEMM-b of chunk i - 2 (its last reader) was issued before this point
        const uint32_t d_tmem = tmem_base + TMEM_S0 + (i & 1) * CHUNK;
        for (int kb = 0; kb < p.kbq; ++kb, cb1.next(p.b1_slots)) {
          const int slot = cb1.slot;
          if (!ptx::mbar_wait(&b1full[slot], cb1.phase, abort_flag)) { ok = false; break; }
          ptx::tc_fence_after();
          const uint64_t a_desc = q_desc0 + static_cast<uint32_t>(kb) * (QKB_BYTES >> 4);
          const uint64_t b_desc = b1_desc0 + static_cast<uint32_t>(slot) * (B1KB_BYTES >> 4);
#pragma unroll
          for (int k = 0; k < KB / 16; ++k)
            ptx::umma_bf16(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc_a, (kb | k) != 0 ? 1u : 0u);
          ptx::umma_commit(&b1empty[slot]);
        }
        if (!ok) break;
        ptx::umma_commit(&sfull[i & 1]);
        if (i > 0) ok = gemm_b(i - 1);
      }
      if (ok && my_chunks > 0) ok = gemm_b(my_chunks - 1);
      if (ok) ptx::umma_commit(pfull);
      if (!ok) {
        ptx::umma_commit(drain);
        const long long t0 = clock64();
        while (!ptx::mbar_try_wait(drain, 0) && clock64() - t0 < ptx::kWaitLimitCycles / 8) {}
      }
    }
    __syncwarp();
  } else {
    // -------------------------------------------------------------- epilogue warps (2 .. 17)
    const int q = warp & 3;              // TMEM lane quarter
    const int cg = (warp - 2) >> 2;      // which 32 of the chunk's 128 columns
    const int row_in_tile = q * 32 + lane;
    const int te = threadIdx.x - 64;     // 0 .. 511
    const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
    const GeluCoef gc = gelu_coef(p.act);
    bool ok = true;
    for (int i = 0; i < my_chunks; ++i) {
      const int sb = i & 1;
      if (!ptx::mbar_wait(&biasfull[i % BIAS_SLOTS], (i / BIAS_SLOTS) & 1, abort_flag)) { ok = false; break; }
      if (!ptx::mbar_wait(&sfull[sb], (i >> 1) & 1, abort_flag)) { ok = false; break; }
      ptx::tc_fence_after();
      const uint32_t t_s = t_lane + TMEM_S0 + sb * CHUNK + cg * 32;
      const float* bias = smem_bias + (i % BIAS_SLOTS) * CHUNK + cg * 32;
      const int n0 = (c_begin + i) * CHUNK + cg * 32;
      // both 16-column loads in flight before the one wait; bias and GELU on the packed fp32 instructions (every
      // component goes through gelu_fast's operations: the same bits)
      uint32_t w[16];
      float va[16], vb[16];
      ptx::tmem_ld16(t_s, va);
      ptx::tmem_ld16(t_s + 16, vb);
      ptx::tmem_ld_wait();
#pragma unroll
      for (int hlf = 0; hlf < 2; ++hlf) {
        const float* v = hlf ? vb : va;
        if (n0 + 16 * hlf + 16 <= p.ml_pad) {   // ml_pad is a multiple of 16
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const float4 b = *reinterpret_cast<const float4*>(bias + 16 * hlf + 4 * j);
            const float2 g0 = gelu_fast2(__fadd2_rn(make_float2(v[4 * j], v[4 * j + 1]), make_float2(b.x, b.y)), gc);
            const float2 g1 = gelu_fast2(__fadd2_rn(make_float2(v[4 * j + 2], v[4 * j + 3]), make_float2(b.z, b.w)), gc);
            w[8 * hlf + 2 * j] = pack_bf16x2(g0.x, g0.y);
            w[8 * hlf + 2 * j + 1] = pack_bf16x2(g1.x, g1.y);
          }
        } else {
#pragma unroll
          for (int j = 0; j < 8; ++j) w[8 * hlf + j] = 0u;
        }
      }
      tmem_st16(t_s, w);   // both 16-column loads of this warp's range have completed
      tmem_st_wait();
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&hfull[sb]);
    }
    // ---- the tile's accumulator: TMEM -> shared memory (fp32, padded rows) -> coalesced global
    if (ok && my_chunks > 0) ok = ptx::mbar_wait(pfull, 0, abort_flag);
    const int pitch = p.r_pad + 4;   // keeps the row-per-thread float4 writes free of bank conflicts
    float* stage = reinterpret_cast<float*>(smem);
    if (ok) {
      ptx::tc_fence_after();
      // every MMA and every TMA load of this CTA has completed: the operand buffers are free
      for (int c = cg * 16; c < p.r_pad; c += 64) {
        float v[16];
        if (my_chunks > 0) {
          ptx::tmem_ld16(t_lane + c, v);
          ptx::tmem_ld_wait();
        } else {
#pragma unroll
          for (int j = 0; j < 16; ++j) v[j] = 0.f;
        }
        float4* dst = reinterpret_cast<float4*>(stage + row_in_tile * pitch + c);
#pragma unroll
        for (int j = 0; j < 4; ++j) dst[j] = make_float4(v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
      }
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(redbar);
      ok = ptx::mbar_wait(redbar, 0, abort_flag);
    }
    if (ok) {
      const int q4 = p.r_pad >> 2;                 // float4 per row
      const int n4 = BLOCK_M * q4;
      const long long row0 = static_cast<long long>(m_blk) * BLOCK_M;
      const long long rows_total = static_cast<long long>(gridDim.y) * BLOCK_M;
      if (p.splits > 1) {
        float4* mine = reinterpret_cast<float4*>(p.partial + (static_cast<long long>(split) * rows_total + row0) * p.r_pad);
        for (int e = te; e < n4; e += EPI_THREADS) {
          const int r = e / q4, c4 = e - r * q4;
          mine[e] = *reinterpret_cast<const float4*>(stage + r * pitch + 4 * c4);
        }
        // publish the partial, take a ticket; the last CTA of this token tile reduces
        __threadfence();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(redbar);
        ok = ptx::mbar_wait(redbar, 1, abort_flag);
        if (ok) {
          if (warp == 2 && lane == 0) {
            const int t = atomicAdd(p.tickets + m_blk, 1);
            *last_flag = (t == p.splits - 1) ? 1 : 0;
            __threadfence();
          }
          __syncwarp();
          if (lane == 0) ptx::mbar_arrive(redbar);
          ok = ptx::mbar_wait(redbar, 0, abort_flag);
        }
      }
      if (ok && (p.splits == 1 || *last_flag)) {
        if (p.splits > 1) __threadfence();
        // Batches of 4 x 3 independent loads per thread: the sum over splits is taken in split order
        // (so it does not depend on which CTA is last) but the loads do not wait for one another.
        constexpr int EG = 3;
        for (int e0 = te; e0 < n4; e0 += EPI_THREADS * EG) {
          float4 acc[EG];
#pragma unroll
          for (int j = 0; j < EG; ++j) acc[j] = make_float4(0.f, 0.f, 0.f, 0.f);
          for (int s0 = 0; s0 < p.splits; s0 += 4) {
            float4 buf[4][EG];
#pragma unroll
            for (int ss = 0; ss < 4; ++ss) {
              const int sp = s0 + ss;
#pragma unroll
              for (int j = 0; j < EG; ++j) {
                const int e = e0 + j * EPI_THREADS;
                buf[ss][j] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (sp < p.splits && e < n4) {
                  if (sp == split) {
                    const int r = e / q4, c4 = e - r * q4;
                    buf[ss][j] = *reinterpret_cast<const float4*>(stage + r * pitch + 4 * c4);
                  } else {
                    buf[ss][j] = __ldcg(reinterpret_cast<const float4*>(
                                            p.partial + (static_cast<long long>(sp) * rows_total + row0) * p.r_pad) + e);
                  }
                }
              }
            }
#pragma unroll
            for (int ss = 0; ss < 4; ++ss) {
              if (s0 + ss < p.splits) {
#pragma unroll
                for (int j = 0; j < EG; ++j) {
                  acc[j].x += buf[ss][j].x; acc[j].y += buf[ss][j].y; acc[j].z += buf[ss][j].z; acc[j].w += buf[ss][j].w;
                }
              }
            }
          }
#pragma unroll
          for (int j = 0; j < EG; ++j) {
            const int e = e0 + j * EPI_THREADS;
            if (e < n4) {
              const int r = e / q4, c4 = e - r * q4;
              if (row0 + r < p.T) {
                uint2 o;
                o.x = pack_bf16x2(acc[j].x, acc[j].y);
                o.y = pack_bf16x2(acc[j].z, acc[j].w);
                *reinterpret_cast<uint2*>(p.P + (row0 + r) * p.ldp + 4 * c4) = o;
              }
            }
          }
        }
        if (p.splits > 1 && warp == 2 && lane == 0) p.tickets[m_blk] = 0;   // ready for the next launch
      }
    }
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) record_status(p.status, FFSPLIT_ERR_TIMEOUT, blockIdx.x, KID_FUSED);
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

}  // namespace fl

bool fused_light_applies(int dtype, int act, int r_pad, int ml_pad) {
  return dtype == FFSPLIT_BF16 && act != FFSPLIT_SWIGLU && r_pad >= 16 && r_pad <= 256 && ml_pad > 0;
}

// Number of CTAs per token tile: enough to cover the SMs, at most 16 and at most one per chunk.
int fused_light_splits(int num_sms, long long tiles_m, int n_chunks) {
  long long s = num_sms / tiles_m;
  if (s < 1) s = 1;
  if (s > 16) s = 16;
  if (s > n_chunks) s = n_chunks;
  return static_cast<int>(s);
}

// Scratch for the fp32 partials, for any SM count (splits <= 16, splits * tiles <= max(tiles, 256)).
size_t fused_light_scratch_bytes(long long T, int r_pad) {
  const long long tiles_m = (T + fl::BLOCK_M - 1) / fl::BLOCK_M;
  long long s = 16;
  if (s * tiles_m > 256 && tiles_m <= 256) s = 256 / tiles_m;
  if (tiles_m > 256) s = 1;
  return static_cast<size_t>(s) * tiles_m * fl::BLOCK_M * r_pad * 4;
}

ffsplit_status launch_fused_light(ffsplit_ctx* ctx, const void* Q, long long ldq, long long T, const void* B1T,
                                  const void* A2T, const float* b1l, int r_pad, int ml_pad, int act, void* P,
                                  long long ldp, char* scratch, int* tickets, double algo_flops,
                                  cudaStream_t st) {
  fl::Params p;
  p.T = T;
  p.r_pad = r_pad;
  p.ml_pad = ml_pad;
  p.kbq = (r_pad + fl::KB - 1) / fl::KB;
  p.n_chunks = (ml_pad + fl::CHUNK - 1) / fl::CHUNK;
  const long long tiles_m = (T + fl::BLOCK_M - 1) / fl::BLOCK_M;
  if (tiles_m > 65535) return fail(ctx, FFSPLIT_ERR_SHAPE, "too many token tiles for one launch");
  p.splits = fused_light_splits(ctx->num_sms, tiles_m, p.n_chunks);
  if (p.splits > 1 && static_cast<long long>(p.splits) * tiles_m > (tiles_m > 256 ? tiles_m : 256)) p.splits = 1;
  p.a2_slot_bytes = r_pad * fl::KB * 2;
  // ring depths: what fits beside the Q tile, balanced in units of chunks (kbq B1 k-blocks, 2 A2 k-blocks)
  const int fixed = p.kbq * fl::QKB_BYTES + fl::BIAS_BYTES + fl::BAR_BYTES + 1024;
  int best_b1 = 0, best_a2 = 0;
  double best = -1.0;
  for (int nb = 1; nb <= fl::MAX_B1_SLOTS; ++nb)
    for (int na = 1; na <= fl::MAX_A2_SLOTS; ++na) {
      if (fixed + nb * fl::B1KB_BYTES + na * p.a2_slot_bytes > fl::MAX_SMEM) continue;
      const double a = static_cast<double>(nb) / p.kbq, b = static_cast<double>(na) / 2.0;
      const double score = (a < b ? a : b) + 1e-3 * (a + b);
      if (score > best) { best = score; best_b1 = nb; best_a2 = na; }
    }
  if (best_b1 < 1 || best_a2 < 1) return fail(ctx, FFSPLIT_ERR_SHAPE, "fused light chain: shared memory too small");
  p.b1_slots = best_b1;
  p.a2_slots = best_a2;
  p.b1l = b1l;
  p.P = static_cast<__nv_bfloat16*>(P);
  p.ldp = ldp;
  p.tickets = tickets;
  p.partial = reinterpret_cast<float*>(scratch);
  p.act = act;
  p.status = ctx->status();
  CUtensorMap tQ, tB1, tA2;
  ffsplit_status s;
  if ((s = get_tmap_bf16(ctx, Q, T, r_pad, ldq, fl::BLOCK_M, &tQ)) != FFSPLIT_OK) return s;
  if ((s = get_tmap_bf16(ctx, B1T, ml_pad, r_pad, r_pad, fl::CHUNK, &tB1)) != FFSPLIT_OK) return s;
  if ((s = get_tmap_bf16(ctx, A2T, r_pad, ml_pad, ml_pad, r_pad, &tA2)) != FFSPLIT_OK) return s;
  const int ring_end = p.kbq * fl::QKB_BYTES + p.b1_slots * fl::B1KB_BYTES + p.a2_slots * p.a2_slot_bytes;
  const int stage_end = (fl::BLOCK_M * (r_pad + 4) * 4 + 1023) / 1024 * 1024;   // the accumulator's way out reuses the operand buffers
  p.bias_off = ring_end > stage_end ? ring_end : stage_end;
  const int smem_bytes = p.bias_off + fl::BIAS_BYTES + fl::BAR_BYTES + 1024;
  if (smem_bytes > fl::MAX_SMEM) return fail(ctx, FFSPLIT_ERR_SHAPE, "fused light chain: shared memory too small");
  if (!ctx->attr_fused_set) {
    cudaError_t e = cudaFuncSetAttribute(fl::fused_light_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         fl::MAX_SMEM);
    if (e != cudaSuccess) return check_cuda(ctx, e, "cudaFuncSetAttribute(fused_light_kernel)");
    ctx->attr_fused_set = true;
  }
  dim3 grid(p.splits, static_cast<unsigned>(tiles_m));
  const int ph = prof_open(ctx, PROF_GEMM_TC, algo_flops, st);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(fl::NUM_THREADS);
  cfg.dynamicSmemBytes = smem_bytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const cudaError_t le = cudaLaunchKernelEx(&cfg, fl::fused_light_kernel, tQ, tB1, tA2, p);
  prof_close(ctx, ph, st);
  ctx->launches++;
  return check_cuda(ctx, le, "fused_light_kernel launch");
}

}  // namespace ffsp
