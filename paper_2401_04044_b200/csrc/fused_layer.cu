// Whole split layer (Eq. 2) in one launch for small hidden widths: GELU layers in bf16 with d <= 1024,
// k_pad <= 256 and r_pad <= 256, at prefill token counts.
//
//     Y = sigma(X U1 + b1[heavy]) V1 + sigma((X A1) B1 + b1[light]) A2 B2 + b2
//
// A cluster of four CTAs owns one tile of 128 tokens.  Nothing but X, the weights and Y crosses HBM; the
// intermediate activations live in shared and tensor memory, and the one exchange between the CTAs of a
// cluster (the partial sums of the light part) goes through L2.  Per CTA (rank c of its cluster):
//   phase A   Q = X_tile A1                     tcgen05.mma, X and A1^T streamed through a ring of k-blocks;
//             Q -> bf16 -> shared memory, laid out as a K-major 128-byte-swizzled MMA operand
//   phase B   the light chain over this rank's quarter of the light neurons, as in fused_light.cu:
//             S = Q B1[:, chunk], H = GELU(S + b1) written back into tensor memory as bf16,
//             Pacc += H A2[chunk, :]
//   phase C   the fp32 partial Pacc goes to global memory; every rank adds the four partials of its
//             quarter of the r columns (in rank order) and stores bf16 P; every rank then reads the whole
//             P tile back into shared memory as an MMA operand.  Meanwhile the tensor pipe computes
//             A_H = X_tile U1, which the epilogue turns into GELU(A_H + b1[heavy]) -> bf16 -> shared memory
//   phase D   Y[:, c d/4 .. (c+1) d/4) = [P | A_H] [B2 ; V1] + b2, the weights of this rank's output
//             columns streamed through the same ring
// Warp roles: warp 0 TMA producer (rings of phases A, C, D; B1 and bias rings of phase B), warp 1 MMA
// issuer, warps 2-17 epilogue, warp 18 TMA producer of the A2 ring.
// CTAs of a cluster signal one another with remote mbarrier arrivals (release at cluster scope after a
// device-wide fence); every wait is bounded as in gemm_tc.cu.  All threads of a cluster meet at a
// cluster barrier after set-up (no remote arrival may reach an uninitialised barrier) and before exit
// (no CTA's shared memory may go away while a peer can still signal it); both are reached on every path.
#include "epilogue.cuh"
#include "internal.h"
#include "ptx.cuh"

namespace ffsp {

ffsplit_status get_tmap_bf16(ffsplit_ctx* ctx, const void* ptr, long long rows, long long cols, long long ld,
                             int box_rows, CUtensorMap* out);

namespace ly {

constexpr int CL = 4;              // CTAs per cluster = per token tile
constexpr int BLOCK_M = 128;
constexpr int CHUNK = 128;         // light neurons per chunk (N of GEMM-a, K of GEMM-b)
constexpr int KB = 64;             // K elements per shared-memory k-block (one 128-byte swizzle row)
constexpr int EPI_WARPS = 16;
constexpr int NUM_THREADS = 32 * (EPI_WARPS + 3);
constexpr int EPI_THREADS = 32 * EPI_WARPS;
constexpr int A2_WARP = EPI_WARPS + 2;
constexpr int MAX_B1_SLOTS = 8;
constexpr int MAX_A2_SLOTS = 6;
constexpr int MAX_RING = 4;
constexpr int BIAS_SLOTS = 8;
constexpr int TMEM_COLS = 512;
constexpr int TMEM_S0 = 256;       // S buffers at columns 256 and 384; Pacc at 0..255; Q, A_H and Y accumulators at 256..
constexpr int KB_BYTES = BLOCK_M * KB * 2;
constexpr int B1KB_BYTES = CHUNK * KB * 2;
constexpr int BIAS_BYTES = BIAS_SLOTS * CHUNK * 4 + 2 * 256 * 4;   // b1[light] ring, b1[heavy], b2 slice
constexpr int BAR_BYTES = 1024;
constexpr int MAX_SMEM = 232448;

struct Params {
  long long T;
  int d, k_pad, r_pad, ml_pad, kp_rp;
  int kbx, kbq, kbh;                // k-blocks of X (d / 64), of Q / P (ceil r_pad / 64), of A_H (ceil k_pad / 64)
  int n_chunks;
  int nq;                           // output columns per CTA, d / CL
  int hsplit;                       // wide heavy part (k_pad > 256): each rank computes k_pad / CL columns of A_H and
                                    // stores them to global memory; the last product streams A_H back by TMA
  int kq;                           // heavy columns this CTA computes: k_pad, or k_pad / CL when hsplit
  __nv_bfloat16* H; long long ldh;  // hsplit: A_H [T, ldh] in global memory
  int b1_slots, a2_slots, a2_slot_bytes;
  int ring_a_slots, ring_a_bytes;   // phase A ring: X k-block + A1^T k-block; starts right behind the Q region
  int ring_c_slots, ring_c_bytes;   // ring of phases C and D
  int ring_c_off;                   // its byte offset: behind the A_H region (behind the Q region when hsplit)
  int bias_off;                     // byte offset of the bias ring
  const float* b1h;
  const float* b1l;
  const float* b2;
  float4* partial;                  // per tile and rank: [r_pad / 4][128 rows] float4 (four columns of one row each)
  uint4* pbuf;                      // per tile: [r_pad / 8][128 rows] pieces of eight bf16 columns, the reduced light output
  __nv_bfloat16* Y; long long ldy;
  int act;
  int* status;
  const unsigned long long* guard;
  unsigned long long guard_hash;
};

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
__device__ __forceinline__ void bulk_load(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                   ptx::smem_u32(smem_dst)),
               "l"(gsrc), "r"(bytes), "r"(ptx::smem_u32(bar))
               : "memory");
}
// Generic-proxy writes to shared memory made visible to the tensor core's (async-proxy) reads.
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// One arrival on the barrier at the same shared-memory offset in CTA `cta` of this cluster.  Relaxed: the
// caller orders its earlier writes with a device-wide fence first (a release per arrival waits on the
// thread's outstanding writes every time: 0.8 us each, measured).
__device__ __forceinline__ void mbar_arrive_remote(uint64_t* bar, uint32_t cta) {
  uint32_t remote;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(remote) : "r"(ptx::smem_u32(bar)), "r"(cta));
  asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(remote) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n"
      ".reg .pred p;\n"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n"
      "selp.u32 %0, 1, 0, p;\n"
      "}\n"
      : "=r"(ok)
      : "r"(ptx::smem_u32(bar)), "r"(parity)
      : "memory");
  return ok != 0;
}
// Bounded wait on a barrier that peers of the cluster arrive on.
__device__ __forceinline__ bool mbar_wait_cluster(uint64_t* bar, uint32_t parity, volatile int* abort_flag) {
  if (mbar_try_wait_cluster(bar, parity)) return true;
  const long long t0 = clock64();
  int spins = 0;
  while (true) {
    if (mbar_try_wait_cluster(bar, parity)) return true;
    if ((++spins & 63) == 0) {
      if (*abort_flag) return false;
      if (clock64() - t0 > ptx::kWaitLimitCycles) {
        *abort_flag = 1;
        return false;
      }
    }
  }
}

// Position in a ring of `n` slots: slot index and the phase bit of its barriers, advanced without divisions
// (the single issuing thread of a role pays every instruction's latency in full).
struct Cursor {
  int slot = 0;
  uint32_t phase = 0;
  __device__ __forceinline__ void next(int n) {
    if (++slot == n) { slot = 0; phase ^= 1u; }
  }
};

// Byte offset of the 16-byte piece holding columns 8 j .. 8 j + 7 (j = 0..7) of row `row` inside one
// 128-row k-block of a K-major operand with 128-byte swizzle (what TMA writes and the MMA descriptor reads).
__device__ __forceinline__ int swz_piece(int row, int j) {
  return (row >> 3) * 1024 + (row & 7) * 128 + ((j ^ (row & 7)) << 4);
}

__global__ void __launch_bounds__(NUM_THREADS, 1)
fused_layer_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmA1,
                   const __grid_constant__ CUtensorMap tmU1, const __grid_constant__ CUtensorMap tmB1,
                   const __grid_constant__ CUtensorMap tmA2, const __grid_constant__ CUtensorMap tmW3,
                   const __grid_constant__ CUtensorMap tmH, const Params p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* smem_z = smem;                                   // Q, later P: kbq k-blocks
  uint8_t* smem_h1 = smem_z + p.kbq * KB_BYTES;             // A_H: kbh k-blocks (phases C, D); [P | A_H] is one operand
  uint8_t* ring_a = smem_h1;                                // phase A ring (A_H is not there yet)
  uint8_t* smem_b1 = smem_h1;                               // phase B rings, over the same bytes
  uint8_t* smem_a2 = smem_b1 + p.b1_slots * B1KB_BYTES;
  uint8_t* ring_c = smem + p.ring_c_off;                    // ring of phases C and D
  float* smem_bias = reinterpret_cast<float*>(smem + p.bias_off);
  float* smem_b1h = smem_bias + BIAS_SLOTS * CHUNK;          // [256] b1 of the heavy neurons
  float* smem_b2 = smem_b1h + 256;                           // [256] b2 of this rank's output columns
  uint64_t* bars = reinterpret_cast<uint64_t*>(reinterpret_cast<uint8_t*>(smem_bias) + BIAS_BYTES);
  uint64_t* b1full = bars;                       // [MAX_B1_SLOTS]
  uint64_t* b1empty = b1full + MAX_B1_SLOTS;     // [MAX_B1_SLOTS]
  uint64_t* a2full = b1empty + MAX_B1_SLOTS;     // [MAX_A2_SLOTS]
  uint64_t* a2empty = a2full + MAX_A2_SLOTS;     // [MAX_A2_SLOTS]
  uint64_t* biasfull = a2empty + MAX_A2_SLOTS;   // [BIAS_SLOTS]
  uint64_t* afull = biasfull + BIAS_SLOTS;       // [MAX_RING] phase A ring
  uint64_t* aempty = afull + MAX_RING;           // [MAX_RING]
  uint64_t* cfull = aempty + MAX_RING;           // [MAX_RING] ring of phases C, D
  uint64_t* cempty = cfull + MAX_RING;           // [MAX_RING]
  uint64_t* sfull = cempty + MAX_RING;           // [2] GEMM-a done -> epilogue
  uint64_t* hfull = sfull + 2;                   // [2] epilogue wrote H -> MMA
  uint64_t* qacc = hfull + 2;                    // [1] phase A MMAs complete
  uint64_t* qsmem = qacc + 1;                    // [1] epilogue wrote Q to shared memory
  uint64_t* pfull = qsmem + 1;                   // [1] all MMAs of phase B complete
  uint64_t* hacc = pfull + 1;                    // [1] A_H MMAs complete
  uint64_t* opfull = hacc + 1;                   // [1] epilogue wrote [P | A_H] to shared memory
  uint64_t* yacc = opfull + 1;                   // [1] phase D MMAs complete
  uint64_t* xbar1 = yacc + 1;                    // [1] all ranks stored their partial (remote arrivals)
  uint64_t* xbar2 = xbar1 + 1;                   // [1] all ranks stored their quarter of P (remote arrivals)
  uint64_t* xbar3 = xbar2 + 1;                   // [1] hsplit: all ranks stored their columns of A_H (remote arrivals)
  uint64_t* drain = xbar3 + 1;                   // [1]
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(drain + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;
  const int rank = static_cast<int>(cluster_rank());
  const int m_blk = blockIdx.y;
  const int c_begin = static_cast<int>(static_cast<long long>(p.n_chunks) * rank / CL);
  const int c_end = static_cast<int>(static_cast<long long>(p.n_chunks) * (rank + 1) / CL);
  const int my_chunks = c_end - c_begin;
  const int kb3 = p.kbq + p.kbh;                 // k-blocks of the last product

  if (threadIdx.x == 0) {
    for (int s = 0; s < MAX_B1_SLOTS; ++s) { ptx::mbar_init(&b1full[s], 1); ptx::mbar_init(&b1empty[s], 1); }
    for (int s = 0; s < MAX_A2_SLOTS; ++s) { ptx::mbar_init(&a2full[s], 1); ptx::mbar_init(&a2empty[s], 1); }
    for (int s = 0; s < BIAS_SLOTS; ++s) ptx::mbar_init(&biasfull[s], 1);
    for (int s = 0; s < MAX_RING; ++s) {
      ptx::mbar_init(&afull[s], 1); ptx::mbar_init(&aempty[s], 1);
      ptx::mbar_init(&cfull[s], 1); ptx::mbar_init(&cempty[s], 1);
    }
    for (int a = 0; a < 2; ++a) { ptx::mbar_init(&sfull[a], 1); ptx::mbar_init(&hfull[a], EPI_WARPS); }
    ptx::mbar_init(qacc, 1);
    ptx::mbar_init(qsmem, EPI_WARPS);
    ptx::mbar_init(pfull, 1);
    ptx::mbar_init(hacc, 1);
    ptx::mbar_init(opfull, EPI_WARPS);
    ptx::mbar_init(yacc, 1);
    ptx::mbar_init(xbar1, CL * EPI_WARPS);
    ptx::mbar_init(xbar2, CL * EPI_WARPS);
    ptx::mbar_init(xbar3, CL * EPI_WARPS);
    ptx::mbar_init(drain, 1);
    *abort_flag = 0;
    ptx::mbar_fence_init();
    ptx::prefetch_tmap(&tmX);
    ptx::prefetch_tmap(&tmA1);
    ptx::prefetch_tmap(&tmU1);
    ptx::prefetch_tmap(&tmB1);
    ptx::prefetch_tmap(&tmA2);
    ptx::prefetch_tmap(&tmW3);
    ptx::prefetch_tmap(&tmH);
  }
  if (warp == 1) {
    ptx::tmem_alloc(tmem_holder, TMEM_COLS);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_holder;
  // Programmatic launch: nothing below may touch global memory before the kernel ahead in the stream is
  // complete; the kernel behind may start its set-up once every CTA here holds its tensor memory.
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  if (warp == 0) {
    if (ptx::elect_one()) {
      // ------------------------------------------------------------ TMA producer: rings A, B1 + bias, C / D
      bool ok = true;
      // phase A: X k-block and the matching k-block of A1^T (r_pad rows)
      const uint32_t a_tx = KB_BYTES + p.r_pad * KB * 2;
      Cursor ca;
      for (int kb = 0; kb < p.kbx && ok; ++kb, ca.next(p.ring_a_slots)) {
        const int slot = ca.slot;
        if (!ptx::mbar_wait(&aempty[slot], ca.phase ^ 1u, abort_flag)) { ok = false; break; }
        ptx::mbar_expect_tx(&afull[slot], a_tx);
        uint8_t* dst = ring_a + slot * p.ring_a_bytes;
        ptx::tma_load_2d(&tmX, dst, &afull[slot], kb * KB, m_blk * BLOCK_M);
        ptx::tma_load_2d(&tmA1, dst + KB_BYTES, &afull[slot], kb * KB, 0);
      }
      // phase B: the rings lie over ring A, free once the MMAs of phase A are complete
      if (ok) ok = ptx::mbar_wait(qacc, 0, abort_flag);
      Cursor cb;
      for (int i = 0; i < my_chunks && ok; ++i) {
        const int chunk = c_begin + i;
        for (int kb = 0; kb < p.kbq; ++kb, cb.next(p.b1_slots)) {
          const int slot = cb.slot;
          if (!ptx::mbar_wait(&b1empty[slot], cb.phase ^ 1u, abort_flag)) { ok = false; break; }
          if (kb == 0) {
            const int n0 = chunk * CHUNK;
            const int cnt = p.ml_pad - n0 < CHUNK ? p.ml_pad - n0 : CHUNK;
            ptx::mbar_expect_tx(&biasfull[i % BIAS_SLOTS], cnt * 4);
            bulk_load(smem_bias + (i % BIAS_SLOTS) * CHUNK, p.b1l + n0, cnt * 4, &biasfull[i % BIAS_SLOTS]);
          }
          ptx::mbar_expect_tx(&b1full[slot], B1KB_BYTES);
          ptx::tma_load_2d(&tmB1, smem_b1 + slot * B1KB_BYTES, &b1full[slot], kb * KB, chunk * CHUNK);
        }
      }
      // phases C and D share one ring, which lies over the rings of phase B: wait for that phase's MMAs
      if (ok) ok = ptx::mbar_wait(pfull, 0, abort_flag);
      Cursor cc;
      const uint32_t c_tx = KB_BYTES + p.kq * KB * 2;
      for (int kb = 0; kb < p.kbx && ok; ++kb, cc.next(p.ring_c_slots)) {
        const int slot = cc.slot;
        if (!ptx::mbar_wait(&cempty[slot], cc.phase ^ 1u, abort_flag)) { ok = false; break; }
        ptx::mbar_expect_tx(&cfull[slot], c_tx);
        uint8_t* dst = ring_c + slot * p.ring_c_bytes;
        ptx::tma_load_2d(&tmX, dst, &cfull[slot], kb * KB, m_blk * BLOCK_M);
        ptx::tma_load_2d(&tmU1, dst + KB_BYTES, &cfull[slot], kb * KB, p.hsplit ? rank * p.kq : 0);
      }
      // phase D: k-blocks of [B2 ; V1]^T for this rank's output columns, in the operand's order [P | A_H]; with a
      // wide heavy part the matching k-block of A_H comes with them, from the global buffer all ranks wrote
      const uint32_t w_off = p.hsplit ? KB_BYTES : 0;
      const uint32_t d_tx = p.nq * KB * 2;
      bool h_ready = false;
      for (int b = 0; b < kb3 && ok; ++b, cc.next(p.ring_c_slots)) {
        const int slot = cc.slot;
        if (!ptx::mbar_wait(&cempty[slot], cc.phase ^ 1u, abort_flag)) { ok = false; break; }
        const bool hblk = p.hsplit && b >= p.kbq;
        if (hblk && !h_ready) {
          if (!mbar_wait_cluster(xbar3, 0, abort_flag)) { ok = false; break; }
          asm volatile("fence.proxy.async;" ::: "memory");   // the peers' generic-proxy stores before this thread's TMA reads
          h_ready = true;
        }
        ptx::mbar_expect_tx(&cfull[slot], d_tx + (hblk ? KB_BYTES : 0));
        const int x = b < p.kbq ? p.k_pad + b * KB : (b - p.kbq) * KB;
        uint8_t* dst = ring_c + slot * p.ring_c_bytes;
        if (hblk) ptx::tma_load_2d(&tmH, dst, &cfull[slot], x, m_blk * BLOCK_M);
        ptx::tma_load_2d(&tmW3, dst + w_off, &cfull[slot], x, rank * p.nq);
      }
      if (!ok) {
        // bounded chance for the copies in flight to land before the CTA goes away
        const long long t0 = clock64();
        while (clock64() - t0 < ptx::kWaitLimitCycles / 64) {}
      }
    }
    __syncwarp();
  } else if (warp == A2_WARP) {
    if (ptx::elect_one()) {
      // ------------------------------------------------------------ TMA producer: A2 ring
      bool ok = ptx::mbar_wait(qacc, 0, abort_flag);
      Cursor c2;
      for (int i = 0; i < my_chunks && ok; ++i) {
        for (int kb = 0; kb < CHUNK / KB; ++kb, c2.next(p.a2_slots)) {
          const int slot = c2.slot;
          if (!ptx::mbar_wait(&a2empty[slot], c2.phase ^ 1u, abort_flag)) { ok = false; break; }
          ptx::mbar_expect_tx(&a2full[slot], p.a2_slot_bytes);
          ptx::tma_load_2d(&tmA2, smem_a2 + slot * p.a2_slot_bytes, &a2full[slot], (c_begin + i) * CHUNK + kb * KB, 0);
        }
      }
      if (!ok) {
        const long long t0 = clock64();
        while (clock64() - t0 < ptx::kWaitLimitCycles / 64) {}
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    if (ptx::elect_one()) {
      // ------------------------------------------------------------ MMA issuer
      bool ok = true;
      // phase A: Q accumulator at TMEM_S0
      {
        const uint32_t idesc = ptx::umma_idesc_bf16(BLOCK_M, p.r_pad);
        Cursor ca;
        for (int kb = 0; kb < p.kbx && ok; ++kb, ca.next(p.ring_a_slots)) {
          const int slot = ca.slot;
          if (!ptx::mbar_wait(&afull[slot], ca.phase, abort_flag)) { ok = false; break; }
          ptx::tc_fence_after();
          const uint64_t a_desc = ptx::umma_desc_k128(ptx::smem_u32(ring_a + slot * p.ring_a_bytes));
          const uint64_t b_desc = ptx::umma_desc_k128(ptx::smem_u32(ring_a + slot * p.ring_a_bytes + KB_BYTES));
#pragma unroll
          for (int k = 0; k < KB / 16; ++k)
            ptx::umma_bf16(tmem_base + TMEM_S0, a_desc + 2 * k, b_desc + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
          ptx::umma_commit(&aempty[slot]);
        }
        if (ok) ptx::umma_commit(qacc);
      }
      // phase B: the light chain (Q now sits in shared memory as the left operand)
      if (ok) ok = ptx::mbar_wait(qsmem, 0, abort_flag);
      ptx::tc_fence_after();
      {
        const uint32_t idesc_a = ptx::umma_idesc_bf16(BLOCK_M, CHUNK);
        const uint32_t idesc_b = ptx::umma_idesc_bf16(BLOCK_M, p.r_pad);
        Cursor c2, cb;
        const uint64_t q_desc = ptx::umma_desc_k128(ptx::smem_u32(smem_z));
        const uint64_t b1_desc0 = ptx::umma_desc_k128(ptx::smem_u32(smem_b1));
        const uint64_t a2_desc0 = ptx::umma_desc_k128(ptx::smem_u32(smem_a2));
        auto gemm_b = [&](int j) -> bool {
          if (!ptx::mbar_wait(&hfull[j & 1], (j >> 1) & 1, abort_flag)) return false;
          ptx::tc_fence_after();
          const uint32_t h_tmem = tmem_base + TMEM_S0 + (j & 1) * CHUNK;
#pragma unroll
          for (int kb = 0; kb < CHUNK / KB; ++kb, c2.next(p.a2_slots)) {
            const int slot = c2.slot;
            if (!ptx::mbar_wait(&a2full[slot], c2.phase, abort_flag)) return false;
            ptx::tc_fence_after();
            const uint64_t b_desc = a2_desc0 + static_cast<uint64_t>((slot * p.a2_slot_bytes) >> 4);
#pragma unroll
            for (int k = 0; k < KB / 16; ++k) {
              const int jj = kb * (KB / 16) + k;
              umma_bf16_ts(tmem_base, h_tmem + 32 * (jj >> 1) + 8 * (jj & 1), b_desc + 2 * k, idesc_b,
                           (j | jj) != 0 ? 1u : 0u);
            }
            ptx::umma_commit(&a2empty[slot]);
          }
          return true;
        };
        for (int i = 0; i < my_chunks && ok; ++i) {
          const uint32_t d_tmem = tmem_base + TMEM_S0 + (i & 1) * CHUNK;
          for (int kb = 0; kb < p.kbq; ++kb, cb.next(p.b1_slots)) {
            const int slot = cb.slot;
            if (!ptx::mbar_wait(&b1full[slot], cb.phase, abort_flag)) { ok = false; break; }
            ptx::tc_fence_after();
            const uint64_t a_desc = q_desc + static_cast<uint64_t>((kb * KB_BYTES) >> 4);
            const uint64_t b_desc = b1_desc0 + static_cast<uint64_t>((slot * B1KB_BYTES) >> 4);
#pragma unroll
            for (int k = 0; k < KB / 16; ++k)   // Q's columns past r_pad are zero
              ptx::umma_bf16(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc_a, (kb | k) != 0 ? 1u : 0u);
            ptx::umma_commit(&b1empty[slot]);
          }
          if (!ok) break;
          ptx::umma_commit(&sfull[i & 1]);
          if (i > 0) ok = gemm_b(i - 1);
        }
        if (ok && my_chunks > 0) ok = gemm_b(my_chunks - 1);
        if (ok) ptx::umma_commit(pfull);
      }
      // phase C: A_H accumulator at TMEM_S0 (the S buffers' last reader was issued above)
      Cursor cc;
      if (ok) {
        const uint32_t idesc = ptx::umma_idesc_bf16(BLOCK_M, p.kq);
        for (int kb = 0; kb < p.kbx && ok; ++kb, cc.next(p.ring_c_slots)) {
          const int slot = cc.slot;
          if (!ptx::mbar_wait(&cfull[slot], cc.phase, abort_flag)) { ok = false; break; }
          ptx::tc_fence_after();
          const uint64_t a_desc = ptx::umma_desc_k128(ptx::smem_u32(ring_c + slot * p.ring_c_bytes));
          const uint64_t b_desc = ptx::umma_desc_k128(ptx::smem_u32(ring_c + slot * p.ring_c_bytes + KB_BYTES));
#pragma unroll
          for (int k = 0; k < KB / 16; ++k)
            ptx::umma_bf16(tmem_base + TMEM_S0, a_desc + 2 * k, b_desc + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
          ptx::umma_commit(&cempty[slot]);
        }
        if (ok) ptx::umma_commit(hacc);
      }
      // phase D: Y accumulator at TMEM_S0 once the epilogue has drained A_H and built [P | A_H]
      if (ok) ok = ptx::mbar_wait(opfull, 0, abort_flag);
      ptx::tc_fence_after();
      if (ok) {
        const uint32_t idesc = ptx::umma_idesc_bf16(BLOCK_M, p.nq);
        for (int b = 0; b < kb3 && ok; ++b, cc.next(p.ring_c_slots)) {
          const int slot = cc.slot;
          if (!ptx::mbar_wait(&cfull[slot], cc.phase, abort_flag)) { ok = false; break; }
          ptx::tc_fence_after();
          uint8_t* slot_p = ring_c + slot * p.ring_c_bytes;
          const bool hblk = p.hsplit && b >= p.kbq;     // A_H block streamed into the slot, in front of the weights
          const uint64_t a_desc = ptx::umma_desc_k128(ptx::smem_u32(hblk ? slot_p : smem_z + b * KB_BYTES));
          const uint64_t b_desc = ptx::umma_desc_k128(ptx::smem_u32(slot_p + (p.hsplit ? KB_BYTES : 0)));
#pragma unroll
          for (int k = 0; k < KB / 16; ++k)   // the operand's columns past r_pad and past k_pad are zero
            ptx::umma_bf16(tmem_base + TMEM_S0, a_desc + 2 * k, b_desc + 2 * k, idesc, (b | k) != 0 ? 1u : 0u);
          ptx::umma_commit(&cempty[slot]);
        }
        if (ok) ptx::umma_commit(yacc);
      }
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
    const int cg = (warp - 2) >> 2;      // column group 0..3
    const int row_in_tile = q * 32 + lane;
    const int te = threadIdx.x - 64;     // 0 .. 511
    const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
    const GeluCoef gc = gelu_coef(p.act);
    const long long row0 = static_cast<long long>(m_blk) * BLOCK_M;
    if (blockIdx.x == 0 && blockIdx.y == 0 && warp == 2) {
      Epilogue ge;
      ge.guard = p.guard;
      ge.guard_hash = p.guard_hash;
      check_blob_guard(ge, p.status, KID_FUSED);
    }
    // 16 accumulator columns of this thread's row -> bf16 -> two 16-byte pieces of a swizzled operand
    auto put16 = [&](uint8_t* region, int col0, const float* v) {
      const int kb = col0 >> 6, j = (col0 & 63) >> 3;
      uint4 a, b;
      a.x = pack_bf16x2(v[0], v[1]);   a.y = pack_bf16x2(v[2], v[3]);
      a.z = pack_bf16x2(v[4], v[5]);   a.w = pack_bf16x2(v[6], v[7]);
      b.x = pack_bf16x2(v[8], v[9]);   b.y = pack_bf16x2(v[10], v[11]);
      b.z = pack_bf16x2(v[12], v[13]); b.w = pack_bf16x2(v[14], v[15]);
      uint8_t* blk = region + kb * KB_BYTES;
      *reinterpret_cast<uint4*>(blk + swz_piece(row_in_tile, j)) = a;
      *reinterpret_cast<uint4*>(blk + swz_piece(row_in_tile, j + 1)) = b;
    };
    // b1[heavy] and this rank's slice of b2 into shared memory, long before they are needed
    if (te < p.kq) smem_b1h[te] = __ldg(p.b1h + (p.hsplit ? rank * p.kq : 0) + te);
    if (te < p.nq) smem_b2[te] = __ldg(p.b2 + rank * p.nq + te);
    asm volatile("bar.sync 1, %0;" ::"n"(EPI_THREADS) : "memory");
    bool ok = ptx::mbar_wait(qacc, 0, abort_flag);
    // ---- phase A: Q accumulator -> shared memory
    if (ok) {
      ptx::tc_fence_after();
      for (int c = cg * 16; c < p.kbq * KB; c += 128) {
        float v[2][16];
#pragma unroll
        for (int u = 0; u < 2; ++u)
          if (c + 64 * u < p.r_pad) ptx::tmem_ld16(t_lane + TMEM_S0 + c + 64 * u, v[u]);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          const int cc = c + 64 * u;
          if (cc >= p.kbq * KB) continue;
          if (cc >= p.r_pad) {
#pragma unroll
            for (int j = 0; j < 16; ++j) v[u][j] = 0.f;
          }
          put16(smem_z, cc, v[u]);
        }
      }
      fence_async_smem();
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(qsmem);
    }
    // ---- phase B: activation of each chunk, written back into tensor memory as bf16
    for (int i = 0; i < my_chunks && ok; ++i) {
      const int sb = i & 1;
      if (!ptx::mbar_wait(&biasfull[i % BIAS_SLOTS], (i / BIAS_SLOTS) & 1, abort_flag)) { ok = false; break; }
      if (!ptx::mbar_wait(&sfull[sb], (i >> 1) & 1, abort_flag)) { ok = false; break; }
      ptx::tc_fence_after();
      const uint32_t t_s = t_lane + TMEM_S0 + sb * CHUNK + cg * 32;
      const float* bias = smem_bias + (i % BIAS_SLOTS) * CHUNK + cg * 32;
      const int n0 = (c_begin + i) * CHUNK + cg * 32;
      uint32_t w[16];
      float v[2][16];
      ptx::tmem_ld16(t_s, v[0]);
      ptx::tmem_ld16(t_s + 16, v[1]);
      ptx::tmem_ld_wait();
#pragma unroll
      for (int hlf = 0; hlf < 2; ++hlf) {
        const bool inside = n0 + 16 * hlf + 16 <= p.ml_pad;   // ml_pad is a multiple of 16
        if (inside) {
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const float4 b = *reinterpret_cast<const float4*>(bias + 16 * hlf + 4 * j);
            v[hlf][4 * j] += b.x; v[hlf][4 * j + 1] += b.y; v[hlf][4 * j + 2] += b.z; v[hlf][4 * j + 3] += b.w;
          }
        }
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const float2 g2 = gelu_fast2(make_float2(v[hlf][2 * j], v[hlf][2 * j + 1]), gc);
          w[8 * hlf + j] = inside ? pack_bf16x2(g2.x, g2.y) : 0u;
        }
      }
      tmem_st16(t_s, w);
      tmem_st_wait();
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&hfull[sb]);
    }
    // ---- phase C: partial of the light part -> global, one arrival per warp on every rank's barrier
    if (ok) ok = ptx::mbar_wait(pfull, 0, abort_flag);
    if (ok) {
      ptx::tc_fence_after();
      // layout: float4 number (c / 4) * 128 + row holds columns c .. c + 3 of `row`, so that the 32 rows of a warp
      // make one contiguous 512-byte store and a rank's quarter of the columns is one contiguous range
      float4* mine = p.partial + (static_cast<long long>(m_blk) * CL + rank) * (p.r_pad / 4) * BLOCK_M;
      for (int c = cg * 16; c < p.r_pad; c += 128) {
        float v[2][16];
        if (my_chunks > 0) {
#pragma unroll
          for (int u = 0; u < 2; ++u)
            if (c + 64 * u < p.r_pad) ptx::tmem_ld16(t_lane + c + 64 * u, v[u]);
          ptx::tmem_ld_wait();
        } else {
#pragma unroll
          for (int u = 0; u < 2; ++u)
#pragma unroll
            for (int j = 0; j < 16; ++j) v[u][j] = 0.f;
        }
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          const int cc = c + 64 * u;
          if (cc >= p.r_pad) continue;
#pragma unroll
          for (int j = 0; j < 4; ++j)
            mine[((cc >> 2) + j) * BLOCK_M + row_in_tile] =
                make_float4(v[u][4 * j], v[u][4 * j + 1], v[u][4 * j + 2], v[u][4 * j + 3]);
        }
      }
      __threadfence();
      __syncwarp();
      if (lane == 0)
        for (int c = 0; c < CL; ++c) mbar_arrive_remote(xbar1, c);
      ok = mbar_wait_cluster(xbar1, 0, abort_flag);
    }
    if (ok) {
      // this rank's quarter of the r columns: the four partials added in rank order, stored as bf16.  All loads
      // of a batch are issued before the first is used.
      const int q4 = p.r_pad / (4 * CL);            // float4 per row in a quarter
      const int n4 = BLOCK_M * q4;
      const float4* src = p.partial + static_cast<long long>(m_blk) * CL * (p.r_pad / 4) * BLOCK_M + rank * n4;
      const long long rstride = static_cast<long long>(p.r_pad / 4) * BLOCK_M;
      uint2* dst = reinterpret_cast<uint2*>(p.pbuf + static_cast<long long>(m_blk) * (p.r_pad / 8) * BLOCK_M);
      constexpr int EB = 3;
      for (int e0 = te; e0 < n4; e0 += EB * EPI_THREADS) {
        float4 buf[EB][CL];
#pragma unroll
        for (int u = 0; u < EB; ++u) {
          const int e = e0 + u * EPI_THREADS;
#pragma unroll
          for (int s = 0; s < CL; ++s)
            buf[u][s] = e < n4 ? __ldcg(src + s * rstride + e) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
#pragma unroll
        for (int u = 0; u < EB; ++u) {
          const int e = e0 + u * EPI_THREADS;
          if (e >= n4) continue;
          float4 acc = buf[u][0];
#pragma unroll
          for (int s = 1; s < CL; ++s) { acc.x += buf[u][s].x; acc.y += buf[u][s].y; acc.z += buf[u][s].z; acc.w += buf[u][s].w; }
          const int c4 = rank * q4 + e / BLOCK_M, r = e % BLOCK_M;     // column quad, row
          uint2 o;
          o.x = pack_bf16x2(acc.x, acc.y);
          o.y = pack_bf16x2(acc.z, acc.w);
          dst[((c4 >> 1) * BLOCK_M + r) * 2 + (c4 & 1)] = o;
        }
      }
      __threadfence();
      __syncwarp();
      if (lane == 0)
        for (int c = 0; c < CL; ++c) mbar_arrive_remote(xbar2, c);
    }
    // ---- A_H accumulator -> bias, GELU -> shared memory (behind P in the operand of the last product)
    if (ok) ok = ptx::mbar_wait(hacc, 0, abort_flag);
    if (ok) {
      ptx::tc_fence_after();
      const int hcols = p.hsplit ? p.kq : p.kbh * KB;      // columns to walk: this rank's slice, or the padded operand
      for (int c = cg * 16; c < hcols; c += 128) {
        float v[2][16];
#pragma unroll
        for (int u = 0; u < 2; ++u)
          if (c + 64 * u < p.kq) ptx::tmem_ld16(t_lane + TMEM_S0 + c + 64 * u, v[u]);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          const int cc = c + 64 * u;
          if (cc >= hcols) continue;
          if (cc < p.kq) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
              const float4 t = *reinterpret_cast<const float4*>(smem_b1h + cc + 4 * j);
              v[u][4 * j] += t.x; v[u][4 * j + 1] += t.y; v[u][4 * j + 2] += t.z; v[u][4 * j + 3] += t.w;
            }
            gelu_fast16(v[u], gc);
          } else {
#pragma unroll
            for (int j = 0; j < 16; ++j) v[u][j] = 0.f;
          }
          if (!p.hsplit) {
            put16(smem_h1, cc, v[u]);
          } else if (row0 + row_in_tile < p.T) {
            uint4 a, bb;
            a.x = pack_bf16x2(v[u][0], v[u][1]);    a.y = pack_bf16x2(v[u][2], v[u][3]);
            a.z = pack_bf16x2(v[u][4], v[u][5]);    a.w = pack_bf16x2(v[u][6], v[u][7]);
            bb.x = pack_bf16x2(v[u][8], v[u][9]);   bb.y = pack_bf16x2(v[u][10], v[u][11]);
            bb.z = pack_bf16x2(v[u][12], v[u][13]); bb.w = pack_bf16x2(v[u][14], v[u][15]);
            uint4* dst = reinterpret_cast<uint4*>(p.H + (row0 + row_in_tile) * p.ldh + rank * p.kq + cc);
            dst[0] = a;
            dst[1] = bb;
          }
        }
      }
      if (p.hsplit) {
        __threadfence();
        __syncwarp();
        if (lane == 0)
          for (int c = 0; c < CL; ++c) mbar_arrive_remote(xbar3, c);
      }
      ok = mbar_wait_cluster(xbar2, 0, abort_flag);
    }
    if (ok) {
      // the whole P tile, bf16, into the operand layout; pieces past r_pad are zero
      const int n8 = p.kbq * 8 * BLOCK_M, real8 = (p.r_pad >> 3) * BLOCK_M;
      const uint4* src = p.pbuf + static_cast<long long>(m_blk) * (p.r_pad / 8) * BLOCK_M;
      constexpr int PB = 4;
      for (int e0 = te; e0 < n8; e0 += PB * EPI_THREADS) {
        uint4 buf[PB];
#pragma unroll
        for (int u = 0; u < PB; ++u) {
          const int e = e0 + u * EPI_THREADS;
          buf[u] = e < real8 ? __ldcg(src + e) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int u = 0; u < PB; ++u) {
          const int e = e0 + u * EPI_THREADS;
          if (e >= n8) continue;
          const int j8 = e / BLOCK_M, r = e % BLOCK_M;
          *reinterpret_cast<uint4*>(smem_z + (j8 >> 3) * KB_BYTES + swz_piece(r, j8 & 7)) = buf[u];
        }
      }
      fence_async_smem();
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(opfull);
      ok = ptx::mbar_wait(yacc, 0, abort_flag);
    }
    // ---- phase D: Y accumulator -> + b2 -> bf16 -> global
    if (ok) {
      ptx::tc_fence_after();
      const long long row = row0 + row_in_tile;
      for (int c = cg * 16; c < p.nq; c += 128) {
        float v[2][16];
#pragma unroll
        for (int u = 0; u < 2; ++u)
          if (c + 64 * u < p.nq) ptx::tmem_ld16(t_lane + TMEM_S0 + c + 64 * u, v[u]);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int u = 0; u < 2; ++u) {
          const int cc = c + 64 * u;
          if (cc >= p.nq || row >= p.T) continue;
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const float4 t = *reinterpret_cast<const float4*>(smem_b2 + cc + 4 * j);
            v[u][4 * j] += t.x; v[u][4 * j + 1] += t.y; v[u][4 * j + 2] += t.z; v[u][4 * j + 3] += t.w;
          }
          uint4 a, bb;
          a.x = pack_bf16x2(v[u][0], v[u][1]);    a.y = pack_bf16x2(v[u][2], v[u][3]);
          a.z = pack_bf16x2(v[u][4], v[u][5]);    a.w = pack_bf16x2(v[u][6], v[u][7]);
          bb.x = pack_bf16x2(v[u][8], v[u][9]);   bb.y = pack_bf16x2(v[u][10], v[u][11]);
          bb.z = pack_bf16x2(v[u][12], v[u][13]); bb.w = pack_bf16x2(v[u][14], v[u][15]);
          __nv_bfloat16* dst = p.Y + row * p.ldy + rank * p.nq + cc;
          if ((reinterpret_cast<uintptr_t>(dst) & 31u) == 0) {
            // one whole 32-byte sector per lane and instruction
            asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(dst), "r"(a.x), "r"(a.y),
                         "r"(a.z), "r"(a.w), "r"(bb.x), "r"(bb.y), "r"(bb.z), "r"(bb.w)
                         : "memory");
          } else {
            reinterpret_cast<uint4*>(dst)[0] = a;
            reinterpret_cast<uint4*>(dst)[1] = bb;
          }
        }
      }
    }
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) record_status(p.status, FFSPLIT_ERR_TIMEOUT, blockIdx.y * CL + rank, KID_FUSED);
  __syncwarp();
  cluster_sync_all();
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

}  // namespace ly

namespace {
struct LayerPlan {
  int b1_slots, a2_slots, ring_a_slots, ring_a_bytes, ring_c_slots, ring_c_bytes, ring_c_off, bias_off, smem_bytes;
  bool ok;
};
// hsplit: the heavy part is wider than one accumulator; each rank computes k_pad / CL of its columns and the
// operand of the last product is streamed from global memory instead of being held in shared memory.
bool layer_hsplit(int k_pad) { return k_pad > 256; }
LayerPlan plan_layer(int d, int k_pad, int r_pad) {
  LayerPlan L{};
  const bool hsplit = layer_hsplit(k_pad);
  const int kq = hsplit ? k_pad / ly::CL : k_pad;
  const int kbq = (r_pad + ly::KB - 1) / ly::KB, kbh = (k_pad + ly::KB - 1) / ly::KB;
  const int nq = d / ly::CL;
  const int z_bytes = kbq * ly::KB_BYTES, h_bytes = hsplit ? 0 : kbh * ly::KB_BYTES;
  const int tail = ly::BIAS_BYTES + ly::BAR_BYTES;
  const int avail = ly::MAX_SMEM - 1024 - z_bytes - tail;   // behind the Q region, before the bias ring
  // phase A ring
  L.ring_a_bytes = ly::KB_BYTES + r_pad * ly::KB * 2;
  L.ring_a_slots = avail / L.ring_a_bytes;
  if (L.ring_a_slots > ly::MAX_RING) L.ring_a_slots = ly::MAX_RING;
  // ring of phases C and D, behind the A_H region
  int cb = ly::KB_BYTES + kq * ly::KB * 2;
  const int db = (hsplit ? ly::KB_BYTES : 0) + nq * ly::KB * 2;
  if (db > cb) cb = db;
  L.ring_c_bytes = (cb + 1023) / 1024 * 1024;
  L.ring_c_off = z_bytes + h_bytes;
  L.ring_c_slots = (avail - h_bytes) / L.ring_c_bytes;
  if (L.ring_c_slots > ly::MAX_RING) L.ring_c_slots = ly::MAX_RING;
  // rings of phase B, balanced in units of chunks
  const int a2_slot = r_pad * ly::KB * 2;
  double best = -1.0;
  for (int nb = 1; nb <= ly::MAX_B1_SLOTS; ++nb)
    for (int na = 1; na <= ly::MAX_A2_SLOTS; ++na) {
      if (nb * ly::B1KB_BYTES + na * a2_slot > avail) continue;
      const double a = static_cast<double>(nb) / kbq, b = static_cast<double>(na) / 2.0;
      const double score = (a < b ? a : b) + 1e-3 * (a + b);
      if (score > best) { best = score; L.b1_slots = nb; L.a2_slots = na; }
    }
  L.bias_off = z_bytes + avail;
  L.smem_bytes = L.bias_off + tail + 1024;
  L.ok = L.ring_a_slots >= 2 && L.ring_c_slots >= 2 && L.b1_slots >= 1 && L.a2_slots >= 2 && L.smem_bytes <= ly::MAX_SMEM;
  return L;
}
}  // namespace

// The one-launch layer takes GELU layers in bf16 whose hidden width splits into four column blocks of at most
// 256 and whose heavy and light widths each fit one accumulator.
// A cluster walks its phases one after the other, so the launch pays off while all clusters are resident at once
// (measured on the BERT-base shape: 31 us per layer up to 4096 tokens against 43 us for the three-launch path, but
// 125 us against 82 us at 16 384 tokens, where the clusters take four turns).
bool fused_layer_applies(int dtype, int act, int d, int k, int k_pad, int r_pad, int ml_pad, long long T, int num_sms) {
  if (dtype != FFSPLIT_BF16 || act == FFSPLIT_SWIGLU) return false;
  if (k < 1 || r_pad < 16 || r_pad > 256 || ml_pad < 1) return false;
  if (k_pad > 256 && (k_pad % (16 * ly::CL) != 0 || k_pad > 256 * ly::CL)) return false;   // wide heavy part: equal column slices
  if (d % 64 != 0 || d / ly::CL > 256 || d / ly::CL < 16) return false;
  if (T <= 64 || (T + ly::BLOCK_M - 1) / ly::BLOCK_M * ly::CL > num_sms) return false;
  return plan_layer(d, k_pad, r_pad).ok;
}

// fp32 partials of the light part (one per rank) and its reduced bf16 form, per token tile
size_t fused_layer_scratch_bytes(long long T, int r_pad) {
  const long long tiles_m = (T + ly::BLOCK_M - 1) / ly::BLOCK_M;
  return static_cast<size_t>(tiles_m) * ly::BLOCK_M * r_pad * (ly::CL * 4 + 2);
}

ffsplit_status launch_fused_layer(ffsplit_ctx* ctx, const BlobHeader& h, const char* blob, const void* X, long long T,
                                  char* scratch, void* H, long long ldh, void* Y, unsigned long long guard_hash,
                                  cudaStream_t st) {
  const int d = h.d, k_pad = h.k_pad, r_pad = h.r_pad, ml_pad = h.ml_pad, kp_rp = h.k_pad + h.r_pad;
  const LayerPlan L = plan_layer(d, k_pad, r_pad);
  if (!L.ok) return fail(ctx, FFSPLIT_ERR_SHAPE, "one-launch layer: shared memory too small");
  ly::Params p;
  p.T = T;
  p.d = d; p.k_pad = k_pad; p.r_pad = r_pad; p.ml_pad = ml_pad; p.kp_rp = kp_rp;
  p.kbx = d / ly::KB;
  p.kbq = (r_pad + ly::KB - 1) / ly::KB;
  p.kbh = (k_pad + ly::KB - 1) / ly::KB;
  p.n_chunks = (ml_pad + ly::CHUNK - 1) / ly::CHUNK;
  p.nq = d / ly::CL;
  p.b1_slots = L.b1_slots; p.a2_slots = L.a2_slots; p.a2_slot_bytes = r_pad * ly::KB * 2;
  p.ring_a_slots = L.ring_a_slots; p.ring_a_bytes = L.ring_a_bytes;
  p.ring_c_slots = L.ring_c_slots; p.ring_c_bytes = L.ring_c_bytes; p.ring_c_off = L.ring_c_off;
  p.hsplit = layer_hsplit(k_pad) ? 1 : 0;
  p.kq = p.hsplit ? k_pad / ly::CL : k_pad;
  p.H = static_cast<__nv_bfloat16*>(H); p.ldh = ldh;
  p.bias_off = L.bias_off;
  p.b1h = reinterpret_cast<const float*>(blob + h.off[SEC_B1H]);
  p.b1l = reinterpret_cast<const float*>(blob + h.off[SEC_B1L]);
  p.b2 = reinterpret_cast<const float*>(blob + h.off[SEC_B2]);
  const long long tiles_m = (T + ly::BLOCK_M - 1) / ly::BLOCK_M;
  p.partial = reinterpret_cast<float4*>(scratch);
  p.pbuf = reinterpret_cast<uint4*>(scratch + static_cast<size_t>(tiles_m) * ly::BLOCK_M * r_pad * ly::CL * 4);
  p.Y = static_cast<__nv_bfloat16*>(Y); p.ldy = d;
  p.act = h.act;
  p.status = ctx->status();
  p.guard = guard_hash ? reinterpret_cast<const unsigned long long*>(blob) : nullptr;
  p.guard_hash = guard_hash;
  const char* u1t = blob + h.off[SEC_U1T];
  CUtensorMap tX, tA1, tU1, tB1, tA2, tW3, tH;
  ffsplit_status s;
  if ((s = get_tmap_bf16(ctx, X, T, d, d, ly::BLOCK_M, &tX)) != FFSPLIT_OK) return s;
  if ((s = get_tmap_bf16(ctx, u1t + static_cast<size_t>(k_pad) * d * 2, r_pad, d, d, r_pad, &tA1)) != FFSPLIT_OK) return s;
  if ((s = get_tmap_bf16(ctx, u1t, k_pad, d, d, p.kq, &tU1)) != FFSPLIT_OK) return s;
  if ((s = get_tmap_bf16(ctx, blob + h.off[SEC_B1T], ml_pad, r_pad, r_pad, ly::CHUNK, &tB1)) != FFSPLIT_OK) return s;
  if ((s = get_tmap_bf16(ctx, blob + h.off[SEC_A2T], r_pad, ml_pad, ml_pad, r_pad, &tA2)) != FFSPLIT_OK) return s;
  if ((s = get_tmap_bf16(ctx, blob + h.off[SEC_V1B2T], d, kp_rp, kp_rp, p.nq, &tW3)) != FFSPLIT_OK) return s;
  // (without hsplit the kernel never uses this map; it is given a valid one all the same)
  if ((s = get_tmap_bf16(ctx, H, T, k_pad, ldh, ly::BLOCK_M, &tH)) != FFSPLIT_OK) return s;
  if (!ctx->attr_layer_set) {
    cudaError_t e = cudaFuncSetAttribute(ly::fused_layer_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         ly::MAX_SMEM);
    if (e != cudaSuccess) return check_cuda(ctx, e, "cudaFuncSetAttribute(fused_layer_kernel)");
    ctx->attr_layer_set = true;
  }
  const double flops = 2.0 * T * (2.0 * d * (h.k + h.r) + 2.0 * h.r * h.ml);
  const int ph = prof_open(ctx, PROF_GEMM_TC, flops, st);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(ly::CL, static_cast<unsigned>(tiles_m));
  cfg.blockDim = dim3(ly::NUM_THREADS);
  cfg.dynamicSmemBytes = L.smem_bytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = ly::CL;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  const cudaError_t le = cudaLaunchKernelEx(&cfg, ly::fused_layer_kernel, tX, tA1, tU1, tB1, tA2, tW3, tH, p);
  prof_close(ctx, ph, st);
  ctx->launches++;
  return check_cuda(ctx, le, "fused_layer_kernel launch");
}

}  // namespace ffsp
