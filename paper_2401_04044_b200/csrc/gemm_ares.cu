// Tensor-core GEMM for a short contraction with the row operand resident in tensor memory:
//
//     C[M, N] = act(A[M, K] B[N, K]^T + bias)        bf16 in, fp32 accumulate, bf16 out, K <= 512
//
// This is the first product of the unfused light chain of Eq. 2, H_L = sigma(Q B1 + b1[light]) with Q [T, r]
// and B1^T [mL, r]: 4096 x 19456 x 512 on the OPT-13B-shaped layer.  With both operands in shared memory a
// 128 x 256 tile needs, per 64-deep k-block, 48 KB written by TMA and 48 KB read by the MMAs in the 512 clocks
// the MMAs take: 187 bytes per clock against the 128 the shared memory of an SM delivers.  Here the 128 x K
// block of A is copied once into tensor memory (two bf16 per 32-bit cell, K / 2 columns) and stays there while
// the CTA walks along N: the MMAs read A from tensor memory and shared memory carries the B tiles only.
//
// Tiles are 128 x 128 and numbered row block by row block; CTA c takes the contiguous range
// [c * tiles / G, (c + 1) * tiles / G), so it changes its row block at most a few times.  Warp roles: warp 0
// TMA producer of the B ring (stages of two k-blocks), warp 1 MMA issuer, warps 2-17 epilogue: two sets of
// eight warps, one per accumulator buffer (even and odd tiles), each warp 32 rows x 64 columns -- the epilogue
// warps also copy A: each thread reads its own row from global memory and stores it into the quarter's lanes.
//
// The output leaves through TMA stores: a lane holds one row (that is how tensor memory is read), so each warp
// writes its 32 x 64 block into 4 KB of shared memory of its own, in the 128-byte swizzle the output's tensor map
// expects (no bank conflicts, no barrier beyond the warp's own), and one lane stores the block with one
// cp.async.bulk.tensor; it waits for that store to have read the buffer only when the warp next writes it, two
// tiles later.
//
// What bounds this product is its output.  Measured on the shape above (single launches): the general GEMM, 32
// bytes per lane straight from the registers, 98.4 us; the same block turned through the warp's buffer and
// written as whole 128-byte lines by ordinary stores 95.6 us; through TMA stores 81.4-83.1 us (tensor pipe 51 ->
// 61 % active); either of the first two without its stores (a working copy) about 47 us -- a plain fill of the
// same 159 MB takes 47 us (3.4 TB/s).  Bit-identical to the general GEMM.
// Every wait is bounded (see gemm_tc.cu).
#include "epilogue.cuh"
#include "internal.h"
#include "ptx.cuh"

namespace ffsp {

ffsplit_status get_tmap_bf16(ffsplit_ctx* ctx, const void* ptr, long long rows, long long cols, long long ld,
                             int box_rows, CUtensorMap* out);

namespace ar {

constexpr int BLOCK_M = 128;
constexpr int BLOCK_N = 128;
constexpr int KB = 64;                              // one 128-byte swizzle row of bf16
constexpr int KB_BYTES = BLOCK_N * KB * 2;          // 16 KB
constexpr int STAGE_KB = 2;                         // k-blocks per ring stage
constexpr int STAGE_BYTES = STAGE_KB * KB_BYTES;
constexpr int MAX_STAGES = 5;
constexpr int MAX_K = 512;
constexpr int EPI_WARPS = 16;
constexpr int NUM_THREADS = 32 * (EPI_WARPS + 2);
constexpr int TMEM_COLS = 512;
constexpr int TMEM_ACC0 = 256;                      // A in columns 0 .. K / 2 - 1, accumulators at 256 and 384
constexpr int BAR_BYTES = 512;
constexpr int TURN_BYTES = 32 * 128;                // one warp's 32 rows x 64 bf16 on their way out
constexpr int SMEM_BYTES = MAX_STAGES * STAGE_BYTES + EPI_WARPS * TURN_BYTES + BAR_BYTES + 1024;

struct Params {
  long long M;
  int N, K;
  int nkb;               // ceil(K / 64)
  int tiles_n;
  long long tiles;       // tiles_m * tiles_n
  const __nv_bfloat16* A;
  long long lda;
  Epilogue epi;
  int* status;
};

struct Cursor {
  int slot = 0;
  uint32_t phase = 0;
  __device__ __forceinline__ void next(int n) {
    if (++slot == n) { slot = 0; phase ^= 1u; }
  }
};

// D[tmem] (+)= A[tmem] * B[smem desc]: A is a 128 x 16 bf16 slab held as 8 columns of tensor memory.
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

__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_ares_kernel(const __grid_constant__ CUtensorMap tmB, const __grid_constant__ CUtensorMap tmC, const Params p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* smem_turn = smem + MAX_STAGES * STAGE_BYTES;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem_turn + EPI_WARPS * TURN_BYTES);
  uint64_t* full = bars;                    // [MAX_STAGES] TMA -> MMA
  uint64_t* empty = full + MAX_STAGES;      // [MAX_STAGES] MMA -> TMA
  uint64_t* tfull = empty + MAX_STAGES;     // [2] MMA -> epilogue: an accumulator is complete
  uint64_t* tempty = tfull + 2;             // [2] epilogue -> MMA: an accumulator has been read
  uint64_t* afull = tempty + 2;             // [1] epilogue -> MMA: the row block of A is in tensor memory
  uint64_t* afree = afull + 1;              // [1] MMA -> epilogue: every MMA that reads it has completed
  uint64_t* drain = afree + 1;              // [1] used only when giving up
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(drain + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < MAX_STAGES; ++s) { ptx::mbar_init(&full[s], 1); ptx::mbar_init(&empty[s], 1); }
    for (int a = 0; a < 2; ++a) { ptx::mbar_init(&tfull[a], 1); ptx::mbar_init(&tempty[a], EPI_WARPS / 2); }
    ptx::mbar_init(afull, EPI_WARPS);
    ptx::mbar_init(afree, 1);
    ptx::mbar_init(drain, 1);
    *abort_flag = 0;
    ptx::mbar_fence_init();
    ptx::prefetch_tmap(&tmB);
  }
  if (warp == 1) {
    ptx::tmem_alloc(tmem_holder, TMEM_COLS);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_holder;
  // programmatic launch: the set-up above ran under the tail of the kernel before; A is that kernel's output
  asm volatile("griddepcontrol.wait;" ::: "memory");
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

  const long long t_begin = p.tiles * blockIdx.x / gridDim.x;
  const long long t_end = p.tiles * (blockIdx.x + 1) / gridDim.x;
  const int n_stage = (p.nkb + STAGE_KB - 1) / STAGE_KB;      // ring stages per tile

  if (warp == 0) {
    if (ptx::elect_one()) {
      // ------------------------------------------------------------ TMA producer: B tiles of every tile in turn
      Cursor cur;
      bool ok = true;
      long long issued = 0;
      int n_blk = static_cast<int>(t_begin % p.tiles_n);
      for (long long t = t_begin; t < t_end && ok; ++t) {
        for (int sg = 0; sg < n_stage; ++sg, cur.next(MAX_STAGES), ++issued) {
          if (!ptx::mbar_wait(&empty[cur.slot], cur.phase ^ 1u, abort_flag)) { ok = false; break; }
          const int kbs = p.nkb - sg * STAGE_KB < STAGE_KB ? p.nkb - sg * STAGE_KB : STAGE_KB;
          ptx::mbar_expect_tx(&full[cur.slot], kbs * KB_BYTES);
          for (int j = 0; j < kbs; ++j)
            ptx::tma_load_2d(&tmB, smem + cur.slot * STAGE_BYTES + j * KB_BYTES, &full[cur.slot], (sg * STAGE_KB + j) * KB,
                             n_blk * BLOCK_N);
        }
        if (++n_blk == p.tiles_n) n_blk = 0;
      }
      if (!ok) {
        // give the copies already issued a bounded chance to land before the CTA exits
        const long long first = issued > MAX_STAGES ? issued - MAX_STAGES : 0;
        for (long long j = first; j < issued; ++j) {
          const long long t0 = clock64();
          while (!ptx::mbar_try_wait(&full[j % MAX_STAGES], (j / MAX_STAGES) & 1) &&
                 clock64() - t0 < ptx::kWaitLimitCycles / 8) {}
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    if (ptx::elect_one()) {
      // ------------------------------------------------------------ MMA issuer
      const uint32_t idesc = ptx::umma_idesc_bf16(BLOCK_M, BLOCK_N);
      const uint64_t b_desc0 = ptx::umma_desc_k128(ptx::smem_u32(smem));
      Cursor cur;
      bool ok = true;
      uint32_t tl = 0, seg = 0;
      int n_blk = static_cast<int>(t_begin % p.tiles_n);
      for (long long t = t_begin; t < t_end && ok; ++t, ++tl) {
        if (t == t_begin || n_blk == 0) {
          // a new row block: its A must have arrived in tensor memory
          if (!ptx::mbar_wait(afull, seg & 1, abort_flag)) { ok = false; break; }
          ptx::tc_fence_after();
          ++seg;
        }
        const uint32_t acc = tl & 1, aph = (tl >> 1) & 1;
        if (!ptx::mbar_wait(&tempty[acc], aph ^ 1, abort_flag)) { ok = false; break; }
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + TMEM_ACC0 + acc * BLOCK_N;
        for (int sg = 0; sg < n_stage; ++sg, cur.next(MAX_STAGES)) {
          if (!ptx::mbar_wait(&full[cur.slot], cur.phase, abort_flag)) { ok = false; break; }
          ptx::tc_fence_after();
          const int kbs = p.nkb - sg * STAGE_KB < STAGE_KB ? p.nkb - sg * STAGE_KB : STAGE_KB;
          const uint64_t b_desc = b_desc0 + static_cast<uint32_t>(cur.slot) * (STAGE_BYTES >> 4);
          for (int j = 0; j < kbs; ++j) {
            const int kb = sg * STAGE_KB + j;
#pragma unroll
            for (int k = 0; k < KB / 16; ++k)   // slab kb * 4 + k of A: 8 columns each
              umma_bf16_ts(d_tmem, tmem_base + (kb * (KB / 16) + k) * 8, b_desc + j * (KB_BYTES >> 4) + 2 * k, idesc,
                           (kb | k) != 0 ? 1u : 0u);
          }
          ptx::umma_commit(&empty[cur.slot]);
        }
        if (!ok) break;
        ptx::umma_commit(&tfull[acc]);
        if (++n_blk == p.tiles_n) n_blk = 0;
        if (n_blk == 0 && t + 1 < t_end) ptx::umma_commit(afree);   // the next tile belongs to another row block
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
    const int q = warp & 3;              // tensor-memory lane quarter
    const int cg = (warp - 2) >> 2;      // which quarter of K this warp copies when A changes
    const uint32_t set = static_cast<uint32_t>(warp - 2) >> 3;   // which accumulator buffer (tile parity) this warp reads
    const int ch = ((warp - 2) >> 2) & 1;                        // which 64 of the tile's 128 columns
    uint8_t* turn = smem_turn + (warp - 2) * TURN_BYTES;
    const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
    const GeluCoef gc = gelu_coef(p.epi.act);
    const Epilogue& e = p.epi;
    if (blockIdx.x == 0 && warp == 2) check_blob_guard(e, p.status, KID_GEMM_AR);
    bool live = true;
    uint32_t tl = 0, seg = 0;
    int n_blk = static_cast<int>(t_begin % p.tiles_n);
    long long m_blk = t_begin / p.tiles_n;
    for (long long t = t_begin; t < t_end && live; ++t, ++tl) {
      if (t == t_begin || n_blk == 0) {
        // ---- copy this row block of A into tensor memory: this thread's row, this warp's quarter of K
        if (seg > 0 && !ptx::mbar_wait(afree, (seg - 1) & 1, abort_flag)) { live = false; break; }
        ptx::tc_fence_after();
        const long long row = m_blk * BLOCK_M + q * 32 + lane;
        const int kq = p.nkb * (KB / 4);                  // elements per warp: a quarter of the padded K
        const __nv_bfloat16* src = p.A + row * p.lda + cg * kq;
        for (int c0 = 0; c0 < kq; c0 += 32) {             // 32 elements = 16 columns per store
          uint32_t w[16];
#pragma unroll
          for (int j = 0; j < 4; ++j) {
            const int kk = cg * kq + c0 + 8 * j;           // K is a multiple of 8: a 16-byte piece is inside or outside
            uint4 v = make_uint4(0u, 0u, 0u, 0u);
            if (row < p.M && kk < p.K) v = __ldg(reinterpret_cast<const uint4*>(src + c0 + 8 * j));
            w[4 * j] = v.x; w[4 * j + 1] = v.y; w[4 * j + 2] = v.z; w[4 * j + 3] = v.w;
          }
          tmem_st16(t_lane + ((cg * kq + c0) >> 1), w);
        }
        tmem_st_wait();
        ptx::tc_fence_before();
        __syncwarp();
        if (lane == 0) ptx::mbar_arrive(afull);
        ++seg;
      }
      const uint32_t acc = tl & 1, aph = (tl >> 1) & 1;
      if (acc == set) {
        if (!ptx::mbar_wait(&tfull[acc], aph, abort_flag)) { live = false; break; }
        ptx::tc_fence_after();
        const uint32_t t_acc = t_lane + TMEM_ACC0 + acc * BLOCK_N + ch * 64;
        const int n0 = n_blk * BLOCK_N + ch * 64;
        // ---- this lane's row, 64 columns: bias, activation, bf16, into the warp's turning buffer (once the store of
        // the warp's tile before has read it: two tiles ago, so this wait does not wait)
        if (lane == 0) asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
        __syncwarp();
#pragma unroll
        for (int pr = 0; pr < 2; ++pr) {
          float va[16], vb[16];
          ptx::tmem_ld16(t_acc + 32 * pr, va);
          ptx::tmem_ld16(t_acc + 32 * pr + 16, vb);
          ptx::tmem_ld_wait();
          if (pr == 1) {
            // the accumulator is in registers: the MMAs of the tile after next may overwrite it
            ptx::tc_fence_before();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(&tempty[acc]);
          }
#pragma unroll
          for (int hlf = 0; hlf < 2; ++hlf) {
            float* v = hlf ? vb : va;
            const int n = n0 + 32 * pr + 16 * hlf;
            if (n + 16 <= e.n_bias) {
#pragma unroll
              for (int j = 0; j < 4; ++j) {
                const float4 b = __ldg(reinterpret_cast<const float4*>(e.bias + n) + j);
                v[4 * j] += b.x; v[4 * j + 1] += b.y; v[4 * j + 2] += b.z; v[4 * j + 3] += b.w;
              }
            } else {
#pragma unroll
              for (int j = 0; j < 16; ++j)
                if (n + j < e.n_bias) v[j] += __ldg(e.bias + n + j);
            }
            if (n < e.n_act) gelu_fast16(v, gc);
            const int piece = 4 * pr + 2 * hlf;          // 16-byte pieces `piece` and `piece + 1` of the row's 128 bytes
            uint8_t* trow = turn + lane * 128;
            *reinterpret_cast<uint4*>(trow + ((piece ^ (lane & 7)) << 4)) =
                make_uint4(pack_bf16x2(v[0], v[1]), pack_bf16x2(v[2], v[3]), pack_bf16x2(v[4], v[5]), pack_bf16x2(v[6], v[7]));
            *reinterpret_cast<uint4*>(trow + (((piece + 1) ^ (lane & 7)) << 4)) =
                make_uint4(pack_bf16x2(v[8], v[9]), pack_bf16x2(v[10], v[11]), pack_bf16x2(v[12], v[13]), pack_bf16x2(v[14], v[15]));
          }
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        __syncwarp();
        // ---- out: one TMA store of the warp's 32 x 64 block (rows past M and columns past N are clipped)
        if (lane == 0) {
          asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];" ::"l"(&tmC),
                       "r"(ptx::smem_u32(turn)), "r"(n0), "r"(static_cast<int>(m_blk * BLOCK_M + q * 32))
                       : "memory");
          asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        }
      }
      if (++n_blk == p.tiles_n) { n_blk = 0; ++m_blk; }
    }
  }

  if (warp >= 2 && lane == 0) asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");
  ptx::tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) record_status(p.status, FFSPLIT_ERR_TIMEOUT, blockIdx.x, KID_GEMM_AR);
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

}  // namespace ar

// Plain or activated bf16 product with one output, a contraction of at most 512 and enough tiles along N for the
// resident row block to pay.
bool gemm_ares_applies(const GemmArgs& g) {
  return g.A1 == nullptr && g.few == nullptr && g.force_split == 0 && !g.epi.col_partial && !g.epi.c0_f32 &&
         g.epi.n_split >= g.N && g.K <= ar::MAX_K && g.K % 8 == 0 && g.K >= 128 && g.M >= 4 * ar::BLOCK_M &&
         g.N >= 16 * ar::BLOCK_N && g.N % 8 == 0 && g.lda0 % 8 == 0 && (reinterpret_cast<uintptr_t>(g.A0) & 15u) == 0 &&
         g.epi.ld0 % 8 == 0 && (reinterpret_cast<uintptr_t>(g.epi.C0) & 15u) == 0;
}

ffsplit_status launch_gemm_ares(ffsplit_ctx* ctx, const GemmArgs& g, cudaStream_t st) {
  ar::Params p;
  p.M = g.M;
  p.N = static_cast<int>(g.N);
  p.K = static_cast<int>(g.K);
  p.nkb = (p.K + ar::KB - 1) / ar::KB;
  p.tiles_n = (p.N + ar::BLOCK_N - 1) / ar::BLOCK_N;
  p.tiles = ((g.M + ar::BLOCK_M - 1) / ar::BLOCK_M) * p.tiles_n;
  p.A = static_cast<const __nv_bfloat16*>(g.A0);
  p.lda = g.lda0;
  p.epi = g.epi;
  p.status = ctx->status();
  CUtensorMap tB, tC;
  ffsplit_status s;
  if ((s = get_tmap_bf16(ctx, g.B0, g.N, g.K, g.ldb0, ar::BLOCK_N, &tB)) != FFSPLIT_OK) return s;
  if ((s = get_tmap_bf16(ctx, g.epi.C0, g.M, g.N, g.epi.ld0, 32, &tC)) != FFSPLIT_OK) return s;
  if (!ctx->attr_ares_set) {
    cudaError_t e = cudaFuncSetAttribute(ar::gemm_ares_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, ar::SMEM_BYTES);
    if (e != cudaSuccess) return check_cuda(ctx, e, "cudaFuncSetAttribute(gemm_ares_kernel)");
    ctx->attr_ares_set = true;
  }
  const int grid = static_cast<int>(p.tiles < ctx->num_sms ? p.tiles : ctx->num_sms);
  const int ph = prof_open(ctx, PROF_GEMM_TC, g.algo_flops, st);
  const cudaError_t le = launch_pdl(ar::gemm_ares_kernel, dim3(grid), dim3(ar::NUM_THREADS), ar::SMEM_BYTES, st, tB, tC, p);
  prof_close(ctx, ph, st);
  ctx->launches++;
  return check_cuda(ctx, le, "gemm_ares_kernel launch");
}

}  // namespace ffsp
