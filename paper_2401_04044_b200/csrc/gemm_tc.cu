// bf16 tensor-core GEMM building block for sm_100a.
//
//   acc[row, n] = sum_k A[row, k] * B[n, k]      A: [M, K], B: [N, K], both K-major bf16
//
// One persistent CTA per SM walks output tiles of 128 x block_n.  Warp roles:
//   warp 0  (one lane)  TMA producer: global -> 128B-swizzled shared tiles, ring of up to 8 stages
//   warp 1  (one lane)  tcgen05.mma issuer; accumulators live in tensor memory (TMEM),
//                       two buffers so the epilogue of tile i overlaps the MMAs of tile i+1
//   warps 2-17          epilogue: tcgen05.ld -> bias / activation / gating -> global; four warps
//                       per TMEM lane quarter, taking every fourth 16-column chunk
// The gated form (SwiGLU) runs two operand pairs into two accumulators of the same
// tile and combines them as silu(acc0) * acc1.
// The score form does not store the tile; it reduces act(acc)^2 over the tile's rows
// with warp shuffles and writes one partial per 32-row group and column (Eq. 3's
// ||sigma(X U_j)||^2 accumulated over tokens).
//
// Every mbarrier wait is bounded; on expiry the CTA records FFSPLIT_ERR_TIMEOUT in
// the status block, drains what it has in flight, frees its TMEM and returns.
#include <cstring>

#include "epilogue.cuh"
#include "internal.h"
#include "ptx.cuh"

namespace ffsp {
namespace tc {

constexpr int BLOCK_M = 128;
constexpr int BLOCK_K = 64;
constexpr int MAX_STAGES = 8;
constexpr int A_STAGE_BYTES = BLOCK_M * BLOCK_K * 2;
constexpr int TMEM_COLS = 512;
constexpr int ACC_STRIDE = 256;   // TMEM columns per accumulator buffer
constexpr int GATE_OFFSET = 128;  // second accumulator of a gated tile
constexpr int EPI_WARPS = 16;
constexpr int NUM_THREADS = 32 * (EPI_WARPS + 2);
constexpr int BAR_BYTES = 256;
constexpr int MAX_SMEM = 232448;

struct Params {
  long long M;
  int N, K;
  int block_n;
  int stages;        // depth of the shared-memory ring (as many as fit, at most 8)
  int tiles_m, tiles_n;
  int dual;
  int shared_a;      // gated pair with one left operand (A0 == A1): A is staged once per k block, the two
                     // weight tiles sit one behind the other and ONE MMA of width 2 block_n fills both accumulators
  int two_m;         // 256 x block_n tiles: two 128-row blocks of A against one weight tile (half the weight
                     // traffic per FLOP); the two accumulator buffers hold the halves, so the epilogue of a tile
                     // does not overlap the MMAs of the next one
  int gate_off;      // tensor-memory column of the second accumulator of a gated tile: 128, or block_n when shared_a
  int panel_m;       // tiles are walked in panels of this many tile rows, column by column inside a panel, so that the
                     // tiles in flight at any time form a block about as high as wide: their operands then fit L2
                     // (row-major order re-read the whole weight matrix from DRAM once per wave: 3.96 GB for 0.29 GB
                     // of operands on the OPT-13B-shaped scoring product)
  int split_k;       // > 1: the K loop is cut into this many ranges, each a tile of its own (tiles_m x tiles_n x split_k
                     // work units) writing an fp32 partial [split][M][N]; a small kernel adds them (thin outputs with a
                     // long contraction: fewer tiles than SMs otherwise)
  int kb_split;      // k-blocks per range
  int early;         // 1: the row operand (A) does not depend on the kernel before this one in the stream (packed weights
                     // in the few-token path): its first stages are loaded before the programmatic-launch wait, under
                     // the tail of that kernel; the other operand and every global write come after the wait
  int trans_tokens;  // > 0: exchanged operands (rows = output columns n, tile columns = tokens), K not cut: the epilogue
                     // applies bias (per row) and activation and stores the transpose, out[t][n], for t < trans_tokens
  Epilogue epi;
  int* status;
};

// Bias, activation and store of 16 consecutive columns of one row.  n_act, n_bias
// and n_split are multiples of 16 (or >= N), so the branches are uniform per chunk.
__device__ __forceinline__ void add_bias16(const Epilogue& e, int n0, float* v) {
  if (n0 + 16 <= e.n_bias) {
    const float4* b = reinterpret_cast<const float4*>(e.bias + n0);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float4 t = __ldg(b + i);
      v[4 * i] += t.x; v[4 * i + 1] += t.y; v[4 * i + 2] += t.z; v[4 * i + 3] += t.w;
    }
  } else {
#pragma unroll
    for (int i = 0; i < 16; ++i)
      if (n0 + i < e.n_bias) v[i] += __ldg(e.bias + n0 + i);
  }
}

__device__ __forceinline__ void epilogue_chunk_store(const Params& p, const GeluCoef& gc, long long row, int n0,
                                                     float* v, int ks) {
  const Epilogue& e = p.epi;
  if (n0 < e.n_bias) add_bias16(e, n0, v);
  if (!p.dual && n0 < e.n_act) {
    gelu_fast16(v, gc);
  }
  if (row >= p.M) return;
  if (e.c0_f32) {
    // fp32 output (n_split >= N): 64 bytes per lane, in 16-byte pieces where the address allows
    float* base = reinterpret_cast<float*>(e.C0) + (row + static_cast<long long>(ks) * p.M) * e.ld0 + n0;   // ks-th partial
    if (n0 + 16 <= p.N && (reinterpret_cast<uintptr_t>(base) & 15u) == 0) {
#pragma unroll
      for (int i = 0; i < 4; ++i)
        reinterpret_cast<float4*>(base)[i] = make_float4(v[4 * i], v[4 * i + 1], v[4 * i + 2], v[4 * i + 3]);
    } else {
#pragma unroll
      for (int i = 0; i < 16; ++i)
        if (n0 + i < p.N) base[i] = v[i];
    }
    return;
  }
  const bool first = n0 < e.n_split;
  __nv_bfloat16* base = first ? reinterpret_cast<__nv_bfloat16*>(e.C0) + row * e.ld0 + n0
                              : reinterpret_cast<__nv_bfloat16*>(e.C1) + row * e.ld1 + (n0 - e.n_split);
  const int limit = first ? (e.n_split < p.N ? e.n_split : p.N) : p.N;
  if (n0 + 16 <= limit && (reinterpret_cast<uintptr_t>(base) & 15u) == 0) {
    uint4 a, b;
    a.x = pack_bf16x2(v[0], v[1]);   a.y = pack_bf16x2(v[2], v[3]);
    a.z = pack_bf16x2(v[4], v[5]);   a.w = pack_bf16x2(v[6], v[7]);
    b.x = pack_bf16x2(v[8], v[9]);   b.y = pack_bf16x2(v[10], v[11]);
    b.z = pack_bf16x2(v[12], v[13]); b.w = pack_bf16x2(v[14], v[15]);
    if ((reinterpret_cast<uintptr_t>(base) & 31u) == 0) {
      // one whole 32-byte sector per lane and instruction: half as many write requests as two 16-byte stores
      asm volatile("st.global.v8.b32 [%0], {%1, %2, %3, %4, %5, %6, %7, %8};" ::"l"(base), "r"(a.x), "r"(a.y), "r"(a.z),
                   "r"(a.w), "r"(b.x), "r"(b.y), "r"(b.z), "r"(b.w)
                   : "memory");
    } else {
      reinterpret_cast<uint4*>(base)[0] = a;
      reinterpret_cast<uint4*>(base)[1] = b;
    }
  } else {
#pragma unroll
    for (int i = 0; i < 16; ++i)
      if (n0 + i < limit) base[i] = __float2bfloat16_rn(v[i]);
  }
}

// Exchanged operands, whole K in one unit: v holds row n (one output column) at tokens t0 .. t0 + 15.  Bias per row,
// activation, and the transposed store: for one token the lanes of a warp write 32 consecutive outputs.
__device__ __forceinline__ void epilogue_chunk_transposed(const Params& p, const GeluCoef& gc, long long n, int t0, float* v) {
  const Epilogue& e = p.epi;
  if (n >= p.M) return;
  const float bias = n < e.n_bias ? __ldg(e.bias + n) : 0.f;
  const bool act = !p.dual && n < e.n_act;   // (a gated pair arrives here as SiLU(gate) * up already)
  const bool first = n < e.n_split;
  __nv_bfloat16* base = first ? reinterpret_cast<__nv_bfloat16*>(e.C0) + n : reinterpret_cast<__nv_bfloat16*>(e.C1) + (n - e.n_split);
  const long long ld = first ? e.ld0 : e.ld1;
#pragma unroll
  for (int i = 0; i < 16; ++i) {
    if (t0 + i < p.trans_tokens) {
      float x = v[i] + bias;
      if (act) x = gelu_fast(x, gc);
      base[static_cast<long long>(t0 + i) * ld] = __float2bfloat16_rn(x);
    }
  }
}

// Sum v[i] over the 32 lanes of the warp for each of 16 columns with a fixed
// exchange tree (16 shuffles).  Afterwards lane l holds the total of column l >> 1.
__device__ __forceinline__ float warp_column_sums16(const float* v, int lane) {
  float w[8], x[4], y[2], z;
  const bool b4 = lane & 16, b3 = lane & 8, b2 = lane & 4, b1 = lane & 2;
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const float send = b4 ? v[i] : v[i + 8];
    const float keep = b4 ? v[i + 8] : v[i];
    w[i] = keep + __shfl_xor_sync(0xffffffffu, send, 16);
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float send = b3 ? w[i] : w[i + 4];
    const float keep = b3 ? w[i + 4] : w[i];
    x[i] = keep + __shfl_xor_sync(0xffffffffu, send, 8);
  }
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    const float send = b2 ? x[i] : x[i + 2];
    const float keep = b2 ? x[i + 2] : x[i];
    y[i] = keep + __shfl_xor_sync(0xffffffffu, send, 4);
  }
  {
    const float send = b1 ? y[0] : y[1];
    const float keep = b1 ? y[1] : y[0];
    z = keep + __shfl_xor_sync(0xffffffffu, send, 2);
  }
  z += __shfl_xor_sync(0xffffffffu, z, 1);
  return z;
}

// Tile number -> (tile row, tile column): panels of panel_m tile rows, inside a panel all rows of a column
// before the next column (the last panel may be lower).
__device__ __forceinline__ void tile_coords(const Params& p, int tile, int* m_blk, int* n_blk) {
  const int per_panel = p.panel_m * p.tiles_n;
  const int panel = tile / per_panel;
  const int in_panel = tile - panel * per_panel;
  const int m0 = panel * p.panel_m;
  const int h = p.tiles_m - m0 < p.panel_m ? p.tiles_m - m0 : p.panel_m;
  *n_blk = in_panel / h;
  *m_blk = m0 + (in_panel - *n_blk * h);
}

__global__ void __launch_bounds__(NUM_THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA0, const __grid_constant__ CUtensorMap tmB0,
               const __grid_constant__ CUtensorMap tmA1, const __grid_constant__ CUtensorMap tmB1, const Params p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  const int STAGES = p.stages;
  const int B_TILE_BYTES = p.block_n * BLOCK_K * 2;
  const int B_STAGE_BYTES = p.shared_a ? 2 * B_TILE_BYTES : B_TILE_BYTES;
  const int MT = p.two_m ? 2 : 1;                 // 128-row blocks of A per tile
  const int A_STAGE = MT * A_STAGE_BYTES;
  uint8_t* smem_a = smem;
  uint8_t* smem_b = smem + STAGES * A_STAGE;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem + STAGES * (A_STAGE + B_STAGE_BYTES));
  uint64_t* full = bars;                      // [MAX_STAGES] TMA -> MMA
  uint64_t* empty = bars + MAX_STAGES;        // [MAX_STAGES] MMA -> TMA
  uint64_t* tfull = bars + 2 * MAX_STAGES;    // [2] MMA -> epilogue
  uint64_t* tempty = tfull + 2;           // [2] epilogue -> MMA
  uint64_t* drain = tempty + 2;           // [1] used only when giving up
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(drain + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);

  const int warp = threadIdx.x >> 5;
  const int lane = threadIdx.x & 31;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) {
      ptx::mbar_init(&full[s], 1);
      ptx::mbar_init(&empty[s], 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(&tfull[a], 1);
      ptx::mbar_init(&tempty[a], EPI_WARPS);
    }
    ptx::mbar_init(drain, 1);
    *abort_flag = 0;
    ptx::mbar_fence_init();
    ptx::prefetch_tmap(&tmA0);
    ptx::prefetch_tmap(&tmB0);
    if (p.dual) {
      ptx::prefetch_tmap(&tmA1);
      ptx::prefetch_tmap(&tmB1);
    }
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
  if (!p.early) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    // Only now may the kernel after this one begin its set-up: it will block in its tensor-memory allocation
    // until this CTA frees its columns, which is safe because this CTA already holds its own (a dependent
    // that got the columns first would wait for this kernel, and this kernel for the columns).
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  }

  const int nkb = (p.K + BLOCK_K - 1) / BLOCK_K;
  const int tiles_mn = p.tiles_m * p.tiles_n;
  const int num_tiles = tiles_mn * p.split_k;
  // k-blocks of a work unit of K range ks (the last range may be shorter)
  const int kb_last = nkb - (p.split_k - 1) * p.kb_split;
  const int kb_mul = (p.dual && !p.shared_a) ? 2 : 1;
#define UNIT_KB(ks) (kb_mul * ((ks) == p.split_k - 1 ? kb_last : p.kb_split))
  const uint32_t stage_tx = A_STAGE + B_STAGE_BYTES;

  if (warp == 0) {
    if (ptx::elect_one()) {
      // ------------------------------------------------------------ TMA producer
      uint32_t it = 0;
      bool ok = true;
      int pre = 0;      // stages of the first unit whose loads were issued ahead of the loop
      if (p.early) {
        // weights first: the ring is empty, no slot needs waiting for
        int m_blk = 0, n_blk = 0, ks = 0;
        if (static_cast<int>(blockIdx.x) < num_tiles) {
          ks = blockIdx.x / tiles_mn;
          tile_coords(p, blockIdx.x - ks * tiles_mn, &m_blk, &n_blk);
          const int total_kb = UNIT_KB(ks);
          pre = total_kb < STAGES ? total_kb : STAGES;
          for (int kb = 0; kb < pre; ++kb) {
            ptx::mbar_expect_tx(&full[kb], stage_tx);
            for (int mt = 0; mt < MT; ++mt)
              ptx::tma_load_2d(&tmA0, smem_a + kb * A_STAGE + mt * A_STAGE_BYTES, &full[kb], (ks * p.kb_split + kb) * BLOCK_K,
                               (m_blk * MT + mt) * BLOCK_M);
          }
        }
        asm volatile("griddepcontrol.wait;" ::: "memory");
        asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
        for (int kb = 0; kb < pre; ++kb)
          ptx::tma_load_2d(&tmB0, smem_b + kb * B_STAGE_BYTES, &full[kb], (ks * p.kb_split + kb) * BLOCK_K, n_blk * p.block_n);
        it = pre;
      }
      // ring position of `it` without divisions (this thread shares its scheduler with epilogue warps)
      int rs = pre == STAGES ? 0 : pre;
      uint32_t rph = pre == STAGES ? 1u : 0u;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x) {
        int m_blk, n_blk;
        const int ks = tile / tiles_mn;
        tile_coords(p, tile - ks * tiles_mn, &m_blk, &n_blk);
        const int total_kb = UNIT_KB(ks), nkb_u = p.split_k > 1 ? total_kb : nkb;
        for (int kb = tile == static_cast<int>(blockIdx.x) ? pre : 0; kb < total_kb; ++kb, ++it) {
          const int s = rs;
          const uint32_t ph = rph;
          if (++rs == STAGES) { rs = 0; rph ^= 1u; }
          if (!ptx::mbar_wait(&empty[s], ph ^ 1, abort_flag)) { ok = false; break; }
          ptx::mbar_expect_tx(&full[s], stage_tx);
          const bool second = p.dual && kb >= nkb_u;
          const int kk = (ks * p.kb_split + (second ? kb - nkb_u : kb)) * BLOCK_K;
          for (int mt = 0; mt < MT; ++mt)
            ptx::tma_load_2d(second ? &tmA1 : &tmA0, smem_a + s * A_STAGE + mt * A_STAGE_BYTES, &full[s], kk,
                             (m_blk * MT + mt) * BLOCK_M);
          ptx::tma_load_2d(second ? &tmB1 : &tmB0, smem_b + s * B_STAGE_BYTES, &full[s], kk, n_blk * p.block_n);
          if (p.shared_a)   // the second weight tile right behind the first: rows block_n .. 2 block_n - 1 of one operand
            ptx::tma_load_2d(&tmB1, smem_b + s * B_STAGE_BYTES + B_TILE_BYTES, &full[s], kk, n_blk * p.block_n);
        }
      }
      if (!ok) {
        // give the copies already issued a bounded chance to land before the CTA exits
        const uint32_t first = it > STAGES ? it - STAGES : 0;
        for (uint32_t j = first; j < it; ++j) {
          const long long t0 = clock64();
          while (!ptx::mbar_try_wait(&full[j % STAGES], (j / STAGES) & 1) &&
                 clock64() - t0 < ptx::kWaitLimitCycles / 8) {}
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    if (ptx::elect_one()) {
      // ------------------------------------------------------------ MMA issuer
      const uint32_t idesc = ptx::umma_idesc_bf16(BLOCK_M, p.shared_a ? 2 * p.block_n : p.block_n);
      uint32_t tl = 0;
      int rs = 0;          // ring position, kept without divisions
      uint32_t rph = 0;
      const uint64_t a_desc0 = ptx::umma_desc_k128(ptx::smem_u32(smem_a));
      const uint64_t b_desc0 = ptx::umma_desc_k128(ptx::smem_u32(smem_b));
      const uint32_t a_step = static_cast<uint32_t>(A_STAGE) >> 4, b_step = static_cast<uint32_t>(B_STAGE_BYTES) >> 4;   // descriptor addresses count 16 bytes
      bool ok = true;
      for (int tile = blockIdx.x; tile < num_tiles && ok; tile += gridDim.x, ++tl) {
        // one buffer per tile, alternating -- or, with 256-row tiles, both buffers for the two halves
        const uint32_t acc = p.two_m ? 0 : (tl & 1), aph = p.two_m ? (tl & 1) : ((tl >> 1) & 1);
        if (!ptx::mbar_wait(&tempty[acc], aph ^ 1, abort_flag)) { ok = false; break; }
        if (p.two_m && !ptx::mbar_wait(&tempty[1], aph ^ 1, abort_flag)) { ok = false; break; }
        ptx::tc_fence_after();
        const int total_kb = UNIT_KB(tile / tiles_mn);
        for (int kb = 0; kb < total_kb; ++kb) {
          const int s = rs;
          const uint32_t ph = rph;
          if (++rs == STAGES) { rs = 0; rph ^= 1u; }
          if (!ptx::mbar_wait(&full[s], ph, abort_flag)) { ok = false; break; }
          ptx::tc_fence_after();
          const bool second = p.dual && kb >= nkb;   // (a gated product is never cut along K)
          const int kbl = second ? kb - nkb : kb;
          const uint32_t d_tmem = tmem_base + acc * ACC_STRIDE + (second ? p.gate_off : 0);
          const uint64_t a_desc = a_desc0 + static_cast<uint32_t>(s) * a_step;
          const uint64_t b_desc = b_desc0 + static_cast<uint32_t>(s) * b_step;
#pragma unroll
          for (int k = 0; k < BLOCK_K / 16; ++k) {
            // 16 elements (32 bytes) further along K inside the swizzled row: +2 in the address field
            ptx::umma_bf16(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc, (kbl | k) != 0 ? 1u : 0u);
          }
          if (p.two_m) {
            // the second 128 rows of A against the same weights, into the other accumulator buffer
            const uint64_t a2_desc = a_desc + (static_cast<uint32_t>(A_STAGE_BYTES) >> 4);
#pragma unroll
            for (int k = 0; k < BLOCK_K / 16; ++k)
              ptx::umma_bf16(d_tmem + ACC_STRIDE, a2_desc + 2 * k, b_desc + 2 * k, idesc, (kbl | k) != 0 ? 1u : 0u);
          }
          ptx::umma_commit(&empty[s]);
        }
        if (ok) {
          ptx::umma_commit(&tfull[acc]);
          if (p.two_m) ptx::umma_commit(&tfull[1]);
        }
      }
      if (!ok) {
        // wait (bounded) until the MMAs issued so far have retired before TMEM is freed
        ptx::umma_commit(drain);
        const long long t0 = clock64();
        while (!ptx::mbar_try_wait(drain, 0) && clock64() - t0 < ptx::kWaitLimitCycles / 8) {}
      }
    }
    __syncwarp();
  } else {
    // -------------------------------------------------------------- epilogue warps
    const int q = warp & 3;             // TMEM lane quarter this warp may read
    const int half = (warp - 2) >> 2;   // which of every EPI_WARPS / 4 consecutive 16-column chunks this warp takes
    const GeluCoef gc = gelu_coef(p.epi.act);
    // The epilogue walks 128-row blocks: one per tile, or the two halves of a 256-row tile one after the
    // other -- either way block number vt uses accumulator buffer vt & 1 in phase (vt >> 1) & 1.
    uint32_t vt = 0;
    bool live = true;
    if (p.early) asm volatile("griddepcontrol.wait;" ::: "memory");   // before this role's first global access
    if (blockIdx.x == 0 && warp == 2) check_blob_guard(p.epi, p.status, KID_GEMM_TC);
    for (int tile = blockIdx.x; tile < num_tiles && live; tile += gridDim.x)
    for (int mt = 0; mt < MT; ++mt, ++vt) {
      int m_tile, n_blk;
      const int ks = tile / tiles_mn;
      tile_coords(p, tile - ks * tiles_mn, &m_tile, &n_blk);
      const int m_blk = m_tile * MT + mt;
      const uint32_t acc = vt & 1, aph = (vt >> 1) & 1;
      if (warp == 2 && p.epi.n_bias > 0) {
        // this tile's slice of the bias vector, on its way to L1 while the MMAs run
        const int nb = n_blk * p.block_n + lane * 32;
        if (lane * 32 < p.block_n && nb < p.epi.n_bias) asm volatile("prefetch.global.L1 [%0];" ::"l"(p.epi.bias + nb));
      }
      if (!ptx::mbar_wait(&tfull[acc], aph, abort_flag)) { live = false; break; }
      ptx::tc_fence_after();
      const long long row = static_cast<long long>(m_blk) * BLOCK_M + q * 32 + lane;
      const uint32_t t_row = tmem_base + (static_cast<uint32_t>(q * 32) << 16) + acc * ACC_STRIDE;
      // one 16-column chunk: v holds the accumulators of this lane's row
      auto finish_chunk = [&](float* v, int n0) {
        if (p.trans_tokens > 0) {
          epilogue_chunk_transposed(p, gc, row, n0, v);
        } else if (p.epi.col_partial == nullptr) {
          epilogue_chunk_store(p, gc, row, n0, v, ks);
        } else {
          const Epilogue& e = p.epi;
          if (n0 < e.n_bias) add_bias16(e, n0, v);
          // scores decide indices: fp32-accurate activation, not the one-MUFU form
          if (!p.dual && e.act == FFSPLIT_GELU_ERF && !e.score_abs) {
            // the common case, without per-element selects
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              const float2 sq = gelu_erf_score_sq2(make_float2(v[2 * i], v[2 * i + 1]));
              v[2 * i] = sq.x;
              v[2 * i + 1] = sq.y;
            }
          } else {
#pragma unroll
            for (int i = 0; i < 16; ++i) {
              float x = v[i];
              if (!p.dual) x = act_gelu_score(x, e.act);
              v[i] = e.score_abs ? fabsf(x) : x * x;
            }
          }
          if (row >= p.M) {
#pragma unroll
            for (int i = 0; i < 16; ++i) v[i] = 0.0f;
          }
          const float tot = warp_column_sums16(v, lane);
          const int n = n0 + (lane >> 1);
          // (the second half of a 256-row tile may lie wholly behind the last row: it has no partial)
          if ((lane & 1) == 0 && n < p.N && static_cast<long long>(m_blk) * BLOCK_M < p.M)
            e.col_partial[(static_cast<long long>(m_blk) * 4 + q) * p.N + n] = tot;
        }
      };
      const int nbase = n_blk * p.block_n;
      constexpr int CSTEP = 4 * EPI_WARPS;
      if (!p.dual) {
        // Two register buffers: the tensor-memory load of the next chunk is in flight while this one goes
        // through bias, activation and stores (a load's registers may be read only after the next wait).
        float va[16], vb[16];
        int c = half * 16;
        bool more = c < p.block_n && nbase + c < p.N;
        if (more) ptx::tmem_ld16(t_row + c, va);
        while (more) {
          ptx::tmem_ld_wait();
          bool next = c + CSTEP < p.block_n && nbase + c + CSTEP < p.N;
          if (next) ptx::tmem_ld16(t_row + c + CSTEP, vb);
          finish_chunk(va, nbase + c);
          if (!next) break;
          c += CSTEP;
          ptx::tmem_ld_wait();
          next = c + CSTEP < p.block_n && nbase + c + CSTEP < p.N;
          if (next) ptx::tmem_ld16(t_row + c + CSTEP, va);
          finish_chunk(vb, nbase + c);
          more = next;
          c += CSTEP;
        }
      } else {
        for (int c = half * 16; c < p.block_n; c += CSTEP) {
          const int n0 = nbase + c;
          if (n0 >= p.N) break;
          float v[16], u[16];
          ptx::tmem_ld16(t_row + c, v);
          ptx::tmem_ld16(t_row + p.gate_off + c, u);
          ptx::tmem_ld_wait();
#pragma unroll
          for (int i = 0; i < 16; ++i)
            v[i] = (p.epi.col_partial ? silu_precise_f(v[i]) : silu_fast(v[i])) * u[i];
          finish_chunk(v, n0);
        }
      }
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&tempty[acc]);
    }
  }

  ptx::tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) record_status(p.status, FFSPLIT_ERR_TIMEOUT, blockIdx.x, KID_GEMM_TC);
  if (warp == 1) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

// C [M, N] (bf16, pitch ldc) = sum over the `split` fp32 partials [split][M][N], in order.  N % 4 == 0.
__global__ void __launch_bounds__(256) splitk_reduce_kernel(const float* partial, int split, long long M, int N,
                                                            __nv_bfloat16* C, long long ldc) {
  pdl_wait();
  const long long q = static_cast<long long>(blockIdx.x) * 256 + threadIdx.x;     // float4 index
  const int n4 = N >> 2;
  if (q >= M * n4) return;
  const long long row = q / n4;
  const int c = static_cast<int>(q - row * n4) * 4;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int s = 0; s < split; ++s) {
    const float4 v = __ldcg(reinterpret_cast<const float4*>(partial + (static_cast<long long>(s) * M + row) * N + c));
    acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
  }
  uint2 o;
  o.x = pack_bf16x2(acc.x, acc.y);
  o.y = pack_bf16x2(acc.z, acc.w);
  *reinterpret_cast<uint2*>(C + row * ldc + c) = o;
}

// Few-token path: Y[t, n] = epi(sum over the `split` partials of acc[n, t]) from the exchanged product's fp32 partials
// [split][n_out][tp] (and a second set for the gated pair), with the epilogue of internal.h read along n:
// bias[n], activation for n < n_act (gated: silu(acc0) * acc1), n < n_split to C0[t, n], else to C1[t, n - n_split].
// Threads run along n, so every token row is written in contiguous runs.
__global__ void __launch_bounds__(256) few_finish_kernel(const float* p0, const float* p1, int split, int n_out, int T, int tp,
                                                         Epilogue e) {
  pdl_wait();
  const int n = blockIdx.x * 256 + threadIdx.x;
  const int t0 = blockIdx.y * 4;
  if (n >= n_out) return;
  float4 a = make_float4(0.f, 0.f, 0.f, 0.f), b = a;
  // the partials are added in order, but eight loads are in flight at a time
  constexpr int FB = 8;
  const size_t stride = static_cast<size_t>(n_out) * tp, at0 = static_cast<size_t>(n) * tp + t0;
  for (int s0 = 0; s0 < split; s0 += FB) {
    float4 v[FB], u[FB];
#pragma unroll
    for (int j = 0; j < FB; ++j) {
      v[j] = make_float4(0.f, 0.f, 0.f, 0.f);
      u[j] = v[j];
      if (s0 + j < split) {
        v[j] = __ldcg(reinterpret_cast<const float4*>(p0 + (s0 + j) * stride + at0));
        if (p1) u[j] = __ldcg(reinterpret_cast<const float4*>(p1 + (s0 + j) * stride + at0));
      }
    }
#pragma unroll
    for (int j = 0; j < FB; ++j) {
      a.x += v[j].x; a.y += v[j].y; a.z += v[j].z; a.w += v[j].w;
      b.x += u[j].x; b.y += u[j].y; b.z += u[j].z; b.w += u[j].w;
    }
  }
  float v[4] = {a.x, a.y, a.z, a.w};
  const float u[4] = {b.x, b.y, b.z, b.w};
  const float bias = n < e.n_bias ? __ldg(e.bias + n) : 0.f;
  const GeluCoef gc = gelu_coef(e.act);
  const bool first = n < e.n_split;
  __nv_bfloat16* base = first ? reinterpret_cast<__nv_bfloat16*>(e.C0) + n : reinterpret_cast<__nv_bfloat16*>(e.C1) + (n - e.n_split);
  const long long ld = first ? e.ld0 : e.ld1;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    if (t0 + i >= T) break;
    float x = v[i] + bias;
    if (p1) x = silu_fast(x) * u[i];
    else if (n < e.n_act) x = gelu_fast(x, gc);
    base[static_cast<long long>(t0 + i) * ld] = __float2bfloat16_rn(x);
  }
}

#undef UNIT_KB

}  // namespace tc

// ---------------------------------------------------------------------------------
// Host side: tensor maps and launch
// ---------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// 2-D bf16 tensor map over a row-major [rows, cols] matrix with pitch ld, box
// [box_rows, 64 columns], 128-byte swizzle, zero fill outside the matrix.
ffsplit_status get_tmap_bf16(ffsplit_ctx* ctx, const void* ptr, long long rows, long long cols, long long ld,
                             int box_rows, CUtensorMap* out) {
  TmapKey key{ptr, rows, cols, ld, box_rows, tc::BLOCK_K};
  auto it = ctx->tmaps.find(key);
  if (it != ctx->tmaps.end()) {
    *out = it->second;
    return FFSPLIT_OK;
  }
  if (!ctx->encode_fn) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn)
      return fail(ctx, FFSPLIT_ERR_CUDA, "cuTensorMapEncodeTiled is not available from the driver");
    ctx->encode_fn = fn;
  }
  if (!aligned16(ptr) || (ld * 2) % 16 != 0)
    return fail(ctx, FFSPLIT_ERR_ALIGN, "tensor-core operand needs a 16-byte aligned base and row pitch");
  cuuint64_t dims[2] = {static_cast<cuuint64_t>(cols), static_cast<cuuint64_t>(rows)};
  cuuint64_t strides[1] = {static_cast<cuuint64_t>(ld) * 2};
  cuuint32_t box[2] = {static_cast<cuuint32_t>(tc::BLOCK_K), static_cast<cuuint32_t>(box_rows)};
  cuuint32_t estr[2] = {1, 1};
  CUtensorMap tm;
  CUresult r = reinterpret_cast<EncodeTiledFn>(ctx->encode_fn)(
      &tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
      CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
      CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS)
    return fail(ctx, FFSPLIT_ERR_CUDA, "cuTensorMapEncodeTiled failed (" + std::to_string((int)r) + ")");
  if (ctx->tmaps.size() > 8192) ctx->tmaps.clear();
  ctx->tmaps.emplace(key, tm);
  *out = tm;
  return FFSPLIT_OK;
}

// Pick the tile width: fewest waves weighted by tile cost, wider tiles on ties.
static int choose_block_n(int N, long long tiles_m, int num_sms, bool dual) {
  const int max_bn = dual ? 128 : 256;
  int best = 32;
  double best_cost = 1e300;
  for (int bn = max_bn; bn >= 32; bn -= 16) {
    const long long tiles = tiles_m * ((N + bn - 1) / bn);
    const long long waves = (tiles + num_sms - 1) / num_sms;
    const double cost = static_cast<double>(waves) * (bn + 40);
    if (cost < best_cost - 1e-9) {
      best_cost = cost;
      best = bn;
    }
  }
  return best;
}

ffsplit_status launch_gemm_tc(ffsplit_ctx* ctx, const GemmArgs& g, cudaStream_t st);

// C [T, N] = epi(X [T, K] . (W [N, K])^T) for T <= 64 on the tensor cores (see GemmArgs::few).
static ffsplit_status launch_gemm_few(ffsplit_ctx* ctx, const GemmArgs& g, cudaStream_t st) {
  const int T = static_cast<int>(g.M), tp = round_up(T, 16), n_out = g.N;
  const bool gated = g.A1 != nullptr;
  const int nmat = gated ? 2 : 1;
  const long long tiles = (n_out + tc::BLOCK_M - 1) / tc::BLOCK_M;
  const int nkb = (g.K + tc::BLOCK_K - 1) / tc::BLOCK_K;
  // K ranges: more of them fill the last wave of work units better but write and re-read more fp32 partials; take the
  // count with the least estimated traffic (weight bytes over the wave efficiency plus twice the partial bytes), with at
  // least four k-blocks per unit and the partials inside the scratch
  int best = 1;
  double best_cost = 1e300;
  const double weight_bytes = 2.0 * n_out * g.K;
  const bool direct_ok = !gated || g.epi.n_bias == 0;   // (the gated epilogue in the kernel adds a bias after the gating)
  for (int s = 1; s <= 16; ++s) {
    if (s > 1 && nkb / s < 4) break;
    if (nkb - (s - 1) * ((nkb + s - 1) / s) <= 0) continue;   // the last range must not be empty
    if (static_cast<size_t>(nmat) * s * n_out * tp * 4 > g.few_bytes) break;
    const long long units = tiles * s;
    const long long waves = (units + ctx->num_sms - 1) / ctx->num_sms;
    const double eff = static_cast<double>(units) / static_cast<double>(waves * ctx->num_sms);
    double cost = weight_bytes / eff + 2.0 * s * n_out * tp * 4;
    // an uncut product finishes its own output (below): no finishing kernel, no launch boundary -- about 3 us, the time
    // in which 16 MB stream from HBM
    if (s == 1 && direct_ok) cost -= 16e6 * nmat;
    if (cost < best_cost) { best_cost = cost; best = s; }
  }
  if (static_cast<size_t>(nmat) * best * n_out * tp * 4 > g.few_bytes)
    return fail(ctx, FFSPLIT_ERR_BUFFER_TOO_SMALL, "workspace too small for the few-token tensor path");
  if (best == 1 && direct_ok) {
    // K in one piece (the light chain's first product: a contraction of r): nothing to add up, so the product's own
    // epilogue finishes the output and the finishing kernel, with its launch boundary, drops out; a gated pair runs
    // as one launch with two accumulators
    GemmArgs h;
    std::memset(&h, 0, sizeof(h));
    h.A0 = g.B0; h.lda0 = g.ldb0;
    h.B0 = g.A0; h.ldb0 = g.lda0;
    if (gated) {
      h.A1 = g.B1; h.lda1 = g.ldb1;
      h.B1 = g.A1; h.ldb1 = g.lda1;
    }
    h.M = n_out; h.N = tp; h.K = g.K;
    h.algo_flops = g.algo_flops;
    h.epi = g.epi;
    h.force_split = 1;
    h.trans_tokens = T;
    h.early_rows = g.weights_stable;
    return launch_gemm_tc(ctx, h, st);
  }
  float* part[2] = {static_cast<float*>(g.few), static_cast<float*>(g.few) + static_cast<size_t>(best) * n_out * tp};
  for (int i = 0; i < nmat; ++i) {
    GemmArgs h;
    std::memset(&h, 0, sizeof(h));
    h.A0 = i == 0 ? g.B0 : g.B1; h.lda0 = i == 0 ? g.ldb0 : g.ldb1;     // the weights: rows of the accumulator
    h.B0 = i == 0 ? g.A0 : g.A1; h.ldb0 = i == 0 ? g.lda0 : g.lda1;     // the tokens: its columns
    h.M = n_out; h.N = tp; h.K = g.K;
    h.algo_flops = g.algo_flops / nmat;
    h.epi.C0 = part[i]; h.epi.ld0 = tp; h.epi.n_split = tp; h.epi.act = FFSPLIT_GELU_ERF;
    h.epi.guard = i == 0 ? g.epi.guard : nullptr; h.epi.guard_hash = g.epi.guard_hash;
    h.force_split = best;
    h.early_rows = g.weights_stable;  // the weights are this product's row operand
    const ffsplit_status s = launch_gemm_tc(ctx, h, st);
    if (s != FFSPLIT_OK) return s;
  }
  Epilogue e = g.epi;
  const cudaError_t le = launch_pdl(tc::few_finish_kernel, dim3((n_out + 255) / 256, (T + 3) / 4), dim3(256), 0, st,
                                    static_cast<const float*>(part[0]), gated ? static_cast<const float*>(part[1]) : nullptr,
                                    best, n_out, T, tp, e);
  ctx->launches++;
  return check_cuda(ctx, le, "few_finish_kernel launch");
}

bool gemm_ares_applies(const GemmArgs& g);
ffsplit_status launch_gemm_ares(ffsplit_ctx* ctx, const GemmArgs& g, cudaStream_t st);

ffsplit_status launch_gemm_tc(ffsplit_ctx* ctx, const GemmArgs& g, cudaStream_t st) {
  if (g.few && g.force_split == 0 && g.M <= 64 && !g.epi.col_partial && !g.epi.c0_f32) return launch_gemm_few(ctx, g, st);
  if (ctx->gemm_ares && gemm_ares_applies(g)) return launch_gemm_ares(ctx, g, st);
  const bool dual = g.A1 != nullptr;
  if (g.M <= 0 || g.N <= 0 || g.K <= 0) return FFSPLIT_OK;
  tc::Params p;
  p.M = g.M;
  p.N = g.N;
  p.K = g.K;
  p.dual = dual ? 1 : 0;
  p.shared_a = (dual && g.A0 == g.A1 && g.lda0 == g.lda1) ? 1 : 0;
  p.tiles_m = static_cast<int>((g.M + tc::BLOCK_M - 1) / tc::BLOCK_M);
  p.block_n = choose_block_n(g.N, p.tiles_m, ctx->num_sms, dual);
  p.two_m = 0;
  if (ctx->gemm_two_m && (!dual || p.shared_a) && g.K >= 2048 && g.M > tc::BLOCK_M) {
    // 256-row tiles halve the weight bytes staged per FLOP (the kernels are bound by the shared-memory
    // fill rate, not by the tensor pipe) but expose each tile's epilogue and make the tiles coarser:
    // taken when the K loop is long and the waves stay about as full as with 128-row tiles.
    const long long tm2 = (g.M + 2 * tc::BLOCK_M - 1) / (2 * tc::BLOCK_M);
    const int bn2 = choose_block_n(g.N, tm2, ctx->num_sms, dual);
    const auto wave_fill = [&](long long tiles) {
      const long long waves = (tiles + ctx->num_sms - 1) / ctx->num_sms;
      return static_cast<double>(tiles) / static_cast<double>(waves * ctx->num_sms);
    };
    const long long t1 = static_cast<long long>(p.tiles_m) * ((g.N + p.block_n - 1) / p.block_n);
    const long long t2 = tm2 * ((g.N + bn2 - 1) / bn2);
    if (ctx->gemm_two_m == 2 || (bn2 >= (dual ? 64 : 128) && wave_fill(t2) >= 0.9 * wave_fill(t1))) {
      p.two_m = 1;
      p.tiles_m = static_cast<int>(tm2);
      p.block_n = bn2;
    }
  }
  p.tiles_n = (g.N + p.block_n - 1) / p.block_n;
  // Thin output, long contraction: with 256-wide tiles of 128 rows there are fewer than half as many tiles as SMs;
  // cut K so that the work units cover the SMs.  (Measured on the OPT-13B-shaped light chain, 4096 x 512 x 19456:
  // 128 tiles of 128 x 128 ran the tensor pipe at 47 %.)
  p.split_k = 1;
  p.kb_split = (g.K + tc::BLOCK_K - 1) / tc::BLOCK_K;
  const bool plain = !dual && !g.epi.col_partial && !g.epi.c0_f32 && g.epi.n_bias == 0 && g.epi.n_act == 0 &&
                     g.epi.n_split >= g.N && g.N % 4 == 0 && (reinterpret_cast<uintptr_t>(g.epi.C0) & 7u) == 0 && g.epi.ld0 % 4 == 0;
  if (g.force_split >= 1) {
    // the few-token path: one tile column as wide as the (padded) token count, K cut as asked
    p.two_m = 0;
    p.tiles_m = static_cast<int>((g.M + tc::BLOCK_M - 1) / tc::BLOCK_M);
    p.block_n = g.N;
    p.tiles_n = 1;
    p.split_k = g.force_split;
    p.kb_split = (p.kb_split + g.force_split - 1) / g.force_split;
  } else if (ctx->gemm_split_k && g.splitk && plain && g.K >= 4096) {
    const int bn = g.N >= 256 ? 256 : round_up(g.N, 16);
    const int nkb = p.kb_split;
    // 128-row tiles (256-row tiles with K cut in four were measured too: 284 us per OPT-13B-shaped split layer against
    // 272 us with 128-row tiles and K cut in two, 283 us without the cut: twice the partials, an exposed epilogue)
    for (int mt = 1; mt >= 1 && p.split_k == 1; --mt) {
      const long long tm = (g.M + mt * tc::BLOCK_M - 1) / (mt * tc::BLOCK_M);
      const long long tiles1 = tm * ((g.N + bn - 1) / bn);
      int split = static_cast<int>(ctx->num_sms / tiles1);
      if (split > 4) split = 4;
      while (split > 1 && (nkb / split < 16 * mt || static_cast<size_t>(split) * g.M * g.N * 4 > g.splitk_bytes)) --split;
      if (split > 1) {
        p.two_m = mt == 2 ? 1 : 0;
        p.tiles_m = static_cast<int>(tm);
        p.block_n = bn;
        p.tiles_n = (g.N + bn - 1) / bn;
        p.split_k = split;
        p.kb_split = (nkb + split - 1) / split;
      }
    }
  }
  {
    // panel height: the tiles of one wave (one per SM) form a block of panel_m x (SMs / panel_m) tiles; the
    // operand bytes that block touches are smallest when its two sides carry about the same bytes
    const double row_bytes = (p.two_m ? 2.0 : 1.0) * tc::BLOCK_M, col_bytes = (dual ? 2.0 : 1.0) * p.block_n;
    int best = 1;
    double best_cost = 1e300;
    for (int h = 1; h <= p.tiles_m && h <= ctx->num_sms; ++h) {
      const double w = static_cast<double>(ctx->num_sms) / h;
      const double cost = h * row_bytes + (w < p.tiles_n ? w : p.tiles_n) * col_bytes;
      if (cost < best_cost - 1e-9) { best_cost = cost; best = h; }
    }
    p.panel_m = ctx->gemm_panel > 0 ? (ctx->gemm_panel < p.tiles_m ? ctx->gemm_panel : p.tiles_m) : best;
  }
  p.gate_off = p.shared_a ? p.block_n : tc::GATE_OFFSET;
  p.early = (g.early_rows && !dual) ? 1 : 0;
  p.epi = g.epi;
  p.trans_tokens = 0;
  if (g.force_split == 1 && g.trans_tokens > 0) {
    p.trans_tokens = g.trans_tokens;   // the caller's epilogue, applied by the one unit of each row tile
  } else if (g.force_split >= 1) {
    p.epi.c0_f32 = 1;         // the caller's C0 is the fp32 partial buffer [split][M][N] already
  } else if (p.split_k > 1) {
    p.epi.C0 = g.splitk;      // fp32 partials [split][M][N]
    p.epi.ld0 = g.N;
    p.epi.c0_f32 = 1;
  }
  p.status = ctx->status();
  CUtensorMap tA0, tB0, tA1, tB1;
  ffsplit_status s;
  if ((s = get_tmap_bf16(ctx, g.A0, g.M, g.K, g.lda0, tc::BLOCK_M, &tA0)) != FFSPLIT_OK) return s;
  if ((s = get_tmap_bf16(ctx, g.B0, g.N, g.K, g.ldb0, p.block_n, &tB0)) != FFSPLIT_OK) return s;
  if (dual) {
    if ((s = get_tmap_bf16(ctx, g.A1, g.M, g.K, g.lda1, tc::BLOCK_M, &tA1)) != FFSPLIT_OK) return s;
    if ((s = get_tmap_bf16(ctx, g.B1, g.N, g.K, g.ldb1, p.block_n, &tB1)) != FFSPLIT_OK) return s;
  } else {
    tA1 = tA0;
    tB1 = tB0;
  }
  if (!ctx->attr_tc_set) {
    cudaError_t e = cudaFuncSetAttribute(tc::gemm_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         tc::MAX_SMEM);
    if (e != cudaSuccess) return check_cuda(ctx, e, "cudaFuncSetAttribute(gemm_tc_kernel)");
    ctx->attr_tc_set = true;
  }
  const int stage_bytes = (p.two_m ? 2 : 1) * tc::A_STAGE_BYTES + (p.shared_a ? 2 : 1) * p.block_n * tc::BLOCK_K * 2;
  p.stages = (tc::MAX_SMEM - tc::BAR_BYTES - 1024) / stage_bytes;
  if (p.stages > tc::MAX_STAGES) p.stages = tc::MAX_STAGES;
  const int smem_bytes = p.stages * stage_bytes + tc::BAR_BYTES + 1024;
  const long long tiles = static_cast<long long>(p.tiles_m) * p.tiles_n * p.split_k;
  const int grid = static_cast<int>(tiles < ctx->num_sms ? tiles : ctx->num_sms);
  const int ph = prof_open(ctx, PROF_GEMM_TC, g.algo_flops, st);
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(grid);
  cfg.blockDim = dim3(tc::NUM_THREADS);
  cfg.dynamicSmemBytes = smem_bytes;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const cudaError_t le = cudaLaunchKernelEx(&cfg, tc::gemm_tc_kernel, tA0, tB0, tA1, tB1, p);
  ctx->launches++;
  if (le != cudaSuccess || p.split_k == 1 || g.force_split >= 1) {
    prof_close(ctx, ph, st);
    return check_cuda(ctx, le, "gemm_tc_kernel launch");
  }
  const long long quads = g.M * (g.N / 4);
  const cudaError_t re = launch_pdl(tc::splitk_reduce_kernel, dim3(static_cast<unsigned>((quads + 255) / 256)), dim3(256), 0, st,
                                    static_cast<const float*>(g.splitk), p.split_k, g.M, g.N,
                                    static_cast<__nv_bfloat16*>(g.epi.C0), g.epi.ld0);
  prof_close(ctx, ph, st);
  ctx->launches++;
  return check_cuda(ctx, re, "splitk_reduce_kernel launch");
}

}  // namespace ffsp
