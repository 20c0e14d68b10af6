// Fused light chain of the split forward (FFN_2 of Eq. 2 with rank-r factors):
//
//     P = sigma(Q B1 + b1[light]) A2          Q: [T, r], B1: [r, mL], A2: [mL, r]
//
// for GELU layers in bf16 with r_pad <= 256.  The T x mL activation matrix never
// leaves the SM: per 128-token tile and 64-neuron chunk
//   GEMM-a   S = Q_tile B1[:, chunk]            tcgen05.mma -> TMEM (double buffered)
//   epilogue H = GELU(S + b1)  -> bf16 -> shared memory in the 128B-swizzled K-major
//            layout the tensor core reads (double buffered)
//   GEMM-b   Pacc += H A2[chunk, :]             tcgen05.mma -> TMEM (resident accumulator)
// Warp roles: warp 0 TMA producer of the Q tile and the B1 ring, warp 1 MMA issuer,
// warps 2-9 epilogue, warp 10 TMA producer of the A2 ring (the two rings drain at
// different times: a B1 tile is free once GEMM-a has read it, an A2 tile one chunk later).
// The mL chunks of one token tile are spread over `splits`
// CTAs so that the grid covers the SMs; each CTA writes its fp32 partial of P and
// the last CTA to finish a token tile (atomic ticket) adds the partials in split
// order -- a fixed order, so the result does not depend on which CTA is last --
// and stores bf16 P.  Every wait is bounded (see gemm_tc.cu).
#include "epilogue.cuh"
#include "internal.h"
#include "ptx.cuh"

namespace ffsp {

ffsplit_status get_tmap_bf16(ffsplit_ctx* ctx, const void* ptr, long long rows, long long cols, long long ld,
                             int box_rows, CUtensorMap* out);

namespace fl {

constexpr int BLOCK_M = 128;
constexpr int CHUNK = 64;          // light neurons per chunk (N of GEMM-a, K of GEMM-b)
constexpr int KB = 64;             // K elements per shared-memory k-block (one 128-byte swizzle row)
constexpr int NUM_THREADS = 352;
constexpr int EPI_WARPS = 8;
constexpr int MAX_STAGES = 4;
constexpr int TMEM_COLS = 512;
constexpr int TMEM_S0 = 256;       // S buffers at columns 256 and 320; P accumulator at 0..255
constexpr int H_BYTES = BLOCK_M * CHUNK * 2;
constexpr int QKB_BYTES = BLOCK_M * KB * 2;
constexpr int B1KB_BYTES = CHUNK * KB * 2;
constexpr int BAR_BYTES = 512;
constexpr int MAX_SMEM = 232448;

struct Params {
  long long T;
  int r_pad, ml_pad, kbq;          // kbq = ceil(r_pad / 64)
  int n_chunks, splits, stages;     // stages: slots in each of the two rings
  int b1_slot_bytes, a2_slot_bytes;
  const float* b1l;
  __nv_bfloat16* P; long long ldp;  // output, bf16
  float* partial;                   // [splits][tiles_m * 128][r_pad] fp32 (splits > 1)
  int* tickets;                     // [tiles_m], zero before the launch, zero again after it
  int act;
  int* status;
};

__global__ void __launch_bounds__(NUM_THREADS, 1)
fused_light_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmB1,
                   const __grid_constant__ CUtensorMap tmA2, const Params p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* smem_q = smem;
  uint8_t* smem_h = smem_q + p.kbq * QKB_BYTES;
  uint8_t* smem_b1 = smem_h + 2 * H_BYTES;
  uint8_t* smem_a2 = smem_b1 + p.stages * p.b1_slot_bytes;
  uint64_t* bars = reinterpret_cast<uint64_t*>(smem_a2 + p.stages * p.a2_slot_bytes);
  uint64_t* b1full = bars;                    // [MAX_STAGES] TMA -> MMA (B1 tile of one chunk)
  uint64_t* b1empty = b1full + MAX_STAGES;    // [MAX_STAGES] GEMM-a done -> TMA
  uint64_t* a2full = b1empty + MAX_STAGES;    // [MAX_STAGES] TMA -> MMA (A2 tile of one chunk)
  uint64_t* a2empty = a2full + MAX_STAGES;    // [MAX_STAGES] GEMM-b done -> TMA
  uint64_t* sfull = a2empty + MAX_STAGES;     // [2] GEMM-a done -> epilogue
  uint64_t* sempty = sfull + 2;               // [2] epilogue has read S -> MMA
  uint64_t* hfull = sempty + 2;               // [2] epilogue wrote H -> MMA
  uint64_t* hempty = hfull + 2;               // [2] GEMM-b has read H -> epilogue
  uint64_t* qfull = hempty + 2;               // [1]
  uint64_t* pfull = qfull + 1;                // [1] all GEMM-b done -> epilogue
  uint64_t* redbar = pfull + 1;               // [1] epilogue warps rendezvous (partials written)
  uint64_t* drain = redbar + 1;               // [1]
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
    for (int s = 0; s < MAX_STAGES; ++s) {
      ptx::mbar_init(&b1full[s], 1);
      ptx::mbar_init(&b1empty[s], 1);
      ptx::mbar_init(&a2full[s], 1);
      ptx::mbar_init(&a2empty[s], 1);
    }
    for (int a = 0; a < 2; ++a) {
      ptx::mbar_init(&sfull[a], 1);
      ptx::mbar_init(&sempty[a], EPI_WARPS);
      ptx::mbar_init(&hfull[a], EPI_WARPS);
      ptx::mbar_init(&hempty[a], 1);
    }
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

  if (warp == 0) {
    if (lane == 0) {
      // ------------------------------------------------------------ TMA producer: Q tile, B1 ring
      bool ok = true;
      ptx::mbar_expect_tx(qfull, p.kbq * QKB_BYTES);
      for (int kb = 0; kb < p.kbq; ++kb) ptx::tma_load_2d(&tmQ, smem_q + kb * QKB_BYTES, qfull, kb * KB, m_blk * BLOCK_M);
      int issued = 0;
      for (int i = 0; i < my_chunks; ++i) {
        const int slot = i % p.stages;
        const uint32_t ph = (i / p.stages) & 1;
        if (!ptx::mbar_wait(&b1empty[slot], ph ^ 1, abort_flag)) { ok = false; break; }
        uint8_t* st = smem_b1 + slot * p.b1_slot_bytes;
        ptx::mbar_expect_tx(&b1full[slot], p.b1_slot_bytes);
        const int chunk = c_begin + i;
        for (int kb = 0; kb < p.kbq; ++kb) ptx::tma_load_2d(&tmB1, st + kb * B1KB_BYTES, &b1full[slot], kb * KB, chunk * CHUNK);
        issued = i + 1;
      }
      if (!ok) {
        const long long t0 = clock64();
        while (!ptx::mbar_try_wait(qfull, 0) && clock64() - t0 < ptx::kWaitLimitCycles / 8) {}
        const int first = issued > p.stages ? issued - p.stages : 0;
        for (int j = first; j < issued; ++j) {
          const long long t1 = clock64();
          while (!ptx::mbar_try_wait(&b1full[j % p.stages], (j / p.stages) & 1) &&
                 clock64() - t1 < ptx::kWaitLimitCycles / 8) {}
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    if (lane == 0) {
      // ------------------------------------------------------------ MMA issuer
      const uint32_t idesc_a = ptx::umma_idesc_bf16(BLOCK_M, CHUNK);
      const uint32_t idesc_b = ptx::umma_idesc_bf16(BLOCK_M, p.r_pad);
      bool ok = ptx::mbar_wait(qfull, 0, abort_flag);
      // GEMM-b of chunk j: Pacc += H[j & 1] * A2 tile of chunk j
      auto gemm_b = [&](int j) -> bool {
        const int hb = j & 1;
        if (!ptx::mbar_wait(&hfull[hb], (j >> 1) & 1, abort_flag)) return false;
        ptx::tc_fence_after();
        const int slot = j % p.stages;
        if (!ptx::mbar_wait(&a2full[slot], (j / p.stages) & 1, abort_flag)) return false;
        ptx::tc_fence_after();
        const uint64_t a_desc = ptx::umma_desc_k128(ptx::smem_u32(smem_h + hb * H_BYTES));
        const uint64_t b_desc = ptx::umma_desc_k128(ptx::smem_u32(smem_a2 + slot * p.a2_slot_bytes));
#pragma unroll
        for (int k = 0; k < CHUNK / 16; ++k)
          ptx::umma_bf16(tmem_base, a_desc + 2 * k, b_desc + 2 * k, idesc_b, (j | k) != 0 ? 1u : 0u);
        ptx::umma_commit(&a2empty[slot]);
        ptx::umma_commit(&hempty[hb]);
        return true;
      };
      for (int i = 0; i < my_chunks && ok; ++i) {
        const int slot = i % p.stages;
        if (!ptx::mbar_wait(&b1full[slot], (i / p.stages) & 1, abort_flag)) { ok = false; break; }
        const int sb = i & 1;
        if (!ptx::mbar_wait(&sempty[sb], ((i >> 1) & 1) ^ 1, abort_flag)) { ok = false; break; }
        ptx::tc_fence_after();
        const uint32_t d_tmem = tmem_base + TMEM_S0 + sb * CHUNK;
        for (int kb = 0; kb < p.kbq; ++kb) {
          const uint64_t a_desc = ptx::umma_desc_k128(ptx::smem_u32(smem_q + kb * QKB_BYTES));
          const uint64_t b_desc = ptx::umma_desc_k128(ptx::smem_u32(smem_b1 + slot * p.b1_slot_bytes + kb * B1KB_BYTES));
#pragma unroll
          for (int k = 0; k < KB / 16; ++k)
            ptx::umma_bf16(d_tmem, a_desc + 2 * k, b_desc + 2 * k, idesc_a, (kb | k) != 0 ? 1u : 0u);
        }
        ptx::umma_commit(&sfull[sb]);
        ptx::umma_commit(&b1empty[slot]);
        if (i > 0) ok = gemm_b(i - 1);   // keeps the tensor core busy while chunk i is in its epilogue
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
  } else if (warp == 10) {
    if (lane == 0) {
      // ------------------------------------------------------------ TMA producer: A2 ring
      bool ok = true;
      int issued = 0;
      for (int i = 0; i < my_chunks; ++i) {
        const int slot = i % p.stages;
        const uint32_t ph = (i / p.stages) & 1;
        if (!ptx::mbar_wait(&a2empty[slot], ph ^ 1, abort_flag)) { ok = false; break; }
        ptx::mbar_expect_tx(&a2full[slot], p.a2_slot_bytes);
        ptx::tma_load_2d(&tmA2, smem_a2 + slot * p.a2_slot_bytes, &a2full[slot], (c_begin + i) * CHUNK, 0);
        issued = i + 1;
      }
      if (!ok) {
        const int first = issued > p.stages ? issued - p.stages : 0;
        for (int j = first; j < issued; ++j) {
          const long long t1 = clock64();
          while (!ptx::mbar_try_wait(&a2full[j % p.stages], (j / p.stages) & 1) &&
                 clock64() - t1 < ptx::kWaitLimitCycles / 8) {}
        }
      }
    }
    __syncwarp();
  } else {
    // -------------------------------------------------------------- epilogue warps
    const int q = warp & 3;
    const int half = (warp - 2) >> 2;
    const int row_in_tile = q * 32 + lane;
    const uint32_t t_lane = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
    const GeluCoef gc = gelu_coef(p.act);
    bool ok = true;
    {
      // bring this CTA's slice of b1[light] towards the SM before the first chunk needs it
      const int te = threadIdx.x - 64;
      const char* b0 = reinterpret_cast<const char*>(p.b1l + static_cast<long long>(c_begin) * CHUNK);
      const long long bytes = (static_cast<long long>(min(c_end * CHUNK, p.ml_pad)) - static_cast<long long>(c_begin) * CHUNK) * 4;
      for (long long off = static_cast<long long>(te) * 128; off < bytes; off += 256 * 128)
        asm volatile("prefetch.global.L2 [%0];" ::"l"(b0 + off));
    }
    for (int i = 0; i < my_chunks; ++i) {
      if (warp == 2 && lane < 2 && i + 1 < my_chunks && (c_begin + i + 1) * CHUNK + lane * 32 < p.ml_pad)
        asm volatile("prefetch.global.L1 [%0];" ::"l"(p.b1l + static_cast<long long>(c_begin + i + 1) * CHUNK + lane * 32));
      const int sb = i & 1;
      const uint32_t ph = (i >> 1) & 1;
      if (!ptx::mbar_wait(&sfull[sb], ph, abort_flag)) { ok = false; break; }
      ptx::tc_fence_after();
      float v[32];
      const int c0 = half * 32;
      ptx::tmem_ld16(t_lane + TMEM_S0 + sb * CHUNK + c0, v);
      ptx::tmem_ld16(t_lane + TMEM_S0 + sb * CHUNK + c0 + 16, v + 16);
      ptx::tmem_ld_wait();
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&sempty[sb]);
      const int n0 = (c_begin + i) * CHUNK + c0;
      if (n0 + 32 <= p.ml_pad) {
        const float4* b = reinterpret_cast<const float4*>(p.b1l + n0);
#pragma unroll
        for (int j = 0; j < 8; ++j) {
          const float4 t = __ldg(b + j);
          v[4 * j] += t.x; v[4 * j + 1] += t.y; v[4 * j + 2] += t.z; v[4 * j + 3] += t.w;
        }
      } else {
#pragma unroll
        for (int j = 0; j < 32; ++j)
          if (n0 + j < p.ml_pad) v[j] += __ldg(p.b1l + n0 + j);
      }
      uint32_t w[16];
#pragma unroll
      for (int j = 0; j < 16; ++j) w[j] = pack_bf16x2(gelu_fast(v[2 * j], gc), gelu_fast(v[2 * j + 1], gc));
      if (!ptx::mbar_wait(&hempty[sb], ph ^ 1, abort_flag)) { ok = false; break; }
      // row `row_in_tile` of the [128 x 64] K-major tile: 128 bytes, 16-byte pieces XOR-swizzled by row % 8
      uint8_t* hrow = smem_h + sb * H_BYTES + row_in_tile * 128;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int piece = (c0 >> 3) + j;
        uint4 val;
        val.x = w[4 * j]; val.y = w[4 * j + 1]; val.z = w[4 * j + 2]; val.w = w[4 * j + 3];
        *reinterpret_cast<uint4*>(hrow + ((piece ^ (row_in_tile & 7)) << 4)) = val;
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(&hfull[sb]);
    }
    // ---- the tile's accumulator: TMEM -> shared memory (fp32, padded rows) -> coalesced global
    if (ok && my_chunks > 0) ok = ptx::mbar_wait(pfull, 0, abort_flag);
    if (ok) {
      ptx::tc_fence_after();
      // every MMA and every TMA load of this CTA has completed: the operand buffers are free
      float* stage = reinterpret_cast<float*>(smem);
      const int pitch = p.r_pad + 4;   // keeps the row-per-thread float4 writes free of bank conflicts
      for (int c = half * 16; c < p.r_pad; c += 32) {
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
      const int te = threadIdx.x - 64;            // 0..255 among the epilogue threads
      const int q4 = p.r_pad >> 2;                 // float4 per row
      const int n4 = BLOCK_M * q4;
      const long long row0 = static_cast<long long>(m_blk) * BLOCK_M;
      const long long rows_total = static_cast<long long>(gridDim.y) * BLOCK_M;
      const int pitch = p.r_pad + 4;
      const float* stage = reinterpret_cast<const float*>(smem);
      if (p.splits > 1) {
        float4* mine = reinterpret_cast<float4*>(p.partial + (static_cast<long long>(split) * rows_total + row0) * p.r_pad);
        for (int e = te; e < n4; e += 256) {
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
        // Batches of 4 x 4 independent loads per thread: the sum over splits is taken in split order
        // (so it does not depend on which CTA is last) but the loads do not wait for one another.
        constexpr int EG = 4;
        for (int e0 = te; e0 < n4; e0 += 256 * EG) {
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
                const int e = e0 + j * 256;
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
            const int e = e0 + j * 256;
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
  p.b1_slot_bytes = p.kbq * fl::B1KB_BYTES;
  p.a2_slot_bytes = r_pad * fl::KB * 2;
  const int fixed = p.kbq * fl::QKB_BYTES + 2 * fl::H_BYTES + fl::BAR_BYTES + 1024;
  int stages = (fl::MAX_SMEM - fixed) / (p.b1_slot_bytes + p.a2_slot_bytes);
  if (stages > fl::MAX_STAGES) stages = fl::MAX_STAGES;
  if (stages < 2) return fail(ctx, FFSPLIT_ERR_SHAPE, "fused light chain: shared memory too small for this rank");
  p.stages = stages;
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
  const int smem_bytes = fixed + stages * (p.b1_slot_bytes + p.a2_slot_bytes);
  if (!ctx->attr_fused_set) {
    cudaError_t e = cudaFuncSetAttribute(fl::fused_light_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         fl::MAX_SMEM);
    if (e != cudaSuccess) return check_cuda(ctx, e, "cudaFuncSetAttribute(fused_light_kernel)");
    ctx->attr_fused_set = true;
  }
  dim3 grid(p.splits, static_cast<unsigned>(tiles_m));
  const int ph = prof_open(ctx, PROF_GEMM_TC, algo_flops, st);
  fl::fused_light_kernel<<<grid, fl::NUM_THREADS, smem_bytes, st>>>(tQ, tB1, tA2, p);
  prof_close(ctx, ph, st);
  ctx->launches++;
  return check_cuda(ctx, cudaGetLastError(), "fused_light_kernel launch");
}

}  // namespace ffsp
