// The transformer block around the feed-forward network, at BERT-base shape (Section 5.1.2 / Table 2 time whole
// BERT-base models, whose layers are: multi-head self-attention, residual + LayerNorm, FFN, residual + LayerNorm).
// Only what the split FFN needs to be timed inside a whole layer: head width 64, sequences of at most 128 tokens
// (one tile), no padding mask, post-LayerNorm order, bf16 activations.
//
//   attention_kernel   one CTA per (sequence, head): S = Q K^T (tcgen05.mma into tensor memory), row softmax in
//                      registers (one thread per query row), P written back into tensor memory as bf16 and used
//                      as the left operand of O = P V; V is transposed in shared memory into the K-major form
//                      the right operand needs.  Q, K, V tiles come by TMA from the fused projection [T, 3 d].
//   add_layernorm_kernel   y = LayerNorm(x + r) * gamma + beta, one warp per token row, fp32 statistics.
// The projections themselves are the library's tensor-core GEMM (bias in its epilogue).
// Every wait is bounded as in gemm_tc.cu.
#include <cstring>

#include "epilogue.cuh"
#include "internal.h"
#include "ptx.cuh"

namespace ffsp {

ffsplit_status get_tmap_bf16(ffsplit_ctx* ctx, const void* ptr, long long rows, long long cols, long long ld,
                             int box_rows, CUtensorMap* out);

namespace enc {

constexpr int SEQ_TILE = 128;     // query rows = key rows per CTA
constexpr int DH = 64;            // head width
constexpr int ATT_THREADS = 160;  // warps 0-3: one query row per thread; warp 4: TMA and MMA issue
constexpr int TILE_BYTES = SEQ_TILE * DH * 2;   // 16 KB: a Q, K or V tile, or the transposed V
constexpr int TMEM_COLS = 128;    // S at columns 0..127; P (bf16, two per column) compacted in place into 0..63; O at 64..127
constexpr int ATT_SMEM = 4 * TILE_BYTES + 1024 + 256;

struct AttParams {
  int seq, heads, d;              // tokens per sequence (<= 128), heads, model width (heads * 64)
  __nv_bfloat16* O;               // [T, d]
  float scale_log2e;              // log2(e) / sqrt(64)
  int* status;
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
__device__ __forceinline__ float ex2_approx(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// Byte offset of element (row, col) of a K-major operand tile with 128-byte swizzle (rows of 64 elements).
__device__ __forceinline__ int swz_elem(int row, int col) {
  return (row >> 3) * 1024 + (row & 7) * 128 + ((((col >> 3) ^ (row & 7))) << 4) + (col & 7) * 2;
}

__global__ void __launch_bounds__(ATT_THREADS)
attention_kernel(const __grid_constant__ CUtensorMap tmQKV, const AttParams p) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~uintptr_t(1023));
  uint8_t* sQ = smem;
  uint8_t* sK = sQ + TILE_BYTES;
  uint8_t* sV = sK + TILE_BYTES;
  uint8_t* sVt = sV + TILE_BYTES;               // two k-blocks of [64 head columns][64 keys]
  uint64_t* bars = reinterpret_cast<uint64_t*>(sVt + TILE_BYTES);
  uint64_t* ld_full = bars;        // TMA: Q, K, V landed
  uint64_t* s_full = bars + 1;     // S = Q K^T complete
  uint64_t* p_full = bars + 2;     // softmax wrote P (4 warps)
  uint64_t* vt_full = bars + 3;    // V^T written (4 warps)
  uint64_t* o_full = bars + 4;     // O = P V complete
  uint32_t* tmem_holder = reinterpret_cast<uint32_t*>(bars + 5);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_holder + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int head = blockIdx.x, seq_id = blockIdx.y;
  const long long row0 = static_cast<long long>(seq_id) * p.seq;

  if (threadIdx.x == 0) {
    ptx::mbar_init(ld_full, 1);
    ptx::mbar_init(s_full, 1);
    ptx::mbar_init(p_full, 4);
    ptx::mbar_init(vt_full, 4);
    ptx::mbar_init(o_full, 1);
    *abort_flag = 0;
    ptx::mbar_fence_init();
    ptx::prefetch_tmap(&tmQKV);
  }
  if (warp == 4) {
    ptx::tmem_alloc(tmem_holder, TMEM_COLS);
    ptx::tmem_relinquish();
  }
  ptx::tc_fence_before();
  __syncthreads();
  ptx::tc_fence_after();
  const uint32_t tmem_base = *tmem_holder;
  pdl_wait();

  if (warp == 4) {
    if (ptx::elect_one()) {
      // rows past the end of the tensor read as zeros; rows past this sequence belong to the next one and are
      // masked (keys) or not stored (queries)
      ptx::mbar_expect_tx(ld_full, 3 * TILE_BYTES);
      ptx::tma_load_2d(&tmQKV, sQ, ld_full, head * DH, static_cast<int>(row0));
      ptx::tma_load_2d(&tmQKV, sK, ld_full, p.d + head * DH, static_cast<int>(row0));
      ptx::tma_load_2d(&tmQKV, sV, ld_full, 2 * p.d + head * DH, static_cast<int>(row0));
      bool ok = ptx::mbar_wait(ld_full, 0, abort_flag);
      if (ok) {
        ptx::tc_fence_after();
        const uint32_t idesc = ptx::umma_idesc_bf16(SEQ_TILE, SEQ_TILE);
        const uint64_t a_desc = ptx::umma_desc_k128(ptx::smem_u32(sQ));
        const uint64_t b_desc = ptx::umma_desc_k128(ptx::smem_u32(sK));
#pragma unroll
        for (int k = 0; k < DH / 16; ++k) ptx::umma_bf16(tmem_base, a_desc + 2 * k, b_desc + 2 * k, idesc, k != 0 ? 1u : 0u);
        ptx::umma_commit(s_full);
      }
      if (ok) ok = ptx::mbar_wait(p_full, 0, abort_flag);
      if (ok) ok = ptx::mbar_wait(vt_full, 0, abort_flag);
      if (ok) {
        ptx::tc_fence_after();
        const uint32_t idesc = ptx::umma_idesc_bf16(SEQ_TILE, DH);
        const uint64_t v_desc = ptx::umma_desc_k128(ptx::smem_u32(sVt));
#pragma unroll
        for (int jj = 0; jj < SEQ_TILE / 16; ++jj) {
          // 16 keys per step: P sits as packed bf16 in columns 0..63, 8 columns per step
          const uint64_t b_desc = v_desc + static_cast<uint64_t>(((jj >> 2) * (TILE_BYTES / 2)) >> 4) + 2 * (jj & 3);
          umma_bf16_ts(tmem_base + 64, tmem_base + 8 * jj, b_desc, idesc, jj != 0 ? 1u : 0u);
        }
        ptx::umma_commit(o_full);
      }
    }
    __syncwarp();
  } else {
    const int row = warp * 32 + lane;                  // query row of this thread = TMEM lane
    const uint32_t t_row = tmem_base + (static_cast<uint32_t>(warp * 32) << 16);
    bool ok = ptx::mbar_wait(ld_full, 0, abort_flag);
    if (ok) {
      // V^T: this thread's key row of V (64 head columns) scattered into the K-major [head column][key] tile
      const int kb = row >> 6, kc = row & 63;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const uint4 piece = *reinterpret_cast<const uint4*>(sV + (row >> 3) * 1024 + (row & 7) * 128 + ((j ^ (row & 7)) << 4));
        const __nv_bfloat16* e = reinterpret_cast<const __nv_bfloat16*>(&piece);
#pragma unroll
        for (int i = 0; i < 8; ++i)
          *reinterpret_cast<__nv_bfloat16*>(sVt + kb * (TILE_BYTES / 2) + swz_elem(8 * j + i, kc)) = e[i];
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(vt_full);
      ok = ptx::mbar_wait(s_full, 0, abort_flag);
    }
    float inv_sum = 0.f;
    if (ok) {
      ptx::tc_fence_after();
      // pass 1: row maximum over the valid keys
      float mx = -INFINITY;
#pragma unroll
      for (int c = 0; c < SEQ_TILE; c += 32) {
        float v[2][16];
        ptx::tmem_ld16(t_row + c, v[0]);
        ptx::tmem_ld16(t_row + c + 16, v[1]);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int u = 0; u < 2; ++u)
#pragma unroll
          for (int i = 0; i < 16; ++i)
            if (c + 16 * u + i < p.seq) mx = fmaxf(mx, v[u][i]);
      }
      // pass 2: exponentials, their sum, P as bf16 compacted into columns 0..63 (the 32 columns of group c become
      // the 16 columns from c / 2: always columns this thread has already consumed)
      float sum = 0.f;
      const float off = mx * p.scale_log2e;
#pragma unroll
      for (int c = 0; c < SEQ_TILE; c += 32) {
        float v[2][16];
        uint32_t w[16];
        ptx::tmem_ld16(t_row + c, v[0]);
        ptx::tmem_ld16(t_row + c + 16, v[1]);
        ptx::tmem_ld_wait();
#pragma unroll
        for (int u = 0; u < 2; ++u)
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            const int k0 = c + 16 * u + 2 * i;
            float e0 = k0 < p.seq ? ex2_approx(fmaf(v[u][2 * i], p.scale_log2e, -off)) : 0.f;
            float e1 = k0 + 1 < p.seq ? ex2_approx(fmaf(v[u][2 * i + 1], p.scale_log2e, -off)) : 0.f;
            // the sum is taken over the rounded values the second product will use
            const uint32_t pk = pack_bf16x2(e0, e1);
            w[8 * u + i] = pk;
            sum += __uint_as_float(pk << 16) + __uint_as_float(pk & 0xffff0000u);
          }
        tmem_st16(t_row + (c >> 1), w);
      }
      tmem_st_wait();
      inv_sum = 1.0f / sum;
      ptx::tc_fence_before();
      __syncwarp();
      if (lane == 0) ptx::mbar_arrive(p_full);
      ok = ptx::mbar_wait(o_full, 0, abort_flag);
    }
    if (ok) {
      ptx::tc_fence_after();
      __nv_bfloat16* dst = p.O + (row0 + row) * p.d + head * DH;
#pragma unroll
      for (int c = 0; c < DH; c += 32) {
        float v[2][16];
        ptx::tmem_ld16(t_row + 64 + c, v[0]);
        ptx::tmem_ld16(t_row + 64 + c + 16, v[1]);
        ptx::tmem_ld_wait();
        if (row < p.seq) {
#pragma unroll
          for (int u = 0; u < 2; ++u) {
            uint4 a, b;
            a.x = pack_bf16x2(v[u][0] * inv_sum, v[u][1] * inv_sum);   a.y = pack_bf16x2(v[u][2] * inv_sum, v[u][3] * inv_sum);
            a.z = pack_bf16x2(v[u][4] * inv_sum, v[u][5] * inv_sum);   a.w = pack_bf16x2(v[u][6] * inv_sum, v[u][7] * inv_sum);
            b.x = pack_bf16x2(v[u][8] * inv_sum, v[u][9] * inv_sum);   b.y = pack_bf16x2(v[u][10] * inv_sum, v[u][11] * inv_sum);
            b.z = pack_bf16x2(v[u][12] * inv_sum, v[u][13] * inv_sum); b.w = pack_bf16x2(v[u][14] * inv_sum, v[u][15] * inv_sum);
            uint4* o = reinterpret_cast<uint4*>(dst + c + 16 * u);
            o[0] = a;
            o[1] = b;
          }
        }
      }
    }
  }
  ptx::tc_fence_before();
  __syncthreads();
  if (threadIdx.x == 0 && *abort_flag) record_status(p.status, FFSPLIT_ERR_TIMEOUT, blockIdx.y * gridDim.x + blockIdx.x, KID_ENCODER);
  if (warp == 4) {
    ptx::tc_fence_after();
    ptx::tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

// y = LayerNorm(x + r) * gamma + beta over rows of d elements (d % 8 == 0), one warp per row.
constexpr int LN_MAX_VEC = 4;   // up to 4 x 8 elements per lane: d <= 1024
__global__ void __launch_bounds__(256) add_layernorm_kernel(const __nv_bfloat16* x, const __nv_bfloat16* r,
                                                            const float* gamma, const float* beta, float eps,
                                                            long long rows, int d, __nv_bfloat16* y) {
  pdl_wait();
  const long long row = static_cast<long long>(blockIdx.x) * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= rows) return;
  const int nvec = d / 8;
  float v[LN_MAX_VEC][8];
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < LN_MAX_VEC; ++i) {
    const int j = lane + 32 * i;
    if (j < nvec) {
      const uint4 a = *reinterpret_cast<const uint4*>(x + row * d + 8 * j);
      const uint4 b = *reinterpret_cast<const uint4*>(r + row * d + 8 * j);
      const __nv_bfloat16* ea = reinterpret_cast<const __nv_bfloat16*>(&a);
      const __nv_bfloat16* eb = reinterpret_cast<const __nv_bfloat16*>(&b);
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        v[i][e] = __bfloat162float(ea[e]) + __bfloat162float(eb[e]);
        s += v[i][e];
      }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  const float mean = s / d;
  float q = 0.f;
#pragma unroll
  for (int i = 0; i < LN_MAX_VEC; ++i) {
    const int j = lane + 32 * i;
    if (j < nvec) {
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        const float t = v[i][e] - mean;
        q = fmaf(t, t, q);
      }
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) q += __shfl_xor_sync(0xffffffffu, q, o);
  const float rstd = rsqrtf(q / d + eps);
#pragma unroll
  for (int i = 0; i < LN_MAX_VEC; ++i) {
    const int j = lane + 32 * i;
    if (j < nvec) {
      uint4 o;
      uint32_t* ow = reinterpret_cast<uint32_t*>(&o);
#pragma unroll
      float gm[8], bt[8];
      *reinterpret_cast<float4*>(gm) = __ldg(reinterpret_cast<const float4*>(gamma + 8 * j));
      *reinterpret_cast<float4*>(gm + 4) = __ldg(reinterpret_cast<const float4*>(gamma + 8 * j) + 1);
      *reinterpret_cast<float4*>(bt) = __ldg(reinterpret_cast<const float4*>(beta + 8 * j));
      *reinterpret_cast<float4*>(bt + 4) = __ldg(reinterpret_cast<const float4*>(beta + 8 * j) + 1);
#pragma unroll
      for (int e = 0; e < 8; e += 2)
        ow[e / 2] = pack_bf16x2(fmaf((v[i][e] - mean) * rstd, gm[e], bt[e]), fmaf((v[i][e + 1] - mean) * rstd, gm[e + 1], bt[e + 1]));
      *reinterpret_cast<uint4*>(y + row * d + 8 * j) = o;
    }
  }
}

}  // namespace enc

namespace {

constexpr size_t kAlignE = 256;
inline size_t align_e(size_t v) { return (v + kAlignE - 1) / kAlignE * kAlignE; }

struct EncLayout { size_t qkv, att, proj, x1, ffn, end; };
EncLayout enc_layout(size_t ffn_end, long long T, int d) {
  EncLayout L;
  size_t off = align_e(ffn_end);
  L.qkv = off;  off = align_e(off + static_cast<size_t>(T) * 3 * d * 2);   // [T, 3 d] fused projection
  L.att = off;  off = align_e(off + static_cast<size_t>(T) * d * 2);       // attention output, heads concatenated
  L.proj = off; off = align_e(off + static_cast<size_t>(T) * d * 2);       // output projection
  L.x1 = off;   off = align_e(off + static_cast<size_t>(T) * d * 2);       // LayerNorm(X + attention)
  L.ffn = off;  off = align_e(off + static_cast<size_t>(T) * d * 2);       // FFN output
  L.end = off;
  return L;
}

ffsplit_status check_encoder(ffsplit_ctx* ctx, const ffsplit_encoder_layer* e) {
  if (!e) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "layer description is NULL");
  if (e->batch < 1 || e->seq < 1 || e->heads < 1) return fail(ctx, FFSPLIT_ERR_SHAPE, "batch, seq and heads must be >= 1");
  if (e->seq > enc::SEQ_TILE) return fail(ctx, FFSPLIT_ERR_SHAPE, "sequences of at most 128 tokens");
  if (e->heads * enc::DH > 1024) return fail(ctx, FFSPLIT_ERR_SHAPE, "model width heads * 64 of at most 1024");
  if (!e->Wqkv_t || !e->bqkv || !e->Wo_t || !e->bo || !e->ln1_gamma || !e->ln1_beta || !e->ln2_gamma || !e->ln2_beta ||
      !e->ffn_blob)
    return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "NULL tensor in the layer description");
  if (!aligned16(e->Wqkv_t) || !aligned16(e->Wo_t) || !aligned16(e->bqkv) || !aligned16(e->bo) || !aligned16(e->ln1_gamma) ||
      !aligned16(e->ln1_beta) || !aligned16(e->ln2_gamma) || !aligned16(e->ln2_beta))
    return fail(ctx, FFSPLIT_ERR_ALIGN, "weights, biases and LayerNorm parameters must be 16-byte aligned");
  return FFSPLIT_OK;
}

ffsplit_status projection(ffsplit_ctx* ctx, const void* X, const void* Wt, const float* bias, long long T, int N, int K,
                          void* C, cudaStream_t st) {
  GemmArgs g;
  std::memset(&g, 0, sizeof(g));
  g.A0 = X; g.lda0 = K; g.B0 = Wt; g.ldb0 = K;
  g.M = T; g.N = N; g.K = K;
  g.algo_flops = 2.0 * T * N * K;
  g.epi.C0 = C; g.epi.ld0 = N; g.epi.n_split = N;
  g.epi.bias = bias; g.epi.n_bias = N;
  g.epi.act = FFSPLIT_GELU_ERF;   // no column is activated (n_act = 0)
  return launch_gemm(ctx, FFSPLIT_BF16, g, st);
}

}  // namespace
}  // namespace ffsp

extern "C" {

ffsplit_status ffsplit_encoder_workspace_size(ffsplit_ctx* ctx, const ffsplit_encoder_layer* layer, size_t* bytes) {
  using namespace ffsp;
  if (!ctx || !bytes) return FFSPLIT_ERR_INVALID_ARG;
  ffsplit_status s = check_encoder(ctx, layer);
  if (s != FFSPLIT_OK) return s;
  const long long T = static_cast<long long>(layer->batch) * layer->seq;
  int fd = 0, fdt = 0;
  const size_t ffn_end = ffn_forward_workspace_end(ctx, layer->ffn_blob, T, &s, &fd, &fdt);
  if (s != FFSPLIT_OK) return s;
  if (fd != layer->heads * enc::DH || fdt != FFSPLIT_BF16)
    return fail(ctx, FFSPLIT_ERR_SHAPE, "the FFN blob must be a bf16 layer of width heads * 64");
  *bytes = kCtrlBytes + enc_layout(ffn_end, T, layer->heads * enc::DH).end;
  return FFSPLIT_OK;
}

ffsplit_status ffsplit_encoder_forward(ffsplit_ctx* ctx, const ffsplit_encoder_layer* layer, const void* X, void* Y,
                                       void* stream) {
  using namespace ffsp;
  if (!ctx) return FFSPLIT_ERR_INVALID_ARG;
  ffsplit_status s = check_encoder(ctx, layer);
  if (s != FFSPLIT_OK) return s;
  if (!X || !Y) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "NULL tensor");
  if (!aligned16(X) || !aligned16(Y)) return fail(ctx, FFSPLIT_ERR_ALIGN, "X and Y must be 16-byte aligned");
  const int d = layer->heads * enc::DH;
  const long long T = static_cast<long long>(layer->batch) * layer->seq;
  int fd = 0, fdt = 0;
  const size_t ffn_end = ffn_forward_workspace_end(ctx, layer->ffn_blob, T, &s, &fd, &fdt);
  if (s != FFSPLIT_OK) return s;
  if (fd != d || fdt != FFSPLIT_BF16) return fail(ctx, FFSPLIT_ERR_SHAPE, "the FFN blob must be a bf16 layer of width heads * 64");
  const EncLayout L = enc_layout(ffn_end, T, d);
  if (!ctx->ws || kCtrlBytes + L.end > ctx->ws_bytes)
    return fail(ctx, FFSPLIT_ERR_BUFFER_TOO_SMALL, "workspace too small for this layer (ffsplit_encoder_workspace_size)");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  char* base = ctx->ws + kCtrlBytes;
  char* QKV = base + L.qkv;
  char* ATT = base + L.att;
  char* PROJ = base + L.proj;
  char* X1 = base + L.x1;
  char* FFN = base + L.ffn;
  // fused Q, K, V projection
  if ((s = projection(ctx, X, layer->Wqkv_t, layer->bqkv, T, 3 * d, d, QKV, st)) != FFSPLIT_OK) return s;
  // attention, one CTA per (sequence, head)
  {
    enc::AttParams p;
    p.seq = layer->seq; p.heads = layer->heads; p.d = d;
    p.O = reinterpret_cast<__nv_bfloat16*>(ATT);
    p.scale_log2e = 1.4426950408889634f / 8.0f;
    p.status = ctx->status();
    CUtensorMap tm;
    if ((s = get_tmap_bf16(ctx, QKV, T, 3 * d, 3 * d, enc::SEQ_TILE, &tm)) != FFSPLIT_OK) return s;
    if (!ctx->attr_att_set) {
      cudaError_t e = cudaFuncSetAttribute(enc::attention_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, enc::ATT_SMEM);
      if (e != cudaSuccess) return check_cuda(ctx, e, "cudaFuncSetAttribute(attention_kernel)");
      ctx->attr_att_set = true;
    }
    const cudaError_t e = launch_pdl(enc::attention_kernel, dim3(layer->heads, layer->batch), dim3(enc::ATT_THREADS),
                                     enc::ATT_SMEM, st, tm, p);
    ctx->launches++;
    if (e != cudaSuccess) return check_cuda(ctx, e, "attention_kernel launch");
  }
  // output projection, residual + LayerNorm
  if ((s = projection(ctx, ATT, layer->Wo_t, layer->bo, T, d, d, PROJ, st)) != FFSPLIT_OK) return s;
  const unsigned ln_blocks = static_cast<unsigned>((T + 7) / 8);
  cudaError_t e = launch_pdl(enc::add_layernorm_kernel, dim3(ln_blocks), dim3(256), 0, st,
                             static_cast<const __nv_bfloat16*>(X), reinterpret_cast<const __nv_bfloat16*>(PROJ),
                             layer->ln1_gamma, layer->ln1_beta, layer->ln_eps, T, d, reinterpret_cast<__nv_bfloat16*>(X1));
  ctx->launches++;
  if (e != cudaSuccess) return check_cuda(ctx, e, "add_layernorm_kernel launch");
  // the feed-forward network (split or dense, as packed), residual + LayerNorm
  if ((s = run_ffn_forward(ctx, layer->ffn_blob, X1, T, FFN, st)) != FFSPLIT_OK) return s;
  e = launch_pdl(enc::add_layernorm_kernel, dim3(ln_blocks), dim3(256), 0, st,
                 reinterpret_cast<const __nv_bfloat16*>(X1), reinterpret_cast<const __nv_bfloat16*>(FFN),
                 layer->ln2_gamma, layer->ln2_beta, layer->ln_eps, T, d, static_cast<__nv_bfloat16*>(Y));
  ctx->launches++;
  return check_cuda(ctx, e, "add_layernorm_kernel launch");
}

}  // extern "C"
