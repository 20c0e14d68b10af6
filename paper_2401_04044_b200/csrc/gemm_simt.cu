// Plain fp32 GEMM (FMA units, no TF32) with the same epilogue contract as the
// tensor-core kernel.  Used for FFSPLIT_F32 layers, whose 1e-5 accuracy bound
// rules out reduced-precision tensor-core products.
//
//   acc[row, n] = sum_k A[row, k] * B[n, k]      A: [M, K], B: [N, K], K-major fp32
//
// 64 x 64 output tile per CTA, 16-deep K slices staged through shared memory,
// 4 x 4 outputs per thread.
#include "epilogue.cuh"
#include "internal.h"

namespace ffsp {
namespace simt {

constexpr int TM = 64, TN = 64, TK = 16, PITCH = TM + 4;

struct Params {
  const float* A0; const float* B0; const float* A1; const float* B1;
  long long lda0, ldb0, lda1, ldb1;
  long long M;
  int N, K;
  Epilogue epi;
  int* status;
};

__device__ __forceinline__ void load_slice(const float* __restrict__ src, long long ld, long long row0,
                                           long long rows, int k0, int K, float (*dst)[PITCH], int tid) {
  const int r = tid >> 2;
  const int kq = (tid & 3) * 4;
  const long long row = row0 + r;
  float v[4] = {0.f, 0.f, 0.f, 0.f};
  if (row < rows) {
    const float* p = src + row * ld + k0 + kq;
    if (k0 + kq + 4 <= K && ((reinterpret_cast<uintptr_t>(p) & 15u) == 0)) {
      const float4 t = *reinterpret_cast<const float4*>(p);
      v[0] = t.x; v[1] = t.y; v[2] = t.z; v[3] = t.w;
    } else {
#pragma unroll
      for (int i = 0; i < 4; ++i)
        if (k0 + kq + i < K) v[i] = p[i];
    }
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) dst[kq + i][r] = v[i];
}

template <bool DUAL>
__global__ void __launch_bounds__(256) gemm_simt_kernel(const Params p) {
  __shared__ __align__(16) float As[TK][PITCH];
  __shared__ __align__(16) float Bs[TK][PITCH];
  __shared__ __align__(16) float A1s[DUAL ? TK : 1][PITCH];
  __shared__ __align__(16) float B1s[DUAL ? TK : 1][PITCH];
  __shared__ float red[16][TN];

  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;
  if (blockIdx.x == 0 && blockIdx.y == 0 && tid < 32) check_blob_guard(p.epi, p.status, KID_GEMM_SIMT);
  const long long row0 = static_cast<long long>(blockIdx.y) * TM;
  const int col0 = blockIdx.x * TN;

  float acc[4][4], acc1[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) { acc[i][j] = 0.f; acc1[i][j] = 0.f; }

  for (int k0 = 0; k0 < p.K; k0 += TK) {
    load_slice(p.A0, p.lda0, row0, p.M, k0, p.K, As, tid);
    load_slice(p.B0, p.ldb0, col0, p.N, k0, p.K, Bs, tid);
    if (DUAL) {
      load_slice(p.A1, p.lda1, row0, p.M, k0, p.K, A1s, tid);
      load_slice(p.B1, p.ldb1, col0, p.N, k0, p.K, B1s, tid);
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < TK; ++kk) {
      const float4 a = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
      const float4 b = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
      const float av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
      if (DUAL) {
        const float4 a1 = *reinterpret_cast<const float4*>(&A1s[kk][ty * 4]);
        const float4 b1 = *reinterpret_cast<const float4*>(&B1s[kk][tx * 4]);
        const float a1v[4] = {a1.x, a1.y, a1.z, a1.w}, b1v[4] = {b1.x, b1.y, b1.z, b1.w};
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 4; ++j) acc1[i][j] = fmaf(a1v[i], b1v[j], acc1[i][j]);
      }
    }
    __syncthreads();
  }

  const Epilogue& e = p.epi;
  const bool score = e.col_partial != nullptr;
  float colsum[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const long long row = row0 + ty * 4 + i;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = col0 + tx * 4 + j;
      float v = acc[i][j];
      if (DUAL) {
        v = silu_precise_f(v) * acc1[i][j];
      } else {
        if (n < e.n_bias) v += e.bias[n];
        if (n < e.n_act || score) v = act_gelu(v, e.act);
      }
      if (score) {
        if (row < p.M) colsum[j] += e.score_abs ? fabsf(v) : v * v;
      } else if (row < p.M && n < p.N) {
        if (n < e.n_split) reinterpret_cast<float*>(e.C0)[row * e.ld0 + n] = v;
        else reinterpret_cast<float*>(e.C1)[row * e.ld1 + (n - e.n_split)] = v;
      }
    }
  }
  if (score) {
#pragma unroll
    for (int j = 0; j < 4; ++j) red[ty][tx * 4 + j] = colsum[j];
    __syncthreads();
    if (tid < TN) {
      float s = 0.f;
#pragma unroll
      for (int t = 0; t < 16; ++t) s += red[t][tid];  // fixed order
      const int n = col0 + tid;
      if (n < p.N) e.col_partial[static_cast<long long>(blockIdx.y) * p.N + n] = s;
    }
  }
}

}  // namespace simt

ffsplit_status launch_gemm_simt(ffsplit_ctx* ctx, const GemmArgs& g, cudaStream_t st) {
  if (g.M <= 0 || g.N <= 0) return FFSPLIT_OK;
  simt::Params p;
  p.A0 = static_cast<const float*>(g.A0); p.B0 = static_cast<const float*>(g.B0);
  p.A1 = static_cast<const float*>(g.A1); p.B1 = static_cast<const float*>(g.B1);
  p.lda0 = g.lda0; p.ldb0 = g.ldb0; p.lda1 = g.lda1; p.ldb1 = g.ldb1;
  p.M = g.M; p.N = g.N; p.K = g.K;
  p.epi = g.epi;
  p.status = ctx->status();
  const long long tiles_m = (g.M + simt::TM - 1) / simt::TM;
  if (tiles_m > 65535) return fail(ctx, FFSPLIT_ERR_SHAPE, "fp32 path: more than 65535*64 rows in one call");
  dim3 grid((g.N + simt::TN - 1) / simt::TN, static_cast<unsigned>(tiles_m));
  const int ph = prof_open(ctx, PROF_GEMM_SIMT, g.algo_flops, st);
  if (g.A1) simt::gemm_simt_kernel<true><<<grid, 256, 0, st>>>(p);
  else simt::gemm_simt_kernel<false><<<grid, 256, 0, st>>>(p);
  prof_close(ctx, ph, st);
  ctx->launches++;
  return check_cuda(ctx, cudaGetLastError(), "gemm_simt_kernel launch");
}

ffsplit_status launch_gemm_tc(ffsplit_ctx* ctx, const GemmArgs& g, cudaStream_t st);

ffsplit_status launch_gemm(ffsplit_ctx* ctx, int dtype, const GemmArgs& g, cudaStream_t st) {
  return dtype == FFSPLIT_BF16 ? launch_gemm_tc(ctx, g, st) : launch_gemm_simt(ctx, g, st);
}

}  // namespace ffsp
