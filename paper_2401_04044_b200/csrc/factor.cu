// On-device rank-r factors of the light slices (Section 5.1.1: the low-rank decomposition is applied to
// U2 and V2 only), so that score -> select -> factor -> pack runs without leaving the GPU.
//
// For W = U2 (d x mL) and for W = V2^T (d x mL) the routine finds an orthonormal basis Q (d x r) of the
// dominant left singular subspace by block power iteration (orthogonal iteration) from a starting basis
// given by the caller:
//     repeat `iters` times:   Y = W (W^T Q),   Q = orth(Y)
// and returns the factors of the projection W ~ Q (Q^T W):
//     U2 ~ A1 B1 with A1 = Q,        B1 = Q^T U2
//     V2 ~ A2 B2 with A2 = V2 Q,     B2 = Q^T
// Q Q^T W is the best approximation of W whose columns lie in span(Q); as span(Q) converges to the span of
// the r leading left singular vectors it becomes the truncated SVD's product (Eckart-Young).  The factors
// differ from the SVD's by an invertible r x r mixing, which the forward never sees.
//
// All thin matrices are kept transposed (r rows), so every product is the library's K-major GEMM:
//     Z^T [r, n] = Q^T [r, d] . (W^T [n, d])^T      Y^T [r, d] = Z^T [r, n] . (W [d, n])^T
//     G   [r, r] = Y^T . (Y^T)^T   in fp32           Q^T = L^-1 Y^T  with G = L L^T (Cholesky QR)
// The two big products run on the tensor cores in bf16 with fp32 accumulation; the Gram matrix, its
// Cholesky factor and the triangular solve are fp32.
#include <cstring>

#include "epilogue.cuh"
#include "internal.h"

namespace ffsp {
namespace fac {

// In-place Cholesky factorisation of the leading r x r block of G (row-major, pitch ld), lower triangle,
// right-looking in block columns of NB: one CTA factors the block column (panel_kernel), then a grid of CTAs
// applies it to the trailing matrix, one 32 x 32 tile of the lower triangle each (update_kernel).  A pivot
// that is not a positive finite number is reported (FFSPLIT_ERR_NONFINITE, detail = column) and replaced by 1
// so that the factorisation finishes with finite numbers.
constexpr int NB = 32;
constexpr int CHOL_THREADS = 1024;
__global__ void __launch_bounds__(CHOL_THREADS) chol_panel_kernel(float* G, int r, int ld, int j0, int* status) {
  __shared__ float col[2048];
  __shared__ float pivot;
  pdl_wait();
  const int j1 = j0 + NB < r ? j0 + NB : r;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int j = j0; j < j1; ++j) {
    if (threadIdx.x == 0) {
      float p = G[static_cast<size_t>(j) * ld + j];
      if (!(p > 0.f) || !isfinite(p)) {
        record_status(status, FFSPLIT_ERR_NONFINITE, j, KID_FACTOR);
        p = 1.f;
      }
      pivot = sqrtf(p);
      G[static_cast<size_t>(j) * ld + j] = pivot;
    }
    __syncthreads();
    const float inv = 1.0f / pivot;
    for (int i = j + 1 + threadIdx.x; i < r; i += CHOL_THREADS) {
      const float v = G[static_cast<size_t>(i) * ld + j] * inv;
      G[static_cast<size_t>(i) * ld + j] = v;
      col[i] = v;
    }
    __syncthreads();
    // the rest of this block column: G[i, l] -= L[i, j] L[l, j] for j < l < j1, l <= i (one warp per row)
    for (int i = j + 1 + warp; i < r; i += CHOL_THREADS / 32) {
      const int l = j + 1 + lane;
      if (l < j1 && l <= i) G[static_cast<size_t>(i) * ld + l] -= col[i] * col[l];
    }
    __syncthreads();
  }
}

// Trailing update with a finished block column P = L[:, j0 .. j0 + NB): G[i, l] -= sum_k P[i, k] P[l, k] for
// j0 + NB <= l <= i.  CTA t owns tile (a, b), b <= a, of the trailing lower triangle (t = a (a + 1) / 2 + b).
__global__ void __launch_bounds__(CHOL_THREADS) chol_update_kernel(float* G, int r, int ld, int j0) {
  __shared__ float Pi[NB][NB + 1];
  __shared__ float Pl[NB][NB + 1];
  pdl_wait();
  const int t = blockIdx.x;
  int a = static_cast<int>((sqrtf(8.0f * t + 1.0f) - 1.0f) * 0.5f);
  while (a * (a + 1) / 2 > t) --a;
  while ((a + 1) * (a + 2) / 2 <= t) ++a;
  const int b = t - a * (a + 1) / 2;
  const int n0 = j0 + NB;
  const int ty = threadIdx.x >> 5, tx = threadIdx.x & 31;
  const int ri = n0 + NB * a + ty, rl = n0 + NB * b + ty;
  Pi[ty][tx] = ri < r ? G[static_cast<size_t>(ri) * ld + j0 + tx] : 0.f;
  Pl[ty][tx] = rl < r ? G[static_cast<size_t>(rl) * ld + j0 + tx] : 0.f;
  __syncthreads();
  const int i = n0 + NB * a + ty, l = n0 + NB * b + tx;
  if (i < r && l <= i) {
    float s = 0.f;
#pragma unroll
    for (int k = 0; k < NB; ++k) s = fmaf(Pi[ty][k], Pl[tx][k], s);
    G[static_cast<size_t>(i) * ld + l] -= s;
  }
}

// Q^T = L^-1 Y^T by forward substitution, one thread per column c of Y^T [r, d] (bf16), L the lower
// triangle of G.  Rows are taken in blocks of TB: the part of the sum over earlier blocks is accumulated
// for all TB rows at once from a tile of L staged in shared memory, then the block's own triangle is
// solved.  The running fp32 solution lives in Qf [r, d] (coalesced across threads); Q^T is stored as bf16.
constexpr int TB = 32;
constexpr int TRSM_THREADS = 128;
__global__ void __launch_bounds__(TRSM_THREADS) trsm_kernel(const float* L, int ldl, const __nv_bfloat16* Yt, int r,
                                                            int d, float* Qf, __nv_bfloat16* Qt) {
  __shared__ float tile[TB][TB + 1];   // tile[t][l]: L[i0 + t, l0 + l]
  pdl_wait();
  const int c = blockIdx.x * TRSM_THREADS + threadIdx.x;
  const bool live = c < d;
  for (int i0 = 0; i0 < r; i0 += TB) {
    const int rows = r - i0 < TB ? r - i0 : TB;
    float acc[TB];
#pragma unroll
    for (int t = 0; t < TB; ++t)
      acc[t] = (live && t < rows) ? __bfloat162float(Yt[static_cast<size_t>(i0 + t) * d + c]) : 0.f;
    for (int l0 = 0; l0 <= i0; l0 += TB) {
      __syncthreads();
      for (int e = threadIdx.x; e < TB * TB; e += TRSM_THREADS) {
        const int t = e / TB, l = e - t * TB;
        const int i = i0 + t, ll = l0 + l;
        tile[t][l] = (i < r && ll <= i && ll < r) ? L[static_cast<size_t>(i) * ldl + ll] : 0.f;
      }
      __syncthreads();
      if (l0 < i0) {
        // earlier block: all of its solution values are final
        for (int l = 0; l < TB; ++l) {
          const float q = live ? Qf[static_cast<size_t>(l0 + l) * d + c] : 0.f;
#pragma unroll
          for (int t = 0; t < TB; ++t) acc[t] = fmaf(-tile[t][l], q, acc[t]);
        }
      } else {
        // the block's own triangle
#pragma unroll
        for (int t = 0; t < TB; ++t) {
          if (t < rows) {
            const float q = acc[t] / tile[t][t];
            acc[t] = q;
#pragma unroll
            for (int u = t + 1; u < TB; ++u) acc[u] = fmaf(-tile[u][t], q, acc[u]);
          }
        }
      }
    }
    if (live) {
#pragma unroll
      for (int t = 0; t < TB; ++t) {
        if (t < rows) {
          Qf[static_cast<size_t>(i0 + t) * d + c] = acc[t];
          Qt[static_cast<size_t>(i0 + t) * d + c] = __float2bfloat16_rn(acc[t]);
        }
      }
    }
  }
}

}  // namespace fac

namespace {

constexpr size_t kAlignF = 256;
inline size_t align_f(size_t v) { return (v + kAlignF - 1) / kAlignF * kAlignF; }

struct FactorLayout { size_t wd, wn, zt, yt, qt, qf, g, end; int np, rp; };
FactorLayout factor_layout(int d, int ml, int r) {
  FactorLayout L;
  L.np = round_up(ml, 16);
  L.rp = round_up(r, 16);
  size_t off = 0;
  L.wd = off; off = align_f(off + static_cast<size_t>(L.np) * d * 2);       // W^T [np, d]
  L.wn = off; off = align_f(off + static_cast<size_t>(d) * L.np * 2);       // W   [d, np]
  L.zt = off; off = align_f(off + static_cast<size_t>(L.rp) * L.np * 2);    // Z^T [r, np]
  L.yt = off; off = align_f(off + static_cast<size_t>(L.rp) * d * 2);       // Y^T [r, d]
  L.qt = off; off = align_f(off + static_cast<size_t>(L.rp) * d * 2);       // Q^T [r, d]
  L.qf = off; off = align_f(off + static_cast<size_t>(L.rp) * d * 4);       // Q^T in fp32 (the solve's running solution)
  L.g = off;  off = align_f(off + static_cast<size_t>(L.rp) * L.rp * 4);    // Gram matrix / Cholesky factor
  L.end = off;
  return L;
}

ffsplit_status check_factor_args(ffsplit_ctx* ctx, const ffsplit_shape* s, int k, int r) {
  if (!s) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "shape is NULL");
  if (s->d < 1 || s->m < 1) return fail(ctx, FFSPLIT_ERR_SHAPE, "d and m must be >= 1");
  if (s->act < 0 || s->act > 2) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "unknown activation");
  if (s->dtype != FFSPLIT_BF16) return fail(ctx, FFSPLIT_ERR_DTYPE, "the on-device factorisation takes bf16 layers");
  if (s->d % 8 != 0) return fail(ctx, FFSPLIT_ERR_SHAPE, "bf16 layers need d to be a multiple of 8");
  if (k < 0 || k >= s->m) return fail(ctx, FFSPLIT_ERR_SHAPE, "k must be in [0, m): there must be light neurons to factor");
  const int ml = s->m - k;
  const int rmax = s->d < ml ? s->d : ml;
  if (r < 1 || r > rmax) return fail(ctx, FFSPLIT_ERR_SHAPE, "r must be in [1, min(d, m - k)]");
  if (r > 2048) return fail(ctx, FFSPLIT_ERR_SHAPE, "the on-device factorisation takes r <= 2048");
  return FFSPLIT_OK;
}

// One GEMM of the iteration: C [M, N] = A [M, K] . (B [N, K])^T, bf16 in; bf16 or fp32 out.
ffsplit_status thin_gemm(ffsplit_ctx* ctx, const void* A, long long lda, const void* B, long long ldb, long long M,
                         int N, int K, void* C, long long ldc, bool f32, cudaStream_t st) {
  GemmArgs g;
  std::memset(&g, 0, sizeof(g));
  g.A0 = A; g.lda0 = lda; g.B0 = B; g.ldb0 = ldb;
  g.M = M; g.N = N; g.K = K;
  g.algo_flops = 2.0 * M * N * K;
  g.epi.C0 = C; g.epi.ld0 = ldc; g.epi.n_split = N;
  g.epi.act = FFSPLIT_GELU_ERF;   // no column is activated (n_act = 0)
  g.epi.c0_f32 = f32 ? 1 : 0;
  return launch_gemm(ctx, FFSPLIT_BF16, g, st);
}

// Q^T <- orth(Q^T W W^T), `iters` times, W given in both K-major forms; Q^T [r, d] starts as `start`.
// Leaves Q^T (bf16) at L.qt and, if want_zt, Z^T = Q^T W [r, np] at L.zt.
ffsplit_status iterate(ffsplit_ctx* ctx, const FactorLayout& L, char* base, int d, int r, int iters, const void* start,
                       cudaStream_t st) {
  char* Wd = base + L.wd;
  char* Wn = base + L.wn;
  char* Zt = base + L.zt;
  char* Yt = base + L.yt;
  char* Qt = base + L.qt;
  float* Qf = reinterpret_cast<float*>(base + L.qf);
  float* G = reinterpret_cast<float*>(base + L.g);
  ffsplit_status s;
  const void* cur = start;
  for (int it = 0; it < iters; ++it) {
    if ((s = thin_gemm(ctx, cur, d, Wd, d, r, L.np, d, Zt, L.np, false, st)) != FFSPLIT_OK) return s;
    if ((s = thin_gemm(ctx, Zt, L.np, Wn, L.np, r, d, L.np, Yt, d, false, st)) != FFSPLIT_OK) return s;
    if ((s = thin_gemm(ctx, Yt, d, Yt, d, r, r, d, G, L.rp, true, st)) != FFSPLIT_OK) return s;
    cudaError_t e = cudaSuccess;
    for (int j0 = 0; j0 < r && e == cudaSuccess; j0 += fac::NB) {
      e = launch_pdl(fac::chol_panel_kernel, dim3(1), dim3(fac::CHOL_THREADS), 0, st, G, r, L.rp, j0, ctx->status());
      ctx->launches++;
      const int tb = (r - j0 - fac::NB + fac::NB - 1) / fac::NB;   // tile rows of the trailing matrix
      if (e == cudaSuccess && tb > 0) {
        e = launch_pdl(fac::chol_update_kernel, dim3(tb * (tb + 1) / 2), dim3(fac::CHOL_THREADS), 0, st, G, r, L.rp, j0);
        ctx->launches++;
      }
    }
    if (e != cudaSuccess) return check_cuda(ctx, e, "Cholesky kernel launch");
    e = launch_pdl(fac::trsm_kernel, dim3((d + fac::TRSM_THREADS - 1) / fac::TRSM_THREADS), dim3(fac::TRSM_THREADS), 0,
                   st, static_cast<const float*>(G), L.rp, reinterpret_cast<const __nv_bfloat16*>(Yt), r, d, Qf,
                   reinterpret_cast<__nv_bfloat16*>(Qt));
    ctx->launches++;
    if (e != cudaSuccess) return check_cuda(ctx, e, "trsm_kernel launch");
    cur = Qt;
  }
  if (iters == 0) {
    const cudaError_t e = cudaMemcpyAsync(Qt, start, static_cast<size_t>(r) * d * 2, cudaMemcpyDeviceToDevice, st);
    if (e != cudaSuccess) return check_cuda(ctx, e, "cudaMemcpyAsync(start basis)");
  }
  return FFSPLIT_OK;
}

}  // namespace
}  // namespace ffsp

extern "C" {

ffsplit_status ffsplit_factor_workspace_size(const ffsplit_shape* shape, int32_t k, int32_t r, size_t* bytes) {
  using namespace ffsp;
  if (!bytes) return FFSPLIT_ERR_INVALID_ARG;
  ffsplit_status s = check_factor_args(nullptr, shape, k, r);
  if (s != FFSPLIT_OK) return s;
  *bytes = kCtrlBytes + factor_layout(shape->d, shape->m - k, r).end;
  return FFSPLIT_OK;
}

ffsplit_status ffsplit_factor_light(ffsplit_ctx* ctx, const ffsplit_shape* shape, const ffsplit_weights* weights,
                                    const int32_t* light_idx, int32_t k, int32_t r, int32_t iters, const void* start,
                                    void* A1, void* B1, void* A2, void* B2, void* A1u, void* B1u, void* stream) {
  using namespace ffsp;
  if (!ctx) return FFSPLIT_ERR_INVALID_ARG;
  ffsplit_status s = check_factor_args(ctx, shape, k, r);
  if (s != FFSPLIT_OK) return s;
  const bool gated = shape->act == FFSPLIT_SWIGLU;
  if (!weights || !weights->W1 || !weights->W2 || !light_idx || !start || !A1 || !B1 || !A2 || !B2)
    return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "NULL tensor");
  if (gated && (!weights->W1u || !A1u || !B1u)) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "SwiGLU needs W1u, A1u and B1u");
  if (iters < 0 || iters > 64) return fail(ctx, FFSPLIT_ERR_INVALID_ARG, "iters must be in [0, 64]");
  if (!aligned16(weights->W1) || !aligned16(weights->W2) || !aligned16(start) || (gated && !aligned16(weights->W1u)))
    return fail(ctx, FFSPLIT_ERR_ALIGN, "weights and the starting bases must be 16-byte aligned");
  const int d = shape->d, m = shape->m, ml = m - k, dt = FFSPLIT_BF16;
  const FactorLayout L = factor_layout(d, ml, r);
  if (!ctx->ws || kCtrlBytes + L.end > ctx->ws_bytes)
    return fail(ctx, FFSPLIT_ERR_BUFFER_TOO_SMALL, "workspace too small for this factorisation (ffsplit_factor_workspace_size)");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  char* base = ctx->ws + kCtrlBytes;
  ctx->score_prep.valid = false;   // the scoring buffers share the workspace
  char* Wd = base + L.wd;
  char* Wn = base + L.wn;
  char* Zt = base + L.zt;
  char* Qt = base + L.qt;
  const size_t start_stride = static_cast<size_t>(r) * d * 2;

  // ---- U-type matrices: W = W1[:, light] (and the SwiGLU up projection): A = Q, B = Q^T W
  for (int which = 0; which < (gated ? 2 : 1); ++which) {
    const void* W = which == 0 ? weights->W1 : weights->W1u;
    void* A = which == 0 ? A1 : A1u;
    void* B = which == 0 ? B1 : B1u;
    const char* st0 = static_cast<const char*>(start) + (which == 0 ? 0 : 2) * start_stride;
    // W^T [np, d] = gathered, transposed columns; W [d, np] = its transpose (pad rows / columns zero)
    if ((s = launch_gather_cols_t(ctx, dt, W, m, d, light_idx, ml, m, Wd, d, L.np, st)) != FFSPLIT_OK) return s;
    if ((s = launch_transpose(ctx, dt, Wd, d, L.np, d, Wn, L.np, L.np, d, nullptr, L.np, st)) != FFSPLIT_OK) return s;
    if ((s = iterate(ctx, L, base, d, r, iters, st0, st)) != FFSPLIT_OK) return s;
    if ((s = thin_gemm(ctx, Qt, d, Wd, d, r, ml, d, B, ml, false, st)) != FFSPLIT_OK) return s;               // B [r, ml]
    if ((s = launch_transpose(ctx, dt, Qt, d, r, d, A, r, r, d, nullptr, r, st)) != FFSPLIT_OK) return s;     // A [d, r]
  }
  // ---- V-type: W = V2^T with V2 = W2[light, :]: A2 = V2 Q = (Q^T V2^T)^T, B2 = Q^T
  {
    const char* st0 = static_cast<const char*>(start) + start_stride;
    if ((s = launch_transpose(ctx, dt, weights->W2, d, ml, d, Wn, L.np, L.np, d, light_idx, m, st)) != FFSPLIT_OK) return s;  // V2^T [d, np]
    if ((s = launch_transpose(ctx, dt, Wn, L.np, d, L.np, Wd, d, d, L.np, nullptr, d, st)) != FFSPLIT_OK) return s;          // V2 [np, d]
    if ((s = iterate(ctx, L, base, d, r, iters, st0, st)) != FFSPLIT_OK) return s;
    if ((s = thin_gemm(ctx, Qt, d, Wd, d, r, L.np, d, Zt, L.np, false, st)) != FFSPLIT_OK) return s;          // Z^T [r, np]
    if ((s = launch_transpose(ctx, dt, Zt, L.np, r, ml, A2, r, r, ml, nullptr, r, st)) != FFSPLIT_OK) return s;   // A2 [ml, r]
    const cudaError_t e = cudaMemcpyAsync(B2, Qt, static_cast<size_t>(r) * d * 2, cudaMemcpyDeviceToDevice, st);
    if (e != cudaSuccess) return check_cuda(ctx, e, "cudaMemcpyAsync(B2)");
  }
  return FFSPLIT_OK;
}

}  // extern "C"
