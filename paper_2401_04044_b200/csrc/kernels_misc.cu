// Selection (radix top-k), row / column energy reductions and the gather /
// transpose kernels of the pack step.
#include "epilogue.cuh"
#include "internal.h"

namespace ffsp {

// ============================================================================
// Top-k selection (Section 4.1: the neurons with the highest score are the heavy
// hitters).  One CTA: 4 radix passes of 8 bits over an order-preserving integer
// image of the float keys find the k-th largest key; an ordered compaction then
// emits heavy and light indices in ascending order.  Keys equal to the threshold
// are taken lowest index first.
// ============================================================================
constexpr int kSelThreads = 1024;

__device__ __forceinline__ unsigned order_key(float f) {
  unsigned b = __float_as_uint(f);
  if (b == 0x80000000u) b = 0u;  // -0.0 ranks as +0.0
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

__global__ void __launch_bounds__(kSelThreads) select_kernel(const float* __restrict__ scores, int m, int k,
                                                             int* __restrict__ heavy, int* __restrict__ light,
                                                             int* status) {
  __shared__ unsigned hist[256];
  __shared__ unsigned s_prefix, s_mask, s_remaining;
  __shared__ unsigned wsum_gt[32], wsum_eq[32];
  const int tid = threadIdx.x;
  const int lane = tid & 31, warp = tid >> 5;

  if (tid == 0) {
    s_prefix = 0u;
    s_mask = 0u;
    s_remaining = static_cast<unsigned>(k);
  }
  bool bad = false;
  for (int i = tid; i < m; i += kSelThreads) {
    const unsigned b = __float_as_uint(scores[i]);
    if ((b & 0x7f800000u) == 0x7f800000u) bad = true;
  }
  if (bad) record_status(status, FFSPLIT_ERR_NONFINITE, 0, KID_SELECT);
  __syncthreads();

  unsigned threshold = 0xFFFFFFFFu, take_eq = 0u;
  if (k > 0) {
    for (int shift = 24; shift >= 0; shift -= 8) {
      for (int b = tid; b < 256; b += kSelThreads) hist[b] = 0u;
      __syncthreads();
      const unsigned prefix = s_prefix, mask = s_mask;
      for (int i = tid; i < m; i += kSelThreads) {
        const unsigned kv = order_key(scores[i]);
        if ((kv & mask) == prefix) atomicAdd(&hist[(kv >> shift) & 255u], 1u);
      }
      __syncthreads();
      if (tid == 0) {
        unsigned cum = 0u, remaining = s_remaining;
        for (int b = 255; b >= 0; --b) {
          const unsigned c = hist[b];
          if (cum + c >= remaining) {
            s_prefix = prefix | (static_cast<unsigned>(b) << shift);
            s_remaining = remaining - cum;
            break;
          }
          cum += c;
        }
        s_mask = mask | (255u << shift);
      }
      __syncthreads();
    }
    threshold = s_prefix;
    take_eq = s_remaining;
  }

  // ordered compaction: thread t owns a contiguous run of indices
  const int chunk = (m + kSelThreads - 1) / kSelThreads;
  const int lo = min(m, tid * chunk), hi = min(m, lo + chunk);
  unsigned n_gt = 0u, n_eq = 0u;
  for (int i = lo; i < hi; ++i) {
    const unsigned kv = order_key(scores[i]);
    n_gt += kv > threshold;
    n_eq += kv == threshold;
  }
  unsigned inc_gt = n_gt, inc_eq = n_eq;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const unsigned a = __shfl_up_sync(0xffffffffu, inc_gt, o);
    const unsigned b = __shfl_up_sync(0xffffffffu, inc_eq, o);
    if (lane >= o) { inc_gt += a; inc_eq += b; }
  }
  if (lane == 31) { wsum_gt[warp] = inc_gt; wsum_eq[warp] = inc_eq; }
  __syncthreads();
  if (warp == 0) {
    const unsigned a = wsum_gt[lane], b = wsum_eq[lane];
    unsigned ia = a, ib = b;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const unsigned x = __shfl_up_sync(0xffffffffu, ia, o);
      const unsigned y = __shfl_up_sync(0xffffffffu, ib, o);
      if (lane >= o) { ia += x; ib += y; }
    }
    wsum_gt[lane] = ia - a;  // exclusive
    wsum_eq[lane] = ib - b;
  }
  __syncthreads();
  const unsigned gt_before = wsum_gt[warp] + inc_gt - n_gt;
  unsigned eq_before = wsum_eq[warp] + inc_eq - n_eq;
  unsigned h_pos = gt_before + min(eq_before, take_eq);
  for (int i = lo; i < hi; ++i) {
    const unsigned kv = order_key(scores[i]);
    bool is_heavy = kv > threshold;
    if (kv == threshold) {
      is_heavy = eq_before < take_eq;
      ++eq_before;
    }
    if (is_heavy) {
      if (heavy && h_pos < static_cast<unsigned>(k)) heavy[h_pos] = i;
      ++h_pos;
    } else if (light) {
      light[i - static_cast<int>(h_pos)] = i;
    }
  }
}

ffsplit_status launch_select(ffsplit_ctx* ctx, const float* scores, int m, int k, int* heavy, int* light,
                             cudaStream_t st) {
  select_kernel<<<1, kSelThreads, 0, st>>>(scores, m, k, heavy, light, ctx->status());
  ctx->launches++;
  return check_cuda(ctx, cudaGetLastError(), "select_kernel launch");
}

// ============================================================================
// w_j = sum_c W2[j, c]^2   (Eq. 3, ||V_{j,:}||^2): one warp per row, 128-bit loads,
// lane-strided partial sums combined by a fixed shuffle tree.
// ============================================================================
template <typename T>
__global__ void __launch_bounds__(256) row_energy_kernel(const T* __restrict__ W, int m, int d, float* __restrict__ w) {
  const int row = blockIdx.x * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= m) return;
  const T* p = W + static_cast<long long>(row) * d;
  constexpr int VEC = 16 / sizeof(T);
  float s = 0.f;
  if (d % VEC == 0 && (reinterpret_cast<uintptr_t>(p) & 15u) == 0) {
    for (int c = lane * VEC; c < d; c += 32 * VEC) {
      const uint4 raw = __ldg(reinterpret_cast<const uint4*>(p + c));
      const T* e = reinterpret_cast<const T*>(&raw);
#pragma unroll
      for (int i = 0; i < VEC; ++i) {
        const float x = to_float<T>(e[i]);
        s = fmaf(x, x, s);
      }
    }
  } else {
    for (int c = lane; c < d; c += 32) {
      const float x = to_float<T>(p[c]);
      s = fmaf(x, x, s);
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  if (lane == 0) w[row] = s;
}

ffsplit_status launch_row_energy(ffsplit_ctx* ctx, int dtype, const void* W2, int m, int d, float* w, cudaStream_t st) {
  const int grid = (m + 7) / 8;
  if (dtype == FFSPLIT_BF16)
    row_energy_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(W2), m, d, w);
  else
    row_energy_kernel<float><<<grid, 256, 0, st>>>(static_cast<const float*>(W2), m, d, w);
  ctx->launches++;
  return check_cuda(ctx, cudaGetLastError(), "row_energy_kernel launch");
}

// ============================================================================
// e_j (+)= sum over row groups of the per-group column partials, in a fixed
// order; then the score of the chosen reading.
// ============================================================================
__global__ void score_finalize_kernel(const float* __restrict__ partial, int groups, int m,
                                      const float* __restrict__ w, float* __restrict__ energy,
                                      float* __restrict__ scores, int mode, int accumulate) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j >= m) return;
  float s = 0.f;
  for (int g = 0; g < groups; ++g) s += partial[static_cast<long long>(g) * m + j];
  const float e = accumulate ? energy[j] + s : s;
  energy[j] = e;
  if (scores) {
    float v = e;
    if (mode == FFSPLIT_SCORE_EQ3) v = e * w[j];
    else if (mode == FFSPLIT_SCORE_SUM_NORM) v = e * sqrtf(w[j]);
    scores[j] = v;
  }
}

ffsplit_status launch_score_finalize(ffsplit_ctx* ctx, const float* partial, int groups, int m, const float* w,
                                     float* energy, float* scores, int mode, int accumulate, cudaStream_t st) {
  score_finalize_kernel<<<(m + 255) / 256, 256, 0, st>>>(partial, groups, m, w, energy, scores, mode, accumulate);
  ctx->launches++;
  return check_cuda(ctx, cudaGetLastError(), "score_finalize_kernel launch");
}

// ============================================================================
// Pack helpers (Figure 3 caption: U1 = U[:, h2], V1 = V[h2, :]).
// ============================================================================
// OUT[c, j] = IN[src(j), c] for j < rows, c < cols; zero elsewhere in the padded
// output [cols_pad, rows_pad].  src(j) = row_idx ? row_idx[j] : j; a source row
// outside [0, idx_limit) reads as zeros.
template <typename T>
__global__ void __launch_bounds__(256) transpose_kernel(const T* __restrict__ in, long long ldi, int rows, int cols,
                                                        T* __restrict__ out, long long ldo, int rows_pad,
                                                        int cols_pad, const int* __restrict__ row_idx, int idx_limit) {
  __shared__ T tile[32][33];
  const int j0 = blockIdx.x * 32, c0 = blockIdx.y * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;  // 32 x 8
  for (int jj = ty; jj < 32; jj += 8) {
    const int j = j0 + jj, c = c0 + tx;
    T v = from_float<T>(0.f);
    if (j < rows && c < cols) {
      const int src = row_idx ? row_idx[j] : j;
      if (src >= 0 && src < idx_limit) v = in[static_cast<long long>(src) * ldi + c];
    }
    tile[jj][tx] = v;
  }
  __syncthreads();
  for (int cc = ty; cc < 32; cc += 8) {
    const int c = c0 + cc, j = j0 + tx;
    if (c < cols_pad && j < rows_pad) out[static_cast<long long>(c) * ldo + j] = tile[tx][cc];
  }
}

ffsplit_status launch_transpose(ffsplit_ctx* ctx, int dtype, const void* in, long long ldi, int rows, int cols,
                                void* out, long long ldo, int rows_pad_out, int cols_pad_out, const int* row_idx,
                                int idx_limit, cudaStream_t st) {
  if (rows_pad_out <= 0 || cols_pad_out <= 0) return FFSPLIT_OK;
  dim3 grid((rows_pad_out + 31) / 32, (cols_pad_out + 31) / 32);
  if (grid.y > 65535) return fail(ctx, FFSPLIT_ERR_SHAPE, "matrix too wide for the transpose kernel");
  if (dtype == FFSPLIT_BF16)
    transpose_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(in), ldi, rows, cols,
                                                          static_cast<__nv_bfloat16*>(out), ldo, rows_pad_out,
                                                          cols_pad_out, row_idx, idx_limit);
  else
    transpose_kernel<float><<<grid, 256, 0, st>>>(static_cast<const float*>(in), ldi, rows, cols,
                                                  static_cast<float*>(out), ldo, rows_pad_out, cols_pad_out, row_idx,
                                                  idx_limit);
  ctx->launches++;
  return check_cuda(ctx, cudaGetLastError(), "transpose_kernel launch");
}

// OUT[j, i] = IN[i, col_idx[j]] for j < ncols, i < rows; zero rows for ncols <= j < rows_out_pad.
template <typename T>
__global__ void __launch_bounds__(256) gather_cols_kernel(const T* __restrict__ in, long long ldi, int rows,
                                                          const int* __restrict__ col_idx, int ncols, int idx_limit,
                                                          T* __restrict__ out, long long ldo, int rows_out_pad) {
  __shared__ T tile[32][33];
  const int j0 = blockIdx.x * 32, i0 = blockIdx.y * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const int j = j0 + tx;
  int src = -1;
  if (j < ncols) {
    src = col_idx[j];
    if (src < 0 || src >= idx_limit) src = -1;
  }
  for (int ii = ty; ii < 32; ii += 8) {
    const int i = i0 + ii;
    T v = from_float<T>(0.f);
    if (src >= 0 && i < rows) v = in[static_cast<long long>(i) * ldi + src];
    tile[ii][tx] = v;
  }
  __syncthreads();
  for (int jj = ty; jj < 32; jj += 8) {
    const int jo = j0 + jj, i = i0 + tx;
    if (jo < rows_out_pad && i < rows) out[static_cast<long long>(jo) * ldo + i] = tile[tx][jj];
  }
}

ffsplit_status launch_gather_cols_t(ffsplit_ctx* ctx, int dtype, const void* in, long long ldi, int rows,
                                    const int* col_idx, int ncols, int idx_limit, void* out, long long ldo,
                                    int rows_out_pad, cudaStream_t st) {
  if (rows_out_pad <= 0 || rows <= 0) return FFSPLIT_OK;
  dim3 grid((rows_out_pad + 31) / 32, (rows + 31) / 32);
  if (grid.y > 65535) return fail(ctx, FFSPLIT_ERR_SHAPE, "matrix too tall for the gather kernel");
  if (dtype == FFSPLIT_BF16)
    gather_cols_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(in), ldi, rows, col_idx,
                                                            ncols, idx_limit, static_cast<__nv_bfloat16*>(out), ldo,
                                                            rows_out_pad);
  else
    gather_cols_kernel<float><<<grid, 256, 0, st>>>(static_cast<const float*>(in), ldi, rows, col_idx, ncols,
                                                    idx_limit, static_cast<float*>(out), ldo, rows_out_pad);
  ctx->launches++;
  return check_cuda(ctx, cudaGetLastError(), "gather_cols_kernel launch");
}

// Biases in fp32: b1[h2] (zero padded), b1[light] (zero padded), b2; also checks
// that heavy_idx is strictly ascending and in range.
template <typename T>
__global__ void pack_bias_kernel(const T* __restrict__ b1, const T* __restrict__ b2, const int* __restrict__ heavy,
                                 int m, int k, int d, float* __restrict__ b1h, int k_pad, float* __restrict__ b1l,
                                 int ml_pad, float* __restrict__ b2o, int* status) {
  const int j = blockIdx.x * blockDim.x + threadIdx.x;
  if (j < k) {
    const int h = heavy[j];
    if (h < 0 || h >= m || (j > 0 && heavy[j - 1] >= h)) record_status(status, FFSPLIT_ERR_BAD_INDEX, j, KID_PACK);
  }
  if (j < m) {
    int lo = 0, hi = k;  // first position with heavy[pos] >= j
    while (lo < hi) {
      const int mid = (lo + hi) >> 1;
      if (heavy[mid] < j) lo = mid + 1; else hi = mid;
    }
    const float v = b1 ? to_float<T>(b1[j]) : 0.f;
    if (lo < k && heavy[lo] == j) b1h[lo] = v;
    else if (j - lo >= 0 && j - lo < ml_pad) b1l[j - lo] = v;
  }
  if (j >= k && j < k_pad) b1h[j] = 0.f;
  const int ml = m - k;
  if (j >= ml && j < ml_pad) b1l[j] = 0.f;
  if (j < d) b2o[j] = b2 ? to_float<T>(b2[j]) : 0.f;
}

ffsplit_status launch_pack_bias(ffsplit_ctx* ctx, int dtype, const void* b1, const void* b2, const int* heavy, int m,
                                int k, int d, float* b1h, int k_pad, float* b1l, int ml_pad, float* b2o,
                                cudaStream_t st) {
  int n = m;
  if (k_pad > n) n = k_pad;
  if (ml_pad > n) n = ml_pad;
  if (d > n) n = d;
  const int grid = (n + 255) / 256;
  if (dtype == FFSPLIT_BF16)
    pack_bias_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(b1),
                                                          static_cast<const __nv_bfloat16*>(b2), heavy, m, k, d, b1h,
                                                          k_pad, b1l, ml_pad, b2o, ctx->status());
  else
    pack_bias_kernel<float><<<grid, 256, 0, st>>>(static_cast<const float*>(b1), static_cast<const float*>(b2), heavy,
                                                  m, k, d, b1h, k_pad, b1l, ml_pad, b2o, ctx->status());
  ctx->launches++;
  return check_cuda(ctx, cudaGetLastError(), "pack_bias_kernel launch");
}

// out[i] = float(in[i]); a NULL input gives zeros.
template <typename T>
__global__ void to_f32_kernel(const T* __restrict__ in, int n, float* __restrict__ out) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) out[i] = in ? to_float<T>(in[i]) : 0.f;
}

ffsplit_status launch_to_f32(ffsplit_ctx* ctx, int dtype, const void* in, int n, float* out, cudaStream_t st) {
  if (n <= 0) return FFSPLIT_OK;
  if (dtype == FFSPLIT_BF16)
    to_f32_kernel<__nv_bfloat16><<<(n + 255) / 256, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(in), n, out);
  else
    to_f32_kernel<float><<<(n + 255) / 256, 256, 0, st>>>(static_cast<const float*>(in), n, out);
  ctx->launches++;
  return check_cuda(ctx, cudaGetLastError(), "to_f32_kernel launch");
}

}  // namespace ffsp
