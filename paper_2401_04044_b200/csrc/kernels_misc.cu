// Selection (radix top-k), row / column energy reductions and the gather /
// transpose kernels of the pack step.
#include "epilogue.cuh"
#include "internal.h"
#include "ptx.cuh"

namespace ffsp {

// ============================================================================
// Self-test of the bounded wait every kernel of the library is built on: one CTA of two warps.  Warp 0
// waits, through the same routine the tensor-core and few-token kernels use, on an mbarrier that nothing
// will ever signal, with a limit of `limit_cycles`; the wait runs out, raises the CTA's abort flag and
// returns; warp 1, waiting on a second unsignalled barrier, sees the flag and leaves too (the way the
// other roles of a kernel leave when one of them gives up).  The kernel then records FFSPLIT_ERR_TIMEOUT
// in the status block and exits normally: no trap, no fault, and the context stays usable.
// ============================================================================
__global__ void __launch_bounds__(64) wait_timeout_probe_kernel(long long limit_cycles, int* status) {
  __shared__ __align__(8) uint64_t bars[2];
  __shared__ int abort_flag;
  __shared__ int gave_up[2];
  if (threadIdx.x == 0) {
    ptx::mbar_init(&bars[0], 1);
    ptx::mbar_init(&bars[1], 1);
    ptx::mbar_fence_init();
    abort_flag = 0;
    gave_up[0] = gave_up[1] = 0;
  }
  __syncthreads();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (lane == 0) {
    // warp 0: the short limit; warp 1: the library's normal limit (about a second), cut short by the flag
    const bool ok = warp == 0 ? ptx::mbar_wait_limit(&bars[0], 0, &abort_flag, limit_cycles)
                              : ptx::mbar_wait(&bars[1], 0, &abort_flag);
    gave_up[warp] = ok ? 0 : 1;
  }
  __syncthreads();
  if (threadIdx.x == 0 && abort_flag)
    record_status(status, FFSPLIT_ERR_TIMEOUT, gave_up[0] + 2 * gave_up[1], KID_PROBE);
}

ffsplit_status launch_wait_timeout_probe(ffsplit_ctx* ctx, long long limit_cycles, cudaStream_t st) {
  wait_timeout_probe_kernel<<<1, 64, 0, st>>>(limit_cycles, ctx->status());
  ctx->launches++;
  return check_cuda(ctx, cudaGetLastError(), "wait_timeout_probe_kernel launch");
}

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
  pdl_wait();

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
      if (warp == 0) {
        // lane l owns bins 8l .. 8l+7; counts of all higher bins by a shuffle suffix scan
        unsigned mine = 0u;
#pragma unroll
        for (int b = 0; b < 8; ++b) mine += hist[8 * lane + b];
        unsigned incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const unsigned up = __shfl_down_sync(0xffffffffu, incl, o);
          if (lane + o < 32) incl += up;
        }
        const unsigned above = incl - mine, remaining = s_remaining;
        __syncwarp();
        if (above < remaining && remaining <= above + mine) {   // exactly one lane
          unsigned cum = above;
          for (int b = 8 * lane + 7; b >= 8 * lane; --b) {
            const unsigned c = hist[b];
            if (cum + c >= remaining) {
              s_prefix = prefix | (static_cast<unsigned>(b) << shift);
              s_remaining = remaining - cum;
              break;
            }
            cum += c;
          }
        }
        if (lane == 0) s_mask = mask | (255u << shift);
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
  const cudaError_t le = launch_pdl(select_kernel, dim3(1), dim3(kSelThreads), 0, st, scores, m, k, heavy, light, ctx->status());
  ctx->launches++;
  return check_cuda(ctx, le, "select_kernel launch");
}

// ============================================================================
// e_j (+)= sum over row groups of the per-group column partials, in a fixed
// order (8 interleaved slices of the groups, then the 8 slice sums in order);
// then the score of the chosen reading.
// ============================================================================
__global__ void __launch_bounds__(256) score_finalize_kernel(const float* __restrict__ partial, int groups, int m,
                                                             const float* __restrict__ w, float* __restrict__ energy,
                                                             float* __restrict__ scores, int mode, int accumulate) {
  __shared__ float part[8][32];
  pdl_wait();
  const int cx = threadIdx.x & 31, gy = threadIdx.x >> 5;
  const int j = blockIdx.x * 32 + cx;
  float s = 0.f;
  if (j < m)
    for (int g = gy; g < groups; g += 8) s += partial[static_cast<long long>(g) * m + j];
  part[gy][cx] = s;
  __syncthreads();
  if (gy != 0 || j >= m) return;
  float tot = 0.f;
#pragma unroll
  for (int i = 0; i < 8; ++i) tot += part[i][cx];
  const float e = accumulate ? energy[j] + tot : tot;
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
  const cudaError_t le = launch_pdl(score_finalize_kernel, dim3((m + 31) / 32), dim3(256), 0, st, partial, groups, m, w, energy, scores, mode, accumulate);
  ctx->launches++;
  return check_cuda(ctx, le, "score_finalize_kernel launch");
}

// ============================================================================
// Column energy of a stored activation matrix (Eq. 3, the factor ||sigma(X U_{:,j})||^2 when the
// activations H [T, m] already exist in memory): partial[g, j] = sum over the rows of group g of
// H[t, j]^2 (or |H[t, j]|).  Pure streaming: every warp-wide load takes 512 contiguous bytes of one
// row; a thread keeps its 16 bytes' worth of columns in registers over the group's rows, the eight
// warps of the CTA are added through shared memory in warp order.  score_finalize_kernel then adds
// the groups.
// ============================================================================
constexpr int kEnergyRows = 256;   // rows of H per group

template <typename T>
__global__ void __launch_bounds__(256) column_energy_kernel(const T* __restrict__ H, long long ldh, long long rows,
                                                            int m, float* __restrict__ partial, int use_abs) {
  constexpr int VEC = 16 / sizeof(T);
  __shared__ float red[8][32 * VEC];
  pdl_wait();
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const int c0 = blockIdx.x * (32 * VEC) + tx * VEC;
  const long long r0 = static_cast<long long>(blockIdx.y) * kEnergyRows;
  const long long r1 = r0 + kEnergyRows < rows ? r0 + kEnergyRows : rows;
  float acc[VEC];
#pragma unroll
  for (int i = 0; i < VEC; ++i) acc[i] = 0.f;
  const bool vec = c0 + VEC <= m && (ldh % VEC) == 0 && (reinterpret_cast<uintptr_t>(H) & 15u) == 0;
  if (vec) {
#pragma unroll 4
    for (long long r = r0 + ty; r < r1; r += 8) {
      const uint4 raw = __ldcs(reinterpret_cast<const uint4*>(H + r * ldh + c0));   // read once: streaming load
      const T* e = reinterpret_cast<const T*>(&raw);
#pragma unroll
      for (int i = 0; i < VEC; ++i) {
        const float x = to_float<T>(e[i]);
        acc[i] = use_abs ? acc[i] + fabsf(x) : fmaf(x, x, acc[i]);
      }
    }
  } else {
    for (long long r = r0 + ty; r < r1; r += 8)
      for (int i = 0; i < VEC; ++i)
        if (c0 + i < m) {
          const float x = to_float<T>(H[r * ldh + c0 + i]);
          acc[i] = use_abs ? acc[i] + fabsf(x) : fmaf(x, x, acc[i]);
        }
  }
#pragma unroll
  for (int i = 0; i < VEC; ++i) red[ty][tx * VEC + i] = acc[i];
  __syncthreads();
  for (int c = threadIdx.x; c < 32 * VEC; c += 256) {
    float s = 0.f;
#pragma unroll
    for (int w = 0; w < 8; ++w) s += red[w][c];   // fixed order
    const int col = blockIdx.x * (32 * VEC) + c;
    if (col < m) partial[static_cast<long long>(blockIdx.y) * m + col] = s;
  }
}

int column_energy_groups(long long rows) { return static_cast<int>((rows + kEnergyRows - 1) / kEnergyRows); }

ffsplit_status launch_column_energy(ffsplit_ctx* ctx, int dtype, const void* H, long long ldh, long long rows, int m,
                                    float* partial, int use_abs, cudaStream_t st) {
  const int groups = column_energy_groups(rows);
  if (groups > 65535) return fail(ctx, FFSPLIT_ERR_SHAPE, "more than 65535*256 activation rows in one call");
  const int ph = prof_open(ctx, PROF_ENERGY, static_cast<double>(rows) * m * elem_size(dtype), st);
  cudaError_t le;
  if (dtype == FFSPLIT_BF16) {
    le = launch_pdl(column_energy_kernel<__nv_bfloat16>, dim3((m + 255) / 256, groups), dim3(256), 0, st,
                    static_cast<const __nv_bfloat16*>(H), ldh, rows, m, partial, use_abs);
  } else {
    le = launch_pdl(column_energy_kernel<float>, dim3((m + 127) / 128, groups), dim3(256), 0, st,
                    static_cast<const float*>(H), ldh, rows, m, partial, use_abs);
  }
  prof_close(ctx, ph, st);
  ctx->launches++;
  return check_cuda(ctx, le, "column_energy_kernel launch");
}

// ============================================================================
// Small data-movement and reduction jobs of scoring and packing, batched: the
// jobs recorded between prep_begin() and prep_flush() run as ONE launch whose
// blocks are dealt out to the jobs (each job is far too small to fill the GPU,
// and a launch per job costs more than the job).
//   TRANSPOSE   OUT[c, j] = IN[src(j), c], zero padded   (factors, V1 = V[h2, :], U^T)
//   GATHER      OUT[j, i] = IN[i, idx[j]], zero padded   (U1^T = (U[:, h2])^T)
//   TO_F32      out[i] = float(in[i])
//   ROW_ENERGY  w_j = sum_c W2[j, c]^2                   (Eq. 3, ||V_{j,:}||^2)
//   PACK_BIAS   b1[h2], b1[light], b2 in fp32 + validation of h2
// ============================================================================
enum PrepKind : int { PREP_TRANSPOSE = 0, PREP_GATHER = 1, PREP_TO_F32 = 2, PREP_ROW_ENERGY = 3, PREP_PACK_BIAS = 4 };

template <typename T>
__device__ __forceinline__ void transpose_tile(const PrepJob& q, int bx, int by, T (*tile)[33]) {
  // OUT[c, j] = IN[src(j), c] for j < rows, c < cols; zero elsewhere in the padded output
  // [cols_pad, rows_pad].  src(j) = idx ? idx[j] : j; a source row outside [0, idx_limit) reads as zeros.
  const T* in = static_cast<const T*>(q.in);
  T* out = static_cast<T*>(q.out);
  const int j0 = bx * 32, c0 = by * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;  // 32 x 8
  for (int jj = ty; jj < 32; jj += 8) {
    const int j = j0 + jj, c = c0 + tx;
    T v = from_float<T>(0.f);
    if (j < q.rows && c < q.cols) {
      const int src = q.idx ? q.idx[j] : j;
      if (src >= 0 && src < q.idx_limit) v = in[static_cast<long long>(src) * q.ldi + c];
    }
    tile[jj][tx] = v;
  }
  __syncthreads();
  for (int cc = ty; cc < 32; cc += 8) {
    const int c = c0 + cc, j = j0 + tx;
    if (c < q.cols_pad && j < q.rows_pad) out[static_cast<long long>(c) * q.ldo + j] = tile[tx][cc];
  }
}

// The same for 2-byte elements with 64 x 64 tiles: pairs of elements move as 4-byte words, so a warp
// reads and writes 128 contiguous bytes per row instead of 64 (the 32 x 32 form above ran the
// 4.7 MB U^T transpose of a BERT-base layer at a third of the copy bandwidth).
template <typename T>
__device__ __forceinline__ void transpose_tile64(const PrepJob& q, int bx, int by, T (*tile)[66]) {
  static_assert(sizeof(T) == 2, "pairs of 2-byte elements");
  const T* in = static_cast<const T*>(q.in);
  T* out = static_cast<T*>(q.out);
  const int j0 = bx * 64, c0 = by * 64;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;  // 32 x 8
  const T zero = from_float<T>(0.f);
  const bool in_pairs = (q.ldi & 1) == 0 && (reinterpret_cast<uintptr_t>(in) & 3u) == 0;
  for (int jj = ty; jj < 64; jj += 8) {
    const int j = j0 + jj, c = c0 + 2 * tx;
    T v0 = zero, v1 = zero;
    if (j < q.rows && c < q.cols) {
      const int src = q.idx ? q.idx[j] : j;
      if (src >= 0 && src < q.idx_limit) {
        const T* p = in + static_cast<long long>(src) * q.ldi + c;
        if (in_pairs && c + 1 < q.cols) {
          const uint32_t w = *reinterpret_cast<const uint32_t*>(p);
          v0 = reinterpret_cast<const T*>(&w)[0];
          v1 = reinterpret_cast<const T*>(&w)[1];
        } else {
          v0 = p[0];
          if (c + 1 < q.cols) v1 = p[1];
        }
      }
    }
    tile[jj][2 * tx] = v0;
    tile[jj][2 * tx + 1] = v1;
  }
  __syncthreads();
  const bool out_pairs = (q.ldo & 1) == 0 && (reinterpret_cast<uintptr_t>(out) & 3u) == 0;
  for (int cc = ty; cc < 64; cc += 8) {
    const int c = c0 + cc, j = j0 + 2 * tx;
    if (c >= q.cols_pad || j >= q.rows_pad) continue;
    T* p = out + static_cast<long long>(c) * q.ldo + j;
    const T a = tile[2 * tx][cc], b = tile[2 * tx + 1][cc];
    if (out_pairs && j + 1 < q.rows_pad) {
      uint32_t w;
      reinterpret_cast<T*>(&w)[0] = a;
      reinterpret_cast<T*>(&w)[1] = b;
      *reinterpret_cast<uint32_t*>(p) = w;
    } else {
      p[0] = a;
      if (j + 1 < q.rows_pad) p[1] = b;
    }
  }
}

template <typename T>
__device__ __forceinline__ void gather_tile(const PrepJob& q, int bx, int by, T (*tile)[33]) {
  // OUT[j, i] = IN[i, idx[j]] for j < cols (count of gathered columns), i < rows; zero rows up to rows_pad
  const T* in = static_cast<const T*>(q.in);
  T* out = static_cast<T*>(q.out);
  const int j0 = bx * 32, i0 = by * 32;
  const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;
  const int j = j0 + tx;
  int src = -1;
  if (j < q.cols) {
    src = q.idx[j];
    if (src < 0 || src >= q.idx_limit) src = -1;
  }
  for (int ii = ty; ii < 32; ii += 8) {
    const int i = i0 + ii;
    T v = from_float<T>(0.f);
    if (src >= 0 && i < q.rows) v = in[static_cast<long long>(i) * q.ldi + src];
    tile[ii][tx] = v;
  }
  __syncthreads();
  for (int jj = ty; jj < 32; jj += 8) {
    const int jo = j0 + jj, i = i0 + tx;
    if (jo < q.rows_pad && i < q.rows) out[static_cast<long long>(jo) * q.ldo + i] = tile[tx][jj];
  }
}

template <typename T>
__device__ __forceinline__ void row_energy_rows(const PrepJob& q, int blk) {
  // one warp per row, 128-bit loads, lane-strided partial sums combined by a fixed shuffle tree
  const int row = blk * 8 + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= q.rows) return;
  const int d = q.cols;
  const T* p = static_cast<const T*>(q.in) + static_cast<long long>(row) * d;
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
  if (lane == 0) static_cast<float*>(q.out)[row] = s;
}

template <typename T>
__device__ __forceinline__ void pack_bias_chunk(const PrepJob& q, int blk, int* status) {
  // rows = m, cols = k, rows_pad = d, cols_pad = k_pad, idx_limit = ml_pad; in = b1, in2 = b2, idx = h2
  const T* b1 = static_cast<const T*>(q.in);
  const T* b2 = static_cast<const T*>(q.in2);
  const int* heavy = q.idx;
  float* b1h = static_cast<float*>(q.out);
  float* b1l = static_cast<float*>(q.out2);
  float* b2o = static_cast<float*>(q.out3);
  const int m = q.rows, k = q.cols, d = q.rows_pad, k_pad = q.cols_pad, ml_pad = q.idx_limit;
  const int j = blk * 256 + threadIdx.x;
  if (heavy == nullptr && k == m && k > 0) {
    // every neuron heavy, in order (k = m): b1[h2] is b1 itself and there is no light bias
    if (j < k) b1h[j] = b1 ? to_float<T>(b1[j]) : 0.f;
    if (j >= k && j < k_pad) b1h[j] = 0.f;
    if (j < ml_pad) b1l[j] = 0.f;
    if (j < d) b2o[j] = b2 ? to_float<T>(b2[j]) : 0.f;
    return;
  }
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

template <typename T>
__global__ void __launch_bounds__(256) prep_kernel(const PrepBatch batch, int* status) {
  // one buffer for both tile shapes: 32 x 33 elements, or 64 x 66 two-byte elements
  __shared__ __align__(4) unsigned char tile_raw[sizeof(T) == 2 ? 64 * 66 * 2 : 32 * 33 * sizeof(T)];
  T (*tile)[33] = reinterpret_cast<T (*)[33]>(tile_raw);
  pdl_wait();
  int i = 0;
  while (i + 1 < batch.n && static_cast<int>(blockIdx.x) >= batch.job[i + 1].block_begin) ++i;
  const PrepJob& q = batch.job[i];
  const int local = blockIdx.x - q.block_begin;
  switch (q.kind) {
    case PREP_TRANSPOSE:
      if constexpr (sizeof(T) == 2) transpose_tile64<T>(q, local % q.tiles_x, local / q.tiles_x, reinterpret_cast<T (*)[66]>(tile_raw));
      else transpose_tile<T>(q, local % q.tiles_x, local / q.tiles_x, tile);
      break;
    case PREP_GATHER: gather_tile<T>(q, local % q.tiles_x, local / q.tiles_x, tile); break;
    case PREP_TO_F32: {
      const int e = local * 256 + threadIdx.x;
      if (e < q.rows) static_cast<float*>(q.out)[e] = q.in ? to_float<T>(static_cast<const T*>(q.in)[e]) : 0.f;
      break;
    }
    case PREP_ROW_ENERGY: row_energy_rows<T>(q, local); break;
    default: pack_bias_chunk<T>(q, local, status); break;
  }
}

void prep_begin(ffsplit_ctx* ctx) {
  ctx->prep.n = 0;
  ctx->prep_blocks = 0;
  ctx->prep_active = true;
}

ffsplit_status prep_flush(ffsplit_ctx* ctx, int dtype, cudaStream_t st) {
  ctx->prep_active = false;
  if (ctx->prep.n == 0) return FFSPLIT_OK;
  const int blocks = ctx->prep_blocks;
  const cudaError_t le = dtype == FFSPLIT_BF16
                             ? launch_pdl(prep_kernel<__nv_bfloat16>, dim3(blocks), dim3(256), 0, st, ctx->prep, ctx->status())
                             : launch_pdl(prep_kernel<float>, dim3(blocks), dim3(256), 0, st, ctx->prep, ctx->status());
  ctx->prep.n = 0;
  ctx->launches++;
  return check_cuda(ctx, le, "prep_kernel launch");
}

// Records a job; outside a prep_begin/prep_flush bracket the job is launched on its own.
static ffsplit_status add_job(ffsplit_ctx* ctx, int dtype, PrepJob q, long long blocks, cudaStream_t st) {
  if (blocks <= 0) return FFSPLIT_OK;
  const bool single = !ctx->prep_active;
  if (single) prep_begin(ctx);
  if (ctx->prep.n >= kMaxPrepJobs || ctx->prep_blocks + blocks > 0x7fffffffLL)
    return fail(ctx, FFSPLIT_ERR_SHAPE, "too many or too large preparation jobs in one batch");
  q.block_begin = ctx->prep_blocks;
  ctx->prep.job[ctx->prep.n++] = q;
  ctx->prep_blocks += static_cast<int>(blocks);
  return single ? prep_flush(ctx, dtype, st) : FFSPLIT_OK;
}

ffsplit_status launch_row_energy(ffsplit_ctx* ctx, int dtype, const void* W2, int m, int d, float* w, cudaStream_t st) {
  PrepJob q{};
  q.kind = PREP_ROW_ENERGY; q.in = W2; q.rows = m; q.cols = d; q.out = w;
  return add_job(ctx, dtype, q, (m + 7) / 8, st);
}

ffsplit_status launch_transpose(ffsplit_ctx* ctx, int dtype, const void* in, long long ldi, int rows, int cols,
                                void* out, long long ldo, int rows_pad_out, int cols_pad_out, const int* row_idx,
                                int idx_limit, cudaStream_t st) {
  if (rows_pad_out <= 0 || cols_pad_out <= 0) return FFSPLIT_OK;
  PrepJob q{};
  q.kind = PREP_TRANSPOSE; q.in = in; q.ldi = ldi; q.rows = rows; q.cols = cols; q.out = out; q.ldo = ldo;
  q.rows_pad = rows_pad_out; q.cols_pad = cols_pad_out; q.idx = row_idx; q.idx_limit = idx_limit;
  const int ts = dtype == FFSPLIT_BF16 ? 64 : 32;   // tile edge of the transpose for this element size
  q.tiles_x = (rows_pad_out + ts - 1) / ts;
  return add_job(ctx, dtype, q, static_cast<long long>(q.tiles_x) * ((cols_pad_out + ts - 1) / ts), st);
}

ffsplit_status launch_gather_cols_t(ffsplit_ctx* ctx, int dtype, const void* in, long long ldi, int rows,
                                    const int* col_idx, int ncols, int idx_limit, void* out, long long ldo,
                                    int rows_out_pad, cudaStream_t st) {
  if (rows_out_pad <= 0 || rows <= 0) return FFSPLIT_OK;
  PrepJob q{};
  q.kind = PREP_GATHER; q.in = in; q.ldi = ldi; q.rows = rows; q.cols = ncols; q.idx = col_idx; q.idx_limit = idx_limit;
  q.out = out; q.ldo = ldo; q.rows_pad = rows_out_pad;
  q.tiles_x = (rows_out_pad + 31) / 32;
  return add_job(ctx, dtype, q, static_cast<long long>(q.tiles_x) * ((rows + 31) / 32), st);
}

ffsplit_status launch_pack_bias(ffsplit_ctx* ctx, int dtype, const void* b1, const void* b2, const int* heavy, int m,
                                int k, int d, float* b1h, int k_pad, float* b1l, int ml_pad, float* b2o,
                                cudaStream_t st) {
  int n = m;
  if (k_pad > n) n = k_pad;
  if (ml_pad > n) n = ml_pad;
  if (d > n) n = d;
  PrepJob q{};
  q.kind = PREP_PACK_BIAS; q.in = b1; q.in2 = b2; q.idx = heavy; q.rows = m; q.cols = k; q.rows_pad = d;
  q.cols_pad = k_pad; q.idx_limit = ml_pad; q.out = b1h; q.out2 = b1l; q.out3 = b2o;
  return add_job(ctx, dtype, q, (n + 255) / 256, st);
}

ffsplit_status launch_to_f32(ffsplit_ctx* ctx, int dtype, const void* in, int n, float* out, cudaStream_t st) {
  if (n <= 0) return FFSPLIT_OK;
  PrepJob q{};
  q.kind = PREP_TO_F32; q.in = in; q.rows = n; q.out = out;
  return add_job(ctx, dtype, q, (n + 255) / 256, st);
}

}  // namespace ffsp
