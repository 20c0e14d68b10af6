// Quantised split (Section 5.2): the round-to-nearest quantiser that builds the packed matrices, and the
// kernel that expands them again for inspection.  See quant.h for the layout.
//
// One warp quantises one group of 128 weights of one output channel: lane l holds the four weights
// 4l .. 4l+3 of the group, minimum and maximum are taken over the group's real weights with shuffles,
//     scale = (max - min) / (2^b - 1),   code = round_half_even((w - min) / scale) clamped to [0, 2^b - 1]
// all in float32 with correctly rounded operations (a constant group has scale 0 and codes 0), and the codes
// are written in the packed form.  Positions past the contraction length get code 0; a group that lies wholly
// past it gets scale = lo = 0.
#include <cuda_bf16.h>

#include "internal.h"
#include "quant.h"

namespace ffsp {
namespace qnt {

struct PackJob {
  const __nv_bfloat16* W;   // source matrix, row-major with pitch ld
  long long ld;
  int utype;                // 1: element (out, kk) = W[kk * ld + idx[out]]   (one neuron's input weights, kk < d)
                            // 0: element (out, kk) = W[idx[kk] * ld + out]   (one output column, kk over the part's neurons)
  const int* idx;           // the part's neuron indices, ascending
  int n_out, n_k;           // rows of the packed matrix, contraction length
  int groups;               // groups per packed row (even)
  int bits;                 // 8 or 3
  unsigned char* dst;
};

__device__ __forceinline__ float elem(const PackJob& j, int out, int kk) {
  const long long at = j.utype ? static_cast<long long>(kk) * j.ld + j.idx[out]
                               : static_cast<long long>(j.idx[kk]) * j.ld + out;
  return __bfloat162float(j.W[at]);
}

__global__ void __launch_bounds__(256) quant_pack_kernel(const PackJob j) {
  const int lane = threadIdx.x & 31;
  const long long task = static_cast<long long>(blockIdx.x) * 8 + (threadIdx.x >> 5);
  if (task >= static_cast<long long>(j.n_out) * j.groups) return;
  const int out = static_cast<int>(task / j.groups), grp = static_cast<int>(task - static_cast<long long>(out) * j.groups);
  const int k0 = grp * kGroup + 4 * lane;
  float w[4];
  float mn = INFINITY, mx = -INFINITY;
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    w[i] = 0.f;
    if (k0 + i < j.n_k) {
      w[i] = elem(j, out, k0 + i);
      mn = fminf(mn, w[i]);
      mx = fmaxf(mx, w[i]);
    }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    mn = fminf(mn, __shfl_xor_sync(0xffffffffu, mn, o));
    mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
  }
  const bool any = grp * kGroup < j.n_k;
  const float qmax = static_cast<float>((1 << j.bits) - 1);
  const float lo = any ? mn : 0.f;
  const float scale = any ? __fdiv_rn(__fsub_rn(mx, mn), qmax) : 0.f;
  unsigned q[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    float c = 0.f;
    if (scale > 0.f && k0 + i < j.n_k) c = fminf(fmaxf(rintf(__fdiv_rn(__fsub_rn(w[i], lo), scale)), 0.f), qmax);
    q[i] = static_cast<unsigned>(c);
  }
  unsigned char* row = j.dst + static_cast<size_t>(out) * j.groups * (j.bits == 8 ? kGroupBytes8 : kGroupBytes3);
  if (j.bits == 8) {
    unsigned char* gp = row + static_cast<size_t>(grp) * kGroupBytes8;
    reinterpret_cast<unsigned*>(gp)[lane] = q[0] | (q[1] << 8) | (q[2] << 16) | (q[3] << 24);
    if (lane == 0) {
      reinterpret_cast<float*>(gp + 128)[0] = scale;
      reinterpret_cast<float*>(gp + 128)[1] = lo;
    }
  } else {
    // this lane's four codes are codes e0 .. e0+3 of run lane / 8: their bits inside the run's three words,
    // then the eight lanes of the run are OR-ed together
    unsigned wd[3] = {0u, 0u, 0u};
    const int e0 = 4 * (lane & 7);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const int e = e0 + i;
      if (e < 30) {
        int word, bit;
        code3_position(e, &word, &bit);
#pragma unroll
        for (int x = 0; x < 3; ++x)
          if (x == word) wd[x] |= q[i] << bit;
      } else {
        const int bit = e == 30 ? 15 : 31;
#pragma unroll
        for (int x = 0; x < 3; ++x) wd[x] |= ((q[i] >> x) & 1u) << bit;
      }
    }
#pragma unroll
    for (int o = 1; o < 8; o <<= 1)
#pragma unroll
      for (int x = 0; x < 3; ++x) wd[x] |= __shfl_xor_sync(0xffffffffu, wd[x], o);
    unsigned char* gp = row + static_cast<size_t>(grp) * kGroupBytes3;
    if ((lane & 7) == 0) {
      unsigned* dstw = reinterpret_cast<unsigned*>(gp) + 3 * (lane >> 3);
      dstw[0] = wd[0]; dstw[1] = wd[1]; dstw[2] = wd[2];
    }
    if (lane == 0) {
      reinterpret_cast<float*>(gp + 48)[0] = scale;
      reinterpret_cast<float*>(gp + 48)[1] = lo;
    }
  }
}

// Expands one packed matrix: codes [n_out, n_k] as bytes, scale and lo [n_out, ceil(n_k / 128)].
__global__ void __launch_bounds__(256) quant_unpack_kernel(const unsigned char* src, int n_out, int n_k, int groups,
                                                           int bits, unsigned char* codes, float* scale, float* lo) {
  const int lane = threadIdx.x & 31;
  const long long task = static_cast<long long>(blockIdx.x) * 8 + (threadIdx.x >> 5);
  const int real_groups = (n_k + kGroup - 1) / kGroup;
  if (task >= static_cast<long long>(n_out) * real_groups) return;
  const int out = static_cast<int>(task / real_groups), grp = static_cast<int>(task - static_cast<long long>(out) * real_groups);
  const int gb = bits == 8 ? kGroupBytes8 : kGroupBytes3;
  const unsigned char* gp = src + (static_cast<size_t>(out) * groups + grp) * gb;
  for (int i = 0; i < 4; ++i) {
    const int kk = grp * kGroup + 4 * lane + i;
    if (kk >= n_k) continue;
    unsigned q;
    if (bits == 8) {
      q = gp[4 * lane + i];
    } else {
      const int run = lane >> 3, e = 4 * (lane & 7) + i;
      const unsigned* wd = reinterpret_cast<const unsigned*>(gp) + 3 * run;
      if (e < 30) {
        int word, bit;
        code3_position(e, &word, &bit);
        q = (wd[word] >> bit) & 7u;
      } else {
        const int bit = e == 30 ? 15 : 31;
        q = ((wd[0] >> bit) & 1u) | (((wd[1] >> bit) & 1u) << 1) | (((wd[2] >> bit) & 1u) << 2);
      }
    }
    codes[static_cast<size_t>(out) * n_k + kk] = static_cast<unsigned char>(q);
  }
  if (lane == 0) {
    const float* par = reinterpret_cast<const float*>(gp + (bits == 8 ? 128 : 48));
    scale[static_cast<size_t>(out) * real_groups + grp] = par[0];
    lo[static_cast<size_t>(out) * real_groups + grp] = par[1];
  }
}

}  // namespace qnt

ffsplit_status launch_quant_pack(ffsplit_ctx* ctx, const __nv_bfloat16* W, long long ld, int utype, const int* idx,
                                 int n_out, int n_k, int groups, int bits, unsigned char* dst, cudaStream_t st) {
  if (n_out <= 0 || groups <= 0) return FFSPLIT_OK;
  qnt::PackJob j;
  j.W = W; j.ld = ld; j.utype = utype; j.idx = idx; j.n_out = n_out; j.n_k = n_k; j.groups = groups; j.bits = bits;
  j.dst = dst;
  const long long tasks = static_cast<long long>(n_out) * groups;
  const long long blocks = (tasks + 7) / 8;
  if (blocks > 0x7fffffffLL) return fail(ctx, FFSPLIT_ERR_SHAPE, "quantised pack: matrix too large for one launch");
  qnt::quant_pack_kernel<<<static_cast<unsigned>(blocks), 256, 0, st>>>(j);
  ctx->launches++;
  return check_cuda(ctx, cudaGetLastError(), "quant_pack_kernel launch");
}

ffsplit_status launch_quant_unpack(ffsplit_ctx* ctx, const unsigned char* src, int n_out, int n_k, int groups, int bits,
                                   unsigned char* codes, float* scale, float* lo, cudaStream_t st) {
  if (n_out <= 0 || n_k <= 0) return FFSPLIT_OK;
  const long long tasks = static_cast<long long>(n_out) * ((n_k + qnt::kGroup - 1) / qnt::kGroup);
  const long long blocks = (tasks + 7) / 8;
  if (blocks > 0x7fffffffLL) return fail(ctx, FFSPLIT_ERR_SHAPE, "quantised unpack: matrix too large for one launch");
  qnt::quant_unpack_kernel<<<static_cast<unsigned>(blocks), 256, 0, st>>>(src, n_out, n_k, groups, bits, codes, scale, lo);
  ctx->launches++;
  return check_cuda(ctx, cudaGetLastError(), "quant_unpack_kernel launch");
}

}  // namespace ffsp
