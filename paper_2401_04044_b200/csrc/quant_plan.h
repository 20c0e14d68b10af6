// Plan of the quantised few-token forward (decode_quant.cu): filled by the host (quant_api.cu).  Not part of
// the public ABI.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "decode_stream.h"

struct ffsplit_ctx;

namespace ffsp {

constexpr int kQuantXBytes = 41472;    // activation operand of a pass in shared memory (fp16), as in decode_stream.h
constexpr int kQuantMaxPhases = 5;
// longest group range of a pass for a given number of token rows (even, at most 160: the activation sums' room)
inline int quant_groups_max(int x_rows) {
  int g = stream_kx_max(x_rows) / 128;
  g = g / 2 * 2;
  return g > 160 ? 160 : g;
}

// Rows of one packed matrix (quant.h): row_bytes apart, `bits` wide codes; multiplied by columns
// [x_off, x_off + 128 G) of the phase's activation matrix; results in output columns [out_col, out_col + rows).
struct QSegment {
  const unsigned char* W;
  long long row_bytes;
  int rows;
  int bits;
  int x_off;
  int out_col;
};

struct QPhase {
  int kind;                 // 0: product; 1: closing reduction
  int sync_before;          // product phases: wait for every CTA to have finished the phase before
  int nseg, nin;
  int G;                    // groups of the contraction (even)
  int S;                    // k ranges (on even group numbers), one output slice each
  int slice0;               // this phase's slices are slice0 .. slice0 + S - 1 of `out`
  int reserved;
  QSegment seg[4];
  StreamInPart in[1];
  float* out;               // raw sums, float [slices][8][out_ld]
  long long out_ld;
  __nv_bfloat16* y;         // closing reduction: layer output [T, y_ld] = sum of in[0]'s slices + y_bias
  long long y_ld;
  const float* y_bias;
  int y_cols;
};

struct QParams {
  QPhase ph[kQuantMaxPhases];
  int nph;
  int T;
  int act;
  int x_rows, x_pitch;
  int* ctrl;
  const unsigned long long* guard;
  unsigned long long guard_hash;
};

ffsplit_status decode_quant_launch(ffsplit_ctx* ctx, const QParams& p, double algo_bytes, cudaStream_t st);

}  // namespace ffsp
