// Plan of the few-token (1..8 tokens) forward run by decode_stream_kernel: the phases of one layer, what
// each multiplies by and where its activation operand comes from.  Filled by the host (decode.cu), read by
// the kernel (decode_stream.cu).  Not part of the public ABI.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "ffsplit.h"

struct ffsplit_ctx;

namespace ffsp {

constexpr int kStreamKxMax = 2560;     // longest k range of one pass (elements): the activation operand of a pass
                                       // lives in shared memory, 8 token rows of this many bf16 values
constexpr int kStreamMaxPhases = 6;
constexpr int kStreamMaxSegments = 4;

enum StreamInKind : int {
  STREAM_IN_BF16 = 0,    // bf16 rows as they are (the layer input X)
  STREAM_IN_LINEAR = 1,  // sum of the fp32 slices (+ bias)
  STREAM_IN_ACT = 2,     // sigma(sum of the slices + bias): the neurons' activations (Section 2)
  STREAM_IN_GATED = 3    // SiLU(sum of gate slices) * (sum of up slices), the up columns gate_off further on
};

// Columns [col_begin, col_end) of a phase's activation matrix and the memory they are formed from.
struct StreamInPart {
  int col_begin, col_end;
  int kind;               // StreamInKind
  int nslices;            // fp32 kinds: slices to add, in order
  const void* src;        // bf16 [T, ld] or float [nslices][8][ld]
  long long ld;           // elements between token rows
  long long slice_stride; // elements between slices
  int src_col;            // column of src that col_begin maps to
  int gate_off;
  const float* bias;      // indexed by column - col_begin, or nullptr
};

// A block of weight rows that share the phase's contraction: rows of W [rows, K] K-major with pitch ldw,
// multiplied by columns [x_off, x_off + K) of the activation matrix, results in output columns
// [out_col, out_col + rows).
struct StreamSegment {
  const __nv_bfloat16* W;
  long long ldw;
  int rows;
  int x_off;
  int out_col;
};

struct StreamPhase {
  int kind;                 // 0: product; 1: closing reduction (y = sum of in[0]'s slices + y_bias)
  int nseg, nin;
  int K;                    // contraction length of every segment (multiple of 8)
  int S;                    // k ranges the contraction is cut into (one output slice each)
  int Nall;                 // sum of the segments' rows
  StreamSegment seg[kStreamMaxSegments];
  StreamInPart in[2];
  float* out;               // raw sums, float [S][8][out_ld]; nullptr for the phase that writes the layer output
  long long out_ld;
  __nv_bfloat16* y;         // layer output [T, y_ld] (+ y_bias), written when out == nullptr
  long long y_ld;
  const float* y_bias;
  int y_cols;
};

struct StreamParams {
  StreamPhase ph[kStreamMaxPhases];
  int nph;
  int T;                    // 1..8
  int act;                  // ffsplit_act of the layer
  int* ctrl;                // control block: status words, grid-barrier words
  const unsigned long long* guard;   // blob header to verify (or nullptr) and its registered hash
  unsigned long long guard_hash;
};

ffsplit_status decode_stream_launch(ffsplit_ctx* ctx, const StreamParams& p, double algo_bytes, cudaStream_t st);

}  // namespace ffsp
