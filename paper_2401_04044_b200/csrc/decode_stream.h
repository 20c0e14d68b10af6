// Plan of the few-token (1..8 tokens) forward run by decode_stream_kernel: the phases of one layer, what
// each multiplies by and where its activation operand comes from.  Filled by the host (decode.cu), read by
// the kernel (decode_stream.cu).  Not part of the public ABI.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include "ffsplit.h"

struct ffsplit_ctx;

namespace ffsp {

// The activation operand of a pass lives in shared memory: x_rows token rows (1, 2, 4 or 8: the token count
// rounded up) of x_pitch bytes, kStreamXBytes in all.  The fewer tokens, the longer the k range a pass may cover
// (20672 elements for one token, 2560 for eight), and the fewer slices a long contraction has to be cut into.
constexpr int kStreamXBytes = 41472;
inline int stream_x_rows(int T) { return T <= 1 ? 1 : T <= 2 ? 2 : T <= 4 ? 4 : 8; }
inline int stream_kx_max(int x_rows) { return (kStreamXBytes / x_rows - 64) / 128 * 64; }   // elements; pitch = 2 kx + 64
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
  int fin_kind;             // when the phase writes finished values: STREAM_IN_LINEAR (sum + bias) or STREAM_IN_ACT
  const float* fin_bias;    // indexed by the row inside the segment, or nullptr
};

// Geometry of one ring stage: a block of `rows` weight rows (at most 32) times a k chunk of 256 * sub elements;
// the fewer rows a block has, the longer its chunks, so that a stage carries about the same bytes either way
// (a stage of 7 rows x 512 bytes would leave most of the ring, and of the memory pipeline, empty).
constexpr int kStreamStageBytes = 32 * 576;
__host__ __device__ inline int stream_stage_sub(int rows) {
  const int s = (kStreamStageBytes / rows - 64) / 512;
  return s < 1 ? 1 : (s > 8 ? 8 : s);
}

struct StreamPhase {
  static constexpr unsigned kQuantum = 32;   // k ranges start on multiples of 32 elements
  int kind;                 // 0: product; 1: closing reduction (y = sum of in[0]'s slices + y_bias)
  int nseg, nin;
  int K;                    // contraction length of every segment (multiple of 8)
  int S;                    // k ranges the contraction is cut into (one output slice each)
  int Nall;                 // sum of the segments' rows
  StreamSegment seg[kStreamMaxSegments];
  StreamInPart in[2];
  float* out;               // raw sums, float [S][8][out_ld]; nullptr for the phase that writes the layer output
  __nv_bfloat16* outb;      // S == 1 only: finished values (bias, activation, rounded), bf16 [8][out_ld], instead of `out`
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
  int x_rows, x_pitch;      // geometry of the activation operand in shared memory
  int act;                  // ffsplit_act of the layer
  int* ctrl;                // control block: status words, grid-barrier words
  const unsigned long long* guard;   // blob header to verify (or nullptr) and its registered hash
  unsigned long long guard_hash;
};

ffsplit_status decode_stream_launch(ffsplit_ctx* ctx, const StreamParams& p, double algo_bytes, cudaStream_t st);

}  // namespace ffsp
