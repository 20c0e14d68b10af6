// Quantised split layer (Section 5.2: heavy-hitter neurons 8 bits, everything else 3 bits, round to nearest,
// group size 128): the packed blob's layout and the helpers shared by the quantising pack kernels, the unpack
// kernel and the few-token forward.  Not part of the public ABI.
//
// Groups run along the input (contraction) dimension of each linear map, per output channel: along d for one
// neuron's input weights (a column of U), along the part's neuron axis for one output column of V.  A group is
// stored as its codes followed by its two float32 parameters, so that a row of the packed matrix -- one output
// channel, all its groups -- is one contiguous run of bytes that the streaming kernel copies as it is:
//     8 bits:  [128 code bytes][scale][lo]                      136 bytes
//     3 bits:  [12 words of codes][scale][lo]                    56 bytes
// and a weight is lo + code * scale.  Rows hold an even number of groups (every row then starts and ends on a
// 16-byte boundary); groups past the contraction length, and the codes past it inside the last group, are zero.
//
// 3-bit code words.  A group's 128 codes are four runs of 32 (run c = codes 32c .. 32c+31 = words 3c .. 3c+2).
// Inside a run, word w (0..2) holds codes 10w .. 10w+9 as five pairs -- the even code of pair p in bits
// [3p, 3p+3), the odd one in bits [16+3p, 16+3p+3) -- so that one shift and one mask turn a pair into the two
// mantissas of an fp16x2 register; the run's last two codes (30 and 31) are spread over the spare bits 15 and 31
// of the three words (bit w of code 30 in bit 15 of word w, bit w of code 31 in bit 31 of word w).
#pragma once

#include <stdint.h>

#include "ffsplit.h"

namespace ffsp {
namespace qnt {

constexpr int kGroup = 128;
constexpr int kGroupBytes8 = 136;
constexpr int kGroupBytes3 = 56;
constexpr uint32_t kQuantMagic = 0x51534646u;  // "FFSQ"
constexpr uint32_t kQuantVersion = 1;

enum QSection : int { QS_U1 = 0, QS_U2 = 1, QS_U1U = 2, QS_U2U = 3, QS_V1 = 4, QS_V2 = 5, QS_B1H = 6, QS_B1L = 7, QS_B2 = 8, QS_COUNT = 9 };

struct QuantHeader {
  uint32_t magic, version;
  int32_t d, m, act, k, ml, n_in;
  int32_t gd, gk, gl;          // groups per row (even): along d, along the heavy neurons, along the light neurons
  int32_t k8, ml8;             // k and ml rounded up to multiples of 8 (column offsets of intermediate vectors)
  int32_t reserved0;
  uint64_t total_bytes, logical_bytes;
  uint64_t off[QS_COUNT];
  uint8_t pad[256 - 4 * 14 - 8 * 2 - 8 * QS_COUNT];
};
static_assert(sizeof(QuantHeader) == 256, "quantised blob header is 256 bytes");

inline int even_groups(int n) {
  const int g = (n + kGroup - 1) / kGroup;
  return (g + 1) / 2 * 2;
}

// Position of code e (0..31) of a run inside the run's three words: which word, and the bit of its least
// significant bit -- for e < 30.  Codes 30 and 31 are spread: bit w of the code sits in word w at bit 15 (code 30)
// or bit 31 (code 31).
__host__ __device__ inline void code3_position(int e, int* word, int* bit) {
  const int pair = e >> 1;            // 0..14
  *word = pair / 5;
  *bit = 3 * (pair % 5) + ((e & 1) ? 16 : 0);
}

}  // namespace qnt
}  // namespace ffsp
