// Packed index formats (private to the library; oq_unpack_indices is the public way to read them).
//
// A level index idx in [0, L), L = 2^bits, is stored as sign + magnitude rank:
//     sgn = (idx < L/2),   mag = sgn ? L/2 - 1 - idx : idx - L/2       (levels are antisymmetric)
// so that a decoder can look the magnitude up in a table of L/2 entries and flip one bit for the sign.
// Coordinates keep the rotated order k; rows are `dim * bits / 8` bytes, stored as little-endian
// 32-bit words.  The position of each field inside its word is chosen so that the GEMM's decoder
// obtains byte-permute selectors and bf16 sign masks with one mask or one shift+mask per 4 coordinates:
//
//   4 bits  one word per 8 coordinates e = 0..7: magnitude (3 bits) at bits [4e, 4e+3);
//           sign of e < 4 at bit 8e+7, sign of e >= 4 at bit 8(e-4)+3.
//   3 bits  three words per 32 coordinates k' = 0..31: M0, M1 (2-bit magnitudes of k' < 16 / >= 16),
//           S (signs).  Inside an M word coordinate kk = k' & 15 sits at 2-bit field
//           f = 2(kk & 3) + ((kk >> 2) & 1) + 8(kk >> 3);  in S coordinate k' sits at bit 8(k'&3) + 7 - (k'>>2).
//   2 bits  two words per 32 coordinates: M (1-bit magnitudes) and S as above; in M coordinate k' sits
//           at bit 4(k'&3) + ((k'>>2)&3) + 16(k'>>4).
#pragma once
#include <stdint.h>

namespace oq {

struct FieldPos {
  int mag_word, mag_shift, sign_word, sign_bit;
};

__host__ __device__ inline FieldPos field_pos(int bits, int k) {
  FieldPos p;
  if (bits == 4) {
    const int e = k & 7;
    p.mag_word = p.sign_word = k >> 3;
    p.mag_shift = 4 * e;
    p.sign_bit = e < 4 ? 8 * e + 7 : 8 * (e - 4) + 3;
  } else {
    const int g = k >> 5, kp = k & 31;
    p.sign_bit = 8 * (kp & 3) + 7 - (kp >> 2);
    if (bits == 3) {
      const int kk = kp & 15;
      p.mag_word = 3 * g + (kp >> 4);
      p.mag_shift = 2 * (2 * (kk & 3) + ((kk >> 2) & 1) + 8 * (kk >> 3));
      p.sign_word = 3 * g + 2;
    } else {
      p.mag_word = 2 * g;
      p.mag_shift = 4 * (kp & 3) + ((kp >> 2) & 3) + 16 * (kp >> 4);
      p.sign_word = 2 * g + 1;
    }
  }
  return p;
}

}  // namespace oq
