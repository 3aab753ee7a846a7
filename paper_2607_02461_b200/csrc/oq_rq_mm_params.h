// Launch parameters of the token-slab rotate+quantize kernel (shared by its translation unit and the launcher).
#pragma once
#include "oq_internal.h"

namespace oq {

struct RqMmParams {
  const unsigned char* X;   // rows x ldx bf16
  int rows, dim, ldx;
  const uint32_t* table;    // [dim] byte offset of the chunk of rotated position (j, k) inside a slab buffer,
                            // stored at j * 128 + (k % 8) * 16 + k / 8
  const uint32_t* srcmask;  // [dim/2] bf16x2 sign-bit masks indexed by SOURCE position pair
  uint32_t* out_idx;
  int pitch_words;          // words per packed row
  void* out_norm;
  float* dbg;
  QuantPoly poly;
  int nslabs;               // ceil(rows / TOK)
  int nb;                   // dim / 128
  int seg_rows;             // 16-byte rows per segment of the slab buffer (a multiple of 16; 16 segments)
  int pad_rows;             // unused rows at the end of every segment
  int tab_smem;             // 1: the gather table is copied to shared memory
  int mask_smem;            // 1: the sign masks are copied to shared memory
  int bf16_norm;            // 1: norms stored as bf16 (weights), 0: fp32 (activations)
  int* status;
};

}  // namespace oq
