// Decoding packed level indices to bf16 levels with byte-permute table look-ups (shared by the GEMM kernels and
// the kernel that writes an operand out as bf16 levels).
#pragma once
#include <stdint.h>

#include "oq_internal.h"
#include "oq_sm100.cuh"

namespace oq {

// Byte tables of the positive levels: lo/hi bytes of bf16(c_j), j = magnitude rank.
struct Tables {
  uint32_t lo0, lo1, hi0, hi1;
};
__device__ __forceinline__ Tables make_tables(const CodebookParams& cb) {
  const int M = (1 << cb.bits) >> 1;
  Tables t = {0u, 0u, 0u, 0u};
#pragma unroll
  for (int j = 0; j < 8; ++j) {
    const uint32_t v = j < M ? cb.level_bf16[M + j] : 0u;
    if (j < 4) {
      t.lo0 |= (v & 0xFFu) << (8 * j);
      t.hi0 |= (v >> 8) << (8 * j);
    } else {
      t.lo1 |= (v & 0xFFu) << (8 * (j - 4));
      t.hi1 |= (v >> 8) << (8 * (j - 4));
    }
  }
  return t;
}

// Decodes 32 consecutive coordinates (BITS words of one packed row) into four 16-byte chunks of bf16.
// Raw packed words of 32 coordinates of one row (BITS words), fetched ahead of their use.
template <int BITS>
struct Raw {
  uint32_t w[BITS];
};
template <int BITS>
__device__ __forceinline__ Raw<BITS> load_raw(const uint32_t* __restrict__ src) {
  Raw<BITS> r;
  if (BITS == 4) {
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(src));
    r.w[0] = v.x; r.w[1] = v.y; r.w[2] = v.z; r.w[BITS - 1] = v.w;
  } else if (BITS == 3) {
    r.w[0] = __ldg(src); r.w[1] = __ldg(src + 1); r.w[2] = __ldg(src + 2);
  } else {
    const uint2 v = __ldg(reinterpret_cast<const uint2*>(src));
    r.w[0] = v.x; r.w[1] = v.y;
  }
  return r;
}

// The 2 * BITS contiguous words of 64 coordinates of one row, as two 32-coordinate pieces.
template <int BITS>
__device__ __forceinline__ void load_raw64(const uint32_t* __restrict__ src, Raw<BITS>& a, Raw<BITS>& b) {
  if (BITS == 4) {          // 32 bytes, 16-byte aligned
    a = load_raw<BITS>(src);
    b = load_raw<BITS>(src + 4);
  } else if (BITS == 3) {   // 24 bytes, 8-byte aligned
    const uint2 v0 = __ldg(reinterpret_cast<const uint2*>(src));
    const uint2 v1 = __ldg(reinterpret_cast<const uint2*>(src) + 1);
    const uint2 v2 = __ldg(reinterpret_cast<const uint2*>(src) + 2);
    a.w[0] = v0.x; a.w[1] = v0.y; a.w[BITS - 1] = v1.x;
    b.w[0] = v1.y; b.w[1] = v2.x; b.w[BITS - 1] = v2.y;
  } else {                  // 16 bytes, 16-byte aligned
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(src));
    a.w[0] = v.x; a.w[1] = v.y;
    b.w[0] = v.z; b.w[1] = v.w;
  }
}

template <int BITS>
__device__ __forceinline__ void decode32(const Raw<BITS>& raw, const Tables& t, uint4 out[4]) {
  if (BITS == 4) {
    const uint32_t* w = raw.w;
#pragma unroll
    for (int q = 0; q < 4; ++q) {
      const uint32_t sel = w[q] & 0x77777777u;
      const uint32_t loA = prmt(t.lo0, t.lo1, sel), loB = prmt(t.lo0, t.lo1, sel >> 16);
      const uint32_t hiA = prmt(t.hi0, t.hi1, sel) ^ (w[q] & 0x80808080u);
      const uint32_t hiB = prmt(t.hi0, t.hi1, sel >> 16) ^ ((w[q] << 4) & 0x80808080u);
      out[q] = make_uint4(prmt(loA, hiA, 0x5140u), prmt(loA, hiA, 0x7362u), prmt(loB, hiB, 0x5140u),
                          prmt(loB, hiB, 0x7362u));
    }
  } else {
    const uint32_t mw[2] = {raw.w[0], raw.w[BITS == 3 ? 1 : 0]};
    const uint32_t s = raw.w[BITS - 1];
    // byte-permute selectors of the 8 groups of 4 coordinates: the permute reads only the low 16 bits of a
    // selector, so one mask serves two groups (the second after a shift by 16)
    uint32_t selv[8];
    if (BITS == 3) {
#pragma unroll
      for (int u = 0; u < 2; ++u) {
        const uint32_t e = mw[u] & 0x33333333u, o = (mw[u] >> 2) & 0x33333333u;
        selv[4 * u] = e; selv[4 * u + 1] = o; selv[4 * u + 2] = e >> 16; selv[4 * u + 3] = o >> 16;
      }
    } else {
#pragma unroll
      for (int g = 0; g < 4; ++g) {
        const uint32_t e = (mw[0] >> g) & 0x11111111u;
        selv[g] = e; selv[4 + g] = e >> 16;
      }
    }
    uint32_t r[16];
#pragma unroll
    for (int G = 0; G < 8; ++G) {
      const uint32_t sel = selv[G];
      const uint32_t lo = prmt(t.lo0, t.lo0, sel);
      const uint32_t hi = prmt(t.hi0, t.hi0, sel) ^ ((s << G) & 0x80808080u);
      r[2 * G] = prmt(lo, hi, 0x5140u);
      r[2 * G + 1] = prmt(lo, hi, 0x7362u);
    }
#pragma unroll
    for (int q = 0; q < 4; ++q) out[q] = make_uint4(r[4 * q], r[4 * q + 1], r[4 * q + 2], r[4 * q + 3]);
  }
}

}  // namespace oq
