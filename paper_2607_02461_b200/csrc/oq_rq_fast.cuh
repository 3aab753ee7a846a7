// Fast fused rotate+quantize kernel for Hadamard blocks of 64, 128 or 256.
//
// Data flow per CTA iteration (T consecutive rows):
//   0. the rows of the NEXT iteration are copied global -> shared with cp.async into the second buffer
//      while the current one is processed (no registers are held, the copy overlaps phases A and B);
//   A. every thread visits its fixed set of 32-bit words (two bf16) of each row in shared memory, flips
//      the sign bits of elements that the permutation sends to a position with sign -1, and accumulates
//      the squared norm of each row;
//   B. a warp lane owns one row t (lane % T) and 64 consecutive rotated coordinates (a whole 64-block, or
//      one half / quarter of a 128- / 256-block): it gathers its permuted elements from row t in shared
//      memory (lanes that share the coordinates read the same element index, so with an odd word pitch
//      the rows fall into distinct banks), runs six butterfly stages in registers and the remaining one or
//      two through warp shuffles, finds each level with a polynomial on the FMA pipe and packs.
#pragma once
#include <cuda_bf16.h>

#include "oq_internal.h"

namespace oq {

struct RqFastParams {
  const uint32_t* X;        // rows x ldx bf16, viewed as words
  int rows, dim, ldw;       // ldw = ldx / 2 (words per input row)
  const uint32_t* offset;   // [dim] byte offset of the source element of rotated position k
  const uint32_t* srcmask;  // [dim/2]
  uint32_t* out_idx;
  int pitch_words;          // words per packed row
  void* out_norm;
  float* dbg;
  QuantPoly poly;
  int groups;               // number of T-row groups
  int bf16_norm;            // 1: norms stored as bf16 (weights), 0: fp32 (activations)
  int ncopy;                // threads (a multiple of 32) that copy and pre-process rows
};

__device__ __forceinline__ unsigned long long pack2(float a, float b) {
  unsigned long long r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(a), "f"(b));
  return r;
}
__device__ __forceinline__ void unpack2(unsigned long long v, float& a, float& b) {
  asm("mov.b64 {%0, %1}, %2;" : "=f"(a), "=f"(b) : "l"(v));
}
__device__ __forceinline__ unsigned long long add2(unsigned long long a, unsigned long long b) {
  unsigned long long r;
  asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ unsigned long long sub2(unsigned long long a, unsigned long long b) {
  unsigned long long r;
  asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
  return r;
}
__device__ __forceinline__ unsigned long long fma2(unsigned long long a, unsigned long long b, unsigned long long c) {
  unsigned long long r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}

// In-register Walsh-Hadamard transform of E values (natural order), unnormalised.
template <int E>
__device__ __forceinline__ void fwht_regs(float (&v)[E]) {
  unsigned long long p[E / 2];
#pragma unroll
  for (int i = 0; i < E / 2; ++i) {            // stage len = 1 inside each pair
    const float a = v[2 * i], b = v[2 * i + 1];
    p[i] = pack2(a + b, a - b);
  }
#pragma unroll
  for (int len = 1; len < E / 2; len <<= 1) {  // pair index distance len  <=>  element distance 2 len
#pragma unroll
    for (int i = 0; i < E / 2; ++i) {
      if ((i & len) == 0) {
        const unsigned long long a = p[i], b = p[i + len];
        p[i] = add2(a, b);
        p[i + len] = sub2(a, b);
      }
    }
  }
#pragma unroll
  for (int i = 0; i < E / 2; ++i) unpack2(p[i], v[2 * i], v[2 * i + 1]);
}

// Bit position bookkeeping of the packed formats (see oq_packing.cuh), resolved at compile time.
template <int BITS>
struct PackOrder;
// 4 bits: one word per 8 coordinates.  Nibbles are emitted from 7 down to 0; nibble n carries the
// magnitude of coordinate n and, in its top bit, the sign of coordinate (n odd ? (n-1)/2 : 4 + n/2).
template <>
struct PackOrder<4> {
  static constexpr int kWordsPer32 = 4;
};
template <>
struct PackOrder<3> {
  static constexpr int kWordsPer32 = 3;
};
template <>
struct PackOrder<2> {
  static constexpr int kWordsPer32 = 2;
};

// The level polynomial with every constant duplicated into both halves of a 64-bit register, so that two
// coordinates are evaluated per instruction.
template <int DEG>
struct Poly2 {
  unsigned long long two, negc, c[DEG + 1], last;
  __device__ __forceinline__ explicit Poly2(const QuantPoly& q) {
    two = pack2(2.f, 2.f);
    negc = pack2(-q.centre, -q.centre);
#pragma unroll
    for (int k = 1; k <= DEG; ++k) c[k] = pack2(q.coef[k], q.coef[k]);
    c[0] = 0ull;
    last = pack2(q.mid + 12582912.f, q.mid + 12582912.f);
  }
  // x = min(|z| kappa, 1);  y = 2x - centre;  bits of (P(y) - 0.5 + 1.5 * 2^23): low bits = floor(P)
  __device__ __forceinline__ void eval(float z0, float z1, float kappa, uint32_t& b0, uint32_t& b1) const {
    const float x0 = __saturatef(fabsf(z0) * kappa), x1 = __saturatef(fabsf(z1) * kappa);
    const unsigned long long y = fma2(pack2(x0, x1), two, negc);
    unsigned long long acc = c[DEG];
#pragma unroll
    for (int k = DEG - 1; k >= 1; --k) acc = fma2(acc, y, c[k]);
    const unsigned long long v = fma2(acc, y, last);
    float f0, f1;
    unpack2(v, f0, f1);
    b0 = __float_as_uint(f0);
    b1 = __float_as_uint(f1);
  }
};

// Sign sources: z minus the smallest subnormal.  The sign bit of the result is set for z <= 0 and clear
// for z > 0, so a coordinate that is exactly zero (a tie between the two middle levels) goes to the lower
// level, the same choice as counting the boundaries strictly below the value.
template <int N>
__device__ __forceinline__ void sign_sources(const float* z, uint32_t* s) {
  const unsigned long long tiny2 = 0x0000000100000001ull;
#pragma unroll
  for (int i = 0; i < N / 2; ++i) {
    float a, b;
    unpack2(sub2(pack2(z[2 * i], z[2 * i + 1]), tiny2), a, b);
    s[2 * i] = __float_as_uint(a);
    s[2 * i + 1] = __float_as_uint(b);
  }
}

__device__ __forceinline__ uint32_t sign_source(float z) { return __float_as_uint(z - __uint_as_float(1u)); }

// One word of the 4-bit format: 8 consecutive rotated coordinates.  Nibbles are emitted from 7 down to 0; nibble n
// carries the magnitude of coordinate n and, in its top bit, the sign of coordinate (n odd ? (n-1)/2 : 4 + n/2).
__device__ __forceinline__ uint32_t pack8_4bit(const float* z, float kappa, const Poly2<7>& poly) {
  constexpr uint32_t MAGIC = 0x4B400000u;
  uint32_t sgn[8], lvl[8];
  sign_sources<8>(z, sgn);
#pragma unroll
  for (int i = 0; i < 4; ++i) poly.eval(z[2 * i], z[2 * i + 1], kappa, lvl[2 * i], lvl[2 * i + 1]);
  uint32_t word = 0;
#pragma unroll
  for (int n = 7; n >= 0; --n) {
    const int se = (n & 1) ? (n - 1) / 2 : 4 + n / 2;            // whose sign rides in nibble n
    word = __funnelshift_l(sgn[se], word, 1);
    word = (word << 3) + lvl[n];
  }
  // every step added MAGIC at nibble position n: remove MAGIC * (16^0 + ... + 16^7) (mod 2^32)
  return word - MAGIC * 0x11111111u;
}

// Packs 32 consecutive rotated coordinates z[0..32) of one row into BITS words.
template <int BITS>
__device__ __forceinline__ void pack32(const float* z, float kappa, const Poly2<(1 << (BITS - 1)) - 1>& poly,
                                       uint32_t* out) {
  [[maybe_unused]] constexpr uint32_t MAGIC = 0x4B400000u;
  if constexpr (BITS == 4) {
#pragma unroll
    for (int w = 0; w < 4; ++w) out[w] = pack8_4bit(z + 8 * w, kappa, poly);
  } else {
    // sign word: coordinate k' sits at bit 8(k'&3) + 7 - (k'>>2); emit bits 31 .. 0
    uint32_t sw = 0;
#pragma unroll
    for (int bit = 31; bit >= 0; --bit) {
      const int kp = (bit >> 3) + 4 * (7 - (bit & 7));
      sw = __funnelshift_l(sign_source(z[kp]), sw, 1);
    }
    out[BITS - 1] = sw;
    uint32_t word = 0;
#pragma unroll
    for (int u = 1; u >= 0; --u) {            // coordinates 16u .. 16u+15
      uint32_t lvl[16];
#pragma unroll
      for (int i = 0; i < 8; ++i) poly.eval(z[16 * u + 2 * i], z[16 * u + 2 * i + 1], kappa, lvl[2 * i], lvl[2 * i + 1]);
      if (BITS == 3) {
        word = 0;
#pragma unroll
        for (int f = 15; f >= 0; --f) {       // 2-bit field f holds kk with f = 2(kk&3) + ((kk>>2)&1) + 8(kk>>3)
          const int kk = ((f & 7) >> 1) + 4 * (f & 1) + 8 * (f >> 3);
          word = (word << 2) + lvl[kk];
        }
        out[u] = word - MAGIC * 0x55555555u;
      } else {
#pragma unroll
        for (int b = 15; b >= 0; --b) {       // bit 16u + b holds k' = 16u + (b>>2) + 4(b&3)
          const int kk = (b >> 2) + 4 * (b & 3);
          word = (word << 1) + lvl[kk];
        }
      }
    }
    if (BITS == 2) out[0] = word - MAGIC * 0xFFFFFFFFu;
  }
}

constexpr int RQ_MAX_THREADS = 512;
// consecutive 32-bit words of a row handled by one copying thread; odd, so that a warp's accesses at this
// stride fall into distinct shared-memory banks
__host__ __device__ constexpr int rq_words_per_thread(int T) { return T >= 16 ? 3 : T == 8 ? 7 : 15; }

template <int H, int T, int BITS>
__global__ void __launch_bounds__(RQ_MAX_THREADS, 1) rq_fast_kernel(const RqFastParams p) {
  constexpr int MAXW = rq_words_per_thread(T);   // 32-bit words one copying thread handles per row
  constexpr bool TAB_SMEM = T >= 8;              // short rows: the offset table lives in shared memory
  constexpr int E = 64;                     // elements per lane
  constexpr int LPB = H / E;                // lanes per Hadamard block (1, 2 or 4)
  constexpr int G = 32 / (T * LPB);         // blocks handled by one warp at a time
  static_assert(H >= 64 && G >= 1, "T * H / 64 lanes must fit in a warp");
  constexpr int WPL = E / 32 * BITS;        // packed words per lane per block

  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int pitch_w = p.dim / 2 + 1;        // odd word pitch: rows of a warp fall into distinct banks
  uint32_t* rowbuf0 = reinterpret_cast<uint32_t*>(smem_raw);        // two buffers of T rows
  float* s_sumsq = reinterpret_cast<float*>(rowbuf0 + 2 * T * pitch_w);   // [warps][T]
  float* s_norm = s_sumsq + (RQ_MAX_THREADS / 32) * T;                    // [T]
  uint32_t* s_table = reinterpret_cast<uint32_t*>(s_norm + T);            // [dim] when p.table_in_smem

  const int tid = threadIdx.x, nthr = blockDim.x, warp = tid >> 5, lane = tid & 31, nwarps = nthr >> 5;
  const int wd = p.dim / 2;
  // the first p.ncopy threads (whole warps) move and pre-process the rows: thread t owns the MAXW consecutive
  // words [t MAXW, (t+1) MAXW) of every row (immediate offsets, no per-word address arithmetic)
  const int w0 = tid * MAXW;
  const bool copier = tid < p.ncopy && w0 < wd;
  const int nw_thr = copier ? min(MAXW, wd - w0) : 0;

  uint32_t mask[MAXW];
#pragma unroll
  for (int q = 0; q < MAXW; ++q) mask[q] = q < nw_thr ? __ldg(p.srcmask + w0 + q) : 0u;

  // Asynchronous copy of one group of T rows into buffer `buf` (4 bytes per lane per instruction, no
  // registers held while the data is in flight).
  auto issue_group = [&](int grp, int buf) {
    if (!copier) return;
    const int row0 = grp * T;
    uint32_t dst = (uint32_t)__cvta_generic_to_shared(rowbuf0 + buf * T * pitch_w + w0);
    const uint32_t* src = p.X + (size_t)row0 * p.ldw + w0;
    const int last = p.rows - 1 - row0;              // rows past the end re-read the last row
#pragma unroll
    for (int r = 0; r < T; ++r) {
      const uint32_t* s = src + (size_t)min(r, last) * p.ldw;
#pragma unroll
      for (int q = 0; q < MAXW; ++q)
        if (q < nw_thr)
          asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(dst + 4u * q), "l"(s + q) : "memory");
      dst += (uint32_t)pitch_w * 4u;
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };

  if (blockIdx.x < p.groups) issue_group(blockIdx.x, 0);
  const uint32_t* table = p.offset;
  if (TAB_SMEM) {
    for (int i = tid; i < p.dim; i += nthr) s_table[i] = __ldg(p.offset + i);
    table = s_table;
  }

  const int t = lane % T, qi = lane / T, sub = qi % LPB, g = qi / LPB;
  const int kblocks = p.dim / H;
  const float inv_sqrt_h = rsqrtf((float)H);
  const Poly2<(1 << (BITS - 1)) - 1> poly(p.poly);

  int it = 0;
  for (int grp = blockIdx.x; grp < p.groups; grp += gridDim.x, ++it) {
    const int row0 = grp * T;
    uint32_t* rowbuf = rowbuf0 + (it & 1) * T * pitch_w;
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncthreads();                          // this group's rows are in shared memory; the other buffer is free
    if (grp + gridDim.x < p.groups) issue_group(grp + gridDim.x, (it + 1) & 1);   // overlaps everything below

    // ---------------- phase A: flip signs in place, accumulate squared norms ----------------
    float ssq[T];
#pragma unroll
    for (int r = 0; r < T; ++r) ssq[r] = 0.f;
    if (copier) {
      uint32_t* rw = rowbuf + w0;
#pragma unroll
      for (int r = 0; r < T; ++r, rw += pitch_w) {
        uint32_t w[MAXW];
#pragma unroll
        for (int q = 0; q < MAXW; ++q)
          if (q < nw_thr) w[q] = rw[q];
        unsigned long long acc2 = 0ull;
#pragma unroll
        for (int q = 0; q < MAXW; ++q)
          if (q < nw_thr) {
            const unsigned long long x2 = pack2(__uint_as_float(w[q] << 16), __uint_as_float(w[q] & 0xFFFF0000u));
            acc2 = fma2(x2, x2, acc2);
            rw[q] = w[q] ^ mask[q];
          }
        float a0, a1;
        unpack2(acc2, a0, a1);
        ssq[r] = a0 + a1;
      }
    }
    // warp reduce-scatter of the T partial sums: afterwards lane L holds the warp total of row L * T / 32
    {
      int n = T;
#pragma unroll
      for (int o = 16; o >= 1; o >>= 1) {
        const bool up = (lane & o) != 0;
        if (n > 1) {
          const int half = n / 2;
#pragma unroll
          for (int i = 0; i < T / 2; ++i)
            if (i < half) {
              const float keep = up ? ssq[i + half] : ssq[i];
              const float send = up ? ssq[i] : ssq[i + half];
              ssq[i] = keep + __shfl_xor_sync(0xffffffffu, send, o);
            }
          n = half;
        } else {
          ssq[0] += __shfl_xor_sync(0xffffffffu, ssq[0], o);
        }
      }
      if (lane % (32 / T) == 0) s_sumsq[warp * T + lane / (32 / T)] = ssq[0];
    }
    __syncthreads();
    if (tid < T) {
      float tot = 0.f;
      for (int w = 0; w < nwarps; ++w) tot += s_sumsq[w * T + tid];
      const float s = sqrtf(tot);
      s_norm[tid] = s;
      if (row0 + tid < p.rows) {
        if (p.bf16_norm) reinterpret_cast<__nv_bfloat16*>(p.out_norm)[row0 + tid] = __float2bfloat16_rn(s);
        else reinterpret_cast<float*>(p.out_norm)[row0 + tid] = s;
      }
    }
    __syncthreads();
    // ---------------- phase B: gather, butterflies, level search, pack ----------------
    const float s = s_norm[t];
    // |t| / clamp = |z| / (sqrt(h) (s + eps) clamp)
    const float kappa = 1.0f / (sqrtf((float)H) * (s + 1e-10f) * p.poly.clamp);
    const unsigned char* rowbytes = reinterpret_cast<const unsigned char*>(rowbuf + t * pitch_w);
    const bool row_ok = row0 + t < p.rows;
    for (int jb = warp * G; jb < kblocks; jb += nwarps * G) {
      const int j = jb + g;
      const bool active = j < kblocks;
      const int jc = active ? j : kblocks - 1;
      const uint4* tab = reinterpret_cast<const uint4*>(table + jc * H + sub * E);
      float v[E];
      {
        uint32_t off[E];                       // all table loads first (independent), gathers afterwards
#pragma unroll
        for (int e4 = 0; e4 < E / 4; ++e4) {
          const uint4 o = tab[e4];
          off[4 * e4] = o.x; off[4 * e4 + 1] = o.y; off[4 * e4 + 2] = o.z; off[4 * e4 + 3] = o.w;
        }
#pragma unroll
        for (int e = 0; e < E; ++e) {
          const uint32_t raw = *reinterpret_cast<const unsigned short*>(rowbytes + off[e]);
          v[e] = __uint_as_float(raw << 16);
        }
      }
      fwht_regs<E>(v);
      // butterflies across the LPB lanes that share a block: element index = sub * 64 + e
#pragma unroll
      for (int st = 1; st < LPB; st <<= 1) {
        const float sg = (sub & st) ? -1.f : 1.f;
#pragma unroll
        for (int e = 0; e < E; ++e) {
          const float other = __shfl_xor_sync(0xffffffffu, v[e], T * st);
          v[e] = fmaf(v[e], sg, other);     // low lane: mine + other;  high lane: other - mine
        }
      }
      if (p.dbg != nullptr) {
        if (row_ok && active) {
          float* d = p.dbg + (size_t)(row0 + t) * p.dim + j * H + sub * E;
#pragma unroll
          for (int e = 0; e < E; ++e) d[e] = v[e] * inv_sqrt_h;
        }
      }
      uint32_t words[WPL];
#pragma unroll
      for (int c = 0; c < E / 32; ++c) pack32<BITS>(v + 32 * c, kappa, poly, words + c * BITS);
      if (row_ok && active) {
        uint32_t* dst = p.out_idx + (size_t)(row0 + t) * p.pitch_words + (j * H + sub * E) / 32 * BITS;
        if (WPL % 4 == 0) {
#pragma unroll
          for (int c = 0; c < WPL / 4; ++c)
            reinterpret_cast<uint4*>(dst)[c] = make_uint4(words[4 * c], words[4 * c + 1], words[4 * c + 2], words[4 * c + 3]);
        } else {
#pragma unroll
          for (int c = 0; c < WPL / 2; ++c) reinterpret_cast<uint2*>(dst)[c] = make_uint2(words[2 * c], words[2 * c + 1]);
        }
      }
    }
  }
}

}  // namespace oq
