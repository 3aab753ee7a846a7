// AdaLN modulation projections: weight-only INT4 round-to-nearest in groups of 64 input coordinates, bf16
// activations (the supplementary section on quantized layers; Sec. 5.1).  The input is one conditioning token per
// sample, so the layer is a matrix-vector product bound by reading the 4-bit weights once from HBM.
//
//   scale_G = bf16(max_{i in G} |w_i| / 7),   q_i = clamp(rint(w_i / scale_G), -8, 7),
//   y_n[row] = sum_G scale_G * sum_{i in G} q_i x_n[i]
//
// Unpacking a nibble to fp32 and multiplying costs ~3 instructions per weight, which would cap the kernel at about
// half of the HBM bandwidth.  Here a nibble pair becomes a bf16 pair with two instructions ((w >> 4j) & 0x000F000F
// | 0x43004300 is the pair (128 + nibble), minus 136 gives q exactly) and the products run on the tensor cores
// (mma.sync m16n8k16, fp32 accumulation; the up to 8 tokens are the n = 8 columns): ~1.8 instructions per weight.
//
// Packed layout (private): rows in tiles of 16, coordinates in groups of 64.  For tile t, group G, lane L of a
// warp (g = L / 4, i = L % 4) and chunk c of 16 coordinates, ONE 32-bit word holds the lane's whole A fragment
// of the product: nibble j (low half) and nibble j + 4 (high half) form fragment register j,
//     register 0: row g,     coordinates 2i, 2i+1       register 1: row g + 8, coordinates 2i, 2i+1
//     register 2: row g,     coordinates 2i+8, 2i+9     register 3: row g + 8, coordinates 2i+8, 2i+9
// (coordinates relative to 64 G + 16 c; a nibble stores q + 8).  The four words of a lane are adjacent, so a warp
// reads 512 contiguous bytes per (tile, group).  Scales: per (tile, group) 8 words, word g = bf16 scale of row g in
// the low half and of row g + 8 in the high half.
#include <cuda_bf16.h>

#include "oq_internal.h"

namespace oq {
namespace adaln {

constexpr int GROUP = 64;
constexpr int WARPS = 8, THREADS = WARPS * 32;
constexpr int RT = 2;              // row tiles (of 16 rows) per CTA
constexpr int MAXN = 8;            // tokens per launch (the n of m16n8k16)
constexpr int PF = 2;              // groups in flight per warp
constexpr int CTAS_PER_SM = 4;

__device__ __forceinline__ uint32_t sub_bf16x2(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("sub.rn.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}

// d = a * b + c (c may be a literal zero: no register is spent on it)
__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1, float c0, float c1,
                                               float c2, float c3) {
  asm("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%10,%11,%12,%13};"
      : "=f"(d[0]), "=f"(d[1]), "=f"(d[2]), "=f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1), "f"(c0), "f"(c1), "f"(c2), "f"(c3));
}

// Grid: CTA b takes the row tiles [b * tiles_per_cta, (b + 1) * tiles_per_cta), RT at a time (one wave of CTAs for
// the layer's real sizes: the activations are staged once per CTA).  Warp w of the CTA takes the groups w, w + 8,
// ...; the eight partial results meet in shared memory and are added in a fixed order (bit-reproducible output).
__global__ void __launch_bounds__(THREADS, CTAS_PER_SM) adaln_linear_kernel(const uint4* __restrict__ Wq, const uint32_t* __restrict__ S,
                                                               const __nv_bfloat16* __restrict__ X, int n, int ldx, int m,
                                                               int dim, int tiles_per_cta, void* __restrict__ Y, int ldy,
                                                               int f32_out) {
  extern __shared__ uint4 smem_dyn4[];
  uint32_t* xs = reinterpret_cast<uint32_t*>(smem_dyn4);      // [n + 1][dim / 2 + 4] words: rows 4 banks apart; row n is zero
  const int pitch_w = dim / 2 + 4;
  float* red = reinterpret_cast<float*>(xs + (size_t)(n + 1) * pitch_w);   // [WARPS][RT * 16][8]
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, tig = lane & 3;
  const int G = dim / GROUP, tiles = m / 16;
  const int tile_end = min(tiles, ((int)blockIdx.x + 1) * tiles_per_cta);
  int tile0 = blockIdx.x * tiles_per_cta;

  auto load_group = [&](int grp, uint4 (&w)[RT], uint32_t (&sc)[RT]) {
#pragma unroll
    for (int t = 0; t < RT; ++t) {
      if (grp < G && tile0 + t < tile_end) {
        const uint32_t tg = (uint32_t)(tile0 + t) * (uint32_t)G + (uint32_t)grp;      // < 2^26: the host checks m * dim < 2^36
        w[t] = __ldcs(Wq + (tg * 32u + (uint32_t)lane));
        sc[t] = __ldg(S + (tg * 8u + (uint32_t)g));
      } else {
        w[t] = make_uint4(0u, 0u, 0u, 0u);
        sc[t] = 0u;                                  // a zero scale removes whatever the nibbles decode to
      }
    }
  };
  // the weights do not depend on the staged activations: request the first groups before the staging
  uint4 wbuf[PF][RT];
  uint32_t sbuf[PF][RT];
#pragma unroll
  for (int u = 0; u < PF; ++u) load_group(warp + u * WARPS, wbuf[u], sbuf[u]);

  for (int i = tid; i < n * (dim / 8); i += THREADS) {
    const int row = i / (dim / 8), c = i - row * (dim / 8);
    const uint4 v = __ldg(reinterpret_cast<const uint4*>(X + (size_t)row * ldx) + c);
    *reinterpret_cast<uint4*>(xs + (size_t)row * pitch_w + c * 4) = v;
  }
  for (int i = tid; i < pitch_w / 4; i += THREADS) *reinterpret_cast<uint4*>(xs + (size_t)n * pitch_w + i * 4) = make_uint4(0u, 0u, 0u, 0u);
  __syncthreads();
  // column g of the product is token g; the columns past the last token read the zero row
  const uint32_t* xrow = xs + (g < n ? g : n) * pitch_w + tig;

  for (; tile0 < tile_end; tile0 += RT) {
    float acc[RT][4];
#pragma unroll
    for (int t = 0; t < RT; ++t)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[t][e] = 0.f;
    for (int it = 0; warp + it * WARPS < G; it += PF) {
#pragma unroll
      for (int u = 0; u < PF; ++u) {
        const int grp = warp + (it + u) * WARPS;
        if (grp < G) {                                  // warp-uniform
          uint4 w[RT];
          uint32_t sc[RT];
#pragma unroll
          for (int t = 0; t < RT; ++t) {
            w[t] = wbuf[u][t];
            sc[t] = sbuf[u][t];
          }
          load_group(grp + PF * WARPS, wbuf[u], sbuf[u]);
          uint32_t b[4][2];
#pragma unroll
          for (int c = 0; c < 4; ++c) {
            b[c][0] = xrow[grp * 32 + c * 8];
            b[c][1] = xrow[grp * 32 + c * 8 + 4];
          }
#pragma unroll
          for (int t = 0; t < RT; ++t) {
            // two accumulators per group (chunks 0, 1 and 2, 3): two independent chains of tensor-core instructions
            float cg[2][4];
            const uint32_t words[4] = {w[t].x, w[t].y, w[t].z, w[t].w};
#pragma unroll
            for (int c = 0; c < 4; ++c) {
              uint32_t a[4];
#pragma unroll
              for (int j = 0; j < 4; ++j) a[j] = sub_bf16x2(((words[c] >> (4 * j)) & 0x000F000Fu) | 0x43004300u, 0x43084308u);
              if (c & 1) mma_bf16_16816(cg[c >> 1], a, b[c][0], b[c][1], cg[c >> 1][0], cg[c >> 1][1], cg[c >> 1][2], cg[c >> 1][3]);
              else mma_bf16_16816(cg[c >> 1], a, b[c][0], b[c][1], 0.f, 0.f, 0.f, 0.f);
            }
            const float s_lo = __uint_as_float(sc[t] << 16), s_hi = __uint_as_float(sc[t] & 0xFFFF0000u);
            acc[t][0] = fmaf(s_lo, cg[0][0] + cg[1][0], acc[t][0]);
            acc[t][1] = fmaf(s_lo, cg[0][1] + cg[1][1], acc[t][1]);
            acc[t][2] = fmaf(s_hi, cg[0][2] + cg[1][2], acc[t][2]);
            acc[t][3] = fmaf(s_hi, cg[0][3] + cg[1][3], acc[t][3]);
          }
        }
      }
    }
#pragma unroll
    for (int t = 0; t < RT; ++t) {
      float* r0 = red + ((size_t)(warp * RT * 16 + t * 16 + g) * 8 + 2 * tig);
      r0[0] = acc[t][0];
      r0[1] = acc[t][1];
      r0[64] = acc[t][2];        // row g + 8
      r0[65] = acc[t][3];
    }
    // the next tiles' first groups travel during the reduction
    if (tile0 + RT < tile_end) {
      tile0 += RT;
#pragma unroll
      for (int u = 0; u < PF; ++u) load_group(warp + u * WARPS, wbuf[u], sbuf[u]);
      tile0 -= RT;
    }
    __syncthreads();
    // thread -> (token, row of the CTA): a warp stores 32 consecutive outputs of one token
    const int tok = tid >> 5, r = tid & 31;
    const int row = tile0 * 16 + r;
    if (tok < n && row < tile_end * 16) {
      float sum = 0.f;
#pragma unroll
      for (int w = 0; w < WARPS; ++w) sum += red[(size_t)(w * RT * 16 + r) * 8 + tok];
      if (f32_out) reinterpret_cast<float*>(Y)[(size_t)tok * ldy + row] = sum;
      else reinterpret_cast<__nv_bfloat16*>(Y)[(size_t)tok * ldy + row] = __float2bfloat16_rn(sum);
    }
    __syncthreads();               // the partial sums are overwritten by the next tiles
  }
}

// One thread per (row, group): the scale, stored into the paired layout.
__global__ void adaln_scale_kernel(const __nv_bfloat16* __restrict__ W, int m, int dim, int ldw, uint16_t* __restrict__ S16) {
  const int G = dim / GROUP;
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (long long)m * G) return;
  const int row = (int)(idx / G), grp = (int)(idx - (long long)row * G);
  const uint4* src = reinterpret_cast<const uint4*>(W + (size_t)row * ldw + grp * GROUP);
  float amax = 0.f;
#pragma unroll
  for (int v = 0; v < 8; ++v) {
    const uint4 q = __ldg(src + v);
    const uint32_t ws[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      amax = fmaxf(amax, fabsf(__uint_as_float(ws[e] << 16)));
      amax = fmaxf(amax, fabsf(__uint_as_float(ws[e] & 0xFFFF0000u)));
    }
  }
  const __nv_bfloat16 s = __float2bfloat16_rn(__fdiv_rn(amax, 7.0f));
  const int tile = row >> 4, r = row & 15;
  // word (r & 7) of the (tile, group) record, low half for rows 0..7, high half for rows 8..15
  S16[(((size_t)tile * G + grp) * 8 + (r & 7)) * 2 + (r >> 3)] = __bfloat16_as_ushort(s);
}

// One thread per packed word: the eight weights of one A fragment.
__global__ void adaln_pack_kernel(const __nv_bfloat16* __restrict__ W, int m, int dim, int ldw, const uint16_t* __restrict__ S16,
                                  uint32_t* __restrict__ Wq) {
  const int G = dim / GROUP;
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;      // ((tile * G + grp) * 32 + lane) * 4 + c
  if (idx >= (long long)(m / 16) * G * 128) return;
  const int c = (int)(idx & 3), lane = (int)((idx >> 2) & 31);
  const long long tg = idx >> 7;
  const int tile = (int)(tg / G), grp = (int)(tg - (long long)tile * G);
  const int g = lane >> 2, tig = lane & 3;
  const int k0 = grp * GROUP + c * 16 + 2 * tig;
  uint32_t word = 0u;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const int row = tile * 16 + g + ((j & 1) ? 8 : 0);
    const int k = k0 + ((j & 2) ? 8 : 0);
    const float scale = __uint_as_float((uint32_t)S16[(((size_t)tile * G + grp) * 8 + g) * 2 + (j & 1)] << 16);
    const uint32_t pair = __ldg(reinterpret_cast<const uint32_t*>(W + (size_t)row * ldw + k));
    const float w0 = __uint_as_float(pair << 16), w1 = __uint_as_float(pair & 0xFFFF0000u);
    int q0 = 0, q1 = 0;
    if (scale > 0.f) {
      q0 = (int)fminf(fmaxf(rintf(__fdiv_rn(w0, scale)), -8.f), 7.f);
      q1 = (int)fminf(fmaxf(rintf(__fdiv_rn(w1, scale)), -8.f), 7.f);
    }
    word |= (uint32_t)(q0 + 8) << (4 * j);
    word |= (uint32_t)(q1 + 8) << (4 * j + 16);
  }
  Wq[idx] = word;
}

// Test helper: logical values back from the packed layout.
__global__ void adaln_unpack_kernel(const uint32_t* __restrict__ Wq, const uint16_t* __restrict__ S16, int m, int dim,
                                    int8_t* __restrict__ q_out, uint16_t* __restrict__ scale_out) {
  const int G = dim / GROUP;
  const long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (idx >= (long long)m * dim) return;
  const int row = (int)(idx / dim), k = (int)(idx - (long long)row * dim);
  const int tile = row >> 4, r = row & 15, g = r & 7, hi_row = r >> 3;
  const int grp = k / GROUP, kk = k - grp * GROUP, c = kk >> 4, kc = kk & 15;
  const int tig = (kc & 7) >> 1, odd = kc & 1, hi_k = kc >> 3;
  const int j = hi_row + 2 * hi_k;
  const uint32_t word = Wq[(((size_t)tile * G + grp) * 32 + g * 4 + tig) * 4 + c];
  q_out[idx] = (int8_t)((int)((word >> (4 * j + 16 * odd)) & 15u) - 8);
  if (kk == 0) scale_out[(size_t)row * G + grp] = S16[(((size_t)tile * G + grp) * 8 + g) * 2 + hi_row];
}

}  // namespace adaln
}  // namespace oq

using namespace oq;

extern "C" {

int oq_adaln_packed_bytes(int m, int dim, size_t* wq_bytes, size_t* scale_bytes) {
  if (m <= 0 || dim <= 0) return fail(OQ_ERR_INVALID_ARG, "oq_adaln_packed_bytes: bad sizes");
  if (m % 16 || dim % adaln::GROUP) return fail(OQ_ERR_UNSUPPORTED, "oq_adaln_packed_bytes: m must be a multiple of 16, dim of 64");
  if (wq_bytes) *wq_bytes = (size_t)m * dim / 2;
  if (scale_bytes) *scale_bytes = (size_t)m * (dim / adaln::GROUP) * 2;
  return OQ_OK;
}

static int adaln_check_shape(const char* fn, int m, int dim) {
  if (m < 0 || dim <= 0) return fail(OQ_ERR_INVALID_ARG, std::string(fn) + ": bad sizes");
  if (m % 16 || dim % adaln::GROUP) return fail(OQ_ERR_UNSUPPORTED, std::string(fn) + ": m must be a multiple of 16, dim of 64");
  return OQ_OK;
}

int oq_adaln_quantize_weights(const void* W_bf16, int m, int dim, int ldw, void* Wq, void* scales, void* stream) {
  int rc = adaln_check_shape("oq_adaln_quantize_weights", m, dim);
  if (rc != OQ_OK || m == 0) return rc;
  if (!W_bf16 || !Wq || !scales) return fail(OQ_ERR_INVALID_ARG, "oq_adaln_quantize_weights: NULL buffer");
  if (ldw < dim) return fail(OQ_ERR_INVALID_ARG, "oq_adaln_quantize_weights: ldw smaller than dim");
  if (ldw % 8 || !aligned16(W_bf16) || !aligned16(Wq) || !aligned16(scales))
    return fail(OQ_ERR_ALIGNMENT, "oq_adaln_quantize_weights: pointers must be 16-byte aligned and ldw a multiple of 8");
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  const int G = dim / adaln::GROUP;
  const long long nscale = (long long)m * G, nword = (long long)(m / 16) * G * 128;
  const __nv_bfloat16* W = reinterpret_cast<const __nv_bfloat16*>(W_bf16);
  adaln::adaln_scale_kernel<<<(unsigned)((nscale + 255) / 256), 256, 0, st>>>(W, m, dim, ldw, reinterpret_cast<uint16_t*>(scales));
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e, "oq_adaln_quantize_weights (scales)");
  adaln::adaln_pack_kernel<<<(unsigned)((nword + 255) / 256), 256, 0, st>>>(W, m, dim, ldw, reinterpret_cast<const uint16_t*>(scales),
                                                                         reinterpret_cast<uint32_t*>(Wq));
  e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e, "oq_adaln_quantize_weights (pack)");
  return OQ_OK;
}

int oq_adaln_unpack(const void* Wq, const void* scales, int m, int dim, void* q_int8, void* scale_bf16, void* stream) {
  int rc = adaln_check_shape("oq_adaln_unpack", m, dim);
  if (rc != OQ_OK || m == 0) return rc;
  if (!Wq || !scales || !q_int8 || !scale_bf16) return fail(OQ_ERR_INVALID_ARG, "oq_adaln_unpack: NULL buffer");
  const long long total = (long long)m * dim;
  adaln::adaln_unpack_kernel<<<(unsigned)((total + 255) / 256), 256, 0, reinterpret_cast<cudaStream_t>(stream)>>>(
      reinterpret_cast<const uint32_t*>(Wq), reinterpret_cast<const uint16_t*>(scales), m, dim,
      reinterpret_cast<int8_t*>(q_int8), reinterpret_cast<uint16_t*>(scale_bf16));
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e, "oq_adaln_unpack");
  return OQ_OK;
}

int oq_adaln_linear(const void* X_bf16, int n_tokens, int ldx, const void* Wq, const void* scales, int m, int dim,
                    void* Y, int ldy, int y_dtype, void* stream) {
  int rc = adaln_check_shape("oq_adaln_linear", m, dim);
  if (rc != OQ_OK) return rc;
  if (n_tokens < 0) return fail(OQ_ERR_INVALID_ARG, "oq_adaln_linear: bad sizes");
  if (y_dtype != OQ_BF16 && y_dtype != OQ_F32) return fail(OQ_ERR_INVALID_ARG, "oq_adaln_linear: unknown y_dtype");
  if (n_tokens == 0 || m == 0) return OQ_OK;
  if (!X_bf16 || !Wq || !scales || !Y) return fail(OQ_ERR_INVALID_ARG, "oq_adaln_linear: NULL buffer");
  if (ldx < dim || ldy < m) return fail(OQ_ERR_INVALID_ARG, "oq_adaln_linear: leading dimension too small");
  if (ldx % 8 || !aligned16(X_bf16) || !aligned16(Wq) || !aligned16(scales))
    return fail(OQ_ERR_ALIGNMENT, "oq_adaln_linear: pointers must be 16-byte aligned and ldx a multiple of 8");
  const size_t red_bytes = (size_t)adaln::WARPS * adaln::RT * 16 * 8 * 4;
  if ((long long)m * dim >= (1ll << 36)) return fail(OQ_ERR_UNSUPPORTED, "oq_adaln_linear: m * dim must be below 2^36");
  const size_t smem_max = (size_t)((n_tokens < adaln::MAXN ? n_tokens : adaln::MAXN) + 1) * (dim / 2 + 4) * 4 + red_bytes;
  if (smem_max > 227 * 1024) return fail(OQ_ERR_UNSUPPORTED, "oq_adaln_linear: dim too large for the activation staging buffer");
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  if (smem_max > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(adaln::adaln_linear_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_max);
    if (e != cudaSuccess) return cuda_fail(e, "oq_adaln_linear (shared memory attribute)");
  }
  // one wave: as many CTAs as are resident at once, each with an equal share of the row tiles (a multiple of RT)
  int dev = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaError_t ea = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (ea != cudaSuccess) return cuda_fail(ea, "cudaDeviceGetAttribute");
  const int tiles = m / 16;
  const size_t ysz = y_dtype == OQ_F32 ? 4 : 2;
  // the tensor-core tile has 8 columns: more tokens than that take one pass over the weights per 8
  for (int n0 = 0; n0 < n_tokens; n0 += adaln::MAXN) {
    const int n = n_tokens - n0 < adaln::MAXN ? n_tokens - n0 : adaln::MAXN;
    const size_t smem = (size_t)(n + 1) * (dim / 2 + 4) * 4 + red_bytes;
    int per_sm = 1;
    cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, adaln::adaln_linear_kernel, adaln::THREADS, smem);
    if (per_sm < 1) per_sm = 1;
    const int slots = sms * per_sm;
    int per_cta = (tiles + slots - 1) / slots;
    per_cta = (per_cta + adaln::RT - 1) / adaln::RT * adaln::RT;
    const int ctas = (tiles + per_cta - 1) / per_cta;
    adaln::adaln_linear_kernel<<<ctas, adaln::THREADS, smem, st>>>(
        reinterpret_cast<const uint4*>(Wq), reinterpret_cast<const uint32_t*>(scales),
        reinterpret_cast<const __nv_bfloat16*>(X_bf16) + (size_t)n0 * ldx, n, ldx, m, dim, per_cta,
        reinterpret_cast<unsigned char*>(Y) + (size_t)n0 * ldy * ysz, ldy, y_dtype == OQ_F32 ? 1 : 0);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(e, "oq_adaln_linear");
  }
  return OQ_OK;
}

}  // extern "C"
