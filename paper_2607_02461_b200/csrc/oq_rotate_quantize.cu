// Fused per-row pass: norm -> RPBH rotation -> nearest Lloyd-Max level -> bit-pack
// (Eq. 7-8 for activations, Eq. 4-6 for weight rows).
#include <cuda_bf16.h>

#include "oq_internal.h"
#include "oq_packing.cuh"
#include "oq_rq_fast.cuh"
#include "oq_rq_mm_params.h"
#include "oq_rq_tc.cuh"

namespace oq {

// -----------------------------------------------------------------------------------------------------
// General kernel: any power-of-two block size up to dim.  One CTA per row (grid-stride over rows), the
// row lives in shared memory as fp32 and the Walsh-Hadamard butterflies run there.
// -----------------------------------------------------------------------------------------------------
template <bool kBf16Norm>
__global__ void __launch_bounds__(256)
rq_general_kernel(const __nv_bfloat16* __restrict__ X, int rows, int dim, int ldx, int block,
                  const uint32_t* __restrict__ gather, CodebookParams cb, uint32_t* __restrict__ out_idx,
                  int pitch_words, void* __restrict__ out_norm, float* __restrict__ dbg) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  float* z = reinterpret_cast<float*>(smem_raw);
  uint8_t* lvl = reinterpret_cast<uint8_t*>(z + dim);
  __shared__ float red[8];
  __shared__ float s_norm;
  const int tid = threadIdx.x, nthr = blockDim.x;
  const int M = (1 << cb.bits) >> 1;
  const float inv_sqrt_h = rsqrtf((float)block);

  for (int row = blockIdx.x; row < rows; row += gridDim.x) {
    const __nv_bfloat16* x = X + (size_t)row * ldx;
    float ss = 0.f;
    for (int k = tid; k < dim; k += nthr) {
      const uint32_t g = gather[k];
      float v = __bfloat162float(x[g & 0xFFFFu]);
      ss = fmaf(v, v, ss);
      z[k] = (g >> 31) ? -v : v;
    }
    for (int o = 16; o; o >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, o);
    if ((tid & 31) == 0) red[tid >> 5] = ss;
    __syncthreads();
    if (tid == 0) {
      float t = 0.f;
      for (int w = 0; w < (nthr >> 5); ++w) t += red[w];
      s_norm = sqrtf(t);
    }
    for (int len = 1; len < block; len <<= 1) {
      __syncthreads();
      for (int p = tid; p < dim / 2; p += nthr) {
        const int i = ((p / len) * 2 * len) + (p % len);
        const float a = z[i], b = z[i + len];
        z[i] = a + b;
        z[i + len] = a - b;
      }
    }
    __syncthreads();
    const float s = s_norm;
    if (tid == 0) {
      if (kBf16Norm) reinterpret_cast<__nv_bfloat16*>(out_norm)[row] = __float2bfloat16_rn(s);
      else reinterpret_cast<float*>(out_norm)[row] = s;
    }
    // thresholds for the un-normalised butterfly output: beta_j * sqrt(h) * (s + eps)
    const float scale = (s + 1e-10f) * sqrtf((float)block);
    for (int k = tid; k < dim; k += nthr) {
      const float v = z[k];
      const float a = fabsf(v);
      int mag = 0;
      for (int j = 0; j < M - 1; ++j) mag += (a > cb.pos_bound[j] * scale) ? 1 : 0;
      lvl[k] = (uint8_t)((v > 0.f) ? M + mag : M - 1 - mag);
      if (dbg) dbg[(size_t)row * dim + k] = v * inv_sqrt_h;
    }
    __syncthreads();
    uint32_t* orow = out_idx + (size_t)row * pitch_words;
    // one thread per 32 coordinates builds that group's words
    for (int g = tid; g < dim / 32; g += nthr) {
      uint32_t w[4] = {0u, 0u, 0u, 0u};
      const int w0 = field_pos(cb.bits, 32 * g).mag_word < field_pos(cb.bits, 32 * g).sign_word
                         ? field_pos(cb.bits, 32 * g).mag_word : field_pos(cb.bits, 32 * g).sign_word;
      for (int kp = 0; kp < 32; ++kp) {
        const int idx = lvl[32 * g + kp];
        const int sgn = idx < M;
        const uint32_t mag = sgn ? M - 1 - idx : idx - M;
        const FieldPos p = field_pos(cb.bits, 32 * g + kp);
        w[p.mag_word - w0] |= mag << p.mag_shift;
        w[p.sign_word - w0] |= (uint32_t)sgn << p.sign_bit;
      }
      for (int i = 0; i < cb.bits; ++i) orow[w0 + i] = w[i];
    }
    __syncthreads();
  }
}

__global__ void unpack_kernel(const uint32_t* __restrict__ idx, int rows, int dim, int bits, int pitch_words,
                              uint8_t* __restrict__ out) {
  const size_t total = (size_t)rows * dim;
  const int M = (1 << bits) >> 1;
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < total; i += (size_t)gridDim.x * blockDim.x) {
    const int row = (int)(i / dim), k = (int)(i % dim);
    const FieldPos p = field_pos(bits, k);
    const uint32_t* r = idx + (size_t)row * pitch_words;
    const int mag = (r[p.mag_word] >> p.mag_shift) & (M - 1);
    const int sgn = (r[p.sign_word] >> p.sign_bit) & 1;
    out[i] = (uint8_t)(sgn ? M - 1 - mag : M + mag);
  }
}

static int check_common(const char* fn, const void* X, int rows, int dim, int ld, const oq_rpbh* rot,
                        const oq_codebook* cb, const void* out_idx, const void* out_norm) {
  if (!rot || !cb) return fail(OQ_ERR_INVALID_ARG, std::string(fn) + ": NULL handle");
  if (rows < 0 || dim <= 0) return fail(OQ_ERR_INVALID_ARG, std::string(fn) + ": bad sizes");
  if (rot->dim != dim || cb->dim != dim)
    return fail(OQ_ERR_INVALID_ARG, std::string(fn) + ": dim differs from the rotation's or the codebook's");
  if (dim % 128) return fail(OQ_ERR_UNSUPPORTED, std::string(fn) + ": dim must be a multiple of 128");
  if (cb->bits < 2 || cb->bits > 4) return fail(OQ_ERR_UNSUPPORTED, std::string(fn) + ": bits must be 2, 3 or 4");
  if (rows == 0) return OQ_OK;
  if (!X || !out_idx || !out_norm) return fail(OQ_ERR_INVALID_ARG, std::string(fn) + ": NULL buffer");
  if (ld < dim) return fail(OQ_ERR_INVALID_ARG, std::string(fn) + ": leading dimension smaller than dim");
  if (ld % 8 || !aligned16(X) || !aligned16(out_idx))
    return fail(OQ_ERR_ALIGNMENT, std::string(fn) + ": pointers must be 16-byte aligned and ld a multiple of 8");
  return OQ_OK;
}

// Picks rows-per-CTA T and the CTA shape for the fast kernel; returns false when the general kernel
// has to be used (block size other than 64/128/256, no monotone level polynomial, or a row too long
// for 8 rows to fit in shared memory).
struct FastPlan {
  int T, threads, ctas_per_sm, ncopy;
  size_t smem;
};
static bool plan_fast(int dim, int block, const oq_codebook* cb, FastPlan* plan) {
  if (block != 64 && block != 128 && block != 256) return false;
  if (!cb->poly.ok) return false;
  const size_t kMaxSmem = 227 * 1024;
  const int lanes_per_block = block / 64;
  // two buffers of T rows (odd word pitch) + per-warp partial sums + norms (+ the offset table for T >= 8)
  auto smem_of = [&](int T) {
    return (size_t)2 * T * (2 * (size_t)dim + 4) + (size_t)(RQ_MAX_THREADS / 32 + 1) * T * 4 + (T >= 8 ? 4 * (size_t)dim : 0);
  };
  // rows per buffer: the largest of 16/8/4 that fits; then as many CTAs per SM (1, 2 or 4) as fit
  int T = 0;
  for (int c = 16; c >= 4 && !T; c >>= 1) {
    if (c * lanes_per_block > 32) continue;
    if (smem_of(c) + 1024 <= kMaxSmem) T = c;
  }
  if (!T) return false;
  int ctas = 1;
  if (2 * (smem_of(T) + 1024) <= kMaxSmem) ctas = 2;
  if (4 * (smem_of(T) + 1024) <= kMaxSmem) ctas = 4;
  plan->T = T;
  plan->ctas_per_sm = ctas;
  plan->threads = RQ_MAX_THREADS / ctas;
  plan->smem = smem_of(T);
  // copying threads: enough whole warps that each handles rq_words_per_thread(T) consecutive words per row
  const int maxw = rq_words_per_thread(T);
  int ncopy = ((dim / 2 + maxw - 1) / maxw + 31) / 32 * 32;
  if (ncopy > plan->threads) return false;
  plan->ncopy = ncopy;
  return true;
}

template <int H, int T>
static cudaError_t launch_fast_bits(int bits, int grid, const FastPlan& pl, cudaStream_t st, const RqFastParams& prm) {
#define OQ_RQ_LAUNCH(B)                                                                                     \
  {                                                                                                         \
    auto k = rq_fast_kernel<H, T, B>;                                                                       \
    cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)pl.smem);     \
    if (e != cudaSuccess) return e;                                                                         \
    k<<<grid, pl.threads, pl.smem, st>>>(prm);                                                              \
    return cudaGetLastError();                                                                              \
  }
  if (bits == 4) OQ_RQ_LAUNCH(4)
  if (bits == 3) OQ_RQ_LAUNCH(3)
  OQ_RQ_LAUNCH(2)
#undef OQ_RQ_LAUNCH
}

template <int H>
static cudaError_t launch_fast_T(int bits, int grid, const FastPlan& pl, cudaStream_t st, const RqFastParams& prm) {
  if (pl.T == 4) return launch_fast_bits<H, 4>(bits, grid, pl, st, prm);
  if (pl.T == 8) return launch_fast_bits<H, 8>(bits, grid, pl, st, prm);
  if constexpr (H <= 128) {
    if (pl.T == 16) return launch_fast_bits<H, 16>(bits, grid, pl, st, prm);
  }
  return cudaErrorInvalidValue;
}

// Which rotate+quantize kernel to use: 0 = choose by shape (never the token-slab kernel: it measured slower than the
// row-per-thread one on every benchmark shape), 1 = general, 2 = register butterflies, 3 = tensor cores (row-per-thread
// gather), 4 = tensor cores (token-slab gather).  A forced kernel that cannot handle the shape falls back.
static int g_forced_kernel = 0;

// Token-slab kernel: blocks of 64, 128, 256; packed outputs; widths for which rq_mm_shape finds a slab size.
static bool plan_mm(int dim, int block, const oq_codebook* cb, RqMmShape* shape) {
  if (block != 64 && block != 128 && block != 256) return false;
  if (cb->bits < 2 || cb->bits > 4 || !cb->poly.ok) return false;
  if (!rq_mm_shape(dim, shape)) return false;
  if (block == 256 && (dim / 128) % 2) return false;
  return true;
}

cudaError_t rq_mm_launch(int bits, int tok, int block, int grid, size_t smem, cudaStream_t st, const RqMmParams& prm);   // oq_rq_mm.cu

// Plan of the tensor-core kernel: th tokens per half group (1, 2, 4 or 8), the largest for which the
// P = th * dim / 128 (token, block) pairs of a half number at most 192 and three half groups of rows fit in
// shared memory beside the Hadamard tile.
struct TcPlan {
  int ths, pairs, ntiles;
  int stages;       // blocks of 512 and more: log2(block / 128) butterfly stages after the tensor-core product
  int tab;          // 0: tables in global memory, 1: both in shared memory, 2: 16-bit offsets in shared memory
  size_t smem;
  double fill;      // used rows of the operand tiles / all rows
};
static bool plan_tc(int dim, int block, const oq_codebook* cb, TcPlan* plan) {
  if (block < 64 || block > 4096 || (block & (block - 1))) return false;
  if (cb->bits == 6 ? !cb->wide_ok : !cb->poly.ok) return false;
  const size_t kMaxSmem = 227 * 1024;
  const int kblocks = dim / 128;
  // blocks above 256: a row's token must be the same in every tile of a group, i.e. th * 2^stages divides 64
  int stages = 0;
  while ((128 << stages) < block) ++stages;
  plan->stages = stages;
  for (int ths = stages > 3 ? 6 - stages : 3; ths >= 0; --ths) {
    const int th = 1 << ths;
    const int pairs = th * kblocks;
    if (pairs > rqtc::MAX_PAIRS) continue;
    // + partial sums, barriers, counters
    const size_t base = 1024 + rqtc::OFF_ROWS + (size_t)rqtc::ROWBUFS * th * rqtc::row_pitch_bytes(dim) + 2 * 16 * 16 * 4 + 256 +
                        (cb->bits == 6 ? 512 : 0);    // (grid tables of a 64-level codebook)
    if (base > kMaxSmem) continue;
    const size_t with_tab = base + (size_t)kblocks * 4 * (rqtc::TAB_PITCH + rqtc::MSK_PITCH);
    const size_t with_tab16 = base + (size_t)kblocks * 4 * rqtc::MSK_PITCH;   // byte offsets fit 16 bits: dim < 32768
    plan->ths = ths;
    plan->pairs = pairs;
    plan->ntiles = pairs <= 128 ? 2 : 3;
    plan->tab = with_tab <= kMaxSmem ? 1 : (with_tab16 <= kMaxSmem && dim < 32768) ? 2 : 0;
    plan->smem = plan->tab == 1 ? with_tab : plan->tab == 2 ? with_tab16 : base;
    // never two of these CTAs on one SM: they would wait for each other's tensor memory
    if (plan->smem < 120 * 1024) plan->smem = 120 * 1024;
    plan->fill = 2.0 * pairs / (128.0 * plan->ntiles);
    return true;
  }
  return false;
}

template <int BITS, int BLK>
static cudaError_t launch_tc_bits(int tab, int grid, size_t smem, cudaStream_t st, const RqTcParams& prm) {
  auto k = tab == 1 ? rq_tc_kernel<BITS, 1, BLK> : tab == 2 ? rq_tc_kernel<BITS, 2, BLK> : rq_tc_kernel<BITS, 0, BLK>;
  cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  return launch_dependent(k, grid, rqtc::THREADS, smem, st, prm);
}
template <int BITS>
static cudaError_t launch_tc_block(int block, int tab, int grid, size_t smem, cudaStream_t st, const RqTcParams& prm) {
  if (block == 64) return launch_tc_bits<BITS, 64>(tab, grid, smem, st, prm);
  if (block == 256) return launch_tc_bits<BITS, 256>(tab, grid, smem, st, prm);
  if (block > 256) return launch_tc_bits<BITS, 512>(tab, grid, smem, st, prm);
  return launch_tc_bits<BITS, 128>(tab, grid, smem, st, prm);
}

template <bool kBf16Norm>
static int launch_rq(const char* fn, const void* X, int rows, int dim, int ld, const oq_rpbh* rot,
                     const oq_codebook* cb, void* out_idx, void* out_norm, float* dbg, int* status, void* stream) {
  int rc = check_common(fn, X, rows, dim, ld, rot, cb, out_idx, out_norm);
  if (rc != OQ_OK || rows == 0) return rc;
  rc = ensure_device_tables(rot);
  if (rc != OQ_OK) return rc;
  const CodebookParams cp = codebook_params(cb);
  const int pitch_words = dim / 32 * cb->bits;
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  int dev = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaError_t e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return cuda_fail(e, "cudaDeviceGetAttribute");
  RqMmShape ms;
  if (g_forced_kernel == 4 && plan_mm(dim, rot->block, cb, &ms) && rot->mm_tok == ms.tok) {
    if (!status) status = device_status_word();
    if (!status) return fail(OQ_ERR_CUDA, std::string(fn) + ": cannot allocate the device status word");
    RqMmParams prm;
    prm.X = reinterpret_cast<const unsigned char*>(X);
    prm.rows = rows; prm.dim = dim; prm.ldx = ld;
    prm.table = rot->d_mm_table; prm.srcmask = rot->d_srcmask;
    prm.out_idx = reinterpret_cast<uint32_t*>(out_idx); prm.pitch_words = pitch_words;
    prm.out_norm = out_norm; prm.dbg = dbg; prm.poly = cb->poly;
    prm.nslabs = (rows + ms.tok - 1) / ms.tok;
    prm.nb = dim / 128;
    prm.seg_rows = ms.seg_rows; prm.pad_rows = ms.pad_rows; prm.tab_smem = ms.tab_smem; prm.mask_smem = ms.mask_smem;
    prm.bf16_norm = kBf16Norm ? 1 : 0;
    prm.status = status;
    const int grid = sms < prm.nslabs ? sms : prm.nslabs;
    e = rq_mm_launch(cb->bits, ms.tok, rot->block, grid, ms.smem, st, prm);
    if (e != cudaSuccess) return cuda_fail(e, fn);
    return OQ_OK;
  }
  TcPlan tp;
  const bool tc_ok = plan_tc(dim, rot->block, cb, &tp);
  if ((g_forced_kernel == 0 && tc_ok && tp.fill >= 0.6) || (g_forced_kernel == 3 && tc_ok)) {
    if (!status) status = device_status_word();
    if (!status) return fail(OQ_ERR_CUDA, std::string(fn) + ": cannot allocate the device status word");
    RqTcParams prm;
    prm.X = reinterpret_cast<const unsigned char*>(X);
    prm.rows = rows; prm.dim = dim; prm.ldx = ld;
    prm.offset = rot->d_offset; prm.posmask = rot->d_posmask;
    prm.out_idx = reinterpret_cast<uint32_t*>(out_idx); prm.pitch_words = pitch_words;
    prm.out_norm = out_norm; prm.dbg = dbg; prm.poly = cb->poly;
    const int T = 2 << tp.ths;
    prm.groups = (rows + T - 1) / T;
    prm.ths = tp.ths; prm.pairs = tp.pairs; prm.ntiles = tp.ntiles;
    prm.bf16_norm = kBf16Norm ? 1 : 0;
    prm.stages = tp.stages;
    prm.wide = nullptr; prm.out_levels = nullptr; prm.ld_levels = 0; prm.out_idx8 = nullptr; prm.grid_scale = 0.f;
    prm.status = status;
    int grid = sms < prm.groups ? sms : prm.groups;
    if (cb->bits == 4) e = launch_tc_block<4>(rot->block, tp.tab, grid, tp.smem, st, prm);
    else if (cb->bits == 3) e = launch_tc_block<3>(rot->block, tp.tab, grid, tp.smem, st, prm);
    else e = launch_tc_block<2>(rot->block, tp.tab, grid, tp.smem, st, prm);
    if (e != cudaSuccess) return cuda_fail(e, fn);
    return OQ_OK;
  }
  FastPlan pl;
  if (g_forced_kernel != 1 && plan_fast(dim, rot->block, cb, &pl)) {
    RqFastParams prm;
    prm.X = reinterpret_cast<const uint32_t*>(X);
    prm.rows = rows; prm.dim = dim; prm.ldw = ld / 2;
    prm.offset = rot->d_offset; prm.srcmask = rot->d_srcmask;
    prm.out_idx = reinterpret_cast<uint32_t*>(out_idx); prm.pitch_words = pitch_words;
    prm.out_norm = out_norm; prm.dbg = dbg; prm.poly = cb->poly;
    prm.groups = (rows + pl.T - 1) / pl.T;
    prm.bf16_norm = kBf16Norm ? 1 : 0;
    prm.ncopy = pl.ncopy;
    int grid = sms * pl.ctas_per_sm;
    if (grid > prm.groups) grid = prm.groups;
    if (rot->block == 64) e = launch_fast_T<64>(cb->bits, grid, pl, st, prm);
    else if (rot->block == 128) e = launch_fast_T<128>(cb->bits, grid, pl, st, prm);
    else e = launch_fast_T<256>(cb->bits, grid, pl, st, prm);
    if (e != cudaSuccess) return cuda_fail(e, fn);
    return OQ_OK;
  }
  const size_t smem = (size_t)dim * 5;
  auto kern = rq_general_kernel<kBf16Norm>;
  if (smem > 48 * 1024) {
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return cuda_fail(e, "cudaFuncSetAttribute");
  }
  int per_sm = 1;
  cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, 256, smem);
  if (per_sm < 1) per_sm = 1;
  int grid = sms * per_sm;
  if (grid > rows) grid = rows;
  kern<<<grid, 256, smem, st>>>(reinterpret_cast<const __nv_bfloat16*>(X), rows, dim, ld, rot->block, rot->d_gather,
                                cp, reinterpret_cast<uint32_t*>(out_idx), pitch_words, out_norm, dbg);
  e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e, fn);
  return OQ_OK;
}

// 64-level activation codebook: the levels themselves are the output (bf16 matrix), the operand of oq_qlinear_levels.
int rotate_quantize_levels_launch(const void* X, int rows, int dim, int ld, const oq_rpbh* rot, const oq_codebook* cb,
                                  void* out_levels, int ld_levels, float* out_norm, void* out_idx8, float* dbg, int* status,
                                  void* stream) {
  const char* fn = "oq_rotate_quantize_act_levels";
  if (!rot || !cb) return fail(OQ_ERR_INVALID_ARG, std::string(fn) + ": NULL handle");
  if (rows < 0 || dim <= 0) return fail(OQ_ERR_INVALID_ARG, std::string(fn) + ": bad sizes");
  if (rot->dim != dim || cb->dim != dim)
    return fail(OQ_ERR_INVALID_ARG, std::string(fn) + ": dim differs from the rotation's or the codebook's");
  if (dim % 128) return fail(OQ_ERR_UNSUPPORTED, std::string(fn) + ": dim must be a multiple of 128");
  if (cb->bits != 6) return fail(OQ_ERR_UNSUPPORTED, std::string(fn) + ": the codebook must have 6 bits");
  TcPlan tp;
  if (!plan_tc(dim, rot->block, cb, &tp))
    return fail(OQ_ERR_UNSUPPORTED, std::string(fn) + ": block must be 64..4096 and the rows must fit the tensor-core kernel");
  if (rows == 0) return OQ_OK;
  if (!X || !out_levels || !out_norm) return fail(OQ_ERR_INVALID_ARG, std::string(fn) + ": NULL buffer");
  if (ld < dim || ld_levels < dim) return fail(OQ_ERR_INVALID_ARG, std::string(fn) + ": leading dimension smaller than dim");
  if (ld % 8 || ld_levels % 8 || !aligned16(X) || !aligned16(out_levels) || (out_idx8 && !aligned16(out_idx8)))
    return fail(OQ_ERR_ALIGNMENT, std::string(fn) + ": pointers must be 16-byte aligned and leading dimensions multiples of 8");
  int rc = ensure_device_tables(rot);
  if (rc != OQ_OK) return rc;
  rc = ensure_wide_tables(cb);
  if (rc != OQ_OK) return rc;
  if (!status) status = device_status_word();
  if (!status) return fail(OQ_ERR_CUDA, std::string(fn) + ": cannot allocate the device status word");
  int dev = 0, sms = 0;
  cudaGetDevice(&dev);
  cudaError_t e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (e != cudaSuccess) return cuda_fail(e, "cudaDeviceGetAttribute");
  RqTcParams prm;
  prm.X = reinterpret_cast<const unsigned char*>(X);
  prm.rows = rows; prm.dim = dim; prm.ldx = ld;
  prm.offset = rot->d_offset; prm.posmask = rot->d_posmask;
  prm.out_idx = nullptr; prm.pitch_words = 0;
  prm.out_norm = out_norm; prm.dbg = dbg; prm.poly = cb->poly;
  const int T = 2 << tp.ths;
  prm.groups = (rows + T - 1) / T;
  prm.ths = tp.ths; prm.pairs = tp.pairs; prm.ntiles = tp.ntiles;
  prm.bf16_norm = 0;
  prm.stages = tp.stages;
  prm.wide = cb->d_wide;
  prm.out_levels = reinterpret_cast<__nv_bfloat16*>(out_levels);
  prm.ld_levels = ld_levels;
  prm.out_idx8 = reinterpret_cast<uint8_t*>(out_idx8);
  prm.grid_scale = cb->wide.grid_scale;
  prm.status = status;
  const int grid = sms < prm.groups ? sms : prm.groups;
  e = launch_tc_block<6>(rot->block, tp.tab, grid, tp.smem, reinterpret_cast<cudaStream_t>(stream), prm);
  if (e != cudaSuccess) return cuda_fail(e, fn);
  return OQ_OK;
}

int rotate_quantize_act_launch(const void* X_bf16, int n_tokens, int dim, int ldx, const oq_rpbh* rot,
                               const oq_codebook* cb_a, void* Xq_idx, float* Xq_norm, float* dbg_rotated, int* status,
                               void* stream) {
  return launch_rq<false>("oq_rotate_quantize_act", X_bf16, n_tokens, dim, ldx, rot, cb_a, Xq_idx, Xq_norm,
                          dbg_rotated, status, stream);
}

}  // namespace oq

using namespace oq;

extern "C" {

int oq_rotate_quantize_act(const void* X_bf16, int n_tokens, int dim, int ldx, const oq_rpbh* rot,
                           const oq_codebook* cb_a, void* Xq_idx, float* Xq_norm, float* dbg_rotated,
                           void* stream) {
  return rotate_quantize_act_launch(X_bf16, n_tokens, dim, ldx, rot, cb_a, Xq_idx, Xq_norm, dbg_rotated, nullptr,
                                    stream);
}

int oq_rotate_quantize_act_levels(const void* X_bf16, int n_tokens, int dim, int ldx, const oq_rpbh* rot,
                                  const oq_codebook* cb_a, void* Xd_bf16, int ldxd, float* Xq_norm, void* idx_u8,
                                  float* dbg_rotated, void* stream) {
  return rotate_quantize_levels_launch(X_bf16, n_tokens, dim, ldx, rot, cb_a, Xd_bf16, ldxd, Xq_norm, idx_u8, dbg_rotated,
                                       nullptr, stream);
}

int oq_rq_plan(const oq_rpbh* rot, const oq_codebook* cb, int* kernel, int* rows_per_group, int* tiles_per_group,
               size_t* smem_bytes) {
  if (!rot || !cb) return fail(OQ_ERR_INVALID_ARG, "oq_rq_plan: NULL handle");
  if (rot->dim != cb->dim) return fail(OQ_ERR_INVALID_ARG, "oq_rq_plan: dim differs between the rotation and the codebook");
  if (rot->dim % 128) return fail(OQ_ERR_UNSUPPORTED, "oq_rq_plan: dim must be a multiple of 128");
  int k = 1, rows = 1, tiles = 0;
  size_t smem = (size_t)rot->dim * 5;
  TcPlan tp;
  FastPlan fp;
  RqMmShape ms;
  const bool tc_ok = plan_tc(rot->dim, rot->block, cb, &tp);
  if (g_forced_kernel == 4 && plan_mm(rot->dim, rot->block, cb, &ms)) {
    k = 4; rows = ms.tok; tiles = 1; smem = ms.smem;
  } else if ((g_forced_kernel == 0 && tc_ok && tp.fill >= 0.6) || (g_forced_kernel == 3 && tc_ok)) {
    k = 3; rows = 2 << tp.ths; tiles = tp.ntiles; smem = tp.smem;
  } else if (g_forced_kernel != 1 && plan_fast(rot->dim, rot->block, cb, &fp)) {
    k = 2; rows = fp.T; smem = fp.smem;
  }
  if (kernel) *kernel = k;
  if (rows_per_group) *rows_per_group = rows;
  if (tiles_per_group) *tiles_per_group = tiles;
  if (smem_bytes) *smem_bytes = smem;
  return OQ_OK;
}

int oq_debug_select_rq_kernel(int which) {
  if (which < 0 || which > 4) return fail(OQ_ERR_INVALID_ARG, "oq_debug_select_rq_kernel: which must be 0..4");
  g_forced_kernel = which;
  return OQ_OK;
}

int oq_quantize_weights(const void* W_bf16, int m, int dim, int ldw, const oq_rpbh* rot, const oq_codebook* cb_w,
                        void* Wq_idx, void* Wq_norm_bf16, void* dbg_rotated, void* stream) {
  return launch_rq<true>("oq_quantize_weights", W_bf16, m, dim, ldw, rot, cb_w, Wq_idx, Wq_norm_bf16,
                         reinterpret_cast<float*>(dbg_rotated), nullptr, stream);
}

int oq_unpack_indices(const void* idx, int rows, int dim, int bits, uint8_t* out, void* stream) {
  if (rows < 0 || dim <= 0) return fail(OQ_ERR_INVALID_ARG, "oq_unpack_indices: bad sizes");
  if (dim % 128) return fail(OQ_ERR_UNSUPPORTED, "oq_unpack_indices: dim must be a multiple of 128");
  if (bits < 2 || bits > 4) return fail(OQ_ERR_UNSUPPORTED, "oq_unpack_indices: bits must be 2, 3 or 4");
  if (rows == 0) return OQ_OK;
  if (!idx || !out) return fail(OQ_ERR_INVALID_ARG, "oq_unpack_indices: NULL buffer");
  const size_t total = (size_t)rows * dim;
  int grid = (int)((total + 255) / 256 < 148 * 16 ? (total + 255) / 256 : 148 * 16);
  unpack_kernel<<<grid, 256, 0, reinterpret_cast<cudaStream_t>(stream)>>>(
      reinterpret_cast<const uint32_t*>(idx), rows, dim, bits, dim / 32 * bits, out);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e, "oq_unpack_indices");
  return OQ_OK;
}

}  // extern "C"
