// Host side of liboq: error reporting, the two offline constructors (Lloyd-Max codebook, RPBH draw),
// size queries and the device status word.
#include <atomic>
#include <cmath>
#include <cstring>
#include <limits>
#include <mutex>
#include <new>

#include "oq_internal.h"

namespace oq {

static thread_local std::string g_last_error;

int fail(int code, const std::string& msg) {
  g_last_error = msg;
  return code;
}

int cuda_fail(cudaError_t e, const char* what) {
  return fail(OQ_ERR_CUDA, std::string(what) + ": " + cudaGetErrorString(e));
}

// ---------------------------------------------------------------------------------------------------
// Lloyd-Max on the sphere-coordinate marginal (Eq. 2-3).
//
// Unnormalised density g(t) = (1 - t^2)^((d-3)/2).  Cell mass by Gauss-Legendre quadrature on sub-cells
// no wider than half a standard deviation (1/sqrt(d)); the unbounded-looking outer cell is cut 16
// standard deviations above its lower edge, where g has fallen below 1e-55 of its peak.  Cell first
// moment in closed form: int_a^b t g(t) dt = [(1-a^2)^p - (1-b^2)^p] / (d-1), p = (d-1)/2.
// ---------------------------------------------------------------------------------------------------
namespace {

constexpr int kGL = 16;  // 32-point rule, symmetric half stored
// Abscissae / weights of the 32-point Gauss-Legendre rule on [-1, 1] are computed at start-up by
// Newton iteration on the Legendre polynomial (no table to mistype).
struct GL32 {
  double x[2 * kGL], w[2 * kGL];
  GL32() {
    const int n = 2 * kGL;
    for (int i = 0; i < n; ++i) {
      double z = std::cos(M_PI * (i + 0.75) / (n + 0.5));
      double pp = 1.0;
      for (int it = 0; it < 100; ++it) {
        double p1 = 1.0, p2 = 0.0;
        for (int j = 0; j < n; ++j) {
          double p3 = p2;
          p2 = p1;
          p1 = ((2.0 * j + 1.0) * z * p2 - j * p3) / (j + 1.0);
        }
        pp = n * (z * p1 - p2) / (z * z - 1.0);
        double dz = p1 / pp;
        z -= dz;
        if (std::fabs(dz) < 1e-16) break;
      }
      x[i] = z;
      w[i] = 2.0 / ((1.0 - z * z) * pp * pp);
    }
  }
};
const GL32& gl32() {
  static GL32 g;
  return g;
}

double cell_mass(double lo, double hi, int d) {
  const double sigma = 1.0 / std::sqrt((double)d);
  hi = std::fmin(hi, std::fmin(1.0, lo + 16.0 * sigma));
  if (!(hi > lo)) return 0.0;
  const double e = 0.5 * (d - 3);
  int nsub = (int)std::ceil((hi - lo) / (0.5 * sigma));
  if (nsub < 1) nsub = 1;
  const GL32& q = gl32();
  double total = 0.0;
  const double wsub = (hi - lo) / nsub;
  for (int s = 0; s < nsub; ++s) {
    const double a = lo + s * wsub, half = 0.5 * wsub, mid = a + half;
    double acc = 0.0;
    for (int i = 0; i < 2 * kGL; ++i) {
      const double t = mid + half * q.x[i];
      const double u = 1.0 - t * t;
      acc += q.w[i] * (u > 0.0 ? std::exp(e * std::log1p(-t * t)) : 0.0);
    }
    total += acc * half;
  }
  return total;
}

double cell_moment(double lo, double hi, int d) {
  const double p = 0.5 * (d - 1);
  auto prim = [&](double t) { return t < 1.0 ? std::exp(p * std::log1p(-t * t)) : 0.0; };
  return (prim(lo) - prim(hi)) / (d - 1);
}

uint16_t f32_to_bf16_rne(float f) {
  uint32_t u;
  std::memcpy(&u, &f, 4);
  u += 0x7FFFu + ((u >> 16) & 1u);
  return (uint16_t)(u >> 16);
}

// Monotone interpolating polynomial for the level search (see QuantPoly).  nb positive boundaries
// beta[0..nb) in units of the normalised coordinate t.
QuantPoly build_quant_poly(const double* beta, int nb) {
  QuantPoly q;
  q.degree = nb;
  if (nb < 1 || nb > 7) return q;
  const int n = nb + 1;
  double best_slope = 0.0, best_c[8] = {0}, best_clamp = 0.0;
  const double ratios[] = {1.002, 1.005, 1.01, 1.02, 1.03, 1.05};
  for (double ratio : ratios) {
    const double clampv = beta[nb - 1] * ratio;
    for (int ip = 0; ip <= 90; ++ip) {
      const double p0 = 0.05 + 0.01 * ip;
      // nodes y = 2 beta / clamp - 1 (and y = -1 for t = 0), values j (and p0)
      long double A[8][9];
      for (int r = 0; r < n; ++r) {
        const long double y = r == 0 ? -1.0L : 2.0L * beta[r - 1] / clampv - 1.0L;
        long double pw = 1.0L;
        for (int c = 0; c < n; ++c) { A[r][c] = pw; pw *= y; }
        A[r][n] = r == 0 ? p0 : (long double)r;
      }
      bool singular = false;
      for (int c = 0; c < n && !singular; ++c) {
        int piv = c;
        for (int r = c + 1; r < n; ++r) if (fabsl(A[r][c]) > fabsl(A[piv][c])) piv = r;
        if (fabsl(A[piv][c]) < 1e-30L) { singular = true; break; }
        for (int k = 0; k <= n; ++k) { long double t = A[c][k]; A[c][k] = A[piv][k]; A[piv][k] = t; }
        for (int r = 0; r < n; ++r) if (r != c) {
          const long double f = A[r][c] / A[c][c];
          for (int k = c; k <= n; ++k) A[r][k] -= f * A[c][k];
        }
      }
      if (singular) continue;
      double c[8];
      for (int k = 0; k < n; ++k) c[k] = (double)(A[k][n] / A[k][k]);
      auto P = [&](double y) { double a = c[n - 1]; for (int k = n - 2; k >= 0; --k) a = a * y + c[k]; return a; };
      auto dP = [&](double y) { double a = (n - 1) * c[n - 1]; for (int k = n - 2; k >= 1; --k) a = a * y + k * c[k]; return a; };
      const double p1 = P(1.0);
      if (!(p1 > nb + 1e-3 && p1 < nb + 0.9)) continue;
      double slope = 1e300;
      for (int g = 0; g <= 4000; ++g) slope = std::fmin(slope, dP(-1.0 + g / 2000.0));
      if (slope > best_slope) {
        best_slope = slope;
        best_clamp = clampv;
        for (int k = 0; k < 8; ++k) best_c[k] = k < n ? c[k] : 0.0;
      }
    }
  }
  if (!(best_slope > 0.0)) return q;
  // y* with P(y*) = mid + 0.5 (P is increasing on [-1, 1]); then the Taylor shift around y*
  const double mid = (double)(nb / 2);
  auto P = [&](double y) { double a = best_c[n - 1]; for (int k = n - 2; k >= 0; --k) a = a * y + best_c[k]; return a; };
  double lo = -1.0, hi = 1.0;
  for (int it = 0; it < 200; ++it) {
    const double m = 0.5 * (lo + hi);
    if (P(m) < mid + 0.5) lo = m; else hi = m;
  }
  const double ys = 0.5 * (lo + hi);
  double sh[8] = {0};
  for (int k = 0; k < n; ++k)
    for (int j = k; j < n; ++j) {
      double binom = 1.0;
      for (int i = 0; i < k; ++i) binom = binom * (j - i) / (i + 1);
      sh[k] += best_c[j] * binom * std::pow(ys, j - k);
    }
  q.ok = 1;
  q.clamp = (float)best_clamp;
  q.centre = (float)(1.0 + ys);
  q.mid = (float)mid;
  for (int k = 1; k < n; ++k) q.coef[k] = (float)sh[k];
  q.coef[0] = (float)mid;
  return q;
}

}  // namespace

CodebookParams codebook_params(const oq_codebook* cb) {
  CodebookParams p;
  const int L = 1 << cb->bits, M = L / 2;
  for (int j = 0; j < 8; ++j) p.pos_bound[j] = std::numeric_limits<float>::infinity();
  for (int j = 0; j < 16; ++j) p.level_bf16[j] = 0;
  if (cb->bits <= 4) {      // (larger codebooks use WideTables)
    for (int j = 1; j < M; ++j) p.pos_bound[j - 1] = cb->boundaries_f32[M - 1 + j];
    for (int j = 0; j < L; ++j) p.level_bf16[j] = cb->centroids_bf16[j];
  }
  p.bits = cb->bits;
  return p;
}

cudaError_t encode_tensor_map_bf16(CUtensorMap* map, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
                                   const uint32_t* box) {
  typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                               const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                               CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
  static std::atomic<EncodeFn> cached{nullptr};       // (threads racing here store the same pointer)
  EncodeFn encode = cached.load(std::memory_order_acquire);
  if (!encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
    if (e != cudaSuccess) return e;
    if (qres != cudaDriverEntryPointSuccess || !fn) return cudaErrorNotSupported;
    encode = reinterpret_cast<EncodeFn>(fn);
    cached.store(encode, std::memory_order_release);
  }
  cuuint64_t gdim[3] = {1, 1, 1}, gstride[2] = {0, 0};
  cuuint32_t bx[3] = {1, 1, 1}, estride[3] = {1, 1, 1};
  for (int i = 0; i < rank; ++i) { gdim[i] = dims[i]; bx[i] = box[i]; }
  for (int i = 0; i + 1 < rank; ++i) gstride[i] = strides_bytes[i];
  const CUresult r = encode(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank, const_cast<void*>(base), gdim, gstride, bx, estride,
                            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

// First-use state (status words, device tables of the handles) is created under one mutex, so that threads making their
// first call on a device at the same time do not allocate twice or see half-published tables.
static std::mutex g_first_use_mutex;
static int* g_status_word[64] = {nullptr};

int* device_status_word() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(g_first_use_mutex);
  if (!g_status_word[dev]) {
    int* p = nullptr;
    if (cudaMalloc(&p, sizeof(int)) != cudaSuccess) return nullptr;
    if (cudaMemset(p, 0, sizeof(int)) != cudaSuccess) {
      cudaFree(p);
      return nullptr;
    }
    g_status_word[dev] = p;
  }
  return g_status_word[dev];
}

int ensure_wide_tables(const oq_codebook* cb) {
  if (!cb->wide_ok) return fail(OQ_ERR_UNSUPPORTED, "this codebook has no grid tables (6 bits only)");
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
  std::lock_guard<std::mutex> lock(g_first_use_mutex);
  if (cb->d_wide && cb->wide_device == dev) return OQ_OK;
  if (cb->d_wide) return fail(OQ_ERR_INVALID_ARG, "codebook handle was first used on another device");
  WideTables* d = nullptr;
  e = cudaMalloc(&d, sizeof(WideTables));
  if (e != cudaSuccess) return cuda_fail(e, "cudaMalloc(codebook tables)");
  e = cudaMemcpy(d, &cb->wide, sizeof(WideTables), cudaMemcpyHostToDevice);
  if (e != cudaSuccess) {
    cudaFree(d);
    return cuda_fail(e, "cudaMemcpy(codebook tables)");
  }
  cb->wide_device = dev;
  cb->d_wide = d;
  return OQ_OK;
}

// Uploads the four device tables of a rotation.  The handle's pointers are set only after all four exist and hold
// their data; a failure on the way frees what was allocated and leaves the handle as it was (the next call retries).
int ensure_device_tables(const oq_rpbh* rc) {
  oq_rpbh* r = const_cast<oq_rpbh*>(rc);
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
  std::lock_guard<std::mutex> lock(g_first_use_mutex);
  if (r->d_gather && r->device == dev) return OQ_OK;
  if (r->d_gather) return fail(OQ_ERR_INVALID_ARG, "rpbh handle was first used on another device");
  std::vector<uint32_t> g(r->dim), off(r->dim), mask((r->dim + 1) / 2, 0u), pmask((r->dim + 1) / 2, 0u);
  for (int k = 0; k < r->dim; ++k) {
    g[k] = (uint32_t)r->perm[k] | (r->signs[k] < 0 ? 0x80000000u : 0u);
    off[k] = 2u * (uint32_t)r->perm[k];
    if (r->signs[k] < 0) {
      mask[r->perm[k] >> 1] |= (r->perm[k] & 1) ? 0x80000000u : 0x00008000u;
      pmask[k >> 1] |= (k & 1) ? 0x80000000u : 0x00008000u;
    }
  }
  // token-slab kernel: where the chunk of every rotated position sits inside a slab buffer
  std::vector<uint32_t> mm;
  RqMmShape shape;
  const int mm_tok = rq_mm_shape(r->dim, &shape) ? shape.tok : 0;
  if (mm_tok) {
    mm.resize(r->dim);
    const int nb = r->dim / 128;
    for (int j = 0; j < nb; ++j)
      for (int k = 0; k < 128; ++k)
        mm[j * 128 + (k % 8) * 16 + k / 8] = rq_mm_chunk_offset(r->perm[j * 128 + k], mm_tok, nb);
  } else {
    mm.assign(4, 0u);
  }
  const int ntab = 5;
  const std::vector<uint32_t>* host[ntab] = {&g, &off, &mask, &pmask, &mm};
  uint32_t* dev_tab[ntab] = {nullptr, nullptr, nullptr, nullptr, nullptr};
  const char* what = "cudaMalloc(rpbh tables)";
  for (int i = 0; i < ntab && e == cudaSuccess; ++i) {
    what = "cudaMalloc(rpbh tables)";
    e = cudaMalloc(&dev_tab[i], sizeof(uint32_t) * host[i]->size());
    if (e != cudaSuccess) break;
    what = "cudaMemcpy(rpbh tables)";
    e = cudaMemcpy(dev_tab[i], host[i]->data(), sizeof(uint32_t) * host[i]->size(), cudaMemcpyHostToDevice);
  }
  if (e != cudaSuccess) {
    for (int i = 0; i < ntab; ++i)
      if (dev_tab[i]) cudaFree(dev_tab[i]);
    return cuda_fail(e, what);
  }
  r->d_mm_table = dev_tab[4];
  r->mm_tok = mm_tok;
  r->d_offset = dev_tab[1];
  r->d_srcmask = dev_tab[2];
  r->d_posmask = dev_tab[3];
  r->device = dev;
  r->d_gather = dev_tab[0];      // last: the fast path above tests this pointer
  return OQ_OK;
}

}  // namespace oq

using namespace oq;

extern "C" {

const char* oq_last_error(void) { return g_last_error.c_str(); }
const char* oq_version(void) { return "liboq 0.1 (sm_100a)"; }

int oq_build_codebook(int dim, int bits, oq_codebook** out) {
  if (!out) return fail(OQ_ERR_INVALID_ARG, "oq_build_codebook: out is NULL");
  *out = nullptr;
  if (dim < 16) return fail(OQ_ERR_UNSUPPORTED, "oq_build_codebook: dim must be >= 16");
  if (bits < 1 || (bits > 4 && bits != 6)) return fail(OQ_ERR_UNSUPPORTED, "oq_build_codebook: bits must be 1..4 or 6");
  const int L = 1 << bits, M = L / 2;
  const double sigma = 1.0 / std::sqrt((double)dim);
  std::vector<double> c(M), edge(M + 1);
  for (int j = 0; j < M; ++j) c[j] = std::fmin(3.0 * sigma, 1.0) * (2 * j + 1) / (2.0 * M);
  // Plain Lloyd iteration on the positive half (the density is even).  It contracts linearly (ratio
  // about 0.965 at 4 bits), so it runs until the step is at rounding level, with an iteration cap.
  for (int it = 0; it < (bits > 4 ? 200000 : 20000); ++it) {
    edge[0] = 0.0;
    for (int j = 1; j < M; ++j) edge[j] = 0.5 * (c[j - 1] + c[j]);
    edge[M] = 1.0;
    double step = 0.0;
    for (int j = 0; j < M; ++j) {
      const double nc = cell_moment(edge[j], edge[j + 1], dim) / cell_mass(edge[j], edge[j + 1], dim);
      step = std::fmax(step, std::fabs(nc - c[j]));
      c[j] = nc;
    }
    if (step <= 2e-17 * c[M - 1]) break;
  }
  oq_codebook* cb = new (std::nothrow) oq_codebook;
  if (!cb) return fail(OQ_ERR_NOMEM, "oq_build_codebook: out of host memory");
  cb->dim = dim;
  cb->bits = bits;
  cb->centroids.resize(L);
  cb->boundaries.resize(L - 1);
  for (int j = 0; j < M; ++j) {
    cb->centroids[M + j] = c[j];
    cb->centroids[M - 1 - j] = -c[j];
  }
  for (int j = 0; j < L - 1; ++j) cb->boundaries[j] = 0.5 * (cb->centroids[j] + cb->centroids[j + 1]);
  cb->boundaries[M - 1] = 0.0;
  cb->boundaries_f32.resize(L - 1);
  cb->centroids_bf16.resize(L);
  for (int j = 0; j < L - 1; ++j) cb->boundaries_f32[j] = (float)cb->boundaries[j];
  for (int j = 0; j < L; ++j) cb->centroids_bf16[j] = f32_to_bf16_rne((float)cb->centroids[j]);
  if (M > 1 && bits <= 4) cb->poly = build_quant_poly(&cb->boundaries[M], M - 1);
  if (bits == 6) {
    WideTables& w = cb->wide;
    const float gs = (float)(256.0 / (1.01 * cb->boundaries[L - 2]));
    w.grid_scale = gs;
    w.pad[0] = w.pad[1] = w.pad[2] = 0.f;
    for (int j = 0; j < 32; ++j) {
      w.bound_scaled[j] = j < M - 1 ? cb->boundaries_f32[M + j] * gs : std::numeric_limits<float>::infinity();
      w.level_bf16[j] = cb->centroids_bf16[M + j];
    }
    bool ok = true;
    for (int g = 0; g < 256; ++g) {
      int below = 0, inside = 0;
      for (int j = 0; j < M - 1; ++j) {
        if (w.bound_scaled[j] <= (float)g) ++below;
        else if (w.bound_scaled[j] < (float)(g + 1)) ++inside;
      }
      if (inside > 1) ok = false;
      w.cell[g] = (uint8_t)below;
    }
    cb->wide_ok = ok ? 1 : 0;
  }
  *out = cb;
  return OQ_OK;
}

int oq_codebook_get(const oq_codebook* cb, double* centroids, double* boundaries, float* boundaries_f32,
                    uint16_t* centroids_bf16) {
  if (!cb) return fail(OQ_ERR_INVALID_ARG, "oq_codebook_get: handle is NULL");
  const int L = 1 << cb->bits;
  if (centroids) std::memcpy(centroids, cb->centroids.data(), sizeof(double) * L);
  if (boundaries) std::memcpy(boundaries, cb->boundaries.data(), sizeof(double) * (L - 1));
  if (boundaries_f32) std::memcpy(boundaries_f32, cb->boundaries_f32.data(), sizeof(float) * (L - 1));
  if (centroids_bf16) std::memcpy(centroids_bf16, cb->centroids_bf16.data(), sizeof(uint16_t) * L);
  return OQ_OK;
}
int oq_codebook_level_poly(const oq_codebook* cb, float* coef, float* clamp, float* centre, float* mid, int* degree) {
  if (!cb) return fail(OQ_ERR_INVALID_ARG, "oq_codebook_level_poly: handle is NULL");
  if (!cb->poly.ok) return fail(OQ_ERR_UNSUPPORTED, "oq_codebook_level_poly: no polynomial for this codebook");
  if (coef) std::memcpy(coef, cb->poly.coef, sizeof(float) * 8);
  if (clamp) *clamp = cb->poly.clamp;
  if (centre) *centre = cb->poly.centre;
  if (mid) *mid = cb->poly.mid;
  if (degree) *degree = cb->poly.degree;
  return OQ_OK;
}
int oq_codebook_dim(const oq_codebook* cb) { return cb ? cb->dim : 0; }
int oq_codebook_bits(const oq_codebook* cb) { return cb ? cb->bits : 0; }
void oq_codebook_destroy(oq_codebook* cb) {
  if (cb && cb->d_wide) cudaFree(cb->d_wide);
  delete cb;
}

int oq_make_rpbh(int dim, int block, uint64_t seed, oq_rpbh** out) {
  if (!out) return fail(OQ_ERR_INVALID_ARG, "oq_make_rpbh: out is NULL");
  *out = nullptr;
  if (dim <= 0 || dim >= 65536) return fail(OQ_ERR_UNSUPPORTED, "oq_make_rpbh: dim must be in 1..65535");
  if (block <= 0 || (block & (block - 1)) || dim % block)
    return fail(OQ_ERR_INVALID_ARG, "oq_make_rpbh: block must be a power of two that divides dim");
  oq_rpbh* r = new (std::nothrow) oq_rpbh;
  if (!r) return fail(OQ_ERR_NOMEM, "oq_make_rpbh: out of host memory");
  r->dim = dim;
  r->block = block;
  r->seed = seed;
  uint64_t state = seed ^ ((uint64_t)(uint32_t)dim << 32) ^ (uint64_t)block;
  auto next = [&state]() {
    state += 0x9E3779B97F4A7C15ull;
    uint64_t z = state;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
  };
  r->perm.resize(dim);
  for (int i = 0; i < dim; ++i) r->perm[i] = i;
  for (int i = dim - 1; i >= 1; --i) {
    const uint64_t n = (uint64_t)i + 1;
    const uint64_t thr = (0 - n) % n;  // (2^64 - n) mod n
    uint64_t v;
    do v = next();
    while (v < thr);
    const int j = (int)(v % n);
    const int32_t t = r->perm[i];
    r->perm[i] = r->perm[j];
    r->perm[j] = t;
  }
  r->signs.resize(dim);
  for (int base = 0; base < dim; base += 64) {
    const uint64_t word = next();
    for (int b = 0; b < 64 && base + b < dim; ++b) r->signs[base + b] = ((word >> b) & 1) ? -1 : 1;
  }
  *out = r;
  return OQ_OK;
}

int oq_rpbh_get(const oq_rpbh* r, int32_t* perm, int8_t* signs) {
  if (!r) return fail(OQ_ERR_INVALID_ARG, "oq_rpbh_get: handle is NULL");
  if (perm) std::memcpy(perm, r->perm.data(), sizeof(int32_t) * r->dim);
  if (signs) std::memcpy(signs, r->signs.data(), r->dim);
  return OQ_OK;
}
int oq_rpbh_dim(const oq_rpbh* r) { return r ? r->dim : 0; }
int oq_rpbh_block(const oq_rpbh* r) { return r ? r->block : 0; }
void oq_rpbh_destroy(oq_rpbh* r) {
  if (!r) return;
  if (r->d_gather) cudaFree(r->d_gather);
  if (r->d_offset) cudaFree(r->d_offset);
  if (r->d_srcmask) cudaFree(r->d_srcmask);
  if (r->d_posmask) cudaFree(r->d_posmask);
  if (r->d_mm_table) cudaFree(r->d_mm_table);
  delete r;
}

int oq_packed_bytes(int rows, int dim, int bits, size_t* idx_bytes, size_t* row_pitch_bytes) {
  if (rows < 0 || dim <= 0) return fail(OQ_ERR_INVALID_ARG, "oq_packed_bytes: bad sizes");
  if (dim % 128) return fail(OQ_ERR_UNSUPPORTED, "oq_packed_bytes: dim must be a multiple of 128");
  if (bits < 2 || bits > 4) return fail(OQ_ERR_UNSUPPORTED, "oq_packed_bytes: bits must be 2, 3 or 4");
  const size_t pitch = (size_t)dim / 8 * bits;  // dim % 128 == 0 makes this a multiple of 16
  if (row_pitch_bytes) *row_pitch_bytes = pitch;
  if (idx_bytes) *idx_bytes = pitch * (size_t)rows;
  return OQ_OK;
}

int oq_device_status(int* status) {
  if (!status) return fail(OQ_ERR_INVALID_ARG, "oq_device_status: status is NULL");
  *status = 0;
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return cuda_fail(e, "cudaDeviceSynchronize");
  int* w = device_status_word();
  if (!w) return fail(OQ_ERR_CUDA, "oq_device_status: no status word (no usable device?)");
  // Two words exist: the library's own and the one inside the scratch of the allocation-free entry point.  Both are
  // read and both are cleared on every call (a word left set would make every later kernel that shares it give up
  // its waits at once); the first non-zero code is reported.
  int code[2] = {0, 0};
  int* word[2] = {w, noalloc_status_word()};
  for (int i = 0; i < 2; ++i) {
    if (!word[i]) continue;
    e = cudaMemcpy(&code[i], word[i], sizeof(int), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMemcpy(status)");
    if (code[i] != 0) {
      e = cudaMemset(word[i], 0, sizeof(int));
      if (e != cudaSuccess) return cuda_fail(e, "cudaMemset(status)");
    }
  }
  *status = code[0] != 0 ? code[0] : code[1];
  if (*status != 0)
    return fail(OQ_ERR_DEVICE_TIMEOUT, "a bounded device-side wait gave up; status code " + std::to_string(*status));
  return OQ_OK;
}

}  // extern "C"
