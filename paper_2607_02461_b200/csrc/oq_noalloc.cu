// Allocation-free variant of the online layer (rotate+quantize followed by the codebook GEMM).
//
// Some callers cannot allocate device memory at the moment they need a layer evaluated: a serving loop
// that runs under a fixed memory budget handed out at start-up, a host thread that is not allowed to
// block on the allocator, or code that has already frozen its memory pool.  The ordinary path needs two
// pieces of device memory besides the inputs and outputs: the packed activations with their norms (the
// hand-over between the two kernels) and the status word that bounded device-side waits report to.  Here
// both live in a statically sized device array that is part of the library image, so the call performs no
// cudaMalloc / cudaFree and uses no allocating library routine.
#include <mutex>
#include <string>

#include "oq_internal.h"

namespace {

// Scratch of the allocation-free entry point.  Every GPU that loads the library holds these bytes until the
// process exits.  Layout: [0, 256) status word (+ padding), then the norms, then the packed indices.
constexpr size_t kMaxTokens = 32768;                       // norms: 4 bytes per token
constexpr size_t kMaxPackedBytes = 8u << 20;               // packed activation indices: 8 MiB
constexpr size_t kNormOffset = 256;
constexpr size_t kIdxOffset = kNormOffset + kMaxTokens * sizeof(float);
constexpr size_t kScratchBytes = kIdxOffset + kMaxPackedBytes;

static __device__ __align__(256) unsigned char g_noalloc_scratch[kScratchBytes];

// Host code cannot use g_noalloc_scratch as an address (on the host the name is only a handle for the
// symbol); the device address is looked up once per device and cached here.
std::mutex g_scratch_mutex;
unsigned char* g_scratch_dev[64] = {nullptr};

int scratch_for_current_device(unsigned char** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return oq::cuda_fail(e, "cudaGetDevice");
  if (dev < 0 || dev >= 64) return oq::fail(OQ_ERR_UNSUPPORTED, "oq_linear_forward_noalloc: device index above 63");
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (!g_scratch_dev[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_noalloc_scratch);
    if (e != cudaSuccess) return oq::cuda_fail(e, "cudaGetSymbolAddress(scratch)");
    // nothing to clear: a static device array starts zeroed when the module is loaded (the status word must start at
    // zero), and every other byte is written by a call before that call reads it
    g_scratch_dev[dev] = static_cast<unsigned char*>(p);
  }
  *out = g_scratch_dev[dev];
  return OQ_OK;
}

}  // namespace

namespace oq {
int* noalloc_status_word() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return nullptr;
  std::lock_guard<std::mutex> lock(g_scratch_mutex);
  if (!g_scratch_dev[dev]) return nullptr;
  return reinterpret_cast<int*>(g_scratch_dev[dev]);
}
}  // namespace oq

extern "C" int oq_linear_forward_noalloc(const void* X_bf16, int n_tokens, int dim, int ldx, const oq_rpbh* rot,
                                         const oq_codebook* cb_a, const void* Wq_idx, const void* Wq_norm_bf16, int m,
                                         const oq_codebook* cb_w, void* Y, int ldy, int y_dtype, void* stream) {
  using namespace oq;
  if (!rot || !cb_a || !cb_w) return fail(OQ_ERR_INVALID_ARG, "oq_linear_forward_noalloc: NULL handle");
  if (n_tokens < 0 || m < 0 || dim <= 0) return fail(OQ_ERR_INVALID_ARG, "oq_linear_forward_noalloc: bad sizes");
  size_t idx_bytes = 0;
  int rc = oq_packed_bytes(n_tokens, dim, cb_a->bits, &idx_bytes, nullptr);
  if (rc != OQ_OK) return rc;
  if ((size_t)n_tokens > kMaxTokens || idx_bytes > kMaxPackedBytes)
    return fail(OQ_ERR_NOMEM, "oq_linear_forward_noalloc: needs " + std::to_string(idx_bytes) + " bytes of packed activations for " +
                                  std::to_string(n_tokens) + " tokens; the built-in scratch holds " +
                                  std::to_string(kMaxPackedBytes) + " bytes and " + std::to_string(kMaxTokens) +
                                  " tokens (split the batch or use oq_rotate_quantize_act + oq_qlinear)");
  if (n_tokens == 0 || m == 0) return OQ_OK;
  // The rotation's device tables are uploaded (and allocated) by the first ordinary GPU call that uses the
  // handle -- in practice oq_quantize_weights, which has to run before any forward pass.  This entry point
  // must not allocate, so it refuses a handle that has never been on the device.
  if (!rot->d_offset || !rot->d_gather || !rot->d_srcmask || !rot->d_posmask)
    return fail(OQ_ERR_INVALID_ARG,
                "oq_linear_forward_noalloc: the rotation handle has no device tables yet (they are created by the first "
                "oq_quantize_weights / oq_rotate_quantize_act call with this handle)");
  unsigned char* scratch = nullptr;
  rc = scratch_for_current_device(&scratch);
  if (rc != OQ_OK) return rc;
  int* status = reinterpret_cast<int*>(scratch);
  float* norms = reinterpret_cast<float*>(scratch + kNormOffset);
  void* idx = scratch + kIdxOffset;
  rc = rotate_quantize_act_launch(X_bf16, n_tokens, dim, ldx, rot, cb_a, idx, norms, nullptr, status, stream);
  if (rc != OQ_OK) return rc;
  return qlinear_launch(idx, norms, n_tokens, cb_a, Wq_idx, Wq_norm_bf16, m, cb_w, dim, Y, ldy, y_dtype, status, stream);
}
