// Whole layer from HOST buffers: copy tokens in, rotate+quantize, codebook GEMM, copy Y out.
#include "oq_internal.h"

using namespace oq;

namespace {
inline size_t up256(size_t v) { return (v + 255) & ~size_t(255); }
}

extern "C" {

int oq_forward_workspace_bytes(int n_tokens, int dim, int m, int bits_a, size_t* bytes) {
  if (!bytes) return fail(OQ_ERR_INVALID_ARG, "oq_forward_workspace_bytes: bytes is NULL");
  size_t idx = 0, pitch = 0;
  int rc = oq_packed_bytes(n_tokens, dim, bits_a, &idx, &pitch);
  if (rc != OQ_OK) return rc;
  if (m < 0) return fail(OQ_ERR_INVALID_ARG, "oq_forward_workspace_bytes: bad m");
  *bytes = up256((size_t)n_tokens * dim * 2) + up256(idx) + up256((size_t)n_tokens * 4) + up256((size_t)n_tokens * m * 2);
  return OQ_OK;
}

int oq_linear_forward_host(const void* X_host_bf16, int n_tokens, int dim, const oq_rpbh* rot, const oq_codebook* cb_a,
                           const void* Wq_idx, const void* Wq_norm_bf16, int m, const oq_codebook* cb_w,
                           void* Y_host_bf16, void* workspace, size_t workspace_bytes, void* stream) {
  if (!cb_a) return fail(OQ_ERR_INVALID_ARG, "oq_linear_forward_host: NULL codebook");
  size_t need = 0;
  int rc = oq_forward_workspace_bytes(n_tokens, dim, m, cb_a->bits, &need);
  if (rc != OQ_OK) return rc;
  if (n_tokens == 0 || m == 0) return OQ_OK;
  if (!X_host_bf16 || !Y_host_bf16 || !workspace) return fail(OQ_ERR_INVALID_ARG, "oq_linear_forward_host: NULL buffer");
  if (workspace_bytes < need) return fail(OQ_ERR_NOMEM, "oq_linear_forward_host: workspace too small");
  if (!aligned16(workspace)) return fail(OQ_ERR_ALIGNMENT, "oq_linear_forward_host: workspace must be 16-byte aligned");
  cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
  size_t idx = 0;
  oq_packed_bytes(n_tokens, dim, cb_a->bits, &idx, nullptr);
  unsigned char* p = reinterpret_cast<unsigned char*>(workspace);
  void* Xd = p;                 p += up256((size_t)n_tokens * dim * 2);
  void* Xq = p;                 p += up256(idx);
  float* Xn = reinterpret_cast<float*>(p); p += up256((size_t)n_tokens * 4);
  void* Yd = p;
  cudaError_t e = cudaMemcpyAsync(Xd, X_host_bf16, (size_t)n_tokens * dim * 2, cudaMemcpyHostToDevice, st);
  if (e != cudaSuccess) return cuda_fail(e, "cudaMemcpyAsync(X)");
  rc = oq_rotate_quantize_act(Xd, n_tokens, dim, dim, rot, cb_a, Xq, Xn, nullptr, stream);
  if (rc != OQ_OK) return rc;
  rc = oq_qlinear(Xq, Xn, n_tokens, cb_a, Wq_idx, Wq_norm_bf16, m, cb_w, dim, Yd, m, OQ_BF16, stream);
  if (rc != OQ_OK) return rc;
  e = cudaMemcpyAsync(Y_host_bf16, Yd, (size_t)n_tokens * m * 2, cudaMemcpyDeviceToHost, st);
  if (e != cudaSuccess) return cuda_fail(e, "cudaMemcpyAsync(Y)");
  return OQ_OK;
}

}  // extern "C"
