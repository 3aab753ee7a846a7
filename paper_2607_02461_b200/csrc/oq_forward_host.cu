// Whole layer from HOST buffers: copy tokens in, rotate+quantize, codebook GEMM, copy Y out.
#include "oq_internal.h"

using namespace oq;

namespace oq {
int rotate_quantize_levels_launch(const void* X, int rows, int dim, int ld, const oq_rpbh* rot, const oq_codebook* cb,
                                  void* out_levels, int ld_levels, float* out_norm, void* out_idx8, float* dbg, int* status,
                                  void* stream);
int qlinear_levels_launch(const void* Xd_bf16, int ldxd, const float* Xq_norm, int n_tokens, const void* Wq_idx,
                          const void* Wq_norm_bf16, int m, const oq_codebook* cb_w, int dim, void* Y, int ldy, int y_dtype,
                          int* status, void* stream);
}

namespace {
inline size_t up256(size_t v) { return (v + 255) & ~size_t(255); }
// bytes of the quantized activations between the two kernels: packed indices, or the bf16 level matrix at 6 bits
int act_bytes(int n_tokens, int dim, int bits_a, size_t* bytes) {
  if (bits_a == 6) {
    if (n_tokens < 0 || dim <= 0 || dim % 128) return fail(OQ_ERR_UNSUPPORTED, "6-bit activations: dim must be a positive multiple of 128");
    *bytes = (size_t)n_tokens * dim * 2;
    return OQ_OK;
  }
  return oq_packed_bytes(n_tokens, dim, bits_a, bytes, nullptr);
}
}

extern "C" {

int oq_forward_workspace_bytes(int n_tokens, int dim, int m, int bits_a, size_t* bytes) {
  if (!bytes) return fail(OQ_ERR_INVALID_ARG, "oq_forward_workspace_bytes: bytes is NULL");
  size_t idx = 0;
  int rc = act_bytes(n_tokens, dim, bits_a, &idx);
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
  act_bytes(n_tokens, dim, cb_a->bits, &idx);
  unsigned char* p = reinterpret_cast<unsigned char*>(workspace);
  void* Xd = p;                 p += up256((size_t)n_tokens * dim * 2);
  void* Xq = p;                 p += up256(idx);
  float* Xn = reinterpret_cast<float*>(p); p += up256((size_t)n_tokens * 4);
  void* Yd = p;
  cudaError_t e = cudaMemcpyAsync(Xd, X_host_bf16, (size_t)n_tokens * dim * 2, cudaMemcpyHostToDevice, st);
  if (e != cudaSuccess) return cuda_fail(e, "cudaMemcpyAsync(X)");
  if (cb_a->bits == 6) {      // 64 levels: the level matrix is the hand-over between the two kernels
    rc = rotate_quantize_levels_launch(Xd, n_tokens, dim, dim, rot, cb_a, Xq, dim, Xn, nullptr, nullptr, nullptr, stream);
    if (rc != OQ_OK) return rc;
    rc = qlinear_levels_launch(Xq, dim, Xn, n_tokens, Wq_idx, Wq_norm_bf16, m, cb_w, dim, Yd, m, OQ_BF16, nullptr, stream);
  } else {
    rc = oq_rotate_quantize_act(Xd, n_tokens, dim, dim, rot, cb_a, Xq, Xn, nullptr, stream);
    if (rc != OQ_OK) return rc;
    rc = oq_qlinear(Xq, Xn, n_tokens, cb_a, Wq_idx, Wq_norm_bf16, m, cb_w, dim, Yd, m, OQ_BF16, stream);
  }
  if (rc != OQ_OK) return rc;
  e = cudaMemcpyAsync(Y_host_bf16, Yd, (size_t)n_tokens * m * 2, cudaMemcpyDeviceToHost, st);
  if (e != cudaSuccess) return cuda_fail(e, "cudaMemcpyAsync(Y)");
  return OQ_OK;
}

}  // extern "C"
