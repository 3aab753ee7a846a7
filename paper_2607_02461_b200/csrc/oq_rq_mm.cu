// Launcher of the token-slab rotate+quantize kernel (a translation unit of its own: 27 kernel instances).
#include "oq_rq_mm.cuh"

namespace oq {

namespace {
template <int BITS, int TOK>
cudaError_t launch_mm_block(int block, int grid, size_t smem, cudaStream_t st, const RqMmParams& prm) {
  auto k = block == 64 ? rq_mm_kernel<BITS, TOK, 64> : block == 256 ? rq_mm_kernel<BITS, TOK, 256> : rq_mm_kernel<BITS, TOK, 128>;
  cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  return launch_dependent(k, grid, rqmm::THREADS, smem, st, prm);
}
#ifdef OQ_RQMM_DEV
// development build: only the 4-bit, block-128 kernels
template <int BITS>
cudaError_t launch_mm_tok(int tok, int block, int grid, size_t smem, cudaStream_t st, const RqMmParams& prm) {
  if constexpr (BITS != 4) return cudaErrorNotSupported;
  else {
    if (block != 128) return cudaErrorNotSupported;
    auto k = tok == 8 ? rq_mm_kernel<4, 8, 128> : tok == 4 ? rq_mm_kernel<4, 4, 128> : rq_mm_kernel<4, 2, 128>;
    cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    return launch_dependent(k, grid, rqmm::THREADS, smem, st, prm);
  }
}
#else
template <int BITS>
cudaError_t launch_mm_tok(int tok, int block, int grid, size_t smem, cudaStream_t st, const RqMmParams& prm) {
  if (tok == 8) return launch_mm_block<BITS, 8>(block, grid, smem, st, prm);
  if (tok == 4) return launch_mm_block<BITS, 4>(block, grid, smem, st, prm);
  return launch_mm_block<BITS, 2>(block, grid, smem, st, prm);
}
#endif
}  // namespace

cudaError_t rq_mm_launch(int bits, int tok, int block, int grid, size_t smem, cudaStream_t st, const RqMmParams& prm) {
  if (bits == 4) return launch_mm_tok<4>(tok, block, grid, smem, st, prm);
  if (bits == 3) return launch_mm_tok<3>(tok, block, grid, smem, st, prm);
  return launch_mm_tok<2>(tok, block, grid, smem, st, prm);
}

}  // namespace oq
