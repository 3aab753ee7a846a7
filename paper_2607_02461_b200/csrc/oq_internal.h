// Internal declarations shared by the translation units of liboq (not installed).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <string>
#include <utility>
#include <vector>

#include "../../include/oq.h"

// Level search as a polynomial: for a normalised magnitude x = min(|t| / clamp, 1) the number of positive
// cell boundaries below |t| equals floor(P(x)), with P a monotone polynomial of degree 2^(bits-1) - 1
// that takes the value j at the j-th boundary.  P is stored re-expanded around the point where it equals
// mid + 0.5 so that "P - 0.5 + 1.5 * 2^23" has an exactly representable constant term and the rounding
// of one fused multiply-add leaves floor(P) in the low mantissa bits.
struct QuantPoly {
  int degree = 0;          // 2^(bits-1) - 1
  int ok = 0;              // 1 when a monotone interpolant was found
  float clamp = 0.f;       // |t| is clamped here (just above the largest boundary)
  float centre = 0.f;      // y = 2x - centre
  float coef[8] = {0};     // P(y) - 0.5 = mid + coef[1] y + ... + coef[degree] y^degree
  float mid = 0.f;         // integer constant term
};

// Tables of a codebook with 64 levels (6 bits), whose level search runs on a uniform grid of the normalised
// magnitude instead of a polynomial: u = |t| * grid_scale falls into cell g = min(int(u), 255); cell[g] positive
// boundaries lie at or below the cell's lower edge and at most one lies inside it, so the magnitude rank is
// cell[g] + (u > bound_scaled[cell[g]]).  Device layout (16-byte aligned, 464 bytes).
struct WideTables {
  float bound_scaled[32];    // positive boundaries times grid_scale, ascending; unused entries +inf
  uint16_t level_bf16[32];   // positive levels, ascending
  uint8_t cell[256];
  float grid_scale;          // 256 / (1.01 * largest boundary)
  float pad[3];
};

struct oq_codebook {
  int dim = 0, bits = 0;
  int wide_ok = 0;                   // 6 bits: the grid tables below are valid
  WideTables wide;
  mutable WideTables* d_wide = nullptr;   // device copy, created on first GPU use
  mutable int wide_device = -1;
  QuantPoly poly;
  std::vector<double> centroids;     // 2^bits ascending
  std::vector<double> boundaries;    // 2^bits - 1 midpoints
  std::vector<float> boundaries_f32;
  std::vector<uint16_t> centroids_bf16;
};

struct oq_rpbh {
  int dim = 0, block = 0;
  uint64_t seed = 0;
  std::vector<int32_t> perm;   // (P x)_k = x[perm[k]]
  std::vector<int8_t> signs;   // +1 / -1, indexed by k (after the permutation)
  // device copies, created on first GPU use
  int device = -1;
  uint32_t* d_gather = nullptr;  // [dim] word k: low 16 bits = perm[k], bit 31 = 1 when sign is -1
  uint32_t* d_offset = nullptr;  // [dim] byte offset 2 * perm[k] of the source element of rotated position k
  uint32_t* d_srcmask = nullptr; // [dim/2] bf16x2 sign-bit masks indexed by SOURCE position: 0x8000 where the
                                 // element moves to a position whose sign is -1
  uint32_t* d_posmask = nullptr; // [dim/2] bf16x2 sign-bit masks indexed by ROTATED position: bit 15 / bit 31 set where
                                 // position 2i / 2i+1 has sign -1
  uint32_t* d_mm_table = nullptr; // [dim] token-slab kernel: byte offset, inside a slab buffer, of the chunk of rotated
                                 // position (j, k), stored at j * 128 + (k % 8) * 16 + k / 8; NULL when mm_tok == 0
  int mm_tok = 0;                // tokens per slab of the token-slab kernel for this width (8, 4, 2), 0: not supported
};

namespace oq {

// ---- layout of the token-slab rotate+quantize kernel (shared by the kernel, its launcher and the table builder) ----
// A slab is `tok` consecutive tokens (8, 4 or 2 by row length).  Its rows are transposed into a slab buffer of
// 16-byte rows: a row holds 8 / tok source coordinates (32 apart) of all tok tokens, the tok values of one
// coordinate adjacent (a "chunk").  The tensor cores read the buffer as both operands of a Gram product, as an
// MN-major matrix with the 128-byte swizzle: two halves of 8 * seg_rows rows each (seg_rows a multiple of 16), of which
// the last 8 * pad_rows rows are unused and stay zero.
// position of source coordinate cb (0..31) of a window among the window's 32 rows of the slab buffer: the 8 rows
// that one stmatrix phase writes fall into 8 different 16-byte bank groups
__host__ __device__ constexpr int rq_mm_window_row(int cb) { return (cb & ~7) | ((cb + 2 * (cb >> 3)) & 7); }
// Byte offset, inside a slab buffer, of the chunk (tok tokens x 2 bytes) of source coordinate i.
inline uint32_t rq_mm_chunk_offset(int i, int tok, int nb) {
  const int hw = 8 / tok;                       // coordinates that share one 16-byte row
  const int w = i / (32 * hw), r = i % (32 * hw), h = r / 32, cb = r % 32;
  const int raw = nb * tok, seg_rows = (raw + 15) / 16 * 16;
  const int lin = w * 32 + rq_mm_window_row(cb);
  const int row = lin + (lin >= 8 * raw ? 8 * (seg_rows - raw) : 0);
  return 16u * (uint32_t)row + (uint32_t)(h * 2 * tok);
}
struct RqMmShape {
  int tok, seg_rows, pad_rows, tab_smem, mask_smem;
  size_t smem;
};
// false: this width does not run on the token-slab kernel.  The largest slab that fits in shared memory beside the
// Hadamard tile (32 KB) and the operand tile (32 KB); a tile of 128 / tok chunks must not touch more than the two
// slabs that are resident.
inline bool rq_mm_shape(int dim, RqMmShape* shape) {
  if (dim <= 0 || dim % 128) return false;
  const size_t kMaxSmem = 227 * 1024;
  const int nb = dim / 128;
  for (int tok = 8; tok >= 2; tok >>= 1) {
    const int hw = 8 / tok, bc = 128 / tok;
    if (dim % (32 * hw)) continue;
    if (dim / (32 * hw) > 128) continue;       // 16 front-end warps x 8 windows in registers per slab
    if (!(nb >= bc - 1 || (bc % nb == 0 && bc / nb <= 2))) continue;
    const int raw = nb * tok, seg_rows = (raw + 15) / 16 * 16;
    if (seg_rows > 16383) continue;
    const size_t slab = 256 * (size_t)seg_rows;
    // what else goes to shared memory, in order of preference: the sign masks (read once per 8 coordinates), then the
    // gather table (read once per chunk, in batches); what stays out is read through L1
    for (int opt = 3; opt >= 0; --opt) {
      const int mask = (opt == 3 || opt == 2) ? 1 : 0, tab = (opt == 3 || opt == 1) ? 1 : 0;
      const size_t smem = 1024 + 65536 + 2 * slab + (tab ? 4 * (size_t)dim : 0) + (mask ? 2 * (size_t)dim : 0) + 3072;
      if (smem <= kMaxSmem) {
        shape->tok = tok; shape->seg_rows = seg_rows; shape->pad_rows = seg_rows - raw;
        shape->tab_smem = tab; shape->mask_smem = mask; shape->smem = smem;
        return true;
      }
    }
  }
  return false;
}

int fail(int code, const std::string& msg);   // records the message, returns code
int cuda_fail(cudaError_t e, const char* what);
int ensure_device_tables(const oq_rpbh* r);   // uploads d_gather on first use
int ensure_wide_tables(const oq_codebook* cb); // uploads the grid tables of a 6-bit codebook on first use

// Values a kernel needs from a codebook, passed by value as a launch parameter.
struct CodebookParams {
  float pos_bound[8];    // positive boundaries beta_j (j >= 1 of the upper half), unused entries = +inf
  uint16_t level_bf16[16];
  int bits;
};
CodebookParams codebook_params(const oq_codebook* cb);

// cuTensorMapEncodeTiled through the runtime's driver entry point (no link-time dependency on the driver library).
// bf16 elements, no interleave, no swizzle, out-of-bounds elements read as zero.  rank <= 3.
cudaError_t encode_tensor_map_bf16(CUtensorMap* map, const void* base, int rank, const uint64_t* dims, const uint64_t* strides_bytes,
                                   const uint32_t* box);

// Device status word (bounded waits report here).
int* device_status_word();   // device pointer (allocated on first use), or nullptr on failure

int qlinear_launch(const void* Xq_idx, const float* Xq_norm, int n_tokens, const oq_codebook* cb_a,
                   const void* Wq_idx, const void* Wq_norm_bf16, int m, const oq_codebook* cb_w, int dim, void* Y,
                   int ldy, int y_dtype, int* status, void* stream);
// Rotate+quantize of activations with an explicit status word (NULL: the library's own, allocated on first use).
int rotate_quantize_act_launch(const void* X_bf16, int n_tokens, int dim, int ldx, const oq_rpbh* rot,
                               const oq_codebook* cb_a, void* Xq_idx, float* Xq_norm, float* dbg_rotated, int* status,
                               void* stream);
// Status word of the allocation-free entry point on the current device, or nullptr before its first call.
int* noalloc_status_word();

// Launch with programmatic stream serialisation: the kernel may be scheduled while the previous kernel of the stream
// is still running; it must execute griddepcontrol.wait before it touches anything that kernel reads or writes.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), int grid, int block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)grid);
  cfg.blockDim = dim3((unsigned)block);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, std::forward<Args>(args)...);
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace oq
