/*
 * liboq -- B200 (sm_100a) runtime hot path of an OrbitQuant quantized linear layer.
 *
 * One quantized linear layer y = W x (paper Eq. 1) is computed as
 *
 *     offline   Pi_d  <- RPBH(d)                       oq_make_rpbh        (Eq. 9, Algorithm 1 "Offline")
 *               C^(d,b) <- LloydMax(d, b)              oq_build_codebook   (Eq. 2-3, Sec. 4.5)
 *               W^' <- diag(r') Q_bw(rows of W Pi^T)   oq_quantize_weights (Eq. 4-6)
 *     online    x^' <- s Q_ba(Pi x / (s + eps))        oq_rotate_quantize_act (Eq. 7-8, Algorithm 1 "Online")
 *               y   <- W^' x^'                         oq_qlinear          (Sec. 4.3: the rotation cancels)
 *
 * Conventions
 *   - Plain C ABI.  Every call returns an OQ_* status; oq_last_error() gives a message for the last
 *     failure on the calling thread.  Nothing throws across the boundary.
 *   - "dev" pointers are CUDA device pointers on the current device, owned by the caller (for example a
 *     PyTorch tensor's data_ptr()).  "host" pointers are ordinary host memory.  The library allocates
 *     only the small tables that belong to an oq_rpbh handle (permutation and signs, < 128 KB, uploaded on
 *     first use on the device that is current at that moment and freed by oq_rpbh_destroy).
 *   - `stream` is a cudaStream_t passed as void* (NULL = default stream).  Kernel launches are
 *     asynchronous on that stream; argument validation happens on the host before any launch.
 *   - Matrices are row-major.  X is [n_tokens][ldx] bf16, W is [m][ldw] bf16 (the layout of a linear
 *     layer's weight, W in R^{m x d}); ld* are in elements.
 *   - Quantized operands are PACKED: `bits` bits per coordinate on the wire, in a layout private to the
 *     library (oq_packed_bytes gives the sizes; oq_unpack_indices recovers the logical level indices,
 *     numbered 0 .. 2^bits-1 in ascending order of the level, in rotated-coordinate order).
 *   - There is no CPU fallback: a call that needs the GPU fails with OQ_ERR_CUDA if no device is usable.
 *   - Threads: handles may be shared between host threads (first-use uploads are serialised inside the library);
 *     oq_last_error() is per thread; oq_debug_select_rq_kernel and oq_debug_select_gemm_kernel are process-wide test
 *     switches and not thread-safe.
 */
#ifndef OQ_H_
#define OQ_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  OQ_OK = 0,
  OQ_ERR_INVALID_ARG = 1,    /* null pointer, non-positive size, mismatching handles */
  OQ_ERR_UNSUPPORTED = 2,    /* dim / block / bits outside what the kernels implement */
  OQ_ERR_ALIGNMENT = 3,      /* pointer not 16-byte aligned or leading dimension not a multiple of 8 */
  OQ_ERR_CUDA = 4,           /* a CUDA runtime call failed (message holds the CUDA error string) */
  OQ_ERR_DEVICE_TIMEOUT = 5, /* a bounded device-side wait gave up (see oq_device_status) */
  OQ_ERR_NOMEM = 6           /* workspace too small / allocation failed */
};

enum { OQ_BF16 = 0, OQ_F32 = 1 }; /* output element type of oq_qlinear */

typedef struct oq_codebook oq_codebook; /* Lloyd-Max codebook C^(d,b): host tables only */
typedef struct oq_rpbh oq_rpbh;         /* RPBH rotation Pi_d: permutation + signs (host, and device on first use) */

/* ---- offline constructors (host arithmetic in fp64; usable without a GPU) ------------------------- */

/* Lloyd-Max codebook of 2^bits levels for the coordinate marginal f_dim of a random unit vector
 * (Eq. 2: f_d(t) ~ (1 - t^2)^((d-3)/2) on [-1,1]; Eq. 3: nearest-level map).  The exact f_dim is used,
 * not its Gaussian approximation.  dim >= 16, bits in 1..4 or 6 (6: activations only, see
 * oq_rotate_quantize_act_levels; takes a few seconds).  *out is owned by the caller
 * (oq_codebook_destroy).  Errors: OQ_ERR_INVALID_ARG, OQ_ERR_UNSUPPORTED. */
int oq_build_codebook(int dim, int bits, oq_codebook** out);

/* Copies the tables out (any pointer may be NULL): centroids[2^bits] ascending (fp64),
 * boundaries[2^bits-1] = midpoints of adjacent levels (fp64), boundaries_f32 = those rounded once to
 * fp32, centroids_bf16 = levels rounded fp64 -> fp32 -> bf16 (the values the GEMM decodes to). */
int oq_codebook_get(const oq_codebook* cb, double* centroids, double* boundaries,
                    float* boundaries_f32, uint16_t* centroids_bf16);
/* Test helper: the polynomial the quantization kernels evaluate instead of a boundary search.  For
 * x = min(|t| / *clamp, 1) and y = 2x - *centre, floor(P(y)) with
 * P(y) - 1/2 = *mid + coef[1] y + ... + coef[*degree] y^(*degree) is the number of positive boundaries
 * below |t| (Eq. 3 restricted to one half of the antisymmetric codebook).  coef has 8 entries.
 * Returns OQ_ERR_UNSUPPORTED when no monotone polynomial was found (the kernels then search boundaries). */
int oq_codebook_level_poly(const oq_codebook* cb, float* coef, float* clamp, float* centre, float* mid,
                           int* degree);
int oq_codebook_dim(const oq_codebook* cb);
int oq_codebook_bits(const oq_codebook* cb);
void oq_codebook_destroy(oq_codebook* cb);

/* Randomized permuted block-Hadamard rotation Pi_d = blkdiag(H_h D_1, ..., H_h D_{d/h}) P_pi (Eq. 9):
 * uniform permutation pi (applied first, as a gather: (P x)_k = x[pi(k)]), Rademacher signs indexed by
 * the position after the permutation, Sylvester-ordered Walsh-Hadamard blocks scaled by 1/sqrt(h).
 * The draw is deterministic in (dim, block, seed): SplitMix64 with initial state
 * seed ^ (dim << 32) ^ block, Fisher-Yates from the top with rejection sampling, then one 64-bit word
 * per 64 signs (bit set = -1).  block: power of two, divides dim; dim < 65536. */
int oq_make_rpbh(int dim, int block, uint64_t seed, oq_rpbh** out);
/* perm[dim] (int32) and signs[dim] (int8, +1 / -1); either may be NULL. */
int oq_rpbh_get(const oq_rpbh* r, int32_t* perm, int8_t* signs);
int oq_rpbh_dim(const oq_rpbh* r);
int oq_rpbh_block(const oq_rpbh* r);
void oq_rpbh_destroy(oq_rpbh* r);

/* ---- sizes -------------------------------------------------------------------------------------------- */

/* Bytes of the packed index matrix of `rows` rows of `dim` coordinates at `bits` bits each, and the
 * pitch of one row (a multiple of 16 bytes).  dim must be a multiple of 128; bits in {2,3,4}. */
int oq_packed_bytes(int rows, int dim, int bits, size_t* idx_bytes, size_t* row_pitch_bytes);

/* ---- GPU entry points ---------------------------------------------------------------------------------- */

/* Online activation quantization, one fused pass per token (Eq. 7-8, Algorithm 1 lines "Online"):
 * x' = Pi x, s = ||x'||_2, idx_k = level of C^(d,b_a) nearest to x'_k / (s + 1e-10).
 *   X_bf16     dev  [n_tokens][ldx] bf16, read only
 *   Xq_idx     dev  packed indices, oq_packed_bytes(n_tokens, dim, bits) bytes, written
 *   Xq_norm    dev  [n_tokens] fp32, s per token, written
 *   dbg_rotated dev [n_tokens][dim] fp32 or NULL; when given, receives x' (test hook; slows the kernel)
 * s is accumulated in fp32: by the tensor-core kernel (every benchmark width) from the rotated row, as Eq. 8 writes
 * it; by the register-butterfly and general kernels from the raw row, which is the same number because Pi is
 * orthogonal.  A coordinate that is exactly on a boundary goes to the lower level (Eq. 3 is silent on ties), so a zero
 * token gives s = 0 and the lower middle level (2^(bits-1) - 1) everywhere.  n_tokens may be 0 (no launch).
 * Requires dim == rpbh dim == codebook dim, dim % 128 == 0, ldx >= dim, ldx % 8 == 0, 16-byte aligned
 * pointers.  Errors: INVALID_ARG, UNSUPPORTED, ALIGNMENT, CUDA. */
int oq_rotate_quantize_act(const void* X_bf16, int n_tokens, int dim, int ldx, const oq_rpbh* rot,
                           const oq_codebook* cb_a, void* Xq_idx, float* Xq_norm, float* dbg_rotated,
                           void* stream);

/* Offline weight quantization, run on the GPU (Eq. 4-6): the same pass applied to the m rows of W
 * (row i of W Pi^T is Pi w_i); the row norm r'_i is stored in bf16 (Sec. 4.2).
 *   W_bf16 dev [m][ldw] bf16; Wq_idx dev packed (oq_packed_bytes(m, dim, bits)); Wq_norm_bf16 dev [m] bf16.
 * The GEMM tiles weights in groups of 128 rows; rows beyond m need not exist (they are never read). */
int oq_quantize_weights(const void* W_bf16, int m, int dim, int ldw, const oq_rpbh* rot,
                        const oq_codebook* cb_w, void* Wq_idx, void* Wq_norm_bf16, void* dbg_rotated,
                        void* stream);

/* Quantized linear layer on packed operands (the product W^' x^' of Sec. 4.3 with Eq. 6 and Eq. 8):
 *   Y[n][i] = s_n * r'_i * sum_k C_a[idxA[n][k]] * C_w[idxW[i][k]]
 * Levels are decoded to bf16 on the SM (weights into shared memory, activations into tensor or shared memory, see
 * oq_debug_select_gemm_kernel), contracted on the tensor cores with fp32 accumulation,
 * and both norms are applied in the epilogue (acc * s_n * r'_i, two fp32 multiplies in that order, then
 * one rounding when Y is bf16).
 *   Xq_idx, Xq_norm  dev  as written by oq_rotate_quantize_act with cb_a
 *   Wq_idx, Wq_norm_bf16 dev as written by oq_quantize_weights with cb_w
 *   Y dev [n_tokens][ldy] of y_dtype (OQ_BF16 or OQ_F32), written; ldy >= m, ldy % 8 == 0
 * Requires the two codebooks to have the same dim (= dim), dim % 128 == 0, m % 8 == 0.
 * n_tokens == 0 or m == 0 launches nothing.  Errors: INVALID_ARG, UNSUPPORTED, ALIGNMENT, CUDA. */
int oq_qlinear(const void* Xq_idx, const float* Xq_norm, int n_tokens, const oq_codebook* cb_a,
               const void* Wq_idx, const void* Wq_norm_bf16, int m, const oq_codebook* cb_w, int dim,
               void* Y, int ldy, int y_dtype, void* stream);

/* Whole online layer from HOST memory (Algorithm 1 "Online" followed by the product of Sec. 4.3):
 * copies X (host, bf16 [n_tokens][dim], dense; pinned memory makes the copy asynchronous) to the device,
 * runs oq_rotate_quantize_act and oq_qlinear, and copies Y (bf16 [n_tokens][m], dense) back to
 * Y_host_bf16, all on `stream`.  Wq_idx / Wq_norm_bf16 are device buffers from oq_quantize_weights.
 * `workspace` is a caller-owned device buffer of at least oq_forward_workspace_bytes() bytes (16-byte
 * aligned); it holds X, the packed activations, the norms and Y while the call is in flight.
 * The call returns after enqueueing; synchronise the stream before reading Y_host_bf16.
 * Errors: as the two calls it wraps, OQ_ERR_NOMEM when the workspace is too small.  With a 6-bit activation codebook
 * the two calls are oq_rotate_quantize_act_levels and oq_qlinear_levels (bits_a = 6 in the size query). */
int oq_forward_workspace_bytes(int n_tokens, int dim, int m, int bits_a, size_t* bytes);
int oq_linear_forward_host(const void* X_host_bf16, int n_tokens, int dim, const oq_rpbh* rot,
                           const oq_codebook* cb_a, const void* Wq_idx, const void* Wq_norm_bf16, int m,
                           const oq_codebook* cb_w, void* Y_host_bf16, void* workspace,
                           size_t workspace_bytes, void* stream);

/* Whole online layer on DEVICE buffers without any allocation.  The paper has no counterpart: this is a
 * variant of the layer call for callers that cannot obtain device memory when they need the layer
 * evaluated -- a serving loop confined to a memory budget fixed at start-up, a thread that must not block on
 * the allocator, a process whose memory pool is already frozen.  It runs oq_rotate_quantize_act and then
 * oq_qlinear; the packed activations, their norms and the status word that bounded device-side waits
 * report to are kept in a scratch array that is compiled into the library (about 8.1 MiB of device memory
 * on every GPU that loads the library, held until the process exits).  The call performs no cudaMalloc /
 * cudaFree and calls no allocating library routine.
 *   X_bf16 dev [n_tokens][ldx] bf16;  Wq_idx / Wq_norm_bf16 dev, from oq_quantize_weights;
 *   Y dev [n_tokens][ldy] of y_dtype, written.  Arguments as for the two calls it wraps.
 * Limits: n_tokens <= 32768 and oq_packed_bytes(n_tokens, dim, bits_a) <= 8 MiB, otherwise OQ_ERR_NOMEM
 * with a message that states both sizes.  `rot` must already have been used by an ordinary GPU call
 * (oq_quantize_weights does that), because creating its device tables allocates; otherwise
 * OQ_ERR_INVALID_ARG.
 * The first call on a device looks up the scratch array's device address (cudaGetSymbolAddress, which may load
 * the module): make that first call before starting any stream capture.
 * All calls on a device share the one scratch array, which keeps the previous call's contents: two calls
 * whose kernels may overlap on the GPU (different streams) race on it -- serialise them.  Nothing in the
 * scratch needs clearing between calls (every byte that is read was written by the same call); the status
 * word is sticky until oq_device_status reads it, and while it is set every kernel that reports to it gives up
 * its waits at once, so outputs produced after a time-out are invalid until oq_device_status has been called. */
int oq_linear_forward_noalloc(const void* X_bf16, int n_tokens, int dim, int ldx, const oq_rpbh* rot,
                              const oq_codebook* cb_a, const void* Wq_idx, const void* Wq_norm_bf16, int m,
                              const oq_codebook* cb_w, void* Y, int ldy, int y_dtype, void* stream);

/* ---- the linear layers of one transformer block ---------------------------------------------------------- */

/* The method is applied token-wise to every linear layer of a block (Sec. 3.1), and the layers that share an input
 * dimension share the rotation Pi_d and the activation codebook (Sec. 4.2).  The layers that read the SAME tensor -- the
 * Q, K and V projections of an attention block -- therefore consume the same quantized activations: one
 * rotate+quantize pass (Eq. 7-8) feeds all of them.  oq_block_forward runs the layers of a block in the order given, on
 * one stream, back to back (every kernel is launched with programmatic stream serialisation, so a kernel's set-up
 * overlaps the tail of the one before it); an input is rotated and quantized once, right before the first layer that reads
 * it.  Because everything is ordered on the stream, the Y of a layer may be the X of a later input.
 *   oq_block_input   X_bf16 dev [n_tokens][ldx] bf16; rot / cb_a for its dim; Xq dev scratch owned by the caller:
 *                    oq_packed_bytes(n_tokens, dim, bits) bytes, or n_tokens * dim * 2 bytes when cb_a has 6 bits (the
 *                    bf16 level matrix); Xq_norm dev [n_tokens] fp32.  Both hold the quantized input after the call.
 *   oq_block_layer   input = index into `inputs`; Wq_idx / Wq_norm_bf16 / cb_w from oq_quantize_weights with the input's
 *                    rotation; Y dev [n_tokens][ldy] of y_dtype.
 * All arguments are validated before the first launch.  n_tokens == 0 or n_layers == 0 launches nothing.
 * Errors: as oq_rotate_quantize_act and oq_qlinear (the message names the input or layer). */
typedef struct {
  const void* X_bf16;
  int ldx, dim;
  const oq_rpbh* rot;
  const oq_codebook* cb_a;
  void* Xq;
  float* Xq_norm;
} oq_block_input;
typedef struct {
  int input, m;
  const void* Wq_idx;
  const void* Wq_norm_bf16;
  const oq_codebook* cb_w;
  void* Y;
  int ldy, y_dtype;
} oq_block_layer;
int oq_block_forward(int n_tokens, const oq_block_input* inputs, int n_inputs, const oq_block_layer* layers, int n_layers,
                     void* stream);

/* Test helper: expand packed indices to one byte per coordinate, out dev [rows][dim] uint8, logical level
 * numbers in rotated-coordinate order. */
int oq_unpack_indices(const void* idx, int rows, int dim, int bits, uint8_t* out, void* stream);

/* Synchronises the device and reports (then clears) the device-side status words (the library's own and the one of
 * oq_linear_forward_noalloc): 0 when every bounded wait inside the kernels completed, otherwise a code saying which
 * wait gave up (the first non-zero word; both are cleared).  After a time-out the kernels that report to the same
 * word cut their waits short until this call has cleared it, so treat every output produced since the previous
 * clean status as invalid.  Returns OQ_OK or OQ_ERR_DEVICE_TIMEOUT (with *status set), OQ_ERR_CUDA. */
int oq_device_status(int* status);

/* ---- activations as bf16 levels ("decode once") ----------------------------------------------------- */

/* An activation tile is used by every column tile of the output, so oq_qlinear decodes the same packed indices
 * once per column tile.  These two calls decode them once per layer instead: oq_decode_levels writes
 * out[row][k] = bf16(C[idx[row][k]]) (the level of Eq. 3, not yet multiplied by the norm) for a packed operand
 * (device, rows x dim, the layout oq_rotate_quantize_act / oq_quantize_weights wrote) into out_bf16 (device,
 * [rows][ldo], ldo >= dim, ldo % 8 == 0, 16-byte aligned); oq_qlinear_levels is oq_qlinear with that matrix as the
 * activation operand (fetched by TMA) and all decoding warps on the weights.  Same bf16 operands, same order of
 * accumulation: Y is bit-identical to oq_qlinear's.  dim % 128 == 0, m % 8 == 0, weight bits 2..4; other
 * arguments, asynchrony and errors as for oq_qlinear. */
int oq_decode_levels(const void* idx, int rows, int dim, const oq_codebook* cb, void* out_bf16, int ldo, void* stream);
int oq_qlinear_levels(const void* Xd_bf16, int ldxd, const float* Xq_norm, int n_tokens, const void* Wq_idx,
                      const void* Wq_norm_bf16, int m, const oq_codebook* cb_w, int dim, void* Y, int ldy, int y_dtype,
                      void* stream);

/* 6-bit activations (the W4A6 setting of the video models, Sec. 5.1): 64 levels do not fit the byte-permute decode
 * of oq_qlinear, so the rotate+quantize pass writes the levels themselves: Xd_bf16[n][k] = bf16(C_a[idx[n][k]])
 * (device, [n_tokens][ldxd], ldxd >= dim, ldxd % 8 == 0, 16-byte aligned), the operand of oq_qlinear_levels, and
 * Xq_norm[n] = s (fp32) as oq_rotate_quantize_act does.  cb_a must have 6 bits (oq_build_codebook(dim, 6)); the
 * nearest level is found on a uniform grid of 256 cells over the normalised magnitude, each holding at most one
 * boundary (same rule as Eq. 3 with ties to the lower index).  idx_u8: optional device [n_tokens][dim] bytes that
 * receive the level indices 0..63 (16-byte aligned; NULL to skip); dbg_rotated as in oq_rotate_quantize_act.
 * Hadamard blocks of 64..4096.  Errors as for oq_rotate_quantize_act. */
int oq_rotate_quantize_act_levels(const void* X_bf16, int n_tokens, int dim, int ldx, const oq_rpbh* rot,
                                  const oq_codebook* cb_a, void* Xd_bf16, int ldxd, float* Xq_norm, void* idx_u8,
                                  float* dbg_rotated, void* stream);

/* ---- AdaLN modulation projections (weight-only INT4, bf16 activations) ----------------------------- */

/* The AdaLN modulation projections are not rotated: their weights are quantized to INT4 by round-to-nearest in
 * groups of 64 input coordinates and their input, one conditioning token per sample, stays in bf16 (the
 * supplementary section on quantized layers; Sec. 5.1).  The grid, on which the paper is silent, is symmetric:
 * scale = bf16(max |w| / 7) per (row, group), q = clamp(rint(w / scale), -8, 7), q = 0 where the scale is 0
 * (divisions in fp32).  Bytes of the two device buffers for an m x dim weight: *wq_bytes = m * dim / 2,
 * *scale_bytes = 2 * m * dim / 64.  m must be a multiple of 16, dim of 64 (OQ_ERR_UNSUPPORTED otherwise). */
int oq_adaln_packed_bytes(int m, int dim, size_t* wq_bytes, size_t* scale_bytes);

/* Offline, on the GPU: W_bf16 (device, row-major [m][ldw], ldw >= dim, ldw % 8 == 0, 16-byte aligned) ->
 * Wq (device, wq_bytes, 16-byte aligned; layout private to the library: the order in which the tensor-core
 * fragments of oq_adaln_linear consume the nibbles) and scales (device, scale_bytes, 16-byte aligned).
 * Asynchronous on `stream`.  Errors: OQ_ERR_INVALID_ARG, OQ_ERR_UNSUPPORTED, OQ_ERR_ALIGNMENT, OQ_ERR_CUDA. */
int oq_adaln_quantize_weights(const void* W_bf16, int m, int dim, int ldw, void* Wq, void* scales, void* stream);

/* Y[n][row] = sum over groups of scale * sum_i q_i * X[n][i]  (products of a group accumulated in fp32 on the
 * tensor cores, groups added in fp32 in a fixed order: results are bit-reproducible).  X_bf16: device,
 * [n_tokens][ldx], ldx >= dim, ldx % 8 == 0, 16-byte aligned.  Y: device, [n_tokens][ldy], ldy >= m, OQ_BF16 or
 * OQ_F32.  One pass over the weights per 8 tokens (the layer sees one token per sample).  The tokens of a pass are
 * staged in shared memory: min(n_tokens, 8) * (2 * dim + 16) bytes + 8 KB must fit in 227 KB (dim <= 13952 for 8).
 * Asynchronous on `stream`; nothing is allocated.  Errors as above. */
int oq_adaln_linear(const void* X_bf16, int n_tokens, int ldx, const void* Wq, const void* scales, int m, int dim,
                    void* Y, int ldy, int y_dtype, void* stream);

/* Test helper: logical values of the private layout.  q_int8: device int8 [m][dim] (-8..7); scale_bf16: device
 * bf16 bit patterns [m][dim / 64]. */
int oq_adaln_unpack(const void* Wq, const void* scales, int m, int dim, void* q_int8, void* scale_bf16, void* stream);

/* Self-test of the bounded device-side waits the GEMM pipeline is built on: launches one thread that waits
 * about a millisecond on a barrier nobody arrives at.  The wait gives up by itself (the kernel ends
 * normally, nothing hangs or traps) and records code 9; the following oq_device_status() must return
 * OQ_ERR_DEVICE_TIMEOUT with *status == 9 and leave the word clear again. */
int oq_selftest_bounded_wait(void* stream);

/* Host-only query (no device needed): which kernel oq_rotate_quantize_act / oq_quantize_weights would launch for
 * this rotation and codebook, and its shape: *kernel = 1 general, 2 register butterflies, 3 tensor cores with a
 * row-per-thread gather, 4 tensor cores with a token-slab gather (only when selected);
 * *rows_per_group = rows one CTA holds in shared memory at a time (1 for the general kernel; the tokens of a slab for
 * kernel 4); *tiles_per_group = 128-row tensor-core tiles per group (0 for kernels 1 and 2, 1 for kernel 4);
 * *smem_bytes = dynamic shared memory per CTA.  Any output pointer may be NULL.  Honours oq_debug_select_rq_kernel.
 * Returns OQ_OK, OQ_ERR_INVALID_ARG (NULL handle, dims differ) or OQ_ERR_UNSUPPORTED (dim not a multiple of 128). */
int oq_rq_plan(const oq_rpbh* rot, const oq_codebook* cb, int* kernel, int* rows_per_group, int* tiles_per_group,
               size_t* smem_bytes);

/* Test helper: selects the kernel behind oq_rotate_quantize_act / oq_quantize_weights for the following calls of
 * this process: 0 = choose by shape (default), 1 = general kernel (any block size; butterflies in shared memory),
 * 2 = register-butterfly kernel (blocks of 64, 128, 256), 3 = tensor-core kernel (blocks of 64 to 4096; the block
 * Hadamard transform of Eq. 7 as a product with a 128 x 128 matrix of +-1, plus butterfly stages for larger blocks;
 * every thread gathers the coordinates of one row), 4 = token-slab tensor-core kernel (blocks of 64, 128, 256, rows of
 * 1024 coordinates and more: the rows of 8, 4 or 2 tokens are transposed so that one shared-memory access moves a
 * coordinate of all of them, and the row norms come from a Gram product on the tensor cores; never chosen by shape,
 * it measured slower).  A selected kernel that does not support the shape falls back.  All of them compute the same
 * function; the parity tests run each of them.  Not thread-safe.  Returns OQ_OK or OQ_ERR_INVALID_ARG. */
int oq_debug_select_rq_kernel(int which);

/* Test helper: selects the kernel behind oq_qlinear (and the calls built on it) for the following calls of this
 * process: 0 = choose by output type (default: kernel 2 for bf16 output, kernel 1 for fp32 output), 1 = both operands
 * decoded into shared memory, two accumulators in tensor memory (the epilogue of a tile overlaps the next tile),
 * 2 = the activation operand decoded into tensor memory (tcgen05.st; tcgen05.mma takes A from there), one accumulator,
 * the output tile staged in shared memory; bf16 output only, fp32 output falls back to kernel 1; 3 = kernel 2 with the
 * tile order it otherwise uses only for large inputs (bands of 8 column tiles, chosen by the library when the packed
 * activations exceed 32 MB).  All of them compute the same sums in the same order: their outputs are bit-identical
 * (Sec. 4.3, Eq. 6, Eq. 8).  oq_qlinear_levels always
 * runs the shared-memory kernel.  Not thread-safe.  Returns OQ_OK or OQ_ERR_INVALID_ARG. */
int oq_debug_select_gemm_kernel(int which);

const char* oq_last_error(void);
const char* oq_version(void);

#ifdef __cplusplus
}
#endif
#endif /* OQ_H_ */
