// The linear layers of one transformer block on one stream: every distinct input tensor is rotated and quantized once
// and feeds all the layers that read it (Sec. 4.2: the layers that share an input dimension share Pi_d and the
// codebook, so the Q, K and V projections consume the same quantized activations).
#include <vector>

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

extern "C" int oq_block_forward(int n_tokens, const oq_block_input* inputs, int n_inputs, const oq_block_layer* layers,
                                int n_layers, void* stream) {
  if (n_tokens < 0 || n_inputs < 0 || n_layers < 0) return fail(OQ_ERR_INVALID_ARG, "oq_block_forward: negative count");
  if (n_layers == 0 || n_tokens == 0) return OQ_OK;
  if (!inputs || !layers) return fail(OQ_ERR_INVALID_ARG, "oq_block_forward: NULL inputs or layers");
  // everything is validated before the first launch, so that a bad layer does not leave half a block enqueued
  for (int i = 0; i < n_inputs; ++i) {
    const oq_block_input& in = inputs[i];
    if (!in.rot || !in.cb_a) return fail(OQ_ERR_INVALID_ARG, "oq_block_forward: input " + std::to_string(i) + ": NULL handle");
    if (in.dim <= 0 || in.rot->dim != in.dim || in.cb_a->dim != in.dim)
      return fail(OQ_ERR_INVALID_ARG, "oq_block_forward: input " + std::to_string(i) + ": dim differs from the rotation's or the codebook's");
    if (in.dim % 128) return fail(OQ_ERR_UNSUPPORTED, "oq_block_forward: input " + std::to_string(i) + ": dim must be a multiple of 128");
    const int b = in.cb_a->bits;
    if (!(b == 2 || b == 3 || b == 4 || b == 6))
      return fail(OQ_ERR_UNSUPPORTED, "oq_block_forward: input " + std::to_string(i) + ": activation bits must be 2, 3, 4 or 6");
    if (!in.X_bf16 || !in.Xq || !in.Xq_norm) return fail(OQ_ERR_INVALID_ARG, "oq_block_forward: input " + std::to_string(i) + ": NULL buffer");
    if (in.ldx < in.dim) return fail(OQ_ERR_INVALID_ARG, "oq_block_forward: input " + std::to_string(i) + ": ldx smaller than dim");
    if (in.ldx % 8 || !aligned16(in.X_bf16) || !aligned16(in.Xq))
      return fail(OQ_ERR_ALIGNMENT, "oq_block_forward: input " + std::to_string(i) + ": pointers must be 16-byte aligned and ldx a multiple of 8");
  }
  for (int l = 0; l < n_layers; ++l) {
    const oq_block_layer& ly = layers[l];
    if (ly.input < 0 || ly.input >= n_inputs) return fail(OQ_ERR_INVALID_ARG, "oq_block_forward: layer " + std::to_string(l) + ": input index out of range");
    if (!ly.cb_w || !ly.Wq_idx || !ly.Wq_norm_bf16 || !ly.Y) return fail(OQ_ERR_INVALID_ARG, "oq_block_forward: layer " + std::to_string(l) + ": NULL handle or buffer");
    if (ly.cb_w->dim != inputs[ly.input].dim) return fail(OQ_ERR_INVALID_ARG, "oq_block_forward: layer " + std::to_string(l) + ": weight codebook of another dim than its input");
    if (ly.cb_w->bits < 2 || ly.cb_w->bits > 4) return fail(OQ_ERR_UNSUPPORTED, "oq_block_forward: layer " + std::to_string(l) + ": weight bits must be 2, 3 or 4");
    if (ly.m <= 0 || ly.m % 8) return fail(OQ_ERR_UNSUPPORTED, "oq_block_forward: layer " + std::to_string(l) + ": m must be a positive multiple of 8");
    if (ly.ldy < ly.m || ly.ldy % 8) return fail(OQ_ERR_ALIGNMENT, "oq_block_forward: layer " + std::to_string(l) + ": ldy must be a multiple of 8, at least m");
    if (ly.y_dtype != OQ_BF16 && ly.y_dtype != OQ_F32) return fail(OQ_ERR_INVALID_ARG, "oq_block_forward: layer " + std::to_string(l) + ": bad y_dtype");
    if (!aligned16(ly.Wq_idx) || !aligned16(ly.Y)) return fail(OQ_ERR_ALIGNMENT, "oq_block_forward: layer " + std::to_string(l) + ": pointers must be 16-byte aligned");
  }
  // Layers run in the order given; an input is rotated and quantized right before the first layer that reads it (so a
  // layer's output may be a later layer's input tensor: everything is ordered on the one stream).
  std::vector<char> done(n_inputs, 0);
  for (int l = 0; l < n_layers; ++l) {
    const oq_block_layer& ly = layers[l];
    const oq_block_input& in = inputs[ly.input];
    const bool levels = in.cb_a->bits == 6;      // 64 levels: the hand-over is the bf16 level matrix [n_tokens][dim]
    if (!done[ly.input]) {
      const int rc = levels ? rotate_quantize_levels_launch(in.X_bf16, n_tokens, in.dim, in.ldx, in.rot, in.cb_a, in.Xq, in.dim,
                                                            in.Xq_norm, nullptr, nullptr, nullptr, stream)
                            : rotate_quantize_act_launch(in.X_bf16, n_tokens, in.dim, in.ldx, in.rot, in.cb_a, in.Xq, in.Xq_norm,
                                                         nullptr, nullptr, stream);
      if (rc != OQ_OK) return rc;
      done[ly.input] = 1;
    }
    const int rc = levels ? qlinear_levels_launch(in.Xq, in.dim, in.Xq_norm, n_tokens, ly.Wq_idx, ly.Wq_norm_bf16, ly.m, ly.cb_w,
                                                  in.dim, ly.Y, ly.ldy, ly.y_dtype, nullptr, stream)
                          : qlinear_launch(in.Xq, in.Xq_norm, n_tokens, in.cb_a, ly.Wq_idx, ly.Wq_norm_bf16, ly.m, ly.cb_w, in.dim,
                                           ly.Y, ly.ldy, ly.y_dtype, nullptr, stream);
    if (rc != OQ_OK) return rc;
  }
  return OQ_OK;
}
