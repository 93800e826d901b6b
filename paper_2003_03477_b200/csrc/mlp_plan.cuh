// Host-side description of one replica's MLP: layer list, flat parameter layout, workspace layout.
#pragma once
#include "common.cuh"

namespace ss {

constexpr int kMaxLayers = 16;

struct LayerInfo {
  int in, out;
  int64_t w_off, b_off;   // element offsets into the flat parameter vector (multiples of 32)
  bool relu;              // ReLU after the Linear (all but the last top layer)
};

struct MlpPlan {
  int nl, nb;             // layers in total, bottom layers
  int n_dense, D0, W;     // dense features, bottom output width, concat width
  bool bf16;
  LayerInfo layer[kMaxLayers];
  int64_t P;              // padded parameter count
  // workspace byte offsets; act[l] = output of layer l ([B,out]), dact[l] = gradient of the loss with
  // respect to it after the ReLU mask.  The last bottom layer's output lives in the concat buffer and
  // the last top layer's in logit[], so act[] is unused for those two.
  size_t act[kMaxLayers], dact[kMaxLayers];
  // bits[l]: one bit per element of layer l's output, "positive" (the ReLU-gradient mask of the backward pass),
  // rows of ld_bits[l] 32-bit words (a multiple of 4); bf16 mode only
  size_t bits[kMaxLayers];
  int ld_bits[kMaxLayers];
  size_t grads, red_partial, gpart, loss_part, ctrl, total;   // loss_part: a ticket word, then one partial loss per 8 samples
  int ctrl_rows;          // most rows of a product that another product of a tensor-core flow may wait for
  size_t ctrl_bytes;      // control words of the tensor-core flows (directly behind the loss ticket: one memset clears both)
  int k_splits[kMaxLayers];      // K slices of the weight-gradient GEMM of each layer (1 = none)
  int64_t gpart_off[kMaxLayers]; // float offset of the layer's slice buffer inside the gpart region
  int red_splits;         // batch slices of the two-stage reductions (bias and skinny weight gradients)
};

inline int64_t pad32(int64_t x) { return (x + 31) & ~(int64_t)31; }

// Returns SS_OK and fills `p` (workspace offsets for batch B; pass B = 0 when only the layout is wanted).
inline ss_status make_mlp_plan(const ss_mlp_desc* d, int B, MlpPlan* p) {
  if (!d || !d->bottom_dims || !d->top_dims) return SS_ERR_NULL;
  if (d->n_bottom < 1 || d->n_top < 1 || d->n_bottom + d->n_top > kMaxLayers || B < 0) return SS_ERR_SHAPE;
  if (d->gemm_dtype != 0 && d->gemm_dtype != 1) return SS_ERR_DTYPE;
  p->nb = d->n_bottom;
  p->nl = d->n_bottom + d->n_top;
  p->bf16 = d->gemm_dtype == 1;
  p->n_dense = d->bottom_dims[0];
  p->D0 = d->bottom_dims[d->n_bottom];
  p->W = d->top_dims[0];
  if (d->top_dims[d->n_top] != 1 || p->W < p->D0 || (p->W & 7) || (p->D0 & 7)) return SS_ERR_SHAPE;
  int64_t off = 0;
  for (int l = 0; l < p->nl; ++l) {
    const int* dims = l < p->nb ? d->bottom_dims + l : d->top_dims + (l - p->nb);
    LayerInfo& L = p->layer[l];
    L.in = dims[0];
    L.out = dims[1];
    if (L.in < 1 || L.out < 1 || L.in > (1 << 20) || L.out > (1 << 20)) return SS_ERR_SHAPE;
    // hidden widths feed 128-bit accesses: multiples of 8 (the first input and the logit are exempt)
    if (l != p->nl - 1 && (L.out & 7)) return SS_ERR_SHAPE;
    L.relu = l != p->nl - 1;
    L.w_off = off; off += pad32((int64_t)L.in * L.out);
    L.b_off = off; off += pad32(L.out);
  }
  p->P = off;
  const size_t es = p->bf16 ? 2 : 4;
  size_t o = 0;
  auto take = [&](size_t bytes) { size_t r = o; o += (bytes + 255) & ~(size_t)255; return r; };
  for (int l = 0; l < p->nl; ++l) {
    const size_t bytes = (size_t)B * p->layer[l].out * es;
    p->act[l] = take(bytes);
    p->dact[l] = take(bytes);
    p->ld_bits[l] = ((p->layer[l].out + 31) / 32 + 3) & ~3;
    p->bits[l] = take(p->bf16 ? (size_t)B * p->ld_bits[l] * 4 : 0);
  }
  p->grads = take((size_t)p->P * 4);
  p->red_splits = B >= 1024 ? (B + 127) / 128 : (B >= 256 ? 8 : (B >= 64 ? 2 : 1));   // at most 128-row slices
  size_t red_total = 0;
  for (int l = 0; l < p->nl; ++l) red_total += (size_t)p->layer[l].out;
  red_total += (size_t)p->layer[p->nl - 1].in;
  if (p->layer[0].in <= 16) red_total += (size_t)p->layer[0].in * p->layer[0].out;
  p->red_partial = take(red_total * 4 * (size_t)p->red_splits);
  // Weight-gradient GEMMs contract over the batch (K = B: dozens of k steps per tile) and have small outputs: few,
  // long tiles.  They are part of the backward flow, where they are what the tail of the launch waits for, so K is cut
  // into slices until their tiles are about as many as the SMs (slices of at least 8 k steps); the update kernel adds
  // the slices in order.
  int64_t gp = 0;
  const int nk = (B + 63) / 64;
  auto sliced = [&](int l) {
    const LayerInfo& L = p->layer[l];
    return p->bf16 && l != p->nl - 1 && !(l == 0 && L.in <= 16) && B >= 16;
  };
  int64_t all_tiles = 0;
  for (int l = 0; l < p->nl; ++l)
    if (sliced(l)) all_tiles += (int64_t)((p->layer[l].out + 127) / 128) * ((p->layer[l].in + 127) / 128);
  for (int l = 0; l < p->nl; ++l) {
    const LayerInfo& L = p->layer[l];
    int s = 1;
    if (sliced(l)) {
      s = (int)((148 + all_tiles / 2) / all_tiles);
      if (s > 8) s = 8;
      if (s > nk / 8) s = nk / 8;                          // slices of at least 8 k-steps: a tile's fixed cost outweighs shorter ones
      if (s > nk) s = nk;
      if (s < 1) s = 1;
    }
    p->k_splits[l] = s;
    p->gpart_off[l] = gp;
    if (s > 1) gp += (int64_t)s * L.in * L.out;
  }
  p->gpart = take((size_t)gp * 4);
  p->loss_part = take(((size_t)(B + 7) / 8 + 4) * 4);
  int widest = B;
  for (int l = 0; l < p->nl; ++l) widest = p->layer[l].out > widest ? p->layer[l].out : widest;
  p->ctrl_rows = widest;
  p->ctrl_bytes = (2 + (size_t)12 * (size_t)((widest + 127) / 128 + 1)) * 4;
  p->ctrl = take(p->ctrl_bytes);
  p->total = o;
  return SS_OK;
}

}  // namespace ss
