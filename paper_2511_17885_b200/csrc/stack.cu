// A stack of MoE layers of one shape with residual adds (attention omitted), expert-activation
// reduction from layer l_v on (Section 3.1) and pruning stages after designated layers
// (Section 3.2; multi-stage schedule of Appendices A and D).  Host code only: it sequences the
// library's own entry points on one stream.  Every size is known on the host before anything
// runs (kept counts do not depend on the data), so the whole stack is enqueued without a
// single synchronisation.
//
// Layer l:   x_{l+1} = x_l + MoE_l(x_l)            vision tokens use K_v iff l >= reduce_from
// Stage at l: prune x_{l+1} with layer l's routing probabilities (computed on x_l); the shorter
//            sequence is the input of layer l+1.  A stage's retention is a fraction of the
//            ORIGINAL vision-token count of each sequence.
#include <math.h>
#include <string.h>

#include <vector>

#include "internal.h"

using namespace fmmoe;

namespace {

struct StackPlan {
  size_t xa, xb, probs, mask_a, mask_b, layer_ws, prune_ws, total;
  size_t layer_ws_bytes, prune_ws_bytes;
};

bool plan_stack(const fmmoe_layer_desc* d, int64_t T, int32_t n_seq, uint32_t flags, StackPlan* p) {
  const size_t elem = d->dtype == FMMOE_BF16 ? 2 : 4;
  const size_t lw = fmmoe_workspace_bytes(d, T, flags | FMMOE_FLAG_RESIDUAL);
  const size_t pw = fmmoe_prune_workspace_bytes(T, n_seq);
  if (lw == 0 || pw == 0) return false;
  size_t o = 0;
  auto take = [&](size_t bytes) { const size_t at = o; o = align_up(o + bytes, 256); return at; };
  p->xa = take((size_t)T * d->hidden * elem);
  p->xb = take((size_t)T * d->hidden * elem);
  p->probs = take((size_t)T * d->n_experts * 4);
  p->mask_a = take((size_t)T);
  p->mask_b = take((size_t)T);
  p->layer_ws = take(lw);
  p->prune_ws = take(pw);
  p->layer_ws_bytes = lw;
  p->prune_ws_bytes = pw;
  p->total = o;
  return true;
}

const fmmoe_stack_stage* stage_after(const fmmoe_stack_stage* st, int32_t n, int32_t layer) {
  for (int32_t i = 0; i < n; ++i)
    if (st[i].after_layer == layer) return &st[i];
  return nullptr;
}

// Sequence layout after every stage up to and including `upto_layer` (host arithmetic only).
bool stack_shapes(const fmmoe_stack_stage* st, int32_t n_stages, int32_t n_layers, const int64_t* seq_off,
                  const int64_t* n_vis, int32_t n_seq, std::vector<int64_t>* off, std::vector<int64_t>* vis) {
  off->assign(seq_off, seq_off + n_seq + 1);
  vis->assign(n_vis, n_vis + n_seq);
  for (int32_t l = 0; l < n_layers; ++l) {
    const fmmoe_stack_stage* s = stage_after(st, n_stages, l);
    if (!s) continue;
    std::vector<int64_t> noff(n_seq + 1, 0);
    for (int32_t b = 0; b < n_seq; ++b) {
      const int64_t L = (*off)[b + 1] - (*off)[b];
      const int64_t eta = (int64_t)floor((double)n_vis[b] * s->retain + 1e-9);
      const int64_t kept = fmmoe_prune_kept_count((*vis)[b], eta, &s->params, nullptr, nullptr);
      if (kept < 0) return false;
      noff[b + 1] = noff[b] + (L - (*vis)[b]) + kept;
      (*vis)[b] = kept;
    }
    *off = noff;
  }
  return true;
}

bool stages_ok(const fmmoe_stack_stage* st, int32_t n_stages, int32_t n_layers) {
  if (n_stages < 0 || (n_stages > 0 && !st)) return false;
  for (int32_t i = 0; i < n_stages; ++i) {
    if (st[i].after_layer < 0 || st[i].after_layer >= n_layers) return false;
    if (!(st[i].retain >= 0.0 && st[i].retain <= 1.0)) return false;
    for (int32_t j = 0; j < i; ++j)
      if (st[j].after_layer == st[i].after_layer) return false;
  }
  return true;
}

}  // namespace

extern "C" __attribute__((visibility("default"))) size_t fmmoe_stack_workspace_bytes(const fmmoe_layer_desc* d, int64_t n_tokens,
                                                                                     int32_t n_seq, uint32_t flags) {
  StackPlan p;
  if (!d || n_tokens < 0 || n_seq < 0 || !plan_stack(d, n_tokens, n_seq, flags, &p)) return 0;
  return p.total + 256;
}

extern "C" __attribute__((visibility("default"))) fmmoe_status fmmoe_stack_output_layout(
    const fmmoe_stack_stage* stages, int32_t n_stages, int32_t n_layers, const int64_t* seq_off, const int64_t* n_vis,
    int32_t n_seq, int64_t* out_seq_off, int64_t* out_n_vis) {
  if (!seq_off || !n_vis || !out_seq_off || n_seq < 0 || n_layers < 0 || !stages_ok(stages, n_stages, n_layers))
    return FMMOE_ERR_INVALID_ARG;
  std::vector<int64_t> off, vis;
  if (!stack_shapes(stages, n_stages, n_layers, seq_off, n_vis, n_seq, &off, &vis)) return FMMOE_ERR_INVALID_ARG;
  memcpy(out_seq_off, off.data(), sizeof(int64_t) * (n_seq + 1));
  if (out_n_vis) memcpy(out_n_vis, vis.data(), sizeof(int64_t) * n_seq);
  return FMMOE_OK;
}

extern "C" __attribute__((visibility("default"))) fmmoe_status fmmoe_stack_forward(
    fmmoe_handle* h, const fmmoe_layer_desc* d, const fmmoe_weights* layer_w, int32_t n_layers, int32_t reduce_from,
    const fmmoe_stack_stage* stages, int32_t n_stages, const void* x, const uint8_t* is_visual, const int64_t* seq_off,
    const int64_t* n_vis, int32_t n_seq, uint32_t flags, void* x_out, uint8_t* is_visual_out, int64_t* out_seq_off,
    void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!h || !d || !layer_w || n_layers < 1 || !seq_off || !n_vis || n_seq < 1 || !out_seq_off) return FMMOE_ERR_INVALID_ARG;
  if (!stages_ok(stages, n_stages, n_layers)) return FMMOE_ERR_INVALID_ARG;
  if (seq_off[0] != 0) return FMMOE_ERR_INVALID_ARG;
  const int64_t T0 = seq_off[n_seq];
  if (T0 < 0) return FMMOE_ERR_INVALID_ARG;
  for (int32_t b = 0; b < n_seq; ++b)
    if (n_vis[b] < 0 || n_vis[b] > seq_off[b + 1] - seq_off[b]) return FMMOE_ERR_INVALID_ARG;
  const uint32_t base_flags = (flags & FMMOE_FLAG_DETERMINISTIC) | FMMOE_FLAG_RESIDUAL;
  StackPlan pl;
  if (!plan_stack(d, T0, n_seq, base_flags, &pl)) return FMMOE_ERR_INVALID_ARG;
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) || workspace_bytes < pl.total) return FMMOE_ERR_WORKSPACE;
  if (T0 > 0 && (!x || !is_visual || !x_out)) return FMMOE_ERR_INVALID_ARG;
  char* ws = static_cast<char*>(workspace);
  std::vector<int64_t> off(seq_off, seq_off + n_seq + 1), vis(n_vis, n_vis + n_seq), eta(n_seq), noff(n_seq + 1);
  // exactly one activation tensor and one mask are live at any time, so "the buffer that is not
  // the live one" is always free
  void* bufs[2] = {ws + pl.xa, ws + pl.xb};
  uint8_t* masks[2] = {reinterpret_cast<uint8_t*>(ws + pl.mask_a), reinterpret_cast<uint8_t*>(ws + pl.mask_b)};
  auto free_buf = [&](const void* live) -> void* { return live == bufs[0] ? bufs[1] : bufs[0]; };
  auto free_mask = [&](const uint8_t* live) -> uint8_t* { return live == masks[0] ? masks[1] : masks[0]; };
  const void* cur_x = x;
  const uint8_t* cur_mask = is_visual;
  float* probs = reinterpret_cast<float*>(ws + pl.probs);

  for (int32_t l = 0; l < n_layers; ++l) {
    const int64_t T = off[n_seq];
    const fmmoe_stack_stage* s = stage_after(stages, n_stages, l);
    const bool last = l == n_layers - 1;
    const uint32_t lf = base_flags | (l >= reduce_from ? FMMOE_FLAG_REDUCE_ON : 0u);
    fmmoe_route_out ro;
    memset(&ro, 0, sizeof(ro));
    ro.probs = s ? probs : nullptr;
    // the layer writes straight into the caller's buffer when nothing follows it
    void* layer_out = (last && !s) ? x_out : free_buf(cur_x);
    fmmoe_status st;
    if (!s) {
      st = fmmoe_moe_forward(h, d, &layer_w[l], cur_x, cur_mask, T, lf, layer_out, &ro, ws + pl.layer_ws,
                             pl.layer_ws_bytes, cuda_stream);
      if (st != FMMOE_OK) return st;
      cur_x = layer_out;
    } else {
      // A pruning layer: the layer and its stage as the single call, whose scoring and selection kernels run
      // beside the expert GEMMs instead of after them.  Three activation tensors are involved (the layer's
      // input, its output, the pruned rows) and the workspace has two buffers: the pruned rows take the place
      // of the layer's input, which nothing reads after the layer's last kernel.  That needs the input to be
      // one of this workspace's buffers, i.e. any layer but the first (the caller's x is never written).
      for (int32_t b = 0; b < n_seq; ++b) eta[b] = (int64_t)floor((double)n_vis[b] * s->retain + 1e-9);
      const bool in_place_ok = cur_x != x;      // the layer's input is dead once GEMM-1 and the router have read it
      void* pruned = last ? x_out : (in_place_ok ? const_cast<void*>(cur_x) : nullptr);
      uint8_t* pmask = (last && is_visual_out) ? is_visual_out : free_mask(cur_mask);
      if (pruned) {
        st = fmmoe_moe_forward_prune(h, d, &layer_w[l], cur_x, cur_mask, T, lf, layer_out, &ro, &s->params, s->attn,
                                     off.data(), vis.data(), eta.data(), n_seq, pruned, pmask, nullptr, nullptr,
                                     noff.data(), ws + pl.layer_ws, pl.layer_ws_bytes + pl.prune_ws_bytes, cuda_stream);
        if (st != FMMOE_OK) return st;
        cur_x = layer_out;
      } else {
        // stage right after the first layer: no third buffer is free, so the two calls in sequence
        st = fmmoe_moe_forward(h, d, &layer_w[l], cur_x, cur_mask, T, lf, layer_out, &ro, ws + pl.layer_ws,
                               pl.layer_ws_bytes, cuda_stream);
        if (st != FMMOE_OK) return st;
        cur_x = layer_out;
        pruned = free_buf(cur_x);
        st = fmmoe_prune_visual(h, &s->params, probs, d->n_experts, s->attn, cur_x, d->dtype, d->hidden, cur_mask,
                                off.data(), vis.data(), eta.data(), n_seq, pruned, pmask, nullptr, nullptr, noff.data(),
                                ws + pl.prune_ws, pl.prune_ws_bytes, cuda_stream);
        if (st != FMMOE_OK) return st;
      }
      for (int32_t b = 0; b < n_seq; ++b) {
        const int64_t n_text = (off[b + 1] - off[b]) - vis[b];
        vis[b] = (noff[b + 1] - noff[b]) - n_text;
      }
      off = noff;
      cur_x = pruned;
      cur_mask = pmask;
    }
  }
  memcpy(out_seq_off, off.data(), sizeof(int64_t) * (n_seq + 1));
  // the final modality mask: copy it out unless the last stage already wrote it there
  if (is_visual_out && cur_mask != is_visual_out && off[n_seq] > 0)
    FMMOE_CUDA_TRY(cudaMemcpyAsync(is_visual_out, cur_mask, (size_t)off[n_seq], cudaMemcpyDeviceToDevice,
                                   static_cast<cudaStream_t>(cuda_stream)));
  return FMMOE_OK;
}
