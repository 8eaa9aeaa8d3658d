// C-ABI entry points: handle, workspace planning, argument validation, and the launch
// sequence of one MoE layer (Section 3.1):
//   route (Eq. 1-3, 5; block counts and in-block ranks) -> permute-by-expert (scan, scatter)
//   -> [copy of the routed rows into expert order, small batches] -> GEMM-1 (+ row gather by
//   token, large batches) + SwiGLU -> GEMM-2 + combine (Eq. 4) -> finalize.
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#include "internal.h"

namespace fmmoe {

static bool desc_ok(const fmmoe_layer_desc* d) {
  if (!d) return false;
  if (d->hidden < 1 || d->n_experts < 1 || d->n_experts > FMMOE_MAX_EXPERTS || d->inter < 1) return false;
  if (d->n_shared < 0 || (d->n_shared > 0 && d->shared_inter < 1)) return false;
  if (d->top_k < 1 || d->top_k > FMMOE_MAX_TOPK || d->top_k > d->n_experts) return false;
  if (d->top_k_vis < 0 || d->top_k_vis > d->top_k) return false;
  if (d->top_k_vis == 0 && d->n_shared == 0) return false;   // p = 0 needs shared experts (Section 3.1)
  if (d->dtype != FMMOE_F32 && d->dtype != FMMOE_BF16) return false;
  if (d->weight_format != FMMOE_WEIGHTS_AS_DTYPE && d->weight_format != FMMOE_WEIGHTS_FP8_BLOCK128) return false;
  if (d->weight_format == FMMOE_WEIGHTS_FP8_BLOCK128 && d->dtype != FMMOE_BF16) return false;
  return true;
}

static fmmoe_status shape_supported(const fmmoe_layer_desc& d, bool forward) {
  const int elem = d.dtype == FMMOE_BF16 ? 2 : 4;
  if ((d.hidden * elem) % 16) return FMMOE_ERR_UNSUPPORTED;
  if (d.dtype == FMMOE_BF16) {
    if (d.hidden % 64) return FMMOE_ERR_UNSUPPORTED;
    if (forward && (d.inter % 64 || (d.n_shared && d.shared_inter % 64))) return FMMOE_ERR_UNSUPPORTED;
    if (forward && d.weight_format == FMMOE_WEIGHTS_FP8_BLOCK128 &&
        (d.hidden % 128 || d.inter % 128 || (d.n_shared && d.shared_inter % 128)))
      return FMMOE_ERR_UNSUPPORTED;
  } else if (forward && (d.hidden % 4 || d.inter % 4 || (d.n_shared && d.shared_inter % 4))) {
    return FMMOE_ERR_UNSUPPORTED;
  }
  return FMMOE_OK;
}

bool plan_workspace(const fmmoe_layer_desc& d, int64_t T, uint32_t flags, WsPlan* p) {
  if (T < 0) return false;
  const size_t elem = d.dtype == FMMOE_BF16 ? 2 : 4;
  const bool det = flags & FMMOE_FLAG_DETERMINISTIC;
  const int block_m = d.dtype == FMMOE_BF16 ? TC_BLOCK_M : F32_BLOCK_M;
  const size_t Tz = (size_t)T, K = d.top_k, H = d.hidden, I = d.inter;
  const size_t P = Tz * K;
  p->p_max = (int64_t)P;
  p->max_mtiles = (int32_t)(d.n_experts + P / block_m + 1);
  size_t o = 0;
  auto take = [&](size_t bytes) { const size_t at = o; o = align_up(o + bytes, 256); return at; };
  p->misc_off = take(8 * 4);
  {
    const size_t acc_bytes = Tz * H * 4;
    const size_t pair_bytes = d.dtype == FMMOE_BF16 ? (P + (size_t)d.n_shared * Tz) * H * 2 : 0;
    p->acc_off = take(det ? 0 : (acc_bytes > pair_bytes ? acc_bytes : pair_bytes));
  }
  p->blk_cnt_off = take((size_t)d.n_experts * ((Tz + 31) / 32 + 4) * 4);
  p->topk_idx_off = take(P * 4);
  p->topk_w_off = take(P * 4);
  p->inv_row_off = take(P * 4);
  p->expert_off_off = take((FMMOE_MAX_EXPERTS + 1) * 4);
  p->row_token_off = take(P * 4);
  p->row_gate_off = take(P * 4);
  p->mtiles_off = take((size_t)p->max_mtiles * sizeof(MTile));
  p->xp_off = take(d.dtype == FMMOE_BF16 ? P * H * elem : 0);
  p->act_off = take(P * I * elem);
  p->act_sh_off = take((size_t)d.n_shared * Tz * d.shared_inter * elem);
  p->y_off = take(det ? P * H * 4 : 0);
  p->ysh_off = take(det ? (size_t)d.n_shared * Tz * H * 4 : 0);
  p->total = o;
  return true;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

struct RoutePtrs {
  float* logits; float* probs; int32_t* topk_idx; float* topk_w; int32_t* inv_row;
  int32_t* expert_off; int32_t* row_token; float* row_gate; int32_t* blk_cnt; int32_t* misc; MTile* mtiles;
};

static RoutePtrs bind_route(const WsPlan& pl, char* ws, const fmmoe_route_out* out) {
  RoutePtrs r;
  r.logits = out ? out->logits : nullptr;
  r.probs = out ? out->probs : nullptr;
  r.topk_idx = (out && out->topk_idx) ? out->topk_idx : reinterpret_cast<int32_t*>(ws + pl.topk_idx_off);
  r.topk_w = (out && out->topk_w) ? out->topk_w : reinterpret_cast<float*>(ws + pl.topk_w_off);
  r.inv_row = (out && out->inv_row) ? out->inv_row : reinterpret_cast<int32_t*>(ws + pl.inv_row_off);
  r.expert_off = (out && out->expert_off) ? out->expert_off : reinterpret_cast<int32_t*>(ws + pl.expert_off_off);
  r.row_token = (out && out->row_token) ? out->row_token : reinterpret_cast<int32_t*>(ws + pl.row_token_off);
  r.row_gate = reinterpret_cast<float*>(ws + pl.row_gate_off);
  r.blk_cnt = reinterpret_cast<int32_t*>(ws + pl.blk_cnt_off);
  r.misc = reinterpret_cast<int32_t*>(ws + pl.misc_off);
  r.mtiles = reinterpret_cast<MTile*>(ws + pl.mtiles_off);
  return r;
}

static fmmoe_status check_common(fmmoe_handle* h, const fmmoe_layer_desc* d, const fmmoe_weights* w, const void* x,
                                 const uint8_t* is_visual, int64_t T, bool forward) {
  if (!h || !desc_ok(d) || !w || T < 0) return FMMOE_ERR_INVALID_ARG;
  if (T > (int64_t)0x7fffffff / d->top_k) return FMMOE_ERR_UNSUPPORTED;
  const fmmoe_status st = shape_supported(*d, forward);
  if (st != FMMOE_OK) return st;
  if (!w->router_w || !aligned16(w->router_w)) return FMMOE_ERR_INVALID_ARG;
  if (T > 0 && (!x || !is_visual || !aligned16(x))) return FMMOE_ERR_INVALID_ARG;
  if (forward) {
    if (!w->w_gate || !w->w_up || !w->w_down) return FMMOE_ERR_INVALID_ARG;
    if (!aligned16(w->w_gate) || !aligned16(w->w_up) || !aligned16(w->w_down)) return FMMOE_ERR_INVALID_ARG;
    if (d->n_shared) {
      if (!w->ws_gate || !w->ws_up || !w->ws_down) return FMMOE_ERR_INVALID_ARG;
      if (!aligned16(w->ws_gate) || !aligned16(w->ws_up) || !aligned16(w->ws_down)) return FMMOE_ERR_INVALID_ARG;
    }
    if (d->weight_format == FMMOE_WEIGHTS_FP8_BLOCK128) {
      if (!w->w_gate_scale || !w->w_up_scale || !w->w_down_scale) return FMMOE_ERR_INVALID_ARG;
      if (d->n_shared && (!w->ws_gate_scale || !w->ws_up_scale || !w->ws_down_scale)) return FMMOE_ERR_INVALID_ARG;
    }
  }
  return FMMOE_OK;
}

static fmmoe_status run_route(fmmoe_handle* h, const fmmoe_layer_desc& d, const fmmoe_weights& w, const void* x,
                              const uint8_t* is_visual, int64_t T, uint32_t flags, const RoutePtrs& r,
                              bool need_permute, float* acc_zero, cudaStream_t s, void* gather_xp = nullptr,
                              int block_m = 0) {
  RouteArgs ra;
  ra.x = x; ra.router_w = w.router_w; ra.router_b = w.router_b; ra.is_visual = is_visual;
  ra.T = T; ra.H = d.hidden; ra.E = d.n_experts; ra.K = d.top_k; ra.Kv = d.top_k_vis;
  ra.reduce_on = (flags & FMMOE_FLAG_REDUCE_ON) ? 1 : 0; ra.dtype = d.dtype;
  ra.logits = r.logits; ra.probs = r.probs; ra.topk_idx = r.topk_idx; ra.topk_w = r.topk_w;
  ra.inv_row = r.inv_row; ra.blk_cnt = r.blk_cnt; ra.acc_zero = acc_zero; ra.misc_zero = r.misc;
  fmmoe_status st = launch_route(h, ra, s);
  if (st != FMMOE_OK || !need_permute) return st;
  PermuteArgs pa;
  pa.topk_idx = r.topk_idx; pa.topk_w = r.topk_w; pa.blk_cnt = r.blk_cnt;
  pa.blk_tokens = route_block_tokens(d.dtype, T, d.hidden);
  pa.n_blk = route_num_blocks(d.dtype, T, d.hidden);
  pa.T = T; pa.K = d.top_k; pa.E = d.n_experts;
  pa.block_m = block_m ? block_m : (d.dtype == FMMOE_BF16 ? TC_BLOCK_M : F32_BLOCK_M);
  pa.expert_off = r.expert_off; pa.row_token = r.row_token; pa.row_gate = r.row_gate; pa.inv_row = r.inv_row;
  pa.mtiles = r.mtiles; pa.n_mtiles = r.misc;
  pa.gather_x = gather_xp ? x : nullptr; pa.gather_xp = gather_xp;
  pa.gather_row_bytes = d.hidden * (d.dtype == FMMOE_BF16 ? 2 : 4);
  return launch_permute(h, pa, s);
}

}  // namespace fmmoe

using namespace fmmoe;

extern "C" __attribute__((visibility("default"))) const char* fmmoe_status_string(fmmoe_status s) {
  switch (s) {
    case FMMOE_OK: return "ok";
    case FMMOE_ERR_INVALID_ARG: return "invalid argument";
    case FMMOE_ERR_UNSUPPORTED: return "unsupported shape or type";
    case FMMOE_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case FMMOE_ERR_CUDA: return "CUDA call failed";
    case FMMOE_ERR_TIMEOUT: return "device-side wait timed out";
    case FMMOE_ERR_INTERNAL: return "internal consistency check failed";
    case FMMOE_ERR_TOO_LARGE: return "problem exceeds the built-in scratch of the no-allocation entry point";
  }
  return "unknown status";
}

extern "C" __attribute__((visibility("default"))) fmmoe_status fmmoe_create(fmmoe_handle** out, int device) {
  if (!out) return FMMOE_ERR_INVALID_ARG;
  *out = nullptr;
  int n = 0;
  if (cudaGetDeviceCount(&n) != cudaSuccess || device < 0 || device >= n) return FMMOE_ERR_CUDA;
  FMMOE_CUDA_TRY(cudaSetDevice(device));
  cudaDeviceProp prop;
  FMMOE_CUDA_TRY(cudaGetDeviceProperties(&prop, device));
  if (prop.major != 10) return FMMOE_ERR_UNSUPPORTED;   // kernels are built for sm_100a only
  fmmoe_handle* h = new fmmoe_handle();
  h->device = device;
  h->sm_count = prop.multiProcessorCount;
  h->max_smem_optin = (int)prop.sharedMemPerBlockOptin;
  h->launches = 0;
  h->d_status = nullptr; h->h_status = nullptr; h->encode_tiled = nullptr;
  h->tc_attr_set = false; h->route_attr_set = false; h->route_f32_attr_mask = 0; h->profiling = false; h->prof_repeat = 1; h->ev_used = 0;
  h->gather_min_tokens = kGatherMinTokensDefault;
  if (const char* g = getenv("FMMOE_GATHER_MIN_TOKENS")) {
    char* end = nullptr;
    const long long v = strtoll(g, &end, 10);
    if (end != g && v >= 0) h->gather_min_tokens = v;
  }
  h->wait_budget_ns = 2000000000ull;
  h->sm_attr_set = false; h->smq_attr_set = false; h->tc2_attr_set = false;
  h->small_m_max_tokens = kSmallMMaxTokensDefault;
  if (const char* g = getenv("FMMOE_SMALL_M_MAX_TOKENS")) {
    char* end = nullptr;
    const long long v = strtoll(g, &end, 10);
    if (end != g && v >= 0) h->small_m_max_tokens = v;
  }
  h->test_withhold_stage = -1; h->test_budget_ns = 0;
  h->cta_pair_min_tokens = INT64_MAX;      // off unless asked for: measured no faster than the one-CTA form (power-capped)
  if (const char* g = getenv("FMMOE_CTA_PAIR_MIN_TOKENS")) {
    char* end = nullptr;
    const long long v = strtoll(g, &end, 10);
    if (end != g && v >= 0) h->cta_pair_min_tokens = v;
  }
  h->pair_min_tokens = kPairMinTokensDefault;
  if (const char* g = getenv("FMMOE_PAIR_ROWS_MIN_TOKENS")) {
    char* end = nullptr;
    const long long v = strtoll(g, &end, 10);
    if (end != g && v >= 0) h->pair_min_tokens = v;
  }
  h->pipe_ready = false; h->pipe_next = 0; h->ticket_next = 0; h->side_ready = false;
  { const char* dbg = getenv("FMMOE_DEBUG_SYNC"); h->debug_sync = dbg && dbg[0] == '1'; h->debug_seq = 0; }
  if (cudaMalloc(&h->d_status, 256) != cudaSuccess || cudaMemset(h->d_status, 0, 256) != cudaSuccess ||
      cudaMallocHost(&h->h_status, 256) != cudaSuccess) {
    if (h->d_status) cudaFree(h->d_status);
    delete h;
    return FMMOE_ERR_CUDA;
  }
  cudaDriverEntryPointQueryResult qres;
  void* fn = nullptr;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
      qres == cudaDriverEntryPointSuccess)
    h->encode_tiled = fn;
  if (prune_prepare(h) != FMMOE_OK) {
    cudaFree(h->d_status); cudaFreeHost(h->h_status);
    delete h;
    return FMMOE_ERR_CUDA;
  }
  *out = h;
  return FMMOE_OK;
}

extern "C" __attribute__((visibility("default"))) fmmoe_status fmmoe_destroy(fmmoe_handle* h) {
  if (!h) return FMMOE_OK;
  cudaSetDevice(h->device);
  if (h->d_status) cudaFree(h->d_status);
  if (h->h_status) cudaFreeHost(h->h_status);
  for (cudaEvent_t e : h->ev_pool) cudaEventDestroy(e);
  if (h->pipe_ready) {
    cudaStreamSynchronize(h->up_stream); cudaStreamSynchronize(h->down_stream);
    for (cudaEvent_t e : h->pipe_ev) cudaEventDestroy(e);
    for (cudaEvent_t e : h->ticket_ev) cudaEventDestroy(e);
    cudaStreamDestroy(h->up_stream); cudaStreamDestroy(h->down_stream);
  }
  if (h->side_ready) {
    cudaStreamSynchronize(h->side_stream);
    cudaEventDestroy(h->side_fork); cudaEventDestroy(h->side_join);
    cudaStreamDestroy(h->side_stream);
  }
  delete h;
  return FMMOE_OK;
}

extern "C" __attribute__((visibility("default"))) fmmoe_status fmmoe_get_status(fmmoe_handle* h, void* cuda_stream) {
  if (!h) return FMMOE_ERR_INVALID_ARG;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  FMMOE_CUDA_TRY(cudaMemcpyAsync(h->h_status, h->d_status, 4, cudaMemcpyDeviceToHost, s));
  FMMOE_CUDA_TRY(cudaMemsetAsync(h->d_status, 0, 4, s));
  FMMOE_CUDA_TRY(cudaStreamSynchronize(s));
  const int v = h->h_status[0];
  if (v == 0) return FMMOE_OK;
  return v == FMMOE_ERR_TIMEOUT ? FMMOE_ERR_TIMEOUT : FMMOE_ERR_INTERNAL;
}

extern "C" __attribute__((visibility("default"))) int64_t fmmoe_launch_count(const fmmoe_handle* h) { return h ? h->launches : -1; }

extern "C" __attribute__((visibility("default"))) size_t fmmoe_workspace_bytes(const fmmoe_layer_desc* d, int64_t n_tokens, uint32_t flags) {
  WsPlan p;
  if (!desc_ok(d) || !plan_workspace(*d, n_tokens, flags, &p)) return 0;
  return p.total + 256;
}

extern "C" __attribute__((visibility("default"))) fmmoe_status fmmoe_route(fmmoe_handle* h, const fmmoe_layer_desc* d, const fmmoe_weights* w, const void* x,
                                    const uint8_t* is_visual, int64_t T, uint32_t flags, const fmmoe_route_out* out,
                                    void* workspace, size_t workspace_bytes, void* cuda_stream) {
  fmmoe_status st = check_common(h, d, w, x, is_visual, T, false);
  if (st != FMMOE_OK) return st;
  WsPlan pl;
  plan_workspace(*d, T, flags, &pl);
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) || workspace_bytes < pl.total) return FMMOE_ERR_WORKSPACE;
  if (T == 0) return FMMOE_OK;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  char* ws = static_cast<char*>(workspace);
  const RoutePtrs r = bind_route(pl, ws, out);
  const bool need_permute = out && (out->expert_off || out->row_token || out->inv_row);
  return run_route(h, *d, *w, x, is_visual, T, flags, r, need_permute, nullptr, s);
}

// The layer.  `after_route` (may be NULL) is called once the router and the permutation have been
// enqueued: the routing record is then ordered on the stream, the expert GEMMs are not yet.
struct AfterRoute { fmmoe_status (*fn)(void*); void* ctx; };
static fmmoe_status forward_impl(fmmoe_handle* h, const fmmoe_layer_desc* d, const fmmoe_weights* w,
                                 const void* x, const uint8_t* is_visual, int64_t T, uint32_t flags, void* out,
                                 const fmmoe_route_out* route, void* workspace, size_t workspace_bytes,
                                 void* cuda_stream, const AfterRoute* after_route) {
  fmmoe_status st = check_common(h, d, w, x, is_visual, T, true);
  if (st != FMMOE_OK) return st;
  if (T > 0 && (!out || !aligned16(out) || out == x)) return FMMOE_ERR_INVALID_ARG;
  WsPlan pl;
  plan_workspace(*d, T, flags, &pl);
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) || workspace_bytes < pl.total) return FMMOE_ERR_WORKSPACE;
  if (T == 0) return FMMOE_OK;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  char* ws = static_cast<char*>(workspace);
  const bool det = flags & FMMOE_FLAG_DETERMINISTIC;
  const RoutePtrs r = bind_route(pl, ws, route);
  // the router clears the scheduler words and (atomic mode) the fp32 accumulator it owns rows of
  // bf16 at small batch: the permutation's scatter pass also writes the expert-grouped copy of x
  const bool pair = use_pair_rows(h, *d, T, flags);
  const bool cta_pairs = use_cta_pairs(h, *d, T);
  // an armed wait self-test runs on the small-M form whatever the size thresholds say
  const bool small_m = !cta_pairs && (use_small_m(h, *d, T) || (h->test_withhold_stage >= 0 && d->dtype == FMMOE_BF16));
  const bool copy_rows = d->dtype == FMMOE_BF16 && (cta_pairs || small_m || !gather_rows_in_gemm(h, T));
  st = run_route(h, *d, *w, x, is_visual, T, flags, r, true, (det || pair) ? nullptr : reinterpret_cast<float*>(ws + pl.acc_off), s,
                 copy_rows ? ws + pl.xp_off : nullptr, cta_pairs ? 2 * TC_BLOCK_M : 0);
  if (st != FMMOE_OK) return st;
  if (after_route) {
    st = after_route->fn(after_route->ctx);
    if (st != FMMOE_OK) return st;
  }

  FfnArgs fa = {};
  fa.d = d; fa.w = w; fa.x = x; fa.T = T; fa.p_max = pl.p_max;
  fa.mtiles = r.mtiles; fa.n_mtiles = r.misc; fa.max_mtiles = pl.max_mtiles;
  fa.tile_counters = r.misc + 1;
  fa.row_token = r.row_token; fa.row_gate = r.row_gate;
  fa.xp = ws + pl.xp_off; fa.act = ws + pl.act_off; fa.act_sh = ws + pl.act_sh_off;
  fa.acc = (det || pair) ? nullptr : reinterpret_cast<float*>(ws + pl.acc_off);
  fa.pair = pair ? 1 : 0;
  fa.yb = pair ? ws + pl.acc_off : nullptr;
  fa.ybsh = pair ? ws + pl.acc_off + (size_t)pl.p_max * d->hidden * 2 : nullptr;
  fa.y = det ? reinterpret_cast<float*>(ws + pl.y_off) : nullptr;
  fa.ysh = det ? reinterpret_cast<float*>(ws + pl.ysh_off) : nullptr;
  fa.deterministic = det; fa.d_status = h->d_status;
  fa.test_withhold_stage = -1; fa.grid_override = 0;
  if (cta_pairs) {
    st = launch_ffn_tc2(h, fa, s);
  } else if (small_m) {
    const uint64_t budget = h->wait_budget_ns;
    if (h->test_withhold_stage >= 0) {     // armed self-test: this call only
      fa.test_withhold_stage = h->test_withhold_stage; fa.grid_override = 1;
      h->wait_budget_ns = h->test_budget_ns;
      h->test_withhold_stage = -1;
    }
    st = launch_ffn_sm(h, fa, s);
    h->wait_budget_ns = budget;
  } else if (d->dtype == FMMOE_BF16) {
    fa.gather_in_gemm = gather_rows_in_gemm(h, T) ? 1 : 0;
    st = launch_ffn_tc(h, fa, s);
  } else {
    st = launch_ffn_f32(h, fa, s);
  }
  if (st != FMMOE_OK) return st;

  FinalizeArgs fin = {};
  fin.x = x; fin.out = out; fin.T = T; fin.H = d->hidden; fin.K = d->top_k; fin.n_shared = d->n_shared;
  fin.dtype = d->dtype; fin.add_residual = (flags & FMMOE_FLAG_RESIDUAL) ? 1 : 0; fin.deterministic = det;
  fin.acc = fa.acc; fin.y = fa.y; fin.ysh = fa.ysh; fin.inv_row = r.inv_row; fin.topk_w = r.topk_w;
  fin.pair = fa.pair; fin.yb = fa.yb; fin.ybsh = fa.ybsh;
  return launch_finalize(h, fin, s);
}

extern "C" __attribute__((visibility("default"))) fmmoe_status fmmoe_moe_forward(fmmoe_handle* h, const fmmoe_layer_desc* d, const fmmoe_weights* w,
                                          const void* x, const uint8_t* is_visual, int64_t T, uint32_t flags, void* out,
                                          const fmmoe_route_out* route, void* workspace, size_t workspace_bytes,
                                          void* cuda_stream) {
  return forward_impl(h, d, w, x, is_visual, T, flags, out, route, workspace, workspace_bytes, cuda_stream, nullptr);
}

// ---------------------------------------------------------------- layer + pruning stage in one call
namespace {
struct FusedPrune {
  fmmoe_handle* h; const fmmoe_prune_params* p; const float* probs; int32_t n_experts; const float* attn;
  const void* x; int32_t dtype, hidden; const uint8_t* is_visual; const int64_t* seq_off; const int64_t* n_vis;
  const int64_t* n_retain; int32_t n_seq; void* x_out; uint8_t* is_visual_out; int32_t* keep_idx; uint8_t* kind;
  int64_t* out_seq_off; void* ws; size_t ws_bytes; cudaStream_t s;
};
fmmoe_status fused_run(const FusedPrune& f, int phases, cudaStream_t s_select, cudaStream_t s_rows) {
  return prune_visual_phases(f.h, f.p, f.probs, f.n_experts, f.attn, f.x, f.dtype, f.hidden, f.is_visual, f.seq_off,
                             f.n_vis, f.n_retain, f.n_seq, f.x_out, f.is_visual_out, f.keep_idx, f.kind, f.out_seq_off,
                             f.ws, f.ws_bytes, phases, s_select, s_rows);
}
// after the router: the selection half of the pruning pass goes to the side stream
fmmoe_status fused_after_route(void* ctx) {
  const FusedPrune& f = *static_cast<const FusedPrune*>(ctx);
  FMMOE_CUDA_TRY(cudaEventRecord(f.h->side_fork, f.s));
  FMMOE_CUDA_TRY(cudaStreamWaitEvent(f.h->side_stream, f.h->side_fork, 0));
  const fmmoe_status st = fused_run(f, 1, f.h->side_stream, f.h->side_stream);
  if (st != FMMOE_OK) return st;
  FMMOE_CUDA_TRY(cudaEventRecord(f.h->side_join, f.h->side_stream));
  return FMMOE_OK;
}
}  // namespace

extern "C" __attribute__((visibility("default"))) fmmoe_status fmmoe_moe_forward_prune(
    fmmoe_handle* h, const fmmoe_layer_desc* d, const fmmoe_weights* w, const void* x, const uint8_t* is_visual,
    int64_t T, uint32_t flags, void* out, const fmmoe_route_out* route, const fmmoe_prune_params* p, const float* attn,
    const int64_t* seq_off, const int64_t* n_vis, const int64_t* n_retain, int32_t n_seq, void* x_out,
    uint8_t* is_visual_out, int32_t* keep_idx, uint8_t* kind, int64_t* out_seq_off, void* workspace,
    size_t workspace_bytes, void* cuda_stream) {
  if (!h || !desc_ok(d) || T < 0 || !route || !route->probs || !seq_off || n_seq < 0) return FMMOE_ERR_INVALID_ARG;
  if ((n_seq ? seq_off[n_seq] : 0) != T) return FMMOE_ERR_INVALID_ARG;
  const size_t layer_ws = fmmoe_workspace_bytes(d, T, flags);
  const size_t prune_ws = fmmoe_prune_workspace_bytes(T, n_seq);
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) || workspace_bytes < layer_ws + prune_ws) return FMMOE_ERR_WORKSPACE;
  if (!h->side_ready) {
    FMMOE_CUDA_TRY(cudaSetDevice(h->device));
    FMMOE_CUDA_TRY(cudaStreamCreateWithFlags(&h->side_stream, cudaStreamNonBlocking));
    FMMOE_CUDA_TRY(cudaEventCreateWithFlags(&h->side_fork, cudaEventDisableTiming));
    FMMOE_CUDA_TRY(cudaEventCreateWithFlags(&h->side_join, cudaEventDisableTiming));
    h->side_ready = true;
  }
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  char* ws = static_cast<char*>(workspace);
  FusedPrune f = {h, p, route->probs, d->n_experts, attn, out, d->dtype, d->hidden, is_visual, seq_off, n_vis, n_retain,
                  n_seq, x_out, is_visual_out, keep_idx, kind, out_seq_off, ws + align_up(layer_ws, 256),
                  workspace_bytes - align_up(layer_ws, 256), s};
  if (T == 0) return fused_run(f, 3, s, s);   // nothing to enqueue: validation and the output layout only
  // every argument check of the pruning pass happens before anything is enqueued
  {
    const fmmoe_status st = fused_run(f, 0, s, s);
    if (st != FMMOE_OK) return st;
  }
  const AfterRoute hook = {fused_after_route, &f};
  fmmoe_status st = forward_impl(h, d, w, x, is_visual, T, flags, out, route, ws, layer_ws, cuda_stream, &hook);
  if (st != FMMOE_OK) return st;
  FMMOE_CUDA_TRY(cudaStreamWaitEvent(s, h->side_join, 0));
  return fused_run(f, 2, s, s);
}

extern "C" __attribute__((visibility("default"))) size_t fmmoe_host_staging_bytes(const fmmoe_layer_desc* d, int64_t T) {
  if (!desc_ok(d) || T < 0) return 0;
  const size_t elem = d->dtype == FMMOE_BF16 ? 2 : 4;
  return 2 * align_up((size_t)T * d->hidden * elem, 256) + align_up((size_t)T, 256);
}

extern "C" __attribute__((visibility("default"))) fmmoe_status fmmoe_moe_forward_host(fmmoe_handle* h, const fmmoe_layer_desc* d, const fmmoe_weights* w,
                                               const void* x_host, const uint8_t* is_visual_host, int64_t T,
                                               uint32_t flags, void* out_host, const fmmoe_route_out* route,
                                               void* out_dev, uint8_t* is_visual_dev, void* workspace,
                                               size_t workspace_bytes, void* cuda_stream) {
  if (!h || !desc_ok(d) || T < 0) return FMMOE_ERR_INVALID_ARG;
  if (T > 0 && (!x_host || !is_visual_host || !out_host)) return FMMOE_ERR_INVALID_ARG;
  const size_t elem = d->dtype == FMMOE_BF16 ? 2 : 4;
  const size_t xb = (size_t)T * d->hidden * elem;
  const size_t stage = fmmoe_host_staging_bytes(d, T);
  const size_t inner = fmmoe_workspace_bytes(d, T, flags);
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) || workspace_bytes < stage + inner) return FMMOE_ERR_WORKSPACE;
  if (T == 0) return FMMOE_OK;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  char* ws = static_cast<char*>(workspace);
  char* dx = ws;
  char* dout = out_dev ? static_cast<char*>(out_dev) : ws + align_up(xb, 256);
  uint8_t* dvis = is_visual_dev ? is_visual_dev : reinterpret_cast<uint8_t*>(ws + 2 * align_up(xb, 256));
  FMMOE_CUDA_TRY(cudaMemcpyAsync(dx, x_host, xb, cudaMemcpyHostToDevice, s));
  FMMOE_CUDA_TRY(cudaMemcpyAsync(dvis, is_visual_host, (size_t)T, cudaMemcpyHostToDevice, s));
  const fmmoe_status st = fmmoe_moe_forward(h, d, w, dx, dvis, T, flags, dout, route, ws + stage, workspace_bytes - stage, s);
  if (st != FMMOE_OK) return st;
  FMMOE_CUDA_TRY(cudaMemcpyAsync(out_host, dout, xb, cudaMemcpyDeviceToHost, s));
  FMMOE_CUDA_TRY(cudaStreamSynchronize(s));
  return FMMOE_OK;
}

// ---------------------------------------------------------------- pipelined host I/O
// Copies run on two streams of the handle, one per direction, ordered against the caller's compute
// stream by events, so that the upload of one batch, the layer of the previous one and the download
// of the one before overlap.  Nothing here waits on the host except fmmoe_host_wait.
static fmmoe_status pipe_init(fmmoe_handle* h) {
  if (h->pipe_ready) return FMMOE_OK;
  FMMOE_CUDA_TRY(cudaSetDevice(h->device));
  FMMOE_CUDA_TRY(cudaStreamCreateWithFlags(&h->up_stream, cudaStreamNonBlocking));
  FMMOE_CUDA_TRY(cudaStreamCreateWithFlags(&h->down_stream, cudaStreamNonBlocking));
  for (cudaEvent_t& e : h->pipe_ev) FMMOE_CUDA_TRY(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
  for (cudaEvent_t& e : h->ticket_ev) FMMOE_CUDA_TRY(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
  h->pipe_ready = true;
  return FMMOE_OK;
}
static cudaEvent_t pipe_event(fmmoe_handle* h) { return h->pipe_ev[h->pipe_next++ % fmmoe_handle::kPipeEvents]; }

extern "C" __attribute__((visibility("default"))) fmmoe_status fmmoe_moe_forward_host_async(
    fmmoe_handle* h, const fmmoe_layer_desc* d, const fmmoe_weights* w, const void* x_host, const uint8_t* is_visual_host,
    int64_t T, uint32_t flags, void* out_host, const fmmoe_route_out* route, void* out_dev, uint8_t* is_visual_dev,
    void* workspace, size_t workspace_bytes, void* cuda_stream) {
  if (!h || !desc_ok(d) || T < 0) return FMMOE_ERR_INVALID_ARG;
  if (T > 0 && (!x_host || !is_visual_host)) return FMMOE_ERR_INVALID_ARG;
  const size_t elem = d->dtype == FMMOE_BF16 ? 2 : 4;
  const size_t xb = (size_t)T * d->hidden * elem;
  const size_t stage = fmmoe_host_staging_bytes(d, T);
  const size_t inner = fmmoe_workspace_bytes(d, T, flags);
  if (!workspace || (reinterpret_cast<uintptr_t>(workspace) & 255) || workspace_bytes < stage + inner) return FMMOE_ERR_WORKSPACE;
  if (T == 0) return FMMOE_OK;
  fmmoe_status st = pipe_init(h);
  if (st != FMMOE_OK) return st;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  char* ws = static_cast<char*>(workspace);
  char* dx = ws;
  char* dout = out_dev ? static_cast<char*>(out_dev) : ws + align_up(xb, 256);
  uint8_t* dvis = is_visual_dev ? is_visual_dev : reinterpret_cast<uint8_t*>(ws + 2 * align_up(xb, 256));
  const cudaEvent_t uploaded = pipe_event(h);
  FMMOE_CUDA_TRY(cudaMemcpyAsync(dx, x_host, xb, cudaMemcpyHostToDevice, h->up_stream));
  FMMOE_CUDA_TRY(cudaMemcpyAsync(dvis, is_visual_host, (size_t)T, cudaMemcpyHostToDevice, h->up_stream));
  FMMOE_CUDA_TRY(cudaEventRecord(uploaded, h->up_stream));
  FMMOE_CUDA_TRY(cudaStreamWaitEvent(s, uploaded, 0));
  st = fmmoe_moe_forward(h, d, w, dx, dvis, T, flags, dout, route, ws + stage, workspace_bytes - stage, s);
  if (st != FMMOE_OK) return st;
  if (out_host) {
    const cudaEvent_t computed = pipe_event(h);
    FMMOE_CUDA_TRY(cudaEventRecord(computed, s));
    FMMOE_CUDA_TRY(cudaStreamWaitEvent(h->down_stream, computed, 0));
    FMMOE_CUDA_TRY(cudaMemcpyAsync(out_host, dout, xb, cudaMemcpyDeviceToHost, h->down_stream));
  }
  return FMMOE_OK;
}

extern "C" __attribute__((visibility("default"))) fmmoe_status fmmoe_upload_async(fmmoe_handle* h, void* dst_dev, const void* src_host,
                                                                                   size_t bytes, void* cuda_stream) {
  if (!h || (bytes && (!dst_dev || !src_host))) return FMMOE_ERR_INVALID_ARG;
  if (bytes == 0) return FMMOE_OK;
  const fmmoe_status st = pipe_init(h);
  if (st != FMMOE_OK) return st;
  const cudaEvent_t uploaded = pipe_event(h);
  FMMOE_CUDA_TRY(cudaMemcpyAsync(dst_dev, src_host, bytes, cudaMemcpyHostToDevice, h->up_stream));
  FMMOE_CUDA_TRY(cudaEventRecord(uploaded, h->up_stream));
  FMMOE_CUDA_TRY(cudaStreamWaitEvent(static_cast<cudaStream_t>(cuda_stream), uploaded, 0));
  return FMMOE_OK;
}

extern "C" __attribute__((visibility("default"))) fmmoe_status fmmoe_download_async(fmmoe_handle* h, void* dst_host, const void* src_dev,
                                                                                     size_t bytes, void* cuda_stream) {
  if (!h || (bytes && (!dst_host || !src_dev))) return FMMOE_ERR_INVALID_ARG;
  if (bytes == 0) return FMMOE_OK;
  const fmmoe_status st = pipe_init(h);
  if (st != FMMOE_OK) return st;
  const cudaEvent_t produced = pipe_event(h);
  FMMOE_CUDA_TRY(cudaEventRecord(produced, static_cast<cudaStream_t>(cuda_stream)));
  FMMOE_CUDA_TRY(cudaStreamWaitEvent(h->down_stream, produced, 0));
  FMMOE_CUDA_TRY(cudaMemcpyAsync(dst_host, src_dev, bytes, cudaMemcpyDeviceToHost, h->down_stream));
  return FMMOE_OK;
}

extern "C" __attribute__((visibility("default"))) fmmoe_status fmmoe_host_fence(fmmoe_handle* h, uint64_t* ticket) {
  if (!h || !ticket) return FMMOE_ERR_INVALID_ARG;
  const fmmoe_status st = pipe_init(h);
  if (st != FMMOE_OK) return st;
  FMMOE_CUDA_TRY(cudaEventRecord(h->ticket_ev[h->ticket_next % fmmoe_handle::kTickets], h->down_stream));
  *ticket = h->ticket_next++;
  return FMMOE_OK;
}

extern "C" __attribute__((visibility("default"))) fmmoe_status fmmoe_host_wait(fmmoe_handle* h, uint64_t ticket) {
  if (!h || !h->pipe_ready || ticket >= h->ticket_next) return FMMOE_ERR_INVALID_ARG;
  // a slot that a later fence has reused completes after the ticket asked for: waiting on it is safe
  FMMOE_CUDA_TRY(cudaEventSynchronize(h->ticket_ev[ticket % fmmoe_handle::kTickets]));
  return FMMOE_OK;
}

extern "C" __attribute__((visibility("default"))) fmmoe_status fmmoe_profile_enable(fmmoe_handle* h, int enable) {
  if (!h) return FMMOE_ERR_INVALID_ARG;
  h->profiling = enable != 0;
  h->prof_repeat = enable > 1 ? enable : 1;
  return FMMOE_OK;
}

extern "C" __attribute__((visibility("default"))) fmmoe_status fmmoe_profile_reset(fmmoe_handle* h) {
  if (!h) return FMMOE_ERR_INVALID_ARG;
  FMMOE_CUDA_TRY(cudaDeviceSynchronize());
  h->prof.clear();
  h->ev_used = 0;
  return FMMOE_OK;
}

extern "C" __attribute__((visibility("default"))) fmmoe_status fmmoe_profile_read(fmmoe_handle* h, int kernel_id,
                                                                                  double* total_ms, int64_t* launches) {
  if (!h || kernel_id < 0 || kernel_id >= FMMOE_KERNEL_COUNT || !total_ms || !launches) return FMMOE_ERR_INVALID_ARG;
  FMMOE_CUDA_TRY(cudaDeviceSynchronize());
  double tot = 0.0;
  int64_t n = 0;
  for (const auto& r : h->prof) {
    if (r.id != kernel_id) continue;
    float ms = 0.f;
    FMMOE_CUDA_TRY(cudaEventElapsedTime(&ms, h->ev_pool[r.start], h->ev_pool[r.stop]));
    tot += ms / (r.reps > 0 ? r.reps : 1);
    ++n;
  }
  *total_ms = tot;
  *launches = n;
  return FMMOE_OK;
}

// Self-test of the bounded device-side waits: see include/fmmoe.h.
extern "C" __attribute__((visibility("default"))) fmmoe_status fmmoe_test_expire_wait(fmmoe_handle* h, uint64_t budget_ns,
                                                                                       int32_t k_block) {
  if (!h || k_block < 0 || budget_ns < 1000 || budget_ns > 1000000000ull) return FMMOE_ERR_INVALID_ARG;
  h->test_withhold_stage = k_block;
  h->test_budget_ns = budget_ns;
  return FMMOE_OK;
}
