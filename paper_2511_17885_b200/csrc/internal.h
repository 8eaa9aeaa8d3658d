// Internal declarations shared by the library's translation units (host side).
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>
#include <stdio.h>

#include <utility>
#include <vector>

#include "../../include/fmmoe.h"

struct fmmoe_handle {
  int device;
  int sm_count;
  int max_smem_optin;
  int* d_status;        // device status word (0 = ok)
  int* h_status;        // pinned host mirror
  int64_t launches;     // kernels launched through this handle
  void* encode_tiled;   // cuTensorMapEncodeTiled entry point
  bool tc_attr_set;     // dynamic shared memory opt-in done for the tensor-core kernels
  bool route_attr_set;  // ... for the bf16 router
  bool sm_attr_set;     // ... for the small-M form of the expert GEMMs
  bool smq_attr_set;    // ... and its FP8 weight stream
  bool tc2_attr_set;    // ... for the CTA-pair form
  int64_t cta_pair_min_tokens;    // from this many tokens on the expert GEMMs run on CTA pairs (cta_group::2)
  int64_t small_m_max_tokens;     // below this many tokens the expert GEMMs run in their small-M form
  int64_t pair_min_tokens;        // from this many tokens on the combine goes through per-pair bf16 rows (no atomics)
  int test_withhold_stage;        // self-test (fmmoe_test_expire_wait): armed for the next layer call, else -1
  uint64_t test_budget_ns;
  uint32_t route_f32_attr_mask;   // ... for the fp32 router instantiations (bit = logits per lane)
  int64_t gather_min_tokens;      // from this many tokens on GEMM-1 gathers the routed rows of x itself
  uint64_t wait_budget_ns;        // time budget of every bounded device-side wait
  // optional kernel timeline
  bool profiling;
  int prof_repeat;      // timeline on: launches of a short idempotent kernel issued back to back inside one event pair
  bool debug_sync;      // FMMOE_DEBUG_SYNC=1: synchronise after every kernel and report the first CUDA error on stderr
  int64_t debug_seq;    // kernels launched so far in debug mode
  std::vector<cudaEvent_t> ev_pool;
  size_t ev_used;
  struct ProfRec { int id; size_t start, stop; int reps; };
  std::vector<ProfRec> prof;
  // pipelined host I/O (created on first use): one stream per copy direction, a ring of events that
  // order them against the caller's compute stream, and a ring of events behind the host tickets
  static constexpr int kPipeEvents = 32, kTickets = 64;
  bool pipe_ready;
  cudaStream_t up_stream, down_stream;
  cudaEvent_t pipe_ev[kPipeEvents];
  uint64_t pipe_next;
  cudaEvent_t ticket_ev[kTickets];
  uint64_t ticket_next;
  // fmmoe_moe_forward_prune: the selection half of the pruning pass runs beside the expert GEMMs
  bool side_ready;
  cudaStream_t side_stream;
  cudaEvent_t side_fork, side_join;
};

namespace fmmoe {

// Device-side status codes written to the status word (first writer wins).
enum : int { DEV_OK = 0, DEV_TIMEOUT = FMMOE_ERR_TIMEOUT, DEV_INTERNAL = FMMOE_ERR_INTERNAL };

constexpr int TC_BLOCK_M = 128;   // token rows per tile on the tensor-core path
constexpr int F32_BLOCK_M = 32;   // token rows per tile on the fp32 FMA path

// One M-tile of the expert-grouped row space.
struct MTile {
  int32_t group;  // expert id
  int32_t row0;   // first row (in the grouped order)
  int32_t rows;   // valid rows in this tile (1..block_m)
  int32_t pad;    // 1 if this is the only tile of its expert
};

static inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Workspace layout of fmmoe_route / fmmoe_moe_forward (byte offsets).
struct WsPlan {
  size_t blk_cnt_off;           // int32 [E][ceil(T/32)] per-block expert counts / offsets (not cleared)
  size_t misc_off;              // int32 [8]: [0] number of routed M-tiles, [1],[2] GEMM tile counters
  size_t acc_off;               // fp32 [T,H] combine accumulator (atomic mode); the same region holds the bf16
                                // per-pair outputs [P_max + N_s*T, H] in pair-row mode (sized for the larger)
  size_t topk_idx_off, topk_w_off, inv_row_off;
  size_t expert_off_off, row_token_off, row_gate_off, mtiles_off;
  size_t xp_off;                // dtype [P_max,H] rows gathered by expert (bf16 path)
  size_t act_off;               // dtype [P_max,I] SwiGLU activations
  size_t act_sh_off;            // dtype [N_s*T,I_s]
  size_t y_off;                 // fp32 [P_max,H]    (deterministic mode)
  size_t ysh_off;               // fp32 [N_s*T,H]    (deterministic mode)
  size_t total;
  int64_t p_max;
  int32_t max_mtiles;
};
bool plan_workspace(const fmmoe_layer_desc& d, int64_t T, uint32_t flags, WsPlan* p);

// Brackets one kernel launch with events when the handle's timeline is on.
// Kernels that give the same result when run twice in a row on the same arguments: with the timeline's repeat
// count above 1 their launch is issued that many times inside the event pair (`reps`), so that the launch
// latency an event pair adds to a 10-30 us kernel is amortised.  The scan / scatter pass works in place and
// the GEMMs consume a tile counter, so they always run once.
static inline bool prof_idempotent(int id) {
  return id == FMMOE_KERNEL_ROUTE || id == FMMOE_KERNEL_FINALIZE || id == FMMOE_KERNEL_PRUNE_INDEX ||
         id == FMMOE_KERNEL_PRUNE_SCORE || id == FMMOE_KERNEL_PRUNE_SELECT || id == FMMOE_KERNEL_PRUNE_COMPACT;
}
struct ProfScope {
  fmmoe_handle* h; cudaStream_t s; size_t rec; bool on; int kid; int reps;
  ProfScope(fmmoe_handle* h_, int id, cudaStream_t s_) : h(h_), s(s_), rec(0), on(h_->profiling), kid(id), reps(1) {
    if (!on) return;
    if (h->prof_repeat > 1 && prof_idempotent(id)) reps = h->prof_repeat;
    while (h->ev_pool.size() < h->ev_used + 2) {
      cudaEvent_t e;
      if (cudaEventCreate(&e) != cudaSuccess) { on = false; return; }
      h->ev_pool.push_back(e);
    }
    fmmoe_handle::ProfRec r{id, h->ev_used, h->ev_used + 1, reps};
    h->ev_used += 2;
    h->prof.push_back(r);
    rec = h->prof.size() - 1;
    cudaEventRecord(h->ev_pool[r.start], s);
  }
  ~ProfScope() {
    if (on) cudaEventRecord(h->ev_pool[h->prof[rec].stop], s);
    if (h->debug_sync) {
      ++h->debug_seq;
      cudaError_t e = cudaStreamSynchronize(s);
      if (e == cudaSuccess) e = cudaGetLastError();
      if (e != cudaSuccess) {
        fprintf(stderr, "fmmoe: kernel class %d (launch scope #%lld) failed: %s\n", kid, (long long)h->debug_seq, cudaGetErrorString(e));
        h->debug_sync = false;   // report the first failure only
      }
    }
  }
};

#define FMMOE_CUDA_TRY(expr)                         \
  do {                                               \
    cudaError_t _e = (expr);                         \
    if (_e != cudaSuccess) return FMMOE_ERR_CUDA;    \
  } while (0)

// Launch with programmatic dependent launch allowed (the kernel calls pdl_wait() before it touches
// data of earlier kernels), optionally as clusters of `cluster_x` CTAs.
template <typename... KArgs, typename... Args>
static inline cudaError_t launch_ex(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                                    unsigned cluster_x, bool pdl, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = s;
  cudaLaunchAttribute attr[2];
  int n = 0;
  if (pdl) {
    attr[n].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[n].val.programmaticStreamSerializationAllowed = 1;
    ++n;
  }
  if (cluster_x > 1) {
    attr[n].id = cudaLaunchAttributeClusterDimension;
    attr[n].val.clusterDim.x = cluster_x; attr[n].val.clusterDim.y = 1; attr[n].val.clusterDim.z = 1;
    ++n;
  }
  cfg.attrs = attr; cfg.numAttrs = n;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
template <typename... KArgs, typename... Args>
static inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s,
                                     unsigned cluster_x, Args&&... args) {
  return launch_ex(kernel, grid, block, smem, s, cluster_x, true, std::forward<Args>(args)...);
}

// ---- launchers (each returns after enqueueing; *launches is incremented per kernel) ----
struct RouteArgs {
  const void* x; const void* router_w; const float* router_b; const uint8_t* is_visual;
  int64_t T; int H, E, K, Kv; int reduce_on; int dtype;
  float* logits; float* probs; int32_t* topk_idx; float* topk_w; int32_t* inv_row;
  int32_t* blk_cnt;   // [E][n_blk]: per token block (route_block_tokens) and expert, the number of selections
  float* acc_zero;    // [T,H] fp32 combine accumulator to clear (each CTA its own tokens' rows), or NULL
  int32_t* misc_zero; // int32 [8] scheduler words to clear, or NULL
};
// bf16 router: number of CTAs (a cluster) that share one 128-token tile by splitting the
// contraction.  Few tiles => split, so that more SMs stream X.
static inline int route_split(int64_t T, int H) {
  const int64_t tiles = (T + 127) / 128;
  const int kblocks = H / 64;
  if (tiles * 4 <= 160 && kblocks % 4 == 0) return 4;
  if (tiles * 2 <= 160 && kblocks % 2 == 0) return 2;
  return 1;
}
// Tokens per router CTA (= granularity of blk_cnt and of the in-block ranks the router leaves in inv_row).
static inline int route_block_tokens(int dtype, int64_t T, int H) {
  return dtype == FMMOE_BF16 ? 128 / route_split(T, H) : 32;
}
// Number of router CTAs = number of token blocks (the last tile's blocks may lie past T: they are empty).
static inline int route_num_blocks(int dtype, int64_t T, int H) {
  return dtype == FMMOE_BF16 ? (int)((T + 127) / 128) * route_split(T, H) : (int)((T + 31) / 32);
}
fmmoe_status launch_route(fmmoe_handle* h, const RouteArgs& a, cudaStream_t s);

struct PermuteArgs {
  const int32_t* topk_idx; const float* topk_w;
  int32_t* blk_cnt; int n_blk; int blk_tokens;   // router's block counts (turned into offsets in place)
  int64_t T; int K, E; int block_m;
  int32_t* expert_off; int32_t* row_token; float* row_gate; int32_t* inv_row;
  MTile* mtiles; int32_t* n_mtiles;
  // optional: also write the expert-grouped copy of x (xp[row] = x[token]) in the scatter pass
  const void* gather_x; void* gather_xp; int gather_row_bytes;
};
fmmoe_status launch_permute(fmmoe_handle* h, const PermuteArgs& a, cudaStream_t s);

struct FfnArgs {   // both paths
  const fmmoe_layer_desc* d; const fmmoe_weights* w;
  const void* x; int64_t T; int64_t p_max;
  const MTile* mtiles; const int32_t* n_mtiles; int32_t max_mtiles;
  int32_t* tile_counters;   // [2] zeroed per call: tile schedulers of GEMM-1 and GEMM-2
  const int32_t* row_token; const float* row_gate;
  void* xp; void* act; void* act_sh;
  float* acc;            // atomic mode
  float* y; float* ysh;  // deterministic mode
  void* yb; void* ybsh;  // pair-row mode (bf16)
  int deterministic;
  int pair;              // GEMM-2 stores gate-scaled bf16 rows per pair; the finalize pass sums them per token
  int gather_in_gemm;    // bf16: GEMM-1 gathers the routed rows of x itself (xp is not read)
  int* d_status;
  int test_withhold_stage;   // small-M form, self-test only (-1: off)
  int grid_override;         // small-M form, self-test only: CTAs to launch (0: one per SM)
};
// From a few hundred tokens on GEMM-1's loader warps gather the routed rows of x themselves and no
// expert-ordered copy of x is written (measured faster than the copy + plain TMA boxes from 256 tokens on,
// by 3-12 % of a step between 2,432 and 14,336 tokens).  Below that the small-M form runs on the copy.
// The threshold is a property of the handle (default 256 tokens; FMMOE_GATHER_MIN_TOKENS, read once
// in fmmoe_create, overrides it so that either path can be exercised at any size).
constexpr int64_t kGatherMinTokensDefault = 256;
// Decode-sized batches: token rows as the MMA's N dimension (FMMOE_SMALL_M_MAX_TOKENS).
constexpr int64_t kSmallMMaxTokensDefault = 256;
static inline bool gather_rows_in_gemm(const fmmoe_handle* h, int64_t T) { return T >= h->gather_min_tokens; }
fmmoe_status launch_ffn_tc(fmmoe_handle* h, const FfnArgs& a, cudaStream_t s);    // bf16, tcgen05, token rows as M
fmmoe_status launch_ffn_sm(fmmoe_handle* h, const FfnArgs& a, cudaStream_t s);    // bf16, tcgen05, token rows as N (reads xp)
fmmoe_status launch_ffn_tc2(fmmoe_handle* h, const FfnArgs& a, cudaStream_t s);   // bf16, tcgen05, CTA pairs, 256-row tiles (reads xp)
// Large batches (experts with several hundred rows): 256-row tiles on CTA pairs.
static inline bool use_cta_pairs(const fmmoe_handle* h, const fmmoe_layer_desc& d, int64_t T) {
  return d.dtype == FMMOE_BF16 && d.weight_format == FMMOE_WEIGHTS_AS_DTYPE && T >= h->cta_pair_min_tokens;
}
// Which form runs: below small_m_max_tokens (and below the in-GEMM gather threshold) the small-M form.
// Combine: every pair's gate-scaled row is written once in bf16 and summed per token in a fixed order
// (no atomics, reproducible bit for bit).  Measured against the atomic fp32 accumulator it is equal below
// 512 tokens and 2-4 % of a step faster from there on (the accumulator, T*H*4 bytes, stops fitting the L2
// cache next to the activations around 8,192 tokens and then pages through HBM), so it is the default at
// every size; FMMOE_PAIR_ROWS_MIN_TOKENS=n keeps the atomic combine below n tokens.
constexpr int64_t kPairMinTokensDefault = 0;
static inline bool use_pair_rows(const fmmoe_handle* h, const fmmoe_layer_desc& d, int64_t T, uint32_t flags) {
  return d.dtype == FMMOE_BF16 && !(flags & FMMOE_FLAG_DETERMINISTIC) && T >= h->pair_min_tokens;
}
// FP8 weights exist only in that form (the weight boxes are expanded in shared memory there).
static inline bool use_small_m(const fmmoe_handle* h, const fmmoe_layer_desc& d, int64_t T) {
  if (d.dtype != FMMOE_BF16) return false;
  if (d.weight_format == FMMOE_WEIGHTS_FP8_BLOCK128) return true;
  return T < h->small_m_max_tokens && T < h->gather_min_tokens && T < h->cta_pair_min_tokens;
}
fmmoe_status launch_ffn_f32(fmmoe_handle* h, const FfnArgs& a, cudaStream_t s);   // fp32 FMA

struct FinalizeArgs {
  const void* x; void* out; int64_t T; int H, K, n_shared; int dtype; int add_residual; int deterministic;
  const float* acc; const float* y; const float* ysh; const int32_t* inv_row; const float* topk_w;
  int pair; const void* yb; const void* ybsh;   // pair-row mode: bf16 [P,H] gate-scaled rows, [N_s*T,H] shared rows
};
fmmoe_status launch_finalize(fmmoe_handle* h, const FinalizeArgs& a, cudaStream_t s);

// start-up work of the pruning pass (module load, scratch address, shared-memory opt-in); device current
fmmoe_status prune_prepare(fmmoe_handle* h);

// fmmoe_prune_visual in two phases (bit 0: ranks, scores, selection on s_select; bit 1: rows on s_rows)
fmmoe_status prune_visual_phases(fmmoe_handle* h, const fmmoe_prune_params* p, const float* probs, int32_t n_experts,
                                 const float* attn, const void* x, int32_t dtype, int32_t hidden,
                                 const uint8_t* is_visual, const int64_t* seq_off, const int64_t* n_vis,
                                 const int64_t* n_retain, int32_t n_seq, void* x_out, uint8_t* is_visual_out,
                                 int32_t* keep_idx, uint8_t* kind, int64_t* out_seq_off, void* workspace,
                                 size_t workspace_bytes, int phases, cudaStream_t s_select, cudaStream_t s_rows);

}  // namespace fmmoe
