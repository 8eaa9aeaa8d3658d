// Permute-by-expert: from the per-expert histogram (filled by the router) to the
// stable grouping of the routed (token, expert) pairs by expert.  The paper only
// states that an unselected expert costs nothing (Section 3.1); the grouped order
// used here is the unique stable one (rows of an expert ascend by token index), so
// it is reproducible bit for bit: ranks come from ballots and scans, never from
// the arrival order of atomics.
//
// One CTA per expert: it scans the histogram for its first row and its first
// M-tile, then walks the tokens in order, 1024 at a time, and assigns consecutive
// rows to those that selected the expert.
#include <cuda_bf16.h>

#include "internal.h"

namespace fmmoe {

constexpr int P_THREADS = 1024;

struct PermuteDev {
  const int32_t* topk_idx; const float* topk_w; const int32_t* counts;
  long long T; int K, E, block_m;
  int32_t* expert_off; int32_t* row_token; float* row_gate; int32_t* inv_row;
  MTile* mtiles; int32_t* n_mtiles;
};

__global__ void __launch_bounds__(P_THREADS) permute_kernel(const PermuteDev a) {
  __shared__ int s_off, s_tile0, s_total_rows, s_total_tiles;
  __shared__ int s_warp[P_THREADS / 32];
  __shared__ int s_running;
  const int e = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  if (warp == 0) {   // prefix over the (<= 256) expert counts
    int off = 0, tiles = 0, tot = 0, tot_tiles = 0;
    for (int i = lane; i < a.E; i += 32) {
      const int c = a.counts[i];
      const int nt = (c + a.block_m - 1) / a.block_m;
      if (i < e) { off += c; tiles += nt; }
      tot += c; tot_tiles += nt;
    }
#pragma unroll
    for (int o = 16; o; o >>= 1) {
      off += __shfl_xor_sync(0xffffffffu, off, o);
      tiles += __shfl_xor_sync(0xffffffffu, tiles, o);
      tot += __shfl_xor_sync(0xffffffffu, tot, o);
      tot_tiles += __shfl_xor_sync(0xffffffffu, tot_tiles, o);
    }
    if (lane == 0) { s_off = off; s_tile0 = tiles; s_total_rows = tot; s_total_tiles = tot_tiles; s_running = 0; }
  }
  __syncthreads();
  const int base = s_off;
  const int cnt = a.counts[e];
  if (tid == 0) {
    if (a.expert_off) {
      a.expert_off[e] = base;
      if (e == a.E - 1) a.expert_off[a.E] = s_total_rows;
    }
    if (e == a.E - 1 && a.n_mtiles) a.n_mtiles[0] = s_total_tiles;
  }
  if (a.mtiles) {
    const int nt = (cnt + a.block_m - 1) / a.block_m;
    for (int i = tid; i < nt; i += P_THREADS) {
      MTile m;
      m.group = e; m.row0 = base + i * a.block_m;
      m.rows = min(a.block_m, cnt - i * a.block_m); m.pad = 0;
      a.mtiles[s_tile0 + i] = m;
    }
  }
  if (cnt == 0) return;

  for (long long t0 = 0; t0 < a.T; t0 += P_THREADS) {
    const long long t = t0 + tid;
    int slot = -1;
    if (t < a.T) {
      for (int s = 0; s < a.K; ++s)
        if (a.topk_idx[t * a.K + s] == e) { slot = s; break; }
    }
    const unsigned bal = __ballot_sync(0xffffffffu, slot >= 0);
    if (lane == 0) s_warp[warp] = __popc(bal);
    __syncthreads();
    if (warp == 0) {   // inclusive scan of the 32 warp counts
      int v = s_warp[lane];
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int n = __shfl_up_sync(0xffffffffu, v, o);
        if (lane >= o) v += n;
      }
      s_warp[lane] = v;
    }
    __syncthreads();
    const int running = s_running;
    if (slot >= 0) {
      const int pos = running + (warp ? s_warp[warp - 1] : 0) + __popc(bal & ((1u << lane) - 1u));
      const int row = base + pos;
      if (a.row_token) a.row_token[row] = (int)t;
      if (a.row_gate) a.row_gate[row] = a.topk_w[t * a.K + slot];
      if (a.inv_row) a.inv_row[t * a.K + slot] = row;
    }
    __syncthreads();
    if (tid == 0) s_running = running + s_warp[31];
    __syncthreads();
    if (s_running >= cnt) break;   // all rows of this expert placed
  }
}

// Copy the routed rows of X into expert-grouped order: xp[row] = x[row_token[row]].
// One warp per row, 16-byte accesses.
__global__ void gather_rows_kernel(const uint4* __restrict__ x, const int32_t* __restrict__ row_token,
                                   const int32_t* __restrict__ expert_off, int E, long long p_max, int row_vec,
                                   uint4* __restrict__ xp) {
  const int P = expert_off[E];
  const int warps = blockDim.x >> 5;
  const int lane = threadIdx.x & 31;
  for (long long row = (long long)blockIdx.x * warps + (threadIdx.x >> 5); row < P; row += (long long)gridDim.x * warps) {
    const long long t = row_token[row];
    const uint4* src = x + t * row_vec;
    uint4* dst = xp + row * row_vec;
    for (int i = lane; i < row_vec; i += 32) dst[i] = src[i];
  }
}

fmmoe_status launch_permute(fmmoe_handle* h, const PermuteArgs& a, cudaStream_t s) {
  if (a.E <= 0) return FMMOE_OK;
  PermuteDev d;
  d.topk_idx = a.topk_idx; d.topk_w = a.topk_w; d.counts = a.counts;
  d.T = a.T; d.K = a.K; d.E = a.E; d.block_m = a.block_m;
  d.expert_off = a.expert_off; d.row_token = a.row_token; d.row_gate = a.row_gate; d.inv_row = a.inv_row;
  d.mtiles = a.mtiles; d.n_mtiles = a.n_mtiles;
  { ProfScope ps(h, FMMOE_KERNEL_PERMUTE, s); permute_kernel<<<a.E, P_THREADS, 0, s>>>(d); }
  FMMOE_CUDA_TRY(cudaGetLastError());
  h->launches += 1;
  return FMMOE_OK;
}

fmmoe_status launch_gather_rows(fmmoe_handle* h, const void* x, const int32_t* row_token, const int32_t* expert_off,
                                int E, int64_t p_max, int H, int elem_bytes, void* xp, cudaStream_t s) {
  if (p_max == 0) return FMMOE_OK;
  const int row_vec = H * elem_bytes / 16;
  const int threads = 256;
  long long blocks = (p_max + 7) / 8;
  const long long cap = (long long)h->sm_count * 8;
  if (blocks > cap) blocks = cap;
  {
    ProfScope ps(h, FMMOE_KERNEL_GATHER, s);
    gather_rows_kernel<<<(int)blocks, threads, 0, s>>>(static_cast<const uint4*>(x), row_token, expert_off, E, p_max,
                                                       row_vec, static_cast<uint4*>(xp));
  }
  FMMOE_CUDA_TRY(cudaGetLastError());
  h->launches += 1;
  return FMMOE_OK;
}

}  // namespace fmmoe
