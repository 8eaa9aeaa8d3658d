// Permute-by-expert: the stable grouping of the routed (token, expert) pairs by expert.  The
// paper only states that an unselected expert costs nothing (Section 3.1); the grouped order
// used here is the unique stable one (rows of an expert ascend by token index), so it is
// reproducible bit for bit: every rank comes from counts and scans, never from the arrival
// order of atomics.
//
// The router leaves, per block of tokens, the number of selections of every expert (blk_cnt)
// and, per (token, slot), the token's rank among its block's tokens that chose that expert.
//   scan_kernel    : per expert an exclusive scan of the block counts (in place), the scan of
//                    the expert totals (expert_off) and the list of 128-row M-tiles
//   scatter_kernel : row = expert_off[e] + block offset + in-block rank, for every pair
//   scatter_gather_kernel : the same, and the pair's row of x copied to its row of the expert-grouped copy
#include <cuda_bf16.h>

#include "internal.h"
#include "ptx.cuh"

namespace fmmoe {

constexpr int P_THREADS = 1024;

struct PermuteDev {
  const int32_t* topk_idx; const float* topk_w;
  int32_t* blk_cnt; int n_blk, blk_tokens;
  long long T; int K, E, block_m;
  int32_t* expert_off; int32_t* row_token; float* row_gate; int32_t* inv_row;
  MTile* mtiles; int32_t* n_mtiles;
};

__global__ void __launch_bounds__(P_THREADS) scan_kernel(const PermuteDev a) {
  __shared__ int s_cnt[FMMOE_MAX_EXPERTS], s_off[FMMOE_MAX_EXPERTS + 1], s_tile0[FMMOE_MAX_EXPERTS + 1];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  pdl_launch_dependents();
  pdl_wait();
  // per expert: exclusive scan over the token blocks, 32 blocks per step
  for (int e = warp; e < a.E; e += P_THREADS / 32) {
    int32_t* row = a.blk_cnt + (long long)e * a.n_blk;
    int running = 0;
    for (int b0 = 0; b0 < a.n_blk; b0 += 128) {   // four independent loads per lane, then the scans
      int v[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int b = b0 + 32 * j + lane;
        v[j] = b < a.n_blk ? row[b] : 0;
      }
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int b = b0 + 32 * j + lane;
        int incl = v[j];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const int n = __shfl_up_sync(0xffffffffu, incl, o);
          if (lane >= o) incl += n;
        }
        if (b < a.n_blk) row[b] = running + incl - v[j];
        running += __shfl_sync(0xffffffffu, incl, 31);
      }
    }
    if (lane == 0) s_cnt[e] = running;
  }
  __syncthreads();
  if (warp == 0) {   // scan over the (<= 256) expert totals: first row and first M-tile of each expert
    int run_rows = 0, run_tiles = 0;
    for (int e0 = 0; e0 < a.E; e0 += 32) {
      const int e = e0 + lane;
      const int c = e < a.E ? s_cnt[e] : 0;
      const int nt = (c + a.block_m - 1) / a.block_m;
      int ic = c, it = nt;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int n1 = __shfl_up_sync(0xffffffffu, ic, o);
        const int n2 = __shfl_up_sync(0xffffffffu, it, o);
        if (lane >= o) { ic += n1; it += n2; }
      }
      if (e < a.E) { s_off[e] = run_rows + ic - c; s_tile0[e] = run_tiles + it - nt; }
      run_rows += __shfl_sync(0xffffffffu, ic, 31);
      run_tiles += __shfl_sync(0xffffffffu, it, 31);
    }
    if (lane == 0) {
      s_off[a.E] = run_rows; s_tile0[a.E] = run_tiles;
      if (a.n_mtiles) a.n_mtiles[0] = run_tiles;
    }
  }
  __syncthreads();
  for (int e = tid; e <= a.E; e += P_THREADS) a.expert_off[e] = s_off[e];
  if (a.mtiles) {
    for (int e = warp; e < a.E; e += P_THREADS / 32) {
      const int cnt = s_cnt[e], base = s_off[e], nt = s_tile0[e + 1] - s_tile0[e];
      for (int i = lane; i < nt; i += 32) {
        MTile m;
        m.group = e; m.row0 = base + i * a.block_m;
        m.rows = min(a.block_m, cnt - i * a.block_m); m.pad = nt == 1;   // 1: the expert's only tile
        a.mtiles[s_tile0[e] + i] = m;
      }
    }
  }
}

__global__ void __launch_bounds__(256) scatter_kernel(const PermuteDev a) {
  pdl_launch_dependents();
  pdl_wait();
  const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= a.T * a.K) return;
  const int e = a.topk_idx[i];
  if (e < 0 || e >= a.E) return;           // padded slot: inv_row already holds -1
  const long long t = i / a.K;
  const int row = a.expert_off[e] + a.blk_cnt[(long long)e * a.n_blk + (int)(t / a.blk_tokens)] + a.inv_row[i];
  if (row < 0 || row >= a.expert_off[a.E]) return;   // cannot happen for a consistent routing record
  a.row_token[row] = (int32_t)t;
  a.row_gate[row] = a.topk_w[i];
  a.inv_row[i] = row;
}

// scatter_kernel and gather_rows_kernel in one pass for small batches: one warp per (token, slot)
// pair computes the pair's row (lane 0, as scatter_kernel does) and then copies the token's row of X
// to that row of the expert-grouped copy.  Saves a dependent launch on the way to GEMM-1.
__global__ void __launch_bounds__(256) scatter_gather_kernel(const PermuteDev a, const uint4* __restrict__ x, int row_vec,
                                                             uint4* __restrict__ xp) {
  pdl_launch_dependents();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const long long i = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (i >= a.T * a.K) return;
  const long long t = i / a.K;
  int row = -1;
  if (lane == 0) {
    const int e = a.topk_idx[i];
    if (e >= 0 && e < a.E) {
      row = a.expert_off[e] + a.blk_cnt[(long long)e * a.n_blk + (int)(t / a.blk_tokens)] + a.inv_row[i];
      if (row < 0 || row >= a.expert_off[a.E]) {
        row = -1;                            // cannot happen for a consistent routing record
      } else {
        a.row_token[row] = (int32_t)t;
        a.row_gate[row] = a.topk_w[i];
        a.inv_row[i] = row;
      }
    }
  }
  row = __shfl_sync(0xffffffffu, row, 0);
  if (row < 0) return;
  const uint4* src = x + t * row_vec;
  uint4* dst = xp + (long long)row * row_vec;
  for (int j = lane; j < row_vec; j += 32) dst[j] = src[j];
}

fmmoe_status launch_permute(fmmoe_handle* h, const PermuteArgs& a, cudaStream_t s) {
  if (a.E <= 0 || a.T <= 0) return FMMOE_OK;
  PermuteDev d;
  d.topk_idx = a.topk_idx; d.topk_w = a.topk_w; d.blk_cnt = a.blk_cnt; d.n_blk = a.n_blk; d.blk_tokens = a.blk_tokens;
  d.T = a.T; d.K = a.K; d.E = a.E; d.block_m = a.block_m;
  d.expert_off = a.expert_off; d.row_token = a.row_token; d.row_gate = a.row_gate; d.inv_row = a.inv_row;
  d.mtiles = a.mtiles; d.n_mtiles = a.n_mtiles;
  const long long pairs = a.T * a.K;
  {
    ProfScope ps(h, FMMOE_KERNEL_PERMUTE, s);
    FMMOE_CUDA_TRY(launch_pdl(scan_kernel, dim3(1), dim3(P_THREADS), 0, s, 1, d));
    if (a.gather_x) {
      FMMOE_CUDA_TRY(launch_pdl(scatter_gather_kernel, dim3((unsigned)((pairs + 7) / 8)), dim3(256), 0, s, 1, d,
                                static_cast<const uint4*>(a.gather_x), a.gather_row_bytes / 16, static_cast<uint4*>(a.gather_xp)));
    } else {
      FMMOE_CUDA_TRY(launch_pdl(scatter_kernel, dim3((unsigned)((pairs + 255) / 256)), dim3(256), 0, s, 1, d));
    }
  }
  FMMOE_CUDA_TRY(cudaGetLastError());
  h->launches += 2;
  return FMMOE_OK;
}

}  // namespace fmmoe
