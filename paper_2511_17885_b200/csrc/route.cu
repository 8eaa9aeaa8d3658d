// Router: logits (Eq. 1), softmax (Eq. 2), modality-aware top-k (Eq. 3, with K_v
// for vision tokens once the layer has reached l_v) and renormalised gates (Eq. 5),
// fused in one kernel per storage type.
//   bf16: the logits tile [128 tokens, E] is a tcgen05 GEMM fed by TMA with its accumulator
//         in tensor memory; the tile is then copied to shared memory and eight lanes per
//         token run the softmax / top-k / gate step across the expert dimension.
//   fp32: a CTA owns 32 tokens, forms their logits with plain FMA in shared memory (TF32
//         would miss an fp32 tolerance), then each warp takes 8 tokens and runs the
//         softmax / top-k / gate step across the expert dimension with warp shuffles.
// Both kernels also start the permutation: a CTA records, per expert, which of its tokens
// selected it (a bit mask in shared memory), from which it writes the block's expert counts
// and, for every (token, slot), the rank of the token among the block's tokens that chose
// the same expert.  Ranks come from bit counts, never from the arrival order of atomics.
#include <cuda_bf16.h>
#include <float.h>

#include "internal.h"
#include "ptx.cuh"

namespace fmmoe {

constexpr int R_BM = 32;
constexpr int R_THREADS = 128;

struct RouteDev {
  const void* x; const void* w; const float* bias; const uint8_t* is_visual;
  long long T; int H, E, K, Kv, reduce_on, e_pad;
  float* logits; float* probs; int32_t* topk_idx; float* topk_w; int32_t* inv_row;
  int32_t* blk_cnt; int n_blk;   // [E][n_blk] selections of each token block per expert
  float* acc_zero; int32_t* misc_zero;   // combine accumulator [T,H] / scheduler words to clear (or NULL)
};

__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Softmax / top-k / gates for the CTA's tokens, logits already in shared memory.
// NTL = e_pad / 32 values per lane.
template <int NTL>
__device__ __forceinline__ void route_tail(const float* Ls, int ldl, long long t0, const RouteDev& a, uint32_t* emask) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  for (int r = warp; r < R_BM; r += R_THREADS / 32) {
    const long long t = t0 + r;
    if (t >= a.T) break;
    float v[NTL];
#pragma unroll
    for (int j = 0; j < NTL; ++j) {
      const int e = lane + 32 * j;
      v[j] = e < a.E ? Ls[r * ldl + e] : -INFINITY;
    }
    if (a.logits) {
#pragma unroll
      for (int j = 0; j < NTL; ++j)
        if (lane + 32 * j < a.E) a.logits[t * a.E + lane + 32 * j] = v[j];
    }
    // The shuffle reductions below need a total order: non-finite logits (overflowed activations
    // upstream) are clamped and NaN counts as the lowest value, so that all lanes agree on every
    // round's winner and each selected index is a valid, distinct expert.  Finite inputs are untouched.
#pragma unroll
    for (int j = 0; j < NTL; ++j)
      if (lane + 32 * j < a.E) v[j] = fminf(fmaxf(v[j], -FLT_MAX), FLT_MAX);
    float m = v[0];
#pragma unroll
    for (int j = 1; j < NTL; ++j) m = fmaxf(m, v[j]);
    m = warp_max(m);
    float s = 0.f;
#pragma unroll
    for (int j = 0; j < NTL; ++j) s += expf(v[j] - m);   // exp(-inf) = 0 for padded lanes
    s = warp_sum(s);
    if (a.probs) {
      const float inv = 1.f / s;
#pragma unroll
      for (int j = 0; j < NTL; ++j)
        if (lane + 32 * j < a.E) a.probs[t * a.E + lane + 32 * j] = expf(v[j] - m) * inv;
    }
    const int k_t = (a.reduce_on && a.is_visual[t]) ? a.Kv : a.K;
    uint32_t taken = 0;
    float my_val = -INFINITY;
    int my_idx = -1;
    for (int i = 0; i < k_t; ++i) {
      float bv = -INFINITY;
      int be = 0x7fffffff;
#pragma unroll
      for (int j = 0; j < NTL; ++j) {
        const int e = lane + 32 * j;
        if (e < a.E && !((taken >> j) & 1u) && (v[j] > bv || be == 0x7fffffff)) { bv = v[j]; be = e; }
      }
#pragma unroll
      for (int o = 16; o; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
        const int oe = __shfl_xor_sync(0xffffffffu, be, o);
        if (oe != 0x7fffffff && (be == 0x7fffffff || ov > bv || (ov == bv && oe < be))) { bv = ov; be = oe; }
      }
      if ((be & 31) == lane) taken |= 1u << (be >> 5);
      if (lane == i) { my_val = bv; my_idx = be; }
    }
    const float p = lane < k_t ? expf(my_val - m) : 0.f;
    const float denom = warp_sum(p);
    if (lane < a.K) {
      const bool sel = lane < k_t;
      a.topk_idx[t * a.K + lane] = sel ? my_idx : -1;
      a.topk_w[t * a.K + lane] = sel ? p / denom : 0.f;
      if (sel && (unsigned)my_idx < (unsigned)a.E) atomicOr(&emask[my_idx], 1u << r);   // one 32-bit word per expert: the block has 32 tokens
    }
  }
}

// After the block's selections are in `emask` ([E][WORDS] bit masks over the block's tokens):
// write the block's per-expert counts and the in-block rank of every (token, slot).
template <int WORDS>
__device__ __forceinline__ void emit_block_ranks(const uint32_t* emask, long long t0, int blk, const RouteDev& a) {
  __syncthreads();
  for (int e = threadIdx.x; e < a.E; e += blockDim.x) {
    int c = 0;
#pragma unroll
    for (int w = 0; w < WORDS; ++w) c += __popc(emask[e * WORDS + w]);
    a.blk_cnt[(long long)e * a.n_blk + blk] = c;
  }
  const int items = WORDS * 32 * a.K;
  for (int it = threadIdx.x; it < items; it += blockDim.x) {
    const int r = it / a.K;
    const long long t = t0 + r;
    if (t >= a.T) break;
    const int e = __ldcg(a.topk_idx + t * a.K + (it - r * a.K));   // written by this CTA before the barrier
    int rank = -1;
    if (e >= 0 && e < a.E) {
      rank = __popc(emask[e * WORDS + (r >> 5)] & ((1u << (r & 31)) - 1u));
#pragma unroll
      for (int w = 0; w < WORDS; ++w)
        if (w < (r >> 5)) rank += __popc(emask[e * WORDS + w]);
    }
    a.inv_row[t * a.K + (it - r * a.K)] = rank;
  }
}

// ---------------------------------------------------------------------------------------
// bf16 router on the tcgen05 tensor cores.  A CTA of 16 warps owns 128 tokens:
//   warp 0    : TMA producer  (X tile 128x64 and the router matrix tile e_pad x 64 per stage)
//   warp 1    : UMMA issuer   (128 x e_pad x 16 tcgen05.mma; the logits tile lives in TMEM)
//   warps 4-11: once the accumulator is complete, copy it (+ bias) from TMEM to shared memory,
//               reusing the pipeline's stage buffers
//   cluster   : with few token tiles the contraction is split over a cluster of 2 or 4 CTAs
//               (more SMs pulling X); every CTA then owns 128/split rows of the tile and adds
//               the partial tiles of its peers, in rank order, through distributed shared memory
//   all warps : softmax / top-k / gates with 8 lanes per token (4 tokens per warp at a time):
//               every lane holds E/8 logits of its token in registers, the row maximum, the
//               sum and each top-k round are a local scan plus three shuffle steps across
//               the expert dimension.
// The router matrix is read once per 128 tokens (from L2 after the first CTA), X once.
// ---------------------------------------------------------------------------------------
constexpr int RT_BM = 128;
constexpr int RT_BK = 64;
constexpr int RT_THREADS = 512;
constexpr int RT_A_BYTES = RT_BM * RT_BK * 2;
constexpr int RT_MAX_STAGES = 8;

__device__ __forceinline__ float group8_max(float v) {
#pragma unroll
  for (int o = 4; o; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ __forceinline__ float group8_sum(float v) {
#pragma unroll
  for (int o = 4; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

__device__ __forceinline__ int group8_min_int(int v) {
#pragma unroll
  for (int o = 4; o; o >>= 1) v = min(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Softmax / top-k / gates for n_rows (a multiple of 32) token rows whose logits (bias included)
// sit in shared memory, row pitch ldl (odd).  Eight lanes per token, four tokens per warp.
// NV = logits per lane (expert e = lane8 + 8 j), NV * 8 >= E.
template <int NV>
__device__ __forceinline__ void route_tail_group8(const float* Lr, int ldl, long long t_first, int n_rows, uint32_t* emask,
                                                  int words, const RouteDev& a) {
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int g = lane >> 3, l8 = lane & 7;
  const int E = a.E;
  for (int base = (warp >> 3) * 32; base < n_rows; base += 32 * (RT_THREADS / 256)) {
    // eight warps share 32 rows; rows of one warp are 8 apart: with an odd row pitch the four groups hit
    // distinct banks
    const int rl = base + g * 8 + (warp & 7);
    const long long t = t_first + rl;
    const bool tok_ok = t < a.T;
    float z[NV];
#pragma unroll
    for (int j = 0; j < NV; ++j) {
      const int e = l8 + 8 * j;
      z[j] = e < E ? Lr[rl * ldl + e] : -INFINITY;
    }
    if (a.logits && tok_ok) {
#pragma unroll
      for (int j = 0; j < NV; ++j)
        if (l8 + 8 * j < E) a.logits[t * E + l8 + 8 * j] = z[j];
    }
    // The selection below marks a taken entry with -inf and looks experts up by value, so it needs
    // finite logits: non-finite ones (overflowed activations upstream) are clamped, NaN counts as the
    // lowest value.  Finite inputs are untouched; whatever the input, every selected index is a
    // valid, distinct expert.
#pragma unroll
    for (int j = 0; j < NV; ++j)
      if (l8 + 8 * j < E) z[j] = fminf(fmaxf(z[j], -FLT_MAX), FLT_MAX);
    float m = z[0];
#pragma unroll
    for (int j = 1; j < NV; ++j) m = fmaxf(m, z[j]);
    m = group8_max(m);
    float s = 0.f;
#pragma unroll
    for (int j = 0; j < NV; ++j) s += __expf(z[j] - m);   // exp(-inf) = 0 for padded entries
    s = group8_sum(s);
    if (a.probs && tok_ok) {
      const float inv = 1.f / s;
#pragma unroll
      for (int j = 0; j < NV; ++j)
        if (l8 + 8 * j < E) a.probs[t * E + l8 + 8 * j] = __expf(z[j] - m) * inv;
    }
    const int k_t = tok_ok ? ((a.reduce_on && a.is_visual[t]) ? a.Kv : a.K) : 0;
    const int k_warp = __reduce_max_sync(0xffffffffu, k_t);
    float denom = 0.f;
    float sel_p[2] = {0.f, 0.f};
    int sel_e[2] = {-1, -1};
    for (int i = 0; i < k_warp; ++i) {
      // largest remaining logit of the token, then the lowest expert index that holds it
      // (a taken entry is overwritten with -inf; real logits are finite)
      float bv = z[0];
#pragma unroll
      for (int j = 1; j < NV; ++j) bv = fmaxf(bv, z[j]);
      bv = group8_max(bv);
      int be = 0x7fffffff;
#pragma unroll
      for (int j = NV - 1; j >= 0; --j)
        if (z[j] == bv) be = l8 + 8 * j;
      be = group8_min_int(be);
      if (i < k_t) {
#pragma unroll
        for (int j = 0; j < NV; ++j)
          if (l8 + 8 * j == be) z[j] = -INFINITY;
        const float p = __expf(bv - m);
        denom += p;
        if ((i & 7) == l8) { sel_p[i >> 3] = p; sel_e[i >> 3] = be; }
      }
    }
    if (tok_ok) {
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const int slot = l8 + 8 * h;
        if (slot < a.K) {
          const bool sel = slot < k_t;
          a.topk_idx[t * a.K + slot] = sel ? sel_e[h] : -1;
          a.topk_w[t * a.K + slot] = sel ? sel_p[h] / denom : 0.f;   // Eq. 5
          if (sel && (unsigned)sel_e[h] < (unsigned)E) atomicOr(&emask[sel_e[h] * words + (rl >> 5)], 1u << (rl & 31));
        }
      }
    }
  }
}

__global__ void __launch_bounds__(RT_THREADS, 1)
route_tc_kernel(const __grid_constant__ CUtensorMap tmX, const __grid_constant__ CUtensorMap tmW, const RouteDev a,
                const int stages, const int tmem_cols, const int tile_bytes, const int split, int* status) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  unsigned char* smem = smem_raw + ((1024 - (raw & 1023)) & 1023);
  const int b_bytes = a.e_pad * RT_BK * 2;
  const int stage_bytes = RT_A_BYTES + b_bytes;
  float* bias_s = reinterpret_cast<float*>(smem + tile_bytes);              // [256]
  uint32_t* emask = reinterpret_cast<uint32_t*>(bias_s + FMMOE_MAX_EXPERTS);   // [256][4] token masks per expert
  uint64_t* full_bar = reinterpret_cast<uint64_t*>(emask + FMMOE_MAX_EXPERTS * 4);
  uint64_t* empty_bar = full_bar + RT_MAX_STAGES;
  uint64_t* tfull_bar = empty_bar + RT_MAX_STAGES;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(tfull_bar + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int krank = (int)cluster_ctarank();            // this CTA's slice of the contraction
  const int kblocks = a.H / RT_BK / split;
  const int kb0 = krank * kblocks;
  const int nch = (a.E + 31) / 32;
  const int ldl = nch * 32 + 1;                 // odd pitch of the logits tile in shared memory
  float* Ls = reinterpret_cast<float*>(smem);   // [128][ldl], overlays the stage buffers after the GEMM

  pdl_launch_dependents();
  if (threadIdx.x == 0) {
    for (int i = 0; i < stages; ++i) { mbar_init(&full_bar[i], 1); mbar_init(&empty_bar[i], 1); }
    mbar_init(tfull_bar, 1);
    *abort_flag = 0;
    mbar_fence_init();
  }
  if (warp == 1) {
    tmem_alloc(tmem_slot, (uint32_t)tmem_cols);
    tmem_relinquish();
  }
  pdl_wait();   // from here on: global memory that earlier kernels of the stream may have written
  for (int e = threadIdx.x; e < FMMOE_MAX_EXPERTS; e += RT_THREADS) {
    bias_s[e] = (a.bias && e < a.E) ? a.bias[e] : 0.f;
#pragma unroll
    for (int w = 0; w < 4; ++w) emask[e * 4 + w] = 0;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_slot;
  const int row0 = (blockIdx.x / split) * RT_BM;

  if (warp == 0) {
    if (lane == 0) {
      tma_prefetch_desc(&tmX); tma_prefetch_desc(&tmW);
      int stage = 0; uint32_t phase = 0;
      bool ok = true;
      for (int kb = 0; kb < kblocks; ++kb) {
        if (!mbar_wait(&empty_bar[stage], phase ^ 1, abort_flag)) { ok = false; break; }
        unsigned char* sA = smem + stage * stage_bytes;
        mbar_arrive_expect_tx(&full_bar[stage], (uint32_t)stage_bytes);
        tma_load_2d(sA, &tmX, &full_bar[stage], (kb0 + kb) * RT_BK, row0);
        tma_load_2d(sA + RT_A_BYTES, &tmW, &full_bar[stage], (kb0 + kb) * RT_BK, 0);
        if (++stage == stages) { stage = 0; phase ^= 1; }
      }
      if (!ok) { atomicCAS(status, 0, DEV_TIMEOUT); *abort_flag = 1; }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = umma_idesc_bf16(RT_BM, a.e_pad);
      int stage = 0; uint32_t phase = 0;
      bool ok = true;
      for (int kb = 0; kb < kblocks; ++kb) {
        if (!mbar_wait(&full_bar[stage], phase, abort_flag)) { ok = false; break; }
        tc_fence_after();
        const uint32_t sA = smem_u32(smem + stage * stage_bytes);
        const uint64_t da = umma_desc_sw128(sA);
        const uint64_t db = umma_desc_sw128(sA + RT_A_BYTES);
#pragma unroll
        for (int k = 0; k < RT_BK / 16; ++k) umma_bf16(tmem_base, da + 2 * k, db + 2 * k, idesc, (kb | k) != 0);
        umma_commit(&empty_bar[stage]);
        if (++stage == stages) { stage = 0; phase ^= 1; }
      }
      if (ok) umma_commit(tfull_bar);
      else { atomicCAS(status, 0, DEV_TIMEOUT); *abort_flag = 1; }
    }
  } else {
    // warps 2-15 have nothing to do while the GEMM streams: clear this CTA's rows of the layer's
    // fp32 combine accumulator (and, once, the tile schedulers' counters)
    if (a.misc_zero && blockIdx.x == 0 && threadIdx.x == 64)
      for (int i = 1; i < 8; ++i) a.misc_zero[i] = 0;
    if (a.acc_zero) {
      const int n_rows = RT_BM / split;
      const long long t_lo = (long long)row0 + krank * n_rows;
      long long t_hi = t_lo + n_rows;
      if (t_hi > a.T) t_hi = a.T;
      if (t_lo < t_hi) {
        float4* dst = reinterpret_cast<float4*>(a.acc_zero + t_lo * a.H);
        const long long n4 = (t_hi - t_lo) * a.H / 4;
        for (long long i = threadIdx.x - 64; i < n4; i += RT_THREADS - 64) dst[i] = make_float4(0.f, 0.f, 0.f, 0.f);
      }
    }
  }
  if (warp >= 4 && warp < 12) {
    // accumulator complete => every stage buffer has been consumed: reuse them for the logits
    // (two warps per TMEM lane quarter, alternate 32-column chunks)
    const int q = warp & 3;
    if (mbar_wait(tfull_bar, 0, abort_flag)) {
      tc_fence_after();
      const uint32_t taddr = tmem_base + (static_cast<uint32_t>(q * 32) << 16);
      float* dst = Ls + (q * 32 + lane) * ldl;
      for (int c = (warp - 4) >> 2; c < nch; c += 2) {
        uint32_t v[32];
        tmem_ld32(taddr + c * 32, v);
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 32; ++j) dst[c * 32 + j] = __uint_as_float(v[j]);   // this CTA's partial sums
      }
    } else {
      atomicCAS(status, 0, DEV_TIMEOUT); *abort_flag = 1;
    }
  }
  __syncwarp();
  tc_fence_before();
  __syncthreads();
  const bool failed = *abort_flag != 0;
  if (failed) {
    const uint64_t t0 = global_timer_ns();
    while (global_timer_ns() - t0 < 200000ull) { }
    __syncthreads();
  }
  // Every CTA of the cluster now holds its partial logits tile in shared memory.  Both cluster
  // barriers are executed unconditionally (a CTA that gave up still arrives), so no peer can
  // be left waiting.
  cluster_sync_all();
  if (!failed) {
    const int n_rows = RT_BM / split, row_lo = krank * n_rows, words = n_rows / 32;
    // This CTA's rows of the logits tile = sum over the cluster's partial tiles, in rank order,
    // plus the bias.  The rows are one contiguous, 16-byte aligned run of every CTA's tile
    // (32 rows * pitch * 4 bytes), read from the peers with 16-byte distributed-shared-memory
    // loads and written to Lr (row pitch ldl, after the tile).
    // (a single-CTA cluster owns the whole tile and adds the bias in place)
    float* Lr = split == 1 ? Ls : reinterpret_cast<float*>((reinterpret_cast<uintptr_t>(Ls + RT_BM * ldl) + 15) & ~uintptr_t(15));
    {
      uint32_t peer[4];
#pragma unroll
      for (int q = 0; q < 4; ++q) peer[q] = cluster_map_shared(smem_u32(Ls + row_lo * ldl), q < split ? q : 0);
      const int n4 = n_rows * ldl / 4;
      for (int i = threadIdx.x; i < n4; i += RT_THREADS) {
        float4 acc4 = ld_cluster_v4f32(peer[0] + i * 16);
#pragma unroll
        for (int q = 1; q < 4; ++q) {
          if (q < split) {
            const float4 v = ld_cluster_v4f32(peer[q] + i * 16);
            acc4.x += v.x; acc4.y += v.y; acc4.z += v.z; acc4.w += v.w;
          }
        }
        // bias by column: element index -> column
        const int e0 = (i * 4) % ldl;
        float vals[4] = {acc4.x, acc4.y, acc4.z, acc4.w};
#pragma unroll
        for (int c = 0; c < 4; ++c) {
          int e = e0 + c; if (e >= ldl) e -= ldl;
          Lr[i * 4 + c] = vals[c] + (e < FMMOE_MAX_EXPERTS ? bias_s[e] : 0.f);
        }
      }
    }
    __syncthreads();
    const long long t_first = (long long)row0 + row_lo;
    switch ((a.E + 31) / 32) {
      case 1: route_tail_group8<4>(Lr, ldl, t_first, n_rows, emask, words, a); break;
      case 2: route_tail_group8<8>(Lr, ldl, t_first, n_rows, emask, words, a); break;
      case 3: route_tail_group8<12>(Lr, ldl, t_first, n_rows, emask, words, a); break;
      case 4: route_tail_group8<16>(Lr, ldl, t_first, n_rows, emask, words, a); break;
      case 5: route_tail_group8<20>(Lr, ldl, t_first, n_rows, emask, words, a); break;
      case 6: route_tail_group8<24>(Lr, ldl, t_first, n_rows, emask, words, a); break;
      case 7: route_tail_group8<28>(Lr, ldl, t_first, n_rows, emask, words, a); break;
      default: route_tail_group8<32>(Lr, ldl, t_first, n_rows, emask, words, a); break;
    }
    // the token block of this CTA: rows [row_lo, row_lo + n_rows) of the tile
    if (split == 1) emit_block_ranks<4>(emask, (long long)row0, blockIdx.x, a);
    else if (split == 2) emit_block_ranks<2>(emask, (long long)row0 + row_lo, blockIdx.x, a);
    else emit_block_ranks<1>(emask, (long long)row0 + row_lo, blockIdx.x, a);
  }
  cluster_sync_all();   // peers may still be reading this CTA's tile until here
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, (uint32_t)tmem_cols);
  }
}

// fp32 router (no tensor cores: TF32 would miss the fp32 tolerance).  Thread (warp w,
// lane l) accumulates rows w, w+4, ... and columns l, l+32, ...
template <int NT>
__global__ void __launch_bounds__(R_THREADS) route_f32_kernel(const RouteDev a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  constexpr int BK = 32;
  const int e_pad = NT * 32;
  const int ldl = e_pad + 1;
  float* Xs = reinterpret_cast<float*>(smem_raw);   // [R_BM][BK+1]
  float* Ws = Xs + R_BM * (BK + 1);                 // [e_pad][BK+1]
  float* Ls = Ws + e_pad * (BK + 1);                // [R_BM][ldl]
  uint32_t* emask = reinterpret_cast<uint32_t*>(Ls + R_BM * ldl);   // [e_pad] one word per expert (32 tokens)
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const long long t0 = (long long)blockIdx.x * R_BM;
  pdl_launch_dependents();
  pdl_wait();
  if (a.misc_zero && blockIdx.x == 0 && tid == 0)
    for (int i = 1; i < 8; ++i) a.misc_zero[i] = 0;
  if (a.acc_zero) {   // clear this block's rows of the combine accumulator
    long long t_hi = t0 + R_BM;
    if (t_hi > a.T) t_hi = a.T;
    const long long n = (t_hi - t0) * a.H;
    for (long long i = tid; i < n; i += R_THREADS) a.acc_zero[t0 * a.H + i] = 0.f;
  }
  const float* X = static_cast<const float*>(a.x);
  const float* W = static_cast<const float*>(a.w);
  for (int i = tid; i < e_pad; i += R_THREADS) emask[i] = 0;
  float acc[R_BM / 4][NT];
#pragma unroll
  for (int i = 0; i < R_BM / 4; ++i)
#pragma unroll
    for (int j = 0; j < NT; ++j) acc[i][j] = 0.f;
  for (int k0 = 0; k0 < a.H; k0 += BK) {
    __syncthreads();
    for (int c = tid; c < R_BM * BK; c += R_THREADS) {
      const int r = c / BK, k = c % BK;
      Xs[r * (BK + 1) + k] = (t0 + r < a.T && k0 + k < a.H) ? X[(t0 + r) * a.H + k0 + k] : 0.f;
    }
    for (int c = tid; c < e_pad * BK; c += R_THREADS) {
      const int r = c / BK, k = c % BK;
      Ws[r * (BK + 1) + k] = (r < a.E && k0 + k < a.H) ? W[(long long)r * a.H + k0 + k] : 0.f;
    }
    __syncthreads();
#pragma unroll 4
    for (int k = 0; k < BK; ++k) {
      float wv[NT];
#pragma unroll
      for (int j = 0; j < NT; ++j) wv[j] = Ws[(lane + 32 * j) * (BK + 1) + k];
#pragma unroll
      for (int i = 0; i < R_BM / 4; ++i) {
        const float xv = Xs[(warp + 4 * i) * (BK + 1) + k];
#pragma unroll
        for (int j = 0; j < NT; ++j) acc[i][j] = fmaf(xv, wv[j], acc[i][j]);
      }
    }
  }
#pragma unroll
  for (int i = 0; i < R_BM / 4; ++i)
#pragma unroll
    for (int j = 0; j < NT; ++j) {
      const int col = lane + 32 * j;
      Ls[(warp + 4 * i) * ldl + col] = acc[i][j] + ((a.bias && col < a.E) ? a.bias[col] : 0.f);
    }
  __syncthreads();
  route_tail<NT>(Ls, ldl, t0, a, emask);
  emit_block_ranks<1>(emask, t0, blockIdx.x, a);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static bool route_map(fmmoe_handle* h, CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {cols * 2};
  const cuuint32_t box[2] = {RT_BK, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return reinterpret_cast<EncodeTiledFn>(h->encode_tiled)(
             m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

static fmmoe_status launch_route_tc(fmmoe_handle* h, RouteDev d, cudaStream_t s) {
  if (!h->encode_tiled) return FMMOE_ERR_CUDA;
  d.e_pad = (d.E + 15) / 16 * 16;                       // UMMA N: a multiple of 16 for M = 128
  const int stage_bytes = RT_A_BYTES + d.e_pad * RT_BK * 2;
  int stages = (200 * 1024) / stage_bytes;
  if (stages > RT_MAX_STAGES) stages = RT_MAX_STAGES;
  const int split = route_split(d.T, d.H);
  const int kblocks = d.H / RT_BK / split;
  if (stages > kblocks) stages = kblocks;
  if (stages < 1) return FMMOE_ERR_UNSUPPORTED;
  int tmem_cols = 32;
  while (tmem_cols < (d.E + 31) / 32 * 32) tmem_cols *= 2;
  // the logits tile [128][32*ceil(E/32)+1] fp32 overlays the stage buffers once the GEMM is done
  size_t tile_bytes = (size_t)stages * stage_bytes;
  const size_t ldl_bytes = (size_t)((d.E + 31) / 32 * 32 + 1) * 4;
  const size_t logit_bytes = RT_BM * ldl_bytes + (split > 1 ? (RT_BM / split) * ldl_bytes + 16 : 0);   // partial tile (+ this CTA's summed rows)
  if (logit_bytes > tile_bytes) tile_bytes = (logit_bytes + 1023) / 1024 * 1024;
  const size_t smem = tile_bytes + FMMOE_MAX_EXPERTS * 20 + (2 * RT_MAX_STAGES + 1) * 8 + 16 + 1024;
  CUtensorMap mx, mw;
  if (!route_map(h, &mx, d.x, (uint64_t)d.T, (uint64_t)d.H, RT_BM)) return FMMOE_ERR_CUDA;
  if (!route_map(h, &mw, d.w, (uint64_t)d.E, (uint64_t)d.H, (uint32_t)d.e_pad)) return FMMOE_ERR_CUDA;
  if (!h->route_attr_set) {   // once per handle: the largest size any shape can ask for
    FMMOE_CUDA_TRY(cudaFuncSetAttribute(route_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, h->max_smem_optin));
    h->route_attr_set = true;
  }
  if (smem > (size_t)h->max_smem_optin) return FMMOE_ERR_UNSUPPORTED;
  const int tiles = (int)((d.T + RT_BM - 1) / RT_BM);
  {
    ProfScope ps(h, FMMOE_KERNEL_ROUTE, s);
    for (int rep = 0; rep < ps.reps; ++rep) {
      FMMOE_CUDA_TRY(launch_pdl(route_tc_kernel, dim3((unsigned)(tiles * split)), dim3(RT_THREADS), smem, s, (unsigned)split, mx, mw, d,
                                stages, tmem_cols, (int)tile_bytes, split, h->d_status));
      h->launches += 1;
    }
  }
  FMMOE_CUDA_TRY(cudaGetLastError());
  return FMMOE_OK;
}

template <int NT>
static fmmoe_status launch_nt(fmmoe_handle* h, const RouteDev& d, int grid, cudaStream_t s) {
  const int e_pad = NT * 32;
  const size_t tail = (size_t)R_BM * (e_pad + 1) * 4 + (size_t)e_pad * 4;
  const size_t smem = (size_t)(R_BM + e_pad) * 33 * 4 + tail;
  if (!(h->route_f32_attr_mask & (1u << NT))) {
    FMMOE_CUDA_TRY(cudaFuncSetAttribute(route_f32_kernel<NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    h->route_f32_attr_mask |= 1u << NT;
  }
  {
    ProfScope ps(h, FMMOE_KERNEL_ROUTE, s);
    for (int rep = 0; rep < ps.reps; ++rep) {
      FMMOE_CUDA_TRY(launch_pdl(route_f32_kernel<NT>, dim3(grid), dim3(R_THREADS), smem, s, 1, d));
      h->launches += 1;
    }
  }
  FMMOE_CUDA_TRY(cudaGetLastError());
  return FMMOE_OK;
}

fmmoe_status launch_route(fmmoe_handle* h, const RouteArgs& a, cudaStream_t s) {
  if (a.T == 0) return FMMOE_OK;
  RouteDev d;
  d.x = a.x; d.w = a.router_w; d.bias = a.router_b; d.is_visual = a.is_visual;
  d.T = a.T; d.H = a.H; d.E = a.E; d.K = a.K; d.Kv = a.Kv; d.reduce_on = a.reduce_on;
  d.e_pad = (a.E + 31) / 32 * 32;
  d.logits = a.logits; d.probs = a.probs; d.topk_idx = a.topk_idx; d.topk_w = a.topk_w;
  d.inv_row = a.inv_row; d.blk_cnt = a.blk_cnt; d.acc_zero = a.acc_zero; d.misc_zero = a.misc_zero;
  d.n_blk = route_num_blocks(a.dtype, a.T, a.H);
  fmmoe_status st;
  if (a.dtype == FMMOE_BF16) {
    st = launch_route_tc(h, d, s);
  } else {
    const int grid = (int)((a.T + R_BM - 1) / R_BM);
    switch (d.e_pad / 32) {
      case 1: st = launch_nt<1>(h, d, grid, s); break;
      case 2: st = launch_nt<2>(h, d, grid, s); break;
      case 3: st = launch_nt<3>(h, d, grid, s); break;
      case 4: st = launch_nt<4>(h, d, grid, s); break;
      case 5: st = launch_nt<5>(h, d, grid, s); break;
      case 6: st = launch_nt<6>(h, d, grid, s); break;
      case 7: st = launch_nt<7>(h, d, grid, s); break;
      case 8: st = launch_nt<8>(h, d, grid, s); break;
      default: return FMMOE_ERR_UNSUPPORTED;
    }
  }
  return st;
}

}  // namespace fmmoe
