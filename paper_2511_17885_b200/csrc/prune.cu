// Routing-aware sliding-window pruning of vision tokens (Section 3.2).
//   vis_index_kernel   : rank of every vision token inside its sequence (scan of the mask)
//   window_score_kernel: per window, routing similarity S (Eq. 8 or Eq. 9-10) and the
//                        attention sum (Eq. 11); one warp per window, fp64 accumulation
//   select_kernel      : per sequence, A_bar (Eq. 12), C (Eq. 13) rounded once to fp32,
//                        merge set = m highest C (Eq. 15), drop set = d smallest A_bar among
//                        the rest (both by an in-CTA bitonic sort of (score, window) keys),
//                        then the stable compaction map (scan of keep flags)
//   compact_kernel     : copies kept rows (a warp per row, four rows per CTA); a merged window becomes
//                        mean(rows) rescaled to the largest member norm (Eq. 16-18) at its first token's
//                        position, formed by the whole CTA
// Ranks come from sorting unique (value, window index) keys, so the keep-set does not depend
// on thread order; ties go to the lower window index.
#include <cuda_bf16.h>
#include <math.h>
#include <pthread.h>

#include "internal.h"
#include "ptx.cuh"

namespace fmmoe {

constexpr int MAXS = FMMOE_MAX_SEQS_PER_LAUNCH;
constexpr int MAXW = FMMOE_MAX_WINDOW;

struct PruneSeqs {
  int n_seq;
  int n_vis[MAXS], m[MAXS], d[MAXS];
  int win_off[MAXS + 1];          // first window of each sequence in this launch
  long long seq_off[MAXS + 1];    // token offsets
  long long out_off[MAXS + 1];    // output row offsets
};

struct PruneDev {
  const float* probs; const float* attn; const void* x; const uint8_t* is_visual;
  int E, H, W, sim_mode, merge_mode, dtype;
  double alpha;
  // workspace
  int32_t* vrank;      // [T] rank of a vision token inside its sequence, -1 for text
  int32_t* vis_list;   // [T] token index of the v-th vision token of sequence b at seq_off[b]+v
  double* sim;         // [windows]
  double* asum;        // [windows]
  // outputs
  void* x_out; uint8_t* is_visual_out; int32_t* keep_idx; uint8_t* kind;
  int32_t* keep_idx_ws; uint8_t* kind_ws;   // always-present copies in the workspace
  int* status;
};

// ------------------------------------------------------------------ vision ranks
__global__ void __launch_bounds__(1024) vis_index_kernel(const PruneDev a, const PruneSeqs sq) {
  __shared__ int s_warp[32];
  __shared__ int s_running;
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  pdl_launch_dependents();
  pdl_wait();
  const long long lo = sq.seq_off[b], hi = sq.seq_off[b + 1];
  if (tid == 0) s_running = 0;
  __syncthreads();
  for (long long t0 = lo; t0 < hi; t0 += 1024) {
    const long long t = t0 + tid;
    const bool v = t < hi && a.is_visual[t] != 0;
    const unsigned bal = __ballot_sync(0xffffffffu, v);
    if (lane == 0) s_warp[warp] = __popc(bal);
    __syncthreads();
    if (warp == 0) {
      int c = s_warp[lane];
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const int n = __shfl_up_sync(0xffffffffu, c, o);
        if (lane >= o) c += n;
      }
      s_warp[lane] = c;
    }
    __syncthreads();
    const int running = s_running;
    if (t < hi) {
      int rank = -1;
      if (v) {
        rank = running + (warp ? s_warp[warp - 1] : 0) + __popc(bal & ((1u << lane) - 1u));
        a.vis_list[lo + rank] = (int32_t)t;
      }
      a.vrank[t] = rank;
    }
    __syncthreads();
    if (tid == 0) s_running = running + s_warp[31];
    __syncthreads();
  }
  // A mask with fewer set bytes than the host's count leaves the tail of this sequence's list unwritten;
  // the scoring and merge kernels index probs and x with these entries, so they must hold a token of the
  // sequence whatever the mask says (the mismatch itself is reported through the status word).
  const int found = s_running;
  for (int i = found + tid; i < sq.n_vis[b]; i += 1024) a.vis_list[lo + i] = (int32_t)lo;
  if (tid == 0 && found != sq.n_vis[b]) atomicCAS(a.status, 0, DEV_INTERNAL);
}

// ------------------------------------------------------------------ window scores
__device__ __forceinline__ double warp_sum_d(double v) {
#pragma unroll
  for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

template <int W>
__device__ __forceinline__ void score_window(const PruneDev& a, const int32_t* members, int lane, double* sim_out,
                                             double* asum_out) {
  // dots[i][j] for j <= i (norms on the diagonal), partial over this lane's experts
  double dots[W * (W + 1) / 2];
#pragma unroll
  for (int i = 0; i < W * (W + 1) / 2; ++i) dots[i] = 0.0;
  const float* rows[W];
#pragma unroll
  for (int i = 0; i < W; ++i) rows[i] = a.probs + (long long)members[i] * a.E;
  for (int e = lane; e < a.E; e += 32) {
    double v[W];
#pragma unroll
    for (int i = 0; i < W; ++i) v[i] = (double)rows[i][e];
    int q = 0;
#pragma unroll
    for (int i = 0; i < W; ++i)
#pragma unroll
      for (int j = 0; j <= i; ++j) { dots[q] = fma(v[i], v[j], dots[q]); ++q; }
  }
#pragma unroll
  for (int i = 0; i < W * (W + 1) / 2; ++i) dots[i] = warp_sum_d(dots[i]);
  // every lane now holds the full dot products
  auto D = [&](int i, int j) { return dots[i * (i + 1) / 2 + j]; };   // j <= i
  double s = 0.0;
  if (a.sim_mode == 0) {
#pragma unroll
    for (int i = 0; i < W; ++i)
#pragma unroll
      for (int j = 0; j < i; ++j) s += D(i, j) / (sqrt(D(i, i)) * sqrt(D(j, j)));
    s = s / (double)(W * (W - 1) / 2);
  } else {
    // mean row rbar = sum(rows)/W:  rows_i . rbar = sum_j D(i,j)/W ;  rbar . rbar = sum_ij D(i,j)/W^2
    double rr = 0.0;
    double rd[W];
#pragma unroll
    for (int i = 0; i < W; ++i) {
      double t = 0.0;
#pragma unroll
      for (int j = 0; j < W; ++j) t += (j <= i) ? D(i, j) : D(j, i);
      rd[i] = t / (double)W;
      rr += t;
    }
    rr = rr / (double)(W * W);
#pragma unroll
    for (int i = 0; i < W; ++i) s += rd[i] / (sqrt(D(i, i)) * sqrt(rr));
    s = s / (double)W;
  }
  double asum = 0.0;
  if (a.attn) {
#pragma unroll
    for (int i = 0; i < W; ++i) asum += (double)a.attn[members[i]];
  }
  if (lane == 0) { *sim_out = s; *asum_out = asum; }
}

__global__ void __launch_bounds__(256) window_score_kernel(const PruneDev a, const PruneSeqs sq) {
  const int lane = threadIdx.x & 31;
  const int gw = blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  pdl_launch_dependents();
  pdl_wait();
  if (gw >= sq.win_off[sq.n_seq]) return;
  int b = 0;
  while (b + 1 < sq.n_seq && gw >= sq.win_off[b + 1]) ++b;
  const int i = gw - sq.win_off[b];
  int32_t members[MAXW];
  const long long s_lo = sq.seq_off[b], s_hi = sq.seq_off[b + 1];
#pragma unroll
  for (int k = 0; k < MAXW; ++k) {
    long long tkn = k < a.W ? a.vis_list[s_lo + (long long)i * a.W + k] : s_lo;
    if (tkn < s_lo || tkn >= s_hi) tkn = s_lo;   // only with a mask that contradicts the host's count (status word set)
    members[k] = (int32_t)tkn;
  }
  switch (a.W) {
    case 2: score_window<2>(a, members, lane, a.sim + gw, a.asum + gw); break;
    case 3: score_window<3>(a, members, lane, a.sim + gw, a.asum + gw); break;
    case 4: score_window<4>(a, members, lane, a.sim + gw, a.asum + gw); break;
    case 5: score_window<5>(a, members, lane, a.sim + gw, a.asum + gw); break;
    case 6: score_window<6>(a, members, lane, a.sim + gw, a.asum + gw); break;
    case 7: score_window<7>(a, members, lane, a.sim + gw, a.asum + gw); break;
    case 8: score_window<8>(a, members, lane, a.sim + gw, a.asum + gw); break;
    default: break;
  }
}

// ------------------------------------------------------------------ select + compaction map
// Order-preserving map float -> uint32 (-0 is folded onto +0 so that equal values tie).
__device__ __forceinline__ uint32_t ordered_bits(float f) {
  if (f == 0.f) f = 0.f;
  const uint32_t u = __float_as_uint(f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// Ascending bitonic sort of n (a power of two) 64-bit keys in shared memory by the whole CTA.
// Keys are unique (the window index is part of them), so the result does not depend on the
// network's comparison order.  One thread per compare-exchange pair; pair p of warp w only ever
// touches elements 64w .. 64w+63 while the partner distance j is <= 32, so those steps need a
// warp barrier only.
__device__ __forceinline__ void bitonic_sort_u64(unsigned long long* keys, int n) {
  const int half = n >> 1;
  for (int k = 2; k <= n; k <<= 1) {
    for (int j = k >> 1; j > 0; j >>= 1) {
      for (int p = threadIdx.x; p < half; p += blockDim.x) {
        const int lo = ((p & ~(j - 1)) << 1) | (p & (j - 1));
        const int hi = lo | j;
        const unsigned long long x = keys[lo], y = keys[hi];
        const bool up = (lo & k) == 0;
        if ((x > y) == up) { keys[lo] = y; keys[hi] = x; }
      }
      if (j > 32 || half > (int)blockDim.x) __syncthreads();
      else __syncwarp();
    }
    if (k >= 64) __syncthreads();   // the next merge starts with partners in other warps' ranges
  }
  __syncthreads();
}

// Ascending bitonic sort of up to 1024 keys, ONE key per thread of a 1024-thread CTA (threads
// past the data hold the maximum key).  Partners less than 32 apart exchange by shuffle, the
// others through `xch` (1024 keys of shared memory).  Returns the key of position threadIdx.x.
__device__ __forceinline__ unsigned long long bitonic_sort_1024_regs(unsigned long long key, int n, unsigned long long* xch) {
  const int tid = threadIdx.x;
  for (int k = 2; k <= n; k <<= 1) {
    for (int j = k >> 1; j > 0; j >>= 1) {
      unsigned long long other;
      if (j < 32) {
        other = __shfl_xor_sync(0xffffffffu, key, j);
      } else {
        xch[tid] = key;
        __syncthreads();
        other = xch[tid ^ j];
        __syncthreads();
      }
      const bool up = (tid & k) == 0;          // this block of k keys sorts ascending
      const bool lower = (tid & j) == 0;       // this thread keeps the smaller of the pair if ascending
      const bool take_min = up == lower;
      key = take_min ? (key < other ? key : other) : (key > other ? key : other);
    }
  }
  return key;
}

// One CTA per sequence.  Eq. 12-13 (one rounding to fp32), then the merge set (Eq. 15) and the
// drop set by SORTING (score, window index) keys: position p of the sorted order is rank p.
__global__ void __launch_bounds__(1024) select_kernel(const PruneDev a, const PruneSeqs sq) {
  extern __shared__ unsigned long long s_keys[];   // [max(n_pad, 1024)] keys, then [n_pad] action bytes
  __shared__ double s_red[32];
  __shared__ int s_warp[32];
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  pdl_launch_dependents();
  pdl_wait();
  const int n_f = sq.n_vis[b] / a.W;
  const int w0 = sq.win_off[b];
  const int m = sq.m[b], d = sq.d[b];
  const bool have_attn = a.attn != nullptr;
  int n_pad = 2;
  while (n_pad < n_f) n_pad <<= 1;
  const bool in_regs = n_pad <= 1024;
  uint8_t* s_action = reinterpret_cast<uint8_t*>(s_keys + (n_pad > 1024 ? n_pad : 1024));   // [n_pad]

  // Eq. 12: divide by the largest window sum (0 if all sums are 0)
  double amax = 0.0;
  if (have_attn) {
    for (int i = tid; i < n_f; i += 1024) amax = fmax(amax, a.asum[w0 + i]);
#pragma unroll
    for (int o = 16; o; o >>= 1) amax = fmax(amax, __shfl_xor_sync(0xffffffffu, amax, o));
    if (lane == 0) s_red[warp] = amax;
    __syncthreads();
    amax = s_red[0];
    for (int i = 1; i < 32; ++i) amax = fmax(amax, s_red[i]);
  }
  // key of the redundancy ranking: (C descending, window ascending); Eq. 13 in fp64 without
  // contraction, then ONE rounding to fp32
  auto c_key = [&](int i) -> unsigned long long {
    if (i >= n_f) return ~0ull;
    const double S = a.sim[w0 + i];
    float c32;
    if (have_attn) {
      const double ab = amax > 0.0 ? a.asum[w0 + i] / amax : 0.0;
      c32 = (float)__dsub_rn(__dmul_rn(a.alpha, S), __dmul_rn(__dsub_rn(1.0, a.alpha), ab));
    } else {
      c32 = (float)S;
    }
    return ((unsigned long long)(~ordered_bits(c32)) << 32) | (unsigned)i;
  };
  // key of the drop ranking among the windows that were not merged: (A_bar ascending, window ascending)
  auto a_key = [&](int i) -> unsigned long long {
    if (i >= n_f || s_action[i] != 0) return ~0ull;
    const float a32 = (float)(amax > 0.0 ? a.asum[w0 + i] / amax : 0.0);
    return ((unsigned long long)ordered_bits(a32) << 32) | (unsigned)i;
  };
  for (int i = tid; i < n_pad; i += 1024) s_action[i] = 0;
  __syncthreads();
  if (m + d > 0) {
    const int n_act = have_attn ? m : m + d;
    if (in_regs) {
      const unsigned long long k = bitonic_sort_1024_regs(c_key(tid), n_pad, s_keys);
      if (tid < n_act && tid < n_f) s_action[(int)(k & 0xffffffffu)] = tid < m ? 1 : 2;
    } else {
      for (int i = tid; i < n_pad; i += 1024) s_keys[i] = c_key(i);
      __syncthreads();
      bitonic_sort_u64(s_keys, n_pad);
      for (int p = tid; p < n_act && p < n_f; p += 1024) s_action[(int)(s_keys[p] & 0xffffffffu)] = p < m ? 1 : 2;
    }
    __syncthreads();
    if (have_attn && d > 0) {
      if (in_regs) {
        const unsigned long long k = bitonic_sort_1024_regs(a_key(tid), n_pad, s_keys);
        __syncthreads();
        if (tid < d && tid < n_f - m) s_action[(int)(k & 0xffffffffu)] = 2;
      } else {
        for (int i = tid; i < n_pad; i += 1024) s_keys[i] = a_key(i);
        __syncthreads();
        bitonic_sort_u64(s_keys, n_pad);
        for (int p = tid; p < d && p < n_f - m; p += 1024) s_action[(int)(s_keys[p] & 0xffffffffu)] = 2;
      }
      __syncthreads();
    }
  }

  // stable compaction map over the sequence's tokens: every thread owns a run of consecutive tokens
  const long long lo = sq.seq_off[b], hi = sq.seq_off[b + 1];
  const int per = (int)((hi - lo + 1023) / 1024);
  const long long t_begin = lo + (long long)tid * per;
  auto kind_of = [&](int v) -> int {   // kind of the emitted row for a token of vision rank v, -1 = nothing emitted
    if (v < 0) return 0;
    const int w = v / a.W;
    if (w >= n_f) return 1;
    const uint8_t act = s_action[w];
    if (act == 0) return 1;
    return (act == 1 && v - w * a.W == 0) ? 2 : -1;
  };
  constexpr int CACHE = 8;             // kinds of the first tokens of the run stay in registers
  int kinds[CACHE];
#pragma unroll
  for (int i = 0; i < CACHE; ++i) {
    const long long t = t_begin + i;
    kinds[i] = (i < per && t < hi) ? a.vrank[t] : -2;      // independent loads first
  }
  int cnt = 0;
#pragma unroll
  for (int i = 0; i < CACHE; ++i) {
    kinds[i] = kinds[i] == -2 ? -1 : kind_of(kinds[i]);
    cnt += kinds[i] >= 0;
  }
  for (int i = CACHE; i < per; ++i) {
    const long long t = t_begin + i;
    if (t < hi && kind_of(a.vrank[t]) >= 0) ++cnt;
  }
  int incl = cnt;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int n = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += n;
  }
  if (lane == 31) s_warp[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    int c = s_warp[lane];
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int n = __shfl_up_sync(0xffffffffu, c, o);
      if (lane >= o) c += n;
    }
    s_warp[lane] = c;
  }
  __syncthreads();
  long long pos = sq.out_off[b] + (warp ? s_warp[warp - 1] : 0) + (incl - cnt);
  auto emit = [&](long long t, int kd) {
    if (pos < sq.out_off[b + 1]) {
      a.keep_idx_ws[pos] = (int32_t)t;
      a.kind_ws[pos] = (uint8_t)kd;
      if (a.keep_idx) a.keep_idx[pos] = (int32_t)t;
      if (a.kind) a.kind[pos] = (uint8_t)kd;
      if (a.is_visual_out) a.is_visual_out[pos] = kd != 0;
    }
    ++pos;
  };
#pragma unroll
  for (int i = 0; i < CACHE; ++i)
    if (kinds[i] >= 0) emit(t_begin + i, kinds[i]);
  for (int i = CACHE; i < per; ++i) {
    const long long t = t_begin + i;
    if (t >= hi) break;
    const int kd = kind_of(a.vrank[t]);
    if (kd >= 0) emit(t, kd);
  }
  if (tid == 0 && s_warp[31] != (int)(sq.out_off[b + 1] - sq.out_off[b])) atomicCAS(a.status, 0, DEV_INTERNAL);
}

// ------------------------------------------------------------------ gather / merge rows
template <typename T> struct Row8;   // 8 elements (bf16) or 4 elements (fp32) per 16 bytes
template <> struct Row8<__nv_bfloat16> {
  static constexpr int N = 8;
  static __device__ __forceinline__ void load(const __nv_bfloat16* p, float* f) {
    const uint4 u = *reinterpret_cast<const uint4*>(p);
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 v = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&w[i]));
      f[2 * i] = v.x; f[2 * i + 1] = v.y;
    }
  }
  static __device__ __forceinline__ void store(__nv_bfloat16* p, const float* f) {
    uint32_t w[4];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const __nv_bfloat162 h = __floats2bfloat162_rn(f[2 * i], f[2 * i + 1]);
      w[i] = *reinterpret_cast<const uint32_t*>(&h);
    }
    *reinterpret_cast<uint4*>(p) = make_uint4(w[0], w[1], w[2], w[3]);
  }
};
template <> struct Row8<float> {
  static constexpr int N = 4;
  static __device__ __forceinline__ void load(const float* p, float* f) {
    const float4 v = *reinterpret_cast<const float4*>(p);
    f[0] = v.x; f[1] = v.y; f[2] = v.z; f[3] = v.w;
  }
  static __device__ __forceinline__ void store(float* p, const float* f) {
    *reinterpret_cast<float4*>(p) = make_float4(f[0], f[1], f[2], f[3]);
  }
};

// Rows per CTA of compact_kernel: one warp copies one kept row (the common case: with the paper's merge
// rates about 3 % of the output rows are merged windows), then the whole CTA forms the block's merged rows
// one after another, so that a merge still has 256 threads behind it.  Four rows per CTA (warps 0-3 copy):
// a CTA then rarely holds more than one merged row, whose dependent steps set the kernel's duration
// (measured 23.9 / 10.2 us with four, 26.9 / 15.2 us with eight and 25.2 / 10.1 us with two rows per CTA on
// 14,336 / 2,432 tokens).
constexpr int CP_ROWS = 4;

template <typename T>
__global__ void __launch_bounds__(256) compact_kernel(const PruneDev a, const PruneSeqs sq, long long row_base, long long n_rows) {
  constexpr int N = Row8<T>::N;
  __shared__ float s_red[8][MAXW + 1];
  __shared__ float s_scale;
  __shared__ unsigned s_merged;                  // bit w: row w of this block is a merged window
  __shared__ long long s_mem[CP_ROWS][MAXW];     // member tokens of the block's merged rows (validated)
  pdl_launch_dependents();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  if (tid == 0) s_merged = 0;
  __syncthreads();
  pdl_wait();
  const T* X = static_cast<const T*>(a.x);
  const int vec = a.H / N;                       // 16-byte pieces per row
  const long long blk_row0 = (long long)blockIdx.x * CP_ROWS;
  // ---- phase 1: warp w copies row blk_row0 + w (all loads of a row in flight before its stores)
  int my_kind = -1;
  {
    const long long rel = blk_row0 + warp;
    if (warp < CP_ROWS && rel < n_rows) {
      const long long row = row_base + rel;
      int b = 0;
      while (b + 1 < sq.n_seq && row >= sq.out_off[b + 1]) ++b;
      const long long t0 = a.keep_idx_ws[row];
      my_kind = a.kind_ws[row];
      uint4* dst = reinterpret_cast<uint4*>(static_cast<T*>(a.x_out) + row * a.H);
      if (t0 < sq.seq_off[b] || t0 >= sq.seq_off[b + 1]) {
        // a slot the selection pass did not fill: only possible when the mask contradicts the host's vision
        // count (reported through the status word).  Never index x with it.
        for (int i = lane; i < vec; i += 32) dst[i] = make_uint4(0u, 0u, 0u, 0u);
        my_kind = -1;
      } else if (my_kind == 2) {
        // a merged window: look its member tokens up now, so that the dependent index loads are behind the
        // block's copies when the whole CTA turns to this row
        int v0 = a.vrank[t0];
        if (v0 < 0 || v0 + a.W > sq.n_vis[b]) v0 = 0;   // inconsistent mask / count (status word set): stay inside the list
        const long long s_lo = sq.seq_off[b], s_hi = sq.seq_off[b + 1];
        if (lane < MAXW) {
          long long tkn = lane < a.W ? a.vis_list[s_lo + v0 + lane] : s_lo;
          if (tkn < s_lo || tkn >= s_hi) tkn = s_lo;
          s_mem[warp][lane] = tkn;
        }
      } else {
        const uint4* src = reinterpret_cast<const uint4*>(X + t0 * a.H);
        for (int i0 = 0; i0 < vec; i0 += 256) {
          uint4 v[8];
#pragma unroll
          for (int u = 0; u < 8; ++u) { const int i = i0 + u * 32 + lane; if (i < vec) v[u] = src[i]; }
#pragma unroll
          for (int u = 0; u < 8; ++u) { const int i = i0 + u * 32 + lane; if (i < vec) dst[i] = v[u]; }
        }
      }
    }
  }
  // ---- phase 2: the block's merged rows, one at a time, by the whole CTA
  if (lane == 0 && my_kind == 2) atomicOr(&s_merged, 1u << warp);
  __syncthreads();
  const unsigned merged_mask = s_merged;
  for (int w = 0; w < CP_ROWS; ++w) {
    if (!((merged_mask >> w) & 1)) continue;
    const long long row = row_base + blk_row0 + w;
    T* O = static_cast<T*>(a.x_out) + row * a.H;
    long long mem[MAXW];
#pragma unroll
    for (int k = 0; k < MAXW; ++k) mem[k] = s_mem[w][k];
    const float invW = 1.f / (float)a.W;
    float part[MAXW + 1];
#pragma unroll
    for (int k = 0; k <= MAXW; ++k) part[k] = 0.f;
    if (vec <= 256) {
      // One 16-byte piece per thread and member row: the W pieces stay in registers between the norm pass and
      // the store, so the member rows are read once (the same sums in the same order as the two-pass form below).
      float mean[N];
#pragma unroll
      for (int j = 0; j < N; ++j) mean[j] = 0.f;
      if (tid < vec) {
#pragma unroll
        for (int k = 0; k < MAXW; ++k) {
          if (k < a.W) {
            float f[N];
            Row8<T>::load(X + mem[k] * a.H + tid * N, f);
#pragma unroll
            for (int j = 0; j < N; ++j) { part[k] = fmaf(f[j], f[j], part[k]); mean[j] += f[j]; }
          }
        }
#pragma unroll
        for (int j = 0; j < N; ++j) { const float mv = mean[j] * invW; part[MAXW] = fmaf(mv, mv, part[MAXW]); }
      }
#pragma unroll
      for (int k = 0; k <= MAXW; ++k) {
        float v = part[k];
#pragma unroll
        for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
        if (lane == 0) s_red[warp][k] = v;
      }
      __syncthreads();
      if (tid == 0) {
        float tot[MAXW + 1];
        for (int k = 0; k <= MAXW; ++k) { tot[k] = 0.f; for (int ww = 0; ww < 8; ++ww) tot[k] += s_red[ww][k]; }
        float nmax = 0.f;
        for (int k = 0; k < a.W; ++k) nmax = fmaxf(nmax, sqrtf(tot[k]));
        const float nb = sqrtf(tot[MAXW]);
        s_scale = a.merge_mode == 1 ? 1.f : (nb > 0.f ? nmax / nb : 0.f);   // Eq. 18
      }
      __syncthreads();
      if (tid < vec) {
        const float scale = s_scale * invW;
#pragma unroll
        for (int j = 0; j < N; ++j) mean[j] *= scale;
        Row8<T>::store(O + tid * N, mean);
      }
      __syncthreads();   // s_red / s_scale are reused by the block's next merged row
      continue;
    }
    // pass 1: squared norms of the members and of the mean
    for (int i = tid; i < vec; i += 256) {
      float mean[N];
#pragma unroll
      for (int j = 0; j < N; ++j) mean[j] = 0.f;
#pragma unroll
      for (int k = 0; k < MAXW; ++k) {
        if (k < a.W) {
          float f[N];
          Row8<T>::load(X + mem[k] * a.H + i * N, f);
#pragma unroll
          for (int j = 0; j < N; ++j) { part[k] = fmaf(f[j], f[j], part[k]); mean[j] += f[j]; }
        }
      }
#pragma unroll
      for (int j = 0; j < N; ++j) { const float mv = mean[j] * invW; part[MAXW] = fmaf(mv, mv, part[MAXW]); }
    }
#pragma unroll
    for (int k = 0; k <= MAXW; ++k) {
      float v = part[k];
#pragma unroll
      for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      if (lane == 0) s_red[warp][k] = v;
    }
    __syncthreads();
    if (tid == 0) {
      float tot[MAXW + 1];
      for (int k = 0; k <= MAXW; ++k) { tot[k] = 0.f; for (int ww = 0; ww < 8; ++ww) tot[k] += s_red[ww][k]; }
      float nmax = 0.f;
      for (int k = 0; k < a.W; ++k) nmax = fmaxf(nmax, sqrtf(tot[k]));
      const float nb = sqrtf(tot[MAXW]);
      s_scale = a.merge_mode == 1 ? 1.f : (nb > 0.f ? nmax / nb : 0.f);   // Eq. 18
    }
    __syncthreads();
    const float scale = s_scale * invW;
    for (int i = tid; i < vec; i += 256) {
      float mean[N];
#pragma unroll
      for (int j = 0; j < N; ++j) mean[j] = 0.f;
#pragma unroll
      for (int k = 0; k < MAXW; ++k) {
        if (k < a.W) {
          float f[N];
          Row8<T>::load(X + mem[k] * a.H + i * N, f);
#pragma unroll
          for (int j = 0; j < N; ++j) mean[j] += f[j];
        }
      }
#pragma unroll
      for (int j = 0; j < N; ++j) mean[j] *= scale;
      Row8<T>::store(O + i * N, mean);
    }
    __syncthreads();   // s_red / s_scale are reused by the block's next merged row
  }
}

static int64_t counts_for(int64_t n_vis, int64_t n_retain, const fmmoe_prune_params* p, int64_t* m_out, int64_t* d_out) {
  const int64_t W = p->window;
  const int64_t eps = n_vis - n_retain;
  const int64_t n_f = n_vis / W;
  int64_t m = 0, d = 0;
  if (!(n_retain >= n_vis || eps <= W)) {
    if (p->merge_mode != 2) {
      m = (int64_t)floor((double)n_retain * p->gamma + 1e-9);
      if (m > eps / (W - 1)) m = eps / (W - 1);
      if (m > n_f) m = n_f;
      if (m < 0) m = 0;
    }
    const int64_t u = eps - m * (W - 1);
    d = u / W;
    if (d > n_f - m) d = n_f - m;
  }
  if (m_out) *m_out = m;
  if (d_out) *d_out = d;
  return n_vis - m * (W - 1) - d * W;
}

}  // namespace fmmoe

using namespace fmmoe;

static bool prune_params_ok(const fmmoe_prune_params* p) {
  return p && p->window >= 2 && p->window <= FMMOE_MAX_WINDOW && p->sim_mode >= 0 && p->sim_mode <= 1 &&
         p->merge_mode >= 0 && p->merge_mode <= 2 && p->alpha >= 0.0 && p->alpha <= 1.0 && p->gamma >= 0.0;
}

extern "C" __attribute__((visibility("default"))) int64_t fmmoe_prune_kept_count(int64_t n_vis, int64_t n_retain, const fmmoe_prune_params* p,
                                          int64_t* n_merge, int64_t* n_drop) {
  if (!prune_params_ok(p) || n_vis < 0 || n_retain < 0) return -1;
  return counts_for(n_vis, n_retain, p, n_merge, n_drop);
}

namespace {
struct PruneWs { size_t vrank, vis_list, sim, asum, keep_idx, kind, total; };
PruneWs plan_prune(int64_t T) {
  PruneWs w; size_t o = 0;
  const size_t nw = (size_t)T / 2 + 1;
  w.vrank = o; o = align_up(o + (size_t)T * 4, 256);
  w.vis_list = o; o = align_up(o + (size_t)T * 4, 256);
  w.sim = o; o = align_up(o + nw * 8, 256);
  w.asum = o; o = align_up(o + nw * 8, 256);
  w.keep_idx = o; o = align_up(o + (size_t)T * 4, 256);
  w.kind = o; o = align_up(o + (size_t)T, 256);
  w.total = o;
  return w;
}
}  // namespace

extern "C" __attribute__((visibility("default"))) size_t fmmoe_prune_workspace_bytes(int64_t n_tokens, int32_t n_seq) {
  (void)n_seq;
  if (n_tokens < 0) return 0;
  return plan_prune(n_tokens).total + 256;
}

// The pruning pass in two phases: phase 1 (vision ranks, window scores, selection + compaction map)
// needs the routing probabilities and the mask only, phase 2 (row gather / merge) needs the rows.
// phases & 1 enqueues phase 1 on s_select, phases & 2 enqueues phase 2 on s_rows.  A caller that
// uses two streams orders phase 2 after phase 1 itself.
fmmoe_status fmmoe::prune_visual_phases(fmmoe_handle* h, const fmmoe_prune_params* p, const float* probs,
                                        int32_t n_experts, const float* attn, const void* x, int32_t dtype,
                                        int32_t hidden, const uint8_t* is_visual, const int64_t* seq_off,
                                        const int64_t* n_vis, const int64_t* n_retain, int32_t n_seq, void* x_out,
                                        uint8_t* is_visual_out, int32_t* keep_idx, uint8_t* kind,
                                        int64_t* out_seq_off, void* workspace, size_t workspace_bytes,
                                        int phases, cudaStream_t s_select, cudaStream_t s_rows) {
  if (!h || !prune_params_ok(p) || !seq_off || !n_vis || !n_retain || !out_seq_off || n_seq < 0)
    return FMMOE_ERR_INVALID_ARG;
  if (n_experts < 1 || hidden < 1 || (dtype != FMMOE_F32 && dtype != FMMOE_BF16)) return FMMOE_ERR_INVALID_ARG;
  const int elem = dtype == FMMOE_BF16 ? 2 : 4;
  if ((hidden * elem) % 16 != 0) return FMMOE_ERR_UNSUPPORTED;
  int64_t max_nf = 0;
  out_seq_off[0] = 0;
  for (int b = 0; b < n_seq; ++b) {
    const int64_t L = seq_off[b + 1] - seq_off[b];
    if (L < 0 || n_vis[b] < 0 || n_vis[b] > L || n_retain[b] < 0) return FMMOE_ERR_INVALID_ARG;
    const int64_t kept = counts_for(n_vis[b], n_retain[b], p, nullptr, nullptr);
    out_seq_off[b + 1] = out_seq_off[b] + (L - n_vis[b]) + kept;
    if (n_vis[b] / p->window > max_nf) max_nf = n_vis[b] / p->window;
  }
  const int64_t T = n_seq ? seq_off[n_seq] : 0;
  if (n_seq && seq_off[0] != 0) return FMMOE_ERR_INVALID_ARG;
  if (T > 0x7fffffff) return FMMOE_ERR_UNSUPPORTED;
  if (T == 0) return FMMOE_OK;
  const int64_t T_out = out_seq_off[n_seq];
  if (!probs || !x || !is_visual || (T_out > 0 && !x_out)) return FMMOE_ERR_INVALID_ARG;
  if (x == x_out) return FMMOE_ERR_INVALID_ARG;
  if (((uintptr_t)x | (uintptr_t)x_out | (uintptr_t)probs) & 15) return FMMOE_ERR_INVALID_ARG;
  const PruneWs wp = plan_prune(T);
  if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < wp.total) return FMMOE_ERR_WORKSPACE;
  size_t sel_pad = 2;
  while ((int64_t)sel_pad < max_nf) sel_pad <<= 1;
  const size_t sel_smem = (sel_pad > 1024 ? sel_pad : 1024) * 8 + sel_pad;   // sort keys + action bytes of the longest sequence
  if (sel_smem > (size_t)h->max_smem_optin - 1024) return FMMOE_ERR_UNSUPPORTED;
  char* ws = static_cast<char*>(workspace);

  PruneDev a = {};
  a.probs = probs; a.attn = attn; a.x = x; a.is_visual = is_visual;
  a.E = n_experts; a.H = hidden; a.W = p->window; a.sim_mode = p->sim_mode; a.merge_mode = p->merge_mode;
  a.dtype = dtype; a.alpha = p->alpha;
  a.vrank = reinterpret_cast<int32_t*>(ws + wp.vrank); a.vis_list = reinterpret_cast<int32_t*>(ws + wp.vis_list);
  a.sim = reinterpret_cast<double*>(ws + wp.sim); a.asum = reinterpret_cast<double*>(ws + wp.asum);
  a.keep_idx_ws = reinterpret_cast<int32_t*>(ws + wp.keep_idx); a.kind_ws = reinterpret_cast<uint8_t*>(ws + wp.kind);
  a.x_out = x_out; a.is_visual_out = is_visual_out; a.keep_idx = keep_idx; a.kind = kind;
  a.status = h->d_status;

  // select_kernel's dynamic shared-memory opt-in was raised to the device's maximum once, in fmmoe_create

  int win_base = 0;
  for (int b0 = 0; b0 < n_seq; b0 += MAXS) {
    const int nb = n_seq - b0 < MAXS ? n_seq - b0 : MAXS;
    PruneSeqs sq = {};
    sq.n_seq = nb;
    sq.win_off[0] = win_base;
    for (int i = 0; i < nb; ++i) {
      const int b = b0 + i;
      int64_t m, d;
      counts_for(n_vis[b], n_retain[b], p, &m, &d);
      sq.n_vis[i] = (int)n_vis[b]; sq.m[i] = (int)m; sq.d[i] = (int)d;
      sq.win_off[i + 1] = sq.win_off[i] + (int)(n_vis[b] / p->window);
      sq.seq_off[i] = seq_off[b]; sq.out_off[i] = out_seq_off[b];
    }
    sq.seq_off[nb] = seq_off[b0 + nb]; sq.out_off[nb] = out_seq_off[b0 + nb];
    const int n_win = sq.win_off[nb] - win_base;
    // window ids inside a launch are relative to the launch's first window
    PruneSeqs rel = sq;
    for (int i = 0; i <= nb; ++i) rel.win_off[i] -= win_base;
    PruneDev al = a;
    al.sim = a.sim + win_base; al.asum = a.asum + win_base;
    if (phases & 1) {
      cudaStream_t s = s_select;
      {
        ProfScope ps(h, FMMOE_KERNEL_PRUNE_INDEX, s);
        for (int rep = 0; rep < ps.reps; ++rep, ++h->launches)
          FMMOE_CUDA_TRY(launch_pdl(vis_index_kernel, dim3(nb), dim3(1024), 0, s, 1, al, rel));
      }
      FMMOE_CUDA_TRY(cudaGetLastError());
      if (n_win > 0) {
        ProfScope ps(h, FMMOE_KERNEL_PRUNE_SCORE, s);
        for (int rep = 0; rep < ps.reps; ++rep, ++h->launches)
          FMMOE_CUDA_TRY(launch_pdl(window_score_kernel, dim3((n_win + 7) / 8), dim3(256), 0, s, 1, al, rel));
      }
      FMMOE_CUDA_TRY(cudaGetLastError());
      {
        ProfScope ps(h, FMMOE_KERNEL_PRUNE_SELECT, s);
        for (int rep = 0; rep < ps.reps; ++rep, ++h->launches)
          FMMOE_CUDA_TRY(launch_pdl(select_kernel, dim3(nb), dim3(1024), sel_smem, s, 1, al, rel));
      }
      FMMOE_CUDA_TRY(cudaGetLastError());
    }
    const long long rows = rel.out_off[nb] - rel.out_off[0];
    if ((phases & 2) && rows > 0) {
      cudaStream_t s = s_rows;
      ProfScope ps(h, FMMOE_KERNEL_PRUNE_COMPACT, s);
      for (int rep = 0; rep < ps.reps; ++rep, ++h->launches) {
        if (dtype == FMMOE_BF16)
          FMMOE_CUDA_TRY(launch_pdl(compact_kernel<__nv_bfloat16>, dim3((unsigned)((rows + CP_ROWS - 1) / CP_ROWS)), dim3(256), 0, s, 1, al, rel, (long long)rel.out_off[0], (long long)rows));
        else
          FMMOE_CUDA_TRY(launch_pdl(compact_kernel<float>, dim3((unsigned)((rows + CP_ROWS - 1) / CP_ROWS)), dim3(256), 0, s, 1, al, rel, (long long)rel.out_off[0], (long long)rows));
      }
      FMMOE_CUDA_TRY(cudaGetLastError());
    }
    win_base += n_win;
  }
  return FMMOE_OK;
}

extern "C" __attribute__((visibility("default"))) fmmoe_status fmmoe_prune_visual(fmmoe_handle* h, const fmmoe_prune_params* p, const float* probs,
                                           int32_t n_experts, const float* attn, const void* x, int32_t dtype,
                                           int32_t hidden, const uint8_t* is_visual, const int64_t* seq_off,
                                           const int64_t* n_vis, const int64_t* n_retain, int32_t n_seq, void* x_out,
                                           uint8_t* is_visual_out, int32_t* keep_idx, uint8_t* kind,
                                           int64_t* out_seq_off, void* workspace, size_t workspace_bytes,
                                           void* cuda_stream) {
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  return prune_visual_phases(h, p, probs, n_experts, attn, x, dtype, hidden, is_visual, seq_off, n_vis, n_retain, n_seq,
                             x_out, is_visual_out, keep_idx, kind, out_seq_off, workspace, workspace_bytes, 3, s, s);
}

// ---------------------------------------------------------------------------------------
// fmmoe_prune_visual_static: the same pruning pass, with its scratch memory built into the
// library instead of supplied by the caller.
//
// Who needs it: code that must not ask the CUDA allocator for anything at the point where
// it prunes.  Examples are an inference server whose whole HBM budget was handed to another
// memory pool at start-up (a late cudaMalloc there fails or fragments the pool), and a
// latency-critical loop that cannot afford the device-wide synchronisation an allocation
// or a free may imply.  Such a caller still owns its inputs and outputs (they come from
// its pool); what it cannot do is size and carve out a workspace per call.
//
// The scratch is the file-scope device array below.  Every GPU on which the library is
// loaded holds these FMMOE_STATIC_PRUNE_SCRATCH_BYTES until the process exits.  In host
// code the array's name is only a stand-in for the symbol, never a device address, so the
// address is looked up with cudaGetSymbolAddress once per device (with that device
// current) and cached; kernels receive the looked-up pointer.
// ---------------------------------------------------------------------------------------
#define FMMOE_STATIC_PRUNE_SCRATCH_BYTES (768u * 1024u)
static __device__ __align__(256) unsigned char g_prune_scratch[FMMOE_STATIC_PRUNE_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
void* g_prune_scratch_addr[kMaxDevices] = {};     // device address of g_prune_scratch, per device
pthread_mutex_t g_prune_scratch_mu = PTHREAD_MUTEX_INITIALIZER;

// Device address of the scratch array on the CURRENT device (must be `device`); looked up on
// the first call for that device, cached afterwards.  Returns nullptr on failure.
void* static_scratch_for(int device) {
  if (device < 0 || device >= kMaxDevices) return nullptr;
  pthread_mutex_lock(&g_prune_scratch_mu);
  void* p = g_prune_scratch_addr[device];
  if (!p) {
    void* q = nullptr;
    if (cudaGetSymbolAddress(&q, g_prune_scratch) == cudaSuccess && q) {
      g_prune_scratch_addr[device] = q;
      p = q;
    }
  }
  pthread_mutex_unlock(&g_prune_scratch_mu);
  return p;
}
}  // namespace

// Called by fmmoe_create with the handle's device current.  Everything the pruning pass would
// otherwise do lazily on its first call happens here, at start-up, while the process can still
// obtain device memory: the module that holds the pruning kernels and the scratch array is loaded
// (under lazy module loading that is when the array and the kernel code are placed in device
// memory), the array's device address is looked up and cached, and select_kernel's dynamic
// shared-memory limit is raised once to the device's maximum, so that no later call has to.
fmmoe_status fmmoe::prune_prepare(fmmoe_handle* h) {
  cudaFuncAttributes fa;
  FMMOE_CUDA_TRY(cudaFuncGetAttributes(&fa, vis_index_kernel));
  FMMOE_CUDA_TRY(cudaFuncGetAttributes(&fa, window_score_kernel));
  FMMOE_CUDA_TRY(cudaFuncGetAttributes(&fa, select_kernel));
  FMMOE_CUDA_TRY(cudaFuncGetAttributes(&fa, compact_kernel<__nv_bfloat16>));
  FMMOE_CUDA_TRY(cudaFuncGetAttributes(&fa, compact_kernel<float>));
  FMMOE_CUDA_TRY(cudaFuncGetAttributes(&fa, select_kernel));
  FMMOE_CUDA_TRY(cudaFuncSetAttribute(select_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                      h->max_smem_optin - (int)fa.sharedSizeBytes));
  if (!static_scratch_for(h->device)) return FMMOE_ERR_CUDA;
  return FMMOE_OK;
}

extern "C" __attribute__((visibility("default"))) fmmoe_status fmmoe_prune_visual_static(
    fmmoe_handle* h, const fmmoe_prune_params* p, const float* probs, int32_t n_experts, const float* attn,
    const void* x, int32_t dtype, int32_t hidden, const uint8_t* is_visual, const int64_t* seq_off,
    const int64_t* n_vis, const int64_t* n_retain, int32_t n_seq, void* x_out, uint8_t* is_visual_out,
    int32_t* keep_idx, uint8_t* kind, int64_t* out_seq_off, void* cuda_stream) {
  if (!h || !seq_off || n_seq < 0) return FMMOE_ERR_INVALID_ARG;
  const int64_t T = n_seq ? seq_off[n_seq] : 0;
  if (T < 0) return FMMOE_ERR_INVALID_ARG;
  // the limit is on the token count: refuse before touching the GPU
  if (T > FMMOE_STATIC_PRUNE_MAX_TOKENS) return FMMOE_ERR_TOO_LARGE;
  const size_t need = plan_prune(T).total;
  if (need > (size_t)FMMOE_STATIC_PRUNE_SCRATCH_BYTES) return FMMOE_ERR_TOO_LARGE;
  int cur = -1;
  if (cudaGetDevice(&cur) != cudaSuccess) return FMMOE_ERR_CUDA;
  if (cur != h->device) return FMMOE_ERR_INVALID_ARG;   // the handle's device must be current
  void* scratch = static_scratch_for(cur);
  if (!scratch) return FMMOE_ERR_CUDA;
  // Nothing in the scratch has to start at zero: a pass writes the vision ranks and lists, the
  // window scores and the compaction map before it reads them.  The one exception is a call
  // whose mask contradicts its n_vis: slots the pass then leaves unwritten hold the previous
  // call's values; the kernels range-check every index they take from the scratch, and the
  // mismatch is reported through the status word.
  return fmmoe_prune_visual(h, p, probs, n_experts, attn, x, dtype, hidden, is_visual, seq_off, n_vis, n_retain,
                            n_seq, x_out, is_visual_out, keep_idx, kind, out_seq_off, scratch,
                            (size_t)FMMOE_STATIC_PRUNE_SCRATCH_BYTES, cuda_stream);
}
