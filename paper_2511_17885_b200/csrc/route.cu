// Router: logits (Eq. 1), softmax (Eq. 2), modality-aware top-k (Eq. 3, with K_v
// for vision tokens once the layer has reached l_v) and renormalised gates (Eq. 5),
// fused in one kernel.  A CTA owns 32 tokens: the logits tile [32, E] is formed in
// shared memory (bf16: mma.sync tensor-core tiles fed by a cp.async pipeline; fp32:
// plain FMA), then each warp takes 8 tokens and runs the softmax / top-k / gate
// step across the expert dimension with warp shuffles.  The kernel also adds the
// selections to the per-expert histogram the permutation needs.
#include <cuda_bf16.h>
#include <float.h>

#include "internal.h"

namespace fmmoe {

constexpr int R_BM = 32;
constexpr int R_THREADS = 128;
constexpr int R_BK = 64;
constexpr int R_LDS = R_BK + 8;   // bf16 elements per smem row (144 B: conflict-free ldmatrix)
constexpr int R_STAGES = 3;

struct RouteDev {
  const void* x; const void* w; const float* bias; const uint8_t* is_visual;
  long long T; int H, E, K, Kv, reduce_on, e_pad;
  float* logits; float* probs; int32_t* topk_idx; float* topk_w; int32_t* inv_row; int32_t* counts;
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
__device__ __forceinline__ void route_tail(const float* Ls, int ldl, long long t0, const RouteDev& a, int* hist) {
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
      if (a.inv_row) a.inv_row[t * a.K + lane] = -1;
      if (sel && a.counts) atomicAdd(&hist[my_idx], 1);
    }
  }
}

__device__ __forceinline__ void flush_hist(const int* hist, const RouteDev& a) {
  __syncthreads();
  if (a.counts)
    for (int e = threadIdx.x; e < a.E; e += R_THREADS)
      if (hist[e]) atomicAdd(&a.counts[e], hist[e]);
}

__device__ __forceinline__ void cp_async16(void* smem, const void* gmem) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(smem)), "l"(gmem));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N)); }

// bf16 router.  NT = n8-tiles per warp = e_pad / 32.
template <int NT>
__global__ void __launch_bounds__(R_THREADS) route_bf16_kernel(const RouteDev a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int e_pad = NT * 32;
  const int ldl = e_pad + 1;
  __nv_bfloat16* Xs = reinterpret_cast<__nv_bfloat16*>(smem_raw);                    // [STAGES][R_BM][R_LDS]
  __nv_bfloat16* Ws = Xs + R_STAGES * R_BM * R_LDS;                                   // [STAGES][e_pad][R_LDS]
  float* Ls = reinterpret_cast<float*>(Ws + R_STAGES * e_pad * R_LDS);                // [R_BM][ldl]
  int* hist = reinterpret_cast<int*>(Ls + R_BM * ldl);                                // [e_pad]
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const long long t0 = (long long)blockIdx.x * R_BM;
  const __nv_bfloat16* X = static_cast<const __nv_bfloat16*>(a.x);
  const __nv_bfloat16* W = static_cast<const __nv_bfloat16*>(a.w);

  // rows that are never loaded (tokens >= T, experts >= E) must read as zero
  for (int i = tid; i < R_STAGES * (R_BM + e_pad) * R_LDS / 8; i += R_THREADS)
    reinterpret_cast<uint4*>(smem_raw)[i] = make_uint4(0, 0, 0, 0);
  for (int i = tid; i < e_pad; i += R_THREADS) hist[i] = 0;
  __syncthreads();

  const int kblocks = a.H / R_BK;
  auto load_stage = [&](int st, int kb) {
    const int k0 = kb * R_BK;
    for (int c = tid; c < R_BM * (R_BK / 8); c += R_THREADS) {
      const int r = c >> 3, cc = c & 7;
      if (t0 + r < a.T) cp_async16(Xs + (st * R_BM + r) * R_LDS + cc * 8, X + (t0 + r) * a.H + k0 + cc * 8);
    }
    for (int c = tid; c < a.E * (R_BK / 8); c += R_THREADS) {
      const int r = c >> 3, cc = c & 7;
      cp_async16(Ws + (st * e_pad + r) * R_LDS + cc * 8, W + (long long)r * a.H + k0 + cc * 8);
    }
  };

  float acc[2][NT][4];
#pragma unroll
  for (int mi = 0; mi < 2; ++mi)
#pragma unroll
    for (int ni = 0; ni < NT; ++ni)
#pragma unroll
      for (int q = 0; q < 4; ++q) acc[mi][ni][q] = 0.f;

  for (int s = 0; s < R_STAGES - 1; ++s) {
    if (s < kblocks) load_stage(s, s);
    cp_async_commit();
  }
  for (int kb = 0; kb < kblocks; ++kb) {
    cp_async_wait<R_STAGES - 2>();
    __syncthreads();
    if (kb + R_STAGES - 1 < kblocks) load_stage((kb + R_STAGES - 1) % R_STAGES, kb + R_STAGES - 1);
    cp_async_commit();
    const int st = kb % R_STAGES;
    const __nv_bfloat16* xs = Xs + st * R_BM * R_LDS;
    const __nv_bfloat16* ws = Ws + st * e_pad * R_LDS;
#pragma unroll
    for (int ks = 0; ks < R_BK / 16; ++ks) {
      uint32_t af[2][4];
#pragma unroll
      for (int mi = 0; mi < 2; ++mi) {
        const uint32_t addr = (uint32_t)__cvta_generic_to_shared(xs + (mi * 16 + (lane & 15)) * R_LDS + ks * 16 + (lane >> 4) * 8);
        asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                     : "=r"(af[mi][0]), "=r"(af[mi][1]), "=r"(af[mi][2]), "=r"(af[mi][3]) : "r"(addr));
      }
#pragma unroll
      for (int ni = 0; ni < NT; ++ni) {
        const int n0 = warp * (NT * 8) + ni * 8;
        uint32_t b0, b1;
        const uint32_t addr = (uint32_t)__cvta_generic_to_shared(ws + (n0 + (lane & 7)) * R_LDS + ks * 16 + ((lane >> 3) & 1) * 8);
        asm volatile("ldmatrix.sync.aligned.m8n8.x2.shared.b16 {%0,%1}, [%2];" : "=r"(b0), "=r"(b1) : "r"(addr));
#pragma unroll
        for (int mi = 0; mi < 2; ++mi) {
          asm volatile(
              "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
              : "+f"(acc[mi][ni][0]), "+f"(acc[mi][ni][1]), "+f"(acc[mi][ni][2]), "+f"(acc[mi][ni][3])
              : "r"(af[mi][0]), "r"(af[mi][1]), "r"(af[mi][2]), "r"(af[mi][3]), "r"(b0), "r"(b1));
        }
      }
    }
  }
  cp_async_wait<0>();
  // logits tile (+ bias) to shared memory
  const int g = lane >> 2, tg = lane & 3;
#pragma unroll
  for (int mi = 0; mi < 2; ++mi)
#pragma unroll
    for (int ni = 0; ni < NT; ++ni) {
      const int col = warp * (NT * 8) + ni * 8 + 2 * tg;
      const float b0 = (a.bias && col < a.E) ? a.bias[col] : 0.f;
      const float b1 = (a.bias && col + 1 < a.E) ? a.bias[col + 1] : 0.f;
      Ls[(mi * 16 + g) * ldl + col] = acc[mi][ni][0] + b0;
      Ls[(mi * 16 + g) * ldl + col + 1] = acc[mi][ni][1] + b1;
      Ls[(mi * 16 + g + 8) * ldl + col] = acc[mi][ni][2] + b0;
      Ls[(mi * 16 + g + 8) * ldl + col + 1] = acc[mi][ni][3] + b1;
    }
  __syncthreads();
  route_tail<NT>(Ls, ldl, t0, a, hist);
  flush_hist(hist, a);
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
  int* hist = reinterpret_cast<int*>(Ls + R_BM * ldl);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const long long t0 = (long long)blockIdx.x * R_BM;
  const float* X = static_cast<const float*>(a.x);
  const float* W = static_cast<const float*>(a.w);
  for (int i = tid; i < e_pad; i += R_THREADS) hist[i] = 0;
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
  route_tail<NT>(Ls, ldl, t0, a, hist);
  flush_hist(hist, a);
}

template <int NT>
static fmmoe_status launch_nt(fmmoe_handle* h, const RouteDev& d, int dtype, int grid, cudaStream_t s) {
  const int e_pad = NT * 32;
  const size_t tail = (size_t)R_BM * (e_pad + 1) * 4 + (size_t)e_pad * 4;
  if (dtype == FMMOE_BF16) {
    const size_t smem = (size_t)R_STAGES * (R_BM + e_pad) * R_LDS * 2 + tail;
    FMMOE_CUDA_TRY(cudaFuncSetAttribute(route_bf16_kernel<NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    ProfScope ps(h, FMMOE_KERNEL_ROUTE, s);
    route_bf16_kernel<NT><<<grid, R_THREADS, smem, s>>>(d);
  } else {
    const size_t smem = (size_t)(R_BM + e_pad) * 33 * 4 + tail;
    FMMOE_CUDA_TRY(cudaFuncSetAttribute(route_f32_kernel<NT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem));
    ProfScope ps(h, FMMOE_KERNEL_ROUTE, s);
    route_f32_kernel<NT><<<grid, R_THREADS, smem, s>>>(d);
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
  d.inv_row = a.inv_row; d.counts = a.counts;
  const int grid = (int)((a.T + R_BM - 1) / R_BM);
  fmmoe_status st;
  switch (d.e_pad / 32) {
    case 1: st = launch_nt<1>(h, d, a.dtype, grid, s); break;
    case 2: st = launch_nt<2>(h, d, a.dtype, grid, s); break;
    case 3: st = launch_nt<3>(h, d, a.dtype, grid, s); break;
    case 4: st = launch_nt<4>(h, d, a.dtype, grid, s); break;
    case 5: st = launch_nt<5>(h, d, a.dtype, grid, s); break;
    case 6: st = launch_nt<6>(h, d, a.dtype, grid, s); break;
    case 7: st = launch_nt<7>(h, d, a.dtype, grid, s); break;
    case 8: st = launch_nt<8>(h, d, a.dtype, grid, s); break;
    default: return FMMOE_ERR_UNSUPPORTED;
  }
  if (st == FMMOE_OK) h->launches += 1;
  return st;
}

}  // namespace fmmoe
