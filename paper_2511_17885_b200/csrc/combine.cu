// Last step of Eq. 4: turn the fp32 combine result into the layer output.
// Atomic mode: the GEMM-2 epilogue has already summed g_j * FFN_j(x) and the shared
// experts into `acc`; this kernel adds the residual (optional) and rounds to the
// storage type.  Deterministic mode: the per-pair outputs y were stored instead and
// are summed here in a fixed order (slots 0..K-1, then shared experts 0..N_s-1).
#include <cuda_bf16.h>

#include "internal.h"
#include "ptx.cuh"

namespace fmmoe {

struct FinalizeDev {
  const void* x; void* out; long long T; int H, K, n_shared, add_residual, deterministic;
  const float* acc; const float* y; const float* ysh; const int32_t* inv_row; const float* topk_w;
  const __nv_bfloat16* yb; const __nv_bfloat16* ybsh;
};

__device__ __forceinline__ void add_bf16x8(float (&v)[8], const uint4 u) {
  const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const float2 f = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&w[i]));
    v[2 * i] += f.x; v[2 * i + 1] += f.y;
  }
}

// Pair-row mode (bf16 layers, large batches): GEMM-2 wrote every pair's gate-scaled output row once, in bf16.
// out[t] = sum over the token's slots 0..K-1 (its rows through inv_row), then the shared experts 0..N_s-1,
// then the residual, in that fixed order in fp32; one rounding to bf16.  No atomics anywhere, so the result is
// reproducible bit for bit.  A thread owns 8 neighbouring columns of one token: the rows' 16-byte pieces are
// independent loads.
template <int KK>
__global__ void __launch_bounds__(256) finalize_pair_kernel(const FinalizeDev a) {
  pdl_launch_dependents();
  pdl_wait();
  const int hv = a.H / 8;
  const long long n = a.T * hv;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
    const long long t = i / hv;
    const int c = (int)(i - t * hv) * 8;
    // every row index first, then every row piece (KK independent 16-byte loads in flight), then the sum in slot order
    int rows[KK];
#pragma unroll
    for (int s = 0; s < KK; ++s) rows[s] = a.inv_row[t * KK + s];
    uint4 q[KK];
#pragma unroll
    for (int s = 0; s < KK; ++s)      // a padded slot (-1) reads row 0 and is not added
      q[s] = *reinterpret_cast<const uint4*>(a.yb + (long long)(rows[s] < 0 ? 0 : rows[s]) * a.H + c);
    float v[8];
#pragma unroll
    for (int j = 0; j < 8; ++j) v[j] = 0.f;
#pragma unroll
    for (int s = 0; s < KK; ++s)
      if (rows[s] >= 0) add_bf16x8(v, q[s]);
    for (int s = 0; s < a.n_shared; ++s)
      add_bf16x8(v, *reinterpret_cast<const uint4*>(a.ybsh + ((long long)s * a.T + t) * a.H + c));
    if (a.add_residual) add_bf16x8(v, *reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(a.x) + t * a.H + c));
    uint32_t w[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const __nv_bfloat162 h2 = __floats2bfloat162_rn(v[2 * j], v[2 * j + 1]);
      w[j] = *reinterpret_cast<const uint32_t*>(&h2);
    }
    *reinterpret_cast<uint4*>(static_cast<__nv_bfloat16*>(a.out) + t * a.H + c) = make_uint4(w[0], w[1], w[2], w[3]);
  }
}

template <int KK>
static cudaError_t launch_finalize_pair(const FinalizeDev& d, unsigned blocks, cudaStream_t s) {
  return launch_pdl(finalize_pair_kernel<KK>, dim3(blocks), dim3(256), 0, s, 1, d);
}
typedef cudaError_t (*FinalizePairFn)(const FinalizeDev&, unsigned, cudaStream_t);
static const FinalizePairFn kFinalizePair[FMMOE_MAX_TOPK] = {
    launch_finalize_pair<1>,  launch_finalize_pair<2>,  launch_finalize_pair<3>,  launch_finalize_pair<4>,
    launch_finalize_pair<5>,  launch_finalize_pair<6>,  launch_finalize_pair<7>,  launch_finalize_pair<8>,
    launch_finalize_pair<9>,  launch_finalize_pair<10>, launch_finalize_pair<11>, launch_finalize_pair<12>,
    launch_finalize_pair<13>, launch_finalize_pair<14>, launch_finalize_pair<15>, launch_finalize_pair<16>};

template <typename T> struct Vec4;
template <> struct Vec4<float> {
  static __device__ __forceinline__ float4 load(const float* p) { return *reinterpret_cast<const float4*>(p); }
  static __device__ __forceinline__ void store(float* p, float4 v) { *reinterpret_cast<float4*>(p) = v; }
};
template <> struct Vec4<__nv_bfloat16> {
  static __device__ __forceinline__ float4 load(const __nv_bfloat16* p) {
    const uint2 u = *reinterpret_cast<const uint2*>(p);
    const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&u.x));
    const float2 b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&u.y));
    return make_float4(a.x, a.y, b.x, b.y);
  }
  static __device__ __forceinline__ void store(__nv_bfloat16* p, float4 v) {
    const __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
    uint2 u;
    u.x = *reinterpret_cast<const uint32_t*>(&a);
    u.y = *reinterpret_cast<const uint32_t*>(&b);
    *reinterpret_cast<uint2*>(p) = u;
  }
};

template <typename T>
__global__ void finalize_kernel(const FinalizeDev a) {
  pdl_launch_dependents();
  pdl_wait();
  const int hv = a.H / 4;
  const long long n = a.T * hv;
  for (long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (long long)gridDim.x * blockDim.x) {
    const long long t = i / hv;
    const int c = (int)(i - t * hv) * 4;
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (!a.deterministic) {
      v = *reinterpret_cast<const float4*>(a.acc + t * a.H + c);
    } else {
      for (int s = 0; s < a.K; ++s) {
        const int row = a.inv_row[t * a.K + s];
        if (row < 0) continue;
        const float g = a.topk_w[t * a.K + s];
        const float4 yv = *reinterpret_cast<const float4*>(a.y + (long long)row * a.H + c);
        v.x = fmaf(g, yv.x, v.x); v.y = fmaf(g, yv.y, v.y); v.z = fmaf(g, yv.z, v.z); v.w = fmaf(g, yv.w, v.w);
      }
      for (int s = 0; s < a.n_shared; ++s) {
        const float4 yv = *reinterpret_cast<const float4*>(a.ysh + ((long long)s * a.T + t) * a.H + c);
        v.x += yv.x; v.y += yv.y; v.z += yv.z; v.w += yv.w;
      }
    }
    if (a.add_residual) {
      const float4 xv = Vec4<T>::load(static_cast<const T*>(a.x) + t * a.H + c);
      v.x += xv.x; v.y += xv.y; v.z += xv.z; v.w += xv.w;
    }
    Vec4<T>::store(static_cast<T*>(a.out) + t * a.H + c, v);
  }
}

fmmoe_status launch_finalize(fmmoe_handle* h, const FinalizeArgs& a, cudaStream_t s) {
  if (a.T == 0) return FMMOE_OK;
  FinalizeDev d;
  d.x = a.x; d.out = a.out; d.T = a.T; d.H = a.H; d.K = a.K; d.n_shared = a.n_shared;
  d.add_residual = a.add_residual; d.deterministic = a.deterministic;
  d.acc = a.acc; d.y = a.y; d.ysh = a.ysh; d.inv_row = a.inv_row; d.topk_w = a.topk_w;
  d.yb = static_cast<const __nv_bfloat16*>(a.yb); d.ybsh = static_cast<const __nv_bfloat16*>(a.ybsh);
  if (a.pair) {
    if (a.dtype != FMMOE_BF16 || a.H % 8 || a.K < 1 || a.K > FMMOE_MAX_TOPK) return FMMOE_ERR_INTERNAL;
    const long long n8 = a.T * (a.H / 8);
    long long blocks8 = (n8 + 255) / 256;
    const long long cap8 = (long long)h->sm_count * 32;
    if (blocks8 > cap8) blocks8 = cap8;
    {
      ProfScope ps(h, FMMOE_KERNEL_FINALIZE, s);
      for (int rep = 0; rep < ps.reps; ++rep) {
        FMMOE_CUDA_TRY(kFinalizePair[a.K - 1](d, (unsigned)blocks8, s));
        h->launches += 1;
      }
    }
    FMMOE_CUDA_TRY(cudaGetLastError());
    return FMMOE_OK;
  }
  const long long n = a.T * (a.H / 4);
  const int threads = 256;
  long long blocks = (n + threads - 1) / threads;
  const long long cap = (long long)h->sm_count * 16;
  if (blocks > cap) blocks = cap;
  {
    ProfScope ps(h, FMMOE_KERNEL_FINALIZE, s);
    for (int rep = 0; rep < ps.reps; ++rep) {
      if (a.dtype == FMMOE_BF16) FMMOE_CUDA_TRY(launch_pdl(finalize_kernel<__nv_bfloat16>, dim3((unsigned)blocks), dim3(threads), 0, s, 1, d));
      else FMMOE_CUDA_TRY(launch_pdl(finalize_kernel<float>, dim3((unsigned)blocks), dim3(threads), 0, s, 1, d));
      h->launches += 1;
    }
  }
  FMMOE_CUDA_TRY(cudaGetLastError());
  return FMMOE_OK;
}

}  // namespace fmmoe
