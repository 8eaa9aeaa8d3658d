// Expert FFNs in fp32 (Eq. 4 with SwiGLU experts) for fp32 layers.  Plain FMA on
// CUDA cores: TF32 tensor cores would not meet an fp32 tolerance.  Same grouping,
// same two GEMMs and the same combine as the tensor-core path, tiles of 32 rows x
// 64 columns, 256 threads, 2 x 4 outputs per thread.
#include "internal.h"
#include "ptx.cuh"

namespace fmmoe {

constexpr int F_BM = F32_BLOCK_M;   // 32
constexpr int F_BN = 64;
constexpr int F_BK = 32;
constexpr int F_THREADS = 256;

struct F32Params {
  const MTile* mtiles; const int32_t* n_mtiles;   // routed M-tiles (NULL for the shared launch)
  int mt_per_shared; long long T;                 // shared launch: tiles per shared expert
  int K;                                          // contraction length
  int N;                                          // output columns per group
  const float* a;                                 // MODE 0: x [T, K];  MODE 1: act [rows, K]
  const int32_t* row_token;                       // routed: token of each grouped row
  const float* row_gate;
  const float* b0; const float* b1;               // [groups, N, K] (b1: up projection, MODE 0)
  float* out;                                     // MODE 0: act [rows, N]; MODE 1 det: y [rows, N]
  float* acc;                                     // MODE 1 atomic: [T, N]
  int deterministic;
};

template <int MODE>
__global__ void __launch_bounds__(F_THREADS) ffn_f32_kernel(const F32Params p) {
  __shared__ float As[F_BM][F_BK + 1];
  __shared__ float B0s[F_BN][F_BK + 1];
  __shared__ float B1s[MODE == 0 ? F_BN : 1][F_BK + 1];
  __shared__ long long s_arow[F_BM];   // source row of A for each tile row, -1 if none
  pdl_launch_dependents();
  pdl_wait();
  const bool routed = p.mtiles != nullptr;
  int group, row0, rows;
  if (routed) {
    if ((int)blockIdx.x >= *p.n_mtiles) return;
    const MTile m = p.mtiles[blockIdx.x];
    group = m.group; row0 = m.row0; rows = m.rows;
  } else {
    group = blockIdx.x / p.mt_per_shared;
    row0 = (blockIdx.x - group * p.mt_per_shared) * F_BM;
    const long long left = p.T - row0;
    rows = left < F_BM ? (int)left : F_BM;
  }
  const int n0 = blockIdx.y * F_BN;
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  // output row index in the grouped space (shared experts: group * T + token)
  const long long out_base = routed ? row0 : (long long)group * p.T + row0;
  if (tid < F_BM) {
    long long ar = -1;
    if (tid < rows) {
      if (MODE == 0) ar = routed ? p.row_token[row0 + tid] : row0 + tid;
      else ar = out_base + tid;
    }
    s_arow[tid] = ar;
  }
  __syncthreads();
  const float* B0 = p.b0 + (long long)group * p.N * p.K;
  const float* B1 = MODE == 0 ? p.b1 + (long long)group * p.N * p.K : nullptr;
  float c0[2][4] = {}, c1[2][4] = {};
  for (int k0 = 0; k0 < p.K; k0 += F_BK) {
    for (int i = tid; i < F_BM * F_BK; i += F_THREADS) {
      const int r = i / F_BK, k = i % F_BK;
      const long long ar = s_arow[r];
      As[r][k] = (ar >= 0 && k0 + k < p.K) ? p.a[ar * p.K + k0 + k] : 0.f;
    }
    for (int i = tid; i < F_BN * F_BK; i += F_THREADS) {
      const int r = i / F_BK, k = i % F_BK;
      const bool ok = n0 + r < p.N && k0 + k < p.K;
      B0s[r][k] = ok ? B0[(long long)(n0 + r) * p.K + k0 + k] : 0.f;
      if (MODE == 0) B1s[r][k] = ok ? B1[(long long)(n0 + r) * p.K + k0 + k] : 0.f;
    }
    __syncthreads();
#pragma unroll 8
    for (int k = 0; k < F_BK; ++k) {
      const float a0 = As[ty * 2][k], a1 = As[ty * 2 + 1][k];
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float b = B0s[tx * 4 + j][k];
        c0[0][j] = fmaf(a0, b, c0[0][j]);
        c0[1][j] = fmaf(a1, b, c0[1][j]);
        if (MODE == 0) {
          const float bu = B1s[tx * 4 + j][k];
          c1[0][j] = fmaf(a0, bu, c1[0][j]);
          c1[1][j] = fmaf(a1, bu, c1[1][j]);
        }
      }
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 2; ++i) {
    const int r = ty * 2 + i;
    if (r >= rows) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int col = n0 + tx * 4 + j;
      if (col >= p.N) continue;
      if (MODE == 0) {
        const float g = c0[i][j];
        p.out[(out_base + r) * p.N + col] = g / (1.f + expf(-g)) * c1[i][j];
      } else if (p.deterministic) {
        p.out[(out_base + r) * p.N + col] = c0[i][j];
      } else {
        const long long tok = routed ? p.row_token[row0 + r] : row0 + r;
        const float gate = routed ? p.row_gate[row0 + r] : 1.f;
        atomicAdd(&p.acc[tok * p.N + col], gate * c0[i][j]);
      }
    }
  }
}

fmmoe_status launch_ffn_f32(fmmoe_handle* h, const FfnArgs& a, cudaStream_t s) {
  const fmmoe_layer_desc& d = *a.d;
  const int H = d.hidden, I = d.inter, Ns = d.n_shared, Is = d.shared_inter;
  if (a.T == 0) return FMMOE_OK;
  const int mtps = (int)((a.T + F_BM - 1) / F_BM);
  // routed GEMM-1
  F32Params p = {};
  p.mtiles = a.mtiles; p.n_mtiles = a.n_mtiles; p.T = a.T;
  p.K = H; p.N = I; p.a = static_cast<const float*>(a.x);
  p.row_token = a.row_token; p.row_gate = a.row_gate;
  p.b0 = static_cast<const float*>(a.w->w_gate); p.b1 = static_cast<const float*>(a.w->w_up);
  p.out = static_cast<float*>(a.act);
  if (a.max_mtiles > 0) {
    { ProfScope prof_(h, FMMOE_KERNEL_GEMM1, s); FMMOE_CUDA_TRY(launch_pdl(ffn_f32_kernel<0>, dim3(a.max_mtiles, (I + F_BN - 1) / F_BN), dim3(F_THREADS), 0, s, 1, p)); }
    FMMOE_CUDA_TRY(cudaGetLastError());
    // routed GEMM-2
    F32Params q = p;
    q.K = I; q.N = H; q.a = static_cast<const float*>(a.act);
    q.b0 = static_cast<const float*>(a.w->w_down); q.b1 = nullptr;
    q.out = a.y; q.acc = a.acc; q.deterministic = a.deterministic;
    { ProfScope prof_(h, FMMOE_KERNEL_GEMM2, s); FMMOE_CUDA_TRY(launch_pdl(ffn_f32_kernel<1>, dim3(a.max_mtiles, (H + F_BN - 1) / F_BN), dim3(F_THREADS), 0, s, 1, q)); }
    FMMOE_CUDA_TRY(cudaGetLastError());
    h->launches += 2;
  }
  if (Ns) {
    F32Params ps = {};
    ps.mt_per_shared = mtps; ps.T = a.T; ps.K = H; ps.N = Is; ps.a = static_cast<const float*>(a.x);
    ps.b0 = static_cast<const float*>(a.w->ws_gate); ps.b1 = static_cast<const float*>(a.w->ws_up);
    ps.out = static_cast<float*>(a.act_sh);
    { ProfScope prof_(h, FMMOE_KERNEL_GEMM1, s); FMMOE_CUDA_TRY(launch_pdl(ffn_f32_kernel<0>, dim3(Ns * mtps, (Is + F_BN - 1) / F_BN), dim3(F_THREADS), 0, s, 1, ps)); }
    FMMOE_CUDA_TRY(cudaGetLastError());
    F32Params qs = ps;
    qs.K = Is; qs.N = H; qs.a = static_cast<const float*>(a.act_sh);
    qs.b0 = static_cast<const float*>(a.w->ws_down); qs.b1 = nullptr;
    qs.out = a.ysh; qs.acc = a.acc; qs.deterministic = a.deterministic;
    { ProfScope prof_(h, FMMOE_KERNEL_GEMM2, s); FMMOE_CUDA_TRY(launch_pdl(ffn_f32_kernel<1>, dim3(Ns * mtps, (H + F_BN - 1) / F_BN), dim3(F_THREADS), 0, s, 1, qs)); }
    FMMOE_CUDA_TRY(cudaGetLastError());
    h->launches += 2;
  }
  return FMMOE_OK;
}

}  // namespace fmmoe
