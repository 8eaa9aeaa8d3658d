// Cross-modal attention importance (Eq. 7): the attention weights of the LAST token of every
// sequence (the last text token of [T_v, T_t]) to all tokens, averaged over the attention heads.
// The pruning stage reads the entries at vision tokens (Eq. 11).  Attention layers themselves are
// not part of this library: the caller hands in that layer's keys and the last token's queries.
//
//   logits_kernel  : one warp per (token, kv head): dot products of the key with the queries of the
//                    heads that share this kv head (grouped-query attention), fp32 accumulation
//   stats_kernel   : one CTA per (head, sequence): max and sum of exp over the sequence (softmax)
//   average_kernel : one thread per token: mean over heads, in head order (reproducible)
#include <cuda_bf16.h>
#include <math.h>

#include "internal.h"
#include "ptx.cuh"

namespace fmmoe {

constexpr int A_MAXS = FMMOE_MAX_SEQS_PER_LAUNCH;
constexpr int A_MAX_GROUP = 16;   // query heads per kv head

struct AttnSeqs {
  int n_seq;
  long long seq_off[A_MAXS + 1];
};

struct AttnDev {
  const void* q; const void* k;
  int n_heads, n_kv, d, group;
  float scale;
  long long T;           // tokens of this launch's sequences start at seq_off[0]
  float* logits;         // [n_heads][T_total]
  float2* stats;         // [n_seq_total][n_heads] (max, 1 / sum exp)
  float* out;            // [T_total]
  long long T_total;
  int seq_base;          // index of this launch's first sequence
};

template <typename TT> __device__ __forceinline__ float ld_elem(const TT* p, int i);
template <> __device__ __forceinline__ float ld_elem<float>(const float* p, int i) { return p[i]; }
template <> __device__ __forceinline__ float ld_elem<__nv_bfloat16>(const __nv_bfloat16* p, int i) { return __bfloat162float(p[i]); }

template <typename TT>
__global__ void __launch_bounds__(256) attn_logits_kernel(const AttnDev a, const AttnSeqs sq) {
  pdl_launch_dependents();
  pdl_wait();
  const int lane = threadIdx.x & 31;
  const long long gw = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const long long n_tok = sq.seq_off[sq.n_seq] - sq.seq_off[0];
  if (gw >= n_tok * a.n_kv) return;
  const long long t = sq.seq_off[0] + gw / a.n_kv;
  const int kvh = (int)(gw % a.n_kv);
  int b = 0;
  while (b + 1 < sq.n_seq && t >= sq.seq_off[b + 1]) ++b;
  const TT* kp = static_cast<const TT*>(a.k) + (t * a.n_kv + kvh) * a.d;
  const TT* qp = static_cast<const TT*>(a.q) + ((long long)(a.seq_base + b) * a.n_heads + kvh * a.group) * a.d;
  float acc[A_MAX_GROUP];
#pragma unroll
  for (int g = 0; g < A_MAX_GROUP; ++g) acc[g] = 0.f;
  for (int i = lane; i < a.d; i += 32) {
    const float kv = ld_elem<TT>(kp, i);
#pragma unroll
    for (int g = 0; g < A_MAX_GROUP; ++g)
      if (g < a.group) acc[g] = fmaf(kv, ld_elem<TT>(qp + g * a.d, i), acc[g]);
  }
#pragma unroll
  for (int g = 0; g < A_MAX_GROUP; ++g) {
    if (g < a.group) {
      float v = acc[g];
#pragma unroll
      for (int o = 16; o; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
      if (lane == 0) a.logits[(long long)(kvh * a.group + g) * a.T_total + t] = v * a.scale;
    }
  }
}

__global__ void __launch_bounds__(256) attn_stats_kernel(const AttnDev a, const AttnSeqs sq) {
  __shared__ float s_red[8];
  pdl_launch_dependents();
  pdl_wait();
  const int h = blockIdx.x, b = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const long long lo = sq.seq_off[b], hi = sq.seq_off[b + 1];
  const float* l = a.logits + (long long)h * a.T_total;
  float m = -INFINITY;
  for (long long t = lo + tid; t < hi; t += 256) m = fmaxf(m, l[t]);
#pragma unroll
  for (int o = 16; o; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  if (lane == 0) s_red[warp] = m;
  __syncthreads();
  m = s_red[0];
  for (int i = 1; i < 8; ++i) m = fmaxf(m, s_red[i]);
  __syncthreads();
  float s = 0.f;
  for (long long t = lo + tid; t < hi; t += 256) s += expf(l[t] - m);
#pragma unroll
  for (int o = 16; o; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  if (lane == 0) s_red[warp] = s;
  __syncthreads();
  if (tid == 0) {
    float tot = 0.f;
    for (int i = 0; i < 8; ++i) tot += s_red[i];
    a.stats[(long long)(a.seq_base + b) * a.n_heads + h] = make_float2(m, tot > 0.f ? 1.f / tot : 0.f);
  }
}

__global__ void __launch_bounds__(256) attn_average_kernel(const AttnDev a, const AttnSeqs sq) {
  pdl_launch_dependents();
  pdl_wait();
  const int b = blockIdx.y;
  const long long t = sq.seq_off[b] + (long long)blockIdx.x * 256 + threadIdx.x;
  if (t >= sq.seq_off[b + 1]) return;
  const float2* st = a.stats + (long long)(a.seq_base + b) * a.n_heads;
  float acc = 0.f;
  for (int h = 0; h < a.n_heads; ++h) {
    const float2 ms = st[h];
    acc += expf(a.logits[(long long)h * a.T_total + t] - ms.x) * ms.y;
  }
  a.out[t] = acc / (float)a.n_heads;
}

}  // namespace fmmoe

using namespace fmmoe;

extern "C" __attribute__((visibility("default"))) size_t fmmoe_attention_workspace_bytes(int64_t n_tokens, int32_t n_seq,
                                                                                         int32_t n_heads) {
  if (n_tokens < 0 || n_seq < 0 || n_heads < 1) return 0;
  return align_up((size_t)n_tokens * n_heads * 4, 256) + align_up((size_t)n_seq * n_heads * 8, 256) + 256;
}

extern "C" __attribute__((visibility("default"))) fmmoe_status fmmoe_attention_importance(
    fmmoe_handle* h, const void* q_last, const void* k, int32_t dtype, int32_t n_heads, int32_t n_kv_heads,
    int32_t head_dim, float scale, const int64_t* seq_off, int32_t n_seq, float* attn_out, void* workspace,
    size_t workspace_bytes, void* cuda_stream) {
  if (!h || !seq_off || n_seq < 0 || n_heads < 1 || n_kv_heads < 1 || head_dim < 1) return FMMOE_ERR_INVALID_ARG;
  if (dtype != FMMOE_F32 && dtype != FMMOE_BF16) return FMMOE_ERR_INVALID_ARG;
  if (n_heads % n_kv_heads) return FMMOE_ERR_INVALID_ARG;
  if (n_heads / n_kv_heads > A_MAX_GROUP) return FMMOE_ERR_UNSUPPORTED;
  if (n_seq && seq_off[0] != 0) return FMMOE_ERR_INVALID_ARG;
  for (int b = 0; b < n_seq; ++b)
    if (seq_off[b + 1] < seq_off[b]) return FMMOE_ERR_INVALID_ARG;
  const int64_t T = n_seq ? seq_off[n_seq] : 0;
  if (T == 0) return FMMOE_OK;
  if (!q_last || !k || !attn_out) return FMMOE_ERR_INVALID_ARG;
  const size_t need = fmmoe_attention_workspace_bytes(T, n_seq, n_heads) - 256;
  if (!workspace || ((uintptr_t)workspace & 255) || workspace_bytes < need) return FMMOE_ERR_WORKSPACE;
  cudaStream_t s = static_cast<cudaStream_t>(cuda_stream);
  char* ws = static_cast<char*>(workspace);
  AttnDev a = {};
  a.q = q_last; a.k = k; a.n_heads = n_heads; a.n_kv = n_kv_heads; a.d = head_dim; a.group = n_heads / n_kv_heads;
  a.scale = scale; a.logits = reinterpret_cast<float*>(ws);
  a.stats = reinterpret_cast<float2*>(ws + align_up((size_t)T * n_heads * 4, 256));
  a.out = attn_out; a.T_total = T;
  for (int b0 = 0; b0 < n_seq; b0 += A_MAXS) {
    const int nb = n_seq - b0 < A_MAXS ? n_seq - b0 : A_MAXS;
    AttnSeqs sq = {};
    sq.n_seq = nb;
    for (int i = 0; i <= nb; ++i) sq.seq_off[i] = seq_off[b0 + i];
    a.seq_base = b0;
    const long long n_tok = sq.seq_off[nb] - sq.seq_off[0];
    if (n_tok == 0) continue;
    long long max_len = 0;
    for (int i = 0; i < nb; ++i) max_len = sq.seq_off[i + 1] - sq.seq_off[i] > max_len ? sq.seq_off[i + 1] - sq.seq_off[i] : max_len;
    const long long warps = n_tok * n_kv_heads;
    {
      ProfScope ps(h, FMMOE_KERNEL_ATTN, s);
      if (dtype == FMMOE_BF16)
        FMMOE_CUDA_TRY(launch_pdl(attn_logits_kernel<__nv_bfloat16>, dim3((unsigned)((warps + 7) / 8)), dim3(256), 0, s, 1, a, sq));
      else
        FMMOE_CUDA_TRY(launch_pdl(attn_logits_kernel<float>, dim3((unsigned)((warps + 7) / 8)), dim3(256), 0, s, 1, a, sq));
      FMMOE_CUDA_TRY(launch_pdl(attn_stats_kernel, dim3(n_heads, nb), dim3(256), 0, s, 1, a, sq));
      FMMOE_CUDA_TRY(launch_pdl(attn_average_kernel, dim3((unsigned)((max_len + 255) / 256), nb), dim3(256), 0, s, 1, a, sq));
    }
    FMMOE_CUDA_TRY(cudaGetLastError());
    h->launches += 3;
  }
  return FMMOE_OK;
}
