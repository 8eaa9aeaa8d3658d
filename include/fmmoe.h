/* fmmoe.h -- C ABI of the B200 (sm_100a) FastMMoE MoE-layer hot path.
 *
 * The library implements, as hand-written CUDA kernels, the two components of
 * FastMMoE's prefill path:
 *   - Section 3.1: a mixture-of-experts layer in which vision tokens activate
 *     K_v <= K routed experts (Eq. 1-5) from a start layer l_v on, and
 *   - Section 3.2: routing-aware sliding-window pruning of vision tokens
 *     (Eq. 6-18 and the drop rule stated after Eq. 18).
 *
 * Conventions that hold for every entry point unless its comment says otherwise
 *   - Tensor pointers are DEVICE pointers owned by the caller, 16-byte aligned,
 *     row-major and contiguous.  Pointers marked (host) are host arrays.
 *   - Nothing is allocated on the device after fmmoe_create(); scratch memory is
 *     the caller's `workspace`, sized by the matching *_workspace_bytes() call.
 *   - Work is enqueued on `cuda_stream` (a cudaStream_t passed as void*) and the
 *     call returns without synchronising, except where stated.
 *   - Errors are return codes; arguments are validated on the host before any
 *     launch.  A kernel whose bounded wait expired records FMMOE_ERR_TIMEOUT in
 *     a device status word that fmmoe_get_status() reads back.
 *   - There is no CPU or library fallback: unsupported shapes return
 *     FMMOE_ERR_UNSUPPORTED.
 *   - Tokens are rows.  is_visual[t] != 0 marks a vision token.  Experts are
 *     numbered from 0.  All ties go to the lower index.
 */
#ifndef FMMOE_H_
#define FMMOE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  FMMOE_OK = 0,
  FMMOE_ERR_INVALID_ARG = 1,   /* NULL / misaligned pointer, negative size, K_v > K ...   */
  FMMOE_ERR_UNSUPPORTED = 2,   /* shape outside what the kernels implement               */
  FMMOE_ERR_WORKSPACE = 3,     /* workspace NULL, misaligned or too small                */
  FMMOE_ERR_CUDA = 4,          /* a CUDA runtime/driver call failed                      */
  FMMOE_ERR_TIMEOUT = 5,       /* a device-side bounded wait expired                     */
  FMMOE_ERR_INTERNAL = 6,
  FMMOE_ERR_TOO_LARGE = 7      /* problem exceeds the built-in scratch of a *_static entry point */
} fmmoe_status;

typedef enum { FMMOE_F32 = 0, FMMOE_BF16 = 1 } fmmoe_dtype;

/* Storage format of the expert matrices (w_gate, w_up, w_down and the shared experts').
 * FMMOE_WEIGHTS_FP8_BLOCK128 halves the weight stream that bounds a prefill at small batch
 * (Section 3.1 leaves a few dozen rows per expert; Appendix E: the compressed prefill is
 * memory-bound): every matrix element is one FP8 E4M3 byte (1 sign, 4 exponent bits with
 * bias 7, 3 mantissa bits, subnormals, largest magnitude 448; the NaN encodings 0x7f / 0xff
 * must not occur), and every block of 128 x 128 elements of a matrix [rows, cols] (the last
 * block of a dimension may be partial) shares one power-of-two scale, stored as its exponent:
 *   value(r, c) = e4m3(byte[r][c]) * 2^scale_exp[r / 128][c / 128],   -100 <= scale_exp <= 7.
 * A power of two keeps the conversion to bf16 exact (an E4M3 value has 4 significant bits),
 * so the layer computes with exactly these values: activations, accumulation and outputs are
 * as in the bf16 layer.  Requires dtype == FMMOE_BF16; the router matrix stays bf16. */
typedef enum { FMMOE_WEIGHTS_AS_DTYPE = 0, FMMOE_WEIGHTS_FP8_BLOCK128 = 1 } fmmoe_weight_format;

/* Limits of the kernels. */
#define FMMOE_MAX_EXPERTS 256
#define FMMOE_MAX_TOPK 16
#define FMMOE_MAX_WINDOW 8
#define FMMOE_MAX_SEQS_PER_LAUNCH 64

/* flags of fmmoe_route / fmmoe_moe_forward */
#define FMMOE_FLAG_REDUCE_ON 1u      /* layer index >= l_v: vision tokens use K_v (Section 3.1) */
#define FMMOE_FLAG_RESIDUAL 2u       /* out = x + MoE(x)                                        */
#define FMMOE_FLAG_DETERMINISTIC 4u  /* combine by a fixed-order gather instead of atomic adds  */

/* Static shape of one MoE layer (Section 3.1: H, E, S_m, N_s, K, K_v). */
typedef struct {
  int32_t hidden;        /* H                                                    */
  int32_t n_experts;     /* E routed experts, 1..FMMOE_MAX_EXPERTS               */
  int32_t inter;         /* routed expert intermediate size S_m                  */
  int32_t n_shared;      /* N_s shared experts (>= 0), always active, gate 1     */
  int32_t shared_inter;  /* intermediate size of EACH shared expert              */
  int32_t top_k;         /* K, 1..FMMOE_MAX_TOPK                                 */
  int32_t top_k_vis;     /* K_v = pK, 0..K; 0 only if n_shared > 0 (Section 3.1) */
  int32_t dtype;         /* fmmoe_dtype of x, out and all expert/router weights  */
  int32_t weight_format; /* fmmoe_weight_format of the expert matrices           */
} fmmoe_layer_desc;

/* Layer parameters (device, read-only).  nn.Linear layout: [out_features, in_features]. */
typedef struct {
  const void  *router_w;  /* W_E [E, H] dtype (Eq. 1)                                       */
  const float *router_b;  /* [E] fp32 added to the logits before the softmax, or NULL       */
  const void  *w_gate;    /* [E, S_m, H]                                                    */
  const void  *w_up;      /* [E, S_m, H]                                                    */
  const void  *w_down;    /* [E, H, S_m]                                                    */
  const void  *ws_gate;   /* [N_s, S_s, H] or NULL                                          */
  const void  *ws_up;     /* [N_s, S_s, H] or NULL                                          */
  const void  *ws_down;   /* [N_s, H, S_s] or NULL                                          */
  /* FMMOE_WEIGHTS_FP8_BLOCK128 only (else ignored): the matrices above hold one byte per element
   * and these hold the block scale exponents, int8, row-major, per expert
   * [ceil(rows/128), ceil(cols/128)] of that expert's [rows, cols] matrix:                      */
  const int8_t *w_gate_scale;   /* [E, ceil(S_m/128), ceil(H/128)]                                */
  const int8_t *w_up_scale;     /* [E, ceil(S_m/128), ceil(H/128)]                                */
  const int8_t *w_down_scale;   /* [E, ceil(H/128), ceil(S_m/128)]                                */
  const int8_t *ws_gate_scale;  /* [N_s, ceil(S_s/128), ceil(H/128)] or NULL                      */
  const int8_t *ws_up_scale;    /* [N_s, ceil(S_s/128), ceil(H/128)] or NULL                      */
  const int8_t *ws_down_scale;  /* [N_s, ceil(H/128), ceil(S_s/128)] or NULL                      */
} fmmoe_weights;

/* Optional routing outputs (device).  Any pointer may be NULL = not wanted. */
typedef struct {
  float   *logits;      /* [T, E] fp32  Z (Eq. 1), as the kernel holds them                      */
  float   *probs;       /* [T, E] fp32  P = softmax(Z) (Eq. 2); the R_v rows of Eq. 6            */
  int32_t *topk_idx;    /* [T, K] Q (Eq. 3), descending probability; -1 beyond the token's k     */
  float   *topk_w;      /* [T, K] g (Eq. 5), 0 beyond the token's k                              */
  int32_t *expert_off;  /* [E+1] first row of each expert in the expert-grouped order            */
  int32_t *row_token;   /* [T*K] token of each row (first expert_off[E] entries are valid)       */
  int32_t *inv_row;     /* [T, K] row of each (token, slot), -1 for padded slots                 */
} fmmoe_route_out;

typedef struct fmmoe_handle fmmoe_handle;   /* opaque: device, SM count, status word, launch counter */

/* Create a handle on CUDA device `device` (allocates a few hundred bytes of
 * device memory for the status word, and loads the pruning kernels together with the
 * built-in scratch array of fmmoe_prune_visual_static onto the device).  Not thread-safe
 * per handle.  Environment, read once here: FMMOE_DEBUG_SYNC=1 synchronises after every
 * kernel and reports the first failing one on stderr; FMMOE_GATHER_MIN_TOKENS=n moves the
 * token count from which GEMM-1 gathers the routed rows itself instead of reading an
 * expert-ordered copy of x (default 256);
 * FMMOE_SMALL_M_MAX_TOKENS=n moves the token count below which the expert GEMMs run with the
 * token rows as the MMA's N dimension (default 256: decode-sized batches; 0 turns that form
 * off; layers with FP8 weights always run in it);
 * FMMOE_CTA_PAIR_MIN_TOKENS=n makes them run on CTA pairs with 256-row tiles from n tokens on
 * (off by default: measured no faster than the one-CTA form on a power-capped B200); FMMOE_PAIR_ROWS_MIN_TOKENS=n keeps the atomic fp32 combine below n tokens
 * (default 0: the combine always goes through per-pair bf16 rows summed in a fixed order). */
fmmoe_status fmmoe_create(fmmoe_handle **handle, int device);
fmmoe_status fmmoe_destroy(fmmoe_handle *handle);
const char  *fmmoe_status_string(fmmoe_status s);

/* Synchronises `cuda_stream`, reads and clears the device status word.
 * Returns FMMOE_OK, FMMOE_ERR_TIMEOUT (a bounded wait expired in a kernel; its
 * outputs are invalid) or FMMOE_ERR_CUDA. */
fmmoe_status fmmoe_get_status(fmmoe_handle *handle, void *cuda_stream);

/* Number of kernels this handle has launched so far (host counter). */
int64_t fmmoe_launch_count(const fmmoe_handle *handle);

/* Bytes of workspace fmmoe_route / fmmoe_moe_forward need for n_tokens tokens of
 * this layer with these flags (only FMMOE_FLAG_DETERMINISTIC changes the size).
 * Host-only, no GPU work.  Returns 0 for an invalid description. */
size_t fmmoe_workspace_bytes(const fmmoe_layer_desc *desc, int64_t n_tokens, uint32_t flags);

/* Section 3.1, Eq. 1-3 and 5: router logits, softmax, per-token top-k with
 * k = K_v for vision tokens when FMMOE_FLAG_REDUCE_ON is set (K otherwise),
 * gates renormalised over the selected set.  The selection is taken on the
 * fp32 logits (softmax is monotone); equal logits go to the lower expert.
 * If expert_off / row_token / inv_row are requested, the stable grouping of the
 * (token, expert) pairs by expert (rows of one expert ascend by token) is
 * produced too.  x: [T, H] dtype; is_visual: [T] bytes.  n_tokens may be 0. */
fmmoe_status fmmoe_route(fmmoe_handle *handle, const fmmoe_layer_desc *desc, const fmmoe_weights *w,
                         const void *x, const uint8_t *is_visual, int64_t n_tokens, uint32_t flags,
                         const fmmoe_route_out *out, void *workspace, size_t workspace_bytes,
                         void *cuda_stream);

/* Section 3.1, Eq. 1-5 (whole layer):
 *   out[t] = sum_s FFN^s(x[t]) + sum_{j in Q_t} g_j FFN^e_j(x[t])   (+ x[t] with FMMOE_FLAG_RESIDUAL)
 * with SwiGLU experts FFN(x) = W_down (silu(W_gate x) * (W_up x)).  Experts a
 * token did not select are not evaluated for it.  bf16 layers run the expert
 * contractions on tcgen05 tensor cores with fp32 accumulation and round the
 * SwiGLU activations once to bf16; fp32 layers use fp32 FMA throughout.
 * out: [T, H] dtype, must not alias x.  `route` (may be NULL) receives the
 * routing record of the call.  bf16 requires H % 64 == 0, S_m % 64 == 0,
 * S_s % 64 == 0.  With FMMOE_WEIGHTS_FP8_BLOCK128 the expert matrices are streamed as FP8 bytes,
 * expanded to bf16 in shared memory (exactly) and fed to the same tensor-core contraction; it
 * additionally requires H % 128 == 0, S_m % 128 == 0 and S_s % 128 == 0. */
fmmoe_status fmmoe_moe_forward(fmmoe_handle *handle, const fmmoe_layer_desc *desc, const fmmoe_weights *w,
                               const void *x, const uint8_t *is_visual, int64_t n_tokens, uint32_t flags,
                               void *out, const fmmoe_route_out *route, void *workspace,
                               size_t workspace_bytes, void *cuda_stream);

/* Same layer as fmmoe_moe_forward with the step's activations in HOST memory:
 * copies x_host [T,H] and is_visual_host [T] to the device, runs the layer, copies
 * out back to out_host [T,H] and SYNCHRONISES the stream before returning.
 * Pinned host buffers make the copies asynchronous.  `workspace` must hold
 * fmmoe_workspace_bytes() + fmmoe_host_staging_bytes() bytes.  Weights stay on the device.
 * Optional DEVICE outputs for a caller that continues on the GPU (e.g. with
 * fmmoe_prune_visual): `route` as in fmmoe_moe_forward, `out_dev` [T,H] receives the
 * layer output, `is_visual_dev` [T] the uploaded mask.  Each may be NULL. */
size_t fmmoe_host_staging_bytes(const fmmoe_layer_desc *desc, int64_t n_tokens);
fmmoe_status fmmoe_moe_forward_host(fmmoe_handle *handle, const fmmoe_layer_desc *desc, const fmmoe_weights *w,
                                    const void *x_host, const uint8_t *is_visual_host, int64_t n_tokens,
                                    uint32_t flags, void *out_host, const fmmoe_route_out *route, void *out_dev,
                                    uint8_t *is_visual_dev, void *workspace, size_t workspace_bytes,
                                    void *cuda_stream);

/* Pipelined host I/O.  The paper has no counterpart: these calls only overlap the PCIe copies of
 * consecutive, independent batches with the layer itself, for callers whose activations live in
 * host memory.  Each handle owns one upload and one download stream (created by the first of these
 * calls on the handle).
 *
 * fmmoe_moe_forward_host_async: as fmmoe_moe_forward_host, but returns as soon as everything is
 * enqueued: the uploads of x_host / is_visual_host run on the upload stream, the layer on
 * cuda_stream after them, the copy to out_host (skipped if out_host is NULL) on the download
 * stream after the layer.  Host buffers should be pinned.  A batch in flight owns its workspace,
 * out_dev, is_visual_dev and host buffers until a ticket taken after it has been waited for: give
 * every batch in flight its own set (two sets alternate for a depth of two).
 * fmmoe_upload_async: copies bytes from src_host to dst_dev on the upload stream and makes the work
 * enqueued on cuda_stream AFTER this call wait for the copy (earlier work on cuda_stream is not waited
 * for: dst_dev must not be in use by it; the ticket rule above covers that).
 * fmmoe_download_async: copies bytes from src_dev to dst_host on the download stream, after the
 * work enqueued on cuda_stream so far (e.g. the rows fmmoe_prune_visual has just produced).
 * fmmoe_host_fence: returns a ticket for everything enqueued on the download stream so far.
 * fmmoe_host_wait: blocks the calling thread until the downloads covered by the ticket are in
 * host memory (at most 64 tickets may be outstanding).
 * Errors: FMMOE_ERR_INVALID_ARG (NULL or unknown ticket), FMMOE_ERR_WORKSPACE, FMMOE_ERR_CUDA. */
fmmoe_status fmmoe_moe_forward_host_async(fmmoe_handle *handle, const fmmoe_layer_desc *desc, const fmmoe_weights *w,
                                          const void *x_host, const uint8_t *is_visual_host, int64_t n_tokens,
                                          uint32_t flags, void *out_host, const fmmoe_route_out *route,
                                          void *out_dev, uint8_t *is_visual_dev, void *workspace,
                                          size_t workspace_bytes, void *cuda_stream);
fmmoe_status fmmoe_upload_async(fmmoe_handle *handle, void *dst_dev, const void *src_host, size_t bytes,
                                void *cuda_stream);
fmmoe_status fmmoe_download_async(fmmoe_handle *handle, void *dst_host, const void *src_dev, size_t bytes,
                                  void *cuda_stream);
fmmoe_status fmmoe_host_fence(fmmoe_handle *handle, uint64_t *ticket);
fmmoe_status fmmoe_host_wait(fmmoe_handle *handle, uint64_t ticket);

/* Optional per-kernel timeline.  While enabled, every kernel the handle launches is
 * bracketed by CUDA events on the launching stream (host-side event objects only; no
 * device memory).  fmmoe_profile_read synchronises the device and returns the summed
 * duration and the number of launches of one kernel since the last reset.
 * An event pair adds the kernel's launch latency to what it measures, which matters for
 * kernels of 10-30 us.  fmmoe_profile_enable(handle, n) with n > 1 therefore issues every
 * launch of a kernel that can be repeated without changing its result (the router, the
 * finalize pass, the four pruning kernels) n times back to back inside its event pair and
 * reports the duration divided by n; outputs are unchanged.  The permutation pass (in
 * place) and the GEMMs (tile counters) always run once.
 * FMMOE_KERNEL_PERMUTE covers the scan and the scatter pass (which also writes the expert-ordered copy of x
 * at small batch); FMMOE_KERNEL_GATHER is kept for numbering only and reports no launches. */
enum {
  FMMOE_KERNEL_ROUTE = 0, FMMOE_KERNEL_PERMUTE = 1, FMMOE_KERNEL_GATHER = 2, FMMOE_KERNEL_GEMM1 = 3,
  FMMOE_KERNEL_GEMM2 = 4, FMMOE_KERNEL_FINALIZE = 5, FMMOE_KERNEL_PRUNE_INDEX = 6, FMMOE_KERNEL_PRUNE_SCORE = 7,
  FMMOE_KERNEL_PRUNE_SELECT = 8, FMMOE_KERNEL_PRUNE_COMPACT = 9, FMMOE_KERNEL_ATTN = 10, FMMOE_KERNEL_COUNT = 11
};
fmmoe_status fmmoe_profile_enable(fmmoe_handle *handle, int enable);
fmmoe_status fmmoe_profile_reset(fmmoe_handle *handle);
fmmoe_status fmmoe_profile_read(fmmoe_handle *handle, int kernel_id, double *total_ms, int64_t *launches);

/* Section 3.2 hyper-parameters. */
typedef struct {
  int32_t window;      /* W, 2..FMMOE_MAX_WINDOW                                                  */
  int32_t sim_mode;    /* 0: mean pairwise cosine (Eq. 8); 1: cosine to the window mean (Eq. 9-10) */
  int32_t merge_mode;  /* 0: mean rescaled to the largest member norm (Eq. 16-18); 1: plain mean;  */
                       /* 2: no merging (gamma ignored, windows are only dropped)                  */
  int32_t reserved;
  double  alpha;       /* Eq. 13 trade-off, 0..1; ignored when attn == NULL                        */
  double  gamma;       /* Eq. 14 merge rate, >= 0                                                  */
} fmmoe_prune_params;

/* Section 3.2.3 budget arithmetic (host only, data-independent): number of
 * vision tokens left when n_vis tokens are pruned towards n_retain.
 * eps = n_vis - n_retain; nothing happens unless eps > W; m = floor(n_retain*gamma)
 * windows are merged (each removes W-1 tokens; m is clamped so no more than eps
 * tokens go), then floor((eps - m(W-1)) / W) windows are dropped.
 * Optionally returns m and the dropped-window count.  Returns -1 on invalid arguments. */
int64_t fmmoe_prune_kept_count(int64_t n_vis, int64_t n_retain, const fmmoe_prune_params *p,
                               int64_t *n_merge, int64_t *n_drop);

size_t fmmoe_prune_workspace_bytes(int64_t n_tokens, int32_t n_seq);

/* Section 3.2 on n_seq independent sequences laid out back to back:
 * sequence b is tokens seq_off[b] .. seq_off[b+1]-1 and holds n_vis[b] vision
 * tokens (must equal the number of set bytes of is_visual in that range; a
 * mismatch is reported through the status word as FMMOE_ERR_INTERNAL).
 * Windows of W consecutive vision tokens (in sequence order, wherever text sits)
 * are scored C = alpha*S - (1-alpha)*A_bar (Eq. 8/10, 11-13) from the routing
 * probabilities `probs` [T, E] fp32 and the attention importance `attn` [T] fp32
 * (entries at vision tokens are used, Eq. 7).  With attn == NULL, C = S and the
 * drop stage takes the most redundant remaining windows.  Scores are
 * accumulated in fp64 and rounded once to fp32 before ranking.  The m highest-C
 * windows are merged into one row at their first token's position (Eq. 15-18),
 * then the d remaining windows with the smallest A_bar are dropped; the
 * N_v mod W trailing vision tokens and all text tokens are kept.
 * Outputs (device): x_out [T', H] dtype, is_visual_out [T'], keep_idx [T'] source
 * token of each output row, kind [T'] (0 text, 1 kept, 2 merged); each may be
 * NULL except x_out.  out_seq_off (host, [n_seq+1]) is filled before return:
 * the counts do not depend on the data.  x_out must not alias x. */
fmmoe_status fmmoe_prune_visual(fmmoe_handle *handle, const fmmoe_prune_params *p,
                                const float *probs, int32_t n_experts, const float *attn,
                                const void *x, int32_t dtype, int32_t hidden, const uint8_t *is_visual,
                                const int64_t *seq_off /* host [n_seq+1] */,
                                const int64_t *n_vis /* host [n_seq] */,
                                const int64_t *n_retain /* host [n_seq] */, int32_t n_seq,
                                void *x_out, uint8_t *is_visual_out, int32_t *keep_idx, uint8_t *kind,
                                int64_t *out_seq_off /* host [n_seq+1] */,
                                void *workspace, size_t workspace_bytes, void *cuda_stream);

/* Section 3.1 followed by Section 3.2 in one call: the layer (as fmmoe_moe_forward) and one pruning
 * stage (as fmmoe_prune_visual) applied to the layer's output `out`, with identical results.  What the
 * single call adds: the scoring and selection half of the pruning stage (Eq. 6-15) reads only the
 * routing probabilities and the mask, so it is enqueued on a stream of the handle as soon as the router
 * has run and executes beside the expert GEMMs; the row gather / merge (Eq. 16-18) follows the layer on
 * cuda_stream, which is also where everything is ordered again before the call's last kernel.
 * route must be non-NULL with route->probs set ([T, E] fp32); seq_off[n_seq] must equal n_tokens.
 * workspace: fmmoe_workspace_bytes() + fmmoe_prune_workspace_bytes() bytes, 256-byte aligned.
 * All other arguments, outputs and errors as in the two calls it replaces. */
fmmoe_status fmmoe_moe_forward_prune(fmmoe_handle *handle, const fmmoe_layer_desc *desc, const fmmoe_weights *w,
                                     const void *x, const uint8_t *is_visual, int64_t n_tokens, uint32_t flags,
                                     void *out, const fmmoe_route_out *route, const fmmoe_prune_params *p,
                                     const float *attn, const int64_t *seq_off, const int64_t *n_vis,
                                     const int64_t *n_retain, int32_t n_seq, void *x_out, uint8_t *is_visual_out,
                                     int32_t *keep_idx, uint8_t *kind, int64_t *out_seq_off, void *workspace,
                                     size_t workspace_bytes, void *cuda_stream);

/* Section 3.2.1, Eq. 7: cross-modal attention importance.  For every sequence, the attention
 * weights of its LAST token (the last text token of [T_v, T_t]) to all tokens of the sequence,
 * averaged over the attention heads:
 *   attn_out[t] = (1 / n_heads) * sum_h softmax_over_the_sequence(scale * q_last[b, h] . k[., kv(h)])[t]
 * with kv(h) = h / (n_heads / n_kv_heads) (grouped-query attention; n_kv_heads == n_heads is the
 * plain multi-head case).  The last token attends to the whole sequence, so no mask is needed.
 * fmmoe_prune_visual reads the entries at vision tokens (Eq. 11).  The attention layer itself is
 * the caller's: q_last [n_seq, n_heads, head_dim] are that layer's queries of the last tokens,
 * k [T, n_kv_heads, head_dim] its keys (as used in its own attention, e.g. after rotary
 * embedding), both `dtype`, device.  attn_out: [T] fp32, device.  The mean over heads is taken in
 * head order (reproducible).  head_dim any positive size; n_heads / n_kv_heads <= 16. */
size_t fmmoe_attention_workspace_bytes(int64_t n_tokens, int32_t n_seq, int32_t n_heads);
fmmoe_status fmmoe_attention_importance(fmmoe_handle *handle, const void *q_last, const void *k, int32_t dtype,
                                        int32_t n_heads, int32_t n_kv_heads, int32_t head_dim, float scale,
                                        const int64_t *seq_off /* host [n_seq+1] */, int32_t n_seq,
                                        float *attn_out, void *workspace, size_t workspace_bytes, void *cuda_stream);

/* A stack of n_layers MoE layers of one shape with residual adds (x <- x + MoE_l(x)), the
 * setting of Section 3.1's start layer and of the multi-stage pruning schedule (Section 3.2,
 * Appendices A and D).  Attention and normalisation layers are not part of this library.
 *   - Layer l (0-based) uses K_v experts for vision tokens iff l >= reduce_from (inclusive).
 *   - A stage with after_layer = l prunes layer l's OUTPUT using layer l's routing
 *     probabilities (computed on that layer's input); layers l+1.. see the shorter sequence.
 *     Its `retain` is a fraction of each sequence's ORIGINAL vision-token count
 *     (eta = floor(n_vis * retain)).  `attn` is the stage's attention-importance vector
 *     (device, one entry per token of the sequence as it is at that layer) or NULL for the
 *     attention-free score.  At most one stage per layer.
 * layer_w: HOST array of n_layers weight structs (device pointers inside).  x / is_visual:
 * the input tokens (not modified).  x_out [T', H], is_visual_out [T'] (may be NULL),
 * out_seq_off (host, [n_seq+1]): the final sequence layout; T' and the offsets follow from
 * fmmoe_stack_output_layout (host only, data-independent).  Flags: FMMOE_FLAG_DETERMINISTIC
 * is honoured; the residual is always added and the reduction flag is set per layer.
 * Everything is enqueued on cuda_stream without synchronising. */
typedef struct {
  int32_t after_layer;          /* prune after this layer, 0 .. n_layers-1                 */
  int32_t reserved;
  double  retain;               /* fraction of the original vision tokens to retain, 0..1 */
  fmmoe_prune_params params;    /* W, gamma, alpha, modes                                  */
  const float *attn;            /* device [T_at_that_layer] or NULL                        */
} fmmoe_stack_stage;

size_t fmmoe_stack_workspace_bytes(const fmmoe_layer_desc *desc, int64_t n_tokens, int32_t n_seq, uint32_t flags);
fmmoe_status fmmoe_stack_output_layout(const fmmoe_stack_stage *stages, int32_t n_stages, int32_t n_layers,
                                       const int64_t *seq_off /* host */, const int64_t *n_vis /* host */,
                                       int32_t n_seq, int64_t *out_seq_off /* host [n_seq+1] */,
                                       int64_t *out_n_vis /* host [n_seq] or NULL */);
fmmoe_status fmmoe_stack_forward(fmmoe_handle *handle, const fmmoe_layer_desc *desc,
                                 const fmmoe_weights *layer_w /* host [n_layers] */, int32_t n_layers,
                                 int32_t reduce_from, const fmmoe_stack_stage *stages, int32_t n_stages,
                                 const void *x, const uint8_t *is_visual, const int64_t *seq_off /* host */,
                                 const int64_t *n_vis /* host */, int32_t n_seq, uint32_t flags,
                                 void *x_out, uint8_t *is_visual_out, int64_t *out_seq_off /* host */,
                                 void *workspace, size_t workspace_bytes, void *cuda_stream);

/* Self-test of the library's bounded device-side waits (no counterpart in the paper).  Every
 * wait of a kernel on a barrier has a time budget; when it runs out the kernel records
 * FMMOE_ERR_TIMEOUT in the status word, releases its tensor memory and returns, so that a protocol
 * error ends as a status code with the context intact.  This call ARMS that path for the next
 * fmmoe_moe_forward on the handle (a bf16 layer; the armed call runs in the small-M form
 * whatever its token count): that call's GEMM-1 runs as a single CTA whose
 * producer stops before it issues any copy or arrival for k-block number `k_block` (0 = the first),
 * and all of that call's waits use `budget_ns` (1 us .. 1 s) instead of the default 2 s.  Nothing
 * faults and nothing spins without a limit: the issuing thread's wait for the missing stage
 * expires, the other roles see the CTA's abort flag, and the kernel leaves through its ordinary
 * tear-down.  The call's outputs are invalid; fmmoe_get_status returns FMMOE_ERR_TIMEOUT once and
 * the handle is back to normal for the next call. */
fmmoe_status fmmoe_test_expire_wait(fmmoe_handle *handle, uint64_t budget_ns, int32_t k_block);

/* fmmoe_prune_visual without a caller-supplied workspace and without any allocation.
 * (The paper has no counterpart: this is a packaging variant of fmmoe_prune_visual above,
 * same arguments minus `workspace`/`workspace_bytes`, same kernels, same results.)
 *
 * For callers that cannot obtain device memory at the point where they prune: a server
 * whose HBM was handed to another memory pool at start-up, or a latency-critical loop that
 * must not run into the device-wide synchronisation an allocation or a free can cause.
 * Inputs and outputs are still the caller's buffers.  The scratch lives in a fixed array
 * inside the library: FMMOE_STATIC_PRUNE_SCRATCH_BYTES (768 KiB) of device memory on every
 * GPU that loads the library, held until the process exits.
 *
 *   - The call makes no cudaMalloc/cudaFree and uses no allocating library routine.  The
 *     handle must exist already (fmmoe_create, done once at start-up, is where the
 *     library's only allocation happens) and its device must be the current device,
 *     otherwise FMMOE_ERR_INVALID_ARG.  Keep the handle's kernel timeline off
 *     (fmmoe_profile_enable) in such a setting: it creates event objects on demand.
 *   - Limit: seq_off[n_seq] <= FMMOE_STATIC_PRUNE_MAX_TOKENS tokens per call; more returns
 *     FMMOE_ERR_TOO_LARGE before anything is enqueued.
 *   - All set-up happens in fmmoe_create, with the handle's device current: the pruning
 *     kernels and the array are loaded onto the device there (under CUDA's lazy module
 *     loading that is the moment their device memory is taken), the array's device address
 *     is looked up and cached per device, and the selection kernel's shared-memory limit is
 *     raised.  So create the handle at start-up, while the process can still obtain device
 *     memory, and before starting any stream capture on that device; the pruning call
 *     itself then does no set-up at all.
 *   - All calls on a device share the one array, and it keeps whatever the previous call
 *     left in it.  No part of it needs clearing: a pass writes what it reads, and every
 *     index a kernel takes from the array is range-checked, so a call whose mask contradicts
 *     its n_vis (reported as FMMOE_ERR_INTERNAL by fmmoe_get_status) cannot be led out of
 *     bounds by the previous call's leftovers.  But two calls whose kernels may overlap on
 *     the GPU - different streams, or different host threads - race on it: serialise them,
 *     or use fmmoe_prune_visual with separate workspaces. */
#define FMMOE_STATIC_PRUNE_MAX_TOKENS 32768
fmmoe_status fmmoe_prune_visual_static(fmmoe_handle *handle, const fmmoe_prune_params *p,
                                       const float *probs, int32_t n_experts, const float *attn,
                                       const void *x, int32_t dtype, int32_t hidden, const uint8_t *is_visual,
                                       const int64_t *seq_off /* host [n_seq+1] */,
                                       const int64_t *n_vis /* host [n_seq] */,
                                       const int64_t *n_retain /* host [n_seq] */, int32_t n_seq,
                                       void *x_out, uint8_t *is_visual_out, int32_t *keep_idx, uint8_t *kind,
                                       int64_t *out_seq_off /* host [n_seq+1] */, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* FMMOE_H_ */
