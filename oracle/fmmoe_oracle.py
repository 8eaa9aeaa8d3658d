"""CPU oracle for the FastMMoE MoE-layer hot path.  TEST INFRASTRUCTURE ONLY.

A plain, slow, float64 numpy restatement of what the paper defines:
modality-aware expert-activation reduction (Section 3.1, Eq. 1-5) inside a
SwiGLU mixture-of-experts layer, and routing-aware sliding-window token pruning
(Section 3.2, Eq. 6-18 and the drop rule that follows Eq. 18).  No blocking,
fusion or reordering beyond what those equations state.  It shares no code with
the CUDA library and must never be imported by the product path: only tests,
the smoke check and the benchmark's cpu-baseline leg may use it.

Where the paper is silent or inconsistent a reading had to be chosen; every such
reading is marked "READING" below.

Pins (tests/test_oracle_*.py): every function here is pinned by closed forms,
invariants the paper states, brute force on tiny inputs, or values the paper
prints (the merge-rate bound table of Appendix D).  Not pinned, because the
paper does not print enough to reproduce them: its whole-model FLOPs-saving
percentages (only the MoE term of the Appendix E cost model is implemented).

Conventions: tokens are rows; `is_visual[t]` is 1 for a vision token; experts
are numbered from 0; all ties go to the lower index.
"""
from __future__ import annotations

import math
from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

F64 = np.float64

KIND_TEXT, KIND_KEPT, KIND_MERGED = 0, 1, 2


# ----------------------------------------------------------------------------
# Section 3.1: routing with fewer experts for vision tokens
# ----------------------------------------------------------------------------
def router_logits(x: np.ndarray, router_w: np.ndarray, router_b: Optional[np.ndarray] = None) -> np.ndarray:
    """Eq. 1: Z = W_E t for every token (rows of x), float64.

    READING: an optional per-expert bias is added to the logit before the
    softmax (the paper's router has none; the DeepSeekMoE-style workload adds one
    to skew expert load).  It therefore shifts probabilities and selection alike.
    """
    z = np.asarray(x, F64) @ np.asarray(router_w, F64).T
    if router_b is not None:
        z = z + np.asarray(router_b, F64)[None, :]
    return z


def routing_probs(logits: np.ndarray) -> np.ndarray:
    """Eq. 2 (and Eq. 6 for the vision rows): P = softmax(Z) over all E experts."""
    z = np.asarray(logits, F64)
    e = np.exp(z - z.max(axis=1, keepdims=True))
    return e / e.sum(axis=1, keepdims=True)


def experts_per_token(is_visual: np.ndarray, top_k: int, top_k_vis: int, reduce_on: bool) -> np.ndarray:
    """Section 3.1: K_v experts for vision tokens once the layer index has reached
    l_v (reduce_on), the full K otherwise and for every text token."""
    v = np.asarray(is_visual).astype(bool)
    k = np.full(v.shape[0], top_k, dtype=np.int64)
    if reduce_on:
        k[v] = top_k_vis
    return k


def select_experts(logits32: np.ndarray, k_t: np.ndarray, top_k: int) -> np.ndarray:
    """Eq. 3: the index set Q of the k_t highest-probability experts, listed by
    descending probability; rows padded with -1 up to K.

    READING: softmax is monotone, so the order of probabilities is the order of
    logits; the decision is taken on the float32 logits handed in (the precision
    the kernel holds them in) and equal logits go to the lower expert index.
    """
    z = np.asarray(logits32, np.float32)
    order = np.argsort(-z, axis=1, kind="stable")      # stable: ties keep ascending index
    idx = np.full((z.shape[0], top_k), -1, dtype=np.int32)
    for j in range(top_k):
        take = k_t > j
        idx[take, j] = order[take, j]
    return idx


def gates(probs: np.ndarray, topk_idx: np.ndarray) -> np.ndarray:
    """Eq. 5: g_j = P_j / sum_{k in Q} P_k on the selected set, 0 elsewhere
    (returned per slot, 0 in the padded slots).  Text tokens are renormalised
    over their own K selected experts in the same way (Appendix C)."""
    p = np.asarray(probs, F64)
    sel = topk_idx >= 0
    g = np.where(sel, np.take_along_axis(p, np.maximum(topk_idx, 0).astype(np.int64), axis=1), 0.0)
    s = g.sum(axis=1, keepdims=True)
    return np.divide(g, s, out=np.zeros_like(g), where=s > 0)


def route(x, router_w, router_b, is_visual, top_k, top_k_vis, reduce_on, logits32=None) -> Dict[str, np.ndarray]:
    """Eq. 1-5 for a batch of tokens.  If `logits32` is given the selection is made
    on it (the kernel's own float32 logits); otherwise on the float64 logits
    rounded once to float32."""
    z = router_logits(x, router_w, router_b)
    p = routing_probs(z)
    k_t = experts_per_token(is_visual, top_k, top_k_vis, reduce_on)
    z32 = z.astype(np.float32) if logits32 is None else np.asarray(logits32, np.float32)
    idx = select_experts(z32, k_t, top_k)
    return {"logits": z, "probs": p, "k_t": k_t, "topk_idx": idx, "topk_w": gates(p, idx)}


def permutation(topk_idx: np.ndarray, n_experts: int) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Group the routed (token, expert) pairs by expert.

    The paper only says an unselected expert costs nothing; the canonical order
    used here is the stable counting sort of the pairs, enumerated token-major,
    by expert: rows of one expert ascend by token index.  Returns
    expert_off[E+1], row_token[P] and inv_row[T,K] (row of each slot, -1 if padded).
    """
    T, K = topk_idx.shape
    flat = topk_idx.reshape(-1)
    valid = np.nonzero(flat >= 0)[0]
    order = valid[np.argsort(flat[valid], kind="stable")]
    counts = np.bincount(flat[valid], minlength=n_experts)
    expert_off = np.zeros(n_experts + 1, dtype=np.int32)
    expert_off[1:] = np.cumsum(counts)
    row_token = (order // K).astype(np.int32)
    inv_row = np.full(T * K, -1, dtype=np.int32)
    inv_row[order] = np.arange(order.size, dtype=np.int32)
    return expert_off, row_token, inv_row.reshape(T, K)


def swiglu_ffn(x: np.ndarray, w_gate: np.ndarray, w_up: np.ndarray, w_down: np.ndarray) -> np.ndarray:
    """One expert: W_d (silu(W_g x) * (W_u x)), weights in [out, in] layout,
    silu(z) = z / (1 + exp(-z)); no intermediate rounding."""
    x = np.asarray(x, F64)
    g = x @ np.asarray(w_gate, F64).T
    u = x @ np.asarray(w_up, F64).T
    a = g / (1.0 + np.exp(-g)) * u
    return a @ np.asarray(w_down, F64).T


def moe_combine(x, topk_idx, topk_w, weights, add_residual=False) -> np.ndarray:
    """Eq. 4: o = sum_s FFN^s(t) + sum_j g_j FFN^e_j(t); experts with g_j = 0 are
    not evaluated.  Shared experts see every token with weight 1."""
    x64 = np.asarray(x, F64)
    T, H = x64.shape
    out = np.zeros((T, H), F64)
    E = weights["w_gate"].shape[0]
    for e in range(E):
        tok, slot = np.nonzero(topk_idx == e)
        if tok.size == 0:
            continue
        y = swiglu_ffn(x64[tok], weights["w_gate"][e], weights["w_up"][e], weights["w_down"][e])
        np.add.at(out, tok, topk_w[tok, slot][:, None] * y)
    if weights.get("ws_gate") is not None:
        for s in range(weights["ws_gate"].shape[0]):
            out += swiglu_ffn(x64, weights["ws_gate"][s], weights["ws_up"][s], weights["ws_down"][s])
    if add_residual:
        out += x64
    return out


def moe_forward(x, is_visual, weights, top_k, top_k_vis, reduce_on, add_residual=False,
                logits32=None) -> Dict[str, np.ndarray]:
    """Eq. 1-5 then Eq. 4 for one layer.  Returns the routing record plus `out`."""
    r = route(x, weights["router_w"], weights.get("router_b"), is_visual, top_k, top_k_vis,
              reduce_on, logits32=logits32)
    r["out"] = moe_combine(x, r["topk_idx"], r["topk_w"], weights, add_residual)
    return r


# ----------------------------------------------------------------------------
# Section 3.2: routing-aware sliding-window pruning
# ----------------------------------------------------------------------------
def cosine(a: np.ndarray, b: np.ndarray) -> float:
    return float(np.dot(a, b) / (math.sqrt(np.dot(a, a)) * math.sqrt(np.dot(b, b))))


def window_similarity_pairwise(rw: np.ndarray) -> float:
    """Eq. 8: mean cosine similarity over the C(W,2) unordered pairs of the
    window's routing-probability rows."""
    W = rw.shape[0]
    s = 0.0
    for a in range(W):
        for b in range(a):
            s += cosine(rw[a], rw[b])
    return s / (W * (W - 1) / 2)


def window_similarity_mean(rw: np.ndarray) -> float:
    """Eq. 9-10: mean cosine of each row to the window's average distribution
    (the paper's cheaper approximation of Eq. 8)."""
    W = rw.shape[0]
    rbar = rw.sum(axis=0) / W
    return sum(cosine(rw[a], rbar) for a in range(W)) / W


def window_scores(probs_vis: np.ndarray, attn_vis: Optional[np.ndarray], window: int, alpha: float,
                  sim_mode: int = 0) -> Tuple[np.ndarray, Optional[np.ndarray], np.ndarray]:
    """Eq. 8 (or 10), Eq. 11-13 over the full windows of one sequence's vision
    tokens.  Returns (C, A_bar, S) with C and A_bar rounded ONCE to float32.

    READING (ragged tail): N_v mod W trailing tokens form no window; only the
    floor(N_v / W) full windows are scored.
    READING (no attention): with attn_vis=None the score is the routing
    similarity alone, C = S (alpha is not applied), and A_bar is None.
    READING (all-zero attention): if max_j A_bar_j = 0 the normalised A_bar is 0.
    """
    r = np.asarray(probs_vis, F64)
    n_f = r.shape[0] // window
    sim = window_similarity_pairwise if sim_mode == 0 else window_similarity_mean
    S = np.array([sim(r[i * window:(i + 1) * window]) for i in range(n_f)], F64)
    if attn_vis is None:
        return S.astype(np.float32), None, S
    a = np.asarray(attn_vis, F64)
    A = np.array([a[i * window:(i + 1) * window].sum() for i in range(n_f)], F64)   # Eq. 11
    amax = A.max() if n_f else 0.0
    A = A / amax if amax > 0 else np.zeros_like(A)                                   # Eq. 12
    C = alpha * S - (1.0 - alpha) * A                                                # Eq. 13
    return C.astype(np.float32), A.astype(np.float32), S


def prune_counts(n_vis: int, n_retain: int, window: int, gamma: float, merge_mode: int = 0) -> Tuple[int, int, int]:
    """Budget arithmetic of Section 3.2.3: (m, d, kept).

    eps = N_v - eta tokens must go.  Nothing happens unless eps > W.
    m = eta * gamma windows are merged (Eq. 14); each merged window turns W
    tokens into one.  The remaining u tokens are removed by dropping
    floor(u / W) whole windows.

    READING: the paper writes u = eps - m, which would count a merged window as
    removing one token; merging W tokens into one removes W - 1, and Appendix D
    derives its bound gamma_hat = ((N_v - eta)/(W - 1)) / eta from exactly that
    accounting (all eps tokens removed by merging alone).  So u = eps - m(W-1).
    READING: m = floor(eta * gamma), clamped so that u >= 0 and m does not exceed
    the number of full windows; d is clamped to the windows left.
    merge_mode 2 disables merging (m = 0).
    """
    eps = n_vis - n_retain
    n_f = n_vis // window
    if n_retain >= n_vis or eps <= window:
        return 0, 0, n_vis
    m = 0 if merge_mode == 2 else min(int(math.floor(n_retain * gamma + 1e-9)), eps // (window - 1), n_f)
    u = eps - m * (window - 1)
    d = min(u // window, n_f - m)
    return m, d, n_vis - m * (window - 1) - d * window


def select_windows(C32: np.ndarray, A32: Optional[np.ndarray], m: int, d: int) -> np.ndarray:
    """Eq. 15 and the drop rule: action per full window, 0 keep / 1 merge / 2 drop.

    Merge set M: the m windows with the highest redundancy score C.  Among the
    others, the d windows with the smallest attention importance A_bar are
    dropped.  READING (no attention): the drop stage continues down the C
    ranking (most redundant first).  Ties: lower window index first.
    """
    n_f = C32.shape[0]
    action = np.zeros(n_f, dtype=np.uint8)
    by_c = np.argsort(-np.asarray(C32, np.float32), kind="stable")
    action[by_c[:m]] = 1
    rest = np.nonzero(action == 0)[0]
    if A32 is not None:
        order = rest[np.argsort(np.asarray(A32, np.float32)[rest], kind="stable")]
    else:
        order = rest[np.argsort(-np.asarray(C32, np.float32)[rest], kind="stable")]
    action[order[:d]] = 2
    return action


def merge_window(rows: np.ndarray, merge_mode: int = 0) -> np.ndarray:
    """Eq. 16-18: the window's arithmetic mean, rescaled (MLERP-style) to the
    largest member norm.  merge_mode 1 returns the plain mean.
    READING: a zero mean vector stays zero."""
    rows = np.asarray(rows, F64)
    xbar = rows.sum(axis=0) / rows.shape[0]                    # Eq. 17
    if merge_mode == 1:
        return xbar
    nb = math.sqrt(float(np.dot(xbar, xbar)))
    if nb == 0.0:
        return xbar
    nmax = max(math.sqrt(float(np.dot(r, r))) for r in rows)
    return xbar / nb * nmax                                    # Eq. 18


def prune_sequence(x, is_visual, probs, attn, n_retain, window, alpha, gamma, sim_mode=0, merge_mode=0):
    """Section 3.2 on ONE sequence.  x [L,H], is_visual [L], probs [L,E] (rows of
    vision tokens used, Eq. 6), attn [L] or None (Eq. 7 values at vision tokens).

    Windows run over the sequence's vision tokens in order, wherever they sit.
    Output keeps the original order; a merged window emits one row at the
    position of its first token (the paper: merged tokens keep their positions);
    dropped windows emit nothing; text tokens and tail tokens are always kept.
    Returns dict(x_out[L',H] f64, is_visual_out, keep_idx (source token of each
    output row), kind (0 text / 1 kept / 2 merged), action, C, A_bar, S).
    """
    x64 = np.asarray(x, F64)
    vis = np.nonzero(np.asarray(is_visual).astype(bool))[0]
    n_vis = vis.size
    m, d, kept = prune_counts(n_vis, int(n_retain), window, gamma, merge_mode)
    C32, A32, S = window_scores(np.asarray(probs)[vis], None if attn is None else np.asarray(attn)[vis],
                                window, alpha, sim_mode)
    action = select_windows(C32, A32, m, d)
    n_f = n_vis // window
    first_of = {int(vis[i * window]): i for i in range(n_f)}
    win_of = {int(vis[v]): v // window for v in range(n_f * window)}
    rows, keep_idx, kind = [], [], []
    for t in range(x64.shape[0]):
        if not is_visual[t]:
            rows.append(x64[t]); keep_idx.append(t); kind.append(KIND_TEXT)
            continue
        w = win_of.get(t)
        if w is None or action[w] == 0:
            rows.append(x64[t]); keep_idx.append(t); kind.append(KIND_KEPT)
        elif action[w] == 1 and t in first_of:
            members = vis[w * window:(w + 1) * window]
            rows.append(merge_window(x64[members], merge_mode)); keep_idx.append(t); kind.append(KIND_MERGED)
    kind = np.array(kind, dtype=np.uint8)
    return {"x_out": np.array(rows, F64).reshape(len(rows), x64.shape[1]),
            "is_visual_out": (kind != KIND_TEXT).astype(np.uint8),
            "keep_idx": np.array(keep_idx, dtype=np.int32), "kind": kind,
            "action": action, "C": C32, "A_bar": A32, "S": S, "m": m, "d": d, "kept_vis": kept}


def prune_visual(x, is_visual, probs, attn, seq_off, n_retain, window, alpha, gamma, sim_mode=0, merge_mode=0):
    """Section 3.2 on a batch of independent sequences given by token offsets
    seq_off[B+1]; outputs concatenated, keep_idx are global token indices."""
    outs = []
    for b in range(len(seq_off) - 1):
        lo, hi = int(seq_off[b]), int(seq_off[b + 1])
        o = prune_sequence(x[lo:hi], is_visual[lo:hi], probs[lo:hi], None if attn is None else attn[lo:hi],
                           n_retain[b], window, alpha, gamma, sim_mode, merge_mode)
        o["keep_idx"] = o["keep_idx"] + lo
        outs.append(o)
    out_off = np.zeros(len(outs) + 1, dtype=np.int64)
    out_off[1:] = np.cumsum([o["x_out"].shape[0] for o in outs])
    return {"x_out": np.concatenate([o["x_out"] for o in outs], axis=0),
            "is_visual_out": np.concatenate([o["is_visual_out"] for o in outs]),
            "keep_idx": np.concatenate([o["keep_idx"] for o in outs]),
            "kind": np.concatenate([o["kind"] for o in outs]),
            "out_seq_off": out_off, "per_seq": outs}


def attention_importance(q_last: np.ndarray, k: np.ndarray, seq_off: Sequence[int],
                         scale: Optional[float] = None) -> np.ndarray:
    """Eq. 7: A_hat = A[:, -1] of the head-averaged attention matrix, i.e. for each sequence the
    attention weights FROM its last token (the last text token of [T_v, T_t]) TO every token of the
    sequence, softmax over the sequence per head, then the mean over heads.  Returned for every
    token; the pruning stage reads the vision entries (Eq. 11).

    q_last [n_seq, n_heads, d]: the last tokens' queries; k [T, n_kv_heads, d]: the keys.
    READING: head h uses kv head h // (n_heads / n_kv_heads) (grouped-query attention, as in the
    paper's backbones); the last token sees the whole sequence, so the causal mask plays no role;
    scale defaults to 1/sqrt(d)."""
    q = np.asarray(q_last, F64)
    kk = np.asarray(k, F64)
    n_seq, n_heads, d = q.shape
    T, n_kv, _ = kk.shape
    group = n_heads // n_kv
    if scale is None:
        scale = 1.0 / math.sqrt(d)
    out = np.zeros(T, F64)
    for b in range(n_seq):
        lo, hi = int(seq_off[b]), int(seq_off[b + 1])
        if hi == lo:
            continue
        for h in range(n_heads):
            z = scale * (kk[lo:hi, h // group, :] @ q[b, h])
            e = np.exp(z - z.max())
            out[lo:hi] += e / e.sum()
    return out / n_heads


# ----------------------------------------------------------------------------
# Appendix D / E: closed forms
# ----------------------------------------------------------------------------
def gamma_hat(beta: float, window: int) -> float:
    """Appendix D: largest merge rate, reached when every removed token is
    removed by merging: gamma_hat = (1/beta - 1) / (W - 1)."""
    return (1.0 / beta - 1.0) / (window - 1)


def stage_beta(overall_retain: float, n_stages: int = 3) -> float:
    """Appendix D: equal per-stage retain ratio, beta = r^(1/stages)."""
    return overall_retain ** (1.0 / n_stages)


def moe_flops(n_tokens: int, n_pairs: int, hidden: int, n_experts: int, inter: int,
              n_shared: int = 0, shared_inter: int = 0) -> int:
    """Appendix E, MoE FFN term: 2*L*H*E for the router plus 6*H*S_m per activated
    (token, expert) pair; the per-token K of the paper becomes the actual pair
    count so that K_v < K is reflected.  Shared experts add 6*H*S_s per token each."""
    return 2 * n_tokens * hidden * n_experts + 6 * hidden * inter * n_pairs \
        + 6 * hidden * shared_inter * n_shared * n_tokens


# ----------------------------------------------------------------------------
# the stack of layers (pruning takes effect for the layers after the pruning layer)
# ----------------------------------------------------------------------------
def stack_forward(x, is_visual, seq_off, layer_weights: Sequence[dict], top_k, top_k_vis, reduce_from,
                  prune_after: Dict[int, dict], n_vis_original: Sequence[int]):
    """Layers 0..L-1 with residual adds.  Layer l uses K_v for vision tokens iff
    l >= reduce_from (inclusive).  A pruning stage "at layer l" scores with layer
    l's routing probabilities (computed on that layer's input), acts after the
    layer's output is formed, and shortens the input of layer l+1.
    READING: each stage's retention fraction refers to the ORIGINAL vision count.
    prune_after[l] = dict(window, alpha, gamma, retain, attn=None)."""
    x = np.asarray(x, F64)
    trace = []
    for l, w in enumerate(layer_weights):
        r = moe_forward(x, is_visual, w, top_k, top_k_vis, l >= reduce_from, add_residual=True)
        x = r["out"]
        if l in prune_after:
            pc = prune_after[l]
            eta = [int(math.floor(n * pc["retain"] + 1e-9)) for n in n_vis_original]
            p = prune_visual(x, is_visual, r["probs"], pc.get("attn"), seq_off, eta, pc["window"],
                             pc.get("alpha", 1.0), pc["gamma"])
            x, is_visual, seq_off = p["x_out"], p["is_visual_out"], p["out_seq_off"]
        trace.append({"n_tokens": x.shape[0], "n_pairs": int((r["topk_idx"] >= 0).sum())})
    return x, is_visual, seq_off, trace
