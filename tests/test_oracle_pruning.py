"""Pins for the oracle's Section 3.2 functions (Eq. 6-18, the drop rule) and the
Appendix D closed forms: printed values, hand-worked examples, library routines,
brute force on tiny inputs and the invariants the paper states (100% retention
is the identity; a merged token takes the largest member norm; order preserved).
"""
import itertools
import math
import os

import numpy as np
import pytest
from scipy.spatial.distance import cosine as scipy_cosine_distance

from oracle import fmmoe_oracle as O

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def rng(seed):
    return np.random.default_rng(seed)


def probs_like(r, n, e):
    z = r.standard_normal((n, e))
    p = np.exp(z)
    return (p / p.sum(1, keepdims=True)).astype(np.float32)


# ---------------------------------------------------------------- Eq. 8-10
def test_similarity_special_cases():
    e = np.eye(6)
    same = np.tile(rng(0).random(6), (5, 1))
    assert abs(O.window_similarity_pairwise(same) - 1) < 1e-12       # identical rows
    assert abs(O.window_similarity_mean(same) - 1) < 1e-12
    assert abs(O.window_similarity_pairwise(e[:4])) < 1e-15           # disjoint one-hots
    # rows (e0, e0, e1): pairs cos = 1, 0, 0 -> 1/3
    assert abs(O.window_similarity_pairwise(e[[0, 0, 1]]) - 1 / 3) < 1e-15
    # Eq. 10 for (e0, e1): mean = (e0+e1)/2, each cosine 1/sqrt(2)
    assert abs(O.window_similarity_mean(e[[0, 1]]) - 1 / math.sqrt(2)) < 1e-15
    # scale invariance of cosine; Eq. 10 for (e0,e0,e1): mean=(2,1,0)/3 -> (2*2/sqrt5 + 1/sqrt5)/3
    assert abs(O.window_similarity_mean(e[[0, 0, 1]]) - (5 / math.sqrt(5)) / 3) < 1e-15


def test_similarity_against_library_pairs():
    r = rng(1)
    for W in (2, 3, 5, 7):
        rw = probs_like(r, W, 17).astype(np.float64)
        ref = np.mean([1.0 - scipy_cosine_distance(rw[a], rw[b]) for a, b in itertools.combinations(range(W), 2)])
        assert abs(O.window_similarity_pairwise(rw) - ref) < 1e-13
        rbar = rw.mean(0)
        ref2 = np.mean([1.0 - scipy_cosine_distance(rw[a], rbar) for a in range(W)])
        assert abs(O.window_similarity_mean(rw) - ref2) < 1e-13
        s = O.window_similarity_pairwise(rw)
        assert 0 < s <= 1 + 1e-15                                    # non-negative vectors


# ---------------------------------------------------------------- Eq. 11-13
def test_scores_hand_example():
    # 2 windows of W=2 over one-hot-ish rows; attention sums 0.2 and 0.8
    e = np.eye(4, dtype=np.float32)
    probs = np.stack([e[0], e[0], e[1], e[2]])
    attn = np.array([0.1, 0.1, 0.5, 0.3], dtype=np.float32)
    C, A, S = O.window_scores(probs, attn, 2, 0.6)
    assert np.allclose(S, [1.0, 0.0])
    a_sum = np.array([float(attn[0]) + float(attn[1]), float(attn[2]) + float(attn[3])])
    assert np.allclose(A, (a_sum / a_sum.max()).astype(np.float32))          # Eq. 11-12: max becomes 1
    assert A.max() == 1.0
    expect = 0.6 * np.array([1.0, 0.0]) - 0.4 * (a_sum / a_sum.max())          # Eq. 13
    assert np.allclose(C, expect.astype(np.float32)) and C.dtype == np.float32
    # alpha = 1 -> C = S ; alpha = 0 -> C = -A_bar
    assert np.allclose(O.window_scores(probs, attn, 2, 1.0)[0], [1.0, 0.0])
    assert np.allclose(O.window_scores(probs, attn, 2, 0.0)[0], -(a_sum / a_sum.max()))
    # attention-free: C = S, no A_bar ; zero attention: A_bar = 0
    C2, A2, _ = O.window_scores(probs, None, 2, 0.3)
    assert A2 is None and np.allclose(C2, [1.0, 0.0])
    assert (O.window_scores(probs, np.zeros(4), 2, 0.5)[1] == 0).all()
    # ragged tail: 5 tokens, W=2 -> two windows only
    assert O.window_scores(np.vstack([probs, e[3:4]]), None, 2, 1.0)[0].shape == (2,)


# ---------------------------------------------------------------- Appendix D
def test_gamma_hat_closed_form_and_printed_table():
    rows = [tuple(map(float, l.split())) for l in open(os.path.join(GOLD, "gamma_hat_table.txt"))
            if l.strip() and not l.startswith("#")]
    assert [r for r, _, _ in rows] == [0.75, 0.5, 0.25]
    closed = []
    for r, beta_p, gh_p in rows:
        beta = O.stage_beta(r, 3)
        assert abs(round(beta, 2) - beta_p) < 1e-9                 # printed 0.91 / 0.79 / 0.63
        closed.append(O.gamma_hat(beta, 5))
    # the three printed bounds, one by one (W = 5, three stages):
    #   75 %: closed form 0.0252 -> printed 0.025 (the closed form to three decimals)
    assert abs(closed[0] - 0.0252) < 5e-5 and rows[0][2] == 0.025 and abs(closed[0] - rows[0][2]) < 5e-4
    #   25 %: closed form 0.1469 -> printed 0.15 (to two decimals)
    assert abs(closed[2] - 0.1469) < 5e-5 and rows[2][2] == 0.15 and round(closed[2], 2) == rows[2][2]
    #   50 %: closed form 0.0650, the paper prints 0.05: its own inconsistency (0.05 is the merge rate the
    #   experiments use at 50 %, a value below the bound); recorded here, not reconciled
    assert abs(closed[1] - 0.0650) < 5e-5 and rows[1][2] == 0.05 and closed[1] > rows[1][2]
    # the identity the bound is derived from: merging alone removes all eps tokens
    for n_v, eta, W in [(1000, 800, 5), (2304, 1152, 3), (3328, 2496, 5)]:
        gh = O.gamma_hat(eta / n_v, W)
        assert abs(gh - ((n_v - eta) / (W - 1)) / eta) < 1e-15


def test_counts_gamma_hat_means_no_drops():
    # eps divisible by W-1: at gamma = gamma_hat every removal is a merge, kept == eta exactly
    n_v, eta, W = 1000, 800, 5                       # eps=200 -> 50 merges
    gh = O.gamma_hat(eta / n_v, W)
    m, d, kept = O.prune_counts(n_v, eta, W, gh)
    assert (m, d, kept) == (50, 0, 800)
    # above the bound it is clamped
    assert O.prune_counts(n_v, eta, W, 0.9) == (50, 0, 800)


def test_counts_identity_cases_and_range():
    assert O.prune_counts(100, 100, 5, 0.05) == (0, 0, 100)        # 100% retention
    assert O.prune_counts(100, 120, 5, 0.05) == (0, 0, 100)
    assert O.prune_counts(100, 95, 5, 0.5) == (0, 0, 100)          # eps <= W: nothing happens
    assert O.prune_counts(100, 94, 5, 0.0)[1:] == (1, 95)          # eps = 6 > W: one window dropped
    for n_v, eta, W, g in itertools.product([97, 224, 3328], [20, 50, 90], [2, 3, 5], [0.0, 0.025, 0.1, 0.3]):
        m, d, kept = O.prune_counts(n_v, eta, W, g)
        assert kept == n_v - m * (W - 1) - d * W
        assert eta <= kept < eta + W
        assert m + d <= n_v // W and m <= math.floor(eta * g + 1e-9)
        assert O.prune_counts(n_v, eta, W, g, merge_mode=2)[0] == 0
    # hand-worked: N_v=3328, eta=2496, W=5, gamma=.025 -> m=62, u=832-248=584, d=116, kept 2500
    assert O.prune_counts(3328, 2496, 5, 0.025) == (62, 116, 2500)
    assert O.prune_counts(2304, 1152, 3, 0.05) == (57, 346, 1152)


# ---------------------------------------------------------------- Eq. 15 + drop rule
def test_select_windows_bruteforce_and_ties():
    r = rng(3)
    for n_f, m, d in [(12, 3, 4), (7, 0, 7), (9, 9, 0), (10, 2, 0), (6, 1, 5)]:
        C = r.standard_normal(n_f).astype(np.float32)
        A = r.random(n_f).astype(np.float32)
        C[1] = C[4]                                   # tie in C
        A[2] = A[5]                                   # tie in A
        act = O.select_windows(C, A, m, d)
        by_c = sorted(range(n_f), key=lambda i: (-float(C[i]), i))
        M = set(by_c[:m])
        rest = sorted((i for i in range(n_f) if i not in M), key=lambda i: (float(A[i]), i))
        D = set(rest[:d])
        assert [int(a) for a in act] == [1 if i in M else 2 if i in D else 0 for i in range(n_f)]
        # attention-free: drops continue down the C ranking
        act2 = O.select_windows(C, None, m, d)
        assert [int(a) for a in act2] == [1 if i in by_c[:m] else 2 if i in by_c[m:m + d] else 0 for i in range(n_f)]


def test_drop_only_sets_are_nested():
    r = rng(4)
    C = r.standard_normal(40).astype(np.float32)
    prev = set()
    for d in (5, 11, 23):
        cur = set(np.nonzero(O.select_windows(C, None, 0, d) == 2)[0].tolist())
        assert prev <= cur and len(cur) == d
        prev = cur


# ---------------------------------------------------------------- Eq. 16-18
def test_merge_norm_and_direction():
    r = rng(5)
    rows = r.standard_normal((5, 16)) * r.random((5, 1)) * 3
    mrg = O.merge_window(rows)
    mean = rows.mean(0)
    assert abs(np.linalg.norm(mrg) - max(np.linalg.norm(x) for x in rows)) < 1e-12
    assert abs(mrg @ mean / np.linalg.norm(mrg) / np.linalg.norm(mean) - 1) < 1e-12
    assert np.allclose(O.merge_window(rows, merge_mode=1), mean, atol=1e-15)
    assert (O.merge_window(np.array([[1.0, -2.0], [-1.0, 2.0]])) == 0).all()
    # hand example: rows (3,0),(0,4): mean (1.5,2) norm 2.5, max norm 4 -> (2.4, 3.2)
    assert np.allclose(O.merge_window(np.array([[3.0, 0.0], [0.0, 4.0]])), [2.4, 3.2])


# ---------------------------------------------------------------- whole sequence
def test_prune_identity_at_full_retention():
    r = rng(6)
    L, H, E = 40, 6, 8
    x = r.standard_normal((L, H)); vis = (np.arange(L) < 30).astype(np.uint8)
    p = probs_like(r, L, E)
    o = O.prune_sequence(x, vis, p, None, 30, 5, 0.5, 0.05)
    assert np.array_equal(o["x_out"], x) and o["keep_idx"].tolist() == list(range(L))
    assert (o["is_visual_out"] == vis).all()


def test_prune_hand_worked_sequence():
    """N_v=12 (W=3 -> 4 windows), 2 text tokens in front and 1 behind, eta=6, gamma=1/6.
    eps=6>3; m=floor(6/6)=1; u=6-2=4; d=1; kept=12-2-3=7.
    Similarities by construction: window 2 identical rows (S=1, merged);
    remaining windows ranked by attention: window 0 has the least -> dropped."""
    e = np.eye(8, dtype=np.float32)
    vis = np.array([0, 0] + [1] * 12 + [0], dtype=np.uint8)
    probs = np.zeros((15, 8), dtype=np.float32)
    probs[[0, 1, 14]] = e[7]
    probs[2:5] = e[[0, 1, 2]]            # window 0: S = 0
    probs[5:8] = e[[0, 0, 1]]            # window 1: S = 1/3
    probs[8:11] = e[[3, 3, 3]]           # window 2: S = 1
    probs[11:14] = e[[4, 4, 5]]          # window 3: S = 1/3
    attn = np.zeros(15, dtype=np.float32)
    attn[2:5] = 0.01; attn[5:8] = 0.2; attn[8:11] = 0.02; attn[11:14] = 0.1
    x = rng(7).standard_normal((15, 4))
    o = O.prune_sequence(x, vis, probs, attn, 6, 3, 0.9, 1 / 6)
    assert (o["m"], o["d"], o["kept_vis"]) == (1, 1, 7)
    assert o["action"].tolist() == [2, 0, 1, 0]
    assert o["keep_idx"].tolist() == [0, 1, 5, 6, 7, 8, 11, 12, 13, 14]
    assert o["kind"].tolist() == [0, 0, 1, 1, 1, 2, 1, 1, 1, 0]
    assert o["is_visual_out"].tolist() == [0, 0, 1, 1, 1, 1, 1, 1, 1, 0]
    assert np.array_equal(o["x_out"][[0, 1, 2, 9]], x[[0, 1, 5, 14]])
    assert np.allclose(o["x_out"][5], O.merge_window(x[8:11]))
    # attention-free: merge window 2, then drop the next most redundant (window 1; tie 1 vs 3 -> lower index)
    o2 = O.prune_sequence(x, vis, probs, None, 6, 3, 0.9, 1 / 6)
    assert o2["action"].tolist() == [0, 2, 1, 0]


def test_prune_interleaved_text_and_tail():
    r = rng(8)
    L, H, E, W = 61, 5, 6, 4
    vis = (r.random(L) < 0.7).astype(np.uint8)
    n_v = int(vis.sum()); eta = n_v // 2
    x = r.standard_normal((L, H)); p = probs_like(r, L, E); a = r.random(L).astype(np.float32)
    o = O.prune_sequence(x, vis, p, a, eta, W, 0.5, 0.1)
    m, d, kept = O.prune_counts(n_v, eta, W, 0.1)
    assert int(o["is_visual_out"].sum()) == kept
    assert (np.diff(o["keep_idx"]) > 0).all()                       # order preserved
    text = np.nonzero(vis == 0)[0]
    assert set(text.tolist()) <= set(o["keep_idx"].tolist())        # text always kept
    vis_idx = np.nonzero(vis)[0]
    tail = vis_idx[(n_v // W) * W:]
    assert set(tail.tolist()) <= set(o["keep_idx"].tolist())        # tail tokens always kept
    merged_rows = np.nonzero(o["kind"] == 2)[0]
    assert merged_rows.size == m
    for row in merged_rows:                                          # merged row sits at its window's first token
        v = int(np.nonzero(vis_idx == o["keep_idx"][row])[0][0])
        assert v % W == 0
        assert np.allclose(o["x_out"][row], O.merge_window(x[vis_idx[v:v + W]]))


def test_prune_batch_concatenation():
    r = rng(9)
    Ls = [30, 44]
    x = r.standard_normal((74, 4)); vis = np.ones(74, dtype=np.uint8); vis[25:30] = 0; vis[70:] = 0
    p = probs_like(r, 74, 5)
    off = np.array([0, 30, 74])
    b = O.prune_visual(x, vis, p, None, off, [12, 20], 3, 1.0, 0.1)
    s0 = O.prune_sequence(x[:30], vis[:30], p[:30], None, 12, 3, 1.0, 0.1)
    s1 = O.prune_sequence(x[30:], vis[30:], p[30:], None, 20, 3, 1.0, 0.1)
    assert b["out_seq_off"].tolist() == [0, len(s0["keep_idx"]), len(s0["keep_idx"]) + len(s1["keep_idx"])]
    assert b["keep_idx"].tolist() == s0["keep_idx"].tolist() + (s1["keep_idx"] + 30).tolist()
    assert np.array_equal(b["x_out"], np.vstack([s0["x_out"], s1["x_out"]]))


def test_stack_pruning_takes_effect_after_the_layer_and_reduce_from_is_inclusive():
    r = rng(10)
    H, E, I, T = 6, 5, 4, 26

    def layer():
        return {"router_w": r.standard_normal((E, H)), "router_b": None,
                "w_gate": 0.3 * r.standard_normal((E, I, H)), "w_up": 0.3 * r.standard_normal((E, I, H)),
                "w_down": 0.3 * r.standard_normal((E, H, I)), "ws_gate": None}
    ws = [layer() for _ in range(3)]
    x = r.standard_normal((T, H)); vis = (np.arange(T) < 20).astype(np.uint8)
    off = np.array([0, T])
    y, vis_o, off_o, trace = O.stack_forward(x, vis, off, ws, 2, 1, 1, {1: dict(window=2, gamma=0.1, retain=0.5)}, [20])
    # layer 0 unreduced (K for all), layer 1 reduced and still full length, layer 2 shortened
    assert trace[0]["n_pairs"] == T * 2
    assert trace[1]["n_pairs"] == 20 * 1 + 6 * 2
    # N_v=20, eta=10, W=2, gamma=.1: m=1, u=10-1=9, d=4 -> 20-1-8 = 11 vision tokens kept
    assert trace[0]["n_tokens"] == T and trace[1]["n_tokens"] == 11 + 6 and trace[2]["n_tokens"] == 17
    assert trace[2]["n_pairs"] == 11 * 1 + 6 * 2
    # manual replay
    a = O.moe_forward(x, vis, ws[0], 2, 1, False, add_residual=True)
    b = O.moe_forward(a["out"], vis, ws[1], 2, 1, True, add_residual=True)
    p = O.prune_visual(b["out"], vis, b["probs"], None, off, [10], 2, 1.0, 0.1)
    c = O.moe_forward(p["x_out"], p["is_visual_out"], ws[2], 2, 1, True, add_residual=True)
    assert np.allclose(y, c["out"], atol=1e-12)


# ---------------------------------------------------------------------------- Eq. 7
def _full_causal_attention(Q, K, scale):
    """Textbook attention probabilities of ONE head: softmax(mask(Q K^T * scale)), pure Python loops."""
    L = Q.shape[0]
    A = np.zeros((L, L))
    for i in range(L):
        z = [scale * sum(Q[i, c] * K[j, c] for c in range(Q.shape[1])) for j in range(i + 1)]
        m = max(z)
        e = [math.exp(v - m) for v in z]
        tot = sum(e)
        for j in range(i + 1):
            A[i, j] = e[j] / tot
    return A


def test_attention_importance_is_the_last_row_of_head_averaged_causal_attention():
    r = np.random.default_rng(0)
    lens, n_heads, n_kv, d = [7, 4], 4, 2, 6
    T = sum(lens)
    seq_off = np.concatenate([[0], np.cumsum(lens)])
    K = r.standard_normal((T, n_kv, d))
    Qfull = r.standard_normal((T, n_heads, d))                 # queries of every token; only the last ones matter
    q_last = np.stack([Qfull[seq_off[b + 1] - 1] for b in range(len(lens))])
    got = O.attention_importance(q_last, K, seq_off)
    want = np.zeros(T)
    for b in range(len(lens)):
        lo, hi = seq_off[b], seq_off[b + 1]
        Abar = sum(_full_causal_attention(Qfull[lo:hi, h], K[lo:hi, h // (n_heads // n_kv)], 1 / math.sqrt(d))
                   for h in range(n_heads)) / n_heads                                           # head-averaged A
        want[lo:hi] = Abar[-1, :]                                                               # A[:, -1] of Eq. 7
    assert np.allclose(got, want, atol=1e-14)


def test_attention_importance_invariants():
    r = np.random.default_rng(1)
    lens = [9, 5, 12]
    seq_off = np.concatenate([[0], np.cumsum(lens)])
    T = sum(lens)
    K = r.standard_normal((T, 2, 8)); q = r.standard_normal((3, 6, 8))
    a = O.attention_importance(q, K, seq_off)
    for b in range(3):
        assert abs(a[seq_off[b]:seq_off[b + 1]].sum() - 1.0) < 1e-14          # a distribution per sequence
    assert (a > 0).all()
    # identical keys (or a zero query): uniform attention
    Ku = np.tile(K[:1], (T, 1, 1))
    au = O.attention_importance(q, Ku, seq_off)
    for b in range(3):
        assert np.allclose(au[seq_off[b]:seq_off[b + 1]], 1.0 / lens[b])
    assert np.allclose(O.attention_importance(np.zeros_like(q), K, seq_off), au)
    # a key aligned with every head's query and a huge scale: all the weight on that token
    K2 = K.copy(); q2 = np.ones((3, 6, 8)); K2[:] = -np.ones(8); K2[4] = np.ones(8)
    a2 = O.attention_importance(q2, K2, seq_off, scale=50.0)
    assert abs(a2[4] - 1.0) < 1e-12 and a2[:4].max() < 1e-12
    # grouped-query attention == multi-head attention on the expanded keys
    Kx = np.repeat(K, 3, axis=1)
    assert np.allclose(O.attention_importance(q, Kx, seq_off), a, atol=1e-15)
    # a sequence's result does not depend on its neighbours
    alone = O.attention_importance(q[1:2], K[seq_off[1]:seq_off[2]], [0, lens[1]])
    assert np.allclose(alone, a[seq_off[1]:seq_off[2]], atol=1e-15)
