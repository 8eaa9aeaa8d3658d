"""Pins for the oracle's Section 3.1 functions (Eq. 1-5) and the MoE output (Eq. 4).

Each test checks the oracle against something other than itself: explicit loops
on tiny non-square inputs, closed forms, library routines (torch fp64), and the
invariants the paper states (renormalised gates sum to one; K_v = K reproduces
the unreduced layer; an unselected expert contributes nothing; the Appendix C
angle identity for orthonormal expert outputs).
"""
import math

import numpy as np
import pytest
import torch

from oracle import fmmoe_oracle as O


def rng(seed):
    return np.random.default_rng(seed)


# ---------------------------------------------------------------- Eq. 1
def test_logits_explicit_loops_nonsquare():
    r = rng(1)
    T, H, E = 3, 4, 5
    x, w, b = r.standard_normal((T, H)), r.standard_normal((E, H)), r.standard_normal(E)
    z = O.router_logits(x, w, b)
    assert z.shape == (T, E)
    for t in range(T):
        for e in range(E):
            ref = sum(w[e, h] * x[t, h] for h in range(H)) + b[e]
            assert abs(z[t, e] - ref) < 1e-12
    z0 = O.router_logits(x, w)
    assert np.allclose(z - z0, b[None, :], atol=1e-12)


# ---------------------------------------------------------------- Eq. 2
def test_probs_closed_forms():
    # two experts: softmax is the logistic function of the logit difference
    z = np.array([[0.3, -1.1], [2.0, 2.0], [-50.0, 50.0]])
    p = O.routing_probs(z)
    for t in range(3):
        assert abs(p[t, 0] - 1.0 / (1.0 + math.exp(z[t, 1] - z[t, 0]))) < 1e-15
    assert np.allclose(p.sum(axis=1), 1.0, atol=1e-15)
    # uniform logits -> 1/E ; shift invariance ; large logits do not overflow
    assert np.allclose(O.routing_probs(np.full((2, 7), 3.0)), 1.0 / 7)
    zz = rng(2).standard_normal((4, 9))
    assert np.allclose(O.routing_probs(zz), O.routing_probs(zz + 1234.5), atol=1e-12)
    assert np.isfinite(O.routing_probs(zz * 1e4)).all()
    # library routine
    assert np.allclose(O.routing_probs(zz), torch.softmax(torch.from_numpy(zz), dim=1).numpy(), atol=1e-15)


# ---------------------------------------------------------------- Eq. 3
def test_experts_per_token_modalities():
    m = np.array([1, 0, 1, 1, 0], dtype=np.uint8)
    assert O.experts_per_token(m, 6, 3, True).tolist() == [3, 6, 3, 3, 6]
    assert O.experts_per_token(m, 6, 3, False).tolist() == [6, 6, 6, 6, 6]   # before layer l_v
    assert O.experts_per_token(m, 6, 0, True).tolist() == [0, 6, 0, 0, 6]     # p = 0 with shared experts


def test_selection_bruteforce_and_ties():
    r = rng(3)
    T, E, K = 40, 11, 4
    z = r.standard_normal((T, E)).astype(np.float32)
    z[5, [2, 7, 9]] = 3.0          # exact three-way tie at the top
    z[6, :] = 0.25                 # all equal
    k_t = r.integers(0, K + 1, size=T)
    idx = O.select_experts(z, k_t, K)
    for t in range(T):
        ranked = sorted(range(E), key=lambda e: (-float(z[t, e]), e))
        assert idx[t, :k_t[t]].tolist() == ranked[:k_t[t]]
        assert (idx[t, k_t[t]:] == -1).all()
        assert len(set(idx[t, :k_t[t]].tolist())) == k_t[t]
    assert idx[5, :3].tolist()[:min(3, k_t[5])] == [2, 7, 9][:min(3, k_t[5])]
    assert idx[6, :k_t[6]].tolist() == list(range(k_t[6]))


def test_selection_matches_library_topk_when_no_ties():
    z = rng(4).standard_normal((64, 32)).astype(np.float32)
    idx = O.select_experts(z, np.full(64, 5), 5)
    ref = torch.topk(torch.from_numpy(z), 5, dim=1).indices.numpy()
    assert (idx == ref).all()


# ---------------------------------------------------------------- Eq. 5
def test_gates_sum_to_one_and_ratio():
    r = rng(5)
    T, E, K, Kv = 50, 16, 6, 3
    z = r.standard_normal((T, E))
    p = O.routing_probs(z)
    vis = (r.random(T) < 0.7).astype(np.uint8)
    k_t = O.experts_per_token(vis, K, Kv, True)
    idx = O.select_experts(z.astype(np.float32), k_t, K)
    g = O.gates(p, idx)
    assert np.allclose(g.sum(axis=1), 1.0, atol=1e-12)           # halved-k weights sum to 1
    assert (g[idx < 0] == 0).all()
    for t in range(T):
        sel = idx[t, :k_t[t]]
        # equals a softmax restricted to the selected logits
        e = np.exp(z[t, sel] - z[t, sel].max())
        assert np.allclose(g[t, :k_t[t]], e / e.sum(), atol=1e-12)
        # g_i / g_j = P_i / P_j
        assert np.allclose(g[t, 0] / g[t, k_t[t] - 1], p[t, sel[0]] / p[t, sel[-1]], rtol=1e-12)


def test_gates_hand_example():
    # P = (.5,.25,.125,.125): top-2 -> (2/3, 1/3); top-1 -> 1
    p = np.array([[0.5, 0.25, 0.125, 0.125]])
    assert np.allclose(O.gates(p, np.array([[0, 1]])), [[2 / 3, 1 / 3]])
    assert np.allclose(O.gates(p, np.array([[0, -1]])), [[1.0, 0.0]])
    assert np.allclose(O.gates(p, np.array([[-1, -1]])), [[0.0, 0.0]])     # K_v = 0


def test_route_kv_equals_k_is_unreduced():
    r = rng(6)
    x, w = r.standard_normal((30, 12)), r.standard_normal((9, 12))
    vis = (r.random(30) < 0.5).astype(np.uint8)
    a = O.route(x, w, None, vis, 4, 4, True)
    b = O.route(x, w, None, vis, 4, 2, False)
    assert (a["topk_idx"] == b["topk_idx"]).all() and np.array_equal(a["topk_w"], b["topk_w"])
    c = O.route(x, w, None, vis, 4, 2, True)
    # reduced selection is the prefix of the full one; text rows untouched
    assert (c["topk_idx"][:, :2] == a["topk_idx"][:, :2]).all()
    assert (c["topk_idx"][vis == 0] == a["topk_idx"][vis == 0]).all()
    assert (c["topk_idx"][vis == 1, 2:] == -1).all()


# ---------------------------------------------------------------- permutation
def test_permutation_bruteforce():
    r = rng(7)
    T, K, E = 37, 3, 6
    idx = np.full((T, K), -1, dtype=np.int32)
    for t in range(T):
        k = int(r.integers(0, K + 1))
        idx[t, :k] = r.choice(E, size=k, replace=False)
    off, row_token, inv = O.permutation(idx, E)
    pairs = sorted((int(idx[t, s]), t, s) for t in range(T) for s in range(K) if idx[t, s] >= 0)
    assert off[-1] == len(pairs) == (idx >= 0).sum()
    assert row_token.tolist() == [p[1] for p in pairs]
    for row, (e, t, s) in enumerate(pairs):
        assert off[e] <= row < off[e + 1]
        assert inv[t, s] == row
    assert (inv[idx < 0] == -1).all()
    for e in range(E):
        seg = row_token[off[e]:off[e + 1]]
        assert (np.diff(seg) > 0).all()          # ascending tokens, each once


# ---------------------------------------------------------------- FFN / Eq. 4
def test_swiglu_against_library_and_loops():
    r = rng(8)
    T, H, I = 3, 5, 4
    x = r.standard_normal((T, H))
    wg, wu, wd = r.standard_normal((I, H)), r.standard_normal((I, H)), r.standard_normal((H, I))
    y = O.swiglu_ffn(x, wg, wu, wd)
    tx = torch.from_numpy(x)
    ref = torch.nn.functional.linear(
        torch.nn.functional.silu(torch.nn.functional.linear(tx, torch.from_numpy(wg)))
        * torch.nn.functional.linear(tx, torch.from_numpy(wu)), torch.from_numpy(wd)).numpy()
    assert np.allclose(y, ref, atol=1e-13)
    for t in range(T):
        a = []
        for i in range(I):
            g = sum(wg[i, h] * x[t, h] for h in range(H))
            u = sum(wu[i, h] * x[t, h] for h in range(H))
            a.append(g / (1 + math.exp(-g)) * u)
        for h in range(H):
            assert abs(y[t, h] - sum(wd[h, i] * a[i] for i in range(I))) < 1e-12


def _tiny_layer(r, T=24, H=8, E=6, I=5, ns=0):
    w = {"router_w": r.standard_normal((E, H)), "router_b": None,
         "w_gate": r.standard_normal((E, I, H)), "w_up": r.standard_normal((E, I, H)),
         "w_down": r.standard_normal((E, H, I)), "ws_gate": None, "ws_up": None, "ws_down": None}
    if ns:
        w["ws_gate"] = r.standard_normal((ns, I, H)); w["ws_up"] = r.standard_normal((ns, I, H))
        w["ws_down"] = r.standard_normal((ns, H, I))
    return r.standard_normal((T, H)), (r.random(T) < 0.6).astype(np.uint8), w


def test_moe_single_expert_is_plain_mlp():
    r = rng(9)
    x, vis, w = _tiny_layer(r, E=1)
    o = O.moe_forward(x, vis, w, 1, 1, True)["out"]
    assert np.allclose(o, O.swiglu_ffn(x, w["w_gate"][0], w["w_up"][0], w["w_down"][0]), atol=1e-12)


def test_moe_dense_sum_definition():
    """Eq. 4 literally: sum over ALL experts of g_j FFN_j with g_j = 0 off the set."""
    r = rng(10)
    x, vis, w = _tiny_layer(r, ns=2)
    rec = O.moe_forward(x, vis, w, 3, 1, True)
    E = w["w_gate"].shape[0]
    ref = np.zeros_like(x)
    for t in range(x.shape[0]):
        gfull = np.zeros(E)
        for s in range(3):
            if rec["topk_idx"][t, s] >= 0:
                gfull[rec["topk_idx"][t, s]] = rec["topk_w"][t, s]
        for e in range(E):
            ref[t] += gfull[e] * O.swiglu_ffn(x[t:t + 1], w["w_gate"][e], w["w_up"][e], w["w_down"][e])[0]
        for s in range(2):
            ref[t] += O.swiglu_ffn(x[t:t + 1], w["ws_gate"][s], w["ws_up"][s], w["ws_down"][s])[0]
    assert np.allclose(rec["out"], ref, atol=1e-11)
    res = O.moe_forward(x, vis, w, 3, 1, True, add_residual=True)["out"]
    assert np.allclose(res - rec["out"], x, atol=1e-12)


def test_moe_kv_equals_k_reproduces_dense_and_unselected_experts_are_skipped():
    r = rng(11)
    x, vis, w = _tiny_layer(r)
    a = O.moe_forward(x, vis, w, 3, 3, True)["out"]
    b = O.moe_forward(x, vis, w, 3, 1, False)["out"]
    assert np.array_equal(a, b)
    # poison an expert nobody selects: output must not change (g_j = 0 => not evaluated)
    w2 = dict(w); w2["router_w"] = w["router_w"].copy(); w2["router_w"][4] = 0.0
    w2["router_b"] = np.zeros(6); w2["router_b"][4] = -1e9
    w2["w_down"] = w["w_down"].copy(); w2["w_down"][4] = np.nan
    out = O.moe_forward(x, vis, w2, 3, 1, True)
    assert (out["topk_idx"] != 4).all() and np.isfinite(out["out"]).all()


def test_shared_only_when_kv_zero():
    r = rng(12)
    x, vis, w = _tiny_layer(r, ns=1)
    rec = O.moe_forward(x, vis, w, 2, 0, True)
    sh = O.swiglu_ffn(x, w["ws_gate"][0], w["ws_up"][0], w["ws_down"][0])
    assert np.allclose(rec["out"][vis == 1], sh[vis == 1], atol=1e-12)
    assert not np.allclose(rec["out"][vis == 0], sh[vis == 0])


def test_appendix_c_angle_identity_with_orthonormal_experts():
    """Appendix C: with orthonormal expert outputs p_i, reducing K -> m experts gives
    cos(theta) = sqrt(sum_{i<=m} a_i^2 / sum_{i<=K} a_i^2) >= sqrt(m/K)."""
    r = rng(13)
    H, E, I, K, m = 8, 8, 1, 6, 3
    x = r.standard_normal((1, H))
    w = {"router_w": r.standard_normal((E, H)), "router_b": None,
         "w_gate": r.standard_normal((E, I, H)), "w_up": r.standard_normal((E, I, H)),
         "w_down": np.zeros((E, H, I)), "ws_gate": None}
    tx = torch.from_numpy(x)
    for e in range(E):   # make FFN_e(x) the e-th basis vector, using the library's silu
        a = (torch.nn.functional.silu(tx @ torch.from_numpy(w["w_gate"][e]).T) * (tx @ torch.from_numpy(w["w_up"][e]).T)).item()
        w["w_down"][e, e, 0] = 1.0 / a
    vis = np.ones(1, dtype=np.uint8)
    full = O.moe_forward(x, vis, w, K, K, True)
    red = O.moe_forward(x, vis, w, K, m, True)
    y, y2 = full["out"][0], red["out"][0]
    cos = float(y @ y2 / np.linalg.norm(y) / np.linalg.norm(y2))
    a = full["topk_w"][0]
    assert (np.diff(a) <= 0).all()
    expect = math.sqrt((a[:m] ** 2).sum() / (a ** 2).sum())
    assert abs(cos - expect) < 1e-12
    assert cos >= math.sqrt(m / K) - 1e-12


def test_moe_flops_matches_appendix_e_formula():
    B, L, H, E, Sm, K = 2, 100, 64, 16, 32, 4
    assert O.moe_flops(B * L, B * L * K, H, E, Sm) == 2 * B * L * H * E + 6 * B * L * H * Sm * K


def test_moe_flops_counted_multiply_adds_with_shared_experts():
    """Every term of moe_flops against a literal count of the multiply-adds of Eq. 1 and Eq. 4 on a tiny layer:
    a matrix-vector product of an [out, in] matrix is out*in multiply-adds = 2*out*in FLOPs; an expert is three of
    them (gate, up, down); a token runs its selected routed experts and every shared expert."""
    T, H, E, Sm, Ns, Ss = 7, 6, 5, 4, 2, 3
    k_t = [3, 1, 1, 3, 1, 3, 1]                      # experts per token (K = 3 for text, K_v = 1 for vision)
    flops = 0
    for t in range(T):
        for e in range(E):                           # Eq. 1: one dot product of length H per expert
            for h in range(H):
                flops += 2
        for j in range(k_t[t]):                      # Eq. 4, routed: gate and up [Sm, H], down [H, Sm]
            for mat_out, mat_in in ((Sm, H), (Sm, H), (H, Sm)):
                for o in range(mat_out):
                    for i in range(mat_in):
                        flops += 2
        for s in range(Ns):                          # Eq. 4, shared: every token, every shared expert
            for mat_out, mat_in in ((Ss, H), (Ss, H), (H, Ss)):
                for o in range(mat_out):
                    for i in range(mat_in):
                        flops += 2
    assert O.moe_flops(T, sum(k_t), H, E, Sm, Ns, Ss) == flops
    assert O.moe_flops(T, sum(k_t), H, E, Sm) == flops - Ns * T * 6 * H * Ss      # the shared term on its own
