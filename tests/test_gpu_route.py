"""GPU parity: router + top-k + gates (Eq. 1-3, 5) and the permutation, through the C ABI,
against the CPU oracle on the same seeded inputs.  Selections and permutation indices are
compared bit-exactly (the oracle takes its decision on the kernel's own fp32 logits);
floating-point outputs within tolerances stated per test."""
import numpy as np
import pytest
import torch

from oracle import fmmoe_oracle as O
from paper_2511_17885_b200 import binding as B
from paper_2511_17885_b200 import inputs as I
from gpu_util import dev, handle, host, TDT

pytestmark = pytest.mark.gpu

CASES = [
    # dtype, T, H, E, K, Kv, bias, reduce_on
    ("f32", 256, 256, 8, 2, 1, False, 1),
    ("f32", 77, 100, 5, 3, 2, True, 1),
    ("bf16", 2432, 2048, 64, 6, 3, True, 1),
    ("bf16", 1000, 512, 72, 6, 2, False, 1),
    ("bf16", 333, 256, 128, 8, 4, False, 1),
    ("bf16", 65, 128, 200, 16, 1, True, 1),
    ("bf16", 31, 64, 256, 8, 8, False, 0),
    ("bf16", 1, 64, 33, 4, 0, False, 1),
]


def check_route(dtype, T, H, E, K, Kv, bias, reduce_on, seed=0, mask=None, x=None, w=None, b=None):
    r = np.random.default_rng(seed)
    x = I.round_to_storage(r.standard_normal((T, H)), dtype) if x is None else x
    w = I.round_to_storage(0.05 * r.standard_normal((E, H)), dtype) if w is None else w
    b = (0.5 * r.standard_normal(E)).astype(np.float32) if (bias and b is None) else b
    mask = (r.random(T) < 0.7).astype(np.uint8) if mask is None else mask
    td = TDT[dtype]
    desc = B.make_desc(H, E, 64, 1 if Kv == 0 else 0, 64, K, Kv, td)
    wd = {"router_w": dev(w, td), "router_b": dev(b)}
    ws = B.make_weights(wd)
    out = handle().fmmoe_route(desc, ws, dev(x, td), dev(mask), B.FLAG_REDUCE_ON if reduce_on else 0)
    handle().check_status()
    g = {k: host(v) for k, v in out.items()}
    ref = O.route(x, w, b, mask, K, Kv, bool(reduce_on), logits32=g["logits"])
    # logits: fp32 accumulation of exact products vs fp64
    scale = np.abs(ref["logits"]).max() + 1e-30
    assert np.abs(g["logits"] - ref["logits"]).max() / scale < 2e-5
    assert np.abs(g["probs"] - ref["probs"]).max() < 2e-5
    assert np.array_equal(g["topk_idx"], ref["topk_idx"])                       # bit-exact selection
    assert np.abs(g["topk_w"] - ref["topk_w"]).max() < 2e-5
    # independent selection check on the oracle's own logits: any disagreement must be a near-tie
    ind = O.route(x, w, b, mask, K, Kv, bool(reduce_on))
    bad = np.nonzero((ind["topk_idx"] != g["topk_idx"]).any(axis=1))[0]
    for t in bad:
        z = np.sort(ref["logits"][t])[::-1]
        k_t = int(ref["k_t"][t])
        gaps = np.abs(np.diff(z[:k_t + 1]))
        assert gaps.min() < 1e-4 * scale, f"token {t}: selection differs without a near-tie"
    assert len(bad) <= max(1, T // 100)
    # permutation: bit-exact
    off, row_token, inv = O.permutation(ref["topk_idx"], E)
    assert np.array_equal(g["expert_off"], off)
    P = off[-1]
    assert np.array_equal(g["row_token"][:P], row_token)
    assert np.array_equal(g["inv_row"], inv)
    return g, ref


@pytest.mark.parametrize("case", CASES)
def test_route_parity(case):
    check_route(*case)


def test_route_exact_ties_go_to_lower_index():
    # duplicate router rows => exactly equal logits
    r = np.random.default_rng(5)
    T, H, E = 64, 128, 16
    w = I.round_to_storage(0.05 * r.standard_normal((E, H)), "bf16")
    w[9] = w[2]; w[11] = w[2]; w[5] = w[4]
    g, ref = check_route("bf16", T, H, E, 4, 2, False, 1, w=w)
    z = g["logits"]
    assert np.array_equal(z[:, 9], z[:, 2]) and np.array_equal(z[:, 11], z[:, 2])
    for t in range(T):
        sel = g["topk_idx"][t][g["topk_idx"][t] >= 0].tolist()
        if 9 in sel:
            assert 2 in sel and sel.index(2) < sel.index(9)
        if 11 in sel:
            assert 9 in sel and sel.index(9) < sel.index(11)


def test_route_all_visual_all_text_and_constant_logits():
    check_route("bf16", 100, 64, 32, 4, 2, False, 1, mask=np.ones(100, np.uint8))
    check_route("bf16", 100, 64, 32, 4, 2, False, 1, mask=np.zeros(100, np.uint8))
    # zero router => all logits equal => experts 0..k-1, uniform gates
    g, _ = check_route("f32", 40, 64, 10, 3, 2, False, 1, w=np.zeros((10, 64), np.float32))
    assert (g["topk_idx"][:, 0] == 0).all() and (g["topk_idx"][:, 1] == 1).all()


def test_route_config_sequences():
    for cfg in (I.C0, I.C2):
        x, m, _, _ = I.make_tokens(cfg)
        w = I.make_weights(cfg)
        check_route(cfg.dtype, cfg.n_tokens, cfg.hidden, cfg.n_experts, cfg.top_k, cfg.top_k_vis, False, 1,
                    mask=m, x=x, w=w["router_w"], b=w["router_b"])


def test_route_empty_and_invalid():
    h = handle()
    desc = B.make_desc(64, 8, 64, 0, 0, 2, 1, torch.bfloat16)
    w = B.make_weights({"router_w": torch.zeros(8, 64, dtype=torch.bfloat16, device="cuda")})
    out = h.fmmoe_route(desc, w, torch.zeros(0, 64, dtype=torch.bfloat16, device="cuda"),
                        torch.zeros(0, dtype=torch.uint8, device="cuda"), 1)
    assert out["topk_idx"].shape == (0, 2)
    bad = B.make_desc(64, 8, 64, 0, 0, 2, 3, torch.bfloat16)       # K_v > K
    with pytest.raises(B.FmmoeError) as e:
        h.fmmoe_route(bad, w, torch.zeros(4, 64, dtype=torch.bfloat16, device="cuda"),
                      torch.zeros(4, dtype=torch.uint8, device="cuda"), 1)
    assert e.value.status == 1
    bad2 = B.make_desc(64, 8, 64, 0, 0, 2, 0, torch.bfloat16)      # K_v = 0 without shared experts
    assert B.fmmoe_workspace_bytes(bad2, 4) == 0
    un = B.make_desc(72, 8, 64, 0, 0, 2, 1, torch.bfloat16)        # H % 64 != 0 on the bf16 path
    with pytest.raises(B.FmmoeError) as e:
        h.fmmoe_route(un, w, torch.zeros(4, 72, dtype=torch.bfloat16, device="cuda"),
                      torch.zeros(4, dtype=torch.uint8, device="cuda"), 1)
    assert e.value.status == 2


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
def test_route_non_finite_activations_still_give_valid_distinct_experts(dtype):
    """Overflowed activations upstream (inf / nan rows) must not turn into out-of-range expert indices:
    the router clamps non-finite logits before it selects, so every token gets k distinct experts in
    [0, E) and the permutation stays consistent."""
    r = np.random.default_rng(8)
    T, H, E, K, Kv = 300, 128, 24, 4, 2
    x = I.round_to_storage(r.standard_normal((T, H)), dtype)
    x[5] = np.inf; x[17] = np.nan; x[40, ::2] = -np.inf; x[41] = 3e38
    w = I.round_to_storage(0.05 * r.standard_normal((E, H)), dtype)
    mask = (r.random(T) < 0.5).astype(np.uint8)
    td = TDT[dtype]
    desc = B.make_desc(H, E, 64, 0, 64, K, Kv, td)
    ws = B.make_weights({"router_w": dev(w, td)})
    out = handle().fmmoe_route(desc, ws, dev(x, td), dev(mask), B.FLAG_REDUCE_ON)
    handle().check_status()
    idx = host(out["topk_idx"])
    for t in range(T):
        k = Kv if mask[t] else K
        sel = idx[t, :k]
        assert (sel >= 0).all() and (sel < E).all() and len(set(sel.tolist())) == k, (t, sel)
        assert (idx[t, k:] == -1).all()
    off, row_token, inv = O.permutation(idx, E)
    assert np.array_equal(host(out["expert_off"]), off)
    assert np.array_equal(host(out["row_token"])[:off[-1]], row_token)
    assert np.array_equal(host(out["inv_row"]), inv)
