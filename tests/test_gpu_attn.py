"""GPU parity: cross-modal attention importance (Eq. 7) through the C ABI against the CPU oracle, and the
self-contained pruning chain (Eq. 7 -> Eq. 11-13 -> keep-set) that it feeds."""
import numpy as np
import pytest
import torch

from oracle import fmmoe_oracle as O
from paper_2511_17885_b200 import binding as B
from paper_2511_17885_b200 import inputs as I
from gpu_util import dev, handle, host, TDT

pytestmark = pytest.mark.gpu

CASES = [
    # dtype, seq_lens, n_heads, n_kv, d
    ("bf16", [2432], 32, 4, 128),
    ("bf16", [301, 77, 512], 8, 8, 64),
    ("f32", [100, 1, 33], 6, 2, 20),
    ("bf16", [64] * 70, 4, 1, 32),           # more sequences than one launch holds
]


@pytest.mark.parametrize("case", CASES)
def test_attention_importance_parity(case):
    dtype, lens, n_heads, n_kv, d = case
    r = np.random.default_rng(len(lens) + d)
    T = sum(lens)
    seq_off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    k = I.round_to_storage(r.standard_normal((T, n_kv, d)), dtype)
    q = I.round_to_storage(2.0 * r.standard_normal((len(lens), n_heads, d)), dtype)
    out = handle().fmmoe_attention_importance(dev(q, TDT[dtype]), dev(k, TDT[dtype]), seq_off)
    handle().check_status()
    ref = O.attention_importance(q, k, seq_off)
    g = host(out)
    assert np.abs(g - ref).max() <= 1e-5 * ref.max() + 1e-9
    for b in range(len(lens)):
        assert abs(g[seq_off[b]:seq_off[b + 1]].sum() - 1.0) < 1e-4
    again = handle().fmmoe_attention_importance(dev(q, TDT[dtype]), dev(k, TDT[dtype]), seq_off)
    assert torch.equal(out, again)                                    # reproducible bit for bit


def test_attention_guided_pruning_end_to_end():
    """Eq. 7 on the GPU feeds Eq. 11-13: the keep-set from the GPU's attention vector and routing
    probabilities equals the oracle's keep-set on the same two inputs."""
    cfg = I.C2
    r = np.random.default_rng(3)
    x, mask, seq_off, n_vis = I.make_tokens(cfg)
    T, E = cfg.n_tokens, cfg.n_experts
    n_heads, n_kv, d = 32, 4, 128
    k = I.round_to_storage(r.standard_normal((T, n_kv, d)), "bf16")
    q = I.round_to_storage(r.standard_normal((1, n_heads, d)), "bf16")
    z = np.cumsum(0.3 * r.standard_normal((T, E)), axis=0).astype(np.float32)
    z -= z.max(1, keepdims=True)
    probs = np.exp(z); probs = (probs / probs.sum(1, keepdims=True)).astype(np.float32)
    h = handle()
    attn = h.fmmoe_attention_importance(dev(q, torch.bfloat16), dev(k, torch.bfloat16), seq_off)
    pc = cfg.prune[1]
    n_ret = I.retain_counts(n_vis, pc.retain)
    out = h.fmmoe_prune_visual(B.prune_params(pc.window, pc.gamma, pc.alpha), dev(probs), attn, dev(x, torch.bfloat16),
                               dev(mask), seq_off, n_vis, n_ret)
    h.check_status()
    ref = O.prune_visual(x, mask, probs, host(attn), seq_off, n_ret, pc.window, pc.alpha, pc.gamma)
    assert np.array_equal(host(out["keep_idx"]), ref["keep_idx"])
    assert np.array_equal(host(out["kind"]), ref["kind"])


def test_attention_importance_invalid_arguments():
    h = handle()
    k = torch.zeros(10, 3, 16, dtype=torch.bfloat16, device="cuda")
    q = torch.zeros(1, 8, 16, dtype=torch.bfloat16, device="cuda")     # 8 heads over 3 kv heads
    with pytest.raises(B.FmmoeError):
        h.fmmoe_attention_importance(q, k, [0, 10])
    q2 = torch.zeros(1, 64, 16, dtype=torch.bfloat16, device="cuda")
    k2 = torch.zeros(10, 2, 16, dtype=torch.bfloat16, device="cuda")   # 32 query heads per kv head
    with pytest.raises(B.FmmoeError):
        h.fmmoe_attention_importance(q2, k2, [0, 10])
