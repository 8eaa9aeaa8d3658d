"""GPU parity: routing-aware pruning (Eq. 6-18 + drop rule) through the C ABI against the
CPU oracle.  Keep-sets, kinds and offsets are compared bit-exactly (both sides rank
fp64-accumulated scores rounded once to fp32); rows within 2e-2 (bf16) / 1e-4 (fp32)."""
import numpy as np
import pytest
import torch

from oracle import fmmoe_oracle as O
from paper_2511_17885_b200 import binding as B
from paper_2511_17885_b200 import inputs as I
from gpu_util import dev, handle, host, row_rel_err, TDT

pytestmark = pytest.mark.gpu


def softmax_rows(r, n, e, smooth=None):
    z = r.standard_normal((n, e)).astype(np.float32)
    if smooth is not None:
        z = smooth
    z = z - z.max(1, keepdims=True)
    p = np.exp(z)
    return (p / p.sum(1, keepdims=True)).astype(np.float32)


def check_prune(dtype, seq_lens, H, E, W, retain, gamma, alpha, use_attn, sim_mode=0, merge_mode=0, seed=0,
                masks=None, contiguous_vision=False):
    r = np.random.default_rng(seed)
    T = int(sum(seq_lens))
    seq_off = np.concatenate([[0], np.cumsum(seq_lens)]).astype(np.int64)
    if masks is None:
        if contiguous_vision:
            mask = np.concatenate([(np.arange(L) < int(L * 0.9)).astype(np.uint8) for L in seq_lens])
        else:
            mask = I.interleaved_mask(T, r)
    else:
        mask = masks
    x = I.round_to_storage(r.standard_normal((T, H)) * (1 + r.random((T, 1))), dtype)
    # smooth logits so that neighbouring rows are similar, like vision tokens
    base = np.cumsum(0.3 * r.standard_normal((T, E)), axis=0).astype(np.float32)
    probs = softmax_rows(r, T, E, smooth=base)
    attn = r.random(T).astype(np.float32) if use_attn else None
    n_vis = np.array([int(mask[seq_off[b]:seq_off[b + 1]].sum()) for b in range(len(seq_lens))], np.int64)
    n_ret = I.retain_counts(n_vis, retain)
    p = B.prune_params(W, gamma, alpha, sim_mode, merge_mode)
    out = handle().fmmoe_prune_visual(p, dev(probs), dev(attn), dev(x, TDT[dtype]), dev(mask), seq_off, n_vis, n_ret)
    handle().check_status()
    ref = O.prune_visual(x, mask, probs, attn, seq_off, n_ret, W, alpha, gamma, sim_mode, merge_mode)
    assert out["out_seq_off"] == ref["out_seq_off"].tolist()
    assert np.array_equal(host(out["keep_idx"]), ref["keep_idx"])          # bit-exact keep-set
    assert np.array_equal(host(out["kind"]), ref["kind"])
    assert np.array_equal(host(out["is_visual_out"]), ref["is_visual_out"])
    y = host(out["x_out"])
    kept = ref["kind"] != 2
    assert np.array_equal(y[kept], x[ref["keep_idx"][kept]])                # copied rows are exact
    tol = 2e-2 if dtype == "bf16" else 1e-4
    assert row_rel_err(y, ref["x_out"]) < tol
    for b in range(len(seq_lens)):
        kc, m, d = B.fmmoe_prune_kept_count(int(n_vis[b]), int(n_ret[b]), p)
        assert (m, d, kc) == O.prune_counts(int(n_vis[b]), int(n_ret[b]), W, gamma, merge_mode)
    return out, ref


@pytest.mark.parametrize("W", [2, 3, 5, 8])
@pytest.mark.parametrize("use_attn", [False, True])
def test_prune_small(W, use_attn):
    check_prune("bf16", [301, 77, 512], 128, 24, W, 0.5, 0.08, 0.6, use_attn, seed=W)


@pytest.mark.parametrize("sim_mode,merge_mode", [(1, 0), (0, 1), (0, 2), (1, 2)])
def test_prune_modes(sim_mode, merge_mode):
    check_prune("bf16", [400, 333], 64, 40, 5, 0.4, 0.1, 0.5, True, sim_mode, merge_mode, seed=11)
    check_prune("f32", [260], 32, 9, 3, 0.25, 0.2, 0.7, False, sim_mode, merge_mode, seed=12)


def test_prune_identity_and_degenerate():
    out, ref = check_prune("bf16", [200, 100], 64, 16, 5, 1.0, 0.05, 0.5, True, seed=20)     # 100% retention
    assert out["x_out"].shape[0] == 300
    check_prune("bf16", [200], 64, 16, 5, 0.99, 0.05, 0.5, True, seed=21)                  # eps <= W: identity
    check_prune("bf16", [64], 64, 16, 5, 0.5, 0.0, 1.0, False, seed=22, masks=np.zeros(64, np.uint8))   # no vision
    check_prune("bf16", [7, 3], 64, 16, 5, 0.5, 0.05, 1.0, False, seed=23, masks=np.ones(10, np.uint8))  # tiny
    check_prune("bf16", [300], 64, 16, 4, 0.02, 0.9, 1.0, False, seed=24, masks=np.ones(300, np.uint8))  # gamma clamped
    check_prune("bf16", [300], 64, 16, 4, 0.0, 0.0, 1.0, True, seed=25, masks=np.ones(300, np.uint8))    # retain 0


def test_prune_ties_go_to_lower_window():
    # identical probability rows everywhere: all S equal (=1) -> merges and drops take the lowest windows
    T, H, E, W = 120, 64, 8, 3
    r = np.random.default_rng(30)
    x = I.round_to_storage(r.standard_normal((T, H)), "bf16")
    probs = np.tile(softmax_rows(r, 1, E), (T, 1))
    mask = np.ones(T, np.uint8)
    p = B.prune_params(W, 0.1, 1.0)
    out = handle().fmmoe_prune_visual(p, dev(probs), None, dev(x, torch.bfloat16), dev(mask), [0, T], [T], [60])
    ref = O.prune_visual(x, mask, probs, None, [0, T], [60], W, 1.0, 0.1)
    assert np.array_equal(host(out["keep_idx"]), ref["keep_idx"])
    act = ref["per_seq"][0]["action"]
    m, d, _ = O.prune_counts(T, 60, W, 0.1)
    assert act[:m].tolist() == [1] * m and act[m:m + d].tolist() == [2] * d


def test_prune_many_sequences_over_launch_chunks():
    lens = [50 + (i % 7) * 9 for i in range(70)]          # more than 64 sequences
    check_prune("bf16", lens, 64, 12, 3, 0.5, 0.05, 0.9, True, seed=40)


def test_prune_c0_and_c3_keep_sets():
    """Keep-sets on the routing probabilities the GPU router itself produces (C0 fp32, C3 sweep)."""
    from gpu_util import upload_weights, desc_of
    for cfg in (I.C0, I.C3):
        x, m, seq_off, n_vis = I.make_tokens(cfg)
        w = I.make_weights(cfg)
        wd = upload_weights(w, cfg.dtype); ws = B.make_weights(wd)
        xd, md = dev(x, TDT[cfg.dtype]), dev(m)
        rt = handle().fmmoe_route(desc_of(cfg), ws, xd, md, B.FLAG_REDUCE_ON, want=("probs", "topk_idx", "topk_w"))
        probs = host(rt["probs"])
        attn = I.make_attention_importance(cfg)
        for pc in cfg.prune:
            n_ret = I.retain_counts(n_vis, pc.retain)
            for a in (None, attn):
                p = B.prune_params(pc.window, pc.gamma, pc.alpha)
                out = handle().fmmoe_prune_visual(p, rt["probs"], dev(a), xd, md, seq_off, n_vis, n_ret)
                handle().check_status()
                ref = O.prune_visual(x, m, probs, a, seq_off, n_ret, pc.window, pc.alpha, pc.gamma)
                assert np.array_equal(host(out["keep_idx"]), ref["keep_idx"])
                assert np.array_equal(host(out["kind"]), ref["kind"])
                assert row_rel_err(host(out["x_out"]), ref["x_out"]) < (2e-2 if cfg.dtype == "bf16" else 1e-4)
    # kept counts of the sweep
    p = B.prune_params(5, 0.025)
    assert B.fmmoe_prune_kept_count(3328, 2496, p)[0] == 2500
    assert B.fmmoe_prune_kept_count(3328, 1664, B.prune_params(5, 0.05))[0] == 1666
    assert B.fmmoe_prune_kept_count(3328, 832, B.prune_params(5, 0.1))[0] == 836


@pytest.mark.parametrize("static", [False, True])
def test_mask_one_bit_short_of_n_vis_is_reported_not_followed(static):
    """The host says a sequence holds n_vis vision tokens, the mask sets one byte fewer.  The pass must end with
    FMMOE_ERR_INTERNAL from the status word - and must not index probs or x with list entries it never wrote,
    whatever the scratch held before (here: the leftovers of a larger earlier call, or a poisoned workspace).
    The next ordinary call on the same handle is unaffected."""
    h = handle()
    r = np.random.default_rng(77)
    H, E, W = 128, 16, 3
    p = B.prune_params(W, 0.1)
    # an earlier, longer call leaves large token indices behind in the shared scratch
    check_prune("bf16", [3000], H, E, W, 0.5, 0.1, 1.0, False, seed=78)
    L = 400
    mask = np.zeros(L, np.uint8); mask[:301] = 1
    n_vis_true = 301
    x = dev(I.round_to_storage(r.standard_normal((L, H)), "bf16"), torch.bfloat16)
    probs = dev(softmax_rows(r, L, E))
    bad = mask.copy(); bad[300] = 0                         # one set byte fewer than the count the host passes
    kept, _, _ = B.fmmoe_prune_kept_count(n_vis_true, 150, p)
    t_out = L - n_vis_true + kept
    if static:
        x_out = torch.zeros((t_out, H), dtype=torch.bfloat16, device="cuda")
        h.fmmoe_prune_visual_static(p, probs, None, x, dev(bad), [0, L], [n_vis_true], [150], x_out)
    else:
        h._ws = None                                        # a fresh workspace, poisoned with out-of-range indices
        ws = h.workspace(int(B.lib().fmmoe_prune_workspace_bytes(L, 1)))
        ws.fill_(0x7f)                                      # every int32 word reads 0x7f7f7f7f
        out = h.fmmoe_prune_visual(p, probs, None, x, dev(bad), [0, L], [n_vis_true], [150])
        assert out["x_out"].shape[0] == t_out
    assert h.get_status() == 6                              # FMMOE_ERR_INTERNAL, read and cleared
    torch.cuda.synchronize()                                # no fault: the context is still usable
    # the consistent call right after it passes parity
    check_prune("bf16", [L], H, E, W, 0.5, 0.1, 1.0, False, seed=79)
