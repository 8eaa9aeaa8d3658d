"""fmmoe_prune_visual_static: pruning for callers that cannot allocate device memory.

Some users of this library prune inside a process where asking CUDA for memory is off the
table at that moment: the HBM was given to another pool at start-up, or the loop cannot
tolerate the synchronisation an allocation can trigger.  For them the library offers a
variant of fmmoe_prune_visual whose scratch is a fixed array built into the library.  This
test calls that variant through the C ABI and checks that it produces what the ordinary,
workspace-taking entry point produces - twice in a row, with different inputs, because the
built-in array is shared by all calls and still holds the previous call's contents.

This file is named so that pytest collects it after every other test file."""
import numpy as np
import pytest
import torch

from paper_2511_17885_b200 import binding as B
from paper_2511_17885_b200 import inputs as I
from gpu_util import dev, handle, host, row_rel_err

pytestmark = pytest.mark.gpu


def _case(seed, seq_lens, H, E):
    r = np.random.default_rng(seed)
    T = int(sum(seq_lens))
    seq_off = np.concatenate([[0], np.cumsum(seq_lens)]).astype(np.int64)
    mask = I.interleaved_mask(T, r)
    x = I.round_to_storage(r.standard_normal((T, H)) * (1 + r.random((T, 1))), "bf16")
    z = np.cumsum(0.3 * r.standard_normal((T, E)), axis=0).astype(np.float32)
    z -= z.max(1, keepdims=True)
    probs = np.exp(z)
    probs = (probs / probs.sum(1, keepdims=True)).astype(np.float32)
    attn = r.random(T).astype(np.float32)
    n_vis = np.array([int(mask[seq_off[b]:seq_off[b + 1]].sum()) for b in range(len(seq_lens))], np.int64)
    return x, mask, probs, attn, seq_off, n_vis


def _compare(h, seed, seq_lens, H, E, W, retain, gamma, alpha, use_attn):
    x, mask, probs, attn, seq_off, n_vis = _case(seed, seq_lens, H, E)
    n_ret = I.retain_counts(n_vis, retain)
    p = B.prune_params(W, gamma, alpha)
    xd, md, pd = dev(x, torch.bfloat16), dev(mask), dev(probs)
    ad = dev(attn) if use_attn else None
    want = h.fmmoe_prune_visual(p, pd, ad, xd, md, seq_off, n_vis, n_ret)          # existing entry point
    t_out = want["x_out"].shape[0]
    x_out = torch.zeros((t_out, H), dtype=torch.bfloat16, device="cuda")
    vis_out = torch.full((t_out,), 255, dtype=torch.uint8, device="cuda")
    keep_idx = torch.full((t_out,), -7, dtype=torch.int32, device="cuda")
    kind = torch.full((t_out,), 255, dtype=torch.uint8, device="cuda")
    off = h.fmmoe_prune_visual_static(p, pd, ad, xd, md, seq_off, n_vis, n_ret, x_out, vis_out, keep_idx, kind)
    h.check_status("fmmoe_prune_visual_static")
    assert off == want["out_seq_off"]
    assert 0 < t_out < x.shape[0]                                                   # something was pruned
    assert torch.equal(keep_idx, want["keep_idx"])                                  # index work: bit-exact
    assert torch.equal(kind, want["kind"])
    assert torch.equal(vis_out, want["is_visual_out"])
    assert row_rel_err(host(x_out), host(want["x_out"])) < 2e-2                     # rows: the bf16 tolerance
    assert (host(kind) == 2).any()                                                  # merged rows were exercised


def test_static_scratch_matches_workspace_entry_point_twice():
    h = handle()
    # first call: three sequences, W = 3, attention-guided score
    _compare(h, 101, [700, 333, 1200], 256, 64, 3, 0.5, 0.08, 0.6, True)
    # second call right after it: other shapes, so the array still holds unrelated leftovers
    _compare(h, 202, [2432, 97], 128, 24, 5, 0.3, 0.1, 1.0, False)


def test_static_scratch_rejects_sizes_beyond_its_limit():
    h = handle()
    T = B.STATIC_PRUNE_MAX_TOKENS + 1
    p = B.prune_params(3, 0.05)
    # the size check comes before any pointer is used, so small dummy buffers are enough
    d = torch.zeros(64, dtype=torch.float32, device="cuda")
    xb = torch.zeros((1, 64), dtype=torch.bfloat16, device="cuda")
    m = torch.zeros(64, dtype=torch.uint8, device="cuda")
    with pytest.raises(B.FmmoeError) as e:
        h.fmmoe_prune_visual_static(p, d.view(1, 64), None, xb, m, [0, T], [T], [T // 2], xb.clone())
    assert e.value.status == 7 and "TOO_LARGE" in str(e.value)
