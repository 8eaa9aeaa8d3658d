"""fmmoe_prune_visual_static: pruning for callers that cannot allocate device memory.

Some users of this library prune inside a process where asking CUDA for memory is off the
table at that moment: the HBM was given to another pool at start-up, or the loop cannot
tolerate the synchronisation an allocation can trigger.  For them the library offers a
variant of fmmoe_prune_visual whose scratch is a fixed array built into the library.  This
test calls that variant through the C ABI and checks that it produces what the ordinary,
workspace-taking entry point produces - twice in a row, with different inputs, because the
built-in array is shared by all calls and still holds the previous call's contents.  Both
entry points run the same kernels on the same inputs, so the comparison is bit for bit: a
race on the shared array or a leftover value that reached a merged row would show.

This file is named so that pytest collects it after every other test file."""
import numpy as np
import pytest
import torch

from paper_2511_17885_b200 import binding as B
from paper_2511_17885_b200 import inputs as I
from gpu_util import dev, handle

pytestmark = pytest.mark.gpu
TD = {"bf16": torch.bfloat16, "f32": torch.float32}


def _case(seed, seq_lens, H, E, dtype="bf16"):
    r = np.random.default_rng(seed)
    T = int(sum(seq_lens))
    seq_off = np.concatenate([[0], np.cumsum(seq_lens)]).astype(np.int64)
    mask = I.interleaved_mask(T, r)
    x = I.round_to_storage(r.standard_normal((T, H)) * (1 + r.random((T, 1))), dtype)
    z = np.cumsum(0.3 * r.standard_normal((T, E)), axis=0).astype(np.float32)
    z -= z.max(1, keepdims=True)
    probs = np.exp(z)
    probs = (probs / probs.sum(1, keepdims=True)).astype(np.float32)
    attn = r.random(T).astype(np.float32)
    n_vis = np.array([int(mask[seq_off[b]:seq_off[b + 1]].sum()) for b in range(len(seq_lens))], np.int64)
    return x, mask, probs, attn, seq_off, n_vis


def _compare(h, seed, seq_lens, H, E, W, retain, gamma, alpha, use_attn, dtype="bf16"):
    x, mask, probs, attn, seq_off, n_vis = _case(seed, seq_lens, H, E, dtype)
    n_ret = I.retain_counts(n_vis, retain)
    p = B.prune_params(W, gamma, alpha)
    xd, md, pd = dev(x, TD[dtype]), dev(mask), dev(probs)
    ad = dev(attn) if use_attn else None
    n0 = h.launch_count()
    want = h.fmmoe_prune_visual(p, pd, ad, xd, md, seq_off, n_vis, n_ret)          # existing entry point
    launches_ws = h.launch_count() - n0
    t_out = want["x_out"].shape[0]
    x_out = torch.zeros((t_out, H), dtype=TD[dtype], device="cuda")
    vis_out = torch.full((t_out,), 255, dtype=torch.uint8, device="cuda")
    keep_idx = torch.full((t_out,), -7, dtype=torch.int32, device="cuda")
    kind = torch.full((t_out,), 255, dtype=torch.uint8, device="cuda")
    torch.cuda.synchronize()
    # the call itself must not reach torch's allocator (cudaMalloc goes through it in this process)
    stats0 = torch.cuda.memory_stats()
    n1 = h.launch_count()
    off = h.fmmoe_prune_visual_static(p, pd, ad, xd, md, seq_off, n_vis, n_ret, x_out, vis_out, keep_idx, kind)
    stats1 = torch.cuda.memory_stats()
    assert stats1["allocation.all.allocated"] == stats0["allocation.all.allocated"]
    assert stats1["segment.all.allocated"] == stats0["segment.all.allocated"]
    assert h.launch_count() - n1 == launches_ws                                     # the same kernels
    h.check_status("fmmoe_prune_visual_static")
    assert off == want["out_seq_off"]
    assert 0 < t_out < x.shape[0]                                                   # something was pruned
    assert torch.equal(keep_idx, want["keep_idx"])                                  # index work: bit-exact
    assert torch.equal(kind, want["kind"])
    assert torch.equal(vis_out, want["is_visual_out"])
    assert torch.equal(x_out, want["x_out"])                                        # same kernels, same inputs: bit for bit
    assert bool((kind == 2).any())                                                  # merged rows were exercised


def test_static_scratch_matches_workspace_entry_point_twice():
    h = handle()
    # first call: three sequences, W = 3, attention-guided score
    _compare(h, 101, [700, 333, 1200], 256, 64, 3, 0.5, 0.08, 0.6, True)
    # second call right after it: other shapes, so the array still holds unrelated leftovers
    _compare(h, 202, [2432, 97], 128, 24, 5, 0.3, 0.1, 1.0, False)


def test_static_scratch_at_its_limit_in_fp32_and_with_many_sequences():
    h = handle()
    # the largest call the array admits: 32,768 tokens, W = 2 (the most windows per token), small rows
    _compare(h, 303, [B.STATIC_PRUNE_MAX_TOKENS], 64, 8, 2, 0.5, 0.05, 1.0, False)
    # fp32 rows
    _compare(h, 404, [900, 410], 64, 16, 4, 0.4, 0.1, 0.5, True, dtype="f32")
    # more sequences than one launch of the per-sequence kernels takes (64): 70 short ones
    _compare(h, 505, [60 + (i % 7) * 9 for i in range(70)], 64, 12, 3, 0.5, 0.1, 1.0, False)


def test_static_scratch_rejects_sizes_beyond_its_limit_and_short_outputs():
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
    # within the limit the wrapper refuses outputs that are too short for the rows the kernels will write
    x, mask, probs, attn, seq_off, n_vis = _case(606, [500], 64, 8)
    with pytest.raises(ValueError):
        h.fmmoe_prune_visual_static(p, dev(probs), None, dev(x, torch.bfloat16), dev(mask), seq_off, n_vis,
                                    I.retain_counts(n_vis, 0.5), torch.zeros((1, 64), dtype=torch.bfloat16, device="cuda"))
