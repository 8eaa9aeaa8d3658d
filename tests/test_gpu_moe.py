"""GPU parity: the whole MoE layer (Eq. 1-5) through the C ABI against the CPU oracle.
Tolerances: fp32 layers 1e-4, bf16 layers 2e-2, both as max over token rows of
|y - ref|_inf / |ref|_inf.  The oracle is teacher-forced on the kernel's fp32 logits for
the (integer) selection, so a near-tie cannot turn into a large output difference."""
import numpy as np
import pytest
import torch

from oracle import fmmoe_oracle as O
from paper_2511_17885_b200 import binding as B
from paper_2511_17885_b200 import inputs as I
from gpu_util import dev, handle, host, row_rel_err, upload_weights, TDT

pytestmark = pytest.mark.gpu
TOL = {"f32": 1e-4, "bf16": 2e-2}


def random_layer(r, dtype, H, E, I_, Ns, Is, std=0.05):
    def d(shape):
        return I.round_to_storage(std * r.standard_normal(shape), dtype)
    w = {"router_w": d((E, H)), "router_b": None, "w_gate": d((E, I_, H)), "w_up": d((E, I_, H)),
         "w_down": d((E, H, I_)), "ws_gate": None, "ws_up": None, "ws_down": None}
    if Ns:
        w["ws_gate"] = d((Ns, Is, H)); w["ws_up"] = d((Ns, Is, H)); w["ws_down"] = d((Ns, H, Is))
    return w


def run_layer(dtype, x, mask, w, K, Kv, flags, Ns=0, Is=0):
    td = TDT[dtype]
    T, H = x.shape
    E, I_ = w["w_gate"].shape[0], w["w_gate"].shape[1]
    desc = B.make_desc(H, E, I_, Ns, Is, K, Kv, td)
    wd = upload_weights(w, dtype)
    ws = B.make_weights(wd)
    route = {"logits": torch.empty(T, E, dtype=torch.float32, device="cuda"),
             "topk_idx": torch.empty(T, K, dtype=torch.int32, device="cuda"),
             "topk_w": torch.empty(T, K, dtype=torch.float32, device="cuda")}
    out = handle().fmmoe_moe_forward(desc, ws, dev(x, td), dev(mask), flags, route=route)
    handle().check_status()
    return host(out), {k: host(v) for k, v in route.items()}


def check_layer(dtype, T, H, E, I_, K, Kv, Ns=0, Is=0, flags=B.FLAG_REDUCE_ON, seed=0, mask=None, bias=False):
    r = np.random.default_rng(seed)
    x = I.round_to_storage(r.standard_normal((T, H)), dtype)
    mask = (r.random(T) < 0.7).astype(np.uint8) if mask is None else mask
    w = random_layer(r, dtype, H, E, I_, Ns, Is)
    if bias:
        w["router_b"] = (0.7 * r.standard_normal(E)).astype(np.float32)
    y, route = run_layer(dtype, x, mask, w, K, Kv, flags, Ns, Is)
    ref = O.moe_forward(x, mask, w, K, Kv, bool(flags & B.FLAG_REDUCE_ON), bool(flags & B.FLAG_RESIDUAL),
                        logits32=route["logits"])
    assert np.array_equal(route["topk_idx"], ref["topk_idx"])
    err = row_rel_err(y, ref["out"])
    assert err < TOL[dtype], f"row-relative error {err}"
    return y, ref


SMALL = [
    # dtype, T, H, E, I, K, Kv, Ns, Is
    ("f32", 256, 256, 8, 512, 2, 1, 0, 0),
    ("f32", 70, 64, 5, 36, 3, 1, 1, 20),
    ("bf16", 300, 128, 8, 128, 2, 1, 0, 0),
    ("bf16", 1000, 256, 16, 192, 4, 2, 2, 192),
    ("bf16", 515, 512, 40, 320, 6, 3, 1, 128),
    ("bf16", 129, 64, 4, 64, 2, 0, 1, 64),
]


@pytest.mark.parametrize("case", SMALL)
@pytest.mark.parametrize("det", [0, B.FLAG_DETERMINISTIC])
def test_layer_small(case, det):
    dtype, T, H, E, I_, K, Kv, Ns, Is = case
    check_layer(dtype, T, H, E, I_, K, Kv, Ns, Is, flags=B.FLAG_REDUCE_ON | det)


def test_layer_residual_and_reduce_off():
    check_layer("bf16", 200, 128, 8, 128, 3, 1, flags=B.FLAG_REDUCE_ON | B.FLAG_RESIDUAL)
    check_layer("bf16", 200, 128, 8, 128, 3, 1, flags=0)
    check_layer("f32", 90, 64, 6, 64, 2, 1, flags=B.FLAG_RESIDUAL)


def test_layer_edge_masks_and_empty_experts():
    T = 260
    check_layer("bf16", T, 128, 8, 128, 2, 1, mask=np.ones(T, np.uint8))
    check_layer("bf16", T, 128, 8, 128, 2, 1, mask=np.zeros(T, np.uint8))
    # a strong bias empties several experts and overloads others (multi-tile groups)
    r = np.random.default_rng(3)
    x = I.round_to_storage(r.standard_normal((T, 128)), "bf16")
    w = random_layer(r, "bf16", 128, 16, 128, 0, 0)
    w["router_b"] = np.array([8, 8, 8] + [-30] * 13, np.float32)
    mask = (r.random(T) < 0.5).astype(np.uint8)
    y, route = run_layer("bf16", x, mask, w, 3, 1, B.FLAG_REDUCE_ON)
    ref = O.moe_forward(x, mask, w, 3, 1, True, logits32=route["logits"])
    assert set(np.unique(route["topk_idx"][route["topk_idx"] >= 0]).tolist()) <= {0, 1, 2}
    assert row_rel_err(y, ref["out"]) < 2e-2


def test_layer_kv_equals_k_reproduces_dense():
    r = np.random.default_rng(4)
    T, H, E, I_ = 150, 128, 8, 128
    x = I.round_to_storage(r.standard_normal((T, H)), "bf16")
    mask = (r.random(T) < 0.6).astype(np.uint8)
    w = random_layer(r, "bf16", H, E, I_, 0, 0)
    a, _ = run_layer("bf16", x, mask, w, 3, 3, B.FLAG_REDUCE_ON | B.FLAG_DETERMINISTIC)
    b, _ = run_layer("bf16", x, mask, w, 3, 1, B.FLAG_DETERMINISTIC)      # reduce off: K for everyone
    assert np.array_equal(a, b)


def test_layer_deterministic_mode_is_reproducible():
    r = np.random.default_rng(6)
    T, H, E, I_ = 400, 256, 16, 128
    x = I.round_to_storage(r.standard_normal((T, H)), "bf16")
    mask = (r.random(T) < 0.6).astype(np.uint8)
    w = random_layer(r, "bf16", H, E, I_, 1, 128)
    a, _ = run_layer("bf16", x, mask, w, 4, 2, B.FLAG_REDUCE_ON | B.FLAG_DETERMINISTIC, 1, 128)
    b, _ = run_layer("bf16", x, mask, w, 4, 2, B.FLAG_REDUCE_ON | B.FLAG_DETERMINISTIC, 1, 128)
    assert np.array_equal(a, b)


def test_layer_c0_full_config():
    cfg = I.C0
    x, m, _, _ = I.make_tokens(cfg)
    w = I.make_weights(cfg)
    y, route = run_layer("f32", x, m, w, cfg.top_k, cfg.top_k_vis, B.FLAG_REDUCE_ON)
    ref = O.moe_forward(x, m, w, cfg.top_k, cfg.top_k_vis, True, logits32=route["logits"])
    assert np.array_equal(route["topk_idx"], ref["topk_idx"])
    assert row_rel_err(y, ref["out"]) < 1e-4
    assert int((ref["topk_idx"] >= 0).sum()) == 224 * 1 + 32 * 2


def test_forward_host_variant_and_empty():
    r = np.random.default_rng(7)
    T, H, E, I_ = 200, 128, 8, 128
    x = I.round_to_storage(r.standard_normal((T, H)), "bf16")
    mask = (r.random(T) < 0.6).astype(np.uint8)
    w = random_layer(r, "bf16", H, E, I_, 0, 0)
    desc = B.make_desc(H, E, I_, 0, 0, 2, 1, torch.bfloat16)
    wd = upload_weights(w, "bf16"); ws = B.make_weights(wd)
    xh = torch.from_numpy(x).to(torch.bfloat16).pin_memory()
    mh = torch.from_numpy(mask).pin_memory()
    oh = torch.empty_like(xh).pin_memory()
    handle().fmmoe_moe_forward_host(desc, ws, xh, mh, B.FLAG_REDUCE_ON | B.FLAG_DETERMINISTIC, oh)
    y, _ = run_layer("bf16", x, mask, w, 2, 1, B.FLAG_REDUCE_ON | B.FLAG_DETERMINISTIC)
    assert np.array_equal(oh.float().numpy(), y)
    # T = 0
    out = handle().fmmoe_moe_forward(desc, ws, torch.zeros(0, H, dtype=torch.bfloat16, device="cuda"),
                                     torch.zeros(0, dtype=torch.uint8, device="cuda"), 1)
    assert out.shape == (0, H)


def test_pipelined_host_batches_match_the_device_path():
    """Five different batches through the pipelined host-buffer calls, two in flight: each batch's layer
    output and pruned rows (downloaded on the library's copy stream) equal the device-resident path's."""
    r = np.random.default_rng(11)
    T, H, E, I_, K, Kv = 300, 128, 8, 128, 2, 1
    w = random_layer(r, "bf16", H, E, I_, 0, 0)
    wd = upload_weights(w, "bf16"); ws = B.make_weights(wd)
    desc = B.make_desc(H, E, I_, 0, 0, K, Kv, torch.bfloat16)
    hd = handle()
    seq_off, n_vis = [0, T], [200]
    pp = B.prune_params(5, 0.05)
    n_ret = [100]
    route = {"probs": torch.empty(T, E, dtype=torch.float32, device="cuda")}
    xs = [torch.from_numpy(I.round_to_storage(r.standard_normal((T, H)), "bf16")).to(torch.bfloat16).pin_memory()
          for _ in range(5)]
    mask_np = np.zeros(T, np.uint8); mask_np[:200] = 1
    mask_h = torch.from_numpy(mask_np).pin_memory()
    slots = [{"out_dev": torch.empty(T, H, dtype=torch.bfloat16, device="cuda"),
              "mask_dev": torch.empty(T, dtype=torch.uint8, device="cuda"), "ticket": None} for _ in range(2)]
    got = []
    for i, xh in enumerate(xs):
        sl = slots[i % 2]
        if sl["ticket"] is not None:
            hd.fmmoe_host_wait(sl["ticket"])
        out_h = torch.empty(T, H, dtype=torch.bfloat16).pin_memory()
        hd.fmmoe_moe_forward_host_async(desc, ws, xh, mask_h, B.FLAG_REDUCE_ON, out_h, slot=i % 2, route=route,
                                        out_dev=sl["out_dev"], is_visual_dev=sl["mask_dev"])
        pr = hd.fmmoe_prune_visual(pp, route["probs"], None, sl["out_dev"], sl["mask_dev"], seq_off, n_vis, n_ret,
                                   want_aux=False)
        pr_h = torch.empty(pr["x_out"].shape, dtype=torch.bfloat16).pin_memory()
        hd.fmmoe_download_async(pr_h, pr["x_out"])
        sl["keep"] = pr["x_out"]
        sl["ticket"] = hd.fmmoe_host_fence()
        got.append((out_h, pr_h, sl["ticket"]))
    for out_h, pr_h, t in got:
        hd.fmmoe_host_wait(t)
    hd.check_status()
    mask_d = dev(mask_np)
    for xh, (out_h, pr_h, _) in zip(xs, got):
        ref = hd.fmmoe_moe_forward(desc, ws, xh.cuda(), mask_d, B.FLAG_REDUCE_ON, route=route)
        pr = hd.fmmoe_prune_visual(pp, route["probs"], None, ref, mask_d, seq_off, n_vis, n_ret, want_aux=False)
        # the combine adds in a different order from call to call (atomics): compare within the bf16 tolerance
        assert row_rel_err(out_h.float().numpy(), ref.float().cpu().numpy()) < 2e-2
        assert pr_h.shape == pr["x_out"].shape
        assert row_rel_err(pr_h.float().numpy(), pr["x_out"].float().cpu().numpy()) < 2e-2
    with pytest.raises(B.FmmoeError):
        hd.fmmoe_host_wait(1 << 40)


@pytest.mark.parametrize("use_attn", [False, True])
def test_layer_and_pruning_in_one_call_equals_the_two_calls(use_attn):
    """fmmoe_moe_forward_prune (selection on a side stream beside the GEMMs) against fmmoe_moe_forward followed by
    fmmoe_prune_visual: the same keep-set bit for bit; with the fixed-order combine also the same rows bit for bit."""
    r = np.random.default_rng(21)
    H, E, I_, K, Kv = 128, 16, 128, 4, 2
    seq_off, n_vis = [0, 700, 1030, 1500], [520, 200, 331]
    T = seq_off[-1]
    mask_np = np.zeros(T, np.uint8)
    for b in range(3):
        idx = r.permutation(seq_off[b + 1] - seq_off[b])[:n_vis[b]] + seq_off[b]   # vision tokens interleaved with text
        mask_np[idx] = 1
    n_ret = [260, 50, 331]
    w = random_layer(r, "bf16", H, E, I_, 1, 64)
    wd = upload_weights(w, "bf16"); ws = B.make_weights(wd)
    desc = B.make_desc(H, E, I_, 1, 64, K, Kv, torch.bfloat16)
    x = dev(I.round_to_storage(r.standard_normal((T, H)), "bf16"), torch.bfloat16)
    mask = dev(mask_np)
    attn = dev(r.random(T).astype(np.float32)) if use_attn else None
    pp = B.prune_params(3, 0.1, 0.6 if use_attn else 1.0)
    hd = handle()
    for flags in (B.FLAG_REDUCE_ON | B.FLAG_DETERMINISTIC, B.FLAG_REDUCE_ON | B.FLAG_RESIDUAL):
        route_a = {"probs": torch.empty(T, E, dtype=torch.float32, device="cuda")}
        route_b = {"probs": torch.empty(T, E, dtype=torch.float32, device="cuda")}
        out_a = hd.fmmoe_moe_forward(desc, ws, x, mask, flags, route=route_a)
        ref = hd.fmmoe_prune_visual(pp, route_a["probs"], attn, out_a, mask, seq_off, n_vis, n_ret)
        out_b = torch.empty_like(x)
        for _ in range(2):   # twice: the side stream's second use must be ordered after the first
            got = hd.fmmoe_moe_forward_prune(desc, ws, x, mask, flags, out_b, route_b, pp, attn, seq_off, n_vis, n_ret)
        hd.check_status()
        assert got["out_seq_off"] == ref["out_seq_off"]
        assert torch.equal(route_a["probs"], route_b["probs"])
        for k in ("keep_idx", "kind", "is_visual_out"):
            assert torch.equal(got[k], ref[k]), k
        if flags & B.FLAG_DETERMINISTIC:
            assert torch.equal(out_a, out_b) and torch.equal(got["x_out"], ref["x_out"])
        else:
            assert row_rel_err(host(got["x_out"]), host(ref["x_out"])) < 2e-2
        # within one call the pruned rows are the call's own layer output: copied rows bit for bit
        copied = got["kind"] != 2
        assert torch.equal(got["x_out"][copied], out_b[got["keep_idx"][copied].long()])
    # argument errors surface before anything is enqueued
    with pytest.raises(B.FmmoeError):
        hd.fmmoe_moe_forward_prune(desc, ws, x, mask, B.FLAG_REDUCE_ON, out_b, route_b, pp, attn, [0, 700, 1030, 1499],
                                   n_vis, n_ret)


def test_upload_and_download_streams_order_against_the_compute_stream():
    """fmmoe_upload_async -> device call -> fmmoe_download_async, four batches over two buffer sets."""
    r = np.random.default_rng(31)
    T, H, E, I_, K, Kv = 260, 128, 8, 128, 2, 1
    w = random_layer(r, "bf16", H, E, I_, 0, 0)
    wd = upload_weights(w, "bf16"); ws = B.make_weights(wd)
    desc = B.make_desc(H, E, I_, 0, 0, K, Kv, torch.bfloat16)
    hd = handle()
    mask = dev((r.random(T) < 0.6).astype(np.uint8))
    xs = [torch.from_numpy(I.round_to_storage(r.standard_normal((T, H)), "bf16")).to(torch.bfloat16).pin_memory()
          for _ in range(4)]
    sets = [{"x": torch.empty(T, H, dtype=torch.bfloat16, device="cuda"),
             "out": torch.empty(T, H, dtype=torch.bfloat16, device="cuda"), "ticket": None} for _ in range(2)]
    res = []
    for i, xh in enumerate(xs):
        st = sets[i % 2]
        if st["ticket"] is not None:
            hd.fmmoe_host_wait(st["ticket"])
        hd.fmmoe_upload_async(st["x"], xh)
        hd.fmmoe_moe_forward(desc, ws, st["x"], mask, B.FLAG_REDUCE_ON | B.FLAG_DETERMINISTIC, out=st["out"])
        oh = torch.empty(T, H, dtype=torch.bfloat16).pin_memory()
        hd.fmmoe_download_async(oh, st["out"])
        st["ticket"] = hd.fmmoe_host_fence()
        res.append((oh, st["ticket"]))
    for oh, t in res:
        hd.fmmoe_host_wait(t)
    hd.check_status()
    for xh, (oh, _) in zip(xs, res):
        ref = hd.fmmoe_moe_forward(desc, ws, xh.cuda(), mask, B.FLAG_REDUCE_ON | B.FLAG_DETERMINISTIC)
        assert torch.equal(oh, ref.cpu())


def test_host_tickets_survive_the_ring_wrapping_around():
    """More fences than the handle keeps events for: every ticket, however old, can still be waited for."""
    hd = handle()
    src = torch.arange(1024, dtype=torch.int32, device="cuda")
    dst = torch.zeros(1024, dtype=torch.int32).pin_memory()
    tickets = []
    for i in range(150):
        src.add_(1)
        hd.fmmoe_download_async(dst, src)
        tickets.append(hd.fmmoe_host_fence())
    assert tickets == list(range(tickets[0], tickets[0] + 150))
    for t in (tickets[0], tickets[70], tickets[-1]):
        hd.fmmoe_host_wait(t)
    assert torch.equal(dst, src.cpu())
    with pytest.raises(B.FmmoeError):
        hd.fmmoe_host_wait(tickets[-1] + 1)


def _rows_per_expert_case(counts, n_text_extra, H=128, I_=192, seed=41):
    """Tokens whose first choice is fixed by construction, so that expert e receives exactly counts[e] first-choice
    rows: vision tokens (K_v = 1) carry their whole weight on that expert.  `n_text_extra` text tokens (K = 2) all
    take the last two experts, which therefore hold several M-tiles."""
    r = np.random.default_rng(seed)
    E = len(counts) + 2
    assign = np.concatenate([np.full(c, e) for e, c in enumerate(counts)]).astype(np.int64)
    r.shuffle(assign)
    T = assign.size + n_text_extra
    x = 0.25 * r.standard_normal((T, H))
    mask = np.ones(T, np.uint8)
    mask[assign.size:] = 0
    w = random_layer(r, "bf16", H, E, I_, 0, 0)
    router = np.zeros((E, H))
    for e in range(E):
        router[e, e] = 1.0                      # logit of expert e = x[t, e]
    w["router_w"] = I.round_to_storage(router, "bf16")
    x[np.arange(assign.size), assign] = 8.0     # first choice of every vision token
    x[assign.size:, E - 2] = 8.0                # text tokens: the two big experts
    x[assign.size:, E - 1] = 6.0
    return I.round_to_storage(x, "bf16"), mask, w, E


_SMALL_M = {"FMMOE_SMALL_M_MAX_TOKENS": "1000000", "FMMOE_GATHER_MIN_TOKENS": "1000000"}
_ATOMIC = {"FMMOE_PAIR_ROWS_MIN_TOKENS": "1000000"}       # the atomic fp32 combine (optional; the default is pair rows)
ROW_PATHS = {
    # name: environment read by fmmoe_create -> which kernels the expert GEMMs run as at this size
    "default": {},                                        # rows as N below 256 tokens, rows as M + gather above; pair rows
    "small_m": dict(_SMALL_M, **_ATOMIC),                 # rows as the MMA's N at every size
    "rows_as_m_copy": dict({"FMMOE_SMALL_M_MAX_TOKENS": "0", "FMMOE_GATHER_MIN_TOKENS": "1000000"}, **_ATOMIC),   # rows as M, expert-ordered copy of x
    "rows_as_m_gather": dict({"FMMOE_SMALL_M_MAX_TOKENS": "0", "FMMOE_GATHER_MIN_TOKENS": "0"}, **_ATOMIC),   # rows as M, in-GEMM gather
    # 256-row tiles on CTA pairs (optional form), with the atomic and the per-pair combine
    "cta_pairs": dict({"FMMOE_CTA_PAIR_MIN_TOKENS": "0"}, **_ATOMIC),
    "cta_pairs_pair_rows": {"FMMOE_CTA_PAIR_MIN_TOKENS": "0", "FMMOE_PAIR_ROWS_MIN_TOKENS": "0"},
    # the combine through per-pair bf16 rows (the default), under both forms
    "small_m_pair_rows": dict(_SMALL_M, FMMOE_PAIR_ROWS_MIN_TOKENS="0"),
    "rows_as_m_gather_pair_rows": {"FMMOE_SMALL_M_MAX_TOKENS": "0", "FMMOE_GATHER_MIN_TOKENS": "0",
                                   "FMMOE_PAIR_ROWS_MIN_TOKENS": "0"},
}


def handle_with_env(monkeypatch, env):
    for k, v in env.items():
        monkeypatch.setenv(k, v)
    h = B.Handle(0)                                  # the thresholds are read once, when the handle is created
    for k in env:
        monkeypatch.delenv(k, raising=False)
    return h


@pytest.mark.parametrize("path", list(ROW_PATHS))
def test_rows_per_expert_boundaries_on_every_gemm_form(path, monkeypatch):
    """Experts holding 0, 1, 15, 16, 17, 33, 64, 65, 96, 97, 128 and 129 rows (and two with several hundred), EVERY
    output row against the oracle, on each form of the expert GEMMs: token rows as the MMA's N dimension (the
    default below 256 tokens), rows as M reading the expert-ordered copy written by the scatter pass, and rows
    as M with the in-GEMM gather by token (the default from 256 tokens on)."""
    counts = [0, 1, 15, 16, 17, 33, 64, 65, 96, 97, 128, 129]
    x, mask, w, E = _rows_per_expert_case(counts, n_text_extra=300)
    h = handle_with_env(monkeypatch, ROW_PATHS[path])
    T, H = x.shape
    I_ = w["w_gate"].shape[1]
    desc = B.make_desc(H, E, I_, 0, 0, 2, 1, torch.bfloat16)
    wd = upload_weights(w, "bf16"); ws = B.make_weights(wd)
    route = {"logits": torch.empty(T, E, dtype=torch.float32, device="cuda"),
             "topk_idx": torch.empty(T, 2, dtype=torch.int32, device="cuda"),
             "expert_off": torch.empty(E + 1, dtype=torch.int32, device="cuda")}
    for flags in (B.FLAG_REDUCE_ON, B.FLAG_REDUCE_ON | B.FLAG_DETERMINISTIC):
        out = h.fmmoe_moe_forward(desc, ws, dev(x, torch.bfloat16), dev(mask), flags, route=route)
        h.check_status()
        got_counts = np.diff(host(route["expert_off"]))
        assert got_counts[:len(counts)].tolist() == counts and got_counts[-1] == 300 and got_counts[-2] == 300
        ref = O.moe_forward(x, mask, w, 2, 1, True, logits32=host(route["logits"]))
        assert np.array_equal(host(route["topk_idx"]), ref["topk_idx"])
        assert row_rel_err(host(out), ref["out"]) < 2e-2
    h.close()


@pytest.mark.parametrize("T", [1, 7, 16, 40])
def test_decode_sized_batches_with_shared_experts(T):
    """A handful of tokens (a decode step): every expert holds 0-3 rows, so each routed tile is one 16-row MMA
    column block; shared experts and odd feature-block counts (S_m = 192 = 128 + 64) included."""
    check_layer("bf16", T, 256, 16, 192, 4, 2, 1, 192, flags=B.FLAG_REDUCE_ON, seed=50 + T)
    check_layer("bf16", T, 128, 8, 64, 2, 1, 0, 0, flags=B.FLAG_REDUCE_ON | B.FLAG_DETERMINISTIC, seed=60 + T)


@pytest.mark.parametrize("T", [255, 256, 257])
def test_default_form_on_both_sides_of_its_size_threshold(T):
    """With the handle's defaults a bf16 layer runs with the token rows as the MMA's N dimension below 256 tokens
    and as its M dimension, gathering its rows, from 256 on: the last size of the one and the first two of the
    other, shared experts and residual included, against the oracle."""
    check_layer("bf16", T, 256, 8, 192, 4, 2, Ns=1, Is=128, flags=B.FLAG_REDUCE_ON | B.FLAG_RESIDUAL, seed=300 + T)


def test_small_m_form_equals_rows_as_m_form_bit_for_bit_in_fixed_order_mode(monkeypatch):
    """The three forms of the expert GEMMs (rows as N, rows as M, rows as M on CTA pairs) accumulate every output element over the same k order in fp32, so with the
    fixed-order combine their layer outputs are identical bit for bit."""
    r = np.random.default_rng(71)
    T, H, E, I_ = 900, 256, 16, 320
    x = I.round_to_storage(r.standard_normal((T, H)), "bf16")
    mask = (r.random(T) < 0.7).astype(np.uint8)
    w = random_layer(r, "bf16", H, E, I_, 1, 128)
    outs = []
    for env in (ROW_PATHS["small_m"], ROW_PATHS["rows_as_m_copy"], ROW_PATHS["cta_pairs"]):
        h = handle_with_env(monkeypatch, env)
        desc = B.make_desc(H, E, I_, 1, 128, 4, 2, torch.bfloat16)
        wd = upload_weights(w, "bf16"); ws = B.make_weights(wd)
        outs.append(h.fmmoe_moe_forward(desc, ws, dev(x, torch.bfloat16), dev(mask),
                                        B.FLAG_REDUCE_ON | B.FLAG_DETERMINISTIC).clone())
        h.check_status()
        h.close()
    assert torch.equal(outs[0], outs[1]) and torch.equal(outs[0], outs[2])


@pytest.mark.parametrize("k_block", [0, 5])
def test_bounded_wait_runs_out_and_the_handle_recovers(k_block):
    """The producer of GEMM-1 (one CTA, tiny shape) stops before it issues k-block `k_block`; the issuing thread's
    wait for that stage has a 3 ms budget and nothing will ever complete it.  Expected: the call returns, the kernels
    finish, fmmoe_get_status reports FMMOE_ERR_TIMEOUT exactly once, and the next ordinary call on the same handle
    passes parity (tensor memory was released, no barrier is left half-way)."""
    h = B.Handle(0)
    r = np.random.default_rng(81)
    T, H, E, I_ = 96, 512, 4, 128            # H = 512: eight k-blocks per GEMM-1 tile
    x = I.round_to_storage(r.standard_normal((T, H)), "bf16")
    mask = (r.random(T) < 0.5).astype(np.uint8)
    w = random_layer(r, "bf16", H, E, I_, 0, 0)
    desc = B.make_desc(H, E, I_, 0, 0, 2, 1, torch.bfloat16)
    wd = upload_weights(w, "bf16"); ws = B.make_weights(wd)
    xd, md = dev(x, torch.bfloat16), dev(mask)
    h.fmmoe_test_expire_wait(3_000_000, k_block)
    h.fmmoe_moe_forward(desc, ws, xd, md, B.FLAG_REDUCE_ON)
    assert h.get_status() == 5                # FMMOE_ERR_TIMEOUT, read and cleared
    assert h.get_status() == 0
    route = {"logits": torch.empty(T, E, dtype=torch.float32, device="cuda")}
    out = h.fmmoe_moe_forward(desc, ws, xd, md, B.FLAG_REDUCE_ON, route=route)
    h.check_status()
    ref = O.moe_forward(x, mask, w, 2, 1, True, logits32=host(route["logits"]))
    assert row_rel_err(host(out), ref["out"]) < 2e-2
    h.close()


@pytest.mark.parametrize("path", ["small_m_pair_rows", "rows_as_m_gather_pair_rows", "cta_pairs_pair_rows", "cta_pairs"])
def test_pair_row_combine_with_shared_experts_residual_and_reproducibility(path, monkeypatch):
    """The combine through per-pair bf16 rows: shared experts, residual, K_v = 0 tokens, against the oracle within
    the bf16 tolerance; it sums in a fixed order without atomics, so two runs agree bit for bit."""
    h = handle_with_env(monkeypatch, ROW_PATHS[path])
    r = np.random.default_rng(91)
    T, H, E, I_, Ns, Is, K, Kv = 700, 256, 16, 192, 2, 128, 4, 0
    x = I.round_to_storage(r.standard_normal((T, H)), "bf16")
    mask = (r.random(T) < 0.6).astype(np.uint8)
    w = random_layer(r, "bf16", H, E, I_, Ns, Is)
    desc = B.make_desc(H, E, I_, Ns, Is, K, Kv, torch.bfloat16)
    wd = upload_weights(w, "bf16"); ws = B.make_weights(wd)
    route = {"logits": torch.empty(T, E, dtype=torch.float32, device="cuda")}
    flags = B.FLAG_REDUCE_ON | B.FLAG_RESIDUAL
    a = h.fmmoe_moe_forward(desc, ws, dev(x, torch.bfloat16), dev(mask), flags, route=route).clone()
    b = h.fmmoe_moe_forward(desc, ws, dev(x, torch.bfloat16), dev(mask), flags, route=route)
    h.check_status()
    if "pair_rows" in path:          # the atomic combine adds in arrival order
        assert torch.equal(a, b)
    ref = O.moe_forward(x, mask, w, K, Kv, True, add_residual=True, logits32=host(route["logits"]))
    assert row_rel_err(host(a), ref["out"]) < 2e-2
    h.close()
