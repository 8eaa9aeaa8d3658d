"""GPU parity at the full workload sizes, in the launch configuration the benchmark times.

C1 (DeepSeekMoE-style, 2,432 tokens), C2 (Qwen3-MoE-style, 3,584 tokens) and its batch of four,
C3 (pruning sweep at 75/50/25 % followed by the layer on the kept tokens) and C4 (24 layers,
8 x 2,432 tokens, K_v = 3 from layer 3, pruning after layers 3 and 12).  Integer results (expert
selections on the kernel's own fp32 logits, permutation, keep-sets) are compared bit-exactly over
ALL tokens, and so are the layer outputs: EVERY token row against the fp64 oracle (every expert a token
selected), within the bf16 tolerance of 2e-2 (max over rows of |y - ref|_inf / |ref|_inf).  C4 is
checked teacher-forced at its first layer, both pruning layers and the last layer, every row of each."""
import numpy as np
import pytest
import torch

from oracle import fmmoe_oracle as O
from paper_2511_17885_b200 import binding as B
from paper_2511_17885_b200 import inputs as I
from paper_2511_17885_b200.workload import LayerWorkload
from gpu_util import handle, host, row_rel_err

pytestmark = pytest.mark.gpu
TOL = 2e-2


def oracle_layer(x, mask, w, K, Kv, reduce_on, logits32, add_residual=False):
    """Oracle routing record and layer output for ALL token rows (routing from the kernel's fp32 logits)."""
    r = O.route(x, w["router_w"], w.get("router_b"), mask, K, Kv, reduce_on, logits32=logits32)
    out = O.moe_combine(x, r["topk_idx"], r["topk_w"], w, add_residual)
    return r, out


def check_layer_workload(cfg, handle_=None, fp8_weights=False):
    h = handle_ or handle()
    wl = LayerWorkload(cfg, h, device=0, prune=None, keep_host=True, fp8_weights=fp8_weights)
    T, E, K = cfg.n_tokens, cfg.n_experts, cfg.top_k
    wl.route = {"logits": torch.empty(T, E, dtype=torch.float32, device="cuda"),
                "probs": torch.empty(T, E, dtype=torch.float32, device="cuda"),
                "topk_idx": torch.empty(T, K, dtype=torch.int32, device="cuda"),
                "topk_w": torch.empty(T, K, dtype=torch.float32, device="cuda"),
                "expert_off": torch.empty(E + 1, dtype=torch.int32, device="cuda"),
                "row_token": torch.empty(T * K, dtype=torch.int32, device="cuda"),
                "inv_row": torch.empty(T, K, dtype=torch.int32, device="cuda")}
    wl.step()
    h.check_status()
    x, mask, w = wl.host["x"], wl.host["mask"], wl.host["w"]
    g = {k: host(v) for k, v in wl.route.items()}
    # every token: selection (on the kernel's logits), gates, permutation, layer output
    full, ref = oracle_layer(x, mask, w, K, cfg.top_k_vis, True, g["logits"])
    assert np.array_equal(g["topk_idx"], full["topk_idx"])
    assert np.abs(g["topk_w"] - full["topk_w"]).max() < 2e-5
    assert np.abs(g["probs"] - full["probs"]).max() < 2e-5
    scale = np.abs(full["logits"]).max()
    assert np.abs(g["logits"] - full["logits"]).max() / scale < 2e-5
    off, row_token, inv = O.permutation(full["topk_idx"], E)
    assert np.array_equal(g["expert_off"], off)
    assert np.array_equal(g["row_token"][:off[-1]], row_token)
    assert np.array_equal(g["inv_row"], inv)
    k_t = (full["topk_idx"] >= 0).sum(1)
    assert set(k_t[mask == 1].tolist()) == {cfg.top_k_vis} and set(k_t[mask == 0].tolist()) == {K}
    assert ref.shape == (T, cfg.hidden)
    err = row_rel_err(host(wl.out), ref)          # all T rows
    assert err < TOL, err
    return wl, g


def test_c1_full():
    wl, g = check_layer_workload(I.C1)
    assert int(g["expert_off"][-1]) == 2304 * 3 + 128 * 6


def test_c1_and_c2_full_with_fp8_expert_weights():
    """The full-size DeepSeekMoE-style and Qwen3-MoE-style layers with their expert matrices stored as FP8 bytes +
    block scales: every output row against the oracle fed the values that storage represents."""
    check_layer_workload(I.C1, fp8_weights=True)
    check_layer_workload(I.C2, fp8_weights=True)


def test_c2_full_and_batch_of_four():
    check_layer_workload(I.C2)
    wl, g = check_layer_workload(I.C2X4)
    assert int(g["expert_off"][-1]) == 4 * (3328 * 4 + 256 * 8)


def test_c3_sweep_keep_sets_and_downstream_forward():
    cfg = I.C3
    h = handle()
    wl = LayerWorkload(cfg, h, device=0, prune=None, keep_host=True)
    T, E, K = cfg.n_tokens, cfg.n_experts, cfg.top_k
    wl.route["logits"] = torch.empty(T, E, dtype=torch.float32, device="cuda")
    wl.step()
    x, mask, w = wl.host["x"], wl.host["mask"], wl.host["w"]
    probs = host(wl.route["probs"])
    kept_expected = {0.75: 2500, 0.5: 1666, 0.25: 836}
    for pc in cfg.prune:
        n_ret = I.retain_counts(wl.n_vis, pc.retain)
        pr = h.fmmoe_prune_visual(B.prune_params(pc.window, pc.gamma, pc.alpha), wl.route["probs"], None, wl.x, wl.mask,
                                  wl.seq_off, wl.n_vis, n_ret)
        h.check_status()
        ref = O.prune_visual(x, mask, probs, None, wl.seq_off, n_ret, pc.window, pc.alpha, pc.gamma)
        assert np.array_equal(host(pr["keep_idx"]), ref["keep_idx"])           # bit-exact keep-set
        assert np.array_equal(host(pr["kind"]), ref["kind"])
        assert int(host(pr["is_visual_out"]).sum()) == kept_expected[pc.retain]
        assert row_rel_err(host(pr["x_out"]), ref["x_out"]) < TOL
        # downstream layer on the kept tokens + 256 text tokens
        xk, mk = pr["x_out"], pr["is_visual_out"]
        Tk = xk.shape[0]
        route = {"logits": torch.empty(Tk, E, dtype=torch.float32, device="cuda"),
                 "topk_idx": torch.empty(Tk, K, dtype=torch.int32, device="cuda")}
        out = h.fmmoe_moe_forward(wl.desc, wl.ws, xk, mk, B.FLAG_REDUCE_ON, route=route)
        h.check_status()
        xk_h, mk_h, lg = host(xk), host(mk), host(route["logits"])
        full = O.route(xk_h, w["router_w"], None, mk_h, K, cfg.top_k_vis, True, logits32=lg)
        assert np.array_equal(host(route["topk_idx"]), full["topk_idx"])
        refo = O.moe_combine(xk_h, full["topk_idx"], full["topk_w"], w)      # every kept row
        assert row_rel_err(host(out), refo) < TOL


def test_c4_stack_full():
    """24 layers at full size: the stack driver against the same sequence of single-layer calls (bit for
    bit with the fixed-order combine), keep-sets of both stages bit-exact against the oracle, and ALL rows of
    the layer outputs teacher-forced against the oracle at the first layer, both pruning layers and the last."""
    sc = I.C4
    lc = sc.layer
    h = handle()
    dev = "cuda:0"
    td = torch.bfloat16
    x, mask, seq_off, n_vis = I.make_tokens(lc)
    xd = torch.from_numpy(x).to(dev).to(td).contiguous()
    md = torch.from_numpy(mask).to(dev)
    layers = [I.stack_layer_weights_torch(sc, l, dev) for l in range(sc.n_layers)]
    wstructs = [B.make_weights(w) for w in layers]
    desc = B.make_desc(lc.hidden, lc.n_experts, lc.inter, lc.n_shared, lc.shared_inter, lc.top_k, lc.top_k_vis, td)
    stages = [(l, pc.retain, B.prune_params(pc.window, pc.gamma, pc.alpha), None) for l, pc in sorted(sc.prune_after.items())]
    y, vis_out, out_off = h.fmmoe_stack_forward(desc, wstructs, sc.reduce_from, stages, xd, md, seq_off, n_vis,
                                                B.FLAG_DETERMINISTIC)
    h.check_status("stack")
    assert out_off[-1] == 8 * (577 + 128)
    assert bool(torch.isfinite(y.float()).all())
    E, K = lc.n_experts, lc.top_k
    checked = {0, 3, 12, sc.n_layers - 1}
    cur_x, cur_m, cur_off, cur_vis = xd, md, list(seq_off), [int(v) for v in n_vis]
    for l in range(sc.n_layers):
        T = cur_x.shape[0]
        reduce_on = l >= sc.reduce_from
        lf = B.FLAG_DETERMINISTIC | B.FLAG_RESIDUAL | (B.FLAG_REDUCE_ON if reduce_on else 0)
        route = {"probs": torch.empty(T, E, dtype=torch.float32, device=dev)}
        if l in checked:
            route["logits"] = torch.empty(T, E, dtype=torch.float32, device=dev)
            route["topk_idx"] = torch.empty(T, K, dtype=torch.int32, device=dev)
        out = h.fmmoe_moe_forward(desc, wstructs[l], cur_x, cur_m, lf, route=route)
        if l in checked:
            wh = {k: (None if v is None else v.float().cpu().numpy()) for k, v in layers[l].items()}
            xh, mh, lg = host(cur_x), host(cur_m), host(route["logits"])
            full = O.route(xh, wh["router_w"], wh["router_b"], mh, K, lc.top_k_vis, reduce_on, logits32=lg)
            assert np.array_equal(host(route["topk_idx"]), full["topk_idx"]), f"layer {l}: selection"
            ref = O.moe_combine(xh, full["topk_idx"], full["topk_w"], wh, add_residual=True)   # every row of the layer
            assert row_rel_err(host(out), ref) < TOL, f"layer {l}: output"
            del wh, ref
        if l in sc.prune_after:
            pc = sc.prune_after[l]
            eta = I.retain_counts(n_vis, pc.retain)
            pr = h.fmmoe_prune_visual(B.prune_params(pc.window, pc.gamma, pc.alpha), route["probs"], None, out, cur_m,
                                      cur_off, cur_vis, eta)
            ref = O.prune_visual(host(out), host(cur_m), host(route["probs"]), None, cur_off, eta, pc.window, pc.alpha,
                                 pc.gamma)
            assert np.array_equal(host(pr["keep_idx"]), ref["keep_idx"]), f"layer {l}: keep-set"
            assert np.array_equal(host(pr["kind"]), ref["kind"])
            n_text = [cur_off[b + 1] - cur_off[b] - cur_vis[b] for b in range(len(cur_vis))]
            cur_off = pr["out_seq_off"]
            cur_vis = [cur_off[b + 1] - cur_off[b] - n_text[b] for b in range(len(n_text))]
            cur_x, cur_m = pr["x_out"], pr["is_visual_out"]
        else:
            cur_x = out
    h.check_status("layerwise")
    assert cur_off == out_off
    assert torch.equal(cur_x, y) and torch.equal(cur_m, vis_out)


@pytest.mark.parametrize("retain", [0.75, 0.5, 0.25])
@pytest.mark.parametrize("model", ["internvl3.5", "deepseek-vl2"])
def test_paper_three_stage_schedules_at_full_size(model, retain):
    """The paper's two schedules (Appendix A: pruning after layers 5/8/12 with W = 5 on the Qwen3-MoE-style layer,
    after layers 2/5/8 with W = 3 on the DeepSeekMoE-style layer) at 75 / 50 / 25 % overall retention with the
    per-stage ratio r^(1/3) (Appendix D) and the (alpha, gamma) of that retention, attention-guided: A_hat comes
    from fmmoe_attention_importance on stand-in queries and keys of each pruning layer.  At every stage the keep-set
    and the kinds are bit-exact against the oracle (fed the kernel's fp32 probabilities and A_hat), A_hat itself is
    within 1e-5 of the oracle's Eq. 7, the kept count is in [eta, eta + W), and the stack driver equals the
    layer-by-layer calls bit for bit (fixed-order combine)."""
    sc = I.paper_stack(model, retain)
    lc = sc.layer
    h = handle()
    dev_, td = "cuda:0", torch.bfloat16
    x, mask, seq_off, n_vis = I.make_tokens(lc)
    xd = torch.from_numpy(x).to(dev_).to(td).contiguous()
    md = torch.from_numpy(mask).to(dev_)
    layers = [I.stack_layer_weights_torch(sc, l, dev_) for l in range(sc.n_layers)]
    wstructs = [B.make_weights(w) for w in layers]
    desc = B.make_desc(lc.hidden, lc.n_experts, lc.inter, lc.n_shared, lc.shared_inter, lc.top_k, lc.top_k_vis, td)
    E = lc.n_experts
    stages, attn_of, done = [], {}, []
    for layer, pc in sorted(sc.prune_after.items()):
        off_here, _ = B.fmmoe_stack_output_layout(done, layer + 1, seq_off, n_vis)
        q, k = I.make_stage_qk(sc, layer, off_here[-1], len(n_vis))
        a = h.fmmoe_attention_importance(torch.from_numpy(q).to(dev_).to(td), torch.from_numpy(k).to(dev_).to(td), off_here)
        ref_a = O.attention_importance(q, k, off_here)
        assert np.abs(host(a) - ref_a).max() <= 1e-5 * max(ref_a.max(), 1e-30) + 1e-9
        attn_of[layer] = a
        st = (layer, pc.retain, B.prune_params(pc.window, pc.gamma, pc.alpha), a)
        stages.append(st); done.append(st)
    flags = B.FLAG_DETERMINISTIC
    y, vis_out, out_off = h.fmmoe_stack_forward(desc, wstructs, sc.reduce_from, stages, xd, md, seq_off, n_vis, flags)
    h.check_status("stack")
    cur_x, cur_m, cur_off, cur_vis = xd, md, list(seq_off), [int(v) for v in n_vis]
    n_v0 = int(n_vis[0])
    for l in range(sc.n_layers):
        T = cur_x.shape[0]
        lf = flags | B.FLAG_RESIDUAL | (B.FLAG_REDUCE_ON if l >= sc.reduce_from else 0)
        route = {"probs": torch.empty(T, E, dtype=torch.float32, device=dev_)}
        out = h.fmmoe_moe_forward(desc, wstructs[l], cur_x, cur_m, lf, route=route)
        if l in sc.prune_after:
            pc = sc.prune_after[l]
            eta = I.retain_counts(n_vis, pc.retain)
            pr = h.fmmoe_prune_visual(B.prune_params(pc.window, pc.gamma, pc.alpha), route["probs"], attn_of[l], out,
                                      cur_m, cur_off, cur_vis, eta)
            ref = O.prune_visual(host(out), host(cur_m), host(route["probs"]), host(attn_of[l]), cur_off, eta, pc.window,
                                 pc.alpha, pc.gamma)
            assert np.array_equal(host(pr["keep_idx"]), ref["keep_idx"]), f"stage after layer {l}"
            assert np.array_equal(host(pr["kind"]), ref["kind"])
            assert row_rel_err(host(pr["x_out"]), ref["x_out"]) < TOL
            n_text = [cur_off[b + 1] - cur_off[b] - cur_vis[b] for b in range(len(cur_vis))]
            cur_off = pr["out_seq_off"]
            cur_vis = [cur_off[b + 1] - cur_off[b] - n_text[b] for b in range(len(n_text))]
            assert int(eta[0]) <= cur_vis[0] < int(eta[0]) + pc.window
            assert abs(pc.retain - retain ** ((sorted(sc.prune_after).index(l) + 1) / 3.0)) < 1e-12   # beta^t of the original
            cur_x, cur_m = pr["x_out"], pr["is_visual_out"]
        else:
            cur_x = out
    h.check_status("layerwise")
    assert cur_off == out_off and torch.equal(cur_x, y) and torch.equal(cur_m, vis_out)
    assert n_v0 * retain <= cur_vis[0] < n_v0 * retain + 3 * sc.prune_after[max(sc.prune_after)].window
    assert bool(torch.isfinite(y.float()).all())
