"""The seeded generators: shapes, determinism, storage-exact values, and the
structure the workloads rely on (smooth vision fields, uncorrelated text)."""
import numpy as np
import torch

from paper_2511_17885_b200 import inputs as I


def test_shapes_and_determinism():
    for cfg in (I.C0, I.C1, I.C2):
        x, m, off, nv = I.make_tokens(cfg)
        assert x.shape == (cfg.n_tokens, cfg.hidden) and m.sum() == cfg.n_vis * cfg.batch
        assert off.tolist() == [0, cfg.seq_len] and nv.tolist() == [cfg.n_vis]
        x2, *_ = I.make_tokens(cfg)
        assert np.array_equal(x, x2)


def test_c0_layout():
    # the tiny workload is 256 tokens = 224 visual + 32 text; 224 = 14 x 16 raster
    assert (I.C0.n_vis, I.C0.n_text, I.C0.seq_len) == (224, 32, 256)


def test_bf16_values_are_storage_exact():
    x, *_ = I.make_tokens(I.C1)
    t = torch.from_numpy(x)
    assert torch.equal(t.to(torch.bfloat16).to(torch.float32), t)


def test_vision_is_smooth_text_is_not():
    x, m, *_ = I.make_tokens(I.C2)
    v = x[m == 1][:256].astype(np.float64)
    t = x[m == 0].astype(np.float64)

    def adj_cos(a):
        return np.mean(np.sum(a[1:] * a[:-1], 1) / np.linalg.norm(a[1:], axis=1) / np.linalg.norm(a[:-1], axis=1))
    rows = v.reshape(16, 16, -1)
    inrow = np.mean([adj_cos(rows[i]) for i in range(16)])
    assert inrow > 0.8 and abs(adj_cos(t)) < 0.1


def test_attention_importance_normalised():
    a = I.make_attention_importance(I.C2)
    assert a.dtype == np.float32 and abs(a[:I.C2.n_vis].sum() - 1) < 1e-4 and (a[I.C2.n_vis:] == 0).all()


def test_paper_three_stage_schedule():
    sch = I.paper_schedule("internvl3.5", 0.5)
    assert sorted(sch) == [5, 8, 12] and all(pc.window == 5 and pc.gamma == 0.05 and pc.alpha == 0.6 for pc in sch.values())
    assert abs(sch[12].retain - 0.5) < 1e-12 and abs(sch[5].retain - 0.5 ** (1 / 3)) < 1e-12      # beta ~ 0.79
    assert abs(round(sch[5].retain, 2) - 0.79) < 1e-9
    d = I.paper_schedule("deepseek-vl2", 0.25)
    assert sorted(d) == [2, 5, 8] and d[2].window == 3 and d[2].gamma == 0.2 and abs(round(d[2].retain, 2) - 0.63) < 1e-9
