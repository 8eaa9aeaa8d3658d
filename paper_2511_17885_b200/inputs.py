"""Seeded synthetic inputs for the FastMMoE MoE-layer hot path.

This module only *draws* tensors (hidden states, weights, modality masks,
attention-importance vectors) and names the workload shapes.  It holds none of
the method's arithmetic: no routing, no softmax, no top-k, no similarity, no
pruning.  Both the CPU oracle's tests and the CUDA path's tests/bench take
their inputs from here, by value, so the two sides see identical numbers.

The shapes stand in for the multimodal prefill workloads the paper measures
(InternVL3.5 on a Qwen3-MoE backbone: 128 routed experts, top-8; DeepSeek-VL2
on a DeepSeekMoE backbone: shared + routed experts), whose images, prompts and
trained weights are not available here.  What is kept is what the method is
sensitive to: thousands of visual tokens laid out tile by tile in raster order
whose neighbouring hidden states are strongly correlated (Section 1 / Figure 1:
adjacent vision tokens route almost identically), followed by a short run of
uncorrelated text tokens (Section 3.2.1: T = [T_v, T_t]).

All float tensors are returned as float32 numpy arrays whose values are exactly
representable in the workload's storage dtype (bf16 values are rounded once,
here), so a float64 upcast (oracle) and a bf16 cast (GPU) are both lossless.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, List, Optional, Tuple

import numpy as np


# ----------------------------------------------------------------------------
# workload descriptions
# ----------------------------------------------------------------------------
@dataclass(frozen=True)
class PruneCfg:
    """Hyper-parameters of one pruning stage (Section 3.2, Appendix A)."""
    window: int            # W
    gamma: float           # merge rate (Eq. 14)
    alpha: float           # score trade-off (Eq. 13); used only with attention
    retain: float          # fraction of the ORIGINAL visual tokens to retain


@dataclass(frozen=True)
class LayerCfg:
    """One MoE layer + one multimodal sequence layout."""
    name: str
    dtype: str                         # "f32" | "bf16"
    hidden: int                        # H
    n_experts: int                     # E
    inter: int                         # S_m (routed expert intermediate size)
    n_shared: int                      # N_s
    shared_inter: int                  # per shared expert
    top_k: int                         # K
    top_k_vis: int                     # K_v
    grids: Tuple[Tuple[int, int], ...]  # visual tiles (rows, cols), raster order
    n_text: int
    router_bias_std: float = 0.0
    seed: int = 0
    batch: int = 1
    prune: Tuple[PruneCfg, ...] = ()

    @property
    def n_vis(self) -> int:
        return int(sum(r * c for r, c in self.grids))

    @property
    def seq_len(self) -> int:
        return self.n_vis + self.n_text

    @property
    def n_tokens(self) -> int:
        return self.seq_len * self.batch


_T16 = (16, 16)

C0 = LayerCfg(name="C0-tiny-f32", dtype="f32", hidden=256, n_experts=8, inter=512,
              n_shared=0, shared_inter=0, top_k=2, top_k_vis=1,
              grids=((14, 16),), n_text=32, seed=0,   # 224 visual tokens: a 14 x 16 raster
              prune=(PruneCfg(window=5, gamma=0.05, alpha=0.6, retain=0.5),))

C1 = LayerCfg(name="C1-deepseekmoe-bf16", dtype="bf16", hidden=2048, n_experts=64,
              inter=1408, n_shared=2, shared_inter=1408, top_k=6, top_k_vis=3,
              grids=(_T16,) * 9, n_text=128, router_bias_std=0.5, seed=1,
              prune=(PruneCfg(window=3, gamma=0.05, alpha=0.9, retain=0.5),))

C2 = LayerCfg(name="C2-qwen3moe-bf16", dtype="bf16", hidden=2048, n_experts=128,
              inter=768, n_shared=0, shared_inter=0, top_k=8, top_k_vis=4,
              grids=(_T16,) * 13, n_text=256, seed=2,
              prune=(PruneCfg(window=5, gamma=0.025, alpha=0.5, retain=0.75),
                     PruneCfg(window=5, gamma=0.05, alpha=0.6, retain=0.50),
                     PruneCfg(window=5, gamma=0.1, alpha=1.0, retain=0.25)))

C2X4 = replace(C2, name="C2x4-qwen3moe-bf16", batch=4)

# C3 is the pruning sweep on the C2 layer: same layer and sequence, the three
# PruneCfg entries above are its three retention points.
C3 = replace(C2, name="C3-prune-sweep", seed=3)


@dataclass(frozen=True)
class StackCfg:
    """C4: a stack of identical-shape MoE layers with residual adds."""
    name: str
    layer: LayerCfg
    n_layers: int
    reduce_from: int                        # l_v (inclusive, 0-based)
    prune_after: Dict[int, PruneCfg] = field(default_factory=dict)
    seed: int = 4


C4 = StackCfg(
    name="C4-stack24-bf16",
    layer=replace(C1, name="C4-layer", batch=8, seed=4, prune=()),
    n_layers=24, reduce_from=3,
    prune_after={3: PruneCfg(window=3, gamma=0.05, alpha=0.9, retain=0.5),
                 12: PruneCfg(window=3, gamma=0.2, alpha=0.7, retain=0.25)},
    seed=4)

CONFIGS = {"C0": C0, "C1": C1, "C2": C2, "C2x4": C2X4, "C3": C3}


# ----------------------------------------------------------------------------
# helpers (storage-dtype rounding only)
# ----------------------------------------------------------------------------
def round_to_storage(a: np.ndarray, dtype: str) -> np.ndarray:
    """Round a float array once to the storage dtype, return as float32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    if dtype == "f32":
        return a
    if dtype == "bf16":
        import torch
        return torch.from_numpy(a).to(torch.bfloat16).to(torch.float32).numpy()
    raise ValueError(dtype)


def _spawn(seed: int, n: int) -> List[np.random.Generator]:
    return [np.random.default_rng(s) for s in np.random.SeedSequence(seed).spawn(n)]


def smooth_field(rng: np.random.Generator, rows: int, cols: int, channels: int,
                 sigma: float = 2.0, noise_std: float = 0.1) -> np.ndarray:
    """A [rows*cols, channels] raster of spatially smooth values plus noise.

    Per channel: an N(0,1) grid, Gaussian-filtered (sigma in patches, reflect
    boundary, truncated at 4 sigma), rescaled to zero mean / unit std over the
    grid, plus N(0, noise_std^2).
    """
    from scipy.ndimage import gaussian_filter
    g = rng.standard_normal((rows, cols, channels))
    g = gaussian_filter(g, sigma=(sigma, sigma, 0.0), mode="reflect", truncate=4.0)
    g -= g.mean(axis=(0, 1), keepdims=True)
    g /= g.std(axis=(0, 1), keepdims=True) + 1e-12
    g += noise_std * rng.standard_normal((rows, cols, channels))
    return g.reshape(rows * cols, channels)


# ----------------------------------------------------------------------------
# tensors
# ----------------------------------------------------------------------------
def make_sequence(cfg: LayerCfg, rng: np.random.Generator) -> Tuple[np.ndarray, np.ndarray]:
    """Hidden states [L, H] and modality mask [L] for one sequence (vision first)."""
    parts = [smooth_field(rng, r, c, cfg.hidden) for r, c in cfg.grids]
    if cfg.n_text:
        parts.append(rng.standard_normal((cfg.n_text, cfg.hidden)))
    x = np.concatenate(parts, axis=0)
    is_visual = np.zeros(cfg.seq_len, dtype=np.uint8)
    is_visual[:cfg.n_vis] = 1
    return round_to_storage(x, cfg.dtype), is_visual


def make_tokens(cfg: LayerCfg, seed: Optional[int] = None):
    """Batch of sequences flattened: x [T,H], is_visual [T], seq_off [B+1], n_vis [B]."""
    seed = cfg.seed if seed is None else seed
    rngs = _spawn(seed * 1000 + 17, cfg.batch)
    xs, ms = zip(*(make_sequence(cfg, r) for r in rngs))
    x = np.concatenate(xs, axis=0)
    is_visual = np.concatenate(ms, axis=0)
    seq_off = np.arange(cfg.batch + 1, dtype=np.int64) * cfg.seq_len
    n_vis = np.full(cfg.batch, cfg.n_vis, dtype=np.int64)
    return x, is_visual, seq_off, n_vis


def make_weights(cfg: LayerCfg, seed: Optional[int] = None, std: float = 0.02) -> Dict[str, Optional[np.ndarray]]:
    """Router + expert weights, N(0, std^2), nn.Linear layout [out, in]."""
    seed = cfg.seed if seed is None else seed
    r = _spawn(seed * 1000 + 29, 8)
    H, E, I = cfg.hidden, cfg.n_experts, cfg.inter

    def draw(rng, shape):
        return round_to_storage(std * rng.standard_normal(shape, dtype=np.float32), cfg.dtype)

    w: Dict[str, Optional[np.ndarray]] = {
        "router_w": draw(r[0], (E, H)),
        "router_b": None,
        "w_gate": draw(r[1], (E, I, H)),
        "w_up": draw(r[2], (E, I, H)),
        "w_down": draw(r[3], (E, H, I)),
        "ws_gate": None, "ws_up": None, "ws_down": None,
    }
    if cfg.router_bias_std > 0:
        w["router_b"] = (cfg.router_bias_std * r[4].standard_normal(E)).astype(np.float32)
    if cfg.n_shared:
        Is = cfg.shared_inter
        w["ws_gate"] = draw(r[5], (cfg.n_shared, Is, H))
        w["ws_up"] = draw(r[6], (cfg.n_shared, Is, H))
        w["ws_down"] = draw(r[7], (cfg.n_shared, H, Is))
    return w


def make_attention_importance(cfg: LayerCfg, seed: Optional[int] = None) -> np.ndarray:
    """Stand-in for the last-text-token -> vision attention row (Eq. 7), per token.

    A positive vector over every token (text entries are ignored by the method)
    that sums to one over each sequence's vision tokens: exp of a smooth field
    per tile, normalised.  float32.
    """
    seed = cfg.seed if seed is None else seed
    rngs = _spawn(seed * 1000 + 43, cfg.batch)
    out = []
    for rng in rngs:
        f = np.concatenate([smooth_field(rng, r, c, 1, noise_std=0.3)[:, 0] for r, c in cfg.grids])
        e = np.exp(f - f.max())
        e /= e.sum()
        out.append(np.concatenate([e, np.zeros(cfg.n_text)]))
    return np.concatenate(out).astype(np.float32)


def retain_counts(n_vis: np.ndarray, retain: float) -> np.ndarray:
    """eta per sequence for a retention fraction (of the counts given)."""
    return np.floor(np.asarray(n_vis, dtype=np.float64) * retain + 1e-9).astype(np.int64)


# Appendix A: per-model pruning hyper-parameters, keyed by the OVERALL retention of the three-stage schedule.
PAPER_SCHEDULES = {
    "internvl3.5": {"layers": (5, 8, 12), "window": 5,
                    0.75: dict(alpha=0.5, gamma=0.025), 0.50: dict(alpha=0.6, gamma=0.05), 0.25: dict(alpha=1.0, gamma=0.1)},
    "deepseek-vl2": {"layers": (2, 5, 8), "window": 3,
                     0.75: dict(alpha=0.3, gamma=0.05), 0.50: dict(alpha=0.9, gamma=0.05), 0.25: dict(alpha=0.7, gamma=0.2)},
}


def paper_schedule(model: str, overall_retain: float) -> Dict[int, PruneCfg]:
    """The paper's three-stage schedule (Appendix A and D): pruning after three designated layers with the
    same per-stage ratio beta = r^(1/3), so that stage t keeps beta^t of the ORIGINAL vision tokens."""
    sc = PAPER_SCHEDULES[model]
    hp = sc[overall_retain]
    beta = overall_retain ** (1.0 / 3.0)
    return {layer: PruneCfg(window=sc["window"], gamma=hp["gamma"], alpha=hp["alpha"], retain=beta ** (t + 1))
            for t, layer in enumerate(sc["layers"])}


def paper_stack(model: str, overall_retain: float) -> StackCfg:
    """A stack that carries the paper's three-stage schedule of one backbone family (Appendix A): the layer shape of
    the matching single-layer workload, one sequence, as many layers as the schedule needs plus one more (so that
    the last stage's output is consumed by a layer), expert reduction from layer 2 on."""
    layer = {"internvl3.5": C2, "deepseek-vl2": C1}[model]
    sched = paper_schedule(model, overall_retain)
    return StackCfg(name=f"paper-{model}-{int(overall_retain * 100)}", layer=replace(layer, name=f"{model}-layer", prune=()),
                    n_layers=max(sched) + 2, reduce_from=2, prune_after=sched, seed=50 + int(overall_retain * 100))


def make_stage_qk(cfg: StackCfg, layer: int, n_tokens: int, n_seq: int, n_heads: int = 16, n_kv_heads: int = 4,
                  head_dim: int = 64):
    """Stand-in for the attention layer's tensors that Eq. 7 reads at a pruning layer: the last tokens' queries
    [n_seq, n_heads, d] and the keys [n_tokens, n_kv_heads, d] of the sequence as it is at that layer.  Keys are a
    smooth random walk over the tokens plus noise (neighbouring vision tokens attend alike), bf16 values."""
    rq, rk = _spawn(cfg.seed * 1000 + 61 + layer, 2)
    q = rq.standard_normal((n_seq, n_heads, head_dim))
    walk = np.cumsum(0.15 * rk.standard_normal((n_tokens, n_kv_heads, head_dim)), axis=0)
    k = walk / (np.abs(walk).max() + 1e-9) * 3.0 + 0.3 * rk.standard_normal((n_tokens, n_kv_heads, head_dim))
    return round_to_storage(q, "bf16"), round_to_storage(k, "bf16")


def interleaved_mask(n_tokens: int, rng: np.random.Generator, p_vis: float = 0.7) -> np.ndarray:
    """A modality mask with text and vision runs interleaved (edge-case tests)."""
    m = np.zeros(n_tokens, dtype=np.uint8)
    t = 0
    while t < n_tokens:
        run = int(rng.integers(1, 12))
        m[t:t + run] = 1 if rng.random() < p_vis else 0
        t += run
    return m


def stack_layer_weights_torch(cfg: StackCfg, layer: int, device: str):
    """Weights of one layer of the C4 stack, drawn ON `device` with a torch generator.

    27 GB of distinct weights are too slow to draw on the host; the same call
    with the same (seed, layer, device type) reproduces the same tensors, and
    the oracle's tests copy the slices they need to the host.
    Returns a dict of torch tensors in the layer's storage dtype (+ fp32 bias).
    """
    import torch
    lc = cfg.layer
    g = torch.Generator(device=device)
    g.manual_seed(cfg.seed * 100003 + layer)
    dt = torch.bfloat16 if lc.dtype == "bf16" else torch.float32
    H, E, I = lc.hidden, lc.n_experts, lc.inter

    def draw(shape, std=0.02):
        t = torch.empty(shape, device=device, dtype=torch.float32)
        t.normal_(0.0, std, generator=g)
        return t.to(dt)

    # Residual-branch scaling: without normalisation layers (the stack has none) a residual stack whose
    # down-projections have the same std as the other weights grows quadratically per layer and
    # overflows bf16 by layer ~9; std / sqrt(2 * n_layers) keeps the activations at unit scale.
    down_std = 0.02 / float(np.sqrt(2.0 * cfg.n_layers))
    w = {"router_w": draw((E, H)),
         "router_b": torch.empty(E, device=device, dtype=torch.float32).normal_(0.0, lc.router_bias_std, generator=g)
         if lc.router_bias_std > 0 else None,
         "w_gate": draw((E, I, H)), "w_up": draw((E, I, H)), "w_down": draw((E, H, I), down_std),
         "ws_gate": None, "ws_up": None, "ws_down": None}
    if lc.n_shared:
        Is = lc.shared_inter
        w["ws_gate"] = draw((lc.n_shared, Is, H))
        w["ws_up"] = draw((lc.n_shared, Is, H))
        w["ws_down"] = draw((lc.n_shared, H, Is), down_std)
    return w


# ----------------------------------------------------------------------------
# FP8 storage of the expert matrices (a storage format, not part of the method)
# ----------------------------------------------------------------------------
EXPERT_MATRICES = ("w_gate", "w_up", "w_down", "ws_gate", "ws_up", "ws_down")


def to_fp8_block128(w: np.ndarray):
    """Store a stack of matrices [G, R, C] as FP8 E4M3 bytes with one power-of-two scale per 128 x 128 block.

    Per block: the smallest exponent s in [-100, 7] with max|w| / 2^s <= 448 (the largest E4M3 magnitude), then
    each element w / 2^s rounded to E4M3 (torch's float8_e4m3fn cast: round to nearest even).
    Returns (bytes uint8 [G, R, C], exponents int8 [G, ceil(R/128), ceil(C/128)], stored values float32 [G, R, C]);
    the stored values are what the bytes and exponents represent, decoded with torch's own float8 type, so that a
    CPU reference can consume them by value."""
    import torch
    G, R, C = w.shape
    rb, cb = (R + 127) // 128, (C + 127) // 128
    t = torch.from_numpy(np.ascontiguousarray(w, dtype=np.float32))
    pad = torch.zeros((G, rb * 128, cb * 128), dtype=torch.float32)
    pad[:, :R, :C] = t
    blocks = pad.view(G, rb, 128, cb, 128)
    amax = blocks.abs().amax(dim=(2, 4))                                    # [G, rb, cb]
    exps = torch.where(amax > 0, torch.ceil(torch.log2(amax / 448.0)), torch.zeros_like(amax)).clamp_(-100, 7)
    scale = torch.exp2(exps)[:, :, None, :, None]
    q = (blocks / scale).to(torch.float8_e4m3fn)
    stored = (q.to(torch.float32) * scale).reshape(G, rb * 128, cb * 128)[:, :R, :C].contiguous()
    qbytes = q.view(torch.uint8).reshape(G, rb * 128, cb * 128)[:, :R, :C].contiguous()
    return qbytes.numpy(), exps.to(torch.int8).numpy(), stored.numpy()


def weights_to_fp8(w: Dict[str, Optional[np.ndarray]]):
    """Expert matrices of a layer in FP8 block storage.  Returns (stored, packed): `stored` is the weight dict with
    every expert matrix replaced by the values its FP8 form represents (float32; router untouched) and `packed`
    maps name -> uint8 bytes and name + "_scale" -> int8 exponents."""
    stored, packed = dict(w), {}
    for k in EXPERT_MATRICES:
        if w.get(k) is None:
            continue
        qb, ex, val = to_fp8_block128(w[k])
        stored[k] = val
        packed[k] = qb
        packed[k + "_scale"] = ex
    return stored, packed
