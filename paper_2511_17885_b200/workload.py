"""Device-resident workloads for the benchmark, the smoke check and the full-size tests.

Marshalling only: tensors come from `inputs`, every computation is a C-ABI call."""
from __future__ import annotations

from typing import Dict, Optional

import numpy as np
import torch

from . import binding as B
from . import inputs as I

TDT = {"f32": torch.float32, "bf16": torch.bfloat16}


def upload_weights(w: Dict[str, Optional[np.ndarray]], dtype: str, device: str) -> Dict[str, Optional[torch.Tensor]]:
    out: Dict[str, Optional[torch.Tensor]] = {}
    for k, v in w.items():
        if v is None:
            out[k] = None
        elif k == "router_b":
            out[k] = torch.from_numpy(v.astype(np.float32)).to(device)
        else:
            out[k] = torch.from_numpy(v).to(device).to(TDT[dtype]).contiguous()
    return out


class LayerWorkload:
    """One MoE layer over one batch of sequences, followed by one pruning stage.

    step()      : inputs resident in HBM  -> fmmoe_moe_forward + fmmoe_prune_visual
    step_host() : inputs in pinned host memory -> fmmoe_moe_forward_host (H2D, layer, D2H of the
                  layer output) + fmmoe_prune_visual on the device copy + D2H of the pruned rows
    """

    def __init__(self, cfg: I.LayerCfg, handle: B.Handle, device: int = 0, prune: Optional[I.PruneCfg] = None,
                 use_attn: bool = False, flags: int = B.FLAG_REDUCE_ON, token_seed: Optional[int] = None,
                 keep_host: bool = False):
        self.cfg, self.h = cfg, handle
        dev = f"cuda:{device}"
        td = TDT[cfg.dtype]
        x, mask, seq_off, n_vis = I.make_tokens(cfg, seed=token_seed)
        w = I.make_weights(cfg)
        self.host = {"x": x, "mask": mask, "w": w} if keep_host else None
        self.seq_off, self.n_vis = seq_off, n_vis
        self.x = torch.from_numpy(x).to(dev).to(td).contiguous()
        self.mask = torch.from_numpy(mask).to(dev)
        self.wd = upload_weights(w, cfg.dtype, dev)
        self.ws = B.make_weights(self.wd)
        self.desc = B.make_desc(cfg.hidden, cfg.n_experts, cfg.inter, cfg.n_shared, cfg.shared_inter, cfg.top_k,
                                cfg.top_k_vis, td)
        self.flags = flags
        T, E, K = cfg.n_tokens, cfg.n_experts, cfg.top_k
        self.out = torch.empty_like(self.x)
        self.route = {"probs": torch.empty(T, E, dtype=torch.float32, device=dev),
                      "topk_idx": torch.empty(T, K, dtype=torch.int32, device=dev),
                      "expert_off": torch.empty(E + 1, dtype=torch.int32, device=dev)}
        self.prune = prune
        self.attn = None
        if prune is not None:
            self.pp = B.prune_params(prune.window, prune.gamma, prune.alpha)
            self.n_retain = I.retain_counts(n_vis, prune.retain)
            if use_attn:
                self.attn = torch.from_numpy(I.make_attention_importance(cfg, seed=token_seed)).to(dev)
        # host side of the end-to-end step
        self.x_host = torch.from_numpy(x).to(td).pin_memory()
        self.mask_host = torch.from_numpy(mask).pin_memory()
        self.out_host = torch.empty_like(self.x_host).pin_memory()
        self.mask_dev2 = torch.empty_like(self.mask)
        self.pruned_host = None
        self.last = None

    @property
    def n_tokens(self) -> int:
        return self.cfg.n_tokens

    def step(self):
        self.h.fmmoe_moe_forward(self.desc, self.ws, self.x, self.mask, self.flags, out=self.out, route=self.route)
        if self.prune is not None:
            self.last = self.h.fmmoe_prune_visual(self.pp, self.route["probs"], self.attn, self.out, self.mask,
                                                  self.seq_off, self.n_vis, self.n_retain)
        return self.last

    def step_host(self):
        self.h.fmmoe_moe_forward_host(self.desc, self.ws, self.x_host, self.mask_host, self.flags, self.out_host,
                                      route=self.route, out_dev=self.out, is_visual_dev=self.mask_dev2)
        if self.prune is not None:
            r = self.h.fmmoe_prune_visual(self.pp, self.route["probs"], self.attn, self.out, self.mask_dev2,
                                          self.seq_off, self.n_vis, self.n_retain, want_aux=False)
            if self.pruned_host is None or self.pruned_host.shape != r["x_out"].shape:
                self.pruned_host = torch.empty(r["x_out"].shape, dtype=r["x_out"].dtype).pin_memory()
            self.pruned_host.copy_(r["x_out"], non_blocking=True)
            torch.cuda.current_stream().synchronize()
        return self.out_host

    def h2d_bytes(self) -> int:
        return self.x_host.numel() * self.x_host.element_size() + self.mask_host.numel()

    def d2h_bytes(self) -> int:
        n = self.out_host.numel() * self.out_host.element_size()
        if self.pruned_host is not None:
            n += self.pruned_host.numel() * self.pruned_host.element_size()
        return n

    def routing_stats(self):
        """(routed pairs P, experts with at least one row) of the last step."""
        off = self.route["expert_off"].cpu().numpy().astype(np.int64)
        cnt = np.diff(off)
        return int(off[-1]), int((cnt > 0).sum())
