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


def upload_weights_fp8(w: Dict[str, Optional[np.ndarray]], packed: Dict[str, np.ndarray], dtype: str,
                       device: str) -> Dict[str, Optional[torch.Tensor]]:
    """Router parameters as usual; expert matrices as FP8 bytes plus their int8 block-scale exponents."""
    out = upload_weights({k: v for k, v in w.items() if k not in I.EXPERT_MATRICES}, dtype, device)
    for k in I.EXPERT_MATRICES:
        out[k] = None
    for k, v in packed.items():
        out[k] = torch.from_numpy(np.ascontiguousarray(v)).to(device)
    return out


class LayerWorkload:
    """One MoE layer over one batch of sequences, followed by one pruning stage.

    step()      : inputs resident in HBM  -> fmmoe_moe_forward_prune (layer, then the pruning stage on its output)
    step_host() : inputs in pinned host memory -> fmmoe_moe_forward_host (H2D, layer, D2H of the
                  layer output) + fmmoe_prune_visual on the device copy + D2H of the pruned rows
    """

    def __init__(self, cfg: I.LayerCfg, handle: B.Handle, device: int = 0, prune: Optional[I.PruneCfg] = None,
                 use_attn: bool = False, flags: int = B.FLAG_REDUCE_ON, token_seed: Optional[int] = None,
                 keep_host: bool = False, fp8_weights: bool = False):
        self.cfg, self.h = cfg, handle
        dev = f"cuda:{device}"
        td = TDT[cfg.dtype]
        x, mask, seq_off, n_vis = I.make_tokens(cfg, seed=token_seed)
        w = I.make_weights(cfg)
        self.fp8_weights = fp8_weights
        if fp8_weights:
            # the layer's expert matrices stored as FP8 bytes + block scales; `w` becomes the values they represent
            w, packed = I.weights_to_fp8(w)
            self.wd = upload_weights_fp8(w, packed, cfg.dtype, dev)
        else:
            self.wd = upload_weights(w, cfg.dtype, dev)
        self.host = {"x": x, "mask": mask, "w": w} if keep_host else None
        self.seq_off, self.n_vis = seq_off, n_vis
        self.x = torch.from_numpy(x).to(dev).to(td).contiguous()
        self.mask = torch.from_numpy(mask).to(dev)
        self.ws = B.make_weights(self.wd)
        self.desc = B.make_desc(cfg.hidden, cfg.n_experts, cfg.inter, cfg.n_shared, cfg.shared_inter, cfg.top_k,
                                cfg.top_k_vis, td, B.WEIGHTS_FP8_BLOCK128 if fp8_weights else B.WEIGHTS_AS_DTYPE)
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

    def step(self, fused: bool = True):
        if self.prune is not None and not fused:     # the same work as two calls, every kernel on one stream
            self.h.fmmoe_moe_forward(self.desc, self.ws, self.x, self.mask, self.flags, out=self.out, route=self.route)
            self.last = self.h.fmmoe_prune_visual(self.pp, self.route["probs"], self.attn, self.out, self.mask,
                                                  self.seq_off, self.n_vis, self.n_retain)
            return self.last
        if self.prune is not None:
            if getattr(self, "_call", None) is None or self._call_route is not self.route:
                # marshalled once: the timed loop is one C call per step and allocates nothing
                self._call = self.h.prepare_forward_prune(self.desc, self.ws, self.x, self.mask, self.flags, self.out,
                                                          self.route, self.pp, self.attn, self.seq_off, self.n_vis,
                                                          self.n_retain)
                self._call_route = self.route
            self.last = self._call.run()
        else:
            self.h.fmmoe_moe_forward(self.desc, self.ws, self.x, self.mask, self.flags, out=self.out, route=self.route)
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

    PIPE_DEPTH = 3   # batches in flight in the pipelined end-to-end step

    def _pipe_slots(self):
        if getattr(self, "_slots", None) is None:
            self._slots = [{"x_dev": torch.empty_like(self.x), "out_dev": torch.empty_like(self.x),
                            "mask_dev": torch.empty_like(self.mask),
                            "out_host": torch.empty_like(self.x_host).pin_memory(), "pruned_host": None,
                            "pruned_dev": None, "ticket": None} for _ in range(self.PIPE_DEPTH)]
        return self._slots

    def step_host_async(self, i: int):
        """Batch i of a stream of independent batches whose activations live in pinned host memory: the upload
        of batch i overlaps the layer of batch i-1 and the downloads of batch i-2 (fmmoe_upload_async, the same
        device call as step(), fmmoe_download_async).  Every batch is uploaded, computed and downloaded in full
        (layer output and pruned rows); drain_host() returns when all results are in host memory."""
        sl = self._pipe_slots()[i % self.PIPE_DEPTH]
        if sl["ticket"] is not None:
            self.h.fmmoe_host_wait(sl["ticket"])       # the slot's previous batch is fully on the host
        self.h.fmmoe_upload_async(sl["x_dev"], self.x_host)
        self.h.fmmoe_upload_async(sl["mask_dev"], self.mask_host)
        if self.prune is not None:
            if sl.get("call") is None:                 # marshalled once per slot: own outputs, own workspace
                sl["call"] = self.h.prepare_forward_prune(self.desc, self.ws, sl["x_dev"], sl["mask_dev"], self.flags,
                                                          sl["out_dev"], self.route, self.pp, self.attn, self.seq_off,
                                                          self.n_vis, self.n_retain, want_aux=False)
            r = sl["call"].run()
            if sl["pruned_host"] is None or sl["pruned_host"].shape != r["x_out"].shape:
                sl["pruned_host"] = torch.empty(r["x_out"].shape, dtype=r["x_out"].dtype).pin_memory()
            sl["pruned_dev"] = r["x_out"]              # owned by the slot's call: rewritten only after the ticket wait
            self.h.fmmoe_download_async(sl["out_host"], sl["out_dev"])
            self.h.fmmoe_download_async(sl["pruned_host"], r["x_out"])
            self.pruned_host = sl["pruned_host"]
        else:
            self.h.fmmoe_moe_forward(self.desc, self.ws, sl["x_dev"], sl["mask_dev"], self.flags, out=sl["out_dev"],
                                     route=self.route)
            self.h.fmmoe_download_async(sl["out_host"], sl["out_dev"])
        sl["ticket"] = self.h.fmmoe_host_fence()
        return sl

    def drain_host(self):
        for sl in self._pipe_slots():
            if sl["ticket"] is not None:
                self.h.fmmoe_host_wait(sl["ticket"])
                sl["ticket"] = None

    def h2d_bytes(self) -> int:
        return self.x_host.numel() * self.x_host.element_size() + self.mask_host.numel()

    def d2h_bytes(self) -> int:
        n = self.out_host.numel() * self.out_host.element_size()
        if self.pruned_host is not None:
            n += self.pruned_host.numel() * self.pruned_host.element_size()
        return n

    def merged_rows(self) -> int:
        """Merged windows of the last step's pruning stage (each read W rows and wrote one)."""
        return int((self.last["kind"] == 2).sum()) if self.last is not None and self.last.get("kind") is not None else 0

    def routing_stats(self):
        """(routed pairs P, experts with at least one row) of the last step."""
        off = self.route["expert_off"].cpu().numpy().astype(np.int64)
        cnt = np.diff(off)
        return int(off[-1]), int((cnt > 0).sum())


class StackWorkload:
    """The 24-layer stack: residual MoE layers of one shape, K_v from layer `reduce_from` on, pruning
    stages after designated layers.  Weights are drawn on the device (distinct per layer).

    step()      : tokens resident in HBM -> fmmoe_stack_forward
    step_host() : tokens in pinned host memory -> H2D copy, fmmoe_stack_forward, D2H copy of the output
    dense=True  : the unreduced, unpruned comparison run (K experts for every token, no stages)."""

    def __init__(self, cfg: I.StackCfg, handle: B.Handle, device: int = 0, token_seed: Optional[int] = None,
                 dense: bool = False, n_layers: Optional[int] = None, attention: bool = False):
        self.cfg, self.h = cfg, handle
        lc = cfg.layer
        dev = f"cuda:{device}"
        td = TDT[lc.dtype]
        self.n_layers = cfg.n_layers if n_layers is None else n_layers
        x, mask, seq_off, n_vis = I.make_tokens(lc, seed=token_seed)
        self.seq_off, self.n_vis = seq_off, n_vis
        self.x = torch.from_numpy(x).to(dev).to(td).contiguous()
        self.mask = torch.from_numpy(mask).to(dev)
        self.layers = [I.stack_layer_weights_torch(cfg, l, dev) for l in range(self.n_layers)]
        self.wstructs = [B.make_weights(w) for w in self.layers]
        self.desc = B.make_desc(lc.hidden, lc.n_experts, lc.inter, lc.n_shared, lc.shared_inter, lc.top_k,
                                lc.top_k_vis, td)
        self.dense = dense
        self.reduce_from = self.n_layers + 1 if dense else cfg.reduce_from
        self.stages = [] if dense else [(l, pc.retain, B.prune_params(pc.window, pc.gamma, pc.alpha), None)
                                        for l, pc in sorted(cfg.prune_after.items()) if l < self.n_layers]
        # attention-guided scoring (Eq. 7, 11-13): every stage gets the attention-importance vector of the sequence
        # as it is at that layer, computed by fmmoe_attention_importance from stand-in queries and keys at every step
        self.attention = attention and not dense
        self.qk = {}
        if self.attention:
            done = []
            for i, (l, r, pp, _) in enumerate(self.stages):
                off_here, _ = B.fmmoe_stack_output_layout(done, l + 1, seq_off, n_vis)
                q, k = I.make_stage_qk(cfg, l, off_here[-1], len(n_vis))
                a = torch.empty(off_here[-1], dtype=torch.float32, device=dev)
                self.qk[l] = (torch.from_numpy(q).to(dev).to(td), torch.from_numpy(k).to(dev).to(td), off_here, a)
                self.stages[i] = (l, r, pp, a)
                done.append(self.stages[i])
        self.out_off, self.out_vis = B.fmmoe_stack_output_layout(self.stages, self.n_layers, seq_off, n_vis)
        self.x_out = torch.empty((self.out_off[-1], lc.hidden), dtype=td, device=dev)
        self.mask_out = torch.empty(self.out_off[-1], dtype=torch.uint8, device=dev)
        self.x_host = torch.from_numpy(x).to(td).pin_memory()
        self.mask_host = torch.from_numpy(mask).pin_memory()
        self.out_host = torch.empty(self.x_out.shape, dtype=td).pin_memory()

    @property
    def n_tokens(self) -> int:
        return self.cfg.layer.n_tokens

    def step(self):
        for l, (q, k, off_here, a) in self.qk.items():      # Eq. 7 for every pruning layer of this step
            self.h.fmmoe_attention_importance(q, k, off_here, out=a)
        self.h.fmmoe_stack_forward(self.desc, self.wstructs, self.reduce_from, self.stages, self.x, self.mask,
                                   self.seq_off, self.n_vis, 0, x_out=self.x_out, is_visual_out=self.mask_out)
        return self.x_out

    PIPE_DEPTH = 2   # batches in flight in the pipelined end-to-end step

    def step_host(self):
        """One batch at a time: upload, the stack, download, host-side wait (all through the library's calls)."""
        self.h.fmmoe_upload_async(self.x, self.x_host)
        self.h.fmmoe_upload_async(self.mask, self.mask_host)
        self.step()
        self.h.fmmoe_download_async(self.out_host, self.x_out)
        self.h.fmmoe_host_wait(self.h.fmmoe_host_fence())
        return self.out_host

    def step_host_async(self, i: int):
        """Batch i of a stream of independent batches in pinned host memory, PIPE_DEPTH in flight: the upload of
        batch i overlaps the stack of batch i-1 and the download of batch i-2."""
        if getattr(self, "_slots", None) is None:
            self._slots = [{"x": torch.empty_like(self.x), "mask": torch.empty_like(self.mask),
                            "x_out": torch.empty_like(self.x_out), "mask_out": torch.empty_like(self.mask_out),
                            "out_host": torch.empty_like(self.out_host).pin_memory(), "ticket": None}
                           for _ in range(self.PIPE_DEPTH)]
        sl = self._slots[i % self.PIPE_DEPTH]
        if sl["ticket"] is not None:
            self.h.fmmoe_host_wait(sl["ticket"])
        self.h.fmmoe_upload_async(sl["x"], self.x_host)
        self.h.fmmoe_upload_async(sl["mask"], self.mask_host)
        for l, (q, k, off_here, a) in self.qk.items():
            self.h.fmmoe_attention_importance(q, k, off_here, out=a)
        self.h.fmmoe_stack_forward(self.desc, self.wstructs, self.reduce_from, self.stages, sl["x"], sl["mask"],
                                   self.seq_off, self.n_vis, 0, x_out=sl["x_out"], is_visual_out=sl["mask_out"])
        self.h.fmmoe_download_async(sl["out_host"], sl["x_out"])
        sl["ticket"] = self.h.fmmoe_host_fence()
        return sl

    def drain_host(self):
        for sl in getattr(self, "_slots", None) or []:
            if sl["ticket"] is not None:
                self.h.fmmoe_host_wait(sl["ticket"])
                sl["ticket"] = None

    def h2d_bytes(self) -> int:
        return self.x_host.numel() * self.x_host.element_size() + self.mask_host.numel()

    def d2h_bytes(self) -> int:
        return self.out_host.numel() * self.out_host.element_size()

    def layer_shapes(self):
        """Per layer (tokens, routed pairs): data-independent, from the kept counts of the stages."""
        lc = self.cfg.layer
        n_text = [int(self.seq_off[b + 1] - self.seq_off[b] - self.n_vis[b]) for b in range(len(self.n_vis))]
        vis = [int(v) for v in self.n_vis]
        out = []
        stage_at = {l: (r, pp) for l, r, pp, _ in self.stages}
        for l in range(self.n_layers):
            kv = lc.top_k_vis if l >= self.reduce_from else lc.top_k
            T = sum(vis) + sum(n_text)
            out.append((T, sum(vis) * kv + sum(n_text) * lc.top_k))
            if l in stage_at:
                r, pp = stage_at[l]
                vis = [B.fmmoe_prune_kept_count(vis[b], int(np.floor(int(self.n_vis[b]) * r + 1e-9)), pp)[0]
                       for b in range(len(vis))]
        return out
