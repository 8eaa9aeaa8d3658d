"""ctypes binding over libfmmoe.so: same names as the C ABI (include/fmmoe.h).

Argument marshalling only: torch supplies device memory, the current stream and
dtypes; every step of the path runs in the library's CUDA kernels.  There is no
fallback: a missing library raises ImportError at first use.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional

import torch

HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(HERE, "libfmmoe.so")

FMMOE_OK = 0
STATUS_NAMES = {0: "OK", 1: "INVALID_ARG", 2: "UNSUPPORTED", 3: "WORKSPACE", 4: "CUDA", 5: "TIMEOUT", 6: "INTERNAL",
                7: "TOO_LARGE"}
F32, BF16 = 0, 1
FLAG_REDUCE_ON, FLAG_RESIDUAL, FLAG_DETERMINISTIC = 1, 2, 4
MAX_EXPERTS, MAX_TOPK, MAX_WINDOW = 256, 16, 8
STATIC_PRUNE_MAX_TOKENS = 32768


class LayerDesc(C.Structure):
    _fields_ = [("hidden", C.c_int32), ("n_experts", C.c_int32), ("inter", C.c_int32), ("n_shared", C.c_int32),
                ("shared_inter", C.c_int32), ("top_k", C.c_int32), ("top_k_vis", C.c_int32), ("dtype", C.c_int32),
                ("weight_format", C.c_int32)]


class Weights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in
                ("router_w", "router_b", "w_gate", "w_up", "w_down", "ws_gate", "ws_up", "ws_down",
                 "w_gate_scale", "w_up_scale", "w_down_scale", "ws_gate_scale", "ws_up_scale", "ws_down_scale")]


class RouteOut(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in
                ("logits", "probs", "topk_idx", "topk_w", "expert_off", "row_token", "inv_row")]


class PruneParams(C.Structure):
    _fields_ = [("window", C.c_int32), ("sim_mode", C.c_int32), ("merge_mode", C.c_int32), ("reserved", C.c_int32),
                ("alpha", C.c_double), ("gamma", C.c_double)]


class StackStage(C.Structure):
    _fields_ = [("after_layer", C.c_int32), ("reserved", C.c_int32), ("retain", C.c_double),
                ("params", PruneParams), ("attn", C.c_void_p)]


class FmmoeError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: FMMOE_ERR_{STATUS_NAMES.get(status, status)}")


_lib = None


def lib() -> C.CDLL:
    """Load libfmmoe.so (built by paper_2511_17885_b200.build).  No fallback."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2511_17885_b200.build` "
                          "(there is no CPU or library fallback)")
    L = C.CDLL(LIB_PATH)
    vp, i64, i32, u32, sz = C.c_void_p, C.c_int64, C.c_int32, C.c_uint32, C.c_size_t
    L.fmmoe_create.argtypes = [C.POINTER(vp), C.c_int]; L.fmmoe_create.restype = C.c_int
    L.fmmoe_destroy.argtypes = [vp]; L.fmmoe_destroy.restype = C.c_int
    L.fmmoe_status_string.argtypes = [C.c_int]; L.fmmoe_status_string.restype = C.c_char_p
    L.fmmoe_get_status.argtypes = [vp, vp]; L.fmmoe_get_status.restype = C.c_int
    L.fmmoe_launch_count.argtypes = [vp]; L.fmmoe_launch_count.restype = i64
    L.fmmoe_workspace_bytes.argtypes = [C.POINTER(LayerDesc), i64, u32]; L.fmmoe_workspace_bytes.restype = sz
    L.fmmoe_host_staging_bytes.argtypes = [C.POINTER(LayerDesc), i64]; L.fmmoe_host_staging_bytes.restype = sz
    L.fmmoe_route.argtypes = [vp, C.POINTER(LayerDesc), C.POINTER(Weights), vp, vp, i64, u32, C.POINTER(RouteOut), vp, sz, vp]
    L.fmmoe_route.restype = C.c_int
    L.fmmoe_moe_forward.argtypes = [vp, C.POINTER(LayerDesc), C.POINTER(Weights), vp, vp, i64, u32, vp,
                                    C.POINTER(RouteOut), vp, sz, vp]
    L.fmmoe_moe_forward.restype = C.c_int
    L.fmmoe_moe_forward_host.argtypes = [vp, C.POINTER(LayerDesc), C.POINTER(Weights), vp, vp, i64, u32, vp,
                                         C.POINTER(RouteOut), vp, vp, vp, sz, vp]
    L.fmmoe_moe_forward_host.restype = C.c_int
    L.fmmoe_moe_forward_prune.argtypes = [vp, C.POINTER(LayerDesc), C.POINTER(Weights), vp, vp, i64, u32, vp,
                                          C.POINTER(RouteOut), C.POINTER(PruneParams), vp, C.POINTER(i64),
                                          C.POINTER(i64), C.POINTER(i64), i32, vp, vp, vp, vp, C.POINTER(i64), vp, sz, vp]
    L.fmmoe_moe_forward_prune.restype = C.c_int
    L.fmmoe_moe_forward_host_async.argtypes = L.fmmoe_moe_forward_host.argtypes
    L.fmmoe_moe_forward_host_async.restype = C.c_int
    L.fmmoe_download_async.argtypes = [vp, vp, vp, sz, vp]; L.fmmoe_download_async.restype = C.c_int
    L.fmmoe_upload_async.argtypes = [vp, vp, vp, sz, vp]; L.fmmoe_upload_async.restype = C.c_int
    L.fmmoe_host_fence.argtypes = [vp, C.POINTER(C.c_uint64)]; L.fmmoe_host_fence.restype = C.c_int
    L.fmmoe_host_wait.argtypes = [vp, C.c_uint64]; L.fmmoe_host_wait.restype = C.c_int
    L.fmmoe_profile_enable.argtypes = [vp, C.c_int]; L.fmmoe_profile_enable.restype = C.c_int
    L.fmmoe_profile_reset.argtypes = [vp]; L.fmmoe_profile_reset.restype = C.c_int
    L.fmmoe_profile_read.argtypes = [vp, C.c_int, C.POINTER(C.c_double), C.POINTER(i64)]
    L.fmmoe_profile_read.restype = C.c_int
    L.fmmoe_prune_kept_count.argtypes = [i64, i64, C.POINTER(PruneParams), C.POINTER(i64), C.POINTER(i64)]
    L.fmmoe_prune_kept_count.restype = i64
    L.fmmoe_prune_workspace_bytes.argtypes = [i64, i32]; L.fmmoe_prune_workspace_bytes.restype = sz
    L.fmmoe_prune_visual.argtypes = [vp, C.POINTER(PruneParams), vp, i32, vp, vp, i32, i32, vp,
                                     C.POINTER(i64), C.POINTER(i64), C.POINTER(i64), i32,
                                     vp, vp, vp, vp, C.POINTER(i64), vp, sz, vp]
    L.fmmoe_prune_visual.restype = C.c_int
    L.fmmoe_attention_workspace_bytes.argtypes = [i64, i32, i32]; L.fmmoe_attention_workspace_bytes.restype = sz
    L.fmmoe_attention_importance.argtypes = [vp, vp, vp, i32, i32, i32, i32, C.c_float, C.POINTER(i64), i32, vp, vp, sz, vp]
    L.fmmoe_attention_importance.restype = C.c_int
    L.fmmoe_stack_workspace_bytes.argtypes = [C.POINTER(LayerDesc), i64, i32, u32]
    L.fmmoe_stack_workspace_bytes.restype = sz
    L.fmmoe_stack_output_layout.argtypes = [C.POINTER(StackStage), i32, i32, C.POINTER(i64), C.POINTER(i64), i32,
                                            C.POINTER(i64), C.POINTER(i64)]
    L.fmmoe_stack_output_layout.restype = C.c_int
    L.fmmoe_stack_forward.argtypes = [vp, C.POINTER(LayerDesc), C.POINTER(Weights), i32, i32, C.POINTER(StackStage), i32,
                                      vp, vp, C.POINTER(i64), C.POINTER(i64), i32, u32, vp, vp, C.POINTER(i64), vp, sz, vp]
    L.fmmoe_stack_forward.restype = C.c_int
    L.fmmoe_test_expire_wait.argtypes = [vp, C.c_uint64, i32]; L.fmmoe_test_expire_wait.restype = C.c_int
    L.fmmoe_prune_visual_static.argtypes = [vp, C.POINTER(PruneParams), vp, i32, vp, vp, i32, i32, vp,
                                            C.POINTER(i64), C.POINTER(i64), C.POINTER(i64), i32,
                                            vp, vp, vp, vp, C.POINTER(i64), vp]
    L.fmmoe_prune_visual_static.restype = C.c_int
    _lib = L
    return L


def _check(st: int, where: str):
    if st != FMMOE_OK:
        raise FmmoeError(st, where)


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    assert t.is_contiguous()
    return C.c_void_p(t.data_ptr())


def _stream() -> C.c_void_p:
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _dtype_code(t: torch.dtype) -> int:
    return {torch.float32: F32, torch.bfloat16: BF16}[t]


def prune_params(window: int, gamma: float, alpha: float = 1.0, sim_mode: int = 0, merge_mode: int = 0) -> PruneParams:
    return PruneParams(window, sim_mode, merge_mode, 0, float(alpha), float(gamma))


def fmmoe_prune_kept_count(n_vis: int, n_retain: int, p: PruneParams):
    """Host-only budget arithmetic of Section 3.2.3 -> (kept, n_merge, n_drop)."""
    m, d = C.c_int64(0), C.c_int64(0)
    kept = lib().fmmoe_prune_kept_count(n_vis, n_retain, C.byref(p), C.byref(m), C.byref(d))
    return int(kept), int(m.value), int(d.value)


def fmmoe_workspace_bytes(desc: LayerDesc, n_tokens: int, flags: int = 0) -> int:
    return int(lib().fmmoe_workspace_bytes(C.byref(desc), n_tokens, flags))


WEIGHTS_AS_DTYPE, WEIGHTS_FP8_BLOCK128 = 0, 1


def make_desc(hidden, n_experts, inter, n_shared, shared_inter, top_k, top_k_vis, dtype: torch.dtype,
              weight_format: int = WEIGHTS_AS_DTYPE) -> LayerDesc:
    return LayerDesc(hidden, n_experts, inter, n_shared, shared_inter, top_k, top_k_vis, _dtype_code(dtype),
                     weight_format)


def make_stages(stages) -> "C.Array":
    """[(after_layer, retain, PruneParams, attn tensor or None), ...] -> C array of fmmoe_stack_stage."""
    arr = (StackStage * max(len(stages), 1))()
    for i, (layer, retain, pp, attn) in enumerate(stages):
        arr[i] = StackStage(int(layer), 0, float(retain), pp, attn.data_ptr() if attn is not None else None)
    return arr


def fmmoe_stack_output_layout(stages, n_layers: int, seq_off, n_vis):
    """Host-only: (out_seq_off, out_n_vis) of a stack with these pruning stages."""
    B = len(n_vis)
    arr = make_stages(stages)
    so = (C.c_int64 * (B + 1))(*[int(v) for v in seq_off])
    nv = (C.c_int64 * max(B, 1))(*[int(v) for v in n_vis])
    oo, ov = (C.c_int64 * (B + 1))(), (C.c_int64 * max(B, 1))()
    _check(lib().fmmoe_stack_output_layout(arr, len(stages), n_layers, so, nv, B, oo, ov), "fmmoe_stack_output_layout")
    return [int(v) for v in oo], [int(v) for v in ov][:B]


def make_weights(w: Dict[str, Optional[torch.Tensor]]) -> Weights:
    """Device tensors -> pointer struct.  The struct keeps a reference to every tensor it points into."""
    ws = Weights()
    ws._tensors = dict(w)
    for name, _ in Weights._fields_:
        t = w.get(name)
        if t is not None:
            assert t.is_cuda and t.is_contiguous(), name
            setattr(ws, name, t.data_ptr())
    return ws


class Handle:
    """fmmoe_handle plus a cached workspace tensor (device memory comes from torch)."""

    def __init__(self, device: int = 0):
        self._h = C.c_void_p()
        self.device = device
        _check(lib().fmmoe_create(C.byref(self._h), device), "fmmoe_create")
        self._ws: Optional[torch.Tensor] = None
        self._ws_slots: Dict[int, torch.Tensor] = {}   # one workspace per batch in flight (pipelined host I/O)

    def close(self):
        if self._h:
            lib().fmmoe_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---- plumbing
    def workspace(self, nbytes: int) -> torch.Tensor:
        if self._ws is None or self._ws.numel() < nbytes:
            self._ws = torch.empty(int(nbytes) + 256, dtype=torch.uint8, device=f"cuda:{self.device}")
        return self._ws

    def _ws_args(self, nbytes: int):
        ws = self.workspace(nbytes)
        base = ws.data_ptr()
        aligned = (base + 255) // 256 * 256
        return C.c_void_p(aligned), C.c_size_t(ws.numel() - (aligned - base))

    def get_status(self) -> int:
        return int(lib().fmmoe_get_status(self._h, _stream()))

    def check_status(self, where: str = "fmmoe_get_status"):
        _check(self.get_status(), where)

    def fmmoe_test_expire_wait(self, budget_ns: int, k_block: int):
        """Self-test: arm the next fmmoe_moe_forward (small-M form) so that one of its bounded waits runs out."""
        _check(lib().fmmoe_test_expire_wait(self._h, C.c_uint64(int(budget_ns)), int(k_block)), "fmmoe_test_expire_wait")

    def launch_count(self) -> int:
        return int(lib().fmmoe_launch_count(self._h))

    KERNELS = ("route", "permute", "gather", "gemm1", "gemm2", "finalize", "prune_index", "prune_score",
               "prune_select", "prune_compact", "attn")

    def profile_enable(self, on: bool = True):
        _check(lib().fmmoe_profile_enable(self._h, 1 if on else 0), "fmmoe_profile_enable")

    def profile_reset(self):
        _check(lib().fmmoe_profile_reset(self._h), "fmmoe_profile_reset")

    def profile_read(self) -> Dict[str, Dict[str, float]]:
        """Per kernel: summed milliseconds and launches since the last reset."""
        out = {}
        for i, name in enumerate(self.KERNELS):
            ms, n = C.c_double(0), C.c_int64(0)
            _check(lib().fmmoe_profile_read(self._h, i, C.byref(ms), C.byref(n)), "fmmoe_profile_read")
            out[name] = {"ms": ms.value, "launches": int(n.value)}
        return out

    # ---- Section 3.1
    def fmmoe_route(self, desc: LayerDesc, w: Weights, x: torch.Tensor, is_visual: torch.Tensor, flags: int,
                    want=("logits", "probs", "topk_idx", "topk_w", "expert_off", "row_token", "inv_row")):
        """Eq. 1-3, 5 (+ grouping by expert).  Returns a dict of freshly allocated device tensors."""
        T, E, K = x.shape[0], desc.n_experts, desc.top_k
        dev = x.device
        shapes = {"logits": ((T, E), torch.float32), "probs": ((T, E), torch.float32),
                  "topk_idx": ((T, K), torch.int32), "topk_w": ((T, K), torch.float32),
                  "expert_off": ((E + 1,), torch.int32), "row_token": ((T * K,), torch.int32),
                  "inv_row": ((T, K), torch.int32)}
        out = {k: torch.empty(shapes[k][0], dtype=shapes[k][1], device=dev) for k in want}
        ro = RouteOut(**{k: v.data_ptr() for k, v in out.items()})
        wsp, wsn = self._ws_args(fmmoe_workspace_bytes(desc, T, flags))
        _check(lib().fmmoe_route(self._h, C.byref(desc), C.byref(w), _ptr(x), _ptr(is_visual), T, flags,
                                 C.byref(ro), wsp, wsn, _stream()), "fmmoe_route")
        return out

    def fmmoe_moe_forward(self, desc: LayerDesc, w: Weights, x: torch.Tensor, is_visual: torch.Tensor, flags: int,
                          out: Optional[torch.Tensor] = None, route: Optional[Dict[str, torch.Tensor]] = None):
        """Eq. 1-5: out[T,H].  `route`: dict of preallocated tensors to receive the routing record."""
        T = x.shape[0]
        if out is None:
            out = torch.empty_like(x)
        ro = RouteOut(**{k: v.data_ptr() for k, v in route.items()}) if route else None
        wsp, wsn = self._ws_args(fmmoe_workspace_bytes(desc, T, flags))
        _check(lib().fmmoe_moe_forward(self._h, C.byref(desc), C.byref(w), _ptr(x), _ptr(is_visual), T, flags,
                                       _ptr(out), C.byref(ro) if ro is not None else None, wsp, wsn, _stream()),
               "fmmoe_moe_forward")
        return out

    def fmmoe_moe_forward_host(self, desc: LayerDesc, w: Weights, x_host: torch.Tensor, is_visual_host: torch.Tensor,
                               flags: int, out_host: torch.Tensor, route: Optional[Dict[str, torch.Tensor]] = None,
                               out_dev: Optional[torch.Tensor] = None, is_visual_dev: Optional[torch.Tensor] = None):
        """Host-buffer variant: H2D copy, layer, D2H copy, stream synchronised on return."""
        T = x_host.shape[0]
        ro = RouteOut(**{k: v.data_ptr() for k, v in route.items()}) if route else None
        assert not x_host.is_cuda and not out_host.is_cuda and x_host.is_contiguous() and out_host.is_contiguous()
        need = fmmoe_workspace_bytes(desc, T, flags) + int(lib().fmmoe_host_staging_bytes(C.byref(desc), T))
        wsp, wsn = self._ws_args(need)
        _check(lib().fmmoe_moe_forward_host(self._h, C.byref(desc), C.byref(w), C.c_void_p(x_host.data_ptr()),
                                            C.c_void_p(is_visual_host.data_ptr()), T, flags,
                                            C.c_void_p(out_host.data_ptr()), C.byref(ro) if ro is not None else None,
                                            _ptr(out_dev), _ptr(is_visual_dev), wsp, wsn, _stream()),
               "fmmoe_moe_forward_host")
        return out_host

    def fmmoe_moe_forward_host_async(self, desc: LayerDesc, w: Weights, x_host: torch.Tensor,
                                     is_visual_host: torch.Tensor, flags: int, out_host: Optional[torch.Tensor],
                                     slot: int, route: Optional[Dict[str, torch.Tensor]] = None,
                                     out_dev: Optional[torch.Tensor] = None,
                                     is_visual_dev: Optional[torch.Tensor] = None):
        """Pipelined host-buffer variant: returns once the upload, the layer and the download are enqueued.
        `slot` selects the workspace of this batch in flight (its staging area is being written by the upload
        stream while other batches compute); take a ticket with fmmoe_host_fence and wait for it before the
        slot and its buffers are reused."""
        T = x_host.shape[0]
        ro = RouteOut(**{k: v.data_ptr() for k, v in route.items()}) if route else None
        assert not x_host.is_cuda and x_host.is_contiguous() and (out_host is None or not out_host.is_cuda)
        need = fmmoe_workspace_bytes(desc, T, flags) + int(lib().fmmoe_host_staging_bytes(C.byref(desc), T))
        ws = self._ws_slots.get(slot)
        if ws is None or ws.numel() < need + 256:
            ws = self._ws_slots[slot] = torch.empty(need + 256, dtype=torch.uint8, device=f"cuda:{self.device}")
        base = ws.data_ptr()
        aligned = (base + 255) // 256 * 256
        _check(lib().fmmoe_moe_forward_host_async(
            self._h, C.byref(desc), C.byref(w), C.c_void_p(x_host.data_ptr()), C.c_void_p(is_visual_host.data_ptr()),
            T, flags, C.c_void_p(out_host.data_ptr()) if out_host is not None else None,
            C.byref(ro) if ro is not None else None, _ptr(out_dev), _ptr(is_visual_dev), C.c_void_p(aligned),
            C.c_size_t(ws.numel() - (aligned - base)), _stream()), "fmmoe_moe_forward_host_async")

    def fmmoe_upload_async(self, dst_dev: torch.Tensor, src_host: torch.Tensor):
        """Host -> device copy on the handle's upload stream; later work on the current stream waits for it."""
        assert dst_dev.is_cuda and not src_host.is_cuda and dst_dev.is_contiguous() and src_host.is_contiguous()
        n = src_host.numel() * src_host.element_size()
        assert dst_dev.numel() * dst_dev.element_size() >= n
        _check(lib().fmmoe_upload_async(self._h, _ptr(dst_dev), C.c_void_p(src_host.data_ptr()), n, _stream()),
               "fmmoe_upload_async")

    def fmmoe_download_async(self, dst_host: torch.Tensor, src_dev: torch.Tensor):
        """Device -> host copy on the handle's download stream, after the work enqueued on the current stream."""
        assert not dst_host.is_cuda and src_dev.is_cuda and dst_host.is_contiguous() and src_dev.is_contiguous()
        n = src_dev.numel() * src_dev.element_size()
        assert dst_host.numel() * dst_host.element_size() >= n
        _check(lib().fmmoe_download_async(self._h, C.c_void_p(dst_host.data_ptr()), _ptr(src_dev), n, _stream()),
               "fmmoe_download_async")

    def fmmoe_host_fence(self) -> int:
        t = C.c_uint64(0)
        _check(lib().fmmoe_host_fence(self._h, C.byref(t)), "fmmoe_host_fence")
        return int(t.value)

    def fmmoe_host_wait(self, ticket: int):
        _check(lib().fmmoe_host_wait(self._h, C.c_uint64(ticket)), "fmmoe_host_wait")

    # ---- Section 3.2
    def fmmoe_prune_visual(self, p: PruneParams, probs: torch.Tensor, attn: Optional[torch.Tensor], x: torch.Tensor,
                           is_visual: torch.Tensor, seq_off, n_vis, n_retain, want_aux: bool = True):
        """Eq. 6-18 + drop rule.  Returns dict(x_out, is_visual_out, keep_idx, kind, out_seq_off)."""
        T, H = x.shape
        B = len(n_vis)
        arr = C.c_int64 * (B + 1)
        so = arr(*[int(v) for v in seq_off])
        nv = (C.c_int64 * max(B, 1))(*[int(v) for v in n_vis])
        nr = (C.c_int64 * max(B, 1))(*[int(v) for v in n_retain])
        oo = arr()
        # output size is data-independent: compute it first, then allocate exactly
        t_out = 0
        for b in range(B):
            kept, _, _ = fmmoe_prune_kept_count(int(n_vis[b]), int(n_retain[b]), p)
            if kept < 0:
                raise FmmoeError(1, "fmmoe_prune_kept_count")
            t_out += int(seq_off[b + 1]) - int(seq_off[b]) - int(n_vis[b]) + kept
        dev = x.device
        x_out = torch.empty((t_out, H), dtype=x.dtype, device=dev)
        vis_out = torch.empty(t_out, dtype=torch.uint8, device=dev) if want_aux else None
        keep_idx = torch.empty(t_out, dtype=torch.int32, device=dev) if want_aux else None
        kind = torch.empty(t_out, dtype=torch.uint8, device=dev) if want_aux else None
        wsp, wsn = self._ws_args(int(lib().fmmoe_prune_workspace_bytes(T, B)))
        _check(lib().fmmoe_prune_visual(self._h, C.byref(p), _ptr(probs), probs.shape[1] if probs is not None else 1,
                                        _ptr(attn), _ptr(x), _dtype_code(x.dtype), H, _ptr(is_visual), so, nv, nr, B,
                                        _ptr(x_out), _ptr(vis_out), _ptr(keep_idx), _ptr(kind), oo, wsp, wsn,
                                        _stream()), "fmmoe_prune_visual")
        return {"x_out": x_out, "is_visual_out": vis_out, "keep_idx": keep_idx, "kind": kind,
                "out_seq_off": [int(v) for v in oo]}

    def fmmoe_moe_forward_prune(self, desc: LayerDesc, w: Weights, x: torch.Tensor, is_visual: torch.Tensor,
                                flags: int, out: torch.Tensor, route: Dict[str, torch.Tensor], p: PruneParams,
                                attn: Optional[torch.Tensor], seq_off, n_vis, n_retain, want_aux: bool = True):
        """Eq. 1-5 then Eq. 6-18 in one call (selection beside the expert GEMMs).  `route` must hold "probs".
        Returns the dict fmmoe_prune_visual returns."""
        T, H = x.shape
        B = len(n_vis)
        arr = C.c_int64 * (B + 1)
        so = arr(*[int(v) for v in seq_off])
        nv = (C.c_int64 * max(B, 1))(*[int(v) for v in n_vis])
        nr = (C.c_int64 * max(B, 1))(*[int(v) for v in n_retain])
        oo = arr()
        t_out = 0
        for b in range(B):
            kept, _, _ = fmmoe_prune_kept_count(int(n_vis[b]), int(n_retain[b]), p)
            if kept < 0:
                raise FmmoeError(1, "fmmoe_prune_kept_count")
            t_out += int(seq_off[b + 1]) - int(seq_off[b]) - int(n_vis[b]) + kept
        dev = x.device
        x_out = torch.empty((t_out, H), dtype=x.dtype, device=dev)
        vis_out = torch.empty(t_out, dtype=torch.uint8, device=dev) if want_aux else None
        keep_idx = torch.empty(t_out, dtype=torch.int32, device=dev) if want_aux else None
        kind = torch.empty(t_out, dtype=torch.uint8, device=dev) if want_aux else None
        ro = RouteOut(**{k: v.data_ptr() for k, v in route.items()})
        need = fmmoe_workspace_bytes(desc, T, flags) + 256 + int(lib().fmmoe_prune_workspace_bytes(T, B))
        wsp, wsn = self._ws_args(need)
        _check(lib().fmmoe_moe_forward_prune(self._h, C.byref(desc), C.byref(w), _ptr(x), _ptr(is_visual), T, flags,
                                             _ptr(out), C.byref(ro), C.byref(p), _ptr(attn), so, nv, nr, B, _ptr(x_out),
                                             _ptr(vis_out), _ptr(keep_idx), _ptr(kind), oo, wsp, wsn, _stream()),
               "fmmoe_moe_forward_prune")
        return {"x_out": x_out, "is_visual_out": vis_out, "keep_idx": keep_idx, "kind": kind,
                "out_seq_off": [int(v) for v in oo]}

    def prepare_forward_prune(self, desc: LayerDesc, w: Weights, x: torch.Tensor, is_visual: torch.Tensor, flags: int,
                              out: torch.Tensor, route: Dict[str, torch.Tensor], p: PruneParams,
                              attn: Optional[torch.Tensor], seq_off, n_vis, n_retain, want_aux: bool = True):
        """fmmoe_moe_forward_prune with every argument marshalled once: the returned object's run() is a single
        C call on the current stream that allocates nothing (outputs and the workspace are created here and reused
        by every run).  For loops that issue the same call many times."""
        return ForwardPruneCall(self, desc, w, x, is_visual, flags, out, route, p, attn, seq_off, n_vis, n_retain,
                                want_aux)

    def fmmoe_attention_importance(self, q_last: torch.Tensor, k: torch.Tensor, seq_off, scale: Optional[float] = None,
                                   out: Optional[torch.Tensor] = None) -> torch.Tensor:
        """Eq. 7: head-averaged attention of each sequence's last token to all its tokens.
        q_last [n_seq, n_heads, d], k [T, n_kv_heads, d] -> attn [T] fp32."""
        n_seq, n_heads, d = q_last.shape
        T, n_kv, _ = k.shape
        if scale is None:
            scale = 1.0 / float(d) ** 0.5
        if out is None:
            out = torch.empty(T, dtype=torch.float32, device=k.device)
        so = (C.c_int64 * (n_seq + 1))(*[int(v) for v in seq_off])
        wsp, wsn = self._ws_args(int(lib().fmmoe_attention_workspace_bytes(T, n_seq, n_heads)))
        _check(lib().fmmoe_attention_importance(self._h, _ptr(q_last), _ptr(k), _dtype_code(k.dtype), n_heads, n_kv, d,
                                                C.c_float(scale), so, n_seq, _ptr(out), wsp, wsn, _stream()),
               "fmmoe_attention_importance")
        return out

    def fmmoe_stack_forward(self, desc: LayerDesc, layer_weights, reduce_from: int, stages, x: torch.Tensor,
                            is_visual: torch.Tensor, seq_off, n_vis, flags: int = 0,
                            x_out: Optional[torch.Tensor] = None, is_visual_out: Optional[torch.Tensor] = None):
        """n_layers x (x <- x + MoE(x)) with K_v from layer `reduce_from` on and pruning stages
        [(after_layer, retain, PruneParams, attn or None), ...].  layer_weights: list of Weights structs.
        Returns (x_out, is_visual_out, out_seq_off)."""
        n_layers, B = len(layer_weights), len(n_vis)
        T, H = x.shape
        out_off, _ = fmmoe_stack_output_layout(stages, n_layers, seq_off, n_vis)
        t_out = out_off[-1]
        if x_out is None:
            x_out = torch.empty((t_out, H), dtype=x.dtype, device=x.device)
        if is_visual_out is None:
            is_visual_out = torch.empty(t_out, dtype=torch.uint8, device=x.device)
        warr = (Weights * n_layers)(*layer_weights)
        sarr = make_stages(stages)
        so = (C.c_int64 * (B + 1))(*[int(v) for v in seq_off])
        nv = (C.c_int64 * max(B, 1))(*[int(v) for v in n_vis])
        oo = (C.c_int64 * (B + 1))()
        wsp, wsn = self._ws_args(int(lib().fmmoe_stack_workspace_bytes(C.byref(desc), T, B, flags)))
        _check(lib().fmmoe_stack_forward(self._h, C.byref(desc), warr, n_layers, reduce_from, sarr, len(stages), _ptr(x),
                                         _ptr(is_visual), so, nv, B, flags, _ptr(x_out), _ptr(is_visual_out), oo, wsp, wsn,
                                         _stream()), "fmmoe_stack_forward")
        assert [int(v) for v in oo] == out_off
        return x_out, is_visual_out, out_off

    def fmmoe_prune_visual_static(self, p: PruneParams, probs: torch.Tensor, attn: Optional[torch.Tensor],
                                  x: torch.Tensor, is_visual: torch.Tensor, seq_off, n_vis, n_retain,
                                  x_out: torch.Tensor, is_visual_out: Optional[torch.Tensor] = None,
                                  keep_idx: Optional[torch.Tensor] = None, kind: Optional[torch.Tensor] = None):
        """fmmoe_prune_visual for callers that cannot allocate device memory when they prune.

        The library call behind this method takes no workspace and allocates nothing: its
        scratch is a fixed array inside the library (at most STATIC_PRUNE_MAX_TOKENS tokens
        per call; more raises FmmoeError TOO_LARGE).  In keeping with that, this wrapper
        allocates nothing either: the caller passes preallocated outputs, x_out [T', H] with
        T' from fmmoe_prune_kept_count, and optionally is_visual_out / keep_idx / kind [T'].
        Calls share the one scratch array, so do not let two of them overlap on the GPU.
        Returns out_seq_off as a list."""
        B = len(n_vis)
        arr = C.c_int64 * (B + 1)
        so = arr(*[int(v) for v in seq_off])
        nv = (C.c_int64 * max(B, 1))(*[int(v) for v in n_vis])
        nr = (C.c_int64 * max(B, 1))(*[int(v) for v in n_retain])
        oo = arr()
        # The kernels write T' rows whatever the buffers hold, so the outputs are checked here against the
        # data-independent output size (host arithmetic only, nothing is allocated).  Problems beyond the
        # built-in scratch are left to the library, which refuses them before it touches any buffer.
        if int(seq_off[B]) <= STATIC_PRUNE_MAX_TOKENS:
            t_out = 0
            for b in range(B):
                kept, _, _ = fmmoe_prune_kept_count(int(n_vis[b]), int(n_retain[b]), p)
                if kept < 0:
                    raise FmmoeError(1, "fmmoe_prune_kept_count")
                t_out += int(seq_off[b + 1]) - int(seq_off[b]) - int(n_vis[b]) + kept
            if (tuple(x_out.shape) != (t_out, x.shape[1]) or x_out.dtype != x.dtype or x_out.device != x.device
                    or not x_out.is_contiguous()):
                raise ValueError(f"x_out must be a contiguous [{t_out}, {x.shape[1]}] {x.dtype} tensor on {x.device}")
            for name, t, dt in (("is_visual_out", is_visual_out, torch.uint8), ("keep_idx", keep_idx, torch.int32),
                                ("kind", kind, torch.uint8)):
                if t is not None and (t.numel() < t_out or t.dtype != dt or t.device != x.device or not t.is_contiguous()):
                    raise ValueError(f"{name} must be a contiguous {dt} tensor of at least {t_out} elements on {x.device}")
        _check(lib().fmmoe_prune_visual_static(self._h, C.byref(p), _ptr(probs), probs.shape[1], _ptr(attn), _ptr(x),
                                               _dtype_code(x.dtype), x.shape[1], _ptr(is_visual), so, nv, nr, B,
                                               _ptr(x_out), _ptr(is_visual_out), _ptr(keep_idx), _ptr(kind), oo,
                                               _stream()), "fmmoe_prune_visual_static")
        return [int(v) for v in oo]


class ForwardPruneCall:
    """A marshalled fmmoe_moe_forward_prune call (see Handle.prepare_forward_prune).  `result` has the keys
    fmmoe_moe_forward_prune returns; its tensors are overwritten by every run()."""

    def __init__(self, handle: Handle, desc, w, x, is_visual, flags, out, route, p, attn, seq_off, n_vis, n_retain,
                 want_aux):
        T, H = x.shape
        B = len(n_vis)
        arr = C.c_int64 * (B + 1)
        self.h = handle
        self.so = arr(*[int(v) for v in seq_off])
        self.nv = (C.c_int64 * max(B, 1))(*[int(v) for v in n_vis])
        self.nr = (C.c_int64 * max(B, 1))(*[int(v) for v in n_retain])
        self.oo = arr()
        t_out = 0
        for b in range(B):
            kept, _, _ = fmmoe_prune_kept_count(int(n_vis[b]), int(n_retain[b]), p)
            if kept < 0:
                raise FmmoeError(1, "fmmoe_prune_kept_count")
            t_out += int(seq_off[b + 1]) - int(seq_off[b]) - int(n_vis[b]) + kept
        dev = x.device
        self.x_out = torch.empty((t_out, H), dtype=x.dtype, device=dev)
        self.vis_out = torch.empty(t_out, dtype=torch.uint8, device=dev) if want_aux else None
        self.keep_idx = torch.empty(t_out, dtype=torch.int32, device=dev) if want_aux else None
        self.kind = torch.empty(t_out, dtype=torch.uint8, device=dev) if want_aux else None
        self.ro = RouteOut(**{k: v.data_ptr() for k, v in route.items()})
        need = fmmoe_workspace_bytes(desc, T, flags) + 256 + int(lib().fmmoe_prune_workspace_bytes(T, B))
        self.ws = torch.empty(need + 256, dtype=torch.uint8, device=dev)     # this call's own workspace
        base = self.ws.data_ptr()
        aligned = (base + 255) // 256 * 256
        self.keep = (desc, w, x, is_visual, out, route, p, attn)             # referenced for as long as the call lives
        self.args = (handle._h, C.byref(desc), C.byref(w), _ptr(x), _ptr(is_visual), T, flags, _ptr(out),
                     C.byref(self.ro), C.byref(p), _ptr(attn), self.so, self.nv, self.nr, B, _ptr(self.x_out),
                     _ptr(self.vis_out), _ptr(self.keep_idx), _ptr(self.kind), self.oo, C.c_void_p(aligned),
                     C.c_size_t(self.ws.numel() - (aligned - base)))
        self.fn = lib().fmmoe_moe_forward_prune
        self.result = {"x_out": self.x_out, "is_visual_out": self.vis_out, "keep_idx": self.keep_idx,
                       "kind": self.kind, "out_seq_off": None}

    def run(self):
        _check(self.fn(*self.args, _stream()), "fmmoe_moe_forward_prune")
        if self.result["out_seq_off"] is None:
            self.result["out_seq_off"] = [int(v) for v in self.oo]
        return self.result
