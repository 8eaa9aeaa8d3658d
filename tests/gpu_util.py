"""Helpers shared by the GPU parity tests (marshalling only)."""
import numpy as np
import torch

from paper_2511_17885_b200 import binding as B

TDT = {"f32": torch.float32, "bf16": torch.bfloat16}


def dev(a, dtype=None):
    if a is None:
        return None
    t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
    return t.to(dtype).contiguous() if dtype is not None else t


def upload_weights(w, dtype):
    td = TDT[dtype]
    out = {}
    for k, v in w.items():
        if v is None:
            out[k] = None
        elif k == "router_b":
            out[k] = dev(v.astype(np.float32))
        else:
            out[k] = dev(v, td)
    return out


def desc_of(cfg):
    return B.make_desc(cfg.hidden, cfg.n_experts, cfg.inter, cfg.n_shared, cfg.shared_inter, cfg.top_k,
                       cfg.top_k_vis, TDT[cfg.dtype])


def host(t):
    return t.detach().float().cpu().numpy() if t.dtype == torch.bfloat16 else t.detach().cpu().numpy()


def row_rel_err(y, ref):
    """max over rows of |y - ref|_inf / |ref|_inf (rows with zero reference use the absolute error)."""
    y = np.asarray(y, np.float64); ref = np.asarray(ref, np.float64)
    if y.size == 0:
        return 0.0
    num = np.abs(y - ref).max(axis=1)
    den = np.abs(ref).max(axis=1)
    return float(np.max(num / np.where(den > 0, den, 1.0)))


_handle = None


def handle():
    global _handle
    if _handle is None:
        _handle = B.Handle(0)
    return _handle
