"""CPU-side checks of the boundary: the library loads without a GPU, exports every symbol
include/fmmoe.h declares, and its host-only entry points agree with the oracle."""
import ctypes
import itertools
import os
import re

import numpy as np
import pytest

from oracle import fmmoe_oracle as O
from paper_2511_17885_b200 import binding as B
from paper_2511_17885_b200 import build as builder

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def L():
    builder.build()
    return B.lib()


def test_every_declared_symbol_is_exported(L):
    hdr = open(os.path.join(ROOT, "include", "fmmoe.h")).read()
    hdr = re.sub(r"/\*.*?\*/", "", hdr, flags=re.S)
    names = set(re.findall(r"\b(fmmoe_[a-z_0-9]+)\s*\(", hdr))
    assert {"fmmoe_route", "fmmoe_moe_forward", "fmmoe_prune_visual"} <= names
    for n in sorted(names):
        assert hasattr(L, n), f"{n} declared in fmmoe.h but not exported"


def test_status_strings(L):
    assert L.fmmoe_status_string(0) == b"ok"
    assert len({L.fmmoe_status_string(i) for i in range(7)}) == 7


def test_kept_count_matches_oracle(L):
    for n_v, eta, W, g, mm in itertools.product([0, 7, 97, 224, 2304, 3328], [0, 20, 90, 1152, 2496, 5000],
                                                [2, 3, 5, 8], [0.0, 0.025, 0.05, 0.2, 0.7, 3.0], [0, 2]):
        p = B.prune_params(W, g, merge_mode=mm)
        kept, m, d = B.fmmoe_prune_kept_count(n_v, eta, p)
        assert (m, d, kept) == O.prune_counts(n_v, eta, W, g, mm), (n_v, eta, W, g, mm)
    assert B.fmmoe_prune_kept_count(10, 5, B.prune_params(1, 0.1))[0] == -1      # W < 2
    assert B.fmmoe_prune_kept_count(10, 5, B.prune_params(9, 0.1))[0] == -1      # W > max
    assert B.fmmoe_prune_kept_count(-1, 5, B.prune_params(3, 0.1))[0] == -1


def test_workspace_sizes(L):
    import torch
    d = B.make_desc(2048, 64, 1408, 2, 1408, 6, 3, torch.bfloat16)
    a = B.fmmoe_workspace_bytes(d, 2432)
    b = B.fmmoe_workspace_bytes(d, 2432, B.FLAG_DETERMINISTIC)
    assert a > 0 and b > a                                   # deterministic mode stores per-pair outputs
    assert B.fmmoe_workspace_bytes(d, 4864) > a
    assert B.fmmoe_workspace_bytes(d, -1) == 0
    bad = B.make_desc(2048, 300, 1408, 0, 0, 6, 3, torch.bfloat16)      # too many experts
    assert B.fmmoe_workspace_bytes(bad, 10) == 0
    assert L.fmmoe_prune_workspace_bytes(1000, 2) > 1000 * 4


def test_no_gpu_means_loud_failure(L):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(B.FmmoeError):
        B.Handle(0)
