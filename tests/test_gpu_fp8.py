"""GPU parity of the FP8 weight stream (expert matrices as FP8 E4M3 bytes with one power-of-two scale per
128 x 128 block, expanded to bf16 in shared memory).

The storage format is exact in bf16, so the layer computes with exactly the values the bytes and scales
represent.  Two checks follow from that: (1) against the fp64 oracle fed those values (decoded on the host
with torch's own float8 type), within the bf16 tolerance 2e-2; (2) against the bf16 layer fed the same values
as bf16 weights, bit for bit in fixed-order mode, because both run the same contraction on the same numbers."""
import numpy as np
import pytest
import torch

from oracle import fmmoe_oracle as O
from paper_2511_17885_b200 import binding as B
from paper_2511_17885_b200 import inputs as I
from paper_2511_17885_b200.workload import upload_weights_fp8
from gpu_util import dev, handle, host, row_rel_err, upload_weights

pytestmark = pytest.mark.gpu


def fp8_layer(seed, T, H, E, I_, Ns, Is, std=0.05, bias=False):
    r = np.random.default_rng(seed)

    def d(shape):
        return I.round_to_storage(std * r.standard_normal(shape), "bf16")
    w = {"router_w": d((E, H)), "router_b": (0.5 * r.standard_normal(E)).astype(np.float32) if bias else None,
         "w_gate": d((E, I_, H)), "w_up": d((E, I_, H)), "w_down": d((E, H, I_)),
         "ws_gate": None, "ws_up": None, "ws_down": None}
    if Ns:
        w["ws_gate"] = d((Ns, Is, H)); w["ws_up"] = d((Ns, Is, H)); w["ws_down"] = d((Ns, H, Is))
    # blocks of very different magnitude, so that the block scales differ inside one matrix
    w["w_gate"][:, :, : H // 2] *= 8.0
    w["w_down"][0] *= 1.0 / 64.0
    stored, packed = I.weights_to_fp8(w)
    x = I.round_to_storage(r.standard_normal((T, H)), "bf16")
    mask = (r.random(T) < 0.7).astype(np.uint8)
    return x, mask, stored, packed


CASES = [
    # T, H, E, I, Ns, Is, K, Kv
    (300, 256, 8, 128, 0, 0, 2, 1),
    (1000, 256, 16, 384, 2, 256, 4, 2),
    (77, 512, 8, 256, 1, 128, 3, 0),
    (5, 128, 4, 128, 0, 0, 2, 1),
]


@pytest.mark.parametrize("case", CASES)
def test_fp8_weight_stream_against_oracle_and_against_the_bf16_layer(case):
    T, H, E, I_, Ns, Is, K, Kv = case
    x, mask, stored, packed = fp8_layer(sum(case), T, H, E, I_, Ns, Is, bias=True)
    if H >= 256:
        assert len({int(v) for v in np.unique(packed["w_gate_scale"])}) > 1      # more than one block scale in play
    h = handle()
    xd, md = dev(x, torch.bfloat16), dev(mask)
    wq = B.make_weights(upload_weights_fp8(stored, packed, "bf16", "cuda"))
    wb = B.make_weights(upload_weights(stored, "bf16"))                            # the same values as bf16 weights
    dq = B.make_desc(H, E, I_, Ns, Is, K, Kv, torch.bfloat16, B.WEIGHTS_FP8_BLOCK128)
    db = B.make_desc(H, E, I_, Ns, Is, K, Kv, torch.bfloat16)
    route = {"logits": torch.empty(T, E, dtype=torch.float32, device="cuda"),
             "topk_idx": torch.empty(T, K, dtype=torch.int32, device="cuda")}
    for flags in (B.FLAG_REDUCE_ON, B.FLAG_REDUCE_ON | B.FLAG_RESIDUAL | B.FLAG_DETERMINISTIC):
        yq = h.fmmoe_moe_forward(dq, wq, xd, md, flags, route=route)
        h.check_status()
        ref = O.moe_forward(x, mask, stored, K, Kv, True, bool(flags & B.FLAG_RESIDUAL), logits32=host(route["logits"]))
        assert np.array_equal(host(route["topk_idx"]), ref["topk_idx"])
        assert row_rel_err(host(yq), ref["out"]) < 2e-2
        if flags & B.FLAG_DETERMINISTIC:
            yb = h.fmmoe_moe_forward(db, wb, xd, md, flags)
            h.check_status()
            assert torch.equal(yq, yb)


def test_fp8_format_is_refused_where_it_cannot_run():
    h = handle()
    x, mask, stored, packed = fp8_layer(3, 64, 256, 4, 128, 0, 0)
    wq = B.make_weights(upload_weights_fp8(stored, packed, "bf16", "cuda"))
    # S_m not a multiple of 128
    with pytest.raises(B.FmmoeError) as e:
        h.fmmoe_moe_forward(B.make_desc(256, 4, 192, 0, 0, 2, 1, torch.bfloat16, B.WEIGHTS_FP8_BLOCK128), wq,
                            dev(x, torch.bfloat16), dev(mask), B.FLAG_REDUCE_ON)
    assert e.value.status == 2
    # fp32 layer with FP8 weights
    with pytest.raises(B.FmmoeError) as e:
        h.fmmoe_moe_forward(B.make_desc(256, 4, 128, 0, 0, 2, 1, torch.float32, B.WEIGHTS_FP8_BLOCK128), wq,
                            dev(x), dev(mask), B.FLAG_REDUCE_ON)
    assert e.value.status == 1
    # scales missing
    wb = B.make_weights(upload_weights(stored, "bf16"))
    with pytest.raises(B.FmmoeError) as e:
        h.fmmoe_moe_forward(B.make_desc(256, 4, 128, 0, 0, 2, 1, torch.bfloat16, B.WEIGHTS_FP8_BLOCK128), wb,
                            dev(x, torch.bfloat16), dev(mask), B.FLAG_REDUCE_ON)
    assert e.value.status == 1
