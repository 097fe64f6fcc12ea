"""GPU parity on seeded random problem shapes: coordinates, budget, packet and header size, longest code,
quantizer and value distribution drawn at random (small enough for the oracle to take milliseconds), so that
combinations nobody thought of listing still meet the bit-exact bar: plan and stream against the oracle with both
selection kernels, the aggregate of three differently weighted copies within 1e-6 rel / 1e-7 abs.  Where the
oracle refuses the parameters the CUDA path must refuse them with the same code."""
import numpy as np
import pytest

import oracle as O
from gpu_util import (assert_aggregate_close, assert_plan_equal, gpu_decode_aggregate, gpu_plan_encode, oracle_params,
                      oracle_plan_encode, params_dict)

pytestmark = pytest.mark.gpu


def draw_case(rng):
    d = int(rng.choice([17, 255, 1000, 4097, 65_537, 200_003, int(rng.integers(5_000, 300_000)), int(rng.integers(5_000, 300_000))]))
    packet_bits = 32 * int(rng.choice([4, 8, 16, 47, 64, 125, 256, 375, 1024]))
    header_bits = int(min(packet_bits - 1, rng.choice([80, 81, 96, 128, 200])))
    quantizer = int(rng.integers(0, 2))
    max_bits = int(rng.choice([3, 8, 12, 16, 24, 32, 32]))
    s_bits = max(1, int(np.ceil(np.log2(d))))
    fit = max(1, int(d * (s_bits + 8) // max(1, packet_bits - header_bits)))   # packets that d coordinates can fill at 8 bits
    packets = int(min(fit, rng.choice([1, 2, 3, 7, 20, 60])))
    kind = rng.choice(["laplace", "ties", "sparse", "constant", "wide"])
    if kind == "laplace":
        x = rng.laplace(0, 1e-3, d)
    elif kind == "ties":
        x = np.round(rng.standard_t(3, d) * 4) / 64.0
    elif kind == "sparse":
        x = rng.laplace(0, 1e-2, d) * (rng.random(d) < 0.05)
    elif kind == "constant":
        x = np.full(d, -0.25)
    else:
        x = rng.standard_normal(d) * 10.0 ** rng.uniform(-30, 30, d)
    pd = params_dict(d, packets * packet_bits + int(rng.integers(0, packet_bits)), packet_bits=packet_bits,
                     header_bits=header_bits, quantizer=quantizer, max_code_bits=max_bits,
                     seed=int(rng.integers(0, 2 ** 63)), client_id=int(rng.integers(0, 2 ** 32)),
                     round=int(rng.integers(0, 2 ** 32)),
                     scale_B=(None if rng.random() < 0.6 else float(rng.choice([1.0, 1.25, 2.0, 17.5]))))
    return x.astype(np.float32), pd, kind


def check_unframed(torch, B, x, pd, framed):
    """where the shape allows it, the unframed stream equals the oracle's byte for byte and decodes to the aggregate of
    the framed one; where it does not (blocks of more than 2048 records), the capacity query says so"""
    from gpu_util import gpu_params
    dev = torch.device("cuda:0")
    p = gpu_params(pd)
    cap = B.cvlc_unframed_stream_capacity(p)
    po = oracle_params(pd)
    s_bits = max(1, int(np.ceil(np.log2(pd["d"]))))
    y_lo = 2 if pd["quantizer"] else 1
    if (pd["packet_bits"] - pd["header_bits"]) // (s_bits + y_lo) > 2048 or pd["max_code_bits"] < y_lo:
        assert cap == 0
        return
    assert cap >= O.unframed_capacity(po)
    ref = O.encode_unframed(x, po, O.plan(x, po))
    enc = B.BatchEncoder([p], dev)
    xd = [torch.from_numpy(x).to(dev)]
    enc.plan(xd)
    out = torch.full((cap,), 0x5A, dtype=torch.uint8, device=dev)
    size = torch.zeros(1, dtype=torch.int64, device=dev)
    uf_ws = B.alloc_bytes(B.cvlc_unframed_workspace_bytes(p, 1), dev)
    B.cvlc_encode_unframed_batch(xd, [p], enc.plans, [out], size, enc.enc_ws, uf_ws, plan_ws=enc.plan_ws)
    assert enc.status() == 0
    n = int(size.item())
    assert n == ref.size and (out[:n].cpu().numpy() == ref).all(), pd
    ptr = torch.tensor([out.data_ptr()], dtype=torch.int64, device=dev)
    w = torch.ones(1, dtype=torch.float32, device=dev)
    ws = B.alloc_bytes(B.cvlc_decode_workspace_bytes(1), dev)
    agg = torch.empty(pd["d"], dtype=torch.float32, device=dev)
    B.cvlc_decode_aggregate_unframed(ptr, size, w, 1, 0.0, pd["d"], agg, False, ws)
    assert B.cvlc_read_status(ws) == 0
    assert_aggregate_close(agg.cpu().numpy(), O.decode_aggregate([framed], np.ones(1, np.float32), pd["d"]))


@pytest.mark.parametrize("seed", range(20))
def test_random_shapes(seed):
    import torch
    from paper_2402_03770_b200 import binding as B
    assert torch.cuda.is_available()
    B.lib()
    B.cvlc_set_device(0)
    rng = np.random.default_rng(9000 + seed)
    done = refused = 0
    for _ in range(12):
        x, pd, kind = draw_case(rng)
        try:
            of, ost = oracle_plan_encode(x, pd)
        except O.OracleError as oe:
            with pytest.raises(B.CvlcError) as e:
                gpu_plan_encode(x, pd)
            assert e.value.code == oe.code, (pd, kind)
            refused += 1
            continue
        for use_plan_ws, compress in ((True, 0), (False, 0), (True, 2 if done % 2 else 1)):
            status, gp, gst = gpu_plan_encode(x, pd, use_plan_ws=use_plan_ws, compress=compress)
            assert status == 0, (status, pd, kind)
            assert_plan_equal(gp, of)
            assert gst.size == ost.size and (gst == ost).all(), (pd, kind, use_plan_ws, compress)
        check_unframed(torch, B, x, pd, ost)
        weights = np.array([1.0, 0.5, 3.0], dtype=np.float32)
        ref = O.decode_aggregate([ost, ost, ost], weights, pd["d"])
        status, out = gpu_decode_aggregate([ost, ost, ost], weights, pd["d"])
        assert status == 0
        assert_aggregate_close(out, ref)
        done += 1
    assert done + refused == 12
