"""GPU parity of the unframed (version 2) stream: cvlc_encode_unframed_batch against the oracle's stream byte for
byte (and its reported length), cvlc_decode_aggregate_unframed against the oracle's aggregate, and both against the
framed path they must agree with."""
import numpy as np
import pytest

import oracle as O
from paper_2402_03770_b200 import workloads as W
from gpu_util import assert_aggregate_close, gpu_params, oracle_params, params_dict

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    from paper_2402_03770_b200 import binding as B
    assert torch.cuda.is_available()
    B.lib()
    B.cvlc_set_device(0)
    return torch, B


def gpu_unframed(torch, B, xs, pds, use_plan_ws=True, fixed_y=0):
    dev = torch.device("cuda:0")
    params = [gpu_params(pd) for pd in pds]
    n = len(xs)
    enc = B.BatchEncoder(params, dev)
    dxs = [torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(dev) for x in xs]
    enc.plan(dxs, fixed_y=fixed_y)
    cap = B.cvlc_unframed_stream_capacity(params[0])
    assert cap > 0
    outs = [torch.full((cap,), 0xAB, dtype=torch.uint8, device=dev) for _ in range(n)]
    sizes = torch.zeros(n, dtype=torch.int64, device=dev)
    uf_ws = B.alloc_bytes(B.cvlc_unframed_workspace_bytes(params[0], n), dev)
    B.cvlc_encode_unframed_batch(dxs, params, enc.plans, outs, sizes, enc.enc_ws, uf_ws,
                                 plan_ws=enc.plan_ws if use_plan_ws else None)
    status = enc.status()
    sz = sizes.cpu().numpy()
    return status, [o.cpu().numpy()[:int(s)].copy() for o, s in zip(outs, sz)], outs, sizes


def gpu_decode_unframed(torch, B, streams, weights, d, **kw):
    dev = torch.device("cuda:0")
    n = len(streams)
    ds = [torch.from_numpy(np.ascontiguousarray(s, dtype=np.uint8)).to(dev) for s in streams]
    ptrs = torch.tensor([s.data_ptr() for s in ds], dtype=torch.int64, device=dev)
    sizes = torch.tensor([s.numel() for s in ds], dtype=torch.int64, device=dev)
    w = torch.from_numpy(np.ascontiguousarray(weights, dtype=np.float32)).to(dev)
    ws = B.alloc_bytes(B.cvlc_decode_workspace_bytes(n), dev)
    out_init = kw.get("out_init")
    out = torch.full((d,), float("nan"), dtype=torch.float32, device=dev) if out_init is None else \
        torch.from_numpy(out_init.astype(np.float32)).to(dev)
    B.cvlc_decode_aggregate_unframed(ptrs, sizes, w, n, kw.get("weight_total", 0.0), d, out, out_init is not None, ws)
    return B.cvlc_read_status(ws), out.cpu().numpy()


@pytest.mark.parametrize("quantizer", [0, 1])
@pytest.mark.parametrize("d,R,pb,n", [(5003, 6, 1024, 1), (60_000, 9, 4096, 3), (300_001, 40, 12000, 5)])
def test_unframed_streams_match_oracle(env, d, R, pb, n, quantizer):
    torch, B = env
    rng = np.random.default_rng(d + quantizer)
    xs = [(rng.laplace(0, 1e-2, d) * (1 + c)).astype(np.float32) for c in range(n)]
    if n > 1:
        xs[1][::5] = 0.0
    pds = [params_dict(d, R * pb + 7, packet_bits=pb, seed=3 + c, client_id=c, round=2, quantizer=quantizer,
                       scale_B=1.0 + 0.01 * c if c else None) for c in range(n)]
    refs = []
    for x, pd in zip(xs, pds):
        po = oracle_params(pd)
        refs.append(O.encode_unframed(x, po, O.plan(x, po)))
    for use_plan_ws in (True, False):
        status, got, _, _ = gpu_unframed(torch, B, xs, pds, use_plan_ws)
        assert status == 0
        for c in range(n):
            assert got[c].size == refs[c].size, (c, got[c].size, refs[c].size)
            assert (got[c] == refs[c]).all(), (c, int(np.nonzero(got[c] != refs[c])[0][0]))
    w = rng.uniform(1, 5, n).astype(np.float32)
    want = O.decode_aggregate_unframed(refs, w, d)
    status, out = gpu_decode_unframed(torch, B, refs, w, d)
    assert status == 0
    assert_aggregate_close(out, want)


def test_unframed_on_workload_shapes_and_fixed_lengths(env):
    torch, B = env
    for name, d, bpc in [("resnet18", 400_000, 2.0), ("resnet50", 500_000, 1.0), ("stress", 1_000_000, 0.25)]:
        w = W.WORKLOADS[name]
        xs = [W.client_update(w, c, d=d) for c in range(2)]
        pds = [params_dict(d, int(bpc * d), seed=c, client_id=c) for c in range(2)]
        refs = [O.encode_unframed(x, oracle_params(pd), O.plan(x, oracle_params(pd))) for x, pd in zip(xs, pds)]
        status, got, _, _ = gpu_unframed(torch, B, xs, pds)
        assert status == 0
        for c in range(2):
            assert got[c].size == refs[c].size and (got[c] == refs[c]).all(), (name, c)
        framed = [O.encode(x, oracle_params(pd), O.plan(x, oracle_params(pd))) for x, pd in zip(xs, pds)]
        assert sum(g.size for g in got) < 0.9 * sum(f.size for f in framed)
        a = O.decode_aggregate(framed, np.ones(2, np.float32), d)
        status, out = gpu_decode_unframed(torch, B, got, np.ones(2, np.float32), d)
        assert status == 0
        assert_aggregate_close(out, a)                                   # the same aggregate as the framed streams
    rng = np.random.default_rng(4)
    x = rng.standard_normal(50_000).astype(np.float32)
    for y in (1, 8, 32):
        pd = params_dict(50_000, 9 * 12000, seed=1, scale_B=1.2)
        po = oracle_params(pd)
        ref = O.encode_unframed(x, po, O.plan_fixed(po, y))
        status, got, _, _ = gpu_unframed(torch, B, [x], [pd], fixed_y=y)
        assert status == 0 and got[0].size == ref.size and (got[0] == ref).all(), y


def test_unframed_encode_then_decode_on_the_device(env):
    """the lengths the encoder leaves on the device feed the decoder directly (no host round trip)"""
    torch, B = env
    dev = torch.device("cuda:0")
    d, n = 120_000, 4
    rng = np.random.default_rng(8)
    xs = [rng.laplace(0, 1e-2, d).astype(np.float32) for _ in range(n)]
    pds = [params_dict(d, 30 * 4096, packet_bits=4096, seed=c, client_id=c) for c in range(n)]
    status, got, outs, sizes = gpu_unframed(torch, B, xs, pds)
    assert status == 0
    ptrs = torch.tensor([o.data_ptr() for o in outs], dtype=torch.int64, device=dev)
    w = torch.tensor([1.0, 2.0, 3.0, 4.0], dtype=torch.float32, device=dev)
    ws = B.alloc_bytes(B.cvlc_decode_workspace_bytes(n), dev)
    out = torch.empty(d, dtype=torch.float32, device=dev)
    B.cvlc_decode_aggregate_unframed(ptrs, sizes, w, n, 0.0, d, out, False, ws)
    assert B.cvlc_read_status(ws) == 0
    want = O.decode_aggregate_unframed(got, np.array([1, 2, 3, 4], np.float32), d)
    assert_aggregate_close(out.cpu().numpy(), want)
    # accumulate over two calls with the total weight given
    status, half = gpu_decode_unframed(torch, B, got[:2], np.array([1, 2], np.float32), d, weight_total=10.0)
    status2, both = gpu_decode_unframed(torch, B, got[2:], np.array([3, 4], np.float32), d, weight_total=10.0, out_init=half)
    assert status == 0 and status2 == 0
    assert_aggregate_close(both, want)


def test_unframed_refusals(env):
    torch, B = env
    # blocks of more than 2048 records are not supported: the capacity query says so, the encoder refuses
    p = gpu_params(params_dict(100_000, 3 * 65536, packet_bits=65536))
    assert B.cvlc_unframed_stream_capacity(p) == 0
    x, pd = np.random.default_rng(1).laplace(0, 1e-2, 20_000).astype(np.float32), params_dict(20_000, 6 * 1024, packet_bits=1024)
    po = oracle_params(pd)
    u = O.encode_unframed(x, po, O.plan(x, po))
    f = O.encode(x, po, O.plan(x, po))
    w = np.ones(1, np.float32)
    bads = [u[:-8], np.concatenate([u, np.zeros(8, np.uint8)]), f]
    for off, val in ((0, 0), (4, 1), (64 + 4 * 8, 99), (64 + 264 + 8 + 8, 0xFF)):
        b = u.copy()
        b[off] = val
        bads.append(b)
    pid_bad = u.copy()
    pid_bad[64 + 264 + 8 + 6 * 8 + 8:64 + 264 + 8 + 6 * 8 + 40] = 0xFF                # a run of one-bits: a position beyond d
    bads.append(pid_bad)
    for bad in bads:
        with pytest.raises(O.OracleError):
            O.decode_aggregate_unframed([bad], w, 20_000)
        status, _ = gpu_decode_unframed(torch, B, [bad], w, 20_000)
        assert status == B.CVLC_ERR_BAD_STREAM
    status, out = gpu_decode_unframed(torch, B, [u], w, 20_000)                          # the context is still usable
    assert status == 0
    assert_aggregate_close(out, O.decode_aggregate_unframed([u], w, 20_000))
    from gpu_util import gpu_decode_aggregate
    status, _ = gpu_decode_aggregate([u], w, 20_000)                                     # the framed decoder refuses it
    assert status == B.CVLC_ERR_BAD_STREAM
