"""GPU parity with the QSGD quantizer: plans, streams (bit-exact) and aggregates against the
CPU oracle on the same seeded inputs, through the C ABI."""
import numpy as np
import pytest

import oracle as O
from paper_2402_03770_b200 import workloads as W
from gpu_util import (assert_aggregate_close, assert_plan_equal, gpu_decode_aggregate, gpu_params, gpu_plan_encode,
                      oracle_params, oracle_plan_encode, params_dict)
from stream_reader import parse, dequantize_qsgd
from test_gpu_parity import run_case

pytestmark = pytest.mark.gpu
QSGD = 1


@pytest.fixture(scope="module")
def torch_cuda():
    import torch
    assert torch.cuda.is_available()
    from paper_2402_03770_b200 import binding as B
    B.lib()
    B.cvlc_set_device(0)
    return torch


def test_default_scale_and_host_checks(torch_cuda):
    from paper_2402_03770_b200 import binding as B
    for d, b in [(5000, 1024), (11_200_000, 12000), (100_000_000, 12000)]:
        pd = params_dict(d, 8 * b, packet_bits=b, quantizer=QSGD)
        assert np.float64(gpu_params(pd).scale_B).view(np.uint64) == np.float64(oracle_params(pd).scale_B).view(np.uint64)
    x = np.random.default_rng(0).standard_normal(5000).astype(np.float32)
    pd = params_dict(5000, 4 * 1024, packet_bits=1024, quantizer=QSGD)
    with pytest.raises(B.CvlcError) as e:                                      # one bit holds no level
        gpu_plan_encode(x, pd, fixed_y=1)
    assert e.value.code == B.CVLC_ERR_INVALID_ARG
    with pytest.raises(B.CvlcError):                                           # an unknown quantizer
        gpu_plan_encode(x, params_dict(5000, 4 * 1024, packet_bits=1024, quantizer=2, scale_B=1.0))


@pytest.mark.parametrize("d", [5, 64, 1000, 4097, 12289, 100_003])
def test_ragged_sizes(torch_cuda, d):
    rng = np.random.default_rng(d)
    x = rng.laplace(0, 1e-2, d).astype(np.float32)
    if d < 1000:
        pd = params_dict(d, 96 * (1 if d < 60 else 5), packet_bits=96, max_code_bits=8, seed=d, client_id=1, round=2,
                         quantizer=QSGD)
    else:
        pd = params_dict(d, min(d // 400, 40) * 2048 + 5, packet_bits=2048, seed=d, client_id=1, round=2, quantizer=QSGD)
    of, ost = run_case(x, pd)
    assert of["n_y"][1] == 0 and of["y_min"] >= 2
    run_case(x, pd, fixed_y=8 if d < 1000 else 3)


@pytest.mark.parametrize("y", [2, 3, 7, 16, 31, 32])
def test_fixed_length_plans(torch_cuda, y):
    rng = np.random.default_rng(y)
    d = 40_000
    x = (rng.standard_normal(d) * 10.0 ** rng.uniform(-4, 0, d)).astype(np.float32)
    pd = params_dict(d, 12 * 4096, packet_bits=4096, seed=5, client_id=y, round=1, quantizer=QSGD, scale_B=1.0)
    of, ost = run_case(x, pd, fixed_y=y)
    ref = O.decode_aggregate([ost], np.ones(1, np.float32), d)
    status, out = gpu_decode_aggregate([ost], np.ones(1, np.float32), d)
    assert status == 0
    assert (out.view(np.uint32) == ref.view(np.uint32)).all()                  # one client: exact per record
    chk = np.zeros(d, dtype=np.float32)
    for pk in parse(ost).packets:                                              # and equal to an independent reader
        chk[pk.pid.astype(np.int64)] = dequantize_qsgd(pk)
    assert (out == chk).all()


def test_ties_zeros_and_a_dominant_coordinate(torch_cuda):
    rng = np.random.default_rng(12)
    d = 30_000
    x = (np.round(rng.standard_normal(d) * 4) / 4).astype(np.float32)          # many exact ties
    x[rng.integers(0, d, 60000)] = 0.0
    x[rng.integers(0, d, 6000)] = -0.0
    x[777] = 1e30                                                              # a packet whose norm is one value
    x[778] = -3e-39                                                            # a subnormal
    pd = params_dict(d, 60 * 2048, packet_bits=2048, seed=9, client_id=2, round=7, quantizer=QSGD)
    run_case(x, pd)
    of, ost = run_case(x, pd, fixed_y=4)
    assert of["k"] > int((x != 0).sum())                                       # zeros are transmitted too
    S = parse(ost)
    assert S.packets[0].pid[0] == 777 and S.packets[-1].lo == 0.0              # an all-zero packet has norm 0
    ref = O.decode_aggregate([ost], np.ones(1, np.float32), d)
    status, out = gpu_decode_aggregate([ost], np.ones(1, np.float32), d)
    assert status == 0 and (out.view(np.uint32) == ref.view(np.uint32)).all()


def test_huge_values_cut_the_norm_at_fp32_max(torch_cuda):
    d = 4096
    x = np.full(d, 3e38, dtype=np.float32)
    x[::2] *= -1
    pd = params_dict(d, 4 * 2048, packet_bits=2048, quantizer=QSGD, scale_B=1.0)
    of, ost = run_case(x, pd, fixed_y=6)
    assert parse(ost).packets[0].lo == np.finfo(np.float32).max


def test_batch_of_clients_and_mixed_aggregate(torch_cuda):
    torch = torch_cuda
    from paper_2402_03770_b200 import binding as B
    w = W.WORKLOADS["small_cnn"]
    d = 150_000
    dev = torch.device("cuda:0")
    clients = [0, 3, 4, 11, 19]
    xs, pds = [], []
    for c in clients:
        x = W.client_update(w, c, d=d)
        seed, cid, rnd = W.philox_ids(w, c)
        xs.append(x)
        pds.append(params_dict(d, 2 * d, seed=seed, client_id=cid, round=rnd, quantizer=QSGD))
    enc = B.BatchEncoder([gpu_params(pd) for pd in pds], dev)
    outs = enc.run([torch.from_numpy(x).to(dev) for x in xs])
    assert enc.status() == B.CVLC_OK
    streams = []
    for i, (x, pd) in enumerate(zip(xs, pds)):
        of, ost = oracle_plan_encode(x, pd)
        assert_plan_equal(enc.read_plan(i), of)
        assert (outs[i].cpu().numpy() == ost).all()
        streams.append(ost)
    # a PQ client joins the same aggregate
    pq = params_dict(d, 2 * d, seed=99, client_id=99, quantizer=0)
    of, ost = oracle_plan_encode(xs[0], pq)
    streams.append(ost)
    wts = np.arange(1, len(streams) + 1, dtype=np.float32)
    ref = O.decode_aggregate(streams, wts, d)
    status, out = gpu_decode_aggregate(streams, wts, d)
    assert status == 0
    assert_aggregate_close(out, ref)
    # quantizers cannot be mixed inside one encode batch
    with pytest.raises(B.CvlcError):
        B.BatchEncoder([gpu_params(pds[0]), gpu_params(pq)], dev).run([torch.from_numpy(xs[0]).to(dev)] * 2)


def test_decode_rejects_malformed_qsgd_streams(torch_cuda):
    from paper_2402_03770_b200 import binding as B
    rng = np.random.default_rng(1)
    d = 5000
    x = rng.laplace(0, 1e-2, d).astype(np.float32)
    pd = params_dict(d, 6 * 1024, packet_bits=1024, quantizer=QSGD)
    of, st = oracle_plan_encode(x, pd)
    w = np.ones(1, np.float32)
    bad_y = st.copy()
    bad_y[64 + 128 * 5 + 1] = 1
    bad_q = st.copy()
    bad_q[6] = 2
    bad_norm = st.copy()
    bits = np.unpackbits(bad_norm[64:64 + 128], bitorder="little")
    bits[16:48] = np.unpackbits(np.array([0x7FC00000], dtype="<u4").view(np.uint8), bitorder="little")
    bad_norm[64:64 + 128] = np.packbits(bits, bitorder="little")
    for bad in (bad_y, bad_q, bad_norm):
        with pytest.raises(O.OracleError):
            O.decode_aggregate([bad], w, d)
        status, out = gpu_decode_aggregate([bad], w, d)
        assert status == B.CVLC_ERR_BAD_STREAM
    status, out = gpu_decode_aggregate([st], w, d)
    assert status == 0
