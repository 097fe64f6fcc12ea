"""GPU parity of the steps either side of one round's compression: planning at the parameter server
from transmitted histograms, two rounds chained through B_next, and the model step."""
import numpy as np
import pytest

import oracle as O
from paper_2402_03770_b200 import workloads as W
from gpu_util import (assert_aggregate_close, assert_plan_equal, gpu_params, gpu_plan_encode, oracle_params,
                      oracle_plan_encode, params_dict)

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env():
    import torch
    from paper_2402_03770_b200 import binding as B
    assert torch.cuda.is_available()
    B.lib()
    B.cvlc_set_device(0)
    return torch, B


def plan_fields(pl):
    return dict(s=pl.s, R=pl.R, y_min=pl.y_min, n_lengths=pl.n_lengths, k=pl.k, alpha=pl.alpha, alpha_q=pl.alpha_q,
                beta=pl.beta, gamma=pl.gamma, B_next=pl.B_next, n_y=[pl.n_y[y] for y in range(33)],
                cap=[pl.cap[y] for y in range(33)])


@pytest.mark.parametrize("quantizer", [0, 1])
def test_server_side_planning_from_histograms(env, quantizer):
    torch, B = env
    dev = torch.device("cuda:0")
    w = W.WORKLOADS["small_cnn"]
    d = 300_001
    clients = [0, 1, 2, 7, 13]
    xs = [W.client_update(w, c, d=d) for c in clients]
    pds = [params_dict(d, 2 * d, seed=c, client_id=c, round=3, quantizer=quantizer) for c in clients]
    params = [gpu_params(pd) for pd in pds]
    n = len(clients)
    xd = [torch.from_numpy(x).to(dev) for x in xs]
    # client side: the histograms
    ws = B.alloc_bytes(B.cvlc_plan_batch_workspace_bytes(params[0], n), dev)
    hist = torch.full((n * B.HIST_BINS,), -1, dtype=torch.int64, device=dev)
    B.cvlc_histogram_batch(xd, params, hist, ws)
    assert B.cvlc_read_status(ws) == B.CVLC_OK
    h = hist.cpu().numpy().view(np.uint64).reshape(n, B.HIST_BINS)
    for i, x in enumerate(xs):
        rc, oh = O.histogram(x)
        assert rc == O.ORC_OK and (h[i] == oh).all()
    # server side: plans from the histograms alone
    plans = B.alloc_bytes(n * B.PLAN_BYTES, dev)
    ws2 = B.alloc_bytes(B.cvlc_plan_batch_workspace_bytes(params[0], n), dev)
    B.cvlc_plan_from_histogram_batch(hist, params, plans, ws2)
    assert B.cvlc_read_status(ws2) == B.CVLC_OK
    enc_ws = B.alloc_bytes(B.cvlc_encode_batch_workspace_bytes(params[0], n, 0), dev)
    outs = [B.alloc_bytes(B.cvlc_stream_bytes(params[0]), dev) for _ in range(n)]
    for i, (x, pd) in enumerate(zip(xs, pds)):
        of = plan_fields(O.plan_from_histogram(h[i], oracle_params(pd)))
        assert_plan_equal(B.read_plan(plans[i * B.PLAN_BYTES:(i + 1) * B.PLAN_BYTES]), of)
    # client side again: encode with the returned plans; their workspace holds no segment tables
    B.cvlc_encode_batch(xd, params, plans, outs, enc_ws, plan_ws=None)
    assert B.cvlc_read_status(enc_ws) == B.CVLC_OK
    for i, (x, pd) in enumerate(zip(xs, pds)):
        of, ost = oracle_plan_encode(x, pd)
        assert (outs[i].cpu().numpy() == ost).all()
    B.cvlc_encode_batch(xd, params, plans, outs, enc_ws, plan_ws=ws2)
    assert B.cvlc_read_status(enc_ws) == B.CVLC_ERR_PLAN_MISMATCH
    B.cvlc_encode_batch(xd, params, plans, outs, enc_ws, plan_ws=ws)           # nor does the histogram call's
    assert B.cvlc_read_status(enc_ws) == B.CVLC_ERR_PLAN_MISMATCH


def test_bad_histograms_are_reported(env):
    torch, B = env
    dev = torch.device("cuda:0")
    d = 50_000
    x = np.random.default_rng(3).laplace(0, 1e-2, d).astype(np.float32)
    pd = params_dict(d, 10 * 2048, packet_bits=2048)
    rc, h = O.histogram(x)
    j = int(np.nonzero(h)[0][0])
    short = h.copy()
    short[j] -= 1
    inf = short.copy()
    inf[0x7F800000 >> 19] += 1
    params = [gpu_params(pd)] * 3
    hist = torch.from_numpy(np.concatenate([h, short, inf]).view(np.int64)).to(dev)
    plans = B.alloc_bytes(3 * B.PLAN_BYTES, dev)
    ws = B.alloc_bytes(B.cvlc_plan_batch_workspace_bytes(params[0], 3), dev)
    B.cvlc_plan_from_histogram_batch(hist, params, plans, ws)
    assert B.cvlc_read_status(ws) in (B.CVLC_ERR_INVALID_ARG, B.CVLC_ERR_NONFINITE_INPUT)
    got = [B.read_plan(plans[i * B.PLAN_BYTES:(i + 1) * B.PLAN_BYTES]).status for i in range(3)]
    assert got == [B.CVLC_OK, B.CVLC_ERR_INVALID_ARG, B.CVLC_ERR_NONFINITE_INPUT]
    for bad, code in ((short, O.ORC_ERR_INVALID_ARG), (inf, O.ORC_ERR_NONFINITE_INPUT)):
        with pytest.raises(O.OracleError) as e:
            O.plan_from_histogram(bad, oracle_params(pd))
        assert e.value.code == code


def test_two_rounds_chained_through_B_next(env):
    """round t+1 runs with B = B_next of round t and its own Philox counter word"""
    torch, B = env
    w = W.WORKLOADS["small_cnn"]
    d = 200_000
    x0 = W.client_update(w, 4, d=d)
    x1 = (W.client_update(w, 5, d=d) * np.float32(0.8)).astype(np.float32)
    pd0 = params_dict(d, 2 * d, seed=4, client_id=4, round=0)
    of0, ost0 = oracle_plan_encode(x0, pd0)
    st, gp0, gst0 = gpu_plan_encode(x0, pd0)
    assert st == 0 and (gst0 == ost0).all()
    assert_plan_equal(gp0, of0)
    pd1 = params_dict(d, 2 * d, seed=4, client_id=4, round=1, scale_B=float(gp0.B_next))
    of1, ost1 = oracle_plan_encode(x1, pd1)
    st, gp1, gst1 = gpu_plan_encode(x1, pd1)
    assert st == 0 and (gst1 == ost1).all()
    assert_plan_equal(gp1, of1)
    assert np.frombuffer(gst1[48:56].tobytes(), dtype="<f8")[0] == gp0.B_next  # the stream carries the scale it used


@pytest.mark.parametrize("d", [4000, 100_003])
def test_model_step(env, d):
    torch, B = env
    dev = torch.device("cuda:0")
    rng = np.random.default_rng(d)
    n = 6
    streams = []
    for i in range(n):
        x = rng.laplace(0, 1e-2, d).astype(np.float32)
        pd = params_dict(d, 8 * 2048, packet_bits=2048, seed=i, client_id=i, quantizer=i % 2)
        streams.append(oracle_plan_encode(x, pd)[1])
    wts = rng.uniform(1, 5, n).astype(np.float32)
    model = rng.standard_normal(d).astype(np.float32)
    ref_agg = O.decode_aggregate(streams, wts, d)
    ref = O.decode_apply(streams, wts, model.copy())
    agg = B.Aggregator(n, d, dev)
    agg.set_clients([torch.from_numpy(s).to(dev) for s in streams], torch.from_numpy(wts))
    md = torch.from_numpy(model).to(dev)
    scratch = torch.full((d,), float("nan"), dtype=torch.float32, device=dev)
    agg.apply(n, md, scratch)
    assert agg.status() == B.CVLC_OK
    got_agg = scratch.cpu().numpy()
    assert_aggregate_close(got_agg, ref_agg)
    got = md.cpu().numpy()
    assert (got == model - got_agg).all()                                     # one fp32 subtraction per weight
    assert np.abs(got.astype(np.float64) - ref.astype(np.float64)).max() <= 1e-7 + 1e-6 * np.abs(ref_agg).max() + 6e-8 * np.abs(model).max()
    assert (got[ref_agg == 0] == model[ref_agg == 0]).all()
    # a malformed stream leaves the model as it was
    bad = streams[0].copy()
    bad[0] = 0
    agg.set_clients([torch.from_numpy(bad).to(dev)] + [torch.from_numpy(s).to(dev) for s in streams[1:]], torch.from_numpy(wts))
    md2 = torch.from_numpy(model).to(dev)
    agg.apply(n, md2, scratch)
    assert agg.status() == B.CVLC_ERR_BAD_STREAM
    assert (md2.cpu().numpy() == model).all()


@pytest.mark.parametrize("quantizer,use_plan_ws", [(0, True), (0, False), (1, True)])
def test_error_compensation_over_rounds(env, quantizer, use_plan_ws):
    """three rounds with the error-compensation memory, three clients per batch: the memories (every coordinate)
    and the streams equal the oracle's bit for bit, round after round"""
    torch, B = env
    dev = torch.device("cuda:0")
    d, n, T = 70_003, 3, 3
    rng = np.random.default_rng(17)
    mem_ref = [np.zeros(d, np.float32) for _ in range(n)]
    mem_gpu = [torch.zeros(d, dtype=torch.float32, device=dev) for _ in range(n)]
    scale = [None] * n
    for t in range(T):
        updates = [(rng.laplace(0, 1e-2, d) * (1.0 + c)).astype(np.float32) for c in range(n)]
        if t == 1:
            updates[1][::3] = -0.0
        pds = [params_dict(d, 9 * 4096, packet_bits=4096, seed=40 + c, client_id=c, round=t, quantizer=quantizer,
                           scale_B=scale[c]) for c in range(n)]
        # oracle: accumulate, plan, encode, residual
        ref_streams, ref_plans = [], []
        for c in range(n):
            a = O.ec_accumulate(mem_ref[c], updates[c])
            po = oracle_params(pds[c])
            pl = O.plan(a, po)
            st = O.encode(a, po, pl)
            mem_ref[c] = O.ec_residual(a, st)
            ref_streams.append(st)
            ref_plans.append(pl)
        # CUDA path
        params = [gpu_params(pd) for pd in pds]
        B.cvlc_ec_accumulate_batch(mem_gpu, [torch.from_numpy(u).to(dev) for u in updates])
        enc = B.BatchEncoder(params, dev)
        enc.plan(mem_gpu)
        B.cvlc_encode_batch_ec(mem_gpu, params, enc.plans, enc.outs, enc.enc_ws, plan_ws=enc.plan_ws if use_plan_ws else None)
        assert enc.status() == B.CVLC_OK
        for c in range(n):
            assert_plan_equal(enc.read_plan(c), plan_fields(ref_plans[c]))
            assert (enc.outs[c].cpu().numpy() == ref_streams[c]).all(), (t, c)
            got = mem_gpu[c].cpu().numpy()
            assert (got.view(np.uint32) == mem_ref[c].view(np.uint32)).all(), (t, c)
            scale[c] = ref_plans[c].B_next
    assert all(np.abs(m).max() > 0 for m in mem_ref)


def test_ec_accumulate_rejects_bad_arguments(env):
    torch, B = env
    dev = torch.device("cuda:0")
    m = torch.zeros(1000, dtype=torch.float32, device=dev)
    with pytest.raises(B.CvlcError) as e:
        B.cvlc_ec_accumulate_batch([m], [m])                      # memory and update must be distinct buffers
    assert e.value.code == B.CVLC_ERR_INVALID_ARG
