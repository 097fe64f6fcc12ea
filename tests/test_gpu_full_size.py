"""GPU parity at the full workload sizes, in the batched launch configuration the
benchmark times: streams bit-exact against the oracle, aggregates within 1e-6 rel /
1e-7 abs.  The oracle runs in spawned worker processes (one client each)."""
import numpy as np
import pytest

import oracle as O
from paper_2402_03770_b200 import workloads as W
from gpu_util import assert_aggregate_close, assert_plan_equal, gpu_params, oracle_encode_clients, params_dict

pytestmark = pytest.mark.gpu


def gpu_batch_encode(workload, clients, d, bpc, max_candidates, torch, B, quantizer=0, one_call=True):
    """one_call: cvlc_compress_batch with the length tuning on a side stream (what the benchmark times); otherwise
    cvlc_plan_batch followed by cvlc_encode_batch"""
    w = W.WORKLOADS[workload]
    dev = torch.device("cuda:0")
    params, xs = [], []
    for c in clients:
        x = W.client_update(w, c, d=d)
        seed, cid, rnd = W.philox_ids(w, c)
        params.append(gpu_params(params_dict(x.size, int(np.floor(bpc * x.size)), seed=seed, client_id=cid, round=rnd,
                                             quantizer=quantizer)))
        xs.append(torch.from_numpy(x).to(dev))
    enc = B.BatchEncoder(params, dev, max_candidates=max_candidates)
    outs = enc.compress(xs, side_stream=torch.cuda.Stream(device=dev)) if one_call else enc.run(xs)
    assert enc.status() == B.CVLC_OK
    del xs
    return enc, outs


def check_against_oracle(enc, outs, oracle_results):
    for i, (client, fields, ost) in enumerate(oracle_results):
        assert_plan_equal(enc.read_plan(i), fields)
        got = outs[i].cpu().numpy()
        assert got.size == ost.size
        if not (got == ost).all():
            bad = np.nonzero(got != ost)[0]
            raise AssertionError(f"client {client}: stream differs at {bad.size} bytes, first at {bad[0]}")


def decode_both(outs, oracle_streams, weights, d, torch, B, batches=1):
    dev = torch.device("cuda:0")
    n = len(outs)
    result = torch.full((d,), float("nan"), dtype=torch.float32, device=dev)
    Wt = float(np.asarray(weights, dtype=np.float64).sum())
    per = (n + batches - 1) // batches
    ref = None
    for b in range(batches):
        sl = slice(b * per, min(n, (b + 1) * per))
        agg = B.Aggregator(sl.stop - sl.start, d, dev)
        agg.set_clients(outs[sl], torch.from_numpy(np.asarray(weights[sl], dtype=np.float32)))
        agg.run(sl.stop - sl.start, result, weight_total=Wt, accumulate=(b > 0))
        assert agg.status() == B.CVLC_OK
        ref = O.decode_aggregate(oracle_streams[sl], np.asarray(weights[sl], dtype=np.float32), d, weight_total=Wt,
                                 out=ref, accumulate=(b > 0))
    assert_aggregate_close(result.cpu().numpy(), ref)
    return ref


@pytest.fixture(scope="module")
def env():
    import torch
    from paper_2402_03770_b200 import binding as B
    assert torch.cuda.is_available()
    B.lib()
    B.cvlc_set_device(0)
    return torch, B


def test_small_cnn_all_20_clients(env):
    torch, B = env
    w = W.WORKLOADS["small_cnn"]
    clients = list(range(w.n_clients))
    ref = oracle_encode_clients("small_cnn", clients, None, 2.0)
    for one_call in (True, False):
        enc, outs = gpu_batch_encode("small_cnn", clients, None, 2.0, 0, torch, B, one_call=one_call)
        check_against_oracle(enc, outs, ref)
    decode_both(outs, [r[2] for r in ref], W.client_weights(w), w.d, torch, B)


@pytest.mark.parametrize("bpc", [0.5, 1.0, 4.0])
def test_resnet18_budget_sweep_two_clients(env, bpc):
    torch, B = env
    w = W.WORKLOADS["resnet18"]
    clients = [0, 57]
    ref = oracle_encode_clients("resnet18", clients, None, bpc)
    enc, outs = gpu_batch_encode("resnet18", clients, None, bpc, 0, torch, B)
    check_against_oracle(enc, outs, ref)
    decode_both(outs, [r[2] for r in ref], W.client_weights(w)[clients], w.d, torch, B)


def test_resnet18_all_100_clients_as_benchmarked(env):
    """the benchmark's step: plan + encode of 100 clients at 2 bits per coordinate in one call, the length tuning on
    a side stream, with the benchmark's reduced candidate workspace, then one decode-aggregate with sample-count
    weights"""
    torch, B = env
    w = W.WORKLOADS["resnet18"]
    clients = list(range(w.n_clients))
    ref = oracle_encode_clients("resnet18", clients, None, 2.0)
    budget = int(2.0 * w.d)
    max_cand = 3 * (budget // 12000) * ((12000 - 80) // (24 + 1))
    enc, outs = gpu_batch_encode("resnet18", clients, None, 2.0, max_cand, torch, B)
    check_against_oracle(enc, outs, ref)
    decode_both(outs, [r[2] for r in ref], W.client_weights(w), w.d, torch, B)


def test_resnet18_qsgd_three_clients(env):
    """the second quantizer of the paper's experiments at the benchmark's size and budget"""
    torch, B = env
    w = W.WORKLOADS["resnet18"]
    clients = [0, 31, 99]
    ref = oracle_encode_clients("resnet18", clients, None, 2.0, quantizer=1)
    enc, outs = gpu_batch_encode("resnet18", clients, None, 2.0, 0, torch, B, quantizer=1)
    check_against_oracle(enc, outs, ref)
    assert enc.read_plan(0).n_y[1] == 0
    decode_both(outs, [r[2] for r in ref], W.client_weights(w)[clients], w.d, torch, B)


def test_resnet50_ties_and_zero_blocks(env):
    torch, B = env
    w = W.WORKLOADS["resnet50"]
    clients = [0, 1, 2]
    ref = oracle_encode_clients("resnet50", clients, None, 1.0)
    enc, outs = gpu_batch_encode("resnet50", clients, None, 1.0, 0, torch, B)
    check_against_oracle(enc, outs, ref)
    decode_both(outs, [r[2] for r in ref], W.client_weights(w)[clients], w.d, torch, B)


def test_stress_1e8_in_accumulate_batches(env):
    torch, B = env
    w = W.WORKLOADS["stress"]
    clients = [0, 1, 2]
    ref = oracle_encode_clients("stress", clients, None, 0.25, procs=3)
    budget = int(0.25 * w.d)
    max_cand = 3 * (budget // 12000) * ((12000 - 80) // (27 + 1))
    enc, outs = gpu_batch_encode("stress", clients, None, 0.25, max_cand, torch, B)
    check_against_oracle(enc, outs, ref)
    lengths = {y for y in range(33) if enc.read_plan(0).n_y[y]}
    assert enc.read_plan(0).k < w.d // 100 and len(lengths) >= 2        # mostly 0-bit (sparsified) coordinates
    decode_both(outs, [r[2] for r in ref], W.client_weights(w)[clients], w.d, torch, B, batches=2)


def test_decode_windows_with_a_ragged_last_window(env):
    # d just above one accumulator window and not a multiple of 4: two windows, the second 1031 coordinates
    # short of the first and ending on a scalar tail; first call overwrites, second accumulates
    torch, B = env
    w = W.WORKLOADS["stress"]
    d = (24 << 20) + 1031
    clients = [0, 1]
    ref = oracle_encode_clients("stress", clients, d, 0.25, procs=2)
    enc, outs = gpu_batch_encode("stress", clients, d, 0.25, 0, torch, B)
    check_against_oracle(enc, outs, ref)
    decode_both(outs, [r[2] for r in ref], np.array([1.0, 3.0], dtype=np.float32), d, torch, B, batches=2)


def test_resnet18_unframed_and_error_compensation_two_clients(env):
    """the unframed writer and the error-compensation residual at the benchmark's size and budget"""
    torch, B = env
    dev = torch.device("cuda:0")
    w = W.WORKLOADS["resnet18"]
    clients = [3, 77]
    xs = [W.client_update(w, c) for c in clients]
    pds = [params_dict(w.d, 2 * w.d, seed=W.philox_ids(w, c)[0], client_id=W.philox_ids(w, c)[1]) for c in clients]
    params = [gpu_params(pd) for pd in pds]
    from gpu_util import oracle_params
    plans = [O.plan(x, oracle_params(pd)) for x, pd in zip(xs, pds)]
    # unframed streams, byte for byte, and the aggregate they decode to
    enc = B.BatchEncoder(params, dev)
    dxs = [torch.from_numpy(x).to(dev) for x in xs]
    enc.plan(dxs)
    cap = B.cvlc_unframed_stream_capacity(params[0])
    outs = [torch.zeros(cap, dtype=torch.uint8, device=dev) for _ in clients]
    sizes = torch.zeros(len(clients), dtype=torch.int64, device=dev)
    uf_ws = B.alloc_bytes(B.cvlc_unframed_workspace_bytes(params[0], len(clients)), dev)
    B.cvlc_encode_unframed_batch(dxs, params, enc.plans, outs, sizes, enc.enc_ws, uf_ws, plan_ws=enc.plan_ws)
    assert enc.status() == B.CVLC_OK
    refs = [O.encode_unframed(x, oracle_params(pd), pl) for x, pd, pl in zip(xs, pds, plans)]
    for i, ref in enumerate(refs):
        n = int(sizes[i].item())
        assert n == ref.size and (outs[i][:n].cpu().numpy() == ref).all(), i
    ptrs = torch.tensor([o.data_ptr() for o in outs], dtype=torch.int64, device=dev)
    wts = torch.tensor([1.0, 3.0], dtype=torch.float32, device=dev)
    dws = B.alloc_bytes(B.cvlc_decode_workspace_bytes(2), dev)
    agg = torch.empty(w.d, dtype=torch.float32, device=dev)
    B.cvlc_decode_aggregate_unframed(ptrs, sizes, wts, 2, 0.0, w.d, agg, False, dws)
    assert B.cvlc_read_status(dws) == B.CVLC_OK
    assert_aggregate_close(agg.cpu().numpy(), O.decode_aggregate_unframed(refs, np.array([1.0, 3.0], np.float32), w.d))
    # error compensation: the framed streams are unchanged, the inputs become the memories
    mems = [torch.from_numpy(x).to(dev) for x in xs]
    enc.plan(mems)
    B.cvlc_encode_batch_ec(mems, params, enc.plans, enc.outs, enc.enc_ws, plan_ws=enc.plan_ws)
    assert enc.status() == B.CVLC_OK
    for i, (x, pd, pl) in enumerate(zip(xs, pds, plans)):
        st = O.encode(x, oracle_params(pd), pl)
        assert (enc.outs[i].cpu().numpy() == st).all(), i
        want = O.ec_residual(x, st)
        assert (mems[i].cpu().numpy().view(np.uint32) == want.view(np.uint32)).all(), i
