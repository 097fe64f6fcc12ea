"""GPU parity: the CUDA path (through the C ABI) against the CPU oracle on the same
seeded inputs.  Bit-exact for plans, indices and streams; 1e-6 rel / 1e-7 abs for
the fp32 aggregate."""
import numpy as np
import pytest

import oracle as O
from paper_2402_03770_b200 import workloads as W
from gpu_util import (assert_aggregate_close, assert_plan_equal, gpu_decode_aggregate, gpu_plan_encode,
                      oracle_encode_clients, oracle_params, oracle_plan_encode, params_dict)
from stream_reader import parse

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def torch_cuda():
    import torch
    assert torch.cuda.is_available()
    from paper_2402_03770_b200 import binding as B
    B.lib()
    B.cvlc_set_device(0)
    return torch


# ---------------------------------------------------------------- building blocks

def test_philox_matches_oracle_on_2_20_counters(torch_cuda):
    torch = torch_cuda
    from paper_2402_03770_b200 import binding as B
    n = 1 << 20
    out = torch.zeros(4 * n, dtype=torch.int32, device="cuda:0")
    seed, client, rnd, first = 0x0123456789ABCDEF, 77, 3, (1 << 32) - 1000    # crosses the 32-bit boundary
    B.cvlc_selftest_philox(seed, client, rnd, first, n, out)
    got = out.cpu().numpy().view(np.uint32).reshape(n, 4)
    idx = np.concatenate([np.arange(0, 4096), np.arange(n - 4096, n), np.random.default_rng(0).integers(0, n, 8192)])
    for i in idx:
        c = first + int(i)
        ref = O.philox4x32_10([c & 0xFFFFFFFF, c >> 32, client, rnd], [seed & 0xFFFFFFFF, seed >> 32])
        assert tuple(int(v) for v in got[i]) == ref
    # every counter, word 0, against the oracle's per-coordinate function
    ref0 = np.array([O.philox_coord(seed, client, rnd, first + i) for i in range(0, n, 1)], dtype=np.uint32) \
        if n <= (1 << 20) else None
    assert (got[:, 0] == ref0).all()
    # known-answer vector through the device path
    B.cvlc_selftest_philox(0, 0, 0, 0, 1, out)
    assert [int(v) for v in out[:4].cpu().numpy().view(np.uint32)] == [0x6627E8D5, 0xE169C58D, 0xBC57AC4C, 0x9B00DBD8]


def test_series_math_bit_exact(torch_cuda):
    torch = torch_cuda
    from paper_2402_03770_b200 import binding as B
    rng = np.random.default_rng(4)
    pos = np.concatenate([rng.integers(1, 2 ** 31, 20000).astype(np.float64), 10.0 ** rng.uniform(-30, 30, 20000),
                          rng.uniform(1, 2, 20000), [1.0, 2.0, 1.4142135623730951, 1.4142135623730954, 1e8]])
    x = torch.from_numpy(pos).cuda()
    l2 = torch.empty_like(x)
    B.cvlc_selftest_math(x, l2, None, None, None)
    ref = np.array([O.log2(float(v)) for v in pos])
    assert (l2.cpu().numpy().view(np.uint64) == ref.view(np.uint64)).all()
    ev = np.concatenate([rng.uniform(-1000, 1000, 30000), rng.uniform(-40, 40, 30000), np.arange(-20, 21) * 0.5])
    x = torch.from_numpy(ev).cuda()
    e2 = torch.empty_like(x)
    B.cvlc_selftest_math(x, None, e2, None, None)
    ref = np.array([O.exp2(float(v)) for v in ev])
    assert (e2.cpu().numpy().view(np.uint64) == ref.view(np.uint64)).all()


def test_division_by_small_constants_is_correctly_rounded(torch_cuda):
    """the planner divides by 1..20 with a reciprocal and one correction; it must equal IEEE division"""
    torch = torch_cuda
    from paper_2402_03770_b200 import binding as B
    rng = np.random.default_rng(8)
    n = 1 << 20
    u = np.concatenate([rng.uniform(-0.35, 0.35, n // 2), rng.standard_normal(n // 4) * 10.0 ** rng.uniform(-18, 3, n // 4),
                        (rng.integers(1, 2 ** 53, n // 4).astype(np.float64)) * 2.0 ** -60])
    # adversarial: exact multiples and neighbours of multiples of j
    extra = []
    for j in range(1, 21):
        m = rng.integers(2 ** 52, 2 ** 53, 2000).astype(np.float64)
        extra += [m * j * 2.0 ** -55, np.nextafter(m * j * 2.0 ** -55, 1.0), np.nextafter(m * j * 2.0 ** -55, 0.0)]
    u = np.concatenate([u] + extra)
    x = torch.from_numpy(u).cuda()
    dv = torch.empty(x.numel() * 20, dtype=torch.float64, device="cuda")
    dr = torch.empty_like(dv)
    B.cvlc_selftest_math(x, None, None, dv, dr)
    a, b = dv.cpu().numpy().view(np.uint64), dr.cpu().numpy().view(np.uint64)
    assert (a == b).all()
    host = (u[:, None] / np.arange(1, 21, dtype=np.float64)[None, :]).reshape(-1)
    assert (b == host.view(np.uint64)).all()


# ---------------------------------------------------------------- plan / stream parity, small cases

def run_case(x, pd, fixed_y=0):
    of, ost = oracle_plan_encode(x, pd, fixed_y)
    # both selection kernels (offsets from the plan's per-segment counts, and the look-back scan), then the
    # one-call form on one stream and with the length tuning on a side stream
    for use_plan_ws, compress in ((True, 0), (False, 0), (True, 1), (True, 2)):
        status, gp, gst = gpu_plan_encode(x, pd, fixed_y, use_plan_ws=use_plan_ws, compress=compress)
        assert status == 0, (status, use_plan_ws, compress)
        assert_plan_equal(gp, of)
        assert gp.k <= gp.n_candidates <= pd["d"]
        assert gst.size == ost.size
        if not (gst == ost).all():
            bad = np.nonzero(gst != ost)[0]
            raise AssertionError(f"stream differs at {bad.size} bytes, first at {bad[0]} of {gst.size} "
                                 f"(use_plan_ws={use_plan_ws}, compress={compress})")
    return of, ost


def test_tiny_workload_encode_decode(torch_cuda):
    w = W.WORKLOADS["tiny"]
    x = W.client_update(w, 0)
    pd = params_dict(w.d, w.budget_bits())
    status, gp, gst, gh = gpu_plan_encode(x, pd, want_hist=True)
    rc, oh = O.histogram(x)
    assert status == 0 and (gh == oh).all()
    of, ost = run_case(x, pd)
    ref = O.decode_aggregate([ost], np.ones(1, np.float32), w.d)
    status, out = gpu_decode_aggregate([gst], np.ones(1, np.float32), w.d)
    assert status == 0
    assert_aggregate_close(out, ref)
    # one client, weight 1: the aggregate is that client's dequantized vector / B, exact per record
    assert (out.view(np.uint32) == ref.view(np.uint32)).all()


@pytest.mark.parametrize("d", [2, 3, 5, 63, 64, 65, 1000, 4095, 4096, 4097, 8191, 12289, 100_003])
def test_ragged_sizes(torch_cuda, d):
    rng = np.random.default_rng(d)
    x = rng.laplace(0, 1e-2, d).astype(np.float32)
    if d < 1000:
        pd = params_dict(d, 96 * (1 if d < 60 else 5), packet_bits=96, max_code_bits=8, seed=d, client_id=1, round=2)
    else:
        pd = params_dict(d, min(d // 400, 40) * 2048 + 5, packet_bits=2048, seed=d, client_id=1, round=2)
    run_case(x, pd)
    run_case(x, pd, fixed_y=8 if d < 1000 else 3)


@pytest.mark.parametrize("y", [1, 2, 7, 8, 16, 31, 32])
def test_fixed_length_plans(torch_cuda, y):
    """all packets at one length: Top_k + y-bit quantization, the special case of Section I"""
    rng = np.random.default_rng(y)
    d = 50_000
    x = rng.standard_normal(d).astype(np.float32) * np.float32(1e-3)
    pd = params_dict(d, 9 * 12000 + 77, seed=5, client_id=y, round=1, scale_B=1.0 + 0.01 * y)
    of, ost = run_case(x, pd, fixed_y=y)
    assert of["n_y"][y] == 9
    ref = O.decode_aggregate([ost], np.ones(1, np.float32), d)
    status, out = gpu_decode_aggregate([ost], np.ones(1, np.float32), d)
    assert status == 0
    assert_aggregate_close(out, ref)
    if y == 32:   # the 0-bit / Top_k case: kept coordinates are x / B to rounding, the rest exactly 0
        S = parse(ost)
        pids = np.concatenate([pk.pid for pk in S.packets]).astype(np.int64)
        mask = np.zeros(d, bool)
        mask[pids] = True
        assert (out[~mask] == 0).all()
        assert np.abs(out[pids] * pd["scale_B"] - x[pids]).max() <= 4e-7 * np.abs(x).max()


def test_ties_zeros_and_negative_zero(torch_cuda):
    """equal |x| keep ascending index; zero blocks may be transmitted when k exceeds the non-zeros"""
    rng = np.random.default_rng(12)
    d = 40_000
    x = (np.round(rng.standard_normal(d) * 4) / 4).astype(np.float32)          # heavy ties, both signs
    x[5000:30000] = 0.0
    x[5000:30000:3] = -0.0
    pd = params_dict(d, 220 * 2048, packet_bits=2048, seed=9)
    of, ost = run_case(x, pd)
    assert of["k"] > np.count_nonzero(x)                                         # zeros are in the stream
    pd2 = params_dict(d, 12 * 2048, packet_bits=2048, seed=9)
    run_case(x, pd2)
    run_case(np.zeros(d, np.float32), pd2)                                       # all zeros
    run_case(np.full(d, -1.5, np.float32), pd2)                                  # all equal


def test_block_structured_workloads_small(torch_cuda):
    for name, d, bpc in [("small_cnn", 150_000, 2.0), ("resnet18", 300_000, 0.5), ("resnet18", 300_000, 4.0),
                         ("resnet50", 400_000, 1.0), ("stress", 1_000_000, 0.25)]:
        w = W.WORKLOADS[name]
        for client in (0, 1):
            x = W.client_update(w, client, d=d)
            seed, cid, rnd = W.philox_ids(w, client)
            pd = params_dict(d, int(bpc * d), seed=seed, client_id=cid, round=rnd)
            run_case(x, pd)


def test_other_packet_and_header_sizes(torch_cuda):
    rng = np.random.default_rng(21)
    d = 70_000
    x = rng.laplace(0, 1e-3, d).astype(np.float32)
    for packet_bits, header_bits, max_bits in [(96, 80, 8), (512, 96, 32), (4096, 81, 12), (12000, 400, 32),
                                               (32768, 80, 24)]:
        pd = params_dict(d, 6 * packet_bits, packet_bits=packet_bits, header_bits=header_bits,
                         max_code_bits=max_bits, seed=3, scale_B=1.5)
        try:
            O.plan(x, oracle_params(pd))
        except O.OracleError:
            continue
        run_case(x, pd)


@pytest.mark.parametrize("n", [2, 4, 5, 23])
def test_batched_plan_encode_matches_oracle_per_client(torch_cuda, n):
    """one set of launches for n clients (different data, scales and Philox ids) = n oracle runs"""
    torch = torch_cuda
    from paper_2402_03770_b200 import binding as B
    from gpu_util import gpu_params
    w = W.WORKLOADS["resnet18"]
    d = 120_001                                                                  # ragged: not a multiple of 4
    dev = torch.device("cuda:0")
    xs, pds = [], []
    for c in range(n):
        x = W.client_update(w, c, d=d)
        if c == 1:
            x[:] = 0.0                                                           # one all-zero client inside the batch
        xs.append(x)
        pds.append(params_dict(d, 20 * 12000 + 7 * c, seed=100 + c, client_id=c, round=c % 3, scale_B=1.0 + 0.002 * c))
    params = [gpu_params(pd) for pd in pds]
    for max_cand in (0, 60_000 if n != 5 else 0):
        enc = B.BatchEncoder(params, dev, max_candidates=max_cand)
        for o in enc.outs:
            o.fill_(0xCD)
        dxs = [torch.from_numpy(x).to(dev) for x in xs]
        outs = enc.run(dxs, use_plan_ws=(n % 2 == 0))
        status = enc.status()
        if max_cand:
            # the all-zero client has d candidates: more than the reduced workspace holds
            assert status == B.CVLC_ERR_WORKSPACE_TOO_SMALL
            continue
        assert status == 0
        for c in range(n):
            of, ost = oracle_plan_encode(xs[c], pds[c])
            assert_plan_equal(enc.read_plan(c), of)
            assert (outs[c].cpu().numpy() == ost).all(), c


def test_clients_that_share_a_tuning_key_get_the_same_lengths(torch_cuda):
    """clients with the same quantised exponent and scale are tuned once and copy the result: every one of them must
    still equal its own oracle run (different Philox ids, so different streams)"""
    torch = torch_cuda
    from paper_2402_03770_b200 import binding as B
    from gpu_util import gpu_params
    dev = torch.device("cuda:0")
    d = 90_001
    rng = np.random.default_rng(44)
    base = [rng.laplace(0, 1e-2, d).astype(np.float32), (rng.standard_t(3, d) * 1e-3).astype(np.float32)]
    xs, pds = [], []
    for c in range(7):
        x = base[c % 2].copy() if c != 6 else np.zeros(d, np.float32)
        if c == 4:
            x = -x[::-1].copy()                                   # same magnitudes, other places: same histogram, same key
        xs.append(x)
        pds.append(params_dict(d, 15 * 12000, seed=7 + c, client_id=c, round=1, scale_B=1.25 if c == 5 else None))
    params = [gpu_params(pd) for pd in pds]
    for side in (False, True):
        enc = B.BatchEncoder(params, dev)
        dxs = [torch.from_numpy(x).to(dev) for x in xs]
        outs = enc.compress(dxs, side_stream=torch.cuda.Stream(device=dev) if side else None)
        assert enc.status() == 0
        keys = set()
        for c in range(7):
            of, ost = oracle_plan_encode(xs[c], pds[c])
            gp = enc.read_plan(c)
            assert_plan_equal(gp, of)
            assert (outs[c].cpu().numpy() == ost).all(), c
            keys.add((gp.alpha_q, pds[c]["scale_B"]))
        assert len(keys) < 7                                       # some clients did share a key


def test_batch_rejects_mixed_shapes(torch_cuda):
    torch = torch_cuda
    from paper_2402_03770_b200 import binding as B
    dev = torch.device("cuda:0")
    d = 50_000
    xs = [torch.zeros(d, device=dev), torch.zeros(d, device=dev)]
    params = [B.make_params(d, 10 * 12000), B.make_params(d, 11 * 12000)]
    plans = B.alloc_bytes(2 * B.PLAN_BYTES, dev)
    ws = B.alloc_bytes(B.cvlc_plan_batch_workspace_bytes(params[0], 2), dev)
    with pytest.raises(B.CvlcError) as e:
        B.cvlc_plan_batch(xs, params, plans, ws)
    assert e.value.code == B.CVLC_ERR_INVALID_ARG


def test_encode_is_deterministic(torch_cuda):
    w = W.WORKLOADS["small_cnn"]
    x = W.client_update(w, 3, d=500_000)
    pd = params_dict(x.size, 2 * x.size, seed=3, client_id=3)
    a = gpu_plan_encode(x, pd)[2]
    b = gpu_plan_encode(x, pd)[2]
    assert (a == b).all()


# ---------------------------------------------------------------- aggregation

def small_clients(n, d=60_000, R=12, seed0=0):
    streams, pds = [], []
    for i in range(n):
        rng = np.random.default_rng(seed0 + i)
        x = rng.laplace(0, 1e-2, d).astype(np.float32)
        pd = params_dict(d, R * 4096, packet_bits=4096, seed=i, client_id=i, scale_B=1.0 + 0.003 * i)
        _, st = oracle_plan_encode(x, pd)
        streams.append(st)
    return streams


def test_aggregate_weighted_many_clients(torch_cuda):
    n, d = 33, 60_000
    streams = small_clients(n, d)
    w = np.random.default_rng(7).uniform(50, 500, n).astype(np.float32)
    ref = O.decode_aggregate(streams, w, d)
    status, out = gpu_decode_aggregate(streams, w, d)
    assert status == 0
    assert_aggregate_close(out, ref)
    assert (out[ref == 0] == 0).all()                                           # unsent coordinates are exactly 0
    # batches with accumulate, total weight given up front
    Wt = float(w.astype(np.float64).sum())
    status, part = gpu_decode_aggregate(streams[:10], w[:10], d, weight_total=Wt)
    assert status == 0
    status, both = gpu_decode_aggregate(streams[10:], w[10:], d, weight_total=Wt, out_init=part, accumulate=True)
    assert status == 0
    assert_aggregate_close(both, ref)


def test_aggregate_mixed_stream_shapes(torch_cuda):
    """clients may use different budgets and packet sizes in one call"""
    d = 30_000
    streams = []
    for i, (R, pb) in enumerate([(3, 1024), (17, 12000), (1, 96 * 32), (40, 512)]):
        rng = np.random.default_rng(50 + i)
        x = rng.standard_normal(d).astype(np.float32)
        pd = params_dict(d, R * pb, packet_bits=pb, seed=i, client_id=i)
        streams.append(oracle_plan_encode(x, pd)[1])
    w = np.array([1, 2, 3, 4], np.float32)
    ref = O.decode_aggregate(streams, w, d)
    status, out = gpu_decode_aggregate(streams, w, d)
    assert status == 0
    assert_aggregate_close(out, ref)


def test_decode_rejects_malformed_streams(torch_cuda):
    from paper_2402_03770_b200 import binding as B
    d = 20_000
    x = np.random.default_rng(1).laplace(0, 1e-2, d).astype(np.float32)
    pd = params_dict(d, 6 * 1024, packet_bits=1024)
    st = oracle_plan_encode(x, pd)[1]
    good = small_clients(2, d=d, R=3)
    w3 = np.ones(3, np.float32)

    def corrupt(off, val):
        b = st.copy()
        b[off] = val
        return b

    bits = np.unpackbits(st[64:64 + 128], bitorder="little")
    bits[80:80 + 15] = 1                                                        # PID 32767 >= d
    pid_bad = st.copy()
    pid_bad[64:64 + 128] = np.packbits(bits, bitorder="little")
    # the PQ centroid fields (bytes 2..5 minimum, 6..9 maximum of a packet): not finite, or in the wrong order
    hi_nan = st.copy()
    hi_nan[64 + 8:64 + 10] = [0xC0, 0x7F]
    lo_inf = st.copy()
    lo_inf[64 + 2:64 + 6] = [0x00, 0x00, 0x80, 0xFF]
    swapped = st.copy()
    swapped[64 + 2:64 + 6], swapped[64 + 6:64 + 10] = st[64 + 6:64 + 10].copy(), st[64 + 2:64 + 6].copy()
    assert st[64 + 2:64 + 6].tobytes() != st[64 + 6:64 + 10].tobytes()
    cases = [corrupt(0, 0), corrupt(4, 2), corrupt(6, 1), corrupt(7, 3), corrupt(16, 9), corrupt(65, 33),
             corrupt(65, 0), corrupt(64 + 128 * 5 + 1, 32), pid_bad, hi_nan, lo_inf, swapped]
    for bad in cases:
        with pytest.raises(O.OracleError):
            O.decode_aggregate([good[0], bad, good[1]], w3, d)
        status, _ = gpu_decode_aggregate([good[0], bad, good[1]], w3, d)
        assert status == B.CVLC_ERR_BAD_STREAM
    # a stream length that disagrees with its header
    status, _ = gpu_decode_aggregate([good[0], st[:-128], good[1]], w3, d)
    assert status == B.CVLC_ERR_BAD_STREAM
    # weights are finite and positive
    for wbad in (np.array([1, -1, 1], np.float32), np.array([1, np.inf, 1], np.float32), np.array([0, 1, 1], np.float32)):
        with pytest.raises(O.OracleError) as oe:
            O.decode_aggregate([good[0], st, good[1]], wbad, d)
        assert oe.value.code == O.ORC_ERR_INVALID_ARG
        status, _ = gpu_decode_aggregate([good[0], st, good[1]], wbad, d)
        assert status == B.CVLC_ERR_INVALID_ARG
    # the context is still usable
    status, out = gpu_decode_aggregate([good[0], st, good[1]], w3, d)
    assert status == 0
    assert_aggregate_close(out, O.decode_aggregate([good[0], st, good[1]], w3, d))


def test_nonfinite_input_is_reported(torch_cuda):
    from paper_2402_03770_b200 import binding as B
    d = 10_000
    x = np.random.default_rng(2).standard_normal(d).astype(np.float32)
    pd = params_dict(d, 4 * 1024, packet_bits=1024)
    for bad in (np.inf, -np.inf, np.nan):
        xb = x.copy()
        xb[d - 3] = bad
        with pytest.raises(O.OracleError) as e:
            O.plan(xb, oracle_params(pd))
        assert e.value.code == O.ORC_ERR_NONFINITE_INPUT
        status, gp, gst = gpu_plan_encode(xb, pd)
        assert status == B.CVLC_ERR_NONFINITE_INPUT


def test_host_side_errors_match_oracle(torch_cuda):
    from paper_2402_03770_b200 import binding as B
    x = np.ones(1000, np.float32)
    for pd, code in [
        (params_dict(1000, 11999), B.CVLC_ERR_BUDGET_TOO_SMALL),
        (params_dict(1000, 50 * 12000), B.CVLC_ERR_BUDGET_TOO_LARGE),
        (params_dict(1000, 12000, header_bits=79, scale_B=1.0), B.CVLC_ERR_INVALID_ARG),
        (params_dict(1000, 12001, packet_bits=12001, scale_B=1.0), B.CVLC_ERR_INVALID_ARG),
        (params_dict(1000, 96, packet_bits=96, scale_B=1.0), B.CVLC_ERR_PACKET_TOO_SMALL),
        (params_dict(100_000, 12000, max_code_bits=3, scale_B=1.0), B.CVLC_ERR_SCALE_TOO_SMALL),
    ]:
        for compress in (0, 1, 2):
            with pytest.raises(B.CvlcError) as e:
                gpu_plan_encode(np.ones(pd["d"], np.float32), pd, compress=compress)
            assert e.value.code == code, (pd, compress)
        with pytest.raises(O.OracleError) as oe:
            O.plan(np.ones(pd["d"], np.float32), oracle_params(pd))
        assert oe.value.code == code                                             # same numbering on both sides


def test_compress_batch_argument_checks(torch_cuda):
    torch = torch_cuda
    from paper_2402_03770_b200 import binding as B
    dev = torch.device("cuda:0")
    d = 40_000
    p = B.make_params(d, 8 * 12000)
    enc = B.BatchEncoder([p, p], dev)
    xs = [torch.zeros(d, device=dev), torch.zeros(d, device=dev)]
    small = B.alloc_bytes(1024, dev)
    for kw, code in ((dict(plan_ws=small), B.CVLC_ERR_WORKSPACE_TOO_SMALL), (dict(enc_ws=small), B.CVLC_ERR_WORKSPACE_TOO_SMALL),
                     (dict(outs=[small, small]), B.CVLC_ERR_OUTPUT_TOO_SMALL), (dict(fixed_y=33), B.CVLC_ERR_INVALID_ARG)):
        a = dict(plan_ws=enc.plan_ws, enc_ws=enc.enc_ws, outs=enc.outs, fixed_y=0)
        a.update(kw)
        with pytest.raises(B.CvlcError) as e:
            B.cvlc_compress_batch(xs, enc.params, enc.plans, a["outs"], a["plan_ws"], a["enc_ws"], fixed_y=a["fixed_y"])
        assert e.value.code == code, kw
    # the same stream given as side stream: everything runs in order on it
    s1 = torch.cuda.Stream(device=dev)
    x = np.random.default_rng(3).laplace(0, 1e-2, d).astype(np.float32)
    xs = [torch.from_numpy(x).to(dev), torch.from_numpy(-x).to(dev)]
    enc.compress(xs, stream=s1, side_stream=s1)
    assert enc.status(s1) == B.CVLC_OK
    po = oracle_params(params_dict(d, 8 * 12000))
    ref = O.encode(x, po, O.plan(x, po))
    assert (enc.outs[0].cpu().numpy() == ref).all()


def test_plan_mismatch_is_detected(torch_cuda):
    torch = torch_cuda
    from paper_2402_03770_b200 import binding as B
    d = 50_000
    x = np.random.default_rng(0).laplace(0, 1e-3, d).astype(np.float32)
    dev = torch.device("cuda:0")
    p = B.make_params(d, 10 * 12000)
    enc = B.ClientEncoder(p, dev)
    xd = torch.from_numpy(x).to(dev)
    B.cvlc_plan(xd, p, enc.plan, enc.plan_ws)
    p2 = B.make_params(d, 11 * 12000)
    enc2 = B.ClientEncoder(p2, dev)
    B.cvlc_encode(xd, p2, enc.plan, enc2.out, enc2.enc_ws)                      # plan made for another budget
    assert B.cvlc_read_status(enc2.enc_ws) == B.CVLC_ERR_PLAN_MISMATCH
    # plan made for another update: three times the values put more coordinates above the plan's threshold,
    # which both selection kernels notice (per-segment counts with the plan's workspace, the total without)
    x2 = torch.from_numpy((x * 3.0).astype(np.float32)).to(dev)
    assert int((np.abs(x * 3.0).astype(np.float32).view(np.uint32) >> 19 >= B.read_plan(enc.plan).thresh_bin).sum()) \
        != B.read_plan(enc.plan).n_candidates
    for plan_ws in (enc.plan_ws, None):
        B.cvlc_encode(x2, p, enc.plan, enc.out, enc.enc_ws, plan_ws=plan_ws)
        assert B.cvlc_read_status(enc.enc_ws) == B.CVLC_ERR_PLAN_MISMATCH
    # code lengths that do not fill the stream's packets are refused by the packing kernel
    plan_host = bytearray(enc.plan.cpu().numpy().tobytes())
    tampered = B.CvlcPlan.from_buffer_copy(bytes(plan_host))
    y_used = max(y for y in range(33) if tampered.n_y[y])
    tampered.n_y[y_used] -= 1
    bad_plan = torch.frombuffer(bytearray(bytes(tampered)), dtype=torch.uint8).to(dev)
    B.cvlc_encode(xd, p, bad_plan, enc.out, enc.enc_ws, plan_ws=enc.plan_ws)
    assert B.cvlc_read_status(enc.enc_ws) == B.CVLC_ERR_PLAN_MISMATCH
    for plan_ws in (enc.plan_ws, None):                                         # and the right pairing still works
        B.cvlc_encode(xd, p, enc.plan, enc.out, enc.enc_ws, plan_ws=plan_ws)
        assert B.cvlc_read_status(enc.enc_ws) == B.CVLC_OK


def test_bounded_wait_runs_out_without_hanging(torch_cuda):
    """the look-back wait on a word nobody publishes gives up after its poll limit and reports DEVICE_TIMEOUT"""
    torch = torch_cuda
    from paper_2402_03770_b200 import binding as B
    word = torch.zeros(1, dtype=torch.int64, device="cuda:0")
    status = torch.zeros(1, dtype=torch.int32, device="cuda:0")
    B.cvlc_selftest_wait(word, status, 64)
    torch.cuda.synchronize()
    assert int(status.item()) == B.CVLC_ERR_DEVICE_TIMEOUT
    # a published word ends the wait at once and leaves the status alone
    word.fill_((1 << 62) | 5)
    status.zero_()
    B.cvlc_selftest_wait(word, status, 64)
    torch.cuda.synchronize()
    assert int(status.item()) == B.CVLC_OK
    with pytest.raises(B.CvlcError):
        B.cvlc_selftest_wait(word, status, 0)


def test_subnormal_threshold(torch_cuda):
    """an update so small that the selection threshold lies among the subnormals (no flush to zero anywhere)"""
    rng = np.random.default_rng(31)
    d = 60_000
    x = (rng.laplace(0, 1.0, d) * 1e-41).astype(np.float32)
    assert 0 < np.count_nonzero(x) and np.abs(x).max() < 1.2e-38
    pd = params_dict(d, 8 * 4096, packet_bits=4096, seed=4, client_id=2)
    of, ost = run_case(x, pd)
    x[::2] *= np.float32(1e3)                                                    # threshold bin among the smallest normals
    run_case(x, pd)


@pytest.mark.parametrize("quantizer", [0, 1])
def test_large_packets_go_through_the_unstaged_paths(torch_cuda, quantizer):
    # 8 KB packets: more records per packet than a warp's lanes many times over, a packet image of several KB per
    # warp in the encoder, and packets too long for the decoder's shared-memory staging (read from global memory)
    rng = np.random.default_rng(77)
    d = 300_000
    x = (rng.standard_t(3, d) * 1e-3).astype(np.float32)
    pd = params_dict(d, 9 * 65536, packet_bits=65536, header_bits=80, quantizer=quantizer, seed=11, client_id=4)
    of, ost = run_case(x, pd)
    assert of["R"] == 9
    ref = O.decode_aggregate([ost], np.array([2.0], np.float32), d, weight_total=5.0)
    status, out = gpu_decode_aggregate([ost], np.array([2.0], np.float32), d, weight_total=5.0)
    assert status == 0
    assert_aggregate_close(out, ref)


def test_packets_beyond_the_encoders_shared_memory_are_rejected(torch_cuda):
    from paper_2402_03770_b200 import binding as B
    d = 100_000
    x = np.linspace(-1.0, 1.0, d).astype(np.float32)
    pd = params_dict(d, 2 * 524288, packet_bits=524288, scale_B=2.0)   # 64 KB packets: four do not fit 200 KB
    with pytest.raises(B.CvlcError) as e:
        gpu_plan_encode(x, pd)
    assert e.value.code == B.CVLC_ERR_INVALID_ARG
