"""The largest problem the interface admits: d = 2^31 coordinates (31-bit position IDs, an 8.6 GB update and
an 8.6 GB aggregate filled in 86 windows).

The oracle's encoder ranks by sorting all d coordinates, which would take hours here, so this size is checked
piece by piece against what the oracle can compute one value at a time: the plan against the oracle's planner
run on the histogram (known by construction: about two thousand non-zero coordinates, the rest zero), the
stream, read by the independent reader, record by record against the ranking (a sort of the non-zero
coordinates alone), the oracle's Philox word and quantizer of every transmitted value, and the aggregate
against the oracle's dequantizer."""
import numpy as np
import pytest

import oracle as O
import stream_reader as SR
from gpu_util import assert_plan_equal, gpu_params, oracle_params, params_dict

pytestmark = pytest.mark.gpu

D = 1 << 31


def test_d_2_pow_31_encode_and_decode():
    import torch
    from paper_2402_03770_b200 import binding as B
    assert torch.cuda.is_available()
    B.lib()
    B.cvlc_set_device(0)
    dev = torch.device("cuda:0")

    rng = np.random.default_rng(31)
    m = 2000
    pos = np.unique(np.concatenate([rng.integers(0, D, size=m - 8, dtype=np.int64),
                                    np.array([0, 1, 5, (1 << 30) - 1, 1 << 30, D - 6, D - 2, D - 1], dtype=np.int64)]))
    m = pos.size
    vals = (rng.uniform(1e-3, 1.0, size=m) * rng.choice([-1.0, 1.0], size=m)).astype(np.float32)
    vals[pos == D - 1] = np.float32(-3.5)        # the last coordinate ranks first
    vals[pos == 0] = np.float32(2.25)            # a tie in magnitude between the first coordinate ...
    vals[pos == D - 2] = np.float32(-2.25)       # ... and the last but one: the lower index ranks first
    keys = vals.view(np.uint32) & np.uint32(0x7FFFFFFF)

    pd = params_dict(D, 3 * 12000, seed=77, client_id=5, round=2)      # three packets
    po = oracle_params(pd)
    h = np.bincount((keys >> np.uint32(19)).astype(np.int64), minlength=4096).astype(np.uint64)
    h[0] += np.uint64(D - m)
    pl = O.plan_from_histogram(h, po)
    fields = dict(s=pl.s, R=pl.R, y_min=pl.y_min, n_lengths=pl.n_lengths, k=pl.k, alpha=pl.alpha, alpha_q=pl.alpha_q,
                  beta=pl.beta, gamma=pl.gamma, B_next=pl.B_next, n_y=[pl.n_y[y] for y in range(33)],
                  cap=[pl.cap[y] for y in range(33)])
    assert pl.s == 31 and pl.R == 3 and 0 < pl.k < m

    x = torch.zeros(D, dtype=torch.float32, device=dev)
    x[torch.from_numpy(pos).to(dev)] = torch.from_numpy(vals).to(dev)
    enc = B.BatchEncoder([gpu_params(pd)], dev, max_candidates=1 << 20)
    outs = enc.run([x])
    assert enc.status() == B.CVLC_OK
    del x
    assert_plan_equal(enc.read_plan(0), fields)

    # ranking of the non-zero coordinates: magnitude descending, ties by ascending index
    order = np.lexsort((pos, -keys.astype(np.int64)))
    st = SR.parse(outs[0].cpu().numpy())
    assert (st.s, st.d, st.R, st.k, st.client_id, st.seed, st.round) == (31, D, 3, pl.k, 5, 77, 2)
    lengths = [y for y in range(32, 0, -1) for _ in range(pl.n_y[y])]
    expected = {}
    z = 0
    for pk, y in zip(st.packets, lengths):
        P = pl.cap[y]
        sel = order[z:z + P]
        z += P
        assert pk.y == y and pk.s == 31 and pk.pad_bits_zero
        assert (pk.pid == pos[sel].astype(np.uint64)).all()
        lo, hi = float(vals[sel].min()), float(vals[sel].max())
        assert (pk.lo, pk.hi) == (lo, hi)
        for j, i in enumerate(sel):
            code = O.pq_quantize(float(vals[i]), lo, hi, y, O.philox_coord(77, 5, 2, int(pos[i])))
            assert int(pk.cid[j]) == code, (int(pos[i]), y, code, int(pk.cid[j]))
            expected[int(pos[i])] = O.pq_dequantize(code, lo, hi, y)
    assert z == pl.k

    # decode-aggregate: weight 1 of a total of 2, scale B of the stream
    agg = B.Aggregator(1, D, dev)
    agg.set_clients(outs, torch.ones(1))
    out = torch.full((D,), float("nan"), dtype=torch.float32, device=dev)
    agg.run(1, out, weight_total=2.0)
    assert agg.status() == B.CVLC_OK
    coef = np.float32(1.0 / (2.0 * st.scale_B))
    pids = np.array(sorted(expected), dtype=np.int64)
    want = np.array([np.float32(np.float64(coef) * np.float64(expected[int(p)])) for p in pids], dtype=np.float32)
    got = out[torch.from_numpy(pids).to(dev)].cpu().numpy()
    assert np.abs(got.astype(np.float64) - want) .max() <= 1e-7 + 1e-6 * np.abs(want).max()
    assert (np.abs(got.astype(np.float64) - want) <= 1e-7 + 1e-6 * np.abs(want)).all()
    assert int(torch.count_nonzero(out).item()) == int(np.count_nonzero(want))   # every other coordinate is exactly 0
