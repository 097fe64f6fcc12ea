"""Pins of the oracle's unframed stream (version 2): the records of every packet without the packet frame, positions
sorted and sent as Golomb-Rice coded differences.  It must carry exactly what the framed stream carries (same
positions per block, same centroid distribution, same centroid IDs), parse with a reader written from the format
alone, meet its own length bookkeeping, and decode to the identical aggregate."""
import numpy as np
import pytest

import oracle as O
from paper_2402_03770_b200 import workloads as W
from stream_reader import parse, parse_unframed
from test_oracle_codec import small_case


def both_streams(x, p, fixed_y=0):
    pl = O.plan_fixed(p, fixed_y) if fixed_y else O.plan(x, p)
    return pl, O.encode(x, p, pl), O.encode_unframed(x, p, pl)


@pytest.mark.parametrize("quantizer", [0, 1])
@pytest.mark.parametrize("d,R,pb", [(5000, 6, 1024), (60_000, 9, 4096), (300_000, 20, 12000)])
def test_same_records_as_the_framed_stream(d, R, pb, quantizer):
    x, p = small_case(d=d, R=R, packet_bits=pb, quantizer=quantizer)
    pl, framed, unframed = both_streams(x, p)
    F, U = parse(framed), parse_unframed(unframed)
    assert U.tail_zero and U.head.k == F.k == pl.k and U.head.R == F.R
    assert U.n_y == [pl.n_y[y] for y in range(33)] and U.cap[1:] == [pl.cap[y] for y in range(1, 33)]
    assert (U.head.scale_B, U.head.seed, U.head.client_id, U.head.round, U.head.quantizer) == \
           (F.scale_B, F.seed, F.client_id, F.round, F.quantizer)
    for fp, up in zip(F.packets, U.head.packets):
        assert up.y == fp.y and (up.lo, up.hi) == (fp.lo, fp.hi)
        order = np.argsort(fp.pid, kind="stable")
        assert (up.pid == fp.pid[order]).all() and (np.diff(up.pid.astype(np.int64)) > 0).all()
        assert (up.cid == fp.cid[order]).all()
    # length bookkeeping: header bits per block plus, per record, the unary part, the stop bit, m and y bits
    bits = 0
    for up in U.head.packets:
        m = max(0, (d // up.pid.size).bit_length() - 1)
        delta = np.diff(np.concatenate([[-1], up.pid.astype(np.int64)])) - 1
        bits += 64 + int((delta >> m).sum()) + up.pid.size * (1 + m + up.y)
    assert bits == U.total_bits
    assert unframed.size <= O.unframed_capacity(p)
    assert U.total_bits < 8 * (framed.size - 64)                        # the body shrinks (the table and the directory
                                                                        # in the header only pay off on longer streams)


@pytest.mark.parametrize("quantizer", [0, 1])
def test_decodes_to_the_same_aggregate(quantizer):
    d = 40_000
    framed, unframed = [], []
    for c in range(4):
        x, _ = small_case(d=d, R=8, seed=c)
        p = O.make_params(d, 8 * 2048 + c, packet_bits=2048, seed=c, client_id=c, round=1, quantizer=quantizer,
                          scale_B=None if c else 1.25)
        pl, f, u = both_streams(x, p)
        framed.append(f)
        unframed.append(u)
    w = np.array([1.0, 2.5, 0.5, 4.0], np.float32)
    a = O.decode_aggregate(framed, w, d)
    b = O.decode_aggregate_unframed(unframed, w, d)
    assert (a.view(np.uint32) == b.view(np.uint32)).all()
    half = O.decode_aggregate_unframed(unframed[:2], w[:2], d, weight_total=8.0)
    both = O.decode_aggregate_unframed(unframed[2:], w[2:], d, weight_total=8.0, out=half.copy(), accumulate=True)
    assert np.abs(both.astype(np.float64) - a).max() <= 1e-7 + 1e-6 * np.abs(a).max()


def test_sparse_and_dense_gaps():
    """few records in a long vector (long unary runs, large Rice parameter) and nearly every coordinate sent (m = 0)"""
    rng = np.random.default_rng(9)
    x = rng.standard_normal(3_000_000).astype(np.float32)
    p = O.make_params(x.size, 2 * 1024, packet_bits=1024)
    pl, f, u = both_streams(x, p, fixed_y=8)
    U = parse_unframed(u)
    assert sorted(np.concatenate([pk.pid for pk in U.head.packets]).tolist()) == \
           sorted(np.concatenate([pk.pid for pk in parse(f).packets]).tolist())
    a = O.decode_aggregate([f], np.ones(1, np.float32), x.size)
    assert (O.decode_aggregate_unframed([u], np.ones(1, np.float32), x.size).view(np.uint32) == a.view(np.uint32)).all()
    x = rng.standard_normal(600).astype(np.float32)
    p = O.make_params(600, 3 * 4096, packet_bits=4096, scale_B=1.5)
    pl, f, u = both_streams(x, p, fixed_y=10)
    assert pl.k >= 500                                                    # 3 blocks of 200 of 600 coordinates: m = 1
    U = parse_unframed(u)
    a = O.decode_aggregate([f], np.ones(1, np.float32), 600)
    assert (O.decode_aggregate_unframed([u], np.ones(1, np.float32), 600).view(np.uint32) == a.view(np.uint32)).all()


def test_workload_sizes_report_the_saving():
    w = W.WORKLOADS["resnet18"]
    x = W.client_update(w, 0, d=400_000)
    p = O.make_params(x.size, 2 * x.size)
    pl, f, u = both_streams(x, p)
    assert 0.6 < u.size / f.size < 0.85                                   # about a quarter of the traffic is frame and position bits


def test_malformed_unframed_streams_are_rejected():
    x, p = small_case(d=20000, R=6, packet_bits=1024)
    pl, f, u = both_streams(x, p)
    w = np.ones(1, np.float32)
    O.decode_aggregate_unframed([u], w, 20000)
    for bad in (u[:-8], np.concatenate([u, np.zeros(8, np.uint8)])):
        with pytest.raises(O.OracleError):
            O.decode_aggregate_unframed([bad], w, 20000)
    for off, val in ((0, 0), (4, 1), (64 + 4 * 8, 99), (64 + 264 + 8 + 8, 0xFF), (64 + 264 + 8 + 8, 1)):     # magic, version, n_y, directory
        b = u.copy()
        b[off] = val
        with pytest.raises(O.OracleError):
            O.decode_aggregate_unframed([b], w, 20000)
    with pytest.raises(O.OracleError):
        O.decode_aggregate_unframed([f], w, 20000)                        # a framed stream is not an unframed one
    with pytest.raises(O.OracleError):
        O.decode_aggregate([u], w, 20000)
