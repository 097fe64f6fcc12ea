"""Pins for the oracle's ranking, PQ quantizer, packet stream and aggregation."""
import math

import numpy as np
import pytest

import oracle as O
from paper_2402_03770_b200 import workloads as W
from stream_reader import parse, dequantize


# ---------------------------------------------------------------- ranking

def numpy_rank(x, k):
    key = (x.view(np.uint32) & np.uint32(0x7FFFFFFF)).astype(np.int64)
    order = np.lexsort((np.arange(x.size), -key))        # |x| descending, index ascending
    return order[:k].astype(np.uint32)


def test_rank_against_lexsort_with_ties_and_zeros():
    rng = np.random.default_rng(3)
    x = (np.round(rng.standard_normal(20000) * 8) / 8).astype(np.float32)   # many exact ties, both signs
    x[rng.integers(0, x.size, 3000)] = 0.0
    x[rng.integers(0, x.size, 500)] = -0.0
    for k in [0, 1, 17, 5000, 19999, 20000]:
        got = O.rank(x, k)
        assert (got == numpy_rank(x, k)).all()
    full = O.rank(x, x.size)
    assert sorted(full.tolist()) == list(range(x.size))                      # a permutation
    mags = np.abs(x[full])
    assert (np.diff(mags) <= 0).all()
    same = np.diff(mags) == 0
    assert (np.diff(full.astype(np.int64))[same] > 0).all()                  # equal |x|: ascending index


# ---------------------------------------------------------------- PQ quantizer

def test_pq_code_range_and_error_bound():
    rng = np.random.default_rng(5)
    for y in [1, 2, 5, 8, 13, 24, 31, 32]:
        lo, hi = np.float32(-0.37), np.float32(1.91)
        L = 2 ** y - 1
        step = (float(hi) - float(lo)) / L
        xs = rng.uniform(lo, hi, 300).astype(np.float32)
        xs[:2] = [lo, hi]
        for x in xs:
            rnd = int(rng.integers(0, 2 ** 32))
            c = O.pq_quantize(float(x), float(lo), float(hi), y, rnd)
            assert 0 <= c <= L
            v = O.pq_dequantize(c, float(lo), float(hi), y)
            assert abs(v - float(x)) <= step * (1 + 1e-6) + abs(float(x)) * 1.2e-7
            assert float(lo) <= v <= float(hi)
        assert O.pq_quantize(float(lo), float(lo), float(hi), y, 0xFFFFFFFF) == 0
        assert O.pq_quantize(float(hi), float(lo), float(hi), y, 0) == L
    assert O.pq_quantize(0.5, 0.5, 0.5, 7, 123) == 0
    assert O.pq_dequantize(0, 0.5, 0.5, 7) == 0.5


def test_pq_unbiased_over_many_seeds():
    """E[quantized value] = value (the unbiasedness Lemma 1 rests on), measured
    over 4096 Philox seeds per coordinate."""
    n_seeds = 4096
    lo, hi, y = -1.0, 2.0, 3
    step = (hi - lo) / (2 ** y - 1)
    xs = np.array([-1.0, -0.9, -0.31, 0.0, 0.123, 0.77, 1.5, 1.999, 2.0], dtype=np.float32)
    for i, x in enumerate(xs):
        vals = np.array([
            O.pq_dequantize(O.pq_quantize(float(x), lo, hi, y, O.philox_coord(seed, 1, 0, i)), lo, hi, y)
            for seed in range(n_seeds)
        ])
        assert abs(vals.mean() - float(x)) <= 4.0 * step / math.sqrt(4.0 * n_seeds) + 1e-6
        assert len(set(vals.tolist())) <= 2                                   # upper or lower centroid only


def test_lemma1_bound_per_segment():
    """E||U~/B - U||^2 <= (Q + (B-1)^2) / B^2 * ||U||^2 with Q = P / (2^y - 1)^2."""
    rng = np.random.default_rng(9)
    P, y, B = 384, 4, 1.05
    x = rng.laplace(0, 1e-3, P).astype(np.float32)
    lo, hi = float(x.min()), float(x.max())
    Q = P / float((2 ** y - 1) ** 2)
    errs = []
    for seed in range(300):
        v = np.array([O.pq_dequantize(O.pq_quantize(float(x[i]), lo, hi, y, O.philox_coord(seed, 0, 0, i)),
                                      lo, hi, y) for i in range(P)], dtype=np.float64)
        errs.append(((v / B - x.astype(np.float64)) ** 2).sum())
    bound = (Q + (B - 1) ** 2) / B ** 2 * float((x.astype(np.float64) ** 2).sum())
    assert np.mean(errs) <= bound


# ---------------------------------------------------------------- stream

def small_case(d=5000, R=6, packet_bits=1024, seed=0, **kw):
    rng = np.random.default_rng(seed)
    x = rng.laplace(0, 1e-2, d).astype(np.float32)
    p = O.make_params(d, R * packet_bits + 13, packet_bits=packet_bits, seed=77, client_id=3, round=5, **kw)
    return x, p


def test_stream_layout_and_budget():
    x, p = small_case()
    pl = O.plan(x, p)
    st, ranked = O.encode(x, p, pl, want_rank=True)
    assert st.size == 64 + 6 * 128 == O.stream_bytes(p)                       # budget met in whole packets
    S = parse(st)
    assert (S.magic, S.version, S.quantizer) == (0x434C5643, 1, 0)
    assert (S.d, S.R, S.packet_bits, S.header_bits) == (5000, 6, 1024, 80)
    assert (S.client_id, S.seed, S.round, S.scale_B, S.k) == (3, 77, 5, p.scale_B, pl.k)
    assert S.s == 13
    ys = [pk.y for pk in S.packets]
    assert ys == sorted(ys, reverse=True)                                     # y_1 >= ... >= y_R
    counts = [0] * 33
    for y in ys:
        counts[y] += 1
    assert counts == [pl.n_y[y] for y in range(33)]
    pids = np.concatenate([pk.pid for pk in S.packets])
    assert pids.size == pl.k and (pids == ranked).all()
    assert (pids == numpy_rank(x, pl.k)).all()                                # exactly the top-k, in rank order
    Z = 0
    for pk in S.packets:
        P = pk.pid.size
        assert pk.s == 13 and pk.pad_bits_zero
        assert P * (pk.s + pk.y) + 80 <= 1024 < (P + 1) * (pk.s + pk.y) + 80   # Eq. (3)
        seg = x[ranked[Z:Z + P]]
        assert pk.lo == seg.min() and pk.hi == seg.max()                       # centroid distribution
        for j in range(P):
            i = int(ranked[Z + j])
            rnd = O.philox_coord(77, 3, 5, i)
            assert int(pk.cid[j]) == O.pq_quantize(float(x[i]), pk.lo, pk.hi, pk.y, rnd)
        Z += P


@pytest.mark.parametrize("s", list(range(1, 17)))
def test_pack_unpack_every_width(s):
    """records of every (s, y) width survive the bit packing"""
    d = 2 ** s if s > 1 else 2
    rng = np.random.default_rng(s)
    x = rng.standard_normal(d).astype(np.float32)
    for y in range(1, 33):
        w = s + y
        per = max(1, min(d, 4))                                               # records per packet
        packet_bits = ((80 + per * w + 31) // 32) * 32
        p = O.make_params(d, packet_bits, packet_bits=packet_bits, scale_B=1.0, seed=y, max_code_bits=y)
        rc, s_, R, cap = O.derive(p)
        assert rc == O.ORC_OK and s_ == s and R == 1
        if cap[y] > d:
            continue
        pl = O.plan_fixed(p, y)
        st, ranked = O.encode(x, p, pl, want_rank=True)
        S = parse(st)
        pk = S.packets[0]
        assert (pk.s, pk.y) == (s, y) and pk.pad_bits_zero
        assert (pk.pid == ranked).all()
        for j, i in enumerate(ranked):
            assert int(pk.cid[j]) == O.pq_quantize(float(x[i]), pk.lo, pk.hi, y, O.philox_coord(y, 0, 0, int(i)))


@pytest.mark.parametrize("s,d", [(20, 2 ** 20 - 5), (24, 11_200_000 // 1)])
def test_pack_wide_position_ids(s, d):
    rng = np.random.default_rng(s)
    x = rng.standard_normal(d).astype(np.float32)
    p = O.make_params(d, 3 * 12000, scale_B=1.0)
    for y in (1, 32):
        pl = O.plan_fixed(p, y)
        st, ranked = O.encode(x, p, pl, want_rank=True)
        S = parse(st)
        assert S.s == s
        assert (np.concatenate([pk.pid for pk in S.packets]) == ranked).all()


def test_zero_bit_case_is_topk_sparsification():
    """Fixed length for the top k and nothing for the rest = Top_k: at 32 bits the decoded
    vector is Top_k(x)/B to fp32 rounding and exactly zero elsewhere (Algorithm 1, last step)."""
    x, p = small_case(d=8000, R=4, packet_bits=2048, scale_B=1.25)
    pl = O.plan_fixed(p, 32)
    st = O.encode(x, p, pl)
    out = O.decode_aggregate([st], np.ones(1, np.float32), x.size)
    top = numpy_rank(x, pl.k)
    mask = np.zeros(x.size, bool)
    mask[top] = True
    assert (out[~mask] == 0).all()
    ref = x[top].astype(np.float64) / 1.25
    # centroid grid of 2^32 points on a range of width <= 2 max|x|: spacing far below fp32 ulp
    assert np.abs(out[top] - ref).max() <= 2.0 * np.spacing(np.abs(x).max()).astype(np.float64)


@pytest.mark.parametrize("y", [1, 4, 8])
def test_equal_length_case_is_topk_plus_fixed_quantization(y):
    """Every packet at one length = Top_k followed by y-bit PQ on consecutive blocks of the
    ranking (the P_y Top_k baselines); rebuilt here with numpy, compared bit for bit."""
    x, p = small_case(d=6000, R=5, packet_bits=1024, seed=y, scale_B=1.0)
    rc, s, R, cap = O.derive(p)
    pl = O.plan_fixed(p, y)
    st = O.encode(x, p, pl)
    out = O.decode_aggregate([st], np.ones(1, np.float32), x.size)
    top = numpy_rank(x, R * cap[y])
    ref = np.zeros(x.size, dtype=np.float32)
    L = float(2 ** y - 1)
    for r in range(R):
        ids = top[r * cap[y]:(r + 1) * cap[y]]
        seg = x[ids].astype(np.float64)
        lo, hi = np.float64(x[ids].min()), np.float64(x[ids].max())
        t = (seg - lo) / (hi - lo) * L
        j0 = np.minimum(np.floor(t), L)
        u = np.array([O.philox_coord(77, 3, 5, int(i)) for i in ids], dtype=np.float64) / 2.0 ** 32
        code = j0 + (u < (t - j0))
        ref[ids] = (lo + code * ((hi - lo) / L)).astype(np.float32)
    assert (out.view(np.uint32) == ref.view(np.uint32)).all()


def test_negative_zero_is_stored_as_positive_zero():
    d = 64
    x = np.zeros(d, dtype=np.float32)
    x[::2] = -0.0
    p = O.make_params(d, 1024, packet_bits=1024, scale_B=1.0)
    pl = O.plan_fixed(p, 32)
    S = parse(O.encode(x, p, pl))
    for pk in S.packets:
        assert np.float32(pk.lo).view(np.uint32) == 0 and np.float32(pk.hi).view(np.uint32) == 0
        assert (pk.cid == 0).all()
    assert (np.concatenate([pk.pid for pk in S.packets]) == np.arange(pl.k)).all()


def test_encode_rejects_bad_input():
    x, p = small_case()
    pl = O.plan(x, p)
    xb = x.copy()
    xb[5] = np.nan
    with pytest.raises(O.OracleError) as e:
        O.encode(xb, p, pl)
    assert e.value.code == O.ORC_ERR_NONFINITE_INPUT
    pl.n_y[9] += 1
    with pytest.raises(O.OracleError):
        O.encode(x, p, pl)


# ---------------------------------------------------------------- aggregation

def test_single_client_aggregate_is_the_dequantized_vector():
    x, p = small_case(scale_B=1.0)
    pl = O.plan(x, p)
    st = O.encode(x, p, pl)
    out = O.decode_aggregate([st], np.ones(1, np.float32), x.size)
    ref = np.zeros(x.size, dtype=np.float32)
    for pk in parse(st).packets:
        ref[pk.pid.astype(np.int64)] = dequantize(pk)
    assert (out.view(np.uint32) == ref.view(np.uint32)).all()


def make_clients(n, d=4000, R=5):
    streams, xs, Bs = [], [], []
    for i in range(n):
        rng = np.random.default_rng(100 + i)
        x = rng.laplace(0, 1e-2, d).astype(np.float32)
        p = O.make_params(d, R * 1024, packet_bits=1024, seed=i, client_id=i, scale_B=1.0 + 0.01 * i)
        streams.append(O.encode(x, p, O.plan(x, p)))
        xs.append(x)
        Bs.append(p.scale_B)
    return streams, xs, Bs


def test_aggregate_is_the_weighted_mean_of_decoded_clients():
    """w_{t+1} - w_t = -(1/|S_t|) sum_i U^_i (Section III, step 3), with sample-count weights"""
    n, d = 7, 4000
    streams, xs, Bs = make_clients(n, d)
    w = np.random.default_rng(7).uniform(50, 500, n).astype(np.float32)
    out = O.decode_aggregate(streams, w, d)
    ref = np.zeros(d, dtype=np.float64)
    W_ = float(w.astype(np.float64).sum())
    for st, wi, B in zip(streams, w, Bs):
        for pk in parse(st).packets:
            np.add.at(ref, pk.pid.astype(np.int64), dequantize(pk).astype(np.float64) * float(np.float32(float(wi) / (W_ * B))))
    np.testing.assert_allclose(out, ref, rtol=2e-7, atol=1e-12)
    # uniform weights: the plain average
    out_u = O.decode_aggregate(streams, np.ones(n, np.float32), d)
    single = [O.decode_aggregate([st], np.ones(1, np.float32), d).astype(np.float64) for st in streams]
    np.testing.assert_allclose(out_u, sum(single) / n, rtol=1e-6, atol=1e-8)
    # linear in the weights
    out2 = O.decode_aggregate(streams, 2 * w, d, weight_total=W_)
    np.testing.assert_allclose(out2, 2 * out.astype(np.float64), rtol=1e-6, atol=1e-8)


def test_accumulate_over_two_batches_equals_one_call():
    n, d = 6, 4000
    streams, xs, Bs = make_clients(n, d)
    w = np.arange(1, n + 1, dtype=np.float32)
    W_ = float(w.sum())
    one = O.decode_aggregate(streams, w, d, weight_total=W_)
    two = O.decode_aggregate(streams[:3], w[:3], d, weight_total=W_)
    two = O.decode_aggregate(streams[3:], w[3:], d, weight_total=W_, out=two, accumulate=True)
    np.testing.assert_allclose(two, one, rtol=1e-6, atol=1e-7)


def _corrupt(st, offset, value):
    bad = st.copy()
    bad[offset] = value
    return bad


def test_decode_rejects_malformed_streams():
    x, p = small_case()
    st = O.encode(x, p, O.plan(x, p))
    w = np.ones(1, np.float32)
    cases = [
        _corrupt(st, 0, 0x00),                 # magic
        _corrupt(st, 4, 2),                    # version
        _corrupt(st, 7, 12),                   # s does not match d
        _corrupt(st, 16, 7),                   # R does not match the length
        st[:-1],                               # truncated
        _corrupt(st, 64 + 1, 33),              # y_1 out of range
        _corrupt(st, 64 + 1, 0),               # y_1 = 0
        _corrupt(st, 64 + 128 * 5 + 1, 32),    # lengths must not increase
    ]
    for bad in cases:
        with pytest.raises(O.OracleError) as e:
            O.decode_aggregate([bad], w, x.size)
        assert e.value.code == O.ORC_ERR_BAD_STREAM
    with pytest.raises(O.OracleError):
        O.decode_aggregate([st], w, x.size + 1)
    # a position ID beyond d
    d = 5000
    S = parse(st)
    bad = st.copy()
    bits = np.unpackbits(bad[64:64 + 128], bitorder="little")
    bits[80:80 + 13] = 1                       # PID 8191 >= 5000
    bad[64:64 + 128] = np.packbits(bits, bitorder="little")
    with pytest.raises(O.OracleError) as e:
        O.decode_aggregate([bad], w, d)
    assert e.value.code == O.ORC_ERR_BAD_STREAM
