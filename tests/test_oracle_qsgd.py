"""Pins for the oracle's QSGD quantizer (the second quantizer of the paper's experiments):
level grid, sign, norm, unbiasedness, the variance its error factor Q bounds, the packet
stream and the planner under this Q."""
import itertools
import math

import numpy as np
import pytest

import oracle as O
from stream_reader import parse, dequantize_qsgd
from test_oracle_codec import numpy_rank, small_case

QSGD = 1


def levels(y):
    return 2 ** (y - 1) - 1


# ---------------------------------------------------------------- quantizer

def test_qsgd_code_layout_range_and_error_bound():
    rng = np.random.default_rng(11)
    for y in [2, 3, 5, 8, 13, 24, 31, 32]:
        sq = levels(y)
        norm = float(np.float32(3.25))
        step = norm / sq
        xs = rng.uniform(-norm, norm, 300).astype(np.float32)
        xs[:5] = [norm, -norm, 0.0, -0.0, np.float32(1e-30)]
        for x in xs:
            rnd = int(rng.integers(0, 2 ** 32))
            c = O.qsgd_quantize(float(x), norm, y, rnd)
            assert 0 <= c < 2 ** y
            level, sign = c & sq, c >> (y - 1)
            assert sign == (1 if x < 0 else 0)                                # the top bit of the code is the sign
            v = O.qsgd_dequantize(c, norm, y)
            assert abs(v - float(x)) <= step * (1 + 1e-6) + abs(float(x)) * 1.2e-7
            assert abs(v) <= norm and (v == 0 or (v < 0) == (x < 0))
            assert level in (math.floor(abs(float(x)) / norm * sq), math.floor(abs(float(x)) / norm * sq) + 1)
        assert O.qsgd_quantize(norm, norm, y, 0) == sq                        # |x| = norm: the top level, no coin
        assert O.qsgd_quantize(-norm, norm, y, 0xFFFFFFFF) == (1 << (y - 1)) | sq
        assert O.qsgd_dequantize(sq, norm, y) == np.float32(norm)
        assert O.qsgd_quantize(0.0, norm, y, 0) == 0
    assert O.qsgd_quantize(0.0, 0.0, 7, 123) == 0                             # an all-zero packet
    assert O.qsgd_dequantize(0, 0.0, 7) == 0.0


def test_qsgd_ternary_at_two_bits():
    """two bits = sign + one level: the values are -norm, 0, +norm with P(|v| = norm) = |x| / norm"""
    norm, y = 2.0, 2
    hits = sum(abs(O.qsgd_dequantize(O.qsgd_quantize(0.5, norm, y, O.philox_coord(s, 0, 0, 0)), norm, y)) == norm
               for s in range(8192))
    assert abs(hits / 8192 - 0.25) < 4 * math.sqrt(0.25 * 0.75 / 8192)
    assert {O.qsgd_dequantize(c, norm, y) for c in range(4)} == {0.0, 2.0, -2.0, -0.0}


def test_qsgd_unbiased_over_many_seeds():
    n_seeds = 4096
    norm, y = 2.5, 4
    step = norm / levels(y)
    xs = np.array([-2.5, -1.9, -0.31, 0.0, 0.123, 0.77, 1.5, 2.4999, 2.5], dtype=np.float32)
    for i, x in enumerate(xs):
        vals = np.array([
            O.qsgd_dequantize(O.qsgd_quantize(float(x), norm, y, O.philox_coord(seed, 1, 0, i)), norm, y)
            for seed in range(n_seeds)
        ])
        assert abs(vals.mean() - float(x)) <= 4.0 * step / math.sqrt(4.0 * n_seeds) + 1e-6
        assert len(set(np.abs(vals).tolist())) <= 2                            # upper or lower level only


def test_qsgd_norm_is_the_l2_norm():
    assert O.qsgd_norm(np.array([3.0, -4.0], np.float32)) == 5.0
    assert O.qsgd_norm(np.array([0.0, -0.0, 0.0], np.float32)) == 0.0
    assert O.qsgd_norm(np.array([2.0 ** -60] * 4, np.float32)) == 2.0 ** -59    # squares far below fp32's range
    assert O.qsgd_norm(np.array([3e38, 3e38], np.float32)) == np.finfo(np.float32).max   # beyond fp32: cut
    rng = np.random.default_rng(2)
    for n in [1, 7, 384, 476]:
        v = (rng.standard_normal(n) * 10.0 ** rng.uniform(-6, 3)).astype(np.float32)
        exact = math.sqrt(math.fsum(float(t) * float(t) for t in v))
        got = O.qsgd_norm(v)
        assert abs(got - exact) <= float(np.spacing(np.float32(exact))) * 0.5 * (1 + 1e-6)
        assert got >= float(np.abs(v).max())                                  # so that every level is <= s_q


def empirical_error(x, norm, y, n_seeds):
    errs = []
    for seed in range(n_seeds):
        v = np.array([O.qsgd_dequantize(O.qsgd_quantize(float(x[i]), norm, y, O.philox_coord(seed, 0, 0, i)), norm, y)
                      for i in range(x.size)], dtype=np.float64)
        errs.append(((v - x.astype(np.float64)) ** 2).sum())
    return float(np.mean(errs))


def test_qsgd_error_factor_Q_bounds_and_nearly_meets_the_variance():
    """Q = min(P / s_q^2, sqrt(P) / s_q) bounds E||v - x||^2 / ||x||^2 (the error factor Lemma 1 takes);
    on equal-magnitude vectors the variance is known in closed form, P (norm / s_q)^2 p (1 - p) with
    p = frac(s_q / sqrt(P)), which comes within 4x of the first branch and 5 % of the second."""
    b, H, d = 12000, 80, 1 << 20
    # first branch: P = 372 records at 8 bits, s_q = 127 > sqrt(P)
    p8 = O.make_params(d, b, packet_bits=b, header_bits=H, quantizer=QSGD, scale_B=1.0, max_code_bits=8)
    rc, s, R, cap = O.derive(p8)
    P = cap[8]
    assert P == (b - H) // (20 + 8)
    Q = O.quant_error_Q(p8, 8)
    x = np.full(P, 1.0, np.float32)
    x[::2] = -1.0
    norm = O.qsgd_norm(x)
    t = 127 / math.sqrt(P)
    frac = t - math.floor(t)
    var = P * (norm / 127) ** 2 * frac * (1 - frac) / float(P)                 # relative to ||x||^2 = P
    emp = empirical_error(x, norm, 8, 200) / float(P)
    assert abs(emp - var) <= 0.1 * var
    assert emp <= Q <= 4.0 * var / (4 * frac * (1 - frac)) * 1.0001            # Q = P / s_q^2 = 4 x the p = 1/2 variance
    rng = np.random.default_rng(4)
    xr = rng.laplace(0, 1e-3, P).astype(np.float32)
    assert empirical_error(xr, O.qsgd_norm(xr), 8, 100) <= Q * float((xr.astype(np.float64) ** 2).sum())
    # second branch: two bits, s_q = 1 < sqrt(P)
    p2 = O.make_params(d, b, packet_bits=b, header_bits=H, quantizer=QSGD, scale_B=1.0, max_code_bits=2)
    rc, s, R, cap = O.derive(p2)
    P2 = cap[2]
    Q2 = O.quant_error_Q(p2, 2)
    x2 = np.full(P2, 0.5, np.float32)
    emp2 = empirical_error(x2, O.qsgd_norm(x2), 2, 400) / float((x2.astype(np.float64) ** 2).sum())
    assert emp2 <= Q2 <= emp2 / (1 - 1 / math.sqrt(P2)) * 1.1
    assert math.isinf(O.quant_error_Q(O.make_params(d, b, quantizer=QSGD, scale_B=1.0), 1))   # one bit holds no level


def test_Q_of_qsgd_falls_with_the_code_length_and_switches_branch_at_sqrt_P():
    p = O.make_params(11_200_000, 12000 * 10, quantizer=QSGD, scale_B=1.0)
    rc, s, R, cap = O.derive(p)
    Qs = [O.quant_error_Q(p, y) for y in range(2, 33)]
    assert all(a > b > 0 for a, b in zip(Qs, Qs[1:]))
    for y in range(2, 33):
        sq, P = levels(y), cap[y]
        ratio = O.quant_error_Q(p, y) * sq / math.sqrt(P)                      # Q / (sqrt(P) / s_q)
        if sq * sq < P:
            assert ratio == pytest.approx(1.0, rel=1e-12)
        else:
            assert ratio == pytest.approx(math.sqrt(P) / sq, rel=1e-12)
    # against PQ at the same length: (2^y - 1)^2 intervals against (2^(y-1) - 1)^2 levels
    ppq = O.make_params(11_200_000, 12000 * 10, quantizer=0, scale_B=1.0)
    for y in (12, 20):
        assert O.quant_error_Q(p, y) / O.quant_error_Q(ppq, y) == pytest.approx(((2 ** y - 1) / levels(y)) ** 2, rel=1e-12)
    assert O.default_scale(p) == 1.0 + O.quant_error_Q(p, 8)


# ---------------------------------------------------------------- planner with this Q

def brute_force(p, beta):
    Y = O.candidates(p)
    rc, s, R, cap = O.derive(p)
    best, bestF = None, -math.inf
    for split in itertools.combinations_with_replacement(range(len(Y)), R):
        n = [0] * 33
        for i in split:
            n[Y[i]] += 1
        F = O.objective(p, beta, n)
        if F > bestF:
            best, bestF = n, F
    return best, bestF


@pytest.mark.parametrize("alpha_q", [-1.0, -0.75, -0.53125, -0.25])
@pytest.mark.parametrize("R", [3, 5])
def test_plan_with_qsgd_equals_brute_force(alpha_q, R):
    d, b = 60000, 2048
    p = O.make_params(d, R * b, packet_bits=b, quantizer=QSGD, max_code_bits=10)
    p.scale_B = O.default_scale(p)
    Y = O.candidates(p)
    assert Y[0] >= 2
    pl = O.plan_from_alpha(p, alpha_q)
    best, bestF = brute_force(p, 2 * alpha_q + 1)
    assert 1.0 - pl.gamma == pytest.approx(bestF, rel=0, abs=1e-12)
    assert list(pl.n_y) == best
    assert pl.n_y[1] == 0 and pl.y_min >= 2
    used = [y for y in range(33) if pl.n_y[y]]
    assert pl.B_next == 1.0 + max(O.quant_error_Q(p, y) for y in used)


def test_fixed_plan_rejects_one_bit_and_closed_form_gamma():
    d, b, R = 50000, 2048, 4
    p = O.make_params(d, R * b, packet_bits=b, quantizer=QSGD, scale_B=1.2)
    with pytest.raises(O.OracleError):
        O.plan_fixed(p, 1)
    pl = O.plan_fixed(p, 6)
    rc, s, R_, cap = O.derive(p)
    # uniform plan, beta = -1: gamma = 1 - g(6) E(R cap(6)), E(Z) = (1 - 1/(Z+1)) / (1 - 1/d)
    Z = R * cap[6]
    E = (1.0 - 1.0 / (Z + 1)) / (1.0 - 1.0 / d)
    Q = min(cap[6] / 31.0 ** 2, math.sqrt(cap[6]) / 31.0)
    g = 1.0 - (Q / 1.2 ** 2 + (1 - 1 / 1.2) ** 2)
    assert pl.gamma == pytest.approx(1.0 - g * E, rel=1e-9)


# ---------------------------------------------------------------- stream

def test_qsgd_stream_layout():
    x, p = small_case(quantizer=QSGD)
    p.scale_B = O.default_scale(p)
    pl = O.plan(x, p)
    st, ranked = O.encode(x, p, pl, want_rank=True)
    S = parse(st)
    assert (S.magic, S.version, S.quantizer) == (0x434C5643, 1, QSGD)
    assert S.k == pl.k and st.size == O.stream_bytes(p)
    pids = np.concatenate([pk.pid for pk in S.packets])
    assert (pids == numpy_rank(x, pl.k)).all()
    Z = 0
    for pk in S.packets:
        P = pk.pid.size
        assert pk.y >= 2 and pk.pad_bits_zero
        assert P * (pk.s + pk.y) + 80 <= 1024 < (P + 1) * (pk.s + pk.y) + 80   # Eq. (3): a record is s + y bits
        seg = x[ranked[Z:Z + P]]
        total = 0.0
        for t in seg:                                                          # rank order, double
            total = total + float(t) * float(t)
        assert pk.lo == np.float32(math.sqrt(total))                           # centroid distribution: the l2-norm
        assert np.float32(pk.hi).view(np.uint32) == 0                          # the other 32 bits stay empty
        for j in range(P):
            i = int(ranked[Z + j])
            assert int(pk.cid[j]) == O.qsgd_quantize(float(x[i]), pk.lo, pk.y, O.philox_coord(77, 3, 5, i))
        Z += P


@pytest.mark.parametrize("y", [2, 5, 9])
def test_equal_length_case_is_topk_plus_fixed_qsgd(y):
    """Every packet at one length = Top_k followed by y-bit QSGD on consecutive blocks of the ranking
    (the Q_y Top_k baselines); rebuilt here with numpy, compared bit for bit."""
    x, p = small_case(d=6000, R=5, packet_bits=1024, seed=y, scale_B=1.0, quantizer=QSGD)
    rc, s, R, cap = O.derive(p)
    pl = O.plan_fixed(p, y)
    st = O.encode(x, p, pl)
    out = O.decode_aggregate([st], np.ones(1, np.float32), x.size)
    top = numpy_rank(x, R * cap[y])
    ref = np.zeros(x.size, dtype=np.float32)
    sq = float(levels(y))
    for r in range(R):
        ids = top[r * cap[y]:(r + 1) * cap[y]]
        seg = x[ids].astype(np.float64)
        norm = np.float64(np.float32(np.sqrt(np.cumsum(seg * seg)[-1])))       # cumsum adds in order
        t = np.abs(seg) / norm * sq
        j0 = np.minimum(np.floor(t), sq)
        u = np.array([O.philox_coord(77, 3, 5, int(i)) for i in ids], dtype=np.float64) / 2.0 ** 32
        level = j0 + (u < (t - j0))
        mag = (level * (norm / sq)).astype(np.float32)
        ref[ids] = np.where(mag == 0, np.float32(0), np.copysign(mag, x[ids]))   # a sum that starts at +0 stays +0
    assert (out.view(np.uint32) == ref.view(np.uint32)).all()


def test_high_resolution_case_is_topk_sparsification():
    x, p = small_case(d=8000, R=4, packet_bits=2048, scale_B=1.25, quantizer=QSGD)
    pl = O.plan_fixed(p, 32)
    st = O.encode(x, p, pl)
    out = O.decode_aggregate([st], np.ones(1, np.float32), x.size)
    top = numpy_rank(x, pl.k)
    mask = np.zeros(x.size, bool)
    mask[top] = True
    assert (out[~mask] == 0).all()
    ref = x[top].astype(np.float64) / 1.25
    # 2^31 - 1 levels on [0, norm], norm <= sqrt(P) max|x|: the grid is far finer than fp32
    assert np.abs(out[top] - ref).max() <= 2.0 * np.spacing(np.abs(x).max()).astype(np.float64)


def test_single_client_aggregate_is_the_dequantized_vector_and_mixed_quantizers_add_up():
    x, p = small_case(scale_B=1.0, quantizer=QSGD)
    st = O.encode(x, p, O.plan(x, p))
    out = O.decode_aggregate([st], np.ones(1, np.float32), x.size)
    ref = np.zeros(x.size, dtype=np.float32)
    for pk in parse(st).packets:
        ref[pk.pid.astype(np.int64)] = dequantize_qsgd(pk)
    assert (out.view(np.uint32) == ref.view(np.uint32)).all()
    # a PQ client and a QSGD client in one aggregate: every stream names its quantizer
    x2, p2 = small_case(seed=4, scale_B=1.0)
    st2 = O.encode(x2, p2, O.plan(x2, p2))
    both = O.decode_aggregate([st, st2], np.ones(2, np.float32), x.size)
    one2 = O.decode_aggregate([st2], np.ones(1, np.float32), x.size)
    np.testing.assert_allclose(both, 0.5 * (out.astype(np.float64) + one2), rtol=1e-6, atol=1e-9)


def test_qsgd_stream_of_zeros_and_ties():
    d = 160
    x = np.zeros(d, dtype=np.float32)
    x[::3] = -0.0
    x[5], x[50] = 0.25, -0.25
    p = O.make_params(d, 2 * 1024, packet_bits=1024, scale_B=1.0, quantizer=QSGD)
    pl = O.plan_fixed(p, 9)
    st = O.encode(x, p, pl)
    S = parse(st)
    assert list(S.packets[0].pid[:2]) == [5, 50]                               # equal |x|: ascending index
    first = S.packets[0]
    assert first.lo == np.float32(math.sqrt(0.125))
    out = O.decode_aggregate([st], np.ones(1, np.float32), d)
    assert (out[[i for i in range(d) if i not in (5, 50)]] == 0).all()
    assert out[5] > 0 > out[50]
    if len(S.packets) > 1 and S.packets[1].pid.size:
        assert S.packets[1].lo == 0.0 and (S.packets[1].cid == 0).all()       # an all-zero packet: norm 0, codes 0


def test_decode_rejects_malformed_qsgd_streams():
    x, p = small_case(quantizer=QSGD)
    st = O.encode(x, p, O.plan(x, p))
    w = np.ones(1, np.float32)
    bad_q = st.copy()
    bad_q[6] = 2                                                               # unknown quantizer
    bad_y = st.copy()
    last = 64 + 128 * 5
    bad_y[last + 1] = 1                                                        # one bit: no room for a level
    bad_norm = st.copy()
    bits = np.unpackbits(bad_norm[64:64 + 128], bitorder="little")
    bits[16:48] = np.unpackbits(np.array([0x7F800000], dtype="<u4").view(np.uint8), bitorder="little")
    bad_norm[64:64 + 128] = np.packbits(bits, bitorder="little")             # norm = +inf
    neg_norm = st.copy()
    bits = np.unpackbits(neg_norm[64:64 + 128], bitorder="little")
    bits[47] = 1                                                               # sign bit of the norm
    neg_norm[64:64 + 128] = np.packbits(bits, bitorder="little")
    for bad in (bad_q, bad_y, bad_norm, neg_norm):
        with pytest.raises(O.OracleError) as e:
            O.decode_aggregate([bad], w, x.size)
        assert e.value.code == O.ORC_ERR_BAD_STREAM
