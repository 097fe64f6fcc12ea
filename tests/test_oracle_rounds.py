"""Pins for the oracle's steps either side of one round's compression: planning at the parameter
server from a transmitted histogram, the scale carried from round to round, and the model step."""
import numpy as np
import pytest

import oracle as O
from stream_reader import parse, dequantize
from test_oracle_codec import small_case, make_clients


def plan_tuple(pl):
    return (pl.s, pl.R, pl.y_min, pl.n_lengths, pl.k, pl.alpha, pl.alpha_q, pl.beta, pl.gamma, pl.B_next, list(pl.n_y))


def test_plan_depends_on_the_update_only_through_its_histogram():
    """Algorithm 1 reads the update through alpha alone, which is why a client may send its
    distribution and let the parameter server plan (Section IV-C, last paragraph)."""
    x, p = small_case(d=20000, R=12)
    rc, h = O.histogram(x)
    assert rc == O.ORC_OK
    ref = plan_tuple(O.plan(x, p))
    assert plan_tuple(O.plan_from_histogram(h, p)) == ref
    rng = np.random.default_rng(1)
    y = rng.permutation(x) * rng.choice(np.array([-1.0, 1.0], np.float32), x.size)   # same |x| multiset
    assert plan_tuple(O.plan(y, p)) == ref
    # a different distribution gives a different fit
    z = (x * np.linspace(0.01, 1.0, x.size, dtype=np.float32))
    assert O.plan(z, p).alpha != O.plan(x, p).alpha


def test_plan_from_histogram_rejects_bad_histograms():
    x, p = small_case(d=20000, R=12)
    rc, h = O.histogram(x)
    short = h.copy()
    short[int(np.nonzero(h)[0][0])] -= 1                                      # counts do not add up to d
    with pytest.raises(O.OracleError) as e:
        O.plan_from_histogram(short, p)
    assert e.value.code == O.ORC_ERR_INVALID_ARG
    inf = h.copy()
    j = int(np.nonzero(h)[0][0])
    inf[j] -= 1
    inf[0x7F800000 >> 19] += 1                                                 # an Inf among the values
    with pytest.raises(O.OracleError) as e:
        O.plan_from_histogram(inf, p)
    assert e.value.code == O.ORC_ERR_NONFINITE_INPUT
    xb = x.copy()
    xb[3] = np.inf
    rc, hb = O.histogram(xb)
    assert rc == O.ORC_ERR_NONFINITE_INPUT and (hb == inf).sum() >= O.HIST_BINS - 2


def test_scale_carried_to_the_next_round():
    """B of a round is 1 + max Q of the previous round's plan (footnote to Proposition 2)"""
    x, p = small_case(d=20000, R=12)
    pl0 = O.plan(x, p)
    used = [y for y in range(1, 33) if pl0.n_y[y]]
    assert pl0.B_next == 1.0 + max(O.quant_error_Q(p, y) for y in used)
    assert pl0.B_next == 1.0 + O.quant_error_Q(p, min(used))                   # Q falls with the code length
    p1 = O.make_params(p.d, p.budget_bits, packet_bits=p.packet_bits, seed=p.seed, client_id=p.client_id, round=p.round + 1,
                       scale_B=pl0.B_next)
    x1 = (x * np.float32(0.9)).astype(np.float32)
    pl1 = O.plan(x1, p1)
    assert 0.0 < pl1.gamma < 1.0
    st0, st1 = O.encode(x, p, pl0), O.encode(x1, p1, pl1)
    S0, S1 = parse(st0), parse(st1)
    assert (S1.round, S1.scale_B) == (S0.round + 1, pl0.B_next)
    # the round enters the Philox counter: same values, other coins
    same = O.encode(x, O.make_params(p.d, p.budget_bits, packet_bits=p.packet_bits, seed=p.seed, client_id=p.client_id,
                                     round=p.round + 1, scale_B=p.scale_B), pl0)
    assert (same[64:] != st0[64:]).any()


def test_model_step_is_minus_the_aggregate():
    """w_{t+1} = w_t - (1/|S_t|) sum_i U_i (Section III, step 3)"""
    n, d = 5, 4000
    streams, xs, Bs = make_clients(n, d)
    w = np.ones(n, np.float32)
    rng = np.random.default_rng(0)
    model = rng.standard_normal(d).astype(np.float32)
    agg = O.decode_aggregate(streams, w, d)
    new = O.decode_apply(streams, w, model.copy())
    assert (new == model - agg).all()
    untouched = agg == 0
    assert untouched.any() and (new[untouched] == model[untouched]).all()
    # against the independent reader: mean of the dequantized clients
    ref = np.zeros(d, np.float64)
    for st, B in zip(streams, Bs):
        for pk in parse(st).packets:
            np.add.at(ref, pk.pid.astype(np.int64), dequantize(pk).astype(np.float64) * float(np.float32(1.0 / (n * B))))
    np.testing.assert_allclose(model.astype(np.float64) - new, ref, rtol=0, atol=2e-7)
    with pytest.raises(O.OracleError):
        O.decode_apply([streams[0][:-1]], w[:1], model.copy())
