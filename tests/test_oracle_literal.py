"""Pins of the oracle's real-valued planner (problem P2 of Section IV-C: packet sizes P_1 <= ... <= P_R as real numbers,
code lengths y_r = (b - H) / P_r - s, k on a grid).

The planner reaches its answer by re-splitting consecutive packets; what it must reach is fixed by the problem itself:
for a given k, the minimum of Eq. (5) over the feasible packet sizes.  That minimum is computed here by a general
constrained optimiser (scipy SLSQP, several starts, libm arithmetic) that shares nothing with the oracle, and by
closed forms where there are any.  Further pins: the ordering of Theorem 1, pairwise optimality (no re-split of two
consecutive packets lowers Eq. (7)), the choice of k*, and the relation to the integer-length planner, which solves
a restriction of the same problem."""
import math

import numpy as np
import pytest
from scipy.optimize import minimize

import oracle as O

H = 80


def gamma_real(P, d, b, s, beta, B, quantizer=0):
    """Eq. (5) for real packet sizes with libm, the energy boundary shifted by one as everywhere in this build"""
    D = d ** beta - 1.0
    Z = np.concatenate([[0.0], np.cumsum(P)])
    E = ((Z + 1.0) ** beta - 1.0) / D
    y = (b - H) / np.asarray(P) - s
    if quantizer == 0:
        Q = P / (2.0 ** y - 1.0) ** 2
    else:
        sq = 2.0 ** (y - 1.0) - 1.0
        Q = np.minimum(P / sq ** 2, np.sqrt(P) / sq)
    c = Q / B ** 2 + (1.0 - 1.0 / B) ** 2
    return float(1.0 - E[-1] + np.sum(c * np.diff(E)))


def slsqp_minimum(k, R, d, b, s, beta, B, y_max, quantizer=0):
    y_lo = 2 if quantizer else 1
    P_min, P_max = (b - H) / (s + y_max), (b - H) / (s + y_lo)
    cons = [{"type": "eq", "fun": lambda P: np.sum(P) - k}]
    cons += [{"type": "ineq", "fun": (lambda P, r=r: P[r] - P[r - 1])} for r in range(1, R)]
    best = math.inf
    rng = np.random.default_rng(1)
    starts = [np.full(R, k / R)] + [np.sort(rng.dirichlet(np.full(R, 40.0)) * k) for _ in range(4)]
    for x0 in starts:
        x0 = np.clip(x0, P_min, P_max)
        g0 = gamma_real(x0, d, b, s, beta, B, quantizer)                 # the objective is scaled to order one
        res = minimize(lambda P: gamma_real(P, d, b, s, beta, B, quantizer) / g0, x0, method="SLSQP",
                       bounds=[(P_min, P_max)] * R, constraints=cons, options={"ftol": 1e-15, "maxiter": 500})
        P = res.x
        if abs(P.sum() - k) < 1e-6 * k and (np.diff(P) > -1e-7).all():
            best = min(best, gamma_real(P, d, b, s, beta, B, quantizer))
    return best


CASES = [(4000, 4, 2016, -0.75, 0), (100_000, 6, 12000, -0.75, 0), (20_000, 5, 1504, -0.40, 0), (300_000, 3, 4096, -1.3, 0),
         (50_000, 4, 2016, -0.6, 1), (1_000_000, 5, 12000, -0.3, 1)]


@pytest.mark.parametrize("d,R,b,alpha_q,quantizer", CASES)
def test_tuned_packets_reach_the_constrained_minimum(d, R, b, alpha_q, quantizer):
    p = O.make_params(d, R * b, packet_bits=b, quantizer=quantizer)
    _, s, R_o, cap = O.derive(p)
    assert R_o == R
    beta = 2.0 * alpha_q + 1.0
    lp = O.plan_literal(p, alpha_q, 7)
    assert (np.diff(lp.k_grid.astype(np.int64)) > 0).all()
    for k, g in zip(lp.k_grid, lp.gamma_of_k):
        ref = slsqp_minimum(float(k), R, d, b, s, beta, p.scale_B, 32, quantizer)
        # the general optimiser stops a little short of the minimum on the flattest instances: the oracle may be
        # below it by a few parts in a million, never above
        assert ref * (1.0 - 2e-5) <= g <= ref * (1.0 + 2e-6), (int(k), g, ref)
    # k* is the grid value with the smallest error bound (first one on ties)
    i = int(np.argmin(lp.gamma_of_k))
    assert (lp.k_star, lp.gamma_star) == (int(lp.k_grid[i]), float(lp.gamma_of_k[i]))
    # its packets: feasible, they add up to k*, in the order of Theorem 1, and Eq. (5) at them is gamma*
    y_lo = 2 if quantizer else 1
    P = lp.P_star
    assert P.sum() == pytest.approx(lp.k_star, rel=1e-12)
    assert (np.diff(P) >= -1e-9).all()
    assert P.min() >= (b - H) / (s + 32) - 1e-9 and P.max() <= (b - H) / (s + y_lo) + 1e-9
    assert gamma_real(P, d, b, s, beta, p.scale_B, quantizer) == pytest.approx(lp.gamma_star, rel=1e-9)


@pytest.mark.parametrize("d,R,b,alpha_q,quantizer", CASES[:4])
def test_no_resplit_of_two_consecutive_packets_helps(d, R, b, alpha_q, quantizer):
    """pairwise optimality (the premise of Theorem 1): moving a little from one packet to its neighbour never lowers
    Eq. (5), unless a bound or the ordering forbids the move"""
    p = O.make_params(d, R * b, packet_bits=b, quantizer=quantizer)
    _, s, _, _ = O.derive(p)
    beta = 2.0 * alpha_q + 1.0
    lp = O.plan_literal(p, alpha_q, 3)
    P = lp.P_star
    g0 = gamma_real(P, d, b, s, beta, p.scale_B, quantizer)
    P_min, P_max = (b - H) / (s + 32), (b - H) / (s + 1)
    for r in range(1, R):
        for delta in (1e-3, -1e-3):
            Pn = P.copy()
            Pn[r] += delta
            Pn[r - 1] -= delta
            if Pn.min() < P_min or Pn.max() > P_max or Pn[r] < Pn[r - 1]:
                continue
            assert gamma_real(Pn, d, b, s, beta, p.scale_B, quantizer) >= g0 - 1e-13


def test_single_packet_closed_form():
    """R = 1: nothing to tune; gamma(k) = 1 - E(k) + c(k) E(k) and k* is its minimiser on the grid"""
    d, b, alpha_q = 80_000, 4096, -0.8
    p = O.make_params(d, b, packet_bits=b)
    _, s, R, _ = O.derive(p)
    assert R == 1
    lp = O.plan_literal(p, alpha_q, 41)
    beta = 2 * alpha_q + 1
    ref = np.array([gamma_real(np.array([float(k)]), d, b, s, beta, p.scale_B) for k in lp.k_grid])
    assert lp.gamma_of_k == pytest.approx(ref, rel=1e-10)
    assert lp.k_star == int(lp.k_grid[np.argmin(ref)])
    assert (lp.sweeps_of_k == 1).all()
    # the grid spans the range of k: one record per packet at the longest code ... every record at one bit
    assert lp.k_grid[0] == math.ceil((b - H) / (s + 32)) and lp.k_grid[-1] == math.floor((b - H) / (s + 1))


@pytest.mark.parametrize("d,R,b,alpha_q", [(4000, 4, 2016, -0.75), (100_000, 8, 12000, -0.75), (20_000, 5, 1504, -0.40),
                                           (1_200_000, 12, 12000, -0.6)])
def test_integer_length_plan_is_a_close_restriction(d, R, b, alpha_q):
    """the planner of the hot path picks integer lengths with full packets: a restriction of P2, so its error bound
    cannot be below the real-valued optimum at the same k, and a sound discretisation stays close to it"""
    p = O.make_params(d, R * b, packet_bits=b)
    _, s, _, cap = O.derive(p)
    plan = O.plan_from_alpha(p, alpha_q)
    lp = O.plan_literal(p, alpha_q, 65)
    # at the k of the integer plan the real-valued optimum is at or below it (checked with the general optimiser)
    ref_at_k = slsqp_minimum(float(plan.k), R, d, b, s, 2 * alpha_q + 1, p.scale_B, 32)
    assert ref_at_k <= plan.gamma * (1.0 + 1e-9)
    assert plan.gamma <= lp.gamma_star * 1.02 and lp.gamma_star <= plan.gamma * 1.02
    assert abs(plan.k - lp.k_star) <= 0.05 * lp.k_star + (lp.k_grid[1] - lp.k_grid[0])
    y_real = (b - H) / lp.P_star - s
    y_int = [y for y in range(32, 0, -1) for _ in range(plan.n_y[y])]
    assert len(y_int) == R
    for yi, yl in zip(y_int, y_real):
        assert abs(yi - yl) <= 1.0, (y_int, np.round(y_real, 2).tolist())


def test_sweep_cap_and_arguments():
    p = O.make_params(100_000, 8 * 12000)
    a = O.plan_literal(p, -0.75, 3, max_sweeps=2)
    assert (a.sweeps_of_k == 2).all()
    b = O.plan_literal(p, -0.75, 3)
    assert (b.gamma_of_k <= a.gamma_of_k + 1e-15).all()          # more sweeps never raise Eq. (5)
    for bad in (dict(alpha_q=0.1), dict(alpha_q=-0.5), dict(n_k=0), dict(max_sweeps=0)):
        kw = dict(alpha_q=-0.75, n_k=3, max_sweeps=4)
        kw.update(bad)
        with pytest.raises(O.OracleError):
            O.plan_literal(p, kw["alpha_q"], kw["n_k"], kw["max_sweeps"])
