"""The discretised length tuning of the oracle against Algorithm 1 as the paper prints it.

Algorithm 1 enumerates k, starts every k from equal packets P_r = k / R, and sweeps r = 2 .. R with the atomic
operation on f(X, P_{r-1}, P_r) (Eq. (7)) until nothing moves, with real-valued packet sizes P_r and code lengths
y_r = (b - H) / P_r - s (text after Proposition 2) and the PQ error factor Q(P_r) = P_r / (2^{y_r} - 1)^2
(appendix, case study).  It is restated here in a few lines of Python with libm arithmetic (the energy boundary
shifted by one as in the oracle, the line search of the atomic operation by golden section, k on an equidistant
grid as Section IV-D suggests) and run on instances small enough for its thousands of sweeps.

The oracle's planner works on integer code lengths with maximal packets, a restriction of this real-valued
problem, so its error bound gamma can only be at or above the literal optimum, and a sound discretisation stays
close to it: same number of transmitted coordinates up to a few percent, the printed ordering P_1 <= ... <= P_R,
and integer lengths that bracket the real-valued ones."""
import math

import numpy as np
import pytest

import oracle as O

GOLD = 0.6180339887498949


def literal_algorithm_1(d, R, b, H, s, beta, B, y_max, n_k):
    D = d ** beta - 1.0

    def E(Z):
        return ((Z + 1.0) ** beta - 1.0) / D

    def c(P):  # bracket of Eq. (5) with 1/B_c = 1 - 1/B
        y = (b - H) / P - s
        return P / (2.0 ** y - 1.0) ** 2 / B ** 2 + (1.0 - 1.0 / B) ** 2

    P_min, P_max = (b - H) / (s + y_max), (b - H) / (s + 1.0)
    k_lo, k_hi = max(R, math.ceil(R * P_min)), min(d, math.floor(R * P_max))
    best = None
    for k in np.unique(np.linspace(k_lo, k_hi, n_k).astype(np.int64)):
        P = np.full(R, k / R)
        for _ in range(20000):
            moved = 0.0
            Z = np.concatenate([[0.0], np.cumsum(P)])
            for r in range(1, R):
                X, Z0, Z2 = P[r - 1] + P[r], Z[r - 1], Z[r + 1]
                lo, hi = max(X / 2.0, P_min, X - P_max), min(X - P_min, P_max)  # Eq. (4): P_{r-1} <= P_r
                if not lo < hi:
                    continue

                def f(p):
                    return c(p) * (E(Z2) - E(Z2 - p)) + c(X - p) * (E(Z2 - p) - E(Z0))

                a, z = lo, hi
                x1, x2 = z - GOLD * (z - a), a + GOLD * (z - a)
                f1, f2 = f(x1), f(x2)
                for _ in range(40):
                    if f1 < f2:
                        z, x2, f2 = x2, x1, f1
                        x1 = z - GOLD * (z - a)
                        f1 = f(x1)
                    else:
                        a, x1, f1 = x1, x2, f2
                        x2 = a + GOLD * (z - a)
                        f2 = f(x2)
                p = 0.5 * (a + z)
                if f(p) < f(P[r]):
                    moved = max(moved, abs(p - P[r]))
                    P[r - 1], P[r] = X - p, p
                    Z[r] = Z0 + P[r - 1]
            if moved < 1e-9 * P_max:
                break
        Z = np.concatenate([[0.0], np.cumsum(P)])
        gamma = 1.0 - E(Z[-1]) + sum(c(P[r]) * (E(Z[r + 1]) - E(Z[r])) for r in range(R))
        if best is None or gamma < best[0]:
            best = (gamma, int(k), P.copy())
    return best


@pytest.mark.parametrize("d,R,b,alpha_q", [(4000, 4, 2016, -0.75), (100000, 8, 12000, -0.75), (20000, 5, 1504, -0.40)])
def test_discretised_tuning_stays_close_to_the_literal_algorithm(d, R, b, alpha_q):
    H = 80
    p = O.make_params(d, R * b, packet_bits=b, header_bits=H)
    _, s, R_o, cap = O.derive(p)
    assert R_o == R
    plan = O.plan_from_alpha(p, alpha_q)
    beta = 2.0 * alpha_q + 1.0
    gamma_lit, k_lit, P = literal_algorithm_1(d, R, b, H, s, beta, p.scale_B, 32, 60)
    y_lit = (b - H) / P - s
    # Theorem 1: the optimum has P_1 <= ... <= P_R, i.e. code lengths never increase along the packets
    assert (np.diff(P) >= -1e-6).all()
    # the integer plan is a restriction of the real-valued problem (up to the k grid of the literal search) ...
    assert gamma_lit <= plan.gamma * (1.0 + 2e-3)
    # ... and a close one: error bound within 2 %, transmitted coordinates within 5 %
    assert plan.gamma <= gamma_lit * 1.02
    assert abs(plan.k - k_lit) <= 0.05 * k_lit
    # the integer lengths, longest first, bracket the real-valued ones packet by packet
    y_int = [y for y in range(32, 0, -1) for _ in range(plan.n_y[y])]
    assert len(y_int) == R
    for yi, yl in zip(y_int, y_lit):
        assert abs(yi - yl) <= 1.0, (y_int, np.round(y_lit, 2).tolist())
