"""Pins for the oracle's planner: histogram, exponent fit, packet constraint,
the error bound of Eq. (5), and the length-tuning rule against brute force."""
import itertools
import math

import numpy as np
import pytest

import oracle as O
from paper_2402_03770_b200 import workloads as W


# ---------------------------------------------------------------- histogram

def test_histogram_brute_force():
    rng = np.random.default_rng(0)
    x = (rng.standard_normal(5000) * 10.0 ** rng.uniform(-8, 3, 5000)).astype(np.float32)
    x[:7] = [0.0, -0.0, 1.0, -1.0, 1e-45, -3.4e38, 2.5]
    rc, h = O.histogram(x)
    assert rc == O.ORC_OK
    keys = x.view(np.uint32) & np.uint32(0x7FFFFFFF)
    ref = np.bincount((keys >> np.uint32(19)).astype(np.int64), minlength=4096)
    assert (h.astype(np.int64) == ref).all()
    assert h.sum() == x.size
    rc2, h2 = O.histogram(-x)
    assert rc2 == O.ORC_OK and (h2 == h).all()        # sign-insensitive
    assert h[0] >= 3                                    # +0, -0 and the denormal share bin 0


@pytest.mark.parametrize("bad", [np.inf, -np.inf, np.nan])
def test_histogram_flags_nonfinite(bad):
    x = np.ones(100, dtype=np.float32)
    x[37] = bad
    rc, _ = O.histogram(x)
    assert rc == O.ORC_ERR_NONFINITE_INPUT


# ---------------------------------------------------------------- alpha fit

@pytest.mark.parametrize("alpha", [-0.3, -0.75, -1.2, -2.0])
def test_alpha_recovered_on_exact_power_law(alpha):
    d = 200_000
    x = W.power_law_vector(d, alpha, phi=0.37, seed=5)
    rc, h = O.histogram(x)
    a, aq = O.alpha_fit(h, d)
    assert abs(a - alpha) < 0.02, (a, alpha)
    assert abs(aq - a) <= 1.0 / 512 + 1e-12 or aq in (-4.0, -1.0 / 256)
    assert aq * 256 == round(aq * 256)


def test_alpha_defaults_and_singularity_bump():
    d = 1000
    rc, h = O.histogram(np.zeros(d, dtype=np.float32))
    assert O.alpha_fit(h, d) == (-1.0, -1.0)
    rc, h = O.histogram(np.full(d, 0.125, dtype=np.float32))
    assert O.alpha_fit(h, d) == (-1.0, -1.0)
    # alpha = -1/2 exactly: |x_l| = l^-1/2 sampled at ranks that are exact bin edges
    # (rank 4^m has magnitude 2^-m): the fit returns -1/2 and is moved off beta = 0
    h = np.zeros(4096, dtype=np.uint64)
    counts = {}
    prev = 0
    for m in range(0, 9):
        j = (127 - m) << 4
        N = 4 ** m
        h[j] = N - prev
        prev = N
    d = 2 * prev
    h[0] = d - prev
    a, aq = O.alpha_fit(h, d)
    assert abs(a + 0.5) < 1e-12
    assert aq == -0.5 - 1.0 / 256


def test_alpha_on_workload_shapes():
    w = W.WORKLOADS["tiny"]
    x = W.client_update(w, 0)
    rc, h = O.histogram(x)
    a, aq = O.alpha_fit(h, w.d)
    assert -0.6 < a < -0.1          # Laplace tails: mild decay
    w = W.WORKLOADS["resnet18"]
    x = W.client_update(w, 0, d=400_000)
    rc, h = O.histogram(x)
    a, aq = O.alpha_fit(h, x.size)
    assert -2.0 < a < -0.2


# ---------------------------------------------------------------- derived constants (Eq. (3))

@pytest.mark.parametrize("d", [2, 3, 4, 5, 1000, 1024, 1025, 100_000, 11_200_000, 2 ** 31])
def test_position_bits_and_capacity(d):
    p = O.make_params(d, 10 * 12000)
    rc, s, R, cap = O.derive(p)
    assert rc == O.ORC_OK
    assert s == max(1, math.ceil(math.log2(d)))
    assert R == 10
    b, H = 12000, 80
    for y in range(1, 33):
        P = cap[y]
        assert P * (s + y) + H <= b < (P + 1) * (s + y) + H          # Eq. (3), packed maximally
    assert O.stream_bytes(p) == 64 + 10 * 1500


def test_budget_and_packet_errors():
    p = O.make_params(1000, 11999)
    assert O.derive(p)[0] == O.ORC_ERR_BUDGET_TOO_SMALL
    p = O.make_params(1000, 12000 * 3 + 11999)
    assert O.derive(p)[1:3] == (10, 3)                                  # leftover bits unused
    p = O.make_params(2 ** 31, 96 * 4, packet_bits=96, header_bits=80, scale_B=1.0)
    assert O.derive(p)[0] == O.ORC_ERR_PACKET_TOO_SMALL               # 16 bits cannot hold s + 32
    p = O.make_params(1000, 12000, header_bits=79, scale_B=1.0)
    assert O.derive(p)[0] == O.ORC_ERR_INVALID_ARG
    p = O.make_params(1000, 12000, packet_bits=12001, scale_B=1.0)
    assert O.derive(p)[0] == O.ORC_ERR_INVALID_ARG
    # budget so large that even the longest code sends more than d coordinates
    p = O.make_params(1000, 12000 * 50)
    with pytest.raises(O.OracleError) as e:
        O.plan_from_alpha(p, -0.75)
    assert e.value.code == O.ORC_ERR_BUDGET_TOO_LARGE


def test_default_scale_and_coefficients():
    p = O.make_params(11_200_000, 22_400_000)
    rc, s, R, cap = O.derive(p)
    assert p.scale_B == 1.0 + cap[8] / 255.0 ** 2
    B = p.scale_B
    for y in range(1, 33):
        Q = cap[y] / float((2 ** y - 1) ** 2)                           # PQ error factor (Appendix)
        assert O.quant_error_Q(p, y) == pytest.approx(Q, rel=1e-15)
        g = 1.0 - (Q / B ** 2 + (1.0 - 1.0 / B) ** 2)
        assert O.coeff_g(p, y) == pytest.approx(g, rel=1e-12, abs=1e-15)
        # g > 0 is the paper's condition B > (Q + 1) / 2 (Proposition 1)
        assert (O.coeff_g(p, y) > 0) == (B > (Q + 1.0) / 2.0)
    Y = O.candidates(p)
    assert Y == sorted(Y) and Y[-1] == 32
    y_min = min(y for y in range(1, 33) if O.coeff_g(p, y) > 0)
    assert Y[0] == y_min
    for y in range(y_min, 32):
        assert (y in Y) == (cap[y] > cap[y + 1])


# ---------------------------------------------------------------- error bound, Eq. (5)

def gamma_eq5(d, beta, B, cap, ys):
    """Eq. (5) packet by packet with libm pow; packet boundaries shifted by one so the
    first term d^beta - (k+1)^beta and the packet terms share their boundary."""
    Bc_inv = 1.0 - 1.0 / B
    D = d ** beta - 1.0
    Z = 0
    total = 0.0
    for y in ys:
        P = cap[y]
        Q = P / float((2 ** y - 1) ** 2)
        total += (Q / B ** 2 + Bc_inv ** 2) * ((Z + P + 1) ** beta - (Z + 1) ** beta) / D
        Z += P
    return (d ** beta - (Z + 1) ** beta) / D + total, Z


@pytest.mark.parametrize("beta", [-3.0, -0.5, -0.0078125, 0.4453125, 0.9])
def test_objective_is_eq5(beta):
    d = 1_200_000
    p = O.make_params(d, 40 * 12000)
    rc, s, R, cap = O.derive(p)
    rng = np.random.default_rng(11)
    Y = O.candidates(p)
    for _ in range(20):
        ys = sorted(rng.choice(Y, size=R).tolist(), reverse=True)        # y_1 >= ... >= y_R
        n = [0] * 33
        for y in ys:
            n[y] += 1
        F = O.objective(p, beta, n)
        g_ref, k = gamma_eq5(d, beta, p.scale_B, cap, ys)
        assert k <= d
        assert 1.0 - F == pytest.approx(g_ref, rel=1e-9, abs=1e-11)


def test_objective_closed_form_uniform_plan():
    d = 100_000
    p = O.make_params(d, 8 * 12000)
    rc, s, R, cap = O.derive(p)
    beta = -0.5
    for y in O.candidates(p):
        n = [0] * 33
        n[y] = R
        E = (O.powr(float(R * cap[y] + 1), beta) - 1.0) / (O.powr(float(d), beta) - 1.0)
        assert O.objective(p, beta, n) == pytest.approx(O.coeff_g(p, y) * E, rel=1e-14)


def test_objective_inadmissible_beyond_d():
    p = O.make_params(3000, 8 * 12000)
    rc, s, R, cap = O.derive(p)
    n = [0] * 33
    y = O.candidates(p)[0]
    n[y] = R
    assert R * cap[y] > 3000
    assert O.objective(p, -0.5, n) == -math.inf


# ---------------------------------------------------------------- length tuning vs brute force

def brute_force(p, beta):
    rc, s, R, cap = O.derive(p)
    Y = O.candidates(p)
    best, best_n, ties = -math.inf, None, 0
    for combo in itertools.combinations_with_replacement(Y, R):
        n = [0] * 33
        for y in combo:
            n[y] += 1
        F = O.objective(p, beta, n)
        if F > best:
            best, best_n, ties = F, n, 1
        elif F == best:
            ties += 1
    return best, best_n, ties


BRUTE_CASES = []
_rng = np.random.default_rng(2024)
for _ in range(60):
    BRUTE_CASES.append(dict(
        d=int(_rng.choice([5_000, 60_000, 1_000_000, 30_000_000])),
        R=int(_rng.integers(1, 6)),
        packet_bits=int(_rng.choice([512, 1024, 4096, 12000])),
        max_code_bits=int(_rng.integers(6, 12)),
        alpha_q=float(_rng.integers(-600, -10)) / 256.0,
        B=float(_rng.choice([1.0, 1.004, 1.05, 1.5])),
    ))


@pytest.mark.parametrize("case", BRUTE_CASES)
def test_length_tuning_equals_brute_force(case):
    """Theorem 1: pairwise-optimal packet sizes are globally optimal, so the tuner must
    land on the exhaustive optimum over all non-increasing length sequences."""
    if case["alpha_q"] == -0.5:
        case["alpha_q"] -= 1.0 / 256
    p = O.make_params(case["d"], case["R"] * case["packet_bits"], packet_bits=case["packet_bits"],
                      max_code_bits=case["max_code_bits"], scale_B=case["B"])
    rc, s, R, cap = O.derive(p)
    Y = O.candidates(p)
    if rc != O.ORC_OK or not Y or 2 * R * cap[Y[0]] > case["d"]:
        pytest.skip("constraint k <= d active or no usable length")
    beta = 2.0 * case["alpha_q"] + 1.0
    pl = O.plan_from_alpha(p, case["alpha_q"])
    bestF, best_n, ties = brute_force(p, beta)
    assert 1.0 - pl.gamma == pytest.approx(bestF, rel=0, abs=0) or pl.gamma == 1.0 - bestF
    if ties == 1:
        assert [pl.n_y[y] for y in range(33)] == best_n


def test_brute_force_cases_not_all_skipped():
    ran = 0
    for case in BRUTE_CASES:
        p = O.make_params(case["d"], case["R"] * case["packet_bits"], packet_bits=case["packet_bits"],
                          max_code_bits=case["max_code_bits"], scale_B=case["B"])
        rc, s, R, cap = O.derive(p)
        Y = O.candidates(p)
        if rc == O.ORC_OK and Y and 2 * R * cap[Y[0]] <= case["d"]:
            ran += 1
    assert ran >= 30


# ---- the same against an enumeration that knows nothing of the oracle's candidate list: every length
# 1 .. max_code_bits may be used, and every plan is scored by Eq. (5) written packet by packet with libm

ALL_LENGTH_CASES = []
_rng2 = np.random.default_rng(77)
while len(ALL_LENGTH_CASES) < 48:
    c = dict(d=int(_rng2.choice([4_000, 50_000, 2_000_000, 60_000_000])), R=int(_rng2.integers(1, 5)),
             packet_bits=int(_rng2.choice([384, 1024, 4096, 12000])), max_code_bits=int(_rng2.integers(4, 10)),
             alpha_q=float(_rng2.integers(-700, -8)) / 256.0, B=float(_rng2.choice([1.0, 1.002, 1.03, 1.4, 2.5])))
    if c["alpha_q"] != -0.5:
        ALL_LENGTH_CASES.append(c)
# scales right above (Q + 1) / 2 of some length: its coefficient is positive but tiny, and it still belongs to the plan
for _d, _pb, _y0, _eps, _aq in [(50_000, 1024, 3, 0.01, -0.3), (50_000, 1024, 3, 0.002, -0.7), (2_000_000, 4096, 3, 0.005, -0.25),
                                (60_000_000, 12000, 4, 0.01, -0.2), (4_000, 384, 2, 0.004, -0.4), (50_000, 1024, 3, 0.02, -1.2)]:
    _s = max(1, math.ceil(math.log2(_d)))
    _Q = ((_pb - 80) // (_s + _y0)) / float((2 ** _y0 - 1) ** 2)
    ALL_LENGTH_CASES.append(dict(d=_d, R=3, packet_bits=_pb, max_code_bits=9, alpha_q=_aq, B=max(1.0, (_Q + 1.0) / 2.0) * (1.0 + _eps),
                                 tiny_g=_y0))


@pytest.mark.parametrize("case", ALL_LENGTH_CASES)
def test_length_tuning_is_optimal_over_all_lengths(case):
    """Dropping the lengths with a non-positive coefficient and the lengths that fit no more records than the next
    longer one must not lose the optimum: the plan's gamma equals the minimum of Eq. (5) over every non-increasing
    sequence of lengths 1 .. max_code_bits (Theorem 1), and no sequence outside the plan's support does better."""
    p = O.make_params(case["d"], case["R"] * case["packet_bits"], packet_bits=case["packet_bits"],
                      max_code_bits=case["max_code_bits"], scale_B=case["B"])
    rc, s, R, cap = O.derive(p)
    if rc != O.ORC_OK:
        pytest.skip("packet too small")
    beta = 2.0 * case["alpha_q"] + 1.0
    try:
        pl = O.plan_from_alpha(p, case["alpha_q"])
    except O.OracleError as e:
        # no usable length at this scale, or even the longest code overshoots d: the enumeration agrees
        if e.code == O.ORC_ERR_BUDGET_TOO_LARGE:
            assert R * cap[case["max_code_bits"]] > case["d"]
        else:
            assert e.code == O.ORC_ERR_SCALE_TOO_SMALL
            assert all(O.coeff_g(p, y) <= 0 for y in range(1, case["max_code_bits"] + 1))
        return
    best = math.inf
    for combo in itertools.combinations_with_replacement(range(case["max_code_bits"], 0, -1), R):  # y_1 >= ... >= y_R
        if sum(cap[y] for y in combo) > case["d"]:
            continue
        g, _ = gamma_eq5(case["d"], beta, case["B"], cap, combo)
        best = min(best, g)
    assert pl.gamma == pytest.approx(best, rel=1e-9, abs=1e-12)
    if "tiny_g" in case:
        # B sits right above (Q + 1) / 2 of this length (Proposition 1's condition): it is the shortest usable one
        assert 0.0 < O.coeff_g(p, case["tiny_g"]) < 0.05 and pl.y_min == case["tiny_g"]


def test_all_length_cases_cover_pruned_lengths():
    """the enumeration above must meet instances where the pruning is active (some length below y_min, some
    length dominated); all of them leave the constraint k <= d slack (with it active the exchange rule is a
    heuristic: the candidate-list brute force above skips those instances for the same reason)"""
    below, dominated = 0, 0
    for case in ALL_LENGTH_CASES:
        p = O.make_params(case["d"], case["R"] * case["packet_bits"], packet_bits=case["packet_bits"],
                          max_code_bits=case["max_code_bits"], scale_B=case["B"])
        rc, s, R, cap = O.derive(p)
        if rc != O.ORC_OK:
            continue
        Y = O.candidates(p)
        if not Y:
            continue
        below += Y[0] > 1
        dominated += any(y not in Y for y in range(Y[0], case["max_code_bits"]))
        assert R * cap[1] <= case["d"]
    assert below >= 10 and dominated >= 5


# ---- which histogram bins enter the fit of the decay exponent (Definition 1): the non-empty normal bins
# 16 .. 4079 whose survival count N_j lies in 1 .. floor(d / 2)

def _fit_reference(h, d):
    """least squares of log2(bin edge) on log2(survival count) with numpy, over the window stated above"""
    h = np.asarray(h, dtype=np.int64)
    N = np.cumsum(h[::-1])[::-1]
    j = np.arange(4096)
    sel = (j >= 16) & (j <= 4079) & (h > 0) & (N >= 1) & (N <= d // 2)
    if sel.sum() < 2:
        return -1.0
    X = np.log2(N[sel].astype(np.float64))
    Y = ((j[sel] >> 4) - 127) + np.log2(1.0 + (j[sel] & 15) / 16.0)
    return float(np.polyfit(X, Y, 1)[0])


def _two_slope_histogram(d, seed):
    """ranks 1 .. d/2 follow |x| ~ l^-0.4, the lower half of the ranks falls off much faster (l^-3): a fit that lets
    points of the lower half in sees a different slope"""
    rng = np.random.default_rng(seed)
    l = np.arange(1, d + 1, dtype=np.float64)
    mag = np.where(l <= d // 2, l ** -0.4, (d // 2) ** -0.4 * (l / (d // 2)) ** -3.0) * 0.8
    x = (mag * rng.choice([-1.0, 1.0], d)).astype(np.float32)
    return x


def test_fit_window_upper_half_of_the_ranks():
    d = 300_000
    x = _two_slope_histogram(d, 3)
    rc, h = O.histogram(x)
    a, aq = O.alpha_fit(h, d)
    ref = _fit_reference(h, d)
    assert a == pytest.approx(ref, abs=1e-9)
    assert abs(a + 0.4) < 0.02
    # the same least squares over all non-empty bins gives a clearly different slope: the window matters here
    hh = np.asarray(h, dtype=np.int64)
    N = np.cumsum(hh[::-1])[::-1]
    j = np.arange(4096)
    sel = (j >= 16) & (j <= 4079) & (hh > 0)
    wide = np.polyfit(np.log2(N[sel].astype(np.float64)), ((j[sel] >> 4) - 127) + np.log2(1.0 + (j[sel] & 15) / 16.0), 1)[0]
    assert abs(wide - a) > 0.05


@pytest.mark.parametrize("which", ["bin15", "bin4080", "half_plus_one", "half_exact"])
def test_fit_window_edges(which):
    """one extra point right outside each edge of the window would change the slope; it must not be used, and the
    point right inside (N_j = floor(d/2)) must"""
    d = 1 << 16
    h = np.zeros(4096, dtype=np.uint64)
    # three points on an exact power law |x| = 2^-2 * l^-1/2 ... ranks 4^m at magnitude 2^-m: slope -1/2
    prev = 0
    for m in range(2, 6):
        h[(127 - m) << 4] = 4 ** m - prev
        prev = 4 ** m
    rest = d - prev
    if which == "bin15":            # the top subnormal bin, far off the line, N = prev + 7 <= d/2
        h[15] = 7
        rest -= 7
    elif which == "bin4080":        # a bin of exponent 255 (the histogram may carry it; the fit must not use it)
        h[4080] = 5
        rest -= 5
    elif which == "half_plus_one":  # a normal bin whose survival count is floor(d/2) + 1: outside
        h[(127 - 40) << 4] = d // 2 + 1 - prev
        rest -= d // 2 + 1 - prev
    else:                           # ... and with floor(d/2) exactly: inside, and it bends the fit
        h[(127 - 40) << 4] = d // 2 - prev
        rest -= d // 2 - prev
    h[0] += rest
    assert int(h.sum()) == d
    a, aq = O.alpha_fit(h, d)
    assert a == pytest.approx(_fit_reference(h, d), abs=1e-9)
    if which == "half_exact":
        assert abs(a + 0.5) > 0.5
    elif which == "bin4080":
        # the counts of the exponent-255 bin still add to every survival count below it: ranks are 5 higher
        assert abs(a + 0.5) < 0.1
    else:
        assert abs(a + 0.5) < 1e-9


# ---------------------------------------------------------------- plan invariants

PLAN_CASES = [
    ("tiny", 100_000, 1.0), ("small", 1_200_000, 2.0), ("r18_05", 11_200_000, 0.5),
    ("r18_2", 11_200_000, 2.0), ("r18_4", 11_200_000, 4.0), ("r50", 23_500_000, 1.0),
    ("stress", 100_000_000, 0.25),
]


@pytest.mark.parametrize("name,d,bpc", PLAN_CASES)
@pytest.mark.parametrize("alpha_q", [-1.5, -0.75, -0.27734375])
def test_plan_invariants(name, d, bpc, alpha_q):
    p = O.make_params(d, int(bpc * d))
    rc, s, R, cap = O.derive(p)
    pl = O.plan_from_alpha(p, alpha_q)
    n = [pl.n_y[y] for y in range(33)]
    assert sum(n) == R and n[0] == 0
    k = sum(n[y] * cap[y] for y in range(33))
    assert pl.k == k <= d
    assert R * cap[32] <= k <= R * cap[1]                               # k_min .. k_max bracket
    assert 0.0 < pl.gamma < 1.0                                          # Proposition 1
    beta = 2 * alpha_q + 1
    Y = O.candidates(p)
    for y in Y:                                                          # baselines are special cases
        u = [0] * 33
        u[y] = R
        Fu = O.objective(p, beta, u)
        assert 1.0 - pl.gamma >= Fu
    used = [y for y in range(33) if n[y]]
    assert all(y in Y for y in used)
    assert pl.B_next == 1.0 + max(O.quant_error_Q(p, y) for y in used)
    # packet sizes P_1 <= ... <= P_R  <=> lengths non-increasing: by construction of the layout;
    # the plan must use a contiguous-ish range where larger magnitude gets more bits
    assert used == sorted(used)


def test_gamma_non_increasing_in_budget():
    d = 1_200_000
    prev = 1.0
    for R in [1, 2, 5, 10, 50, 200, 800]:
        p = O.make_params(d, R * 12000, scale_B=1.0073)
        g = O.plan_from_alpha(p, -0.75).gamma
        assert g <= prev + 1e-15
        prev = g


def test_plan_uses_more_bits_for_larger_magnitudes_and_varies_length():
    p = O.make_params(11_200_000, 22_400_000)
    pl = O.plan_from_alpha(p, -0.75)
    used = [y for y in range(33) if pl.n_y[y]]
    assert len(used) >= 3                 # genuinely variable-length
    # counts fall off toward the long codes (few huge magnitudes, many small ones)
    assert pl.n_y[used[0]] + pl.n_y[used[1]] > pl.n_y[used[-1]]


def test_plan_fixed_is_uniform():
    p = O.make_params(100_000, 100_000)
    rc, s, R, cap = O.derive(p)
    pl = O.plan_fixed(p, 6)
    assert pl.n_y[6] == R and sum(pl.n_y) == R and pl.k == R * cap[6]
    with pytest.raises(O.OracleError):
        O.plan_fixed(p, 0)
    with pytest.raises(O.OracleError):
        O.plan_fixed(p, 33)


def test_plan_end_to_end_on_tiny_workload():
    w = W.WORKLOADS["tiny"]
    x = W.client_update(w, 0)
    p = O.make_params(w.d, w.budget_bits())
    pl = O.plan(x, p)
    rc, h = O.histogram(x)
    a, aq = O.alpha_fit(h, w.d)
    assert (pl.alpha, pl.alpha_q, pl.beta) == (a, aq, 2 * aq + 1)
    pl2 = O.plan_from_alpha(p, aq)
    assert [pl.n_y[y] for y in range(33)] == [pl2.n_y[y] for y in range(33)]
    assert pl.gamma == pl2.gamma
