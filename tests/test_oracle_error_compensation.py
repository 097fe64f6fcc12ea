"""Pins of the oracle's error-compensation step (Section II: Top_k with an error compensation mechanism; the
reading used here: the client compresses memory + update and keeps compensated - U_hat, U_hat being what the
parameter server rebuilds, i.e. the dequantized value divided by B on sent coordinates and zero elsewhere)."""
import numpy as np
import pytest

import oracle as O
from stream_reader import dequantize, dequantize_qsgd, parse
from test_oracle_codec import small_case


def sent_values(stream):
    """(PIDs, what the server rebuilds for them) from the independent stream reader"""
    S = parse(stream)
    pids = np.concatenate([pk.pid for pk in S.packets]).astype(np.int64)
    deq = dequantize_qsgd if S.quantizer == 1 else dequantize
    vals = np.concatenate([deq(pk) for pk in S.packets])
    return pids, (vals.astype(np.float64) / S.scale_B).astype(np.float32)


@pytest.mark.parametrize("quantizer", [0, 1])
def test_residual_is_what_the_server_does_not_get(quantizer):
    x, p = small_case(d=20000, R=12, quantizer=quantizer)
    st = O.encode(x, p, O.plan(x, p))
    m = O.ec_residual(x, st)
    pids, u_hat = sent_values(st)
    sent = np.zeros(x.size, bool)
    sent[pids] = True
    assert (m[~sent] == x[~sent]).all()                               # nothing sent: everything is kept
    assert (m[pids] == x[pids] - u_hat).all()                         # sent: one fp32 subtraction of the rebuilt value
    # compensated = rebuilt + memory, up to that one rounding
    rebuilt = np.zeros(x.size, np.float32)
    rebuilt[pids] = u_hat
    assert np.abs((rebuilt.astype(np.float64) + m) - x).max() <= 2.0 ** -24 * np.abs(x).max()


def test_exact_top_k_leaves_no_residual_on_sent_coordinates():
    """32-bit codes and B = 1 are plain Top_k: the memory is zero (to rounding) where a value was sent"""
    x, _ = small_case(d=20000, R=12)
    p = O.make_params(20000, 12 * 1024, packet_bits=1024, scale_B=1.0)
    pl = O.plan_fixed(p, 32)
    st = O.encode(x, p, pl)
    m = O.ec_residual(x, st)
    pids, _ = sent_values(st)
    assert np.abs(m[pids]).max() <= 2.0 ** -22 * np.abs(x).max()
    kept = np.ones(x.size, bool)
    kept[pids] = False
    assert np.abs(x[pids]).min() >= np.abs(x[kept]).max()            # and the sent ones are the largest


def test_updates_telescope_over_rounds():
    """over T rounds, everything the server rebuilt plus the final memory equals the sum of the updates: nothing is lost"""
    d, T = 8000, 6
    rng = np.random.default_rng(5)
    mem = np.zeros(d, np.float32)
    total_sent = np.zeros(d, np.float64)
    total_updates = np.zeros(d, np.float64)
    B = None
    for t in range(T):
        u = rng.laplace(0, 1e-2, d).astype(np.float32)
        total_updates += u
        a = O.ec_accumulate(mem, u)
        assert a is mem
        p = O.make_params(d, 5 * 1024, packet_bits=1024, seed=3, client_id=1, round=t, scale_B=B)
        pl = O.plan(a, p)
        st = O.encode(a, p, pl)
        pids, u_hat = sent_values(st)
        total_sent[pids] += u_hat
        mem = O.ec_residual(a, st)
        B = pl.B_next
    assert np.abs(total_sent + mem - total_updates).max() <= T * 2.0 ** -22 * np.abs(total_updates).max()
    # without the memory the unsent part is simply gone: the compensated run has rebuilt more of the total
    assert np.abs(mem).sum() > 0 and np.abs(total_sent).sum() > 0


def test_accumulate_is_an_fp32_sum():
    rng = np.random.default_rng(2)
    m = rng.standard_normal(1000).astype(np.float32)
    u = (rng.standard_normal(1000) * 1e-3).astype(np.float32)
    ref = m + u
    assert (O.ec_accumulate(m, u) == ref).all()


def test_residual_rejects_a_foreign_stream():
    x, p = small_case(d=20000, R=12)
    st = O.encode(x, p, O.plan(x, p))
    with pytest.raises(O.OracleError):
        O.ec_residual(x[:-1], st)                                      # another d
    bad = st.copy()
    bad[0] ^= 1
    with pytest.raises(O.OracleError):
        O.ec_residual(x, bad)
