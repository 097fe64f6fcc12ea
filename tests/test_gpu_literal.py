"""GPU parity of cvlc_plan_literal (problem P2 with real-valued packet sizes, plan only) with the CPU oracle:
the same grid of k, and for every k the same error bound, sweep count and packet sizes, bit for bit."""
import numpy as np
import pytest

import oracle as O
from gpu_util import f64_bits, gpu_params, oracle_params, params_dict

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def dev():
    import torch
    assert torch.cuda.is_available()
    from paper_2402_03770_b200 import binding as B
    B.lib()
    B.cvlc_set_device(0)
    return torch.device("cuda:0")


CASES = [  # d, R, packet bits, alpha_q, quantizer, n_k, max_sweeps
    (4000, 4, 2016, -0.75, 0, 9, 1 << 20),
    (100_000, 8, 12000, -0.75, 0, 17, 1 << 20),
    (20_000, 5, 1504, -0.40, 0, 33, 1 << 20),
    (80_000, 1, 4096, -0.8, 0, 41, 1 << 20),           # one packet: nothing to tune
    (50_000, 4, 2016, -0.6, 1, 7, 1 << 20),            # QSGD error factor
    (1_200_000, 16, 12000, -0.6, 0, 5, 1 << 20),
    (11_200_000, 64, 12000, -0.5390625, 0, 3, 60),     # 64 packets, sweeps cut short on both sides
    (300_000, 3, 4096, -1.3, 0, 1, 1 << 20),           # a single value of k
]


@pytest.mark.parametrize("d,R,b,alpha_q,quantizer,n_k,max_sweeps", CASES)
def test_literal_plan_matches_oracle(dev, d, R, b, alpha_q, quantizer, n_k, max_sweeps):
    from paper_2402_03770_b200 import binding as B
    pd = params_dict(d, R * b, packet_bits=b, quantizer=quantizer)
    ref = O.plan_literal(oracle_params(pd), alpha_q, n_k, max_sweeps)
    head, P_star, k_grid, gamma, sweeps = B.cvlc_plan_literal(gpu_params(pd), alpha_q, n_k, max_sweeps, dev)
    assert head.status == 0 and head.R == R and head.n_k == n_k
    assert (k_grid == ref.k_grid).all()
    assert (sweeps == ref.sweeps_of_k).all()
    assert (gamma.view(np.uint64) == ref.gamma_of_k.view(np.uint64)).all()
    assert head.k_star == ref.k_star and f64_bits(head.gamma_star) == f64_bits(ref.gamma_star)
    assert (P_star.view(np.uint64) == ref.P_star.view(np.uint64)).all()
    assert head.sweeps == int(ref.sweeps_of_k[int(np.argmin(ref.gamma_of_k))])


def test_literal_plan_refusals(dev):
    from paper_2402_03770_b200 import binding as B
    p = gpu_params(params_dict(100_000, 8 * 12000))
    for kw in (dict(alpha_q=0.1), dict(alpha_q=-0.5), dict(n_k=0), dict(n_k=5000), dict(max_sweeps=0)):
        a = dict(alpha_q=-0.75, n_k=3, max_sweeps=10)
        a.update(kw)
        with pytest.raises((B.CvlcError, AssertionError)):
            B.cvlc_plan_literal(p, a["alpha_q"], a["n_k"], a["max_sweeps"], dev)
    big = gpu_params(params_dict(100_000_000, 3000 * 12000))           # more packets than the kernel keeps on chip
    with pytest.raises(B.CvlcError) as e:
        B.cvlc_plan_literal(big, -0.75, 3, 10, dev)
    assert e.value.code == B.CVLC_ERR_INVALID_ARG
