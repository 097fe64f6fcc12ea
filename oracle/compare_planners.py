"""Error bound of the real-valued planner (problem P2) next to the integer-length rule, on the five workload shapes
with the packet count reduced to R (the sweeps of the real-valued tuning grow about with R^2).  CPU only: it calls
the oracle and the seeded input generator.

    python -m oracle.compare_planners [R] [n_k]
"""
from __future__ import annotations

import sys

import oracle as O
from paper_2402_03770_b200 import workloads as W


def main(R: int = 12, n_k: int = 33) -> None:
    print("| workload | d | alpha_q (client 0) | R | gamma, real-valued P2 (k*) | gamma, integer lengths (k) | ratio | sweeps at k* |")
    print("|---|---|---|---|---|---|---|---|")
    for name in ("tiny", "small_cnn", "resnet18", "resnet50", "stress"):
        w = W.WORKLOADS[name]
        d = w.d
        x = W.client_update(w, 0)
        rc, h = O.histogram(x)
        _, alpha_q = O.alpha_fit(h, x.size)
        p = O.make_params(d, R * 12000)
        plan = O.plan_from_alpha(p, alpha_q)
        lit = O.plan_literal(p, alpha_q, n_k)
        i = int(lit.gamma_of_k.argmin())
        print(f"| {name} | {d:,} | {alpha_q:.5f} | {R} | {lit.gamma_star:.6f} ({lit.k_star}) | {plan.gamma:.6f} ({plan.k}) | "
              f"{plan.gamma / lit.gamma_star:.4f} | {int(lit.sweeps_of_k[i])} |")


if __name__ == "__main__":
    a = [int(v) for v in sys.argv[1:]]
    main(*a)
