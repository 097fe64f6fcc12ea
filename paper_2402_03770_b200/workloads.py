"""Seeded synthetic update vectors shaped like CNN model updates.

This module only draws random numbers; it contains none of the compression
method's arithmetic, so both the CPU oracle's tests and the CUDA path's tests
may import it.  Every generator returns host ``numpy.float32`` arrays.

The five workloads stand in for the model updates of the CNNs the paper trains
(Section V, "Models": 3e5 .. 5e6 parameters, 10 .. 90 packets of 1500 bytes per
client and round, 100 clients); the datasets and weights are not available, so
the magnitude distributions are synthetic: heavy-tailed, block-structured per
"layer", with the skew the paper's Definition 1 models.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Tuple

import numpy as np

PACKET_BITS = 12000  # 1500-byte packets (Section IV-C, "b = 1,500 bytes")
HEADER_BITS = 80


@dataclass(frozen=True)
class Workload:
    name: str
    d: int
    n_clients: int
    bits_per_coord: Tuple[float, ...]
    n_blocks: int
    data_seed0: int
    weights: str  # "uniform" or "samples"
    kind: str
    decode_batch: Optional[int] = None

    def budget_bits(self, bits_per_coord: Optional[float] = None) -> int:
        bpc = self.bits_per_coord[0] if bits_per_coord is None else bits_per_coord
        return int(np.floor(bpc * self.d))


WORKLOADS = {
    "tiny": Workload("tiny", 100_000, 1, (1.0,), 1, 0, "uniform", "laplace"),
    "small_cnn": Workload("small_cnn", 1_200_000, 20, (2.0,), 8, 1000, "uniform", "laplace_blocks"),
    "resnet18": Workload("resnet18", 11_200_000, 100, (0.5, 1.0, 2.0, 4.0), 62, 2000, "samples",
                         "gauss_blocks_outliers"),
    "resnet50": Workload("resnet50", 23_500_000, 50, (1.0,), 161, 3000, "uniform", "student_blocks_ties"),
    "stress": Workload("stress", 100_000_000, 200, (0.25,), 1, 4000, "uniform", "laplace", decode_batch=25),
}


def block_sizes(d: int, n_blocks: int, seed: int) -> np.ndarray:
    """Split ``d`` coordinates into ``n_blocks`` "layers".

    Raw layer weights are ``10**U(3, 6.5)``; sizes follow by largest-remainder
    apportionment so they sum to ``d`` exactly and every block is non-empty.
    """
    if n_blocks == 1:
        return np.array([d], dtype=np.int64)
    rng = np.random.default_rng(seed)
    w = 10.0 ** rng.uniform(3.0, 6.5, n_blocks)
    quota = w / w.sum() * (d - n_blocks)
    base = np.floor(quota).astype(np.int64)
    rem = int(d - n_blocks - base.sum())
    order = np.argsort(-(quota - base), kind="stable")
    base[order[:rem]] += 1
    sizes = base + 1
    assert sizes.sum() == d and (sizes > 0).all()
    return sizes


def client_update(w: Workload, client: int, d: Optional[int] = None) -> np.ndarray:
    """The fp32 update vector of one client (data seed ``data_seed0 + client``).

    ``d`` may shrink the workload (same recipe, fewer coordinates) for tests
    that need the structure but not the size.
    """
    d = w.d if d is None else int(d)
    rng = np.random.default_rng(w.data_seed0 + client)
    if w.kind == "laplace":
        return rng.laplace(0.0, 1e-3, d).astype(np.float32)
    sizes = block_sizes(d, w.n_blocks, seed=w.data_seed0 - 1)
    out = np.empty(d, dtype=np.float32)
    pos = 0
    nonzero_seen = 0
    for b, n in enumerate(sizes):
        n = int(n)
        if w.kind == "laplace_blocks":
            scale = 10.0 ** rng.uniform(-4.0, -2.0)
            blk = rng.laplace(0.0, scale, n)
        elif w.kind == "gauss_blocks_outliers":
            std = 10.0 ** rng.uniform(-5.0, -2.0)
            blk = rng.normal(0.0, std, n)
            n_out = int(round(n * 1e-3))
            if n_out:
                where = rng.choice(n, size=n_out, replace=False)
                blk[where] = 50.0 * std * rng.choice([-1.0, 1.0], size=n_out)
        elif w.kind == "student_blocks_ties":
            blk = 1e-3 * rng.standard_t(3.0, n)
            if b % 10 == 9:
                blk[:] = 0.0  # an all-zero layer
            else:
                nonzero_seen += 1
                if nonzero_seen % 7 == 0:
                    # exact ties in |x| of both signs: multiples of 2^-14
                    blk = np.round(blk * 16384.0) / 16384.0
        else:
            raise ValueError(w.kind)
        out[pos:pos + n] = blk.astype(np.float32)
        pos += n
    return out


def client_weights(w: Workload, n_clients: Optional[int] = None) -> np.ndarray:
    """Aggregation weights: uniform, or sample counts ~ U(50, 500) (seed 7)."""
    n = w.n_clients if n_clients is None else n_clients
    if w.weights == "uniform":
        return np.ones(n, dtype=np.float32)
    return np.random.default_rng(7).uniform(50.0, 500.0, w.n_clients).astype(np.float32)[:n]


def philox_ids(w: Workload, client: int) -> Tuple[int, int, int]:
    """(seed, client_id, round) handed to the stochastic quantizer for this client."""
    return (client, client, 0)


def power_law_vector(d: int, alpha: float, phi: float = 1.0, seed: int = 0) -> np.ndarray:
    """|x_l| = phi * l**alpha for rank l = 1..d, random signs, random positions."""
    rng = np.random.default_rng(seed)
    mag = phi * np.arange(1, d + 1, dtype=np.float64) ** alpha
    sign = rng.choice([-1.0, 1.0], size=d)
    x = (mag * sign).astype(np.float32)
    rng.shuffle(x)
    return x
