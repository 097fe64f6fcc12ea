"""Helpers of the GPU parity tests: run the CUDA path through the C ABI on numpy
inputs and run the oracle on the same inputs (possibly in worker processes)."""
from __future__ import annotations

import multiprocessing as mp
import os
from typing import List, Optional, Sequence, Tuple

import numpy as np

PARAM_FIELDS = ["d", "budget_bits", "packet_bits", "header_bits", "quantizer", "max_code_bits", "scale_B",
                "seed", "client_id", "round"]


def params_dict(d: int, budget_bits: int, **kw) -> dict:
    out = dict(d=int(d), budget_bits=int(budget_bits), packet_bits=12000, header_bits=80, quantizer=0,
               max_code_bits=32, scale_B=None, seed=0, client_id=0, round=0)
    out.update(kw)
    return out


def oracle_params(pd: dict):
    import oracle as O
    return O.make_params(pd["d"], pd["budget_bits"], packet_bits=pd["packet_bits"], header_bits=pd["header_bits"],
                         quantizer=pd["quantizer"], max_code_bits=pd["max_code_bits"], scale_B=pd["scale_B"],
                         seed=pd["seed"], client_id=pd["client_id"], round=pd["round"])


def gpu_params(pd: dict):
    from paper_2402_03770_b200 import binding as B
    return B.make_params(pd["d"], pd["budget_bits"], packet_bits=pd["packet_bits"], header_bits=pd["header_bits"],
                         quantizer=pd["quantizer"], max_code_bits=pd["max_code_bits"], scale_B=pd["scale_B"],
                         seed=pd["seed"], client_id=pd["client_id"], round=pd["round"])


# ---- oracle side (also used from spawned workers) -------------------------------------

def oracle_plan_encode(x: np.ndarray, pd: dict, fixed_y: int = 0):
    """returns (plan fields dict, stream bytes as np.uint8, histogram)"""
    import oracle as O
    p = oracle_params(pd)
    pl = O.plan_fixed(p, fixed_y) if fixed_y else O.plan(x, p)
    st = O.encode(x, p, pl)
    fields = dict(s=pl.s, R=pl.R, y_min=pl.y_min, n_lengths=pl.n_lengths, k=pl.k, alpha=pl.alpha,
                  alpha_q=pl.alpha_q, beta=pl.beta, gamma=pl.gamma, B_next=pl.B_next,
                  n_y=[pl.n_y[y] for y in range(33)], cap=[pl.cap[y] for y in range(33)])
    return fields, st


def _worker_encode(args):
    workload_name, client, d, bpc, fixed_y, quantizer = args
    from paper_2402_03770_b200 import workloads as W
    w = W.WORKLOADS[workload_name]
    x = W.client_update(w, client, d=d)
    seed, cid, rnd = W.philox_ids(w, client)
    pd = params_dict(x.size, int(np.floor(bpc * x.size)), seed=seed, client_id=cid, round=rnd, quantizer=quantizer)
    fields, st = oracle_plan_encode(x, pd, fixed_y)
    return client, fields, st


def oracle_encode_clients(workload_name: str, clients: Sequence[int], d: Optional[int], bpc: float,
                          fixed_y: int = 0, procs: Optional[int] = None, quantizer: int = 0):
    """Oracle plan+encode of several clients of a workload, in spawned worker processes."""
    jobs = [(workload_name, c, d, bpc, fixed_y, quantizer) for c in clients]
    procs = procs or min(len(jobs), max(1, (os.cpu_count() or 2) - 1), 32)
    if procs <= 1 or len(jobs) == 1:
        return [_worker_encode(j) for j in jobs]
    ctx = mp.get_context("spawn")
    with ctx.Pool(procs) as pool:
        return pool.map(_worker_encode, jobs, chunksize=1)


# ---- GPU side ----------------------------------------------------------------------------

def gpu_plan_encode(x: np.ndarray, pd: dict, fixed_y: int = 0, device: str = "cuda:0", want_hist: bool = False,
                    use_plan_ws: bool = True, compress: int = 0):
    """returns (status, CvlcPlan host copy, stream np.uint8[, histogram np.uint64]).
    compress: 0 = cvlc_plan then cvlc_encode; 1 = cvlc_compress_batch on one stream; 2 = with a side stream"""
    import torch
    from paper_2402_03770_b200 import binding as B
    dev = torch.device(device)
    p = gpu_params(pd)
    xd = torch.from_numpy(np.ascontiguousarray(x, dtype=np.float32)).to(dev)
    if compress:
        enc = B.BatchEncoder([p], dev)
        enc.outs[0].fill_(0xAB)  # the encoder must write every byte of the stream
        enc.plan = enc.plans
        side = torch.cuda.Stream(device=dev) if compress == 2 else None
        out = enc.compress([xd], side_stream=side, fixed_y=fixed_y)[0]
    else:
        enc = B.ClientEncoder(p, dev)
        enc.out.fill_(0xAB)
        out = enc.run(xd, fixed_y=fixed_y, use_plan_ws=use_plan_ws)
    status = enc.status()
    plan = B.read_plan(enc.plan)
    st = out.cpu().numpy().copy()
    if want_hist:
        h = enc.plan_ws[B.PLAN_WS_HIST_OFFSET:B.PLAN_WS_HIST_OFFSET + 8 * B.HIST_BINS].cpu().numpy().view(np.uint64).copy()
        return status, plan, st, h
    return status, plan, st


def gpu_decode_aggregate(streams: Sequence[np.ndarray], weights: np.ndarray, d: int, *, weight_total: float = 0.0,
                         out_init: Optional[np.ndarray] = None, accumulate: bool = False, device: str = "cuda:0"):
    import torch
    from paper_2402_03770_b200 import binding as B
    dev = torch.device(device)
    n = len(streams)
    dstreams = [torch.from_numpy(np.ascontiguousarray(s, dtype=np.uint8)).to(dev) for s in streams]
    agg = B.Aggregator(n, d, dev)
    agg.set_clients(dstreams, torch.from_numpy(np.ascontiguousarray(weights, dtype=np.float32)))
    if out_init is None:
        out = torch.full((d,), float("nan"), dtype=torch.float32, device=dev)  # must be overwritten
    else:
        out = torch.from_numpy(out_init.astype(np.float32)).to(dev)
    agg.run(n, out, weight_total=weight_total, accumulate=accumulate)
    status = agg.status()
    return status, out.cpu().numpy()


def f64_bits(v: float) -> int:
    return int(np.float64(v).view(np.uint64))


def assert_plan_equal(gp, of: dict):
    """bit-exact comparison of a GPU plan with the oracle's plan fields"""
    assert gp.status == 0
    assert (gp.s, gp.R, gp.y_min, gp.n_lengths, gp.k) == (of["s"], of["R"], of["y_min"], of["n_lengths"], of["k"])
    assert [gp.n_y[y] for y in range(33)] == of["n_y"]
    assert [gp.cap[y] for y in range(33)] == of["cap"]
    for name in ("alpha", "alpha_q", "beta", "gamma", "B_next"):
        assert f64_bits(getattr(gp, name)) == f64_bits(of[name]), (name, getattr(gp, name), of[name])


def assert_aggregate_close(got: np.ndarray, ref: np.ndarray):
    """fp32 aggregate: 1e-6 relative / 1e-7 absolute (summation order may differ)"""
    err = np.abs(got.astype(np.float64) - ref.astype(np.float64))
    tol = 1e-7 + 1e-6 * np.abs(ref.astype(np.float64))
    bad = err > tol
    assert not bad.any(), (int(bad.sum()), float(err.max()), int(np.argmax(err - tol)))
