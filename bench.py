#!/usr/bin/env python
"""Benchmark of the Fed-CVLC compression path on B200.

One step = one federated round's compression work for one batch of clients:
plan + encode of every client's fp32 update, then decode-aggregate of all their
streams into the dense averaged update.  Inputs are synthetic (seeded, shaped like
CNN updates) and resident in HBM when the timed region starts; the `e2e` figure
repeats the step with every update copied from pinned host memory and the
aggregate copied back inside the timed region.

    python bench.py --gpus 1 --steps 5 --warmup 3
    python bench.py --impl reference          # the CPU oracle, timed on the host cores
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time
from concurrent.futures import ThreadPoolExecutor

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2402_03770_b200 import workloads as W  # noqa: E402

METRIC = "encode+decode_aggregate throughput (4*d*clients / step time)"
UNIT = "GB/s"
FALLBACK_HBM_GBS = 6650.0

# dram__bytes_read.sum + dram__bytes_write.sum per client and launch, from one ncu capture of the kernels as they
# stand (resnet18 shape, 2 bits per coordinate, PQ, 32 clients per launch: working sets beyond the L2, traffic in
# proportion to the clients); scaled to the clients of a launch, None for any other configuration, for fewer than
# 32 clients per launch, and for a kernel that has changed since its capture.
NCU_TRAFFIC_BYTES_PER_CLIENT = {
    "k_hist": (1434.27e6 + 58.85e6) / 32,          # the update once, plus row maxima and per-segment histograms
    "k_select": (477.15e6 + 164.51e6) / 32,        # the rows that hold candidates (a third of the update), plus the candidates
    "k_sort_pass": (209.78e6 + 174.11e6 + 208.96e6 + 173.35e6 + 206.46e6 + 173.98e6 + 0.08e6) / 32 / 4,  # mean of a step's four launches
    "k_pack": (177.98e6 + 54.22e6) / 32,
}
NOMINAL_HBM_GBS = 8000.0

def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=5)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="resnet18")
    ap.add_argument("--bits-per-coord", type=float, default=2.0)
    ap.add_argument("--quantizer", default="pq", choices=["pq", "qsgd"], help="the two quantizers of the paper's experiments")
    ap.add_argument("--clients", type=int, default=0, help="0 = the workload's client count")
    ap.add_argument("--d", type=int, default=0, help="0 = the workload's d (smaller values are for profiling)")
    ap.add_argument("--batch", type=int, default=0, help="clients per plan/encode call; 0 = all clients in one call")
    ap.add_argument("--streams", type=int, default=2, help="CUDA streams the batches are spread over")
    ap.add_argument("--no-side-stream", action="store_true",
                    help="run the length tuning on the main stream instead of next to selection and ranking")
    ap.add_argument("--max-candidates", type=int, default=0,
                    help="candidate slots per client in the encode workspace; 0 = 3 * R * cap(1)")
    ap.add_argument("--profile-kernel", default="", help="kernel whose roofline is reported; default: the one with the largest total time")
    ap.add_argument("--e2e-steps", type=int, default=2)
    ap.add_argument("--e2e-batch", type=int, default=10, help="clients per call of the end-to-end leg: host-to-device copies of one sub-batch overlap the kernels of the previous ones")
    ap.add_argument("--e2e-streams", type=int, default=3)
    ap.add_argument("--cpu-sample-clients", type=int, default=3)
    ap.add_argument("--sustain-seconds", type=float, default=3.0,
                    help="after the timed steps, repeat the step back to back for this long and report the sustained rate (0 = skip)")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-e2e", action="store_true")
    return ap.parse_args()


def measured_hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    QUERY = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap,power.draw")

    def __init__(self, index: int, period_ms: int = 100):
        self.index = index
        self.period_ms = period_ms
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", str(self.period_ms)], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.thread = threading.Thread(target=self._read, daemon=True)
            self.thread.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def wait_first_sample(self, timeout_s: float = 3.0):
        """nvidia-smi takes a moment to start: wait until it has answered once"""
        t0 = time.time()
        while self.proc is not None and not self.lines and time.time() - t0 < timeout_s:
            time.sleep(0.01)

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in self.lines:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 6:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[2:6]):
                if val.lower().startswith("active"):
                    reasons.add(name)
            if len(parts) > 6:
                try:
                    power.append(float(parts[6]))
                except ValueError:
                    pass
        return {"sm_mhz": float(np.median(sm)) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "reasons": sorted(reasons), "samples": len(sm), "power_w_median": float(np.median(power)) if power else None,
                "power_w_max": max(power) if power else None}


# --------------------------------------------------------------------------------------------
# reference arm: the CPU oracle as it stands, on a bounded sample of the workload
# --------------------------------------------------------------------------------------------

QUANTIZERS = {"pq": 0, "qsgd": 1}


def host_info():
    """cores and CPU model of the host the oracle is timed on"""
    model = None
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.lower().startswith("model name"):
                    model = line.split(":", 1)[1].strip()
                    break
    except OSError:
        pass
    return {"host_cores": os.cpu_count(), "host_cpu": model}


def oracle_step(w, d, bpc, clients, quantizer=0):
    """plan + encode of `clients`, then decode-aggregate of their streams; returns seconds"""
    import oracle as O
    xs = [W.client_update(w, c, d=d) for c in clients]
    weights = W.client_weights(w)[[c % w.n_clients for c in clients]]
    t0 = time.perf_counter()
    streams = []
    for c, x in zip(clients, xs):
        seed, cid, rnd = W.philox_ids(w, c)
        p = O.make_params(d, int(np.floor(bpc * d)), seed=seed, client_id=cid, round=rnd, quantizer=quantizer)
        streams.append(O.encode(x, p, O.plan(x, p)))
    O.decode_aggregate(streams, weights, d)
    return time.perf_counter() - t0


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    w = W.WORKLOADS[args.workload]
    d = args.d or w.d
    n = max(1, args.cpu_sample_clients)
    clients = list(range(n))
    for _ in range(min(args.warmup, 1)):
        oracle_step(w, d, args.bits_per_coord, clients[:1], QUANTIZERS[args.quantizer])
    times = [oracle_step(w, d, args.bits_per_coord, clients, QUANTIZERS[args.quantizer]) for _ in range(args.steps)]
    t = float(np.mean(times))
    value = 4.0 * d * n / t / 1e9
    sample = f"{n} of {args.clients or w.n_clients} clients per step (plan+encode each, decode-aggregate of those {n})"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": t * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64 plan / f32 data", "data": "synthetic",
        "config": {"workload": f"{w.name} d={d} bits_per_coord={args.bits_per_coord} quantizer={args.quantizer}", "sample": sample},
        "cpu_baseline": dict({"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample}, **host_info()),
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "params_per_s": d * n / t,
    }))


# --------------------------------------------------------------------------------------------
# our arm
# --------------------------------------------------------------------------------------------

def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2402_03770_b200 import binding as B
    from paper_2402_03770_b200 import replica as R

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the compression path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    dev = torch.device("cuda", local_rank)
    B.lib()
    B.cvlc_set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    w = W.WORKLOADS[args.workload]
    d = args.d or w.d
    n_clients = args.clients or w.n_clients
    bpc = args.bits_per_coord
    budget = int(np.floor(bpc * d))
    first_client = R.replica_clients(rank, n_clients)[0]  # every rank is an independent replica with its own clients

    # ---- inputs: seeded host generation (threads; numpy releases the GIL), then HBM-resident
    with ThreadPoolExecutor(max_workers=min(16, os.cpu_count() or 4)) as ex:
        host_x = list(ex.map(lambda c: W.client_update(w, first_client + c, d=d), range(n_clients)))
    pinned = [torch.from_numpy(x).pin_memory() for x in host_x] if not args.no_e2e else None
    dev_x = [torch.from_numpy(x).to(dev) for x in host_x]
    weights = torch.from_numpy(W.client_weights(w)[[(first_client + c) % w.n_clients for c in range(n_clients)]].copy())

    params = []
    for c in range(n_clients):
        seed, cid, rnd = W.philox_ids(w, first_client + c)
        params.append(B.make_params(d, budget, seed=seed, client_id=cid, round=rnd, quantizer=QUANTIZERS[args.quantizer]))
    batch = args.batch or n_clients
    groups = [list(range(i, min(i + batch, n_clients))) for i in range(0, n_clients, batch)]
    n_streams = max(1, min(args.streams, len(groups)))
    streams = [torch.cuda.Stream(device=dev) for _ in range(n_streams)]
    side_streams = [None if args.no_side_stream else torch.cuda.Stream(device=dev) for _ in range(n_streams)]
    if args.max_candidates:
        max_cand = args.max_candidates
    else:
        s_bits = max(1, int(np.ceil(np.log2(d))))
        max_cand = min(d, 3 * (budget // 12000) * ((12000 - 80) // (s_bits + 1)))
    encoders = [B.BatchEncoder([params[c] for c in g], dev, max_candidates=max_cand) for g in groups]
    out_streams = [o for enc in encoders for o in enc.outs]
    agg = B.Aggregator(n_clients, d, dev)
    agg.set_clients(out_streams, weights)
    result = torch.empty(d, dtype=torch.float32, device=dev)
    result_host = torch.empty(d, dtype=torch.float32).pin_memory() if not args.no_e2e else None
    main = torch.cuda.current_stream(dev)
    done = [torch.cuda.Event() for _ in range(n_streams)]
    fork = torch.cuda.Event()

    # the end-to-end leg has its own, smaller sub-batches on a few streams, so that the copy of one
    # sub-batch runs under the kernels of the ones before it (same kernels, same results)
    if not args.no_e2e:
        eb = max(1, min(args.e2e_batch, n_clients))
        e2e_groups = [list(range(i, min(i + eb, n_clients))) for i in range(0, n_clients, eb)]
        e2e_streams = [torch.cuda.Stream(device=dev) for _ in range(max(1, min(args.e2e_streams, len(e2e_groups))))]
        e2e_side = [None if args.no_side_stream else torch.cuda.Stream(device=dev) for _ in e2e_streams]
        e2e_encoders = [B.BatchEncoder([params[c] for c in g], dev, max_candidates=max_cand) for g in e2e_groups]
        e2e_agg = B.Aggregator(n_clients, d, dev)
        e2e_agg.set_clients([o for enc in e2e_encoders for o in enc.outs], weights)
        e2e_done = [torch.cuda.Event() for _ in e2e_streams]

    def step(from_host: bool):
        g_list, s_list, e_list, a, dn, sd = (e2e_groups, e2e_streams, e2e_encoders, e2e_agg, e2e_done, e2e_side) if from_host else \
            (groups, streams, encoders, agg, done, side_streams)
        fork.record(main)
        for s in s_list:
            s.wait_event(fork)
        for gi, g in enumerate(g_list):
            s = s_list[gi % len(s_list)]
            if from_host:
                with torch.cuda.stream(s):
                    for c in g:
                        dev_x[c].copy_(pinned[c], non_blocking=True)
            e_list[gi].compress([dev_x[c] for c in g], stream=s, side_stream=sd[gi % len(s_list)])
        for s, e in zip(s_list, dn):
            e.record(s)
            main.wait_event(e)
        a.run(n_clients, result, stream=main)
        if from_host:
            result_host.copy_(result, non_blocking=True)

    def barrier():
        torch.cuda.synchronize(dev)
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize(dev)

    def timed(n_steps: int, from_host: bool):
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(n_steps + 1)]
        barrier()
        ev[0].record(main)
        for i in range(n_steps):
            step(from_host)
            ev[i + 1].record(main)
        barrier()
        total_ms = ev[0].elapsed_time(ev[-1])
        per = [ev[i].elapsed_time(ev[i + 1]) for i in range(n_steps)]
        total_ms = R.max_over_ranks(total_ms, dev)
        return total_ms, per

    # the clock sampler runs from before the warm-up to the end of the timed region, with no idle gap in between
    # (an idle GPU drops its clocks, and the first steps after a pause are slow)
    sampler = ClockSampler(local_rank, period_ms=25)   # the timed region is short: sample often
    if rank == 0:
        sampler.start()
        sampler.wait_first_sample()
    for _ in range(max(args.warmup, 3)):
        step(False)
    barrier()
    for enc in encoders:
        assert enc.status() == B.CVLC_OK, "encode reported a device-side error"
    assert agg.status() == B.CVLC_OK, "decode-aggregate reported a device-side error"

    per_step_launch_cap = 16 * len(groups) + 8 + 3 * (d // (24 << 20) + 1)  # decode: one fill + one launch per window
    B.cvlc_profile_select("*", per_step_launch_cap * args.steps)
    for _ in range(2):        # the GPU idled while the profiling events were created: two more untimed steps
        step(False)
    barrier()
    B.cvlc_profile_reset()    # the per-kernel times cover the timed steps only
    launches_before = B.cvlc_launch_count()
    total_ms, per = timed(args.steps, False)
    clocks = sampler.stop() if rank == 0 else None
    gpu_launches = B.cvlc_launch_count() - launches_before
    kernel_times = {}
    for name in B.KERNEL_NAMES:
        kn, kms = B.cvlc_profile_read(name)
        if kn:
            kernel_times[name] = (kn, kms)
    B.cvlc_profile_select(None, 0)

    ms_per_step = total_ms / args.steps
    units = d * n_clients * world

    # ---- the same step back to back for a few seconds: what the rate settles at under power and temperature
    sustained = None
    if args.sustain_seconds > 0:
        n_sus = max(args.steps, int(np.ceil(args.sustain_seconds * 1e3 / ms_per_step)))
        sampler2 = ClockSampler(local_rank)
        if rank == 0:
            sampler2.start()
        sus_ms, _ = timed(n_sus, False)
        clocks2 = sampler2.stop() if rank == 0 else None
        sustained = {"steps": n_sus, "seconds": sus_ms * 1e-3, "ms_per_step": sus_ms / n_sus,
                     "value": 4.0 * units / (sus_ms / n_sus * 1e-3) / 1e9, "unit": UNIT, "clocks": clocks2}

    # ---- what this GPU moves right now: a read-only pass and a copy over 4 GiB (library kernels, as a yardstick beside
    # the recorded peak: a read-only kernel of the path may exceed a peak that was measured with a copy)
    probe = None
    if rank == 0:
        n_probe = 1 << 30
        a = torch.empty(n_probe, dtype=torch.float32, device=dev).fill_(1.0)
        b = torch.empty_like(a)
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        best_copy = best_read = 0.0
        for _ in range(5):
            ev0.record(main); b.copy_(a); ev1.record(main); torch.cuda.synchronize(dev)
            best_copy = max(best_copy, 8.0 * n_probe / (ev0.elapsed_time(ev1) * 1e-3) / 1e9)
            ev0.record(main); a.sum(); ev1.record(main); torch.cuda.synchronize(dev)
            best_read = max(best_read, 4.0 * n_probe / (ev0.elapsed_time(ev1) * 1e-3) / 1e9)
        probe = {"copy_GBps": best_copy, "read_only_GBps": best_read, "how": "torch copy_ / sum over 2^30 fp32, best of 5, CUDA events"}
        del a, b
    value = 4.0 * units / (ms_per_step * 1e-3) / 1e9

    e2e = None
    if not args.no_e2e:
        step(True)
        e2e_ms, _ = timed(max(1, args.e2e_steps), True)
        e2e_ms /= max(1, args.e2e_steps)
        e2e = {"value": 4.0 * units / (e2e_ms * 1e-3) / 1e9, "unit": UNIT, "ms_per_step": e2e_ms,
               "h2d_bytes_per_step": 4 * d * n_clients, "d2h_bytes_per_step": 4 * d,
               "clients_per_call": eb, "streams": len(e2e_streams)}
        for enc in e2e_encoders:
            assert enc.status() == B.CVLC_OK, "encode reported a device-side error in the end-to-end leg"
        assert e2e_agg.status() == B.CVLC_OK

    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    # ---- per-kernel CUDA-event times of the timed region, and the roofline of the dominant kernel:
    # algorithmic bytes per launch / mean launch duration
    plans = [enc.read_plan(i) for enc in encoders for i in range(enc.n)]
    stream_bytes = B.cvlc_stream_bytes(params[0])
    n_groups = len(groups)
    sum_cand = float(sum(p.n_candidates for p in plans))
    sum_k = float(sum(p.k for p in plans))
    # digit passes that move a client's candidates: its sort key keytop - key has 19 bits below the histogram bins plus
    # the bits of the bin range between the threshold and the top bin; 9 bits per pass
    def moving_passes(p):
        bits = 19 + int(np.ceil(np.log2(max(1, p.top_bin + 1 - p.thresh_bin))))
        return min(4, (bits + 8) // 9)
    sort_bytes = float(sum(16.0 * p.n_candidates * moving_passes(p) for p in plans))
    alg_bytes_per_step = {   # algorithmic bytes all launches of one step move
        "k_hist": 4.0 * d * n_clients,
        "k_select": 4.0 * d * n_clients + 8.0 * sum_cand,
        "k_sort_hist": 8.0 * sum_cand,
        "k_sort_pass": sort_bytes,
        "k_pack": 8.0 * sum_k + float(n_clients) * stream_bytes,
        "k_decode": float(n_clients) * stream_bytes + 4.0 * d,
        "k_fill_zero": 4.0 * d,
    }
    peak, peak_kind = measured_hbm_peak()
    total_kernel_ms = sum(ms for _, ms in kernel_times.values())
    kernels = {}
    for name, (kn, kms) in sorted(kernel_times.items(), key=lambda kv: -kv[1][1]):
        entry = {"launches_per_step": kn / args.steps, "ms_per_step": kms / args.steps,
                 "share": kms / total_kernel_ms if total_kernel_ms else None}
        if name in alg_bytes_per_step:
            entry["achieved_GBps"] = alg_bytes_per_step[name] / (kms / args.steps * 1e-3) / 1e9
            entry["frac_of_hbm_peak"] = entry["achieved_GBps"] / peak
            entry["frac_of_nominal_8TBps"] = entry["achieved_GBps"] / NOMINAL_HBM_GBS
        kernels[name] = entry
    dominant = args.profile_kernel or (max(kernel_times.items(), key=lambda kv: kv[1][1])[0] if kernel_times else "")
    roofline = None
    if dominant in kernel_times:
        kn, kms = kernel_times[dominant]
        if dominant in alg_bytes_per_step:
            per_launch = alg_bytes_per_step[dominant] * args.steps / kn
            captured = (w.name == "resnet18" and d == w.d and bpc == 2.0 and args.quantizer == "pq"
                        and dominant in NCU_TRAFFIC_BYTES_PER_CLIENT and n_clients / n_groups >= 32)
            ncu_traffic = NCU_TRAFFIC_BYTES_PER_CLIENT[dominant] * n_clients / n_groups if captured else None
            achieved = per_launch / (kms / kn * 1e-3) / 1e9
            roofline = {"bound": "hbm", "kernel": dominant, "achieved": achieved, "peak": peak,
                        "peak_kind": f"of {peak_kind}", "unit": "GB/s", "frac": achieved / peak,
                        "frac_of_nominal_8TBps": achieved / NOMINAL_HBM_GBS,
                        "traffic": ncu_traffic, "launches_timed": kn,
                        "mean_launch_us": kms / kn * 1e3, "algorithmic_bytes_per_launch": per_launch}
        else:
            # the single-CTA-per-client planner: FP64 series arithmetic with O(1) data, bound by the
            # FP64 pipe of the SMs it occupies (64 FMA lanes per SM per clock)
            sm_max = (clocks or {}).get("sm_max_mhz") or 1965.0
            fp64_peak = 2.0 * 64 * 148 * sm_max * 1e6 / 1e12
            roofline = {"bound": "alu", "kernel": dominant, "achieved": None, "peak": fp64_peak, "unit": "TFLOP/s",
                        "frac": None, "traffic": None, "launches_timed": kn, "mean_launch_us": kms / kn * 1e3}
    # whole-step minimum bytes (read every update once, write every stream; read the streams, write the aggregate)
    step_min_bytes = n_clients * (4.0 * d + stream_bytes) + n_clients * stream_bytes + 4.0 * d
    step_frac = step_min_bytes / (ms_per_step * 1e-3) / 1e9 / peak
    # the same with every pass counted at its own minimum (histogram read, selection read + candidates, three
    # ranking passes, pack, decode): what this multi-pass design has to move
    pass_bytes = sum(alg_bytes_per_step[k] for k in ("k_hist", "k_select", "k_sort_pass", "k_pack", "k_decode"))
    pass_frac = pass_bytes / (ms_per_step * 1e-3) / 1e9 / peak
    pass_frac_nominal = pass_bytes / (ms_per_step * 1e-3) / 1e9 / NOMINAL_HBM_GBS

    cpu_baseline = None
    if world == 1 and not args.no_cpu_baseline:
        n_s = max(1, min(args.cpu_sample_clients, n_clients))
        t = oracle_step(w, d, bpc, list(range(n_s)), QUANTIZERS[args.quantizer])
        cpu_baseline = dict({"value": 4.0 * d * n_s / t / 1e9, "unit": UNIT, "cores": 1, "kind": "oracle",
                             "sample": f"{n_s} of {n_clients} clients: plan+encode each, decode-aggregate of those {n_s}; {t:.1f} s"},
                            **host_info())

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": max(args.warmup, 3),
        "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "f32 data / f64 plan+quantizer / u32 keys", "data": "synthetic",
        "config": {"workload": f"{w.name} d={d} clients={n_clients} bits_per_coord={bpc} quantizer={args.quantizer} packet=1500B",
                   "l2": "inputs (4*d*clients bytes per step) exceed L2", "streams": n_streams, "side_stream_for_length_tuning": not args.no_side_stream, "clients_per_call": batch, "max_candidates": int(max_cand),
                   "multi_gpu": "replicas only: every rank runs its own clients and aggregator"},
        "params_per_s": units / (ms_per_step * 1e-3),
        "step_min_bytes_frac_of_hbm_peak": step_frac,
        "step_pass_bytes_frac_of_hbm_peak": pass_frac,
        "step_pass_bytes_frac_of_nominal_8TBps": pass_frac_nominal,
        "step_pass_bytes": pass_bytes, "target_frac_of_hbm_peak": 0.5, "target_met": bool(pass_frac >= 0.5),
        "sustained": sustained, "hbm_probe": probe,
        "per_step_ms": per,
        "plan_of_client_0": {"k": int(plans[0].k), "R": int(plans[0].R), "n_candidates": int(plans[0].n_candidates), "alpha_q": plans[0].alpha_q,
                 "lengths": {str(y): int(plans[0].n_y[y]) for y in range(33) if plans[0].n_y[y]}},
        "phase_ms_per_step": {
            "plan": sum(kernels[k]["ms_per_step"] for k in ("k_zero_words", "k_hist", "k_plan_fit", "k_plan_tune", "k_plan_finish")
                        if k in kernels),
            "encode": sum(kernels[k]["ms_per_step"] for k in ("k_encode_init", "k_select", "k_select_lookback", "k_sort_hist",
                                                                "k_sort_scan", "k_sort_pass", "k_pack") if k in kernels),
            "decode_aggregate": sum(kernels[k]["ms_per_step"] for k in ("k_decode_prepare", "k_fill_zero", "k_decode")
                                    if k in kernels)},
        "step_min_bytes_frac_of_nominal_8TBps": step_min_bytes / (ms_per_step * 1e-3) / 8e12,
        "kernels": kernels, "roofline": roofline, "cpu_baseline": cpu_baseline, "e2e": e2e, "gpu_launches": int(gpu_launches),
        "clocks": clocks,
    }
    print(json.dumps(line))
    if world > 1:
        dist.destroy_process_group()


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
