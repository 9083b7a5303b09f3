#!/usr/bin/env python
"""Benchmark of the BMGD hot path on B200.

A step is one buffer of the workload taken through the whole hot path: T rounds of shuffled
mini-batch gradient descent for every chain (one launch of the fused step kernel), theta carried
from step to step.  `value` is sample-gradients per second with all buffers already resident in
HBM; `e2e` is the same metric through load_buffer/run_rounds/get_theta with the buffers in pinned
host memory, the copy of buffer k+1 issued before the compute on buffer k.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2] [--impl reference]

Under torchrun every rank runs the same workload on its own GPU with its own shuffle seeds (the
chains are independent, so there is no collective on the data path); rank 0 prints one JSON line.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import torch  # noqa: E402

from paper_2312_08728_b200 import inputs  # noqa: E402
from paper_2312_08728_b200.inputs import WORKLOADS  # noqa: E402

METRIC = "bmgd_sample_grads_per_s"
UNIT = "sample-grads/s"
FALLBACK_HBM_GBS = 6650.0


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=30)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="cfg2", choices=sorted(WORKLOADS))
    ap.add_argument("--rounds", type=int, default=0, help="override T (cfg5 sweeps it)")
    ap.add_argument("--chains", type=int, default=0, help="override Rc")
    ap.add_argument("--buffers", type=int, default=0, help="use only the first B buffers of the workload")
    ap.add_argument("--cluster-size", type=int, default=0)
    ap.add_argument("--ctas-per-chain", type=int, default=0)
    ap.add_argument("--threads", type=int, default=0)
    ap.add_argument("--depth", type=int, default=0)
    ap.add_argument("--subpasses", type=int, default=0, help="sub-passes per ring stage")
    ap.add_argument("--lanes-per-row", type=int, default=0, help="lanes that share a row in the inner loop (0: library default)")
    ap.add_argument("--producer-warps", type=int, default=0, help="warps per CTA that only fetch rows (0: library default)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    return ap.parse_args()


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def workload_of(args):
    w = WORKLOADS[args.workload]
    if args.rounds:
        w = w.scaled(T=args.rounds)
    if args.chains:
        w = w.scaled(Rc=args.chains)
    return w


def peak_hbm():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def kernel_source_hash():
    """Hash of the CUDA sources: a recorded ncu figure is only reported while the kernels are unchanged."""
    h = hashlib.sha256()
    d = os.path.join(ROOT, "paper_2312_08728_b200", "csrc")
    for name in sorted(os.listdir(d)):
        with open(os.path.join(d, name), "rb") as f:
            h.update(name.encode())
            h.update(f.read())
    return h.hexdigest()[:16]


def recorded_traffic(workload):
    """DRAM bytes per launch from the committed ncu capture, if the kernels have not changed since."""
    try:
        with open(os.path.join(ROOT, "profiles", "traffic.json")) as f:
            rec = json.load(f).get(workload)
        if rec and rec.get("kernel_source_hash") == kernel_source_hash():
            return rec["dram_bytes_per_launch"]
    except Exception:
        pass
    return None


class ClockSampler:
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index):
        self.index = index
        self.proc = None

    def start(self):
        try:
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                 "-lms", "20"], stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2]))
            except ValueError:
                continue
            for name, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(name)
        note = None
        if not sm:  # the timed region was shorter than one sampling period: one reading taken right after it
            try:
                out = subprocess.run(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.QUERY}",
                                      "--format=csv,noheader,nounits"], capture_output=True, text=True, timeout=10).stdout
                f = [x.strip() for x in out.strip().split(",")]
                sm.append(float(f[1])); mx.append(float(f[2]))
                reasons.update(n for n, v in zip(names, f[5:9]) if v.lower().startswith("active"))
                note = "timed region shorter than the sampling period; read once right after it"
            except Exception:
                pass
        res = {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
               "samples": len(sm), "reasons": sorted(reasons)}
        if note:
            res["note"] = note
        return res


# ---------------------------------------------------------------------------------------------- reference arm

def oracle_rate(w, bufs, seconds, chains=1):
    """Time the CPU oracle, as it stands, on whole buffers of the workload until `seconds` have passed."""
    import numpy as np
    import oracle
    oloss = {inputs.LOSS_LINEAR: oracle.LINEAR, inputs.LOSS_LOGISTIC: oracle.LOGISTIC,
             inputs.LOSS_SOFTMAX: oracle.SOFTMAX}[w.loss]
    shape = (w.p, w.C) if w.loss == inputs.LOSS_SOFTMAX else (w.p,)
    th = np.zeros(shape)
    done = 0
    t0 = time.perf_counter()
    k = 0
    while True:
        X, y = bufs[k % len(bufs)]
        oracle.run_rounds(oloss, X, y, th, 1, w.n, w.lr, inputs.buffer_seed(w.seed, 0, k, w.K), chain=0, C=w.C)
        done += X.shape[0]
        k += 1
        el = time.perf_counter() - t0
        if el >= seconds or k >= 10_000:
            break
    return done / el, done, el, oracle.num_threads()


def run_reference(args, w):
    rank, world, _ = dist_env()
    if rank != 0:
        return
    import numpy as np
    import oracle
    nb = min(args.buffers or w.K, 2)
    bufs = [inputs.make_buffer(w, k) for k in range(nb)]
    oloss = {inputs.LOSS_LINEAR: oracle.LINEAR, inputs.LOSS_LOGISTIC: oracle.LOGISTIC,
             inputs.LOSS_SOFTMAX: oracle.SOFTMAX}[w.loss]
    shape = (w.p, w.C) if w.loss == inputs.LOSS_SOFTMAX else (w.p,)
    # one step = one round of one chain over a prefix of one buffer, sized from a short calibration
    th = np.zeros(shape)
    probe_rows = min(bufs[0][0].shape[0], 4 * w.n)
    t0 = time.perf_counter()
    oracle.run_rounds(oloss, bufs[0][0][:probe_rows], bufs[0][1][:probe_rows], th, 1, w.n, w.lr, 1, C=w.C)
    rate = probe_rows / max(time.perf_counter() - t0, 1e-6)
    budget = 120.0 / max(1, args.steps + args.warmup)
    rows = int(min(bufs[0][0].shape[0], max(w.n, rate * min(budget, 2.0))))
    rows = max(w.n, rows // w.n * w.n)
    th = np.zeros(shape)

    def step(i):
        X, y = bufs[i % nb]
        oracle.run_rounds(oloss, X[:rows], y[:rows], th, 1, w.n, w.lr, inputs.buffer_seed(w.seed, 0, i, w.K), C=w.C)

    for i in range(args.warmup):
        step(i)
    t0 = time.perf_counter()
    for i in range(args.steps):
        step(args.warmup + i)
    el = time.perf_counter() - t0
    value = args.steps * rows / el
    sample = f"one chain, one round over the first {rows} rows of a buffer per step"
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * el / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_of(args, w),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


def config_of(args, w):
    names = {0: "linear", 1: "logistic", 2: "softmax"}
    return {"workload": f"{w.name}: {names[w.loss]} regression, N={w.N}, p={w.p}, K={w.K} buffers of {w.N0} rows, "
                        f"n={w.n}, T={w.T}, lr={w.lr}, Rc={w.Rc}" + (f", C={w.C}" if w.C > 1 else ""),
            "step": "one buffer: T rounds x M mini-batch steps x Rc chains in one launch",
            "cache": "steps cycle through the workload's buffers; the buffer set is larger than L2 "
                     f"(a single buffer is not: its Rc*T = {w.Rc * w.T} re-reads per step are served by L2 by design)"
                     if w.Rc > 1 else "steps cycle through the workload's buffers; inputs larger than L2"}


# ---------------------------------------------------------------------------------------------- our arm

def run_ours(args, w):
    import numpy as np
    from paper_2312_08728_b200.binding import Bmgd, FLAG_NO_SLOTS, FLAG_TIMING
    rank, world, local = dist_env()
    extra_flags = 0
    multi = world > 1
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if multi:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    def barrier():
        if multi:
            dist.barrier()
        torch.cuda.synchronize(dev)

    nb = args.buffers or w.K
    host = [inputs.make_buffer(w, k) for k in range(nb)]
    seed0 = w.seed + rank * 1_000_003
    shape = dict(cluster_size=args.cluster_size, ctas_per_chain=args.ctas_per_chain, threads_per_cta=args.threads,
                 pipeline_depth=args.depth, subpasses_per_stage=args.subpasses, producer_warps=args.producer_warps, lanes_per_row=args.lanes_per_row)
    sg_per_step = [x.shape[0] * w.T * w.Rc for x, _ in host]

    # ---- device-resident measurement
    stream = torch.cuda.Stream(dev)
    resident = [(x.to(dev), y.to(dev)) for x, y in host]
    with torch.cuda.stream(stream):
        h = Bmgd(w.N, w.p, w.K, loss=w.loss, dtype=w.dtype, C=w.C, Rc=w.Rc, device=local,
                 flags=FLAG_NO_SLOTS | FLAG_TIMING | extra_flags, use_torch_stream=True, **shape)

        def step(i):
            x, y = resident[i % nb]
            h.run_rounds_resident(x, y, w.T, w.n, w.lr, inputs.buffer_seed(seed0, i // nb, i % nb, nb))

        for i in range(args.warmup):
            step(i)
        h.sync()
        s0 = h.get_stats()
        barrier()
        sampler = ClockSampler(local)
        if rank == 0:
            sampler.start()
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ev0.record(stream)
        for i in range(args.steps):
            step(args.warmup + i)
        ev1.record(stream)
        h.sync()
        barrier()
        clocks = sampler.stop() if rank == 0 else None
        ms = ev0.elapsed_time(ev1)
        s1 = h.get_stats()
        theta = h.get_theta(allow_nonfinite=True)
        h.close()
    sg = sum(sg_per_step[(args.warmup + i) % nb] for i in range(args.steps))
    launches = s1["launches"] - s0["launches"]
    kernel_ms = s1["kernel_ms"] - s0["kernel_ms"]
    t = torch.tensor([ms, kernel_ms], dtype=torch.float64, device=dev)
    if multi:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    ms, kernel_ms = float(t[0]), float(t[1])
    value = world * sg / (ms * 1e-3)

    # ---- end to end: pinned host -> HBM behind the compute, theta read back every step
    e2e = None
    if not args.no_e2e:
        pinned = [(x.pin_memory(), y.pin_memory()) for x, y in host]
        copy = torch.cuda.Stream(dev)
        with torch.cuda.stream(stream):
            h = Bmgd(w.N, w.p, w.K, loss=w.loss, dtype=w.dtype, C=w.C, Rc=w.Rc, device=local,
                     flags=FLAG_TIMING | extra_flags, use_torch_stream=True, **shape)
            total = args.warmup + args.steps
            e2e_s0 = None
            slot = h.load_buffer(*pinned[0], stream=copy)
            d2h = 0
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            for i in range(total):
                if i == args.warmup:
                    h.sync()
                    e2e_s0 = h.get_stats()
                    barrier()
                    e0.record(stream)
                nxt = h.load_buffer(*pinned[(i + 1) % nb], stream=copy) if i + 1 < total else None
                h.run_rounds(slot, w.T, w.n, w.lr, inputs.buffer_seed(seed0, i // nb, i % nb, nb))
                th = h.get_theta(allow_nonfinite=True)
                d2h = th.nbytes
                slot = nxt
            e1.record(stream)
            h.sync()
            barrier()
            ems = e0.elapsed_time(e1)
            e2e_s1 = h.get_stats()
            h.close()
        t = torch.tensor([ems], dtype=torch.float64, device=dev)
        if multi:
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
        ems = float(t[0])
        h2d = host[0][0].numel() * host[0][0].element_size() + host[0][1].numel() * host[0][1].element_size()
        e2e = {"value": world * sg / (ems * 1e-3), "unit": UNIT, "h2d_bytes_per_step": int(h2d),
               "d2h_bytes_per_step": int(d2h), "ms_per_step": ems / args.steps,
               "kernel_ms_per_step": (e2e_s1["kernel_ms"] - e2e_s0["kernel_ms"]) / args.steps,
               "h2d_ms_per_step": (e2e_s1["h2d_ms"] - e2e_s0["h2d_ms"]) / args.steps}
        # the copy of buffer k+1 runs behind the kernel on buffer k: hidden when the step costs no more than the kernel
        e2e["h2d_hidden"] = bool(e2e["ms_per_step"] <= 1.05 * max(e2e["kernel_ms_per_step"], 1e-9) + 0.05)

    if rank != 0:
        if multi:
            dist.destroy_process_group()
        return

    peak, peak_kind = peak_hbm()
    bytes_per_launch = (sg / args.steps) * w.row_bytes
    kdur = kernel_ms / max(1, launches) * 1e-3
    achieved = bytes_per_launch / kdur / 1e9 if kdur > 0 else None
    roofline = {"bound": "hbm", "achieved": achieved, "peak": peak, "peak_kind": peak_kind, "unit": "GB/s",
                "frac": achieved / peak if achieved else None, "frac_of_nominal_8TBps": achieved / 8000.0 if achieved else None,
                "traffic": recorded_traffic(w.name), "kernel": "glm_kernel" if w.loss != inputs.LOSS_SOFTMAX else "softmax_kernel",
                "kernel_ms_per_launch": kdur * 1e3, "algorithmic_bytes_per_launch": bytes_per_launch,
                "us_per_minibatch_step": 1e3 * kernel_ms / max(1, (s1["steps"] - s0["steps"]) / w.Rc),
                "launch_shape": {k: s1[k] for k in ("grid_ctas", "cluster_size", "ctas_per_chain", "threads_per_cta",
                                                    "pipeline_depth", "subpasses_per_stage", "smem_bytes",
                                                    "chains_in_flight")}}
    if w.loss == inputs.LOSS_SOFTMAX:
        flops = 4.0 * w.p * 16 * (sg / args.steps)  # both contractions, classes padded to 16
        roofline["tensor_tflops"] = flops / kdur / 1e12 if kdur > 0 else None
        roofline["note"] = ("bf16 tcgen05 contractions (M=128, N=16, K=16); the step is bound by its two cluster "
                            "barriers and the gather, not by the tensor pipe or HBM")
    if w.Rc > 1:
        roofline["note"] = (f"one {w.N0 * w.p * w.x_itemsize / 1e6:.0f} MB buffer is re-read Rc*T = {w.Rc * w.T} times per launch "
                            "and stays in the 126 MB L2, so algorithmic bytes per second may exceed the HBM peak; "
                            "DRAM traffic is in `traffic`")

    cpu = None
    if not args.no_cpu and world == 1:
        rate, done, el, cores = oracle_rate(w, host[:1], args.cpu_seconds)
        cpu = {"value": rate, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": f"chain 0, whole rounds over buffer 0 ({host[0][0].shape[0]} rows) repeated for "
                         f"{el:.1f} s = {done} sample-gradients"}

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
        "ms_per_step": ms / args.steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": {0: "f64", 1: "f32", 2: "bf16"}[w.dtype], "data": "synthetic",
        "config": config_of(args, w), "clocks": clocks, "e2e": e2e, "gpu_launches": int(launches),
        "roofline": roofline, "cpu_baseline": cpu,
        "theta_check": {"finite": bool(np.isfinite(theta).all()), "mean": float(theta.mean())},
    }
    print(json.dumps(line), flush=True)
    if multi:
        dist.destroy_process_group()


def main():
    args = parse_args()
    w = workload_of(args)
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
