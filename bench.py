#!/usr/bin/env python
"""Benchmark of the BMGD hot path on B200.

A step is one buffer of the workload taken through the whole hot path: T rounds of shuffled
mini-batch gradient descent for every chain (one launch of the fused step kernel), theta carried
from step to step.  `value` is sample-gradients per second with all buffers already resident in
HBM; `e2e` is the same metric through load_buffer/run_rounds/get_theta with the buffers in pinned
host memory, the copy of buffer k+1 issued before the compute on buffer k.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload cfg2] [--impl reference]

The headline workload is cfg2 (64 replicate chains).  On one GPU the same run also measures the
single-chain workloads (cfg3, cfg5 at T = 5, cfg4, cfg1) and reports them under "workloads", each
with its own roofline entry and, beside it, the time per step of the kernel's latency probe (the
step's waits, exchanges and updates without any rows): the floor under a chain of dependent steps.

With --gpus N and no WORLD_SIZE in the environment this script starts the N ranks itself (one
process per GPU); under torchrun it is one of them.  Rank r works on chains r*Rc .. (r+1)*Rc - 1 of a
job with N*Rc chains (the chains are independent, so there is no collective on the data path; theta is
gathered once at the end); rank 0 prints one JSON line.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import math
import os
import socket
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
L2_BYTES = 126e6
# single-chain workloads measured beside the headline on one GPU: (name, buffers kept resident, overrides)
# sim41-K2-n1000-a: the paper's simulation with two buffers of 50,000 x 500 (100 MB each, 100 chains): the replicate-chain
# launch whose buffer does not fit L2
EXTRA_WORKLOADS = (("cfg3", 2, {}), ("cfg5", 2, {"T": 5}), ("cfg4", 2, {}), ("cfg1", 5, {}), ("sim41-K2-n1000-a", 2, {}))
EXTRA_SECONDS = 0.6   # timed region of each of them


def parse_args(argv=None):
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
    ap.add_argument("--no-extra", action="store_true", help="measure only the named workload, not the single-chain ones beside it")
    ap.add_argument("--cpu-seconds", type=float, default=15.0)
    return ap.parse_args(argv)


def dist_env():
    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    return rank, world, local


def free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def spawn_ranks(args, argv):
    """`--gpus N` outside torchrun: start the N ranks of this script on this node and wait for them."""
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
           "--master-addr", "127.0.0.1", "--master-port", str(free_port()), os.path.abspath(__file__)] + list(argv)
    return subprocess.call(cmd)


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
    """nvidia-smi sampling SM clocks and throttle reasons for the whole run; windows are cut out by wall-clock time."""
    QUERY = ("timestamp,index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, index):
        self.index = index
        self.proc = None
        self.rows = None

    def start(self):
        try:
            cmd = ["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                   "-lms", "20"]
            import shutil
            if shutil.which("stdbuf"):  # line-buffered, so that the lines of the last window are not lost in the pipe
                cmd = ["stdbuf", "-oL"] + cmd
            self.proc = subprocess.Popen(cmd, stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    @staticmethod
    def _parse(line):
        f = [x.strip() for x in line.split(",")]
        if len(f) < 10:
            return None
        try:
            t = time.mktime(time.strptime(f[0][:19], "%Y/%m/%d %H:%M:%S")) + float("0" + f[0][19:] if len(f[0]) > 19 else 0)
            return t, float(f[2]), float(f[3]), [n for n, v in zip(ClockSampler.NAMES, f[6:10]) if v.lower().startswith("active")]
        except ValueError:
            return None

    def stop(self):
        if self.proc is None:
            self.rows = []
            return
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        self.rows = [r for r in (self._parse(line) for line in out.splitlines()) if r]

    def read_once(self):
        try:
            out = subprocess.run(["nvidia-smi", f"--id={self.index}", f"--query-gpu={self.QUERY}",
                                  "--format=csv,noheader,nounits"], capture_output=True, text=True, timeout=10).stdout
            return self._parse(out.strip())
        except Exception:
            return None

    def window(self, t0, t1, fallback=None):
        """Summary of the samples taken between wall-clock times t0 and t1 (call after stop())."""
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        rows = [r for r in self.rows if t0 - 0.02 <= r[0] <= t1 + 0.02]
        note = None
        if not rows and fallback is not None:
            rows = [fallback]
            note = "no sampler line inside the timed region; read once right after it"
        res = {"sm_mhz": statistics.median(r[1] for r in rows) if rows else None,
               "sm_max_mhz": max(r[2] for r in rows) if rows else None, "samples": len(rows),
               "reasons": sorted({n for r in rows for n in r[3]})}
        if note:
            res["note"] = note
        return res


def config_of(w):
    names = {0: "linear", 1: "logistic", 2: "softmax"}
    return {"workload": f"{w.name}: {names[w.loss]} regression, N={w.N}, p={w.p}, K={w.K} buffers of {w.N0} rows, "
                        f"n={w.n}, T={w.T}, lr={w.lr}, Rc={w.Rc}" + (f", C={w.C}" if w.C > 1 else ""),
            "step": "one buffer: T rounds x M mini-batch steps x Rc chains in one launch",
            "cache": "steps cycle through the workload's buffers; the buffer set is larger than L2 "
                     f"(a single buffer is not: its Rc*T = {w.Rc * w.T} re-reads per step are served by L2 by design)"
                     if w.Rc > 1 else "steps cycle through the workload's buffers; inputs larger than L2"}


# ---------------------------------------------------------------------------------------------- reference arm

def oracle_consts(w):
    import oracle
    oloss = {inputs.LOSS_LINEAR: oracle.LINEAR, inputs.LOSS_LOGISTIC: oracle.LOGISTIC,
             inputs.LOSS_SOFTMAX: oracle.SOFTMAX}[w.loss]
    shape = (w.p, w.C) if w.loss == inputs.LOSS_SOFTMAX else (w.p,)
    return oloss, shape


def oracle_rate(w, bufs, seconds):
    """Time the CPU oracle, as it stands, on whole rounds over whole buffers of the workload until `seconds` have passed."""
    import numpy as np
    import oracle
    oloss, shape = oracle_consts(w)
    th = np.zeros(shape)
    X, y = bufs[0]
    oracle.run_rounds(oloss, X[:4 * w.n], y[:4 * w.n], np.zeros(shape), 1, w.n, w.lr, 1, C=w.C)  # threads started
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
    """The CPU oracle, unchanged, on the same workload, metric and unit.  A step is `rounds` rounds of one chain over
    the first `rows` rows of a buffer, sized from a short calibration so that the timed region lasts at least two
    seconds and the whole run at most a couple of minutes."""
    rank, world, _ = dist_env()
    if rank != 0:
        return
    import numpy as np
    import oracle
    if world > 1:  # the launcher of the ranks pins OpenMP to one thread; the oracle gets the host's cores as at N = 1
        oracle.set_num_threads(len(os.sched_getaffinity(0)))
    nb = min(args.buffers or w.K, 2)
    bufs = [inputs.make_buffer(w, k) for k in range(nb)]
    oloss, shape = oracle_consts(w)
    th = np.zeros(shape)
    N0 = bufs[0][0].shape[0]
    probe_rows = min(N0, 4 * w.n)
    oracle.run_rounds(oloss, bufs[0][0][:probe_rows], bufs[0][1][:probe_rows], th, 1, w.n, w.lr, 1, C=w.C)  # threads started
    t0 = time.perf_counter()
    reps = 0
    while time.perf_counter() - t0 < 0.5:
        oracle.run_rounds(oloss, bufs[0][0][:probe_rows], bufs[0][1][:probe_rows], th, 1, w.n, w.lr, 1, C=w.C)
        reps += 1
    rate = reps * probe_rows / (time.perf_counter() - t0)
    per_step = min(max(2.5 / max(1, args.steps), 0.1), 100.0 / max(1, args.steps + args.warmup))
    work = max(w.n, rate * per_step)  # sample-gradients per step
    if work <= N0:
        rows, rounds = max(w.n, min(N0, int(work) // w.n * w.n)), 1
    else:
        rows, rounds = N0, int(math.ceil(work / N0))
    th = np.zeros(shape)

    def step(i):
        X, y = bufs[i % nb]
        oracle.run_rounds(oloss, X[:rows], y[:rows], th, rounds, w.n, w.lr, inputs.buffer_seed(w.seed, 0, i, w.K), C=w.C)

    for i in range(args.warmup):
        step(i)
    t0 = time.perf_counter()
    for i in range(args.steps):
        step(args.warmup + i)
    el = time.perf_counter() - t0
    value = args.steps * rows * rounds / el
    sample = (f"one chain, {rounds} round(s) over the first {rows} rows of a buffer per step; "
              f"{args.steps} steps timed for {el:.2f} s")
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * el / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": config_of(w),
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle.num_threads(), "kind": "oracle",
                         "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ---------------------------------------------------------------------------------------------- our arm

class Runner:
    """Measures workloads on this rank's GPU through the library's public calls."""

    def __init__(self, args):
        self.args = args
        self.rank, self.world, self.local = dist_env()
        self.multi = self.world > 1
        torch.cuda.set_device(self.local)
        self.dev = torch.device("cuda", self.local)
        if self.multi:
            import torch.distributed as dist
            dist.init_process_group("nccl", device_id=self.dev)
        self.stream = torch.cuda.Stream(self.dev)
        self.peak, self.peak_kind = peak_hbm()
        self.launches = 0

    def barrier(self):
        if self.multi:
            import torch.distributed as dist
            dist.barrier()
        torch.cuda.synchronize(self.dev)

    def max_over_ranks(self, values):
        t = torch.tensor(values, dtype=torch.float64, device=self.dev)
        if self.multi:
            import torch.distributed as dist
            dist.all_reduce(t, op=dist.ReduceOp.MAX)
        return [float(v) for v in t]

    def measure(self, w, nb, steps, warmup, seconds=None, e2e=True, e2e_steps=None, shape=None, sampler=None):
        """Resident and end-to-end measurement of workload `w` on its first `nb` buffers.

        `seconds`: size the timed region from a pilot so that it lasts about that long (instead of `steps`)."""
        import numpy as np
        from paper_2312_08728_b200.binding import Bmgd, BmgdError, ERR_UNIMPLEMENTED, FLAG_NO_SLOTS, FLAG_TIMING
        shape = shape or {}
        dev, stream, rank, world = self.dev, self.stream, self.rank, self.world
        host = [inputs.make_buffer(w, k) for k in range(nb)]
        # rank r works on chains r*Rc .. (r+1)*Rc - 1 of a job with world*Rc chains
        first_chain = rank * w.Rc
        seed0 = w.seed
        kw = dict(loss=w.loss, dtype=w.dtype, C=w.C, Rc=w.Rc, device=self.local, use_torch_stream=True,
                  first_chain=first_chain, **shape)
        rows_of = [x.shape[0] for x, _ in host]
        M_of = [-(-r // w.n) for r in rows_of]

        # ---- buffers resident in HBM
        resident = [(x.to(dev), y.to(dev)) for x, y in host]
        with torch.cuda.stream(stream):
            h = Bmgd(w.N, w.p, w.K, flags=FLAG_NO_SLOTS | FLAG_TIMING, **kw)

            def step(i):
                x, y = resident[i % nb]
                h.run_rounds_resident(x, y, w.T, w.n, w.lr, inputs.buffer_seed(seed0, i // nb, i % nb, nb))

            for i in range(warmup):
                step(i)
            h.sync()
            if seconds is not None:  # a pilot sizes the timed region
                p0 = h.get_stats()
                for i in range(3):
                    step(warmup + i)
                h.sync()
                pilot_ms = (h.get_stats()["kernel_ms"] - p0["kernel_ms"]) / 3
                steps = int(min(20_000, max(5, math.ceil(seconds * 1e3 / max(pilot_ms, 1e-3)))))
                warmup += 3
            s0 = h.get_stats()
            self.barrier()
            ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            t_wall0 = time.time()
            ev0.record(stream)
            for i in range(steps):
                step(warmup + i)
            ev1.record(stream)
            h.sync()
            t_wall1 = time.time()
            # one reading right after the timed region, used if the sampler's own lines for this window are missing (a
            # region shorter than the sampling period, or the tail of the sampler's output lost in its pipe)
            once = sampler.read_once() if sampler is not None else None
            self.barrier()
            ms = ev0.elapsed_time(ev1)
            s1 = h.get_stats()
            theta = h.get_theta(allow_nonfinite=True)
            # ---- the latency probe in the same launch shape: the step's waits, exchanges and updates without rows
            sync_us = None
            try:
                h.debug_null_rounds(rows_of[0], w.T, w.n)
                h.sync()
                n0 = h.get_stats()
                reps = 3
                for _ in range(reps):
                    h.debug_null_rounds(rows_of[0], w.T, w.n)
                h.sync()
                n1 = h.get_stats()
                sync_us = 1e3 * (n1["kernel_ms"] - n0["kernel_ms"]) / reps / (w.T * M_of[0])
                probe_launches = 1 + reps
            except BmgdError as e:
                if e.status != ERR_UNIMPLEMENTED:
                    raise
                probe_launches = 0
            h.close()
        sg = sum(rows_of[(warmup + i) % nb] * w.T * w.Rc for i in range(steps))
        launches = s1["launches"] - s0["launches"]
        kernel_ms = s1["kernel_ms"] - s0["kernel_ms"]
        ms, kernel_ms = self.max_over_ranks([ms, kernel_ms])
        self.launches += launches
        value = world * sg / (ms * 1e-3)

        # ---- end to end: pinned host -> HBM behind the compute, theta read back every step
        e2e_res = None
        if e2e:
            n_e2e = e2e_steps or steps
            pinned = [(x.pin_memory(), y.pin_memory()) for x, y in host]
            copy = torch.cuda.Stream(dev)
            with torch.cuda.stream(stream):
                h = Bmgd(w.N, w.p, w.K, flags=FLAG_TIMING, **kw)
                total = warmup + n_e2e
                e2e_s0 = None
                slot = h.load_buffer(*pinned[0], stream=copy)
                d2h = 0
                e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                for i in range(total):
                    if i == warmup:
                        h.sync()
                        e2e_s0 = h.get_stats()
                        self.barrier()
                        e0.record(stream)
                    nxt = h.load_buffer(*pinned[(i + 1) % nb], stream=copy) if i + 1 < total else None
                    h.run_rounds(slot, w.T, w.n, w.lr, inputs.buffer_seed(seed0, i // nb, i % nb, nb))
                    th = h.get_theta(allow_nonfinite=True)
                    d2h = th.nbytes
                    slot = nxt
                e1.record(stream)
                h.sync()
                self.barrier()
                ems = e0.elapsed_time(e1)
                e2e_s1 = h.get_stats()
                h.close()
            ems, = self.max_over_ranks([ems])
            sg_e2e = sum(rows_of[(warmup + i) % nb] * w.T * w.Rc for i in range(n_e2e))
            h2d = host[0][0].numel() * host[0][0].element_size() + host[0][1].numel() * host[0][1].element_size()
            e2e_res = {"value": world * sg_e2e / (ems * 1e-3), "unit": UNIT, "h2d_bytes_per_step": int(h2d),
                       "d2h_bytes_per_step": int(d2h), "steps": n_e2e, "ms_per_step": ems / n_e2e,
                       "kernel_ms_per_step": (e2e_s1["kernel_ms"] - e2e_s0["kernel_ms"]) / n_e2e,
                       "h2d_ms_per_step": (e2e_s1["h2d_ms"] - e2e_s0["h2d_ms"]) / n_e2e}
            # the copy of buffer k+1 runs behind the kernel on buffer k: hidden when the step costs no more than the kernel
            e2e_res["h2d_hidden"] = bool(e2e_res["ms_per_step"] <= 1.05 * max(e2e_res["kernel_ms_per_step"], 1e-9) + 0.05)
            self.launches += e2e_s1["launches"] - e2e_s0["launches"]

        # ---- roofline of the step kernel
        bytes_per_launch = (sg / steps) * w.row_bytes
        kdur = kernel_ms / max(1, launches) * 1e-3
        achieved = bytes_per_launch / kdur / 1e9 if kdur > 0 else None
        us_step = 1e3 * kernel_ms / max(1, (s1["steps"] - s0["steps"]) / w.Rc)
        buffer_bytes = rows_of[0] * w.row_bytes
        traffic = recorded_traffic(w.name)
        # Which memory serves the bytes.  A buffer that fits L2 and is swept Rc*T times per launch comes from L2 after
        # its first sweep (ncu: DRAM traffic per launch = one buffer); the algorithmic figure is then a throughput
        # expressed in HBM units, not an HBM utilisation.
        l2_served = (buffer_bytes < 0.6 * L2_BYTES and w.Rc * w.T > 1) or (traffic is not None and traffic < 0.5 * bytes_per_launch)
        roofline = {"bound": "l2" if l2_served else "hbm", "achieved": achieved, "peak": self.peak,
                    "peak_kind": self.peak_kind + " HBM copy bandwidth", "unit": "GB/s",
                    "frac": achieved / self.peak if achieved else None,
                    "frac_of_nominal_8TBps": achieved / 8000.0 if achieved else None,
                    "algorithmic_gbs": achieved, "traffic": traffic,
                    "kernel": "glm_kernel" if w.loss != inputs.LOSS_SOFTMAX else "softmax_kernel",
                    "kernel_ms_per_launch": kdur * 1e3, "algorithmic_bytes_per_launch": bytes_per_launch,
                    "us_per_minibatch_step": us_step,
                    "sync_us_per_step": sync_us,
                    "frac_of_sync_ceiling": (sync_us / us_step) if sync_us else None,
                    "launch_shape": {k: s1[k] for k in ("grid_ctas", "cluster_size", "ctas_per_chain", "threads_per_cta",
                                                        "pipeline_depth", "subpasses_per_stage", "smem_bytes",
                                                        "chains_in_flight")}}
        notes = []
        if l2_served:
            notes.append(f"one {buffer_bytes / 1e6:.1f} MB buffer is swept Rc*T = {w.Rc * w.T} times per launch and stays in the "
                         "126 MB L2 after the first sweep: `achieved` counts algorithmic bytes (it may exceed the HBM peak) and "
                         "`frac` is a throughput in HBM units, not an HBM utilisation; DRAM bytes per launch are in `traffic`")
        if w.Rc == 1:
            notes.append("one chain: every step waits for the theta of the step before it (Eq. (2.1)), so the step time, not "
                         "the memory system, sets the pace; `sync_us_per_step` is the same launch without rows and "
                         "`frac_of_sync_ceiling` = sync_us_per_step / us_per_minibatch_step")
        if w.loss == inputs.LOSS_SOFTMAX:
            flops = 4.0 * w.p * 16 * (sg / steps)  # both contractions, classes padded to 16
            roofline["tensor_tflops"] = flops / kdur / 1e12 if kdur > 0 else None
            notes.append("bf16 tcgen05 contractions (M=128, N=16, K=16): thin tiles, the tensor pipe is mostly idle")
        roofline["note"] = " | ".join(notes)
        self.launches += probe_launches
        res = {"value": value, "unit": UNIT, "steps": steps, "warmup": warmup, "ms_per_step": ms / steps,
               "dtype": {0: "f64", 1: "f32", 2: "bf16"}[w.dtype], "config": config_of(w),
               "us_per_minibatch_step": us_step, "roofline": roofline, "e2e": e2e_res,
               "gpu_launches": int(launches),
               "theta_check": {"finite": bool(np.isfinite(theta).all()), "mean": float(theta.mean())},
               "_window": (t_wall0, t_wall1, once), "_theta": theta, "_host": host}
        del resident
        torch.cuda.empty_cache()
        return res


def run_ours(args, w):
    import numpy as np
    R = Runner(args)
    rank, world = R.rank, R.world
    shape = dict(cluster_size=args.cluster_size, ctas_per_chain=args.ctas_per_chain, threads_per_cta=args.threads,
                 pipeline_depth=args.depth, subpasses_per_stage=args.subpasses, producer_warps=args.producer_warps,
                 lanes_per_row=args.lanes_per_row)
    sampler = ClockSampler(R.local) if rank == 0 else None
    if sampler:
        sampler.start()
    nb = args.buffers or w.K
    head = R.measure(w, nb, args.steps, args.warmup, e2e=not args.no_e2e, shape=shape, sampler=sampler)

    # theta of all chains of the job on rank 0: one all-gather at the end, nothing on the per-step path
    gathered = None
    if R.multi:
        from paper_2312_08728_b200 import multi_gpu
        local = torch.from_numpy(head["_theta"]).to(R.dev)
        gathered = multi_gpu.gather_theta(local, world * w.Rc).cpu().numpy()

    extras = {}
    if world == 1 and not args.no_extra and args.workload == "cfg2":
        for name, xnb, over in EXTRA_WORKLOADS:
            xw = WORKLOADS[name].scaled(**over) if over else WORKLOADS[name]
            extras[name] = R.measure(xw, min(xnb, xw.K), None, max(3, args.warmup), seconds=EXTRA_SECONDS,
                                     e2e=not args.no_e2e, e2e_steps=10, sampler=sampler)
    if sampler:
        sampler.stop()

    if rank != 0:
        if R.multi:
            import torch.distributed as dist
            dist.destroy_process_group()
        return

    def finish(res):
        t0, t1, once = res.pop("_window")
        res.pop("_theta"); res.pop("_host")
        res["clocks"] = sampler.window(t0, t1, once)
        return res

    host0 = head["_host"][:1]
    head = finish(head)
    cpu = None
    if not args.no_cpu and world == 1:
        rate, done, el, cores = oracle_rate(w, host0, args.cpu_seconds)
        cpu = {"value": rate, "unit": UNIT, "cores": cores, "kind": "oracle",
               "sample": f"chain 0, whole rounds over buffer 0 ({host0[0][0].shape[0]} rows) repeated for "
                         f"{el:.1f} s = {done} sample-gradients"}
    line = {
        "metric": METRIC, "value": head["value"], "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": args.warmup, "ms_per_step": head["ms_per_step"], "higher_is_better": True, "scaling": "weak",
        "vs_baseline": None, "dtype": head["dtype"], "data": "synthetic", "config": head["config"],
        "clocks": head["clocks"], "e2e": head["e2e"], "gpu_launches": int(R.launches),
        "roofline": head["roofline"], "cpu_baseline": cpu, "theta_check": head["theta_check"],
    }
    if gathered is not None:
        line["chains"] = {"total": int(world * w.Rc), "per_gpu": int(w.Rc), "gathered_theta_shape": list(gathered.shape),
                          "finite": bool(np.isfinite(gathered).all())}
    if extras:
        line["workloads"] = {name: finish(res) for name, res in extras.items()}
    print(json.dumps(line), flush=True)
    if R.multi:
        import torch.distributed as dist
        dist.destroy_process_group()


def main(argv=None):
    argv = sys.argv[1:] if argv is None else argv
    args = parse_args(argv)
    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        sys.exit(spawn_ranks(args, argv))
    w = workload_of(args)
    if args.impl == "reference":
        run_reference(args, w)
    else:
        run_ours(args, w)


if __name__ == "__main__":
    main()
