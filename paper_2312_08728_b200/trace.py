"""Per-phase cycle counts of the step kernel, from the trace build of the library.

    python -m paper_2312_08728_b200.build --trace          # libbmgd_trace.so: the same sources with -DBMGD_TRACE
    python -m paper_2312_08728_b200.trace cfg5 cfg3 cfg5:null cfg2:chains=8

In the trace build thread 0 of every CTA stamps its SM's cycle counter at the phase boundaries of the first steps of a
launch.  This reader runs one buffer of a workload for one round (or the latency probe, `:null`), reads the stamps back
and prints, per phase, the median over steps of CTA 0 and the spread of that median over all CTAs.  A debugging aid:
numbers taken from the trace build are a little slower than the product build and are never bench values.

Phases of a step (consumer thread 0):  sweep = waiting for and multiplying the CTA's rows;  cta-sum = folding the row
groups and the barrier behind it;  col-sum = one thread per predictor summing the CTA's partial rows;  push = sending the
sums to the peers;  poll = waiting for the peers' sums (one cluster per chain), or, with several clusters per chain,
rs-poll + l2-store = the reduce-scatter inside the cluster and writing the slice sums to global memory,  l2-poll+push =
waiting for the other clusters' slice sums and sending totals to the peers,  totals = waiting for the peers' totals;
update = applying the update rule and publishing theta;  reload = the barrier and re-reading the coefficients.
"""
from __future__ import annotations

import ctypes
import sys

import numpy as np
import torch

from . import binding, build as _build, inputs


def load_trace_library():
    if _build.is_stale(_build.TRACE_LIB_PATH):
        _build.build(trace=True)
    L = binding.load_library(_build.TRACE_LIB_PATH)
    L.bmgd_debug_trace.argtypes = [ctypes.c_int, ctypes.c_void_p, ctypes.c_int]
    L.bmgd_debug_trace.restype = ctypes.c_int
    P = ctypes.POINTER(ctypes.c_int)
    L.bmgd_debug_trace_dims.argtypes = [P, P, P]
    return L


def read_stamps(L, which=0):
    b, s, ph = ctypes.c_int(), ctypes.c_int(), ctypes.c_int()
    assert L.bmgd_debug_trace_dims(ctypes.byref(b), ctypes.byref(s), ctypes.byref(ph)) == 0
    out = np.zeros(b.value * s.value * ph.value, dtype=np.int64)
    assert L.bmgd_debug_trace(which, out.ctypes.data, out.size) == 0
    return out.reshape(b.value, s.value, ph.value)


# (name, from phase, to phase) for one cluster per chain and for several
PHASES_ONE = [("step head", 0, 11), ("wait for 1st stage", 11, 10), ("1st stage's rows", 10, 13), ("sweep", 0, 1), ("cta-sum", 1, 2), ("col-sum", 2, 3), ("push", 3, 8), ("poll", 8, 4), ("update", 6, 9),
              ("reload", 9, 7)]
PHASES_MULTI = [("step head", 0, 11), ("wait for 1st stage", 11, 10), ("1st stage's rows", 10, 13), ("sweep", 0, 1), ("cta-sum", 1, 2), ("col-sum", 2, 3), ("rs-push", 3, 4), ("rs-poll+l2-store", 4, 12),
                ("l2-poll+push", 12, 5), ("totals", 5, 6), ("update", 6, 9), ("reload", 9, 7)]
PHASES_SOFTMAX = [("wait for rows", 0, 1), ("forward + read-out", 1, 2), ("logits exchange", 2, 3), ("softmax + R push", 3, 4),
                  ("R arrival", 4, 5), ("backward + read-out", 5, 6), ("update + barrier", 6, 7)]
PRODUCER = [("shuffle", 0, 1), ("slot wait + copies (A)", 1, 3), ("arrive (A)", 3, 4), ("B (gathered rows)", 4, 6)]


def trace_workload(L, spec):
    name, _, opts = spec.partition(":")
    kw, shape, null, chains, rounds = {}, {}, False, 0, 1
    for o in filter(None, opts.split(",")):
        if o == "null":
            null = True
            continue
        k, v = o.split("=")
        if k == "chains":
            chains = int(v)
        elif k == "rounds":
            rounds = int(v)
        elif k in ("p", "n", "N", "K", "C"):  # another shape of the same workload
            shape[k] = int(v)
        else:
            kw[k] = int(v)
    w = inputs.WORKLOADS[name]
    if shape:
        w = w.scaled(**shape)
    if chains:
        w = w.scaled(Rc=chains)
    x, y = inputs.make_buffer(w, 0)
    dx, dy = x.cuda(), y.cuda()
    binding._lib = L  # handles made below call into the trace build
    with binding.Bmgd(w.N, w.p, w.K, loss=w.loss, dtype=w.dtype, C=w.C, Rc=w.Rc, flags=binding.FLAG_NO_SLOTS, **kw) as h:
        for seed in (1, 2):  # the second launch is the one whose stamps are read
            if null:
                h.debug_null_rounds(x.shape[0], rounds, w.n)
            else:
                h.run_rounds_resident(dx, dy, rounds, w.n, w.lr, seed)
            h.sync()
        st = h.get_stats()
    t = read_stamps(L, 0)
    nblk = min(st["grid_ctas"], t.shape[0])
    multi = st["ctas_per_chain"] > st["cluster_size"]
    steps = slice(8, t.shape[1] - 4)
    print(f"== {spec}: grid {st['grid_ctas']} CTAs, clusters of {st['cluster_size']}, {st['ctas_per_chain']} CTAs per chain, "
          f"{st['threads_per_cta']} threads, ring {st['pipeline_depth']} x {st['subpasses_per_stage']} sub-passes")
    per_blk_step = np.median(t[:nblk, 9:t.shape[1] - 4, 0] - t[:nblk, 8:t.shape[1] - 5, 0], axis=1)
    print(f"   step: {int(per_blk_step[0])} cycles in CTA 0 (min {int(per_blk_step.min())}, max {int(per_blk_step.max())} over CTAs)")
    softmax = w.loss == inputs.LOSS_SOFTMAX
    for label, a, b in (PHASES_SOFTMAX if softmax else PHASES_MULTI if multi else PHASES_ONE):
        d = np.median(t[:nblk, steps, b] - t[:nblk, steps, a], axis=1)
        print(f"   {label:18s} {int(d[0]):6d}   (CTAs: min {int(d.min()):6d}  median {int(np.median(d)):6d}  max {int(d.max()):6d})")
    if softmax:
        return
    pt = read_stamps(L, 1)
    for label, a, b in PRODUCER:
        d = np.median(pt[:nblk, steps, b] - pt[:nblk, steps, a], axis=1)
        print(f"   producer {label:22s} {int(d[0]):6d}   (CTAs: median {int(np.median(d)):6d})")
    pair = np.median(pt[:nblk, 9:t.shape[1] - 4, 0] - pt[:nblk, 8:t.shape[1] - 5, 0], axis=1)
    print(f"   producer warp 0, one turn of its loop (a pair of stages with gathered rows, else one stage of its slot): {int(pair[0])} cycles")


def main(argv):
    if not torch.cuda.is_available():
        raise SystemExit("the trace reader needs a CUDA device")
    L = load_trace_library()
    for spec in argv:
        trace_workload(L, spec)


if __name__ == "__main__":
    main(sys.argv[1:])
