"""Shared test plumbing: run the same BMGD job through the oracle and through the CUDA library."""
import numpy as np
import torch

import oracle
from paper_2312_08728_b200 import inputs

ORACLE_LOSS = {inputs.LOSS_LINEAR: oracle.LINEAR, inputs.LOSS_LOGISTIC: oracle.LOGISTIC,
               inputs.LOSS_SOFTMAX: oracle.SOFTMAX}
TOL = {inputs.DTYPE_F64: 1e-10, inputs.DTYPE_F32: 1e-4, inputs.DTYPE_BF16: 2e-2}


def rel_l2(a, b):
    a = np.asarray(a, dtype=np.float64).ravel()
    b = np.asarray(b, dtype=np.float64).ravel()
    return float(np.linalg.norm(a - b) / max(np.linalg.norm(b), 1e-300))


def oracle_job(w, buffers, chains=None, theta0=None, fixed_partition=False, opt=None):
    """Run w.epochs passes over `buffers` [(X, y), ...] for the listed chains; returns {chain: theta}.

    opt: None, or dict(kind=, a=, b=, eps=, sched=, period=) in the oracle's constants: the update rule and
    learning-rate schedule, with one state per chain carried through the whole job."""
    chains = list(range(w.Rc)) if chains is None else chains
    shape = (w.p, w.C) if w.loss == inputs.LOSS_SOFTMAX else (w.p,)
    out = {}
    for c in chains:
        th = np.zeros(shape) if theta0 is None else np.array(theta0[c], dtype=np.float64).reshape(shape)
        o = None
        if opt is not None:
            o = oracle.Optimizer(opt.get("kind", oracle.OPT_SGD), th.size, a=opt.get("a", 0.0), b=opt.get("b", 0.0),
                                 eps=opt.get("eps", 0.0), sched=opt.get("sched", oracle.LR_CONSTANT),
                                 period=opt.get("period", 0))
        for e in range(w.epochs):
            for k, (X, y) in enumerate(buffers):
                oracle.run_rounds(ORACLE_LOSS[w.loss], X, y, th, w.T, min(w.n, X.shape[0]), w.lr,
                                  inputs.buffer_seed(w.seed, e, k, len(buffers)), chain=c, C=w.C,
                                  fixed_partition=fixed_partition, opt=o)
        out[c] = th
    return out


def gpu_job(w, buffers, mode="slots", flags=0, theta0=None, opt=None, **shape):
    """The same job through the C ABI.  mode: "slots" streams host buffers through load_buffer with the next
    copy issued before the current compute; "resident" keeps all buffers on the device."""
    from paper_2312_08728_b200.binding import Bmgd, FLAG_NO_SLOTS
    N0max = max(X.shape[0] for X, _ in buffers)
    K = len(buffers)
    if mode == "resident":
        flags |= FLAG_NO_SLOTS
    h = Bmgd(N0max * K, w.p, K, loss=w.loss, dtype=w.dtype, C=w.C, Rc=w.Rc, flags=flags, **shape)
    try:
        if theta0 is not None:
            h.set_theta(theta0)
        if opt is not None:  # the library's constants have the oracle's values; checked in the CPU tests
            h.set_optimizer(opt.get("kind", 0), opt.get("a", 0.0), opt.get("b", 0.0), opt.get("eps", 0.0))
            h.set_lr_schedule(opt.get("sched", 0), opt.get("period", 0))
        if mode == "resident":
            dev = [(X.cuda(), y.cuda()) for X, y in buffers]
            for e in range(w.epochs):
                for k, (X, y) in enumerate(dev):
                    h.run_rounds_resident(X, y, w.T, w.n, w.lr, inputs.buffer_seed(w.seed, e, k, K))
        else:
            copy = torch.cuda.Stream()
            pinned = [(X.pin_memory(), y.pin_memory()) for X, y in buffers]
            order = [(e, k) for e in range(w.epochs) for k in range(K)]
            slot = h.load_buffer(*pinned[order[0][1]], stream=copy)
            for i, (e, k) in enumerate(order):
                nxt = None
                if i + 1 < len(order):
                    nxt = h.load_buffer(*pinned[order[i + 1][1]], stream=copy)
                h.run_rounds(slot, w.T, w.n, w.lr, inputs.buffer_seed(w.seed, e, k, K))
                slot = nxt
        theta = h.get_theta()
        stats = h.get_stats()
    finally:
        h.close()
    return theta, stats


def buffers_of(w):
    return [inputs.make_buffer(w, k) for k in range(w.K)]
