"""CPU oracle for BMGD: ctypes access to oracle/bmgd_oracle.c.

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the
benchmark's CPU-baseline leg.  The product package never imports this module and
this module never imports the product package.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "bmgd_oracle.c")
_LIB = os.path.join(_HERE, "libbmgd_oracle.so")

LINEAR, LOGISTIC, SOFTMAX = 0, 1, 2
F64, F32, BF16 = 0, 1, 2

_lib: Optional[ctypes.CDLL] = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP on) if the shared object is missing or stale."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".{os.getpid()}.tmp"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-ffp-contract=off",
             "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        u32p = ctypes.POINTER(ctypes.c_uint32)
        L.orc_philox4x32_10.argtypes = [u32p, u32p, u32p]
        L.orc_philox4x32_10.restype = None
        L.orc_round_keys.argtypes = [ctypes.c_uint64, ctypes.c_uint32, ctypes.c_uint32, u32p]
        L.orc_round_keys.restype = None
        L.orc_perm_index.argtypes = [ctypes.c_uint32, ctypes.c_uint32, u32p]
        L.orc_perm_index.restype = ctypes.c_uint32
        L.orc_domain.argtypes = [ctypes.c_uint32, u32p, u32p]
        L.orc_domain.restype = None
        L.orc_perm.argtypes = [ctypes.c_uint64, ctypes.c_uint32, ctypes.c_uint32, ctypes.c_uint32, ctypes.c_void_p]
        L.orc_perm.restype = None
        L.orc_run_rounds.argtypes = [
            ctypes.c_int, ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p, ctypes.c_int,
            ctypes.c_int64, ctypes.c_int, ctypes.c_int, ctypes.c_void_p,
            ctypes.c_int, ctypes.c_int, ctypes.c_double, ctypes.c_uint64, ctypes.c_uint32,
            ctypes.c_int, ctypes.c_void_p]
        L.orc_run_rounds.restype = ctypes.c_int
        L.orc_run_rounds_opt.argtypes = L.orc_run_rounds.argtypes + [ctypes.c_void_p]
        L.orc_run_rounds_opt.restype = ctypes.c_int
        L.orc_num_threads.restype = ctypes.c_int
        L.orc_set_num_threads.argtypes = [ctypes.c_int]
        _lib = L
    return _lib


def philox4x32_10(ctr, key):
    c = (ctypes.c_uint32 * 4)(*[int(v) & 0xFFFFFFFF for v in ctr])
    k = (ctypes.c_uint32 * 2)(*[int(v) & 0xFFFFFFFF for v in key])
    out = (ctypes.c_uint32 * 4)()
    lib().orc_philox4x32_10(c, k, out)
    return [int(v) for v in out]


def round_keys(seed: int, chain: int, rnd: int):
    out = (ctypes.c_uint32 * 8)()
    lib().orc_round_keys(int(seed) & 0xFFFFFFFFFFFFFFFF, chain, rnd, out)
    return [int(v) for v in out]


def domain(N0: int):
    """(a, c): the sizes of the two halves of the Feistel network for a buffer of N0 rows."""
    a, c = ctypes.c_uint32(), ctypes.c_uint32()
    lib().orc_domain(N0, ctypes.byref(a), ctypes.byref(c))
    return a.value, c.value


def perm(seed: int, chain: int, rnd: int, N0: int) -> np.ndarray:
    """pi_t as an array: out[j] = pi_t(j), uint32."""
    out = np.empty(N0, dtype=np.uint32)
    lib().orc_perm(int(seed) & 0xFFFFFFFFFFFFFFFF, chain, rnd, N0, out.ctypes.data)
    return out


def _as_stored(a):
    """(numpy view, storage code) of a numpy array or torch tensor without changing its bits."""
    try:
        import torch
        if isinstance(a, torch.Tensor):
            a = a.detach().cpu().contiguous()
            if a.dtype == torch.bfloat16:
                return a.view(torch.int16).numpy().view(np.uint16), BF16
            a = a.numpy()
    except ImportError:  # pragma: no cover
        pass
    a = np.ascontiguousarray(a)
    if a.dtype == np.float64:
        return a, F64
    if a.dtype == np.float32:
        return a, F32
    if a.dtype == np.uint16:
        return a, BF16
    if a.dtype == np.int32:
        return a, -1
    raise TypeError(f"unsupported stored dtype {a.dtype}")


def run_rounds(loss: int, X, y, theta: np.ndarray, T: int, n: int, alpha: float, seed: int,
               chain: int = 0, C: int = 1, fixed_partition: bool = False,
               trace: bool = False, opt: "Optimizer | None" = None):
    """T rounds over one buffer; `theta` (float64, [p] or [p, C]) is updated in place.

    X and y are read as stored (fp64 / fp32 / bf16; int32 labels for softmax).
    With trace=True returns theta after every step as [T*M, p*C].
    """
    Xn, xt = _as_stored(X)
    yn, yt = _as_stored(y)
    N0, p = Xn.shape
    if loss == SOFTMAX:
        if yn.dtype != np.int32:
            raise TypeError("softmax labels must be int32")
        if theta.shape != (p, C):
            raise ValueError("theta must be [p, C]")
    else:
        if yt < 0:
            raise TypeError("responses must be floating point")
        if theta.shape != (p,):
            raise ValueError("theta must be [p]")
    if theta.dtype != np.float64 or not theta.flags.c_contiguous:
        raise TypeError("theta must be contiguous float64")
    if yn.shape[0] != N0:
        raise ValueError("y has the wrong length")
    M = -(-N0 // n)
    tr = np.empty((T * M, theta.size), dtype=np.float64) if trace else None
    if opt is not None:
        if opt.s1.size != theta.size:
            raise ValueError("optimizer state has the wrong size")
        st = opt._struct()
        rc = lib().orc_run_rounds_opt(loss, Xn.ctypes.data, xt, yn.ctypes.data, max(yt, 0), N0, p, C,
                                      theta.ctypes.data, T, n, float(alpha),
                                      int(seed) & 0xFFFFFFFFFFFFFFFF, chain, int(fixed_partition),
                                      tr.ctypes.data if trace else None, ctypes.byref(st))
    else:
        rc = lib().orc_run_rounds(loss, Xn.ctypes.data, xt, yn.ctypes.data, max(yt, 0), N0, p, C,
                                  theta.ctypes.data, T, n, float(alpha),
                                  int(seed) & 0xFFFFFFFFFFFFFFFF, chain, int(fixed_partition),
                                  tr.ctypes.data if trace else None)
    if rc != 0:
        raise ValueError("orc_run_rounds rejected its arguments")
    return tr


OPT_SGD, OPT_NESTEROV, OPT_ADAM = 0, 1, 2
LR_CONSTANT, LR_COSINE = 0, 1


class _OrcOpt(ctypes.Structure):
    _fields_ = [("kind", ctypes.c_int), ("a", ctypes.c_double), ("b", ctypes.c_double), ("eps", ctypes.c_double),
                ("s1", ctypes.c_void_p), ("s2", ctypes.c_void_p), ("t", ctypes.c_void_p),
                ("sched", ctypes.c_int), ("period", ctypes.c_int64), ("j_done", ctypes.c_void_p)]


class Optimizer:
    """Update rule and learning-rate schedule with their state, carried from one run_rounds call to the next.

    kind: OPT_SGD (Eq. (2.1)), OPT_NESTEROV (a = momentum) or OPT_ADAM (a = beta1, b = beta2, eps).
    sched: LR_CONSTANT, or LR_COSINE with `period` updates per pass (Section 4.4).
    """

    def __init__(self, kind: int, size: int, a: float = 0.9, b: float = 0.999, eps: float = 1e-7,
                 sched: int = LR_CONSTANT, period: int = 0):
        self.kind, self.a, self.b, self.eps, self.sched, self.period = kind, a, b, eps, sched, period
        self.s1 = np.zeros(size, dtype=np.float64)
        self.s2 = np.zeros(size, dtype=np.float64)
        self.t = np.zeros(1, dtype=np.int64)
        self.j_done = np.zeros(1, dtype=np.int64)

    def _struct(self) -> _OrcOpt:
        return _OrcOpt(self.kind, self.a, self.b, self.eps, self.s1.ctypes.data, self.s2.ctypes.data,
                       self.t.ctypes.data, self.sched, self.period, self.j_done.ctypes.data)


def num_threads() -> int:
    return lib().orc_num_threads()


def set_num_threads(k: int) -> None:
    lib().orc_set_num_threads(k)
