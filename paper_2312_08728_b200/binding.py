"""ctypes binding of the BMGD C ABI (include/bmgd.h).

Argument marshalling only: every step of the computation runs in the CUDA library.
torch is used for device memory (the workspace), pinned host memory and streams.
There is no CPU fallback: if the library cannot be loaded, or no CUDA device is
present, creating a handle raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import numpy as np
import torch

from . import build as _build
from .inputs import DTYPE_BF16, DTYPE_F32, DTYPE_F64, LOSS_LINEAR, LOSS_LOGISTIC, LOSS_SOFTMAX

BMGD_OK = 0
ERR_ARG, ERR_ALLOC, ERR_CUDA, ERR_CAPACITY, ERR_TIMEOUT = -1, -2, -3, -4, -5
ERR_NONFINITE, ERR_LAUNCH, ERR_UNIMPLEMENTED, ERR_STATE = -6, -7, -8, -9

FLAG_FIXED_PARTITION = 1
FLAG_NO_SLOTS = 2
FLAG_TIMING = 4
FLAG_SOFTMAX_CUDA_CORES = 8

# every symbol include/bmgd.h declares
EXPORTS = (
    "bmgd_config_init", "bmgd_workspace_bytes", "bmgd_create", "bmgd_create_ex", "bmgd_destroy",
    "bmgd_load_buffer", "bmgd_run_rounds", "bmgd_run_rounds_resident", "bmgd_sync", "bmgd_get_theta",
    "bmgd_set_theta", "bmgd_get_stats", "bmgd_debug_perm", "bmgd_strerror", "bmgd_last_cuda_error",
    "bmgd_version", "bmgd_run_rounds_noalloc", "bmgd_debug_wait_timeout", "bmgd_partition_index", "bmgd_gather_buffer",
    "bmgd_set_optimizer", "bmgd_set_lr_schedule", "bmgd_set_timeout", "bmgd_debug_null_rounds",
)

OPT_SGD, OPT_NESTEROV, OPT_ADAM = 0, 1, 2
LR_CONSTANT, LR_COSINE = 0, 1


class BmgdConfig(ctypes.Structure):
    _fields_ = [
        ("N", ctypes.c_int64), ("p", ctypes.c_int32), ("K", ctypes.c_int32), ("loss", ctypes.c_int32),
        ("dtype", ctypes.c_int32), ("C", ctypes.c_int32), ("Rc", ctypes.c_int32), ("device", ctypes.c_int32),
        ("flags", ctypes.c_uint32), ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_int64),
        ("compute_stream", ctypes.c_void_p), ("timeout_ms", ctypes.c_double),
        ("cluster_size", ctypes.c_int32), ("ctas_per_chain", ctypes.c_int32),
        ("threads_per_cta", ctypes.c_int32), ("pipeline_depth", ctypes.c_int32),
        ("subpasses_per_stage", ctypes.c_int32), ("producer_warps", ctypes.c_int32),
        ("lanes_per_row", ctypes.c_int32), ("first_chain", ctypes.c_int32), ("reserved", ctypes.c_int32 * 4),
    ]


class BmgdStats(ctypes.Structure):
    _fields_ = [
        ("launches", ctypes.c_int64), ("steps", ctypes.c_int64), ("sample_grads", ctypes.c_int64),
        ("h2d_bytes", ctypes.c_int64), ("kernel_ms", ctypes.c_double), ("h2d_ms", ctypes.c_double),
        ("grid_ctas", ctypes.c_int32), ("cluster_size", ctypes.c_int32), ("ctas_per_chain", ctypes.c_int32),
        ("threads_per_cta", ctypes.c_int32), ("pipeline_depth", ctypes.c_int32), ("smem_bytes", ctypes.c_int32),
        ("chains_in_flight", ctypes.c_int32), ("subpasses_per_stage", ctypes.c_int32),
    ]

    def as_dict(self):
        return {k: getattr(self, k) for k, _ in self._fields_ if k != "reserved"}


class BmgdError(RuntimeError):
    def __init__(self, status: int, where: str, cuda: int = 0):
        self.status = status
        self.cuda_error = cuda
        msg = load_library().bmgd_strerror(status).decode()
        super().__init__(f"{where}: {msg} (status {status}" + (f", cudaError {cuda})" if cuda else ")"))


_lib: Optional[ctypes.CDLL] = None


def load_library(path: Optional[str] = None) -> ctypes.CDLL:
    """Load libbmgd.so (building it first if its sources are newer) and declare the ABI."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    if path is None:
        path = _build.LIB_PATH
        if _build.is_stale():
            if _build.find_nvcc() is not None:
                _build.build()
            elif not os.path.exists(path):
                raise RuntimeError("libbmgd.so is not built and nvcc is not available")
    L = ctypes.CDLL(path)
    vp, i32, i64, u32, u64, dbl = (ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_uint32,
                                  ctypes.c_uint64, ctypes.c_double)
    P = ctypes.POINTER
    L.bmgd_config_init.argtypes = [P(BmgdConfig)]; L.bmgd_config_init.restype = None
    L.bmgd_workspace_bytes.argtypes = [P(BmgdConfig), P(i64)]
    L.bmgd_create.argtypes = [i64, i32, i32, i32, P(vp)]
    L.bmgd_create_ex.argtypes = [P(BmgdConfig), P(vp)]
    L.bmgd_destroy.argtypes = [vp]
    L.bmgd_load_buffer.argtypes = [vp, vp, vp, i64, vp, P(i32)]
    L.bmgd_run_rounds.argtypes = [vp, i32, i32, i32, dbl, u64]
    L.bmgd_run_rounds_resident.argtypes = [vp, vp, vp, i64, i32, i32, dbl, u64]
    L.bmgd_sync.argtypes = [vp]
    L.bmgd_set_optimizer.argtypes = [vp, i32, dbl, dbl, dbl]
    L.bmgd_set_lr_schedule.argtypes = [vp, i32, i64]
    L.bmgd_set_timeout.argtypes = [vp, dbl]
    L.bmgd_get_theta.argtypes = [vp, vp, i64]
    L.bmgd_set_theta.argtypes = [vp, vp, i64]
    L.bmgd_get_stats.argtypes = [vp, P(BmgdStats)]
    L.bmgd_debug_perm.argtypes = [vp, u64, u32, u32, u32, vp]
    L.bmgd_strerror.argtypes = [ctypes.c_int]; L.bmgd_strerror.restype = ctypes.c_char_p
    L.bmgd_last_cuda_error.argtypes = [vp]
    L.bmgd_version.argtypes = []
    L.bmgd_debug_wait_timeout.argtypes = [vp, dbl]
    L.bmgd_debug_null_rounds.argtypes = [vp, i64, i32, i32]
    L.bmgd_partition_index.argtypes = [u64, u32, i64, i64, P(i64)]
    L.bmgd_gather_buffer.argtypes = [vp, vp, i64, i64, i64, i32, u64, u32, i32, vp, vp, i32, P(i64)]
    L.bmgd_run_rounds_noalloc.argtypes = [vp, vp, i64, i32, i32, i32, i32, vp, i32, i32, dbl, u64, vp]
    for name in EXPORTS:
        if getattr(L, name).restype is None or name in ("bmgd_strerror",):
            continue
        getattr(L, name).restype = ctypes.c_int
    if path == _build.LIB_PATH:
        _lib = L
    return L


_NP_THETA = {DTYPE_F64: np.float64, DTYPE_F32: np.float32, DTYPE_BF16: np.float32}


NOALLOC_MAX_P = 256

_TORCH_X = {DTYPE_F64: torch.float64, DTYPE_F32: torch.float32, DTYPE_BF16: torch.bfloat16}
_TORCH_THETA = {DTYPE_F64: torch.float64, DTYPE_F32: torch.float32, DTYPE_BF16: torch.float32}


def check_buffer(x: torch.Tensor, y: torch.Tensor, p: int, loss: int, dtype: int, max_rows: Optional[int] = None) -> int:
    """Refuse a buffer whose tensors do not have the shape and element types the job was created for.

    The C ABI takes bare pointers, so a float32 X handed to a float64 job, an X with another column count, a
    shorter y or labels that are not int32 would make the kernel read past the end of an allocation.  This is
    the only place where the tensors' own metadata can be compared with the job.  Returns the row count."""
    if dtype not in _TORCH_X:
        raise ValueError(f"unknown dtype code {dtype}")
    if x.dim() != 2 or x.shape[1] != p:
        raise ValueError(f"X must be [rows, {p}], got {tuple(x.shape)}")
    if x.dtype != _TORCH_X[dtype]:
        raise ValueError(f"X must be {_TORCH_X[dtype]}, got {x.dtype}")
    want_y = torch.int32 if loss == LOSS_SOFTMAX else _TORCH_THETA[dtype]
    if y.dim() != 1 or y.shape[0] != x.shape[0]:
        raise ValueError(f"y must be [{x.shape[0]}], got {tuple(y.shape)}")
    if y.dtype != want_y:
        raise ValueError(f"y must be {want_y}, got {y.dtype}")
    if not (x.is_contiguous() and y.is_contiguous()):
        raise ValueError("X and y must be contiguous")
    if x.device != y.device:
        raise ValueError("X and y must live on the same device")
    if x.shape[0] < 1:
        raise ValueError("a buffer needs at least one row")
    if max_rows is not None and x.shape[0] > max_rows:
        raise ValueError(f"{x.shape[0]} rows do not fit a slot of {max_rows}")
    return x.shape[0]


def run_rounds_noalloc(dev_x: torch.Tensor, dev_y: torch.Tensor, theta: torch.Tensor, loss: int, dtype: int,
                       rounds: int, batch_size: int, lr: float, seed: int,
                       stream: Optional[torch.cuda.Stream] = None) -> None:
    """Allocation-free computation step: bmgd_run_rounds_noalloc on caller-held device tensors.

    For callers that may not allocate device memory where they call this library (a fixed memory
    budget, an allocator owned by someone else).  `theta` [Rc, p] lives on the device, is the
    starting value and receives the result.  Nothing is allocated here either: the tensors are
    passed as they are and must already be contiguous and on the current device.  Returns once the
    kernel has finished; calls on one GPU must not overlap, they share one fixed scratch array.
    """
    if theta.dim() != 2:
        raise ValueError(f"theta must be [Rc, p], got {tuple(theta.shape)}")
    Rc, p = theta.shape
    # y is checked as a response vector in the parameter type: the entry point has no softmax kernel, and the
    # library itself refuses such a job
    check_buffer(dev_x, dev_y, p, LOSS_LINEAR, dtype)
    if theta.dtype != _TORCH_THETA[dtype]:
        raise ValueError(f"theta must be {_TORCH_THETA[dtype]}, got {theta.dtype}")
    for t in (dev_x, dev_y, theta):
        if t.device.type != "cuda" or not t.is_contiguous():
            raise ValueError("run_rounds_noalloc takes contiguous device tensors")
    if theta.device != dev_x.device:
        raise ValueError("theta and the buffer must live on the same device")
    L = load_library()
    s = stream.cuda_stream if stream is not None else None
    rc = L.bmgd_run_rounds_noalloc(dev_x.data_ptr(), dev_y.data_ptr(), dev_x.shape[0], p, loss, dtype, Rc,
                                   theta.data_ptr(), rounds, batch_size, float(lr),
                                   int(seed) & 0xFFFFFFFFFFFFFFFF, s)
    if rc != BMGD_OK:
        raise BmgdError(rc, "bmgd_run_rounds_noalloc")


PARTITION_CHAIN = 0xFFFFFFFF  # chain word of the sample-level partition


def partition_index(seed: int, epoch: int, N: int, j: int) -> int:
    """Row of the sample that sits at position j of pass `epoch`'s random partition into buffers."""
    out = ctypes.c_int64(-1)
    rc = load_library().bmgd_partition_index(int(seed) & 0xFFFFFFFFFFFFFFFF, epoch, N, j, ctypes.byref(out))
    if rc != BMGD_OK:
        raise BmgdError(rc, "bmgd_partition_index")
    return out.value


def gather_buffer(host_x: torch.Tensor, host_y: torch.Tensor, K: int, seed: int, epoch: int, k: int,
                  stage_x: torch.Tensor, stage_y: torch.Tensor, threads: int = 0) -> int:
    """Gather buffer k of pass `epoch` from the whole host-resident sample into the staging tensors (host threads
    inside the library; the GIL is released for the duration of the call).  Returns the number of rows."""
    for t in (host_x, host_y, stage_x, stage_y):
        if t.device.type != "cpu" or not t.is_contiguous():
            raise ValueError("gather_buffer takes contiguous host tensors")
    N = host_x.shape[0]
    row_bytes = host_x.shape[1] * host_x.element_size()
    if stage_x.shape[1] * stage_x.element_size() != row_bytes or stage_x.shape[0] < -(-N // K) or stage_y.shape[0] < -(-N // K):
        raise ValueError("staging tensors are too small for a buffer")
    rows = ctypes.c_int64(0)
    rc = load_library().bmgd_gather_buffer(host_x.data_ptr(), host_y.data_ptr(), N, row_bytes, host_y.element_size(), K,
                                           int(seed) & 0xFFFFFFFFFFFFFFFF, epoch, k, stage_x.data_ptr(),
                                           stage_y.data_ptr(), threads, ctypes.byref(rows))
    if rc != BMGD_OK:
        raise BmgdError(rc, "bmgd_gather_buffer")
    return rows.value


class Bmgd:
    """One BMGD handle: theta for Rc chains, two device buffer slots, a compute stream.

    Mirrors the C calls one to one: load_buffer, run_rounds, run_rounds_resident, sync,
    get_theta, set_theta, get_stats, debug_perm.
    """

    def __init__(self, N: int, p: int, K: int, loss: int = LOSS_LINEAR, dtype: int = DTYPE_F32, C: int = 1,
                 Rc: int = 1, device: int = 0, flags: int = 0, cluster_size: int = 0, ctas_per_chain: int = 0,
                 threads_per_cta: int = 0, pipeline_depth: int = 0, subpasses_per_stage: int = 0,
                 producer_warps: int = 0, lanes_per_row: int = 0,
                 timeout_ms: float = 0.0, first_chain: int = 0,
                 use_torch_stream: bool = False):
        if not torch.cuda.is_available():
            raise RuntimeError("BMGD needs a CUDA device; there is no CPU path")
        self._lib = load_library()
        self._h = ctypes.c_void_p()
        cfg = BmgdConfig()
        self._lib.bmgd_config_init(ctypes.byref(cfg))
        cfg.N, cfg.p, cfg.K, cfg.loss, cfg.dtype, cfg.C, cfg.Rc = N, p, K, loss, dtype, C, Rc
        cfg.device, cfg.flags = device, flags
        cfg.cluster_size, cfg.ctas_per_chain = cluster_size, ctas_per_chain
        cfg.threads_per_cta, cfg.pipeline_depth, cfg.timeout_ms = threads_per_cta, pipeline_depth, timeout_ms
        cfg.subpasses_per_stage = subpasses_per_stage
        cfg.producer_warps = producer_warps
        cfg.lanes_per_row = lanes_per_row
        cfg.first_chain = first_chain
        need = ctypes.c_int64()
        self._check(self._lib.bmgd_workspace_bytes(ctypes.byref(cfg), ctypes.byref(need)), "bmgd_workspace_bytes")
        self.device = torch.device("cuda", device)
        # device memory comes from torch's allocator; the library carves it up
        self._workspace = torch.empty(need.value + 256, dtype=torch.uint8, device=self.device)
        base = (self._workspace.data_ptr() + 255) // 256 * 256
        cfg.workspace, cfg.workspace_bytes = base, need.value
        if use_torch_stream:
            self._stream = torch.cuda.current_stream(self.device)
            cfg.compute_stream = self._stream.cuda_stream
        self.cfg = cfg
        self.N, self.p, self.K, self.loss, self.dtype, self.C, self.Rc = N, p, K, loss, dtype, C, Rc
        self._check(self._lib.bmgd_create_ex(ctypes.byref(cfg), ctypes.byref(self._h)), "bmgd_create_ex")
        self._keep = []  # host tensors whose copies may still be in flight

    # -- helpers
    def _check(self, status: int, where: str, allow=()):
        if status != BMGD_OK and status not in allow:
            cuda = self._lib.bmgd_last_cuda_error(self._h) if self._h else 0
            raise BmgdError(status, where, cuda)
        return status

    @property
    def theta_shape(self) -> Tuple[int, ...]:
        return (self.Rc, self.p, self.C) if self.loss == LOSS_SOFTMAX else (self.Rc, self.p)

    # -- the calls
    def load_buffer(self, host_x: torch.Tensor, host_y: torch.Tensor, stream: Optional[torch.cuda.Stream] = None) -> int:
        """Start the host-to-device copy of one buffer; returns the slot id."""
        if host_x.device.type != "cpu" or host_y.device.type != "cpu":
            raise ValueError("load_buffer takes host tensors")
        rows = check_buffer(host_x, host_y, self.p, self.loss, self.dtype)
        if rows > -(-self.N // self.K):  # the library refuses it too; said here with the same status
            raise BmgdError(ERR_CAPACITY, "load_buffer")
        slot = ctypes.c_int32(-1)
        s = stream.cuda_stream if stream is not None else None
        self._check(self._lib.bmgd_load_buffer(self._h, host_x.data_ptr(), host_y.data_ptr(), rows, s,
                                               ctypes.byref(slot)), "bmgd_load_buffer")
        self._keep.append((host_x, host_y))
        if len(self._keep) > 4:
            self._keep.pop(0)
        return slot.value

    def run_rounds(self, slot: int, rounds: int, batch_size: int, lr: float, seed: int) -> None:
        self._check(self._lib.bmgd_run_rounds(self._h, slot, rounds, batch_size, float(lr),
                                              int(seed) & 0xFFFFFFFFFFFFFFFF), "bmgd_run_rounds")

    def run_rounds_resident(self, dev_x: torch.Tensor, dev_y: torch.Tensor, rounds: int, batch_size: int,
                            lr: float, seed: int) -> None:
        if dev_x.device != self.device or dev_y.device != self.device:
            raise ValueError("resident buffers must live on the handle's device")
        check_buffer(dev_x, dev_y, self.p, self.loss, self.dtype)
        self._check(self._lib.bmgd_run_rounds_resident(self._h, dev_x.data_ptr(), dev_y.data_ptr(), dev_x.shape[0],
                                                       rounds, batch_size, float(lr),
                                                       int(seed) & 0xFFFFFFFFFFFFFFFF), "bmgd_run_rounds_resident")

    def sync(self) -> None:
        self._check(self._lib.bmgd_sync(self._h), "bmgd_sync")
        self._keep.clear()

    def get_theta(self, allow_nonfinite: bool = False) -> np.ndarray:
        out = np.empty(self.theta_shape, dtype=_NP_THETA[self.dtype])
        self._check(self._lib.bmgd_get_theta(self._h, out.ctypes.data, out.nbytes), "bmgd_get_theta",
                    allow=(ERR_NONFINITE,) if allow_nonfinite else ())
        return out

    def set_theta(self, theta: np.ndarray) -> None:
        a = np.ascontiguousarray(theta, dtype=_NP_THETA[self.dtype]).reshape(self.theta_shape)
        self._check(self._lib.bmgd_set_theta(self._h, a.ctypes.data, a.nbytes), "bmgd_set_theta")

    def set_optimizer(self, kind: int, a: float = 0.0, b: float = 0.0, eps: float = 0.0) -> None:
        """Choose the update rule (OPT_SGD, OPT_NESTEROV with momentum a, OPT_ADAM with beta1 a, beta2 b, eps);
        its state starts from zero."""
        self._check(self._lib.bmgd_set_optimizer(self._h, kind, float(a), float(b), float(eps)), "bmgd_set_optimizer")

    def set_lr_schedule(self, kind: int, updates_per_pass: int = 0) -> None:
        """LR_CONSTANT, or LR_COSINE: the j-th update of a pass of `updates_per_pass` takes lr (1/2 + 1/2 cos(j pi / J))."""
        self._check(self._lib.bmgd_set_lr_schedule(self._h, kind, int(updates_per_pass)), "bmgd_set_lr_schedule")

    def set_timeout(self, timeout_ms: float) -> None:
        """Bound on any single device-side wait of later launches; <= 0 selects the default of 2000 ms."""
        self._check(self._lib.bmgd_set_timeout(self._h, float(timeout_ms)), "bmgd_set_timeout")

    def get_stats(self) -> dict:
        st = BmgdStats()
        self._check(self._lib.bmgd_get_stats(self._h, ctypes.byref(st)), "bmgd_get_stats")
        return st.as_dict()

    def debug_perm(self, seed: int, chain: int, rnd: int, N0: int) -> np.ndarray:
        out = np.empty(N0, dtype=np.uint32)
        self._check(self._lib.bmgd_debug_perm(self._h, int(seed) & 0xFFFFFFFFFFFFFFFF, chain, rnd, N0,
                                              out.ctypes.data), "bmgd_debug_perm")
        return out

    def debug_wait_timeout(self, budget_ms: float) -> None:
        self._check(self._lib.bmgd_debug_wait_timeout(self._h, float(budget_ms)), "bmgd_debug_wait_timeout")

    def debug_null_rounds(self, rows: int, rounds: int, batch_size: int) -> None:
        """Launch the step kernel's latency probe: all waits, exchanges and updates of `rounds` rounds, no rows."""
        self._check(self._lib.bmgd_debug_null_rounds(self._h, rows, rounds, batch_size), "bmgd_debug_null_rounds")

    def close(self) -> None:
        if getattr(self, "_h", None) is not None and self._h:
            self._lib.bmgd_destroy(self._h)
            self._h = ctypes.c_void_p()
        self._workspace = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def __enter__(self):
        return self

    def __exit__(self, *exc):
        self.close()
