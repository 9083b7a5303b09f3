"""The binding refuses tensors that do not match the job before any pointer reaches the library.

The C ABI sees bare pointers and sizes; a tensor of the wrong element type, column count or length would make a
kernel read or write past the end of an allocation.  These checks need no GPU: they run on the tensors' metadata.
"""
import pytest
import torch

from paper_2312_08728_b200 import binding
from paper_2312_08728_b200.inputs import (DTYPE_BF16, DTYPE_F32, DTYPE_F64, LOSS_LINEAR, LOSS_LOGISTIC, LOSS_SOFTMAX)


def good(rows=32, p=8, dtype=torch.float32, ydtype=None):
    return torch.zeros(rows, p, dtype=dtype), torch.zeros(rows, dtype=ydtype or dtype)


def test_a_matching_buffer_passes_and_reports_its_rows():
    x, y = good()
    assert binding.check_buffer(x, y, 8, LOSS_LINEAR, DTYPE_F32) == 32
    x, y = good(dtype=torch.float64)
    assert binding.check_buffer(x, y, 8, LOSS_LOGISTIC, DTYPE_F64, max_rows=32) == 32
    x, y = good(dtype=torch.bfloat16, ydtype=torch.int32)
    assert binding.check_buffer(x, y, 8, LOSS_SOFTMAX, DTYPE_BF16) == 32


@pytest.mark.parametrize("case", [
    "x_dtype", "x_columns", "x_rank", "y_short", "y_dtype", "labels_not_int32", "not_contiguous", "too_many_rows",
    "empty", "dtype_code",
])
def test_mismatches_are_refused(case):
    x, y = good()
    p, loss, dtype, cap = 8, LOSS_LINEAR, DTYPE_F32, None
    if case == "x_dtype":
        dtype = DTYPE_F64          # a float32 X under a float64 job: 8-byte reads past the end
    elif case == "x_columns":
        p = 12
    elif case == "x_rank":
        x = x.reshape(-1)
    elif case == "y_short":
        y = y[:-1].contiguous()
    elif case == "y_dtype":
        y = y.double()
    elif case == "labels_not_int32":
        x, y = good(dtype=torch.bfloat16, ydtype=torch.int64)
        loss, dtype = LOSS_SOFTMAX, DTYPE_BF16
    elif case == "not_contiguous":
        x = torch.zeros(32, 16)[:, :8]
    elif case == "too_many_rows":
        cap = 31
    elif case == "empty":
        x, y = good(rows=0)
    elif case == "dtype_code":
        dtype = 7
    with pytest.raises(ValueError):
        binding.check_buffer(x, y, p, loss, dtype, max_rows=cap)


def handle_without_a_gpu(N=64, p=8, K=2, loss=LOSS_LINEAR, dtype=DTYPE_F32):
    """A Bmgd object with the job's shape but no library handle: enough to reach the checks, which come first."""
    h = binding.Bmgd.__new__(binding.Bmgd)
    h.N, h.p, h.K, h.loss, h.dtype, h.C, h.Rc = N, p, K, loss, dtype, 1, 1
    h.device = torch.device("cpu")
    h._h = None
    h._lib = None
    return h


def test_load_buffer_checks_before_it_calls_the_library():
    h = handle_without_a_gpu()
    x, y = good(rows=32)
    with pytest.raises(ValueError):
        h.load_buffer(x.double(), y)                 # element type
    with pytest.raises(ValueError):
        h.load_buffer(torch.zeros(32, 9), y)         # column count
    with pytest.raises(ValueError):
        h.load_buffer(x, y[:16].contiguous())        # y shorter than X
    big_x, big_y = good(rows=33)
    with pytest.raises(binding.BmgdError) as e:
        h.load_buffer(big_x, big_y)                  # more rows than a slot of ceil(64/2) holds
    assert e.value.status == binding.ERR_CAPACITY
    # (with _lib = None a call that got past the checks would raise AttributeError instead)


def test_run_rounds_resident_checks_before_it_calls_the_library():
    h = handle_without_a_gpu(dtype=DTYPE_F64)
    x, y = good(rows=32)
    with pytest.raises(ValueError):
        h.run_rounds_resident(x, y, 1, 8, 0.1, 0)    # float32 tensors under a float64 job


def test_noalloc_checks_before_it_calls_the_library(monkeypatch):
    monkeypatch.setattr(binding, "load_library", lambda *a, **k: (_ for _ in ()).throw(AssertionError("reached the library")))
    x, y = good(rows=32)
    theta = torch.zeros(1, 8)
    with pytest.raises(ValueError):
        binding.run_rounds_noalloc(x, y, theta.double(), LOSS_LINEAR, DTYPE_F32, 1, 8, 0.1, 0)   # theta's type
    with pytest.raises(ValueError):
        binding.run_rounds_noalloc(x, y, torch.zeros(1, 9), LOSS_LINEAR, DTYPE_F32, 1, 8, 0.1, 0)  # theta's p against X
    with pytest.raises(ValueError):
        binding.run_rounds_noalloc(x, y, theta, LOSS_LINEAR, DTYPE_F64, 1, 8, 0.1, 0)            # float32 under float64
    with pytest.raises(ValueError):
        binding.run_rounds_noalloc(x, y, theta.reshape(-1), LOSS_LINEAR, DTYPE_F32, 1, 8, 0.1, 0)  # theta's rank
    with pytest.raises(ValueError):
        binding.run_rounds_noalloc(x, y, theta, LOSS_LINEAR, DTYPE_F32, 1, 8, 0.1, 0)            # host tensors
