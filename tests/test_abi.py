"""Host-side checks that need no GPU: the library loads, exports what the header declares, and
rejects bad arguments with the documented codes."""
import ctypes
import os
import re

import pytest

from paper_2312_08728_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def header_symbols():
    text = open(os.path.join(ROOT, "include", "bmgd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(bmgd_[a-z_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    L = binding.load_library()
    syms = header_symbols()
    assert len(syms) >= 16
    for s in syms:
        assert hasattr(L, s), s
    assert set(syms) == set(binding.EXPORTS)


def test_version_and_strerror():
    L = binding.load_library()
    assert L.bmgd_version() >= 1000
    for code in range(-9, 1):
        assert L.bmgd_strerror(code)
    assert b"unknown" in L.bmgd_strerror(-99)


def make_cfg(**kw):
    L = binding.load_library()
    c = binding.BmgdConfig()
    L.bmgd_config_init(ctypes.byref(c))
    c.N, c.p, c.K = 1000, 10, 5
    for k, v in kw.items():
        setattr(c, k, v)
    return c


def ws(c):
    b = ctypes.c_int64(-1)
    return binding.load_library().bmgd_workspace_bytes(ctypes.byref(c), ctypes.byref(b)), b.value


def test_config_defaults():
    c = make_cfg()
    assert (c.loss, c.dtype, c.C, c.Rc, c.device) == (0, 1, 1, 1, -1)
    assert ctypes.sizeof(binding.BmgdConfig) == 120
    assert ctypes.sizeof(binding.BmgdStats) == 80


def test_workspace_size_counts_slots_theta_and_exchange():
    rc, b = ws(make_cfg())
    assert rc == 0
    slots = 2 * (200 * 10 * 4 + 200 * 4)
    assert b >= slots
    rc, b2 = ws(make_cfg(flags=binding.FLAG_NO_SLOTS))
    assert rc == 0 and b2 < b and b - b2 >= slots
    rc, b64 = ws(make_cfg(dtype=0))
    assert rc == 0 and b64 > b


@pytest.mark.parametrize("kw,code", [
    (dict(N=0), binding.ERR_ARG), (dict(p=0), binding.ERR_ARG), (dict(K=0), binding.ERR_ARG),
    (dict(K=2000), binding.ERR_ARG), (dict(loss=3), binding.ERR_ARG), (dict(dtype=7), binding.ERR_ARG),
    (dict(Rc=0), binding.ERR_ARG), (dict(C=3), binding.ERR_ARG), (dict(cluster_size=3), binding.ERR_ARG),
    (dict(threads_per_cta=100), binding.ERR_ARG), (dict(threads_per_cta=300), binding.ERR_ARG),
    (dict(producer_warps=9), binding.ERR_ARG), (dict(lanes_per_row=5), binding.ERR_ARG),
    (dict(pipeline_depth=1), binding.ERR_ARG), (dict(pipeline_depth=9), binding.ERR_ARG),
    (dict(loss=2, C=1, dtype=2), binding.ERR_ARG), (dict(loss=2, C=10, dtype=1), binding.ERR_UNIMPLEMENTED),
    (dict(loss=0, dtype=2), binding.ERR_UNIMPLEMENTED), (dict(N=2**40, K=1), binding.ERR_ARG),
])
def test_bad_configs_are_rejected(kw, code):
    assert ws(make_cfg(**kw))[0] == code


def test_null_pointers_are_rejected_without_a_device():
    L = binding.load_library()
    assert L.bmgd_workspace_bytes(None, None) == binding.ERR_ARG
    assert L.bmgd_create_ex(None, None) == binding.ERR_ARG
    assert L.bmgd_sync(None) == binding.ERR_ARG
    assert L.bmgd_get_theta(None, None, 0) == binding.ERR_ARG
    assert L.bmgd_destroy(None) == 0
    assert L.bmgd_last_cuda_error(None) == 0


def test_no_cpu_fallback():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    with pytest.raises(RuntimeError):
        binding.Bmgd(1000, 10, 5)
