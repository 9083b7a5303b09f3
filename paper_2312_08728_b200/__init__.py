"""B200-native buffered mini-batch gradient descent (BMGD).

The computation runs in a CUDA library (csrc/, C ABI in include/bmgd.h); `binding`
wraps it with ctypes, `inputs` draws the seeded synthetic workloads, `build`
compiles the library in-tree with nvcc.
"""
from . import inputs  # noqa: F401
from .inputs import WORKLOADS, Workload, buffer_seed  # noqa: F401


def __getattr__(name):
    # the binding loads (and if need be builds) the CUDA library: only on first use
    if name in ("Bmgd", "BmgdError", "load_library", "binding"):
        import importlib
        binding = importlib.import_module(__name__ + ".binding")
        return binding if name == "binding" else getattr(binding, name)
    raise AttributeError(name)
