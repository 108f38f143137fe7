"""B200-native CWAC-fused quantized linear layer and CWAC calibration (QwT-v2).

The product is the C-ABI library ``libqwt2.so`` (CUDA, sm_100a).  This package is
a thin ctypes binding with the same entry points plus the seeded workload
generators.  There is no CPU fallback: importing :mod:`.binding` fails loudly
when the library has not been built.
"""
from . import workload  # noqa: F401


def __getattr__(name):
    # The binding is loaded on first use so that the workload generators stay
    # importable on machines where the CUDA library has not been built yet.
    if name == "binding":
        import importlib
        return importlib.import_module(".binding", __name__)
    raise AttributeError(name)
