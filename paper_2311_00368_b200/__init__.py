"""B200-native SPMM / SDDMM / FusedMM over a CSR sparsity pattern (sm_100a).

``workloads``  seeded synthetic inputs (no arithmetic of the method)
``binding``    thin ctypes binding over the C-ABI library ``libb2sp.so`` (imported lazily;
               importing it raises if the CUDA library has not been built)
"""
from . import workloads  # noqa: F401

__all__ = ["workloads", "binding"]


def __getattr__(name):
    if name == "binding":
        import importlib
        return importlib.import_module(".binding", __name__)
    raise AttributeError(name)
