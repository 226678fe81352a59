"""B200-native D-PSGD hot path (Lian et al., arXiv 1705.09056): n simulated nodes on one GPU.

`workloads` builds seeded synthetic inputs; `binding` (loaded on first use) wraps the C-ABI
CUDA library `libdpsgd.so`.  There is no CPU fallback: using the binding without the built
library raises.
"""
from . import workloads  # noqa: F401

_LAZY = ("binding", "Dpsgd", "DpsgdError", "load_library")


def __getattr__(name):
    if name in _LAZY:
        import importlib
        b = importlib.import_module(__name__ + ".binding")
        return b if name == "binding" else getattr(b, name)
    raise AttributeError(name)
