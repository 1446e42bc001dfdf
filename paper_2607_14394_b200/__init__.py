"""B200-native truncated spectral layer (the single-GPU hot path of DTST).

`from paper_2607_14394_b200 import Plan` gives the ctypes binding of the C-ABI
library `libdtst.so`; `paper_2607_14394_b200.inputs` holds the seeded synthetic
input generators.  The binding is imported lazily so that the input generators
can be used without torch or the built library.
"""

__all__ = ["Plan", "FNO", "binding", "inputs", "build"]


def __getattr__(name):
    if name == "Plan":
        from .binding import Plan
        return Plan
    if name == "FNO":
        from .fno import FNO
        return FNO
    if name in ("binding", "inputs", "build"):
        import importlib
        return importlib.import_module("." + name, __name__)
    raise AttributeError(name)
