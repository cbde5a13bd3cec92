"""B200-native CoCoA round (local SCD solvers, update aggregation, duality gap) behind a C-ABI library.

``datagen`` draws the synthetic workloads; ``binding`` is the ctypes layer over ``libchicle.so``.
The binding is imported on first use so that the generators can be used without the CUDA library.
"""

__all__ = ["datagen", "binding"]


def __getattr__(name):
    if name in ("binding", "datagen", "build"):
        import importlib
        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
