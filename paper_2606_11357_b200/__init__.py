"""B200-native fused W4A16 / W8A16 linear layer (TileFuse hot path).

`workloads` draws seeded inputs (pure numpy).  The compute entry points live in
`binding`, a thin ctypes layer over the C-ABI library `libtilefuse.so`; it is
imported lazily so that the input generators can be used without the library.
"""
__all__ = ["workloads", "binding"]


def __getattr__(name):
    if name in ("binding", "workloads"):
        import importlib
        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
