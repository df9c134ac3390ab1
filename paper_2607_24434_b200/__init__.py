"""B200-native draft / verify MoE hot path of DraftExpert (expansion-aware
self-speculative decoding).  ``synth`` holds the seeded input generators;
``binding`` is the thin ctypes layer over the C-ABI CUDA library and is
imported on first use so that host-only tooling can import the package
without a GPU."""

__all__ = ["synth", "binding"]


def __getattr__(name):
    if name in __all__:
        import importlib

        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
