"""FLToP CTC on B200: batched, frame-pruned CTC prefix beam search (sm_100a).

``workloads`` holds the seeded input generators.  ``binding`` is the thin
ctypes layer over the C-ABI library; it is imported lazily so that the
generators stay usable on machines without the CUDA library, while every
decoding call fails loudly if the library is missing.
"""

__all__ = ["workloads", "binding"]


def __getattr__(name):
    if name in ("binding", "workloads"):
        import importlib
        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
