"""B200 (sm_100a) k-means-quantised linear layer: thin binding over libkmq.

The compute lives in the CUDA library under ``csrc/``; ``kmq`` (imported on
first use) only marshals arguments.  ``synth`` prepares seeded inputs.
"""
__all__ = ["kmq", "synth"]


def __getattr__(name):
    if name in ("kmq", "synth", "build"):
        import importlib
        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
