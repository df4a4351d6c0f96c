"""B200 (sm_100a) implementation of the AQUA-KV per-token KV-cache codec.

`synth` (seeded synthetic inputs) imports without the CUDA library; `api` (the binding of
libaquakv.so) raises ImportError when the library has not been built -- there is no fallback.
"""
import importlib

__all__ = ["synth", "api", "build"]


def __getattr__(name):
    if name in __all__:
        return importlib.import_module("." + name, __name__)
    raise AttributeError(name)
