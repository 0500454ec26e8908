"""B200-native end-of-prefill KV retention pass of CompilerKV (arxiv 2602.08686).

``binding`` is the thin ctypes layer over the C-ABI library ``libckv.so`` (hand-written
sm_100a CUDA kernels); ``inputs`` builds the seeded synthetic workloads.  There is no CPU
fallback: every call fails loudly when the CUDA library is missing.
"""
from . import inputs  # noqa: F401

__all__ = ["inputs", "binding"]


def __getattr__(name):
    if name == "binding":
        import importlib
        return importlib.import_module(".binding", __name__)
    raise AttributeError(name)
