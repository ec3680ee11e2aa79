"""B200-native implementation of the XKV hot path: importance scoring, per-layer budget
allocation, top-k eviction into a ragged paged KV cache, and decode attention over it.

The compute lives in libxkv.so (hand-written CUDA for sm_100a behind a C ABI, see include/xkv.h);
`xkv` is the thin ctypes binding.  There is no CPU fallback: calling into the binding without the
built library raises.
"""
from . import workloads  # noqa: F401  (pure input generation, no compute)

__all__ = ["workloads", "xkv"]


def __getattr__(name):
    if name == "xkv":
        import importlib
        return importlib.import_module(".xkv", __name__)
    raise AttributeError(name)
