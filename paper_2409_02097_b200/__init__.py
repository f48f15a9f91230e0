"""B200 (sm_100a) implementation of LinFusion's normalized non-causal linear attention.

``workloads`` builds seeded synthetic inputs; ``attn`` is the thin ctypes binding over the
C-ABI CUDA library (``include/linfusion_attn.h``).  The binding is imported lazily so that the
input generators can be used on machines without the compiled library.
"""

__all__ = ["workloads", "attn"]


def __getattr__(name):
    if name in ("attn", "workloads"):
        import importlib
        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
