"""B200-native fused 4-bit AdamW step (arXiv 2309.01507): CUDA kernels behind a C-ABI library.

`paper_2309_01507_b200.lpmm` is the thin ctypes binding of include/lpmm.h; it is imported lazily
so that the shape/gradient generators in `workloads` can be used without the CUDA library.
"""

__all__ = ["lpmm", "workloads"]


def __getattr__(name):
    if name in ("lpmm", "workloads"):
        import importlib
        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
