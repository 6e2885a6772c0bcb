"""B200 library for the local arithmetic of the sparsity-aware secret-shared FFN
(Comet, arXiv 2505.07239): mask compaction, Beaver open/combine over the active
neurons only, and local truncation, behind a small C ABI.

`binding` loads the CUDA shared library and raises if it is missing (there is
no CPU fallback); `workloads` draws the seeded synthetic inputs; `build`
compiles the library in-tree.
"""

__all__ = ["binding", "workloads", "build"]


def __getattr__(name):
    if name in __all__:
        import importlib

        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
