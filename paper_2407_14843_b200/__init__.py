"""B200-native batched solver for the joint horizontal+vertical scaling
problem of multi-model inference pipelines (Themis, arXiv 2407.14843).

``paper_2407_14843_b200.solver`` binds the C-ABI CUDA library;
``paper_2407_14843_b200.workloads`` draws seeded synthetic inputs.  The
solver module is imported lazily so that the input generators can be used
on a machine without the built library.
"""
__all__ = ["solver", "workloads"]


def __getattr__(name):
    if name in __all__:
        import importlib
        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
