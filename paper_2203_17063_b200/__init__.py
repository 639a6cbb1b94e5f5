"""Eventually consistent collectives on one B200 (sm_100a).

``binding``  ctypes front end of the CUDA library (the product path);
``inputs``   seeded synthetic inputs (no method arithmetic);
``build``    compiles the library in-tree with nvcc.

The binding is imported on first use so that the input generators can be used
on machines without the CUDA library.
"""
__all__ = ["binding", "inputs", "build"]


def __getattr__(name):
    if name in __all__:
        import importlib

        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
