"""B200-native DARK random-feature attention (data-aligned kernel exp(q^T Sigma k), Sigma = M^T M).

The compute lives in ``libdarkattn.so`` (hand-written CUDA for sm_100a behind a C ABI, declared in
``include/darkattn.h``); ``binding`` marshals arguments to it. ``inputs`` draws the synthetic
workloads and has no dependency on the CUDA library.
"""

__all__ = ["binding", "inputs"]


def __getattr__(name):
    if name in __all__:
        import importlib
        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
