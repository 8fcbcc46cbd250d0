"""B200-native row-parallel linear layer with partial channel-reduce (CAAT-Net hot path).

``paper_2506_19645_b200.caat`` is the Python binding of the C-ABI library (imported
on first attribute access so that ``synthetic`` can be used without the library).
"""
import importlib

__all__ = ["caat", "synthetic"]


def __getattr__(name):
    if name in __all__:
        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
