"""B200-native hot path of Value-Aware Token Pruning (VATP).

`vatp` (the ctypes binding to libvatp.so) is loaded on first use so that the
synthetic-workload module can be imported on machines without the library.
"""
from importlib import import_module

__all__ = ["synth", "vatp", "build", "presets"]


def __getattr__(name):
    if name in __all__:
        return import_module(f"{__name__}.{name}")
    raise AttributeError(name)
