"""B200-native MoGA routed group-attention forward (CUDA library + thin binding).

``inputs`` holds the seeded synthetic workloads.  ``binding`` (loaded on first
attribute access) opens the C-ABI library ``csrc/libmoga.so``; there is no CPU
fallback, so a missing library raises at that point.
"""
from . import inputs  # noqa: F401

_BINDING_NAMES = ("binding",)


def __getattr__(name):
    if name == "binding":
        import importlib
        return importlib.import_module(".binding", __name__)
    raise AttributeError(name)
