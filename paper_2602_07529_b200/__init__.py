"""B200-native topology-aware (DAG) attention with adaptive position indices.

``synth``   seeded synthetic workloads (inputs only)
``binding`` thin ctypes binding over the C-ABI library ``libmedverse_attn.so`` (loaded on first use;
            raises if the library has not been built -- there is no CPU fallback)
"""
from . import synth  # noqa: F401

__all__ = ["synth", "binding"]


def __getattr__(name):
    if name == "binding":
        import importlib
        return importlib.import_module(".binding", __name__)
    raise AttributeError(name)
