"""B200-native hot path of DEER's draft-verify step (block attention over a
paged KV cache, LM head with fused selection, acceptance rule, KV commit) as a
C-ABI CUDA library with a thin ctypes binding.

``workload`` draws the seeded synthetic inputs; ``binding`` mirrors
``include/deer.h``; ``runner`` owns device buffers for one step.  Nothing here
falls back to the CPU: without ``libdeer.so`` every call raises.
"""
from . import workload  # noqa: F401  (pure input generation; importable without the library)

__all__ = ["workload", "binding", "runner", "build"]


def __getattr__(name):
    if name in ("binding", "runner", "build"):
        import importlib
        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
