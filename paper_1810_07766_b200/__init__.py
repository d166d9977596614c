"""B200-native RPS synchronisation step (unreliable parameter-server averaging).

The compute path lives in ``csrc/`` (CUDA, sm_100a) behind a C ABI declared in
``include/rps.h``; ``binding`` is the thin ctypes layer over it and is imported
lazily so that the input generators can be used without the built library.
"""

__all__ = ["workloads", "binding"]


def __getattr__(name):
    if name in ("binding", "RPS", "load_library"):
        import importlib

        mod = importlib.import_module(".binding", __name__)
        return mod if name == "binding" else getattr(mod, name)
    raise AttributeError(name)
