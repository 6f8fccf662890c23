"""IndexMem decode / chunked-prefill hot path for NVIDIA B200 (sm_100a).

``paper_2605_25475_b200.binding`` is the thin ctypes layer over the C-ABI library
(``include/indexmem.h``); ``paper_2605_25475_b200.synth`` draws the seeded synthetic workloads.
The binding is imported lazily so that the workload generators can be used without the library.
"""

__all__ = ["binding", "synth", "buildlib"]


def __getattr__(name):
    if name in __all__:
        import importlib
        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
