"""B200-native KV-cache store / retrieve / compose (the hot path of a Knowledge Delivery Network).

``paper_2409_13761_b200.kdn``    ctypes binding of the C-ABI library (loads libkdn.so; raises if absent)
``paper_2409_13761_b200.synth``  seeded synthetic pools and block tables
``paper_2409_13761_b200.build``  compiles csrc/ for sm_100a with nvcc
"""

__all__ = ["kdn", "synth", "build"]


def __getattr__(name):
    if name in __all__:
        import importlib
        return importlib.import_module("." + name, __name__)
    raise AttributeError(name)
