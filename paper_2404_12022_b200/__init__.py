"""B200-native tree-verify step of Hidden Transfer decoding.

Four operations behind a C ABI (``libht.so``, hand-written CUDA for sm_100a):
hidden-transfer projection, tree attention against a KV cache, greedy acceptance and
KV compaction.  ``binding`` holds the Python entry points of the same names;
``workloads`` holds the seeded synthetic inputs.  There is no CPU fallback: calling an
operation without the built library raises.
"""
from . import workloads  # noqa: F401

__all__ = ["workloads", "binding"]


def __getattr__(name):
    if name == "binding":
        import importlib
        return importlib.import_module(".binding", __name__)
    raise AttributeError(name)
