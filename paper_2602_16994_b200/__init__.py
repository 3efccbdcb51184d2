"""B200-native batched draft-tree verification (SpecInfer / Traversal) behind a C-ABI library.

``paper_2602_16994_b200.synth`` builds seeded inputs; ``paper_2602_16994_b200.binding`` marshals
arguments into ``libspecverify.so`` (hand-written sm_100a CUDA).  There is no CPU fallback: calling
a verifier without the built library or without a CUDA device raises.
"""
from . import synth  # noqa: F401

__all__ = ["synth", "binding"]


def __getattr__(name):
    if name == "binding":
        import importlib
        return importlib.import_module(".binding", __name__)
    raise AttributeError(name)
