"""B200-native (sm_100a) implementation of the prefill-end KV-cache compression pass of UNComp
(arXiv 2410.03090): truncated matrix entropy -> token budgets -> window scores + selection -> compaction.

`binding` wraps the C ABI of include/uncomp.h; `synth` makes seeded synthetic workloads.  Importing
`binding` loads the CUDA library and fails loudly when it is missing; nothing here computes on the CPU.
"""
from . import synth  # noqa: F401

__all__ = ["synth", "binding", "compress"]


def __getattr__(name):
    if name in ("binding", "compress"):
        import importlib
        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
