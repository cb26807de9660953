"""Batch-invariant paged attention for NVIDIA B200 (sm_100a).

The product is the C-ABI library built from ``csrc/`` (entry points declared
in ``include/vosti.h``); :mod:`paper_2609_38981_b200.binding` marshals
arguments to it and nothing more.  :mod:`paper_2609_38981_b200.inputs` draws
the seeded synthetic workloads.

The binding is loaded on first use so that the input generators can be
imported on a machine without the built library; any use of the binding
without it raises.
"""
__all__ = ["binding", "inputs"]


def __getattr__(name):
    if name in __all__:
        import importlib
        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
