"""pLogP collective-communication tuner on one B200: CUDA evaluation of the Broadcast / Scatter
cost models (Tables 1 and 2 of the paper), segment-size search and strategy selection.

The compute entry points live in the CUDA library and are reached through ``plogp`` (loaded on
first use; importing ``workloads`` alone does not need it)."""
import importlib

__all__ = ["plogp", "workloads"]


def __getattr__(name):
    if name in __all__:
        return importlib.import_module(__name__ + "." + name)
    raise AttributeError(name)
