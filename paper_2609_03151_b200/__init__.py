"""B200-native (sm_100a) BASP attention-layer hot path: group plan, in-HBM all-to-all
reshards, tcgen05 causal attention, and the fused layer, behind the C ABI of include/basp.h.

``binding`` (loaded on first attribute access) is the ctypes front end of libbasp.so;
``synth`` holds the seeded synthetic workloads, ``autograd`` wraps the forward and backward calls of the layer as one
differentiable torch operation, ``dist`` has the multi-GPU plumbing.  Nothing here computes on the CPU.
"""
import importlib

__all__ = ["binding", "synth", "build", "autograd", "dist"]


def __getattr__(name):
    if name in __all__:
        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
