"""B200-native fused policy-gradient loss over the LM head (TRLOO + mismatch rejection sampling).

`binding` wraps the C ABI of libdrk.so one to one; `dp` strings the library calls together with the
`torch.distributed` exchanges of the multi-GPU forms; `build` compiles the library.  Submodules are
imported on first use.
"""
import importlib

__all__ = ["binding", "dp", "build"]


def __getattr__(name):
    if name in __all__:
        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
