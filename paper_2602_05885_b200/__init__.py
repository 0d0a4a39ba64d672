"""B200-native fused policy-gradient loss over the LM head (TRLOO + mismatch rejection sampling).

`binding` wraps the C ABI of libdrk.so one to one; `synth` draws seeded synthetic inputs;
`build` compiles the library.  Submodules are imported on first use so that `synth` can be used
without the shared library.
"""
import importlib

__all__ = ["binding", "synth", "build"]


def __getattr__(name):
    if name in __all__:
        return importlib.import_module(f"{__name__}.{name}")
    raise AttributeError(name)
