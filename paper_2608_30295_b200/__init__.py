"""CateKV hot path for one NVIDIA B200: thin Python binding over libcatekv.so.

The API names are those of the C ABI (include/catekv.h) and are resolved on
first use from `.binding`, which loads the built CUDA library and raises if it
is missing - there is no other implementation behind these names.
`python -m paper_2608_30295_b200.build` compiles the library in-tree.
"""
import importlib

__all__ = ["binding", "build"]


def __getattr__(name):
    if name in ("binding", "build"):
        return importlib.import_module(f"{__name__}.{name}")
    b = importlib.import_module(f"{__name__}.binding")
    try:
        return getattr(b, name)
    except AttributeError:
        raise AttributeError(f"module {__name__!r} has no attribute {name!r}") from None
