"""B200 (sm_100a) token-routing hot path of Cobalt behind a C ABI (libcobalt.so).

`paper_2609_36959_b200.binding` mirrors the C entry points one to one (coact_stats, assign,
permute, combine, ...); `paper_2609_36959_b200.build` compiles the library in-tree.  The
binding is loaded on first use and raises if the shared library is missing: there is no
CPU or eager fallback.
"""
import importlib

__all__ = ["binding", "build"]


def __getattr__(name):
    if name in ("binding", "build", "router"):
        return importlib.import_module(f"{__name__}.{name}")
    binding = importlib.import_module(f"{__name__}.binding")
    try:
        return getattr(binding, name)
    except AttributeError:
        raise AttributeError(f"module {__name__!r} has no attribute {name!r}") from None
