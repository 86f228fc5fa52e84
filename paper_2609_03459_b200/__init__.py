"""B200 (sm_100a) Tensor-Train embedding-bag: CUDA library + thin ctypes binding.

`paper_2609_03459_b200.build` compiles the shared library; everything else lives in
`paper_2609_03459_b200.binding` and is loaded on first use (it raises if the library is missing --
there is no CPU fallback)."""
import importlib

__all__ = ["build", "binding"]


def __getattr__(name):
    if name in ("build", "binding"):
        return importlib.import_module(f"{__name__}.{name}")
    b = importlib.import_module(f"{__name__}.binding")
    try:
        return getattr(b, name)
    except AttributeError:
        raise AttributeError(f"module {__name__!r} has no attribute {name!r}") from None
