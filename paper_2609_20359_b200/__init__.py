"""libfls: the FL+FSDP / FL+HSDP sync step and FedAvg on one B200.

Thin ctypes binding of the C ABI declared in include/fls.h.  Every step of the path runs in the
CUDA library; this package only marshals arguments.  There is no CPU fallback: the first use of any
fls_* name loads libfls.so and raises if it is missing (build it with
`python -m paper_2609_20359_b200.build`).
"""
import importlib

_SUBMODULES = ("build", "session", "_binding")
__all__ = list(_SUBMODULES)


def __getattr__(name):
    # Submodules first (so that `from paper_2609_20359_b200 import build` works before the library exists);
    # every other name is looked up in the binding, which loads libfls.so on first use.
    if name in _SUBMODULES:
        return importlib.import_module("." + name, __name__)
    if name.startswith("__"):
        raise AttributeError(name)
    binding = importlib.import_module("._binding", __name__)
    try:
        return getattr(binding, name)
    except AttributeError:
        raise AttributeError(f"module {__name__!r} has no attribute {name!r}") from None
