"""B200-native gf.apply hot path (CSR and generated-radius traversals) behind a C ABI.

The product is ``libtiga.so`` (hand-written CUDA for sm_100a, declared in ``include/tiga.h``).
This package is only the thin Python binding, :mod:`paper_2609_24802_b200.api`, which marshals
torch CUDA tensors into the C calls; its names are re-exported here on first use.  There is no
CPU fallback: touching any of them raises ImportError when the library has not been built
(``python -m paper_2609_24802_b200.build``).
"""


def __getattr__(name):
    if name in ("api", "build"):
        import importlib
        return importlib.import_module("." + name, __name__)
    from . import api
    try:
        return getattr(api, name)
    except AttributeError:
        raise AttributeError(f"module {__name__!r} has no attribute {name!r}") from None
