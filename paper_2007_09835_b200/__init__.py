"""B200-native library for the RT3D conv3d hot path (KGS / vanilla structured sparsity).

`paper_2007_09835_b200.binding` is the thin ctypes face of librt3d.so (built in-tree by
`paper_2007_09835_b200.build`).  Attribute access on the package forwards to the binding,
so `import paper_2007_09835_b200 as rt3d; rt3d.rt3d_conv3d_sparse(...)` works; the build
module stays importable before the library exists.
"""


_SUBMODULES = ("build", "binding", "nets", "dist", "sweep")


def __getattr__(name):
    import importlib
    if name in _SUBMODULES:             # `from package import build` must not load the (possibly stale) library
        return importlib.import_module(__name__ + "." + name)
    binding = importlib.import_module(__name__ + ".binding")
    try:
        return getattr(binding, name)
    except AttributeError:
        raise AttributeError(f"module {__name__!r} has no attribute {name!r}") from None
