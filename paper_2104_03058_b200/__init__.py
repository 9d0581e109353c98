"""gnnfd: feature-decomposed GNN aggregation (GCN, GraphSAGE mean, GAT) on one B200.

The work is done by libgnnfd.so (hand-written CUDA behind a C ABI, declared in include/gnnfd.h);
``binding`` marshals torch tensors into it.  Build the library with ``build.build_library()``.
"""
import importlib

from . import build  # noqa: F401


def __getattr__(name):
    # the binding is imported on first use so that the package can be imported before the library is built
    if name.startswith("__") or name == "binding":
        raise AttributeError(name)
    binding = importlib.import_module(__name__ + ".binding")
    try:
        return getattr(binding, name)
    except AttributeError:
        raise AttributeError("module %r has no attribute %r" % (__name__, name)) from None
