"""B200-native fused Stochastic Gradient Push step (arXiv 1811.10792).

`binding` wraps the CUDA library (libsgp.so, built in-tree by `build`); `inputs` holds the seeded
synthetic workloads.  Importing `binding` (or any of the names re-exported below) raises if the
library has not been built: there is no CPU implementation behind this package.
"""
_LAZY = {"Sgp", "GraphDesc", "Schedule", "SgpError"}


def __getattr__(name):
    if name in _LAZY:
        from . import binding
        return getattr(binding, name)
    raise AttributeError(name)
