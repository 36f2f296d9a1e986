"""B200 (sm_100a) k-means clustering path of ClusComp: thin Python binding over the C ABI.

`binding` loads `libcluscomp.so` and exposes the `cc_*` calls under the same names;
`workloads` holds the seeded synthetic inputs.  There is no CPU fallback: every call
raises if the CUDA library cannot be loaded.
"""
from . import workloads  # noqa: F401

__all__ = ["workloads", "binding"]


def __getattr__(name):
    if name == "binding":
        import importlib
        return importlib.import_module(".binding", __name__)
    raise AttributeError(name)
