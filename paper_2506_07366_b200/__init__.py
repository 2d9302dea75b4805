"""B200 (sm_100a) hot path of a Mixture-of-Experts layer with prediction-driven expert duplication.

The compute lives in libmoegps.so (hand-written CUDA behind a C ABI, see include/moegps.h);
`binding` marshals torch tensors into it, `layer.MoeLayer` chains the calls, `workloads` draws the
seeded synthetic inputs.  The library is loaded on first use and there is no other path.
"""
import importlib

from .workloads import WORKLOADS, Workload  # noqa: F401

_BINDING_NAMES = ("Context", "Shape", "MoegpsError", "workspace_bytes", "rcap", "error_string")


def __getattr__(name):
    # binding/layer are imported on first use so that the input generators stay usable on machines
    # where the shared library has not been built
    if name in _BINDING_NAMES:
        return getattr(importlib.import_module(__name__ + ".binding"), name)
    if name == "MoeLayer":
        return importlib.import_module(__name__ + ".layer").MoeLayer
    raise AttributeError(name)
