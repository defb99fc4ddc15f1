"""n-softsync parameter-server update (arXiv 1511.05950) as sm_100a CUDA kernels behind a C ABI.

`binding` loads libsoftsync_ps.so and mirrors its entry points; everything it exports is reachable
from this package (`paper_1511_05950_b200.ParameterServer`, `.ps_create`, ...).  The binding is
loaded on first use, so that `paper_1511_05950_b200.build` can be imported to build the library
first; using anything else without the built library raises (there is no CPU fallback).
"""
import importlib


def __getattr__(name):
    if name.startswith("__"):
        raise AttributeError(name)
    if name == "build":                      # importable before the library exists
        return importlib.import_module(".build", __name__)
    binding = importlib.import_module(".binding", __name__)
    if name == "binding":
        return binding
    try:
        return getattr(binding, name)
    except AttributeError:
        raise AttributeError("module %r has no attribute %r" % (__name__, name)) from None
