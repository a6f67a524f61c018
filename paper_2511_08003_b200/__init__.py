"""SharpV pruning hot path for B200 (sm_100a): C-ABI CUDA library plus a thin binding.

``workloads`` draws seeded synthetic inputs and has no dependency on the CUDA
library; the binding (``binding`` and the ``sharpv_*`` names re-exported from
it) loads ``libsharpv.so`` on first use and raises if it is missing.
"""

__all__ = ["workloads"]


def __getattr__(name):
    if name.startswith("sharpv_") or name in ("binding", "Status", "SharpVError"):
        import importlib
        mod = importlib.import_module(__name__ + ".binding")
        return mod if name == "binding" else getattr(mod, name)
    raise AttributeError(name)
