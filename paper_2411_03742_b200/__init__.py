"""AdaCons (arXiv 2411.03742) gradient aggregation for NVIDIA B200 (sm_100a).

The product is the C-ABI shared library built from `csrc/`; `AdaCons` in `binding`
marshals arguments to it.  There is no CPU fallback: using the class without the built
library raises.
"""
from . import workloads  # noqa: F401


def __getattr__(name):
    if name in ("AdaCons", "AdaConsError", "load_library", "binding"):
        import importlib
        mod = importlib.import_module(".binding", __name__)
        return mod if name == "binding" else getattr(mod, name)
    raise AttributeError(name)
