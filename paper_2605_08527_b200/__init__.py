"""B200-native multi-tenant LoRA linear layer (forward + backward) behind a C-ABI CUDA library.

`binding` mirrors include/marlaas.h one to one; `workloads` holds the seeded synthetic inputs.
Importing the package does not load the CUDA library; the first call does, and raises if it is absent.
"""
from . import workloads  # noqa: F401


def __getattr__(name):
    if name == "binding" or name.startswith("marlaas_") or name in ("AdapterPool", "Segments", "MarlaasError",
                                                                    "load_library"):
        import importlib
        b = importlib.import_module(".binding", __name__)
        return b if name == "binding" else getattr(b, name)
    raise AttributeError(name)
