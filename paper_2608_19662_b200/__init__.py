"""Resource-routed attention for B200 (sm_100a): a C-ABI CUDA library
(librecache.so, declared in include/recache.h) plus this thin binding.

    from paper_2608_19662_b200 import ReCache      # needs a CUDA device
    from paper_2608_19662_b200 import workloads    # seeded synthetic inputs (CPU)

Importing the package does not load the shared library; creating a ReCache
context does, and fails loudly if it is missing.
"""
from . import workloads  # noqa: F401


def __getattr__(name):
    if name in ("ReCache", "ReCacheError", "load_library", "PACKED", "PAGED", "F32", "BF16", "binding"):
        import importlib
        binding = importlib.import_module(__name__ + ".binding")
        return binding if name == "binding" else getattr(binding, name)
    raise AttributeError(name)
