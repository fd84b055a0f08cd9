"""B200-native evaluation of bit-accurate GPU MMA arithmetic models (C-ABI library + thin Python binding).

``paper_2511_10909_b200.mmasim`` is the binding (it needs the built ``libmmasim.so`` and fails loudly without
it), ``.build`` compiles the library in-tree, ``.workloads`` holds the seeded input generators.
"""
import importlib

_BINDING = ("ARCH", "FMT", "ACC", "FAMILY", "RHO", "Model", "MmasimError", "create_model", "gemm", "gemm_host",
            "dot_batch", "int_peak", "last_kernel", "library_path", "model_keys", "PEAK_KINDS", "hw_mma", "HW_KINDS", "error_stats", "STAT_NAMES")


def __getattr__(name):
    if name in _BINDING:
        return getattr(importlib.import_module(".mmasim", __name__), name)
    raise AttributeError(name)
