"""Structured tensor algebra on densely packed layouts for NVIDIA B200 (sm_100a).

The product is ``libdastac.so`` (C ABI, see ``include/dastac.h``); this package is its Python
binding.  The binding needs the built library: ``python -m paper_2407_13726_b200.build``.  It is
loaded on first use of any public name, so that the build module itself can be imported before the
library exists; a missing library raises ImportError at that point (there is no other code path).
"""
import importlib

_PUBLIC = ("DastacError", "Structure", "contract", "contract_workspace", "launch_count", "pack",
           "rank", "rank_batch", "status_string", "structure_count", "structure_create", "unpack",
           "unrank", "unrank_batch", "trimm_bf16_noalloc", "device_error", "selftest_wait_expiry", "piecewise_fuse", "KIND_GENERIC", "Rule", "mttkrp_split_tf32", "bandmm_split_tf32", "ttm_split_tf32", "NOALLOC_MAX_N", "F32", "BF16", "MEM_DEVICE", "MEM_HOST", "KIND_EMPTY",
           "KIND_DENSE", "KIND_UPPER", "KIND_LOWER", "KIND_BAND_DIAGONALS", "KIND_TETRAHEDRON", "KIND_BAND_EXACT", "KIND_UPPER_SHIFTED", "KIND_BAND_OFFSETS", "KIND_PLANE",
           "LAYOUT_LEXICOGRAPHIC", "LAYOUT_PADDED_DIAGONALS", "EXPORTS", "LIB_PATH")

__all__ = list(_PUBLIC)


def __getattr__(name):
    if name.startswith("__"):
        raise AttributeError(name)
    if name in ("build", "binding"):
        return importlib.import_module("." + name, __name__)
    binding = importlib.import_module(".binding", __name__)
    try:
        value = getattr(binding, name)
    except AttributeError:
        raise AttributeError(f"module {__name__!r} has no attribute {name!r}") from None
    globals()[name] = value
    return value
