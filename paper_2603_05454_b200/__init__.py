"""B200-native Longest-Stable-Prefix decode path: ctypes binding over the CUDA C-ABI library.

The Python layer only marshals arguments; every step of the path runs in the library's kernels.
The binding is imported on first use and fails loudly when the compiled library is missing
(`python -m paper_2603_05454_b200.build` builds it); there is no CPU or PyTorch fallback.
"""
_NAMES = ("LSPDecoder", "SchedCfg", "lib", "LSPError", "linear_static", "FLAG_SNAPPED", "FLAG_FALLBACK", "FLAG_RANGE_UNACHIEVABLE",
          "FLAG_RUN_TO_END", "FLAG_NEAR_THRESHOLD", "FLAG_NEAR_TIE")
__all__ = list(_NAMES)


def __getattr__(name):
    if name in _NAMES:
        import importlib
        return getattr(importlib.import_module(__name__ + ".binding"), name)
    raise AttributeError(name)
