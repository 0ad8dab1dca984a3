"""The C-ABI library builds, loads and exports every function include/lsp.h declares (no GPU needed)."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = open(os.path.join(ROOT, "include", "lsp.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(lsp_[a-z_0-9]+)\s*\(", src)))


def test_library_exports_every_declared_symbol():
    from paper_2603_05454_b200 import build
    path = build.build()
    l = ctypes.CDLL(path)
    names = _declared()
    assert "lsp_init" in names and "lsp_denoise_step" in names and "lsp_commit" in names and "lsp_generate" in names
    for n in names:
        assert hasattr(l, n), n


def test_binding_lists_the_same_names():
    from paper_2603_05454_b200 import binding
    assert sorted(binding.EXPORTS) == _declared()


def test_sizes_and_argument_errors_without_gpu():
    from paper_2603_05454_b200 import binding as B
    mc = B.ModelCfg(2, 256, 4, 4, 64, 1024, 2048, 1e-5, 10000.0, 0, 2047)
    ws = B.lib.lsp_workspace_bytes(ctypes.byref(mc), 1, 96)
    kv = B.lib.lsp_kv_cache_bytes(ctypes.byref(mc), 1, 96)
    assert kv == 2 * 2 * 1 * 96 * 4 * 64 * 4
    assert ws > 2 * 2 * 96 * 256 * 4          # at least the staging buffer
    bad = B.ModelCfg(2, 250, 4, 4, 64, 1024, 2048, 1e-5, 10000.0, 0, 2047)
    assert B.lib.lsp_workspace_bytes(ctypes.byref(bad), 1, 96) == 0
    h = ctypes.c_void_p()
    assert B.lib.lsp_init(ctypes.byref(h), None, None, None, None, None, 0, 1, 96, None) == -1
    assert B.lib.lsp_commit(None, None) == -1


def test_internal_tuning_entry_is_exported_but_not_public():
    """The tuning and benchmark knobs live behind lsp_debug_set, declared in the package's internal header only."""
    from paper_2603_05454_b200 import build
    l = ctypes.CDLL(build.build())
    internal = open(os.path.join(ROOT, "paper_2603_05454_b200", "csrc", "lsp_tuning.h")).read()
    assert re.search(r"\bint\s+lsp_debug_set\s*\(", internal) and hasattr(l, "lsp_debug_set")
    assert "lsp_debug_set" not in _declared()
    public = re.sub(r"/\*.*?\*/", "", open(os.path.join(ROOT, "include", "lsp.h")).read(), flags=re.S)
    assert "tuning" not in public.lower()
