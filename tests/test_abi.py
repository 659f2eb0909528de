"""Host-side checks that need no GPU: the library loads and exports every symbol the header declares."""
import ctypes
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    src = open(os.path.join(ROOT, "include", "bpc.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    return sorted(set(re.findall(r"\b(bpc_[a-z_0-9]+)\s*\(", src)))


def test_library_exports_every_declared_symbol():
    from paper_2608_04405_b200 import binding as B
    names = _declared()
    assert len(names) >= 20
    lib = ctypes.CDLL(B.LIB_PATH)
    for n in names:
        assert hasattr(lib, n), "missing export %s" % n
    assert set(B.EXPORTS) == set(names)
    assert b"sm_100a" in B.lib.bpc_version()


def test_size_queries_and_config_validation_without_gpu():
    import torch
    from paper_2608_04405_b200 import binding as B
    cfg = B.make_config(4, 32, 8, 131072 + 256, 128, torch.bfloat16)
    assert B.lib.bpc_codes_bytes(ctypes.byref(cfg)) == 4 * 8 * (131072 + 256) * 16
    cfg64 = B.make_config(1, 1, 1, 4096, 64, torch.float32)
    assert B.lib.bpc_codes_bytes(ctypes.byref(cfg64)) == 4096 * 8        # one 64-bit word per key
    cfg32 = B.make_config(1, 4, 1, 4096, 32, torch.float32)
    assert B.lib.bpc_codes_bytes(ctypes.byref(cfg32)) == 4096 * 4        # half a word per key
    bad = B.make_config(1, 4, 1, 1024, 96, torch.bfloat16)
    assert B.lib.bpc_codes_bytes(ctypes.byref(bad)) == 0
    off = B.lib.bpc_fit_codes_offset(ctypes.byref(cfg64))
    assert 0 <= off < B.lib.bpc_fit_workspace_bytes(ctypes.byref(cfg64))   # (the fitted codes open the workspace)
    assert off % 256 == 0


def test_product_path_does_not_import_the_checker():
    pkg = os.path.join(ROOT, "paper_2608_04405_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                txt = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in txt, "%s mentions the checker" % f
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith(".py"):
            txt = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2608_04405_b200" not in txt and "ctypes" not in txt
