"""Host-side checks that need no GPU: the library loads and exports every symbol the header declares."""
import ctypes
import os
import re

import pytest
import torch

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


def test_device_error_word_maps_to_a_status_and_library_reads_no_environment():
    """A non-zero device error word is reported as BPC_ERR_DEVICE (6); diagnostic switches are explicit calls, so no
    source file of the library reads the environment."""
    from paper_2608_04405_b200 import binding as B
    assert B.lib.bpc_status_of_device_error(0) == B.BPC_OK
    for word in (1, 2, 4, 7):
        assert B.lib.bpc_status_of_device_error(word) == 6 and B.STATUS_NAMES[6] == "BPC_ERR_DEVICE"
    csrc = os.path.join(ROOT, "paper_2608_04405_b200", "csrc")
    for f in os.listdir(csrc):
        assert "getenv" not in open(os.path.join(csrc, f)).read(), "%s reads the environment" % f


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


def _binding():
    from paper_2608_04405_b200 import binding as B
    return B


def _b200_like_limits():
    """Resident clusters per size as a 148-SM part answers them: one block per SM, a cluster stays inside one GPC, GPCs of
    unequal size (this split reproduces the counts seen on a B200: 74 clusters of 2, 7 of 12 to 16, fewer than 16 of 8)."""
    gpcs = [10, 18, 20, 20, 20, 20, 20, 20]
    return [0] + [sum(g // c for g in gpcs) for c in range(1, 17)]


@pytest.mark.parametrize("batch,n_kv,n_max,want", [
    (1, 8, 131072 + 256, 10),      # 8 units: the largest size with all clusters resident (12+ hold only 7)
    (4, 8, 131072 + 256, 4),       # 32 units: 5 blocks each would need two waves
    (2, 8, 131072 + 256, 6),       # 16 units: 6 x 16 = 96 blocks in one wave, 8 x 16 would not be resident
    (5, 8, 131072 + 256, 3),       # 40 units
    (16, 8, 65536 + 64, 1),        # 128 units: one block each
    (1, 8, 1048576 + 64, 16),      # needs >= 13 blocks per unit; two waves either way, the smaller blocks win
    (1, 8, 4096, 4),               # a block keeps at least 1024 keys
])
def test_cluster_size_plan_on_given_device_limits(batch, n_kv, n_max, want):
    """The automatic cluster choice is host arithmetic over the device's occupancy answers: checked here on a table
    shaped like a 148-SM part, without a GPU."""
    B = _binding()
    cfg = B.make_config(batch, 4 * n_kv, n_kv, n_max, 128, torch.bfloat16)
    got = B.plan_cluster_size(cfg, _b200_like_limits(), 87000)
    assert got == want, (got, want)


def test_cluster_size_plan_edge_cases():
    B = _binding()
    cfg = B.make_config(1, 8, 8, 131072, 128, torch.bfloat16)
    ma = _b200_like_limits()
    assert B.plan_cluster_size(cfg, [0] * 17, 87000) == 0                 # nothing schedulable
    assert B.plan_cluster_size(cfg, ma, 1024) == 0                         # n_max fits no cluster: streaming applies
    only_pow2 = [v if c in (1, 2, 4, 8, 16) else 0 for c, v in enumerate(ma)]
    assert B.plan_cluster_size(cfg, only_pow2, 87000) == 8                 # sizes the device refuses are never chosen
    small = B.make_config(1, 8, 8, 1500, 128, torch.bfloat16)
    assert B.plan_cluster_size(small, ma, 87000) == 1                      # short contexts stay in one block
    got = B.plan_cluster_size(cfg, ma, 20000)                              # 131072 keys need >= 7 blocks of 20000
    assert got >= 7 and ma[got] >= 8
