"""Host-side checks that need no GPU: the library builds, loads and exports every symbol that
include/ps.h declares; configuration checks run on the host."""
import ctypes as C
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    import paper_2410_05589_b200 as ps
    from paper_2410_05589_b200.binding import EXPORTS
    lib = ps.load_library()
    header = open(os.path.join(ROOT, "include", "ps.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(ps_[a-z_0-9]+)\s*\(", header))
    assert declared == set(EXPORTS), declared ^ set(EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_workspace_bytes_and_config_checks_on_host():
    from paper_2410_05589_b200.binding import load_library, ps_config
    lib = load_library()
    ok = ps_config(1, 5120, 40, 40, 128, 13824, 32000, 4, 1, 1024 + 5, 10000.0, 1e-5, 0)
    n = lib.ps_workspace_bytes(C.byref(ok))
    kv = 2 * 40 * 1029 * 128 * 2
    # (scratch is sized for the 128 rows the tensor-core path takes, whatever max_batch is)
    assert kv < n < kv + (160 << 20)
    for field, bad in (("head_dim", 96), ("hidden", 5121), ("k_masks", 16), ("max_batch", 0),
                       ("max_batch", 129), ("dtype", 2), ("n_kv_heads", 3), ("max_ctx", 2)):
        cfg = ps_config(1, 5120, 40, 40, 128, 13824, 32000, 4, 1, 1029, 10000.0, 1e-5, 0)
        setattr(cfg, field, bad)
        assert lib.ps_workspace_bytes(C.byref(cfg)) == 0, field
    assert lib.ps_workspace_bytes(None) == 0
    # null arguments come back as a status, not a crash
    assert lib.ps_kv_len(None, 0, None) == -1
    assert lib.ps_poll(None, None) == -1
    assert lib.ps_verify(None, 1, 1, 1, None, None, None, 1.0, 0, 0, None, None, None, None) == -1


def test_no_oracle_in_product_path():
    """The package and the benchmark's GPU path never import the oracle."""
    pkg = os.path.join(ROOT, "paper_2410_05589_b200")
    for dp, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dp, f)).read()
                assert "oracle" not in text.lower(), os.path.join(dp, f)
