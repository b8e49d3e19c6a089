"""The C-ABI library builds for sm_100a, loads without a GPU and exports every symbol the header declares."""
import os
import re

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    from paper_2402_05109_b200.build import build
    build()
    import paper_2402_05109_b200 as pkg
    hdr = open(os.path.join(ROOT, "include", "hydra.h")).read()
    names = sorted(set(re.findall(r"\b(hydra_[a-z_0-9]+)\s*\(", hdr)))
    assert len(names) >= 18
    for n in names:
        assert hasattr(pkg.lib, n), n
    assert pkg.lib.hydra_status_str(3).decode() == "call out of order"


def test_workspace_bytes_and_invalid_configs_without_gpu():
    import ctypes as C
    from paper_2402_05109_b200.binding import lib, ModelCfgC, HeadCfgC, TreeCfgC
    mc = ModelCfgC(2, 256, 4, 64, 688, 1024, 1e-6, 1e4, 0, 1, 128)
    hc = HeadCfgC(3, 1, 0, 1)
    par = (C.c_int32 * 4)(-1, 0, 0, 1)
    n = lib.hydra_workspace_bytes(C.byref(mc), C.byref(hc), C.byref(TreeCfgC(4, par)))
    assert n > 2 * 2 * 4 * 128 * 64 * 4 and n % 256 == 0
    bad = (C.c_int32 * 4)(-1, 0, 1, 0)                       # rows not ordered by (depth, rank path)
    assert lib.hydra_workspace_bytes(C.byref(mc), C.byref(hc), C.byref(TreeCfgC(4, bad))) == 0
    deep = (C.c_int32 * 5)(-1, 0, 1, 2, 3)                   # deeper than the number of heads
    assert lib.hydra_workspace_bytes(C.byref(mc), C.byref(hc), C.byref(TreeCfgC(5, deep))) == 0
    mc.n_heads = 3                                           # n_heads * head_dim != d_model
    assert lib.hydra_workspace_bytes(C.byref(mc), C.byref(hc), C.byref(TreeCfgC(4, par))) == 0
