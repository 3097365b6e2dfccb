"""CPU-side checks of the C-ABI library: it loads and exports every function the header declares
(no compute calls here), workspace sizing is host arithmetic, and the oracle and the CUDA sources
are independent of each other."""
import os
import re

import paper_2407_08330_b200 as P
from paper_2407_08330_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_library_exports_every_declared_symbol():
    declared, missing = P.exported_symbols()
    assert {"hdt_build_index", "hdt_attn_fwd", "hdt_attn_bwd"} <= set(declared)
    assert missing == []


def test_workspace_bytes_host_arithmetic():
    assert P.hdt_index_workspace_bytes(4, 32768) > 0
    assert P.hdt_index_workspace_bytes(4, 32768, block_m=256) == 0      # invalid block_m
    assert P.hdt_index_workspace_bytes(-1, 10) == 0
    a = P.hdt_index_workspace_bytes(4, 1000)
    b = P.hdt_index_workspace_bytes(4, 2000)
    assert b > a


def test_oracle_and_cuda_path_share_nothing():
    for dirpath, _, files in os.walk(os.path.join(ROOT, "paper_2407_08330_b200")):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                txt = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"^\s*(from|import)\s+oracle\b", txt, re.M), f
                assert "hdt_oracle" not in txt, f
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".c")):
            txt = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2407_08330_b200" not in txt and "libhdt.so" not in txt, f
