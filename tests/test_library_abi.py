"""The C-ABI library builds, loads and exports every symbol the public header declares (no GPU needed)."""
import ctypes
import os
import re

from paper_2608_15522_b200 import binding as av
from paper_2608_15522_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "avsa.h")).read()
    return sorted(set(re.findall(r"AVSA_API\s+[\w\s\*]+?\b(avsa_\w+)\s*\(", text)))


def test_header_declares_the_three_calls():
    names = _declared_symbols()
    for n in ("avsa_cross_attn_scores", "avsa_build_block_mask", "avsa_sparse_self_attn"):
        assert n in names and n + "_workspace_bytes" in names


def test_library_builds_loads_and_exports_every_declared_symbol():
    path = build.build_library()
    assert os.path.exists(path)
    lib = ctypes.CDLL(path)
    for name in _declared_symbols():
        assert hasattr(lib, name), name
    assert sorted(av.EXPORTS) == sorted(n for n in _declared_symbols())


def test_host_only_entry_points():
    assert av.avsa_version() >= 100
    assert av.status_string(av.AVSA_OK) == "ok"
    assert "column list" in av.status_string(av.AVSA_ERR_BAD_MASK)
    assert av.avsa_count_from_percent(10, 140) == 14
    assert av.avsa_count_from_percent(5, 32760) == 1638
    assert av.avsa_count_from_percent(25, 256) == 64
    assert av.avsa_count_from_percent(20, 384) == 77
    assert av.avsa_count_from_percent(0, 100) == 0
    assert av.avsa_cross_attn_scores_workspace_bytes(1, 24, 256, 32760, 128) > 0
    assert av.avsa_build_block_mask_workspace_bytes(1, 24, 32760, 128, 128) > 2 * 24 * 256 * 128 * 4
    assert av.avsa_sparse_self_attn_workspace_bytes(1, 24, 32760, 128, 128) >= 16
    assert av.avsa_cross_attn_scores_workspace_bytes(1, 1, 1, 1, 96) == 0
