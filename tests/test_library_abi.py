"""The C-ABI library loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "gelo.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(gelo_[a-z_0-9]+)\s*\(", text)))


@pytest.fixture(scope="module")
def lib():
    from paper_2603_05035_b200 import build
    return ctypes.CDLL(build.build())


def test_header_symbols_are_exported(lib):
    names = _declared()
    assert len(names) >= 20
    for name in names:
        assert hasattr(lib, name), f"{name} declared in gelo.h but not exported"


def test_binding_table_matches_header():
    from paper_2603_05035_b200 import binding
    assert sorted(binding.EXPORTS) == _declared()
    binding.load_library()


def test_host_only_entry_points(lib):
    from paper_2603_05035_b200 import binding
    L = binding.load_library()
    assert L.gelo_mixing_ld(1) == 64 and L.gelo_mixing_ld(64) == 64 and L.gelo_mixing_ld(68) == 128
    assert L.gelo_mixing_ld(4300) == 4352 and L.gelo_mixing_ld(0) == 0
    assert L.gelo_status_string(0) == b"ok" and b"condition" in L.gelo_status_string(3)
    small = L.gelo_workspace_bytes(64, 0, 256, 768, 0)
    big = L.gelo_workspace_bytes(4096, 204, 4096, 12288, 1)
    assert 0 < small < big < 4 << 30
    assert L.gelo_workspace_bytes(-1, 0, 8, 8, 0) == 0 and L.gelo_workspace_bytes(4, 0, 8, 8, 7) == 0
    # workspace demand grows with every size
    assert L.gelo_workspace_bytes(4096, 204, 4096, 12288, 1) > L.gelo_workspace_bytes(2048, 102, 4096, 12288, 1)
    # null context is rejected, never dereferenced
    assert L.gelo_set_workspace(None, None, 0) == binding.ERR_INVALID
    assert L.gelo_destroy(None) == binding.ERR_INVALID
    assert L.gelo_launch_count(None, 0) == -1


def test_block_diagonal_grouping_is_checked_on_the_host(lib):
    from paper_2603_05035_b200 import binding
    L = binding.load_library()
    ws = L.gelo_blockdiag_workspace_bytes
    base = ws(4096, 204, 4096, 12288, 1, 512, 32)
    assert base > 0
    assert ws(4096, 204, 4096, 12288, 1, 1024, 32) > base               # larger groups, larger per-lane scratch
    assert ws(4096, 204, 4096, 12288, 1, 500, 32) == 0                  # group size not a multiple of 64
    assert ws(4096, 204, 4096, 12288, 1, 64, 32) == 0                   # 68 groups: more than the 32 lanes
    assert ws(4, 0, 64, 192, 0, 64, 8) > 0 and ws(0, 0, 64, 192, 0, 64, 8) == 0
    assert ws(4096, 204, 4096, 12288, 7, 512, 32) == 0                  # unknown element type
    assert ws(4096, 204, 4096, 12288, 2, 512, 32) == base               # half and bfloat16 have the same footprint
