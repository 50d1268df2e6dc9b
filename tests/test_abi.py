"""The C-ABI library loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

from paper_2609_36954_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "purlin.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = set(re.findall(r"\b(pl_[a-z_0-9]+)\s*\(", text))
    return sorted(names)


def test_library_exports_every_declared_symbol():
    lib = B.load()
    declared = _declared()
    assert len(declared) >= 20
    for name in declared:
        assert hasattr(lib, name), name
    assert sorted(B.EXPORTS) == declared


def test_struct_layouts_match_header_sizes():
    # sizes implied by the header's field lists (natural alignment, LP64)
    assert ctypes.sizeof(B.pl_ref_t) == 24
    assert ctypes.sizeof(B.pl_op_t) == 40 + 8 + 24 + 24 * 16 + 4 * 16 + 4 * 16
    assert ctypes.sizeof(B.pl_bufs_t) == 4 * 16 * 8
    assert ctypes.sizeof(B.pl_devstatus_t) == 32
    assert ctypes.sizeof(B.pl_sched_opts_t) == 64


def test_status_strings():
    assert B.status_string(B.PL_OK) == "ok"
    assert "timed out" in B.status_string(B.PL_ERR_TIMEOUT)
    assert B.pl_launch_count() >= 0
