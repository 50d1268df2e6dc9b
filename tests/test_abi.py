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
    assert ctypes.sizeof(B.pl_bufs_t) == 6 * 16 * 8
    assert ctypes.sizeof(B.pl_devstatus_t) == 32
    assert ctypes.sizeof(B.pl_sched_opts_t) == 72


def test_status_strings():
    assert B.status_string(B.PL_OK) == "ok"
    assert "timed out" in B.status_string(B.PL_ERR_TIMEOUT)
    assert B.pl_launch_count() >= 0


def test_header_is_plain_c99():
    """The boundary is a C ABI: the header must compile as C99 on its own, no CUDA or C++ needed."""
    import subprocess
    import tempfile
    src = '#include "purlin.h"\nint main(void) { pl_sched_opts_t o; o.struct_size = sizeof o; return (int)pl_launch_count() * 0 + (int)o.struct_size * 0; }\n'
    with tempfile.TemporaryDirectory() as d:
        c = os.path.join(d, "t.c")
        open(c, "w").write(src)
        res = subprocess.run(["gcc", "-std=c99", "-pedantic", "-Wall", "-Werror", "-fsyntax-only",
                              "-I", os.path.join(ROOT, "include"), c], capture_output=True, text=True)
        assert res.returncode == 0, res.stderr


def test_product_never_touches_the_oracle():
    """The oracle is test infrastructure: nothing under the package may import, load or run it."""
    pkg = os.path.join(ROOT, "paper_2609_36954_b200")
    for base, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".cpp", ".h")):
                text = open(os.path.join(base, f)).read()
                for line in text.splitlines():
                    code = line.split("#")[0]
                    assert not ("import" in code and "oracle" in code), f"{f} imports the oracle"
                assert "liboracle" not in text and "collectives_oracle" not in text, f"{f} loads the oracle"
    # and the oracle does not reach into the product either
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith((".py", ".c")):
            text = open(os.path.join(ROOT, "oracle", f)).read()
            assert "paper_2609_36954_b200" not in text and "purlin" not in text.lower()
