"""The C-ABI library loads without a GPU and exports every symbol the header declares."""
import ctypes
import os
import re

from paper_2607_17181_b200 import binding as tb

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "talaria.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(talaria_[a-z_]+)\s*\(", text)))


def test_library_builds_loads_and_exports_every_declared_symbol():
    tb.build()
    lib = ctypes.CDLL(tb.LIB_PATH)
    names = _declared()
    assert len(names) >= 20
    for n in names:
        assert hasattr(lib, n), n
    # the binding marshals exactly the declared entry points
    assert sorted(tb._SIGNATURES) == names


def test_status_strings_and_struct_sizes():
    lib = tb.lib()
    assert lib.talaria_strerror(0) == b"ok"
    for code in (-1, -2, -3, -4, -5, -6, -7, -9):
        assert lib.talaria_strerror(code) not in (b"ok", b"unknown status")
    assert ctypes.sizeof(tb.Match) == 32 == tb.MATCH_DTYPE.itemsize
    assert ctypes.sizeof(tb.Copy) == 40 == tb.COPY_DTYPE.itemsize
    assert ctypes.sizeof(tb.KvLayout) == 40 and ctypes.sizeof(tb.HostLayout) == 32
    assert ctypes.sizeof(tb.KvXfer) == 64


def test_prefix_agree_needs_no_gpu():
    import numpy as np
    h = np.array([[1, 2, 3, 4], [1, 2, 9, 4]], dtype=np.uint64)
    assert tb.Talaria.prefix_agree([4, 4], h) == 2
    assert tb.Talaria.prefix_agree([1, 4], h) == 1
    assert tb.Talaria.prefix_agree([4], h[:1]) == 4


def test_header_is_plain_c(tmp_path):
    import subprocess
    src = tmp_path / "hdr.c"
    src.write_text('#include "talaria.h"\nint main(void) { talaria_match_t m; (void)m; return TALARIA_OK; }\n')
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror", "-fsyntax-only",
                           "-I", os.path.join(ROOT, "include"), str(src)])
