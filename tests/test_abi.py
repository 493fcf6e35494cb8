"""The C-ABI library loads and exports every symbol include/ripple.h declares (no GPU needed),
and the binding's struct layouts agree with the header."""
import ctypes
import os
import re

import pytest

from paper_2601_12347_b200 import build as B
from paper_2601_12347_b200 import ripple

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    B.build_library()
    return ripple.load_library()


def header_functions(name="ripple.h"):
    text = open(os.path.join(ROOT, "include", name)).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ripple_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = header_functions()
    assert set(names) == set(ripple.EXPORTED)
    for n in names:
        assert getattr(lib, n) is not None
    part = header_functions("ripple_part.h")
    assert set(part) == set(ripple.EXPORTED_PART)
    for n in part:
        assert getattr(lib, n) is not None
    assert sorted(os.listdir(os.path.join(ROOT, "include"))) == ["ripple.h", "ripple_part.h"]


def test_version_and_null_handling(lib):
    assert b"sm_100a" in lib.ripple_version()
    # calls that need no device work reject null handles with INVALID_ARG instead of crashing
    assert lib.ripple_get_stats(None, None) == ripple.ERR_INVALID_ARG
    assert lib.ripple_apply_batch(None, None, 0, None, 0, 0) == ripple.ERR_INVALID_ARG
    assert lib.ripple_recompute_full(None) == ripple.ERR_INVALID_ARG
    out = ctypes.c_void_p(123)
    assert lib.ripple_create(None, None, 0, None, 2, 0, None, ctypes.byref(out)) == ripple.ERR_INVALID_ARG
    assert out.value is None
    assert b"null" in lib.ripple_last_error(None)
    lib.ripple_destroy(None)


def test_struct_sizes_match_the_header(tmp_path):
    """sizeof of every struct, as a C compiler sees the header, equals the ctypes mirror."""
    import subprocess
    src = tmp_path / "sizes.c"
    src.write_text(
        '#include <stdio.h>\n#include "ripple_part.h"\n'
        'int main(void){printf("%zu %zu %zu %zu %zu %zu %zu\\n", sizeof(ripple_update), sizeof(ripple_graph),'
        ' sizeof(ripple_layer), sizeof(ripple_options), sizeof(ripple_stats), sizeof(ripple_part_exports),'
        ' sizeof(ripple_part_ipc)); return 0;}\n')
    exe = tmp_path / "sizes"
    subprocess.check_call(["gcc", "-I", os.path.join(ROOT, "include"), str(src), "-o", str(exe)])
    got = [int(x) for x in subprocess.check_output([str(exe)]).split()]
    want = [ripple.UPDATE_DTYPE.itemsize] + [ctypes.sizeof(t) for t in
                                             (ripple._Graph, ripple._Layer, ripple._Options, ripple._Stats,
                                              ripple._PartExports, ripple._PartIpc)]
    assert got == want


def test_missing_library_fails_loudly(tmp_path):
    with pytest.raises(FileNotFoundError):
        ripple.load_library(str(tmp_path / "libripple.so"))
