"""The C-ABI library loads and exports every entry point the header declares (no GPU, no compute calls)."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    names = set()
    for f in os.listdir(os.path.join(ROOT, "include")):
        if f.endswith(".h"):
            src = open(os.path.join(ROOT, "include", f)).read()
            src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
            names |= set(re.findall(r"\b(dab_[a-z0-9_]+)\s*\(", src))
    return names


@pytest.fixture(scope="module")
def lib():
    from paper_1804_02941_b200 import build
    build.build()
    import paper_1804_02941_b200 as d
    return d.lib()


def test_every_declared_symbol_is_exported(lib):
    import paper_1804_02941_b200 as d
    declared = _declared()
    assert declared and declared == set(d.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def test_sources_are_built_for_sm_100a():
    from paper_1804_02941_b200 import build
    assert "arch=compute_100a,code=sm_100a" in build.NVCC_FLAGS and build.sources()


def test_host_side_helpers_and_validation(lib):
    import paper_1804_02941_b200 as d
    assert [d.dab_words_per_row(n) for n in (1, 32, 33, 576, 577)] == [1, 1, 2, 18, 19]
    assert [d.dab_default_ld(n) for n in (1, 128, 129, 576, 2400)] == [4, 4, 8, 20, 76]
    assert d.status_string(0) == "ok" and "workspace" in d.status_string(3)
    # argument errors are found on the host before anything touches a device
    assert lib.dab_binarize(None, -1, 8, 8, None, None, None, None, 4, None, None) == 1
    assert lib.dab_binarize(None, 1, 20000, 20000, None, None, None, None, 628, None, None) == 2
    assert lib.dab_binarize(None, 0, 8, 8, None, None, None, None, 4, None, None) == 0
    assert lib.dab_pack(None, 1, 8, 4, None, 4, None, None) == 1
    assert lib.dab_binary_gemm(1, 1, 64, None, 2, None, None, None, None, 4, None, None, None, None, 1, None, 0, None) == 1
    desc = d.make_desc((2, 64, 56, 56), 64, 3, 3, (1, 1), (1, 1))
    assert d.dab_conv_output_size(desc) == (56, 56)
    assert d.dab_binary_conv_workspace(desc) >= 2 * 56 * 56 * (20 * 4 + 12)
    assert d.dab_binary_conv_host_workspace(desc) > d.dab_binary_conv_workspace(desc)
    assert d.dab_conv_output_size(d.make_desc((1, 1, 225, 225), 64, 15, 15, (3, 3), (0, 0))) == (71, 71)
    assert d.dab_binary_conv_workspace(d.make_desc((1, 64, 8, 8), 4, 17, 17, (1, 1), (8, 8))) == 0   # n > DAB_MAX_N
