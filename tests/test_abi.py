"""The C-ABI shared library: it loads without a GPU, exports every function that
include/solo.h declares, and its host-only entry points behave (no compute calls here)."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import oracle

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def B():
    import __graft_entry__ as ge
    ge.build()
    from paper_2505_00347_b200 import binding
    return binding


def declared_functions():
    text = open(os.path.join(ROOT, "include", "solo.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(solo_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(B):
    names = declared_functions()
    assert {"solo_state_create", "solo_step", "solo_multi_step", "solo_dequant"} <= set(names)
    lib = C.CDLL(str(B.LIB_PATH))
    for n in names:
        assert hasattr(lib, n), n


def test_host_only_entry_points(B):
    for numel, bm, bv, blk in [(1, 2, 3, 64), (129, 4, 4, 128), (2049, 3, 8, 2048), (6_738_415_616, 2, 2, 128)]:
        assert B.state_bytes(numel, bm, bv, blk) == oracle.state_bytes(numel, bm, bv, blk)
    with pytest.raises(B.SoloError):
        B.state_bytes(10, 5, 4, 128)
    with pytest.raises(B.SoloError):
        B.state_bytes(10, 4, 4, 100)
    assert "aligned" in B.strerror(B.SOLO_EALIGN) and B.strerror(0) == "ok"
    # the paper's defaults (Sec. 3.4): 4 bit 0.8 / 0.3, 2 bit 0.5 / 0.1
    assert B.default_beta1(4) == pytest.approx(0.8) and B.default_beta1(4, True) == pytest.approx(0.3)
    assert B.default_beta1(2) == pytest.approx(0.5) and B.default_beta1(2, True) == pytest.approx(0.1)
    assert B.default_beta1(3) == pytest.approx(0.6) and B.default_beta1(3, True) == pytest.approx(0.2)
    assert B.default_beta1(8) == pytest.approx(0.9)
    assert B.launch_count() >= 0


def test_library_codebook_equals_oracle_codebook(B):
    """Two independent constructions of the signed DE levels give the same binary32 values."""
    for b in (2, 3, 4, 8):
        assert np.array_equal(B.codebook_m(b).numpy(), oracle.codebook(oracle.DE_SIGNED, b))
        for sel, kind in ((1, oracle.DE_UNSIGNED), (2, oracle.LINEAR_UNSIGNED), (3, oracle.LINEAR_NOZERO)):
            assert np.array_equal(B.codebook_v(sel, b).numpy(), oracle.codebook(kind, b)), (sel, b)
    with pytest.raises(B.SoloError):
        B.codebook_v(0, 4)


def test_hyper_records_agree(B):
    """The oracle's and the library's hyper-parameter records have the same layout."""
    assert C.sizeof(B.Hyper) == C.sizeof(oracle.Hyper) == 72
    for (n1, t1), (n2, t2) in zip(B.Hyper._fields_, oracle.Hyper._fields_):
        assert n1 == n2 and t1 is t2


def test_product_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2505_00347_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "import oracle" not in src and "from oracle" not in src and "solo_oracle" not in src, f
