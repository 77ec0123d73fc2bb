"""The C-ABI library loads and exports every symbol include/aif.h declares; host-side logic of the boundary.
No compute call is made here (no GPU)."""
import ctypes as C
import os
import re

import pytest

from oracle import aif_oracle as orc
from paper_2511_12934_b200 import binding as B
from paper_2511_12934_b200 import build as libbuild
from paper_2511_12934_b200 import synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    libbuild.build()
    return B.load_library()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "aif.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(aif_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert len(names) >= 15
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(B.EXPORTS) == names


def test_struct_layouts_match_the_header(lib):
    # sizes follow from the header's field lists under the C ABI (natural alignment)
    assert C.sizeof(B.aif_config) == 120
    assert C.sizeof(B.aif_weights) == 8 + 4 * 8 + 4 * 8 + 10 * 8
    assert C.sizeof(B.aif_user_inputs) == 8 + 7 * 8 + 8
    assert C.sizeof(B.aif_item_weights) == 16 + 6 * 8
    cfg = B.make_config(dtype=B.BF16, M=1000, d=128, L_max=10, hidden=(512, 256), F=16, B=1024, dc=32)
    assert lib.aif_input_width(C.byref(cfg)) == 128 * 3 + 16 * 32
    assert synth.C2.input_width() == 896 and synth.C1.input_width() == 320 and synth.C5.input_width() == 2816


def test_host_hash_matches_oracle_hash(lib):
    for i in (0, 1, 2, 77, 123456789, 2**31 - 1):
        for f in (0, 1, 15, 63):
            assert B.mix64(i, f) == orc.mix64(i, f)
        for n_cat in (1, 7, 100):
            for mode in (B.BUCKET_MOD, B.BUCKET_HASH):
                assert lib.aif_category(i, n_cat, mode) == orc.category(i, n_cat, mode)


def test_argument_errors_without_a_device(lib):
    h = C.c_void_p()
    assert lib.aif_create(None, C.byref(h)) == B.ERR_ARG
    bad = B.make_config(dtype=B.BF16, M=1000, d=100, L_max=10, hidden=(512, 256))     # d not a multiple of 32
    assert lib.aif_create(C.byref(bad), C.byref(h)) == B.ERR_SHAPE
    bad = B.make_config(dtype=B.BF16, M=0, d=128, L_max=10, hidden=(512, 256))
    assert lib.aif_create(C.byref(bad), C.byref(h)) == B.ERR_SHAPE
    bad = B.make_config(dtype=7, M=10, d=128, L_max=10, hidden=(512, 256))
    assert lib.aif_create(C.byref(bad), C.byref(h)) == B.ERR_ARG
    bad = B.make_config(dtype=B.BF16, M=10, d=128, L_max=10, hidden=(512, 256))
    bad.struct_size = 4
    assert lib.aif_create(C.byref(bad), C.byref(h)) == B.ERR_ARG
    assert lib.aif_destroy(None) == B.ERR_ARG
    assert lib.aif_score(None, None, None, 1, None, None) == B.ERR_ARG
    assert lib.aif_strerror(B.ERR_VERSION).decode().startswith("user state")
    assert lib.aif_kernel_launches() == 0


def test_binding_refuses_to_run_without_cuda():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a CUDA device is present")
    with pytest.raises(RuntimeError):
        B.Aif(B.make_config(dtype=B.BF16, M=10, d=128, L_max=10, hidden=(512, 256)))
    with pytest.raises(FileNotFoundError):
        B.load_library(os.path.join(ROOT, "no_such_dir", "libaif.so"))
