"""The C-ABI library builds, loads and exports every symbol include/wk.h declares; host-only logic (sizes,
status strings, config validation) behaves as documented.  No compute calls: this runs without a GPU."""
import ctypes as C
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2605_22718_b200.build import build_all
    build_all()
    import paper_2605_22718_b200 as pkg
    return pkg.load_library()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "wk.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(wk_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    import paper_2605_22718_b200 as pkg
    names = declared_functions()
    assert len(names) >= 17
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in include/wk.h but not exported"
    assert set(names) == set(pkg.EXPORTED_SYMBOLS)


def test_input_generator_library_loads():
    from paper_2605_22718_b200.build import build_all, LIB_INPUTS
    build_all()
    g = C.CDLL(LIB_INPUTS)
    assert hasattr(g, "wkin_fill_normal_bf16") and hasattr(g, "wkin_fill_keys_bf16")


def test_sizes_and_status_strings(lib):
    import paper_2605_22718_b200 as pkg
    cfg = pkg.wk_config(30, 12, 128, 880, 3, 440, 250, 8, 2, 0, 0.0, 0)
    kv = 30 * 250 * 1320 * 1536 * 2
    total = lib.wk_pool_bytes(C.byref(cfg))
    assert 2 * kv <= total <= 2 * kv + 16384                      # K and V rows, plus poses / flags / status
    s1 = lib.wk_scratch_bytes(C.byref(cfg), 30, 2640, 1)
    s8 = lib.wk_scratch_bytes(C.byref(cfg), 30, 2640, 8)
    assert s8 - s1 >= 8 * 12 * 2640 * 128 * 4                     # fp32 partials for 8 splits
    bad = pkg.wk_config(30, 12, 64, 880, 3, 440, 250, 8, 2, 0, 0.0, 0)   # head_dim must be 128
    assert lib.wk_pool_bytes(C.byref(bad)) == 0
    bad2 = pkg.wk_config(30, 12, 128, 880, 3, 1761, 250, 8, 2, 0, 0.0, 0)  # n_keep > (F-1) T
    assert lib.wk_pool_bytes(C.byref(bad2)) == 0
    assert pkg.status_string(pkg.WK_OK) == "ok"
    for st in range(-9, 0):
        assert pkg.status_string(st) not in ("ok", "unknown status")
    assert pkg.status_string(-99) == "unknown status"


def test_create_fails_loudly_without_a_device_or_with_a_bad_config(lib):
    import torch
    import paper_2605_22718_b200 as pkg
    h = C.c_void_p()
    bad = pkg.wk_config(0, 12, 128, 880, 3, 440, 250, 8, 2, 0, 0.0, 0)
    assert lib.wk_create(C.byref(bad), C.byref(h)) == pkg.WK_ERR_ARG and not h.value
    if not torch.cuda.is_available():
        with pytest.raises(pkg.WkError) as e:
            pkg.WorldKV(n_layers=1, n_heads=2, tokens_per_frame=16, n_keep=8, pool_slots=2, max_k=1)
        assert e.value.status == pkg.WK_ERR_NO_DEVICE


def test_product_does_not_import_the_oracle():
    """The oracle is test infrastructure: nothing under the package may import it."""
    pkg_dir = os.path.join(ROOT, "paper_2605_22718_b200")
    for base, _, files in os.walk(pkg_dir):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(base, f)).read()
                assert "oracle" not in text, f"{f} mentions the oracle"
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith(".py"):
            assert "paper_2605_22718_b200" not in open(os.path.join(ROOT, "oracle", f)).read()
