"""CPU-side checks of the boundary: the C-ABI library builds, loads and exports every
symbol that include/fda.h declares; the binding refuses to work without a device instead of
falling back to anything."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2405_20988_b200 import build
    build.build()
    import paper_2405_20988_b200 as F
    return F.load_library()


def declared_functions():
    text = open(os.path.join(ROOT, "include", "fda.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(fda_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_functions()
    assert len(names) >= 9
    for n in names:
        assert hasattr(lib, n), n
    from paper_2405_20988_b200 import binding
    assert sorted(binding.EXPORTS) == names


def test_estimate_struct_layout_matches_header():
    from paper_2405_20988_b200 import Estimate
    assert ctypes.sizeof(Estimate) == 4 * 4 + 2 * 4 + 16 * 4
    assert Estimate.trigger.offset == 16 and Estimate.row_sq_norm.offset == 24


def test_null_and_range_checks_need_no_device(lib):
    assert lib.fda_create(None, 0, 5, 250, None, 100, 2) == 1            # out == NULL
    h = ctypes.c_void_p()
    assert lib.fda_create(ctypes.byref(h), 0, 17, 250, None, 100, 2) == 1
    assert lib.fda_create(ctypes.byref(h), 0, 5, 250, None, 100, 2) == 1  # coefficients missing
    assert lib.fda_state_len(None) == 0
    assert lib.fda_destroy(None) == 0
    assert lib.fda_local_state(None, None, 0, 0, 0, None, None, 0, None, None) == 1


def test_no_cpu_fallback_without_a_device():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    import paper_2405_20988_b200 as F
    with pytest.raises(F.FdaError):
        F.FdaContext(0, 0, None, 100, 2)


def test_product_path_does_not_touch_the_oracle():
    pkg = os.path.join(ROOT, "paper_2405_20988_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src.replace("test infrastructure", ""), f
