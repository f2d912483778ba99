"""The C-ABI library loads and exports every symbol include/xrl.h declares (no GPU needed)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2304_14698_b200 import build, binding
    build.build()
    return binding.load_library()


def _declared():
    text = open(os.path.join(ROOT, "include", "xrl.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(xrl_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    from paper_2304_14698_b200 import binding
    names = _declared()
    assert len(names) >= 16
    for n in names:
        assert hasattr(lib, n), n
    assert sorted(binding.EXPORTED_SYMBOLS) == names


def test_version_and_argument_errors_without_a_gpu(lib):
    import paper_2304_14698_b200 as xrl
    assert "sm_100a" in xrl.xrl_version()
    # null config / null out are rejected before any CUDA call
    assert lib.xrl_create(None, 0, None) == 1
    m = dict(T=32, S=8, H=64, K=1, L=2, Hm=64, Dg=1, dtype="fp32", A_max=8)
    bad = xrl.model_config(dict(m, H=48), 8, 1, 1024, 4096)       # 48 is not a multiple of 32
    out = ctypes.c_void_p()
    assert lib.xrl_create(ctypes.byref(bad), 0, ctypes.byref(out)) == 8
    bad = xrl.model_config(dict(m, K=3), 8, 1, 1024, 4096)        # heads must divide hidden
    assert lib.xrl_create(ctypes.byref(bad), 0, ctypes.byref(out)) == 1


def test_no_cpu_fallback_without_a_device(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    import paper_2304_14698_b200 as xrl
    m = dict(T=32, S=8, H=64, K=1, L=2, Hm=64, Dg=1, dtype="fp32", A_max=8)
    with pytest.raises(xrl.XrlError) as e:
        xrl.xrl_create(xrl.model_config(m, 8, 1, 1024, 4096), 0)
    assert e.value.status == 5          # XRL_ERR_CUDA: the product path fails loudly


def test_product_package_does_not_import_the_oracle():
    pkg = os.path.join(ROOT, "paper_2304_14698_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in src.lower(), os.path.join(dirpath, f)
