"""Host-side checks of the C-ABI library that need no GPU: it builds for sm_100a, loads, and
exports every function include/moin.h declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "moin.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(moin_[a-z_0-9]+)\s*\(", text)))


@pytest.fixture(scope="module")
def built():
    from paper_2410_09687_b200 import build
    return build.build()


def test_header_functions_are_exported(built):
    L = ctypes.CDLL(built)
    names = _declared()
    assert "moin_route" in names and "moin_lora_linear" in names and "moin_decoder_forward" in names
    for n in names:
        assert hasattr(L, n), f"{n} declared in moin.h but not exported"


def test_binding_lists_every_declared_function(built):
    import paper_2410_09687_b200 as moin
    assert sorted(moin.EXPORTED_SYMBOLS) == _declared()
    L = moin.lib()
    assert L.moin_version() >= 100
    assert L.moin_status_string(0) == b"MOIN_OK"
    assert L.moin_status_string(-5) == b"MOIN_ERR_UNSUPPORTED_RANK"


def test_size_queries_need_no_gpu(built):
    import paper_2410_09687_b200 as moin
    L = moin.lib()
    assert L.moin_plan_bytes(256, 500) >= 4 * (256 * 6 + 501)
    assert L.moin_plan_bytes(16384, 5000) >= 4 * 64 * 5001
    assert L.moin_route_workspace_bytes(65536, 5000, 768) >= 65536 * 8
    assert L.moin_lora_linear_workspace_bytes(256, 2048, 5632, 64) >= 256 * 5632 * 4 + 256 * 64 * 4


def test_no_cpu_fallback_without_gpu(built):
    import torch
    import paper_2410_09687_b200 as moin
    if torch.cuda.is_available():
        pytest.skip("GPU present")
    x = torch.zeros(4, 64, dtype=torch.bfloat16)
    W = torch.zeros(8, 64, dtype=torch.bfloat16)
    with pytest.raises(moin.MoinError):
        moin.lora_linear(None, x, W, None, 1.0, y=torch.zeros(4, 8, dtype=torch.bfloat16),
                         workspace=torch.zeros(1024, dtype=torch.uint8))


def test_product_never_imports_oracle():
    pkg = os.path.join(ROOT, "paper_2410_09687_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                src = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"^\s*(import|from)\s+oracle\b", src, flags=re.M), f
                assert "moin_oracle" not in src and "libmoin_oracle" not in src, f
