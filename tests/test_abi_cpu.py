"""Host-side checks that need no GPU: the C-ABI library builds, loads and exports what the header declares."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2506_18952_b200 import binding
    return binding.load_library()


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "hola_verify.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(hola_[a-z0-9_]+)\s*\(", text)))


def test_library_exports_every_declared_symbol(lib):
    from paper_2506_18952_b200 import binding
    names = _declared_functions()
    assert len(names) >= 12
    for n in names:
        assert hasattr(lib, n), f"{n} is declared in include/hola_verify.h but not exported"
    assert sorted(binding.EXPORTS) == names


def test_strerror_version_and_workspace(lib):
    assert lib.hola_version().decode() == "0.1"
    texts = {lib.hola_strerror(i).decode() for i in range(6)}
    assert len(texts) == 6 and "ok" in texts
    assert lib.hola_strerror(99).decode() == "unknown status"
    # workspace: fp32 logits scratch dominates; 64 x 6 rows of 128256 floats = 197 MB
    ws = lib.hola_workspace_bytes(64, 5, 4096, 128256)
    assert 64 * 6 * 128256 * 4 < ws < 2 * 64 * 6 * 128256 * 4 + (1 << 29)
    assert lib.hola_workspace_bytes(0, 5, 4096, 1000) == 0


def test_struct_layout_matches_header():
    from paper_2506_18952_b200 import binding
    a = binding.hola_verify_args
    # 4 int32, 4 pointers, int32 (+pad), pointer, float (+pad), 6 pointers, 2 int32, pointer, 2 int32, 2 pointers
    assert ctypes.sizeof(a) == 16 + 4 * 8 + 8 + 8 + 8 + 6 * 8 + 8 + 8 + 8 + 8 + 8
    assert a.wmix.offset == 152 and ctypes.sizeof(binding.hola_wmix) == 6 * 8 + 4 * 4
    assert a.w_dtype.offset == 136 and a.w_scale.offset == 144
    assert a.gate_source.offset == 120 and a.fallback.offset == 124 and a.draft_entropy.offset == 128
    assert a.uniforms.offset == 56 and a.tau.offset == 64 and a.accept_len.offset == 72
    assert ctypes.sizeof(binding.hola_plan_info) == 24


def test_no_device_is_an_error_not_a_fallback(lib):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    from paper_2506_18952_b200 import binding
    ctx = ctypes.c_void_p()
    assert lib.hola_create(ctypes.byref(ctx), 0, 1, 4, 64, 1000) == 5       # HOLA_ERR_NO_DEVICE
    assert not ctx.value
    with pytest.raises(binding.HolaError):
        binding.HolaVerify(1, 4, 64, 1000)
    a = binding.hola_verify_args()
    assert lib.hola_verify(None, ctypes.byref(a), None) == 1
    assert lib.hola_destroy(None) == 0


def test_product_package_does_not_touch_the_oracle():
    pkg = os.path.join(ROOT, "paper_2506_18952_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".h", ".cuh")):
                src = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"^\s*(from|import)\s+oracle\b", src, flags=re.M), f"{f} imports the oracle"
                assert "oracle/" not in src and "hola_verify_ref" not in src, f"{f} reaches into the oracle"
