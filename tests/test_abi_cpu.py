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


def test_launch_geometry_for_shapes_without_a_device():
    """hola_plan_for_shape is host arithmetic: the split of the verify rows into passes and of the grid into pairs (and,
    when the passes share a launch, into groups of pairs that walk the same vocabulary tiles) must hold for any shape."""
    from paper_2506_18952_b200 import binding as b
    sms = 148
    expansion = (b.HOLA_W_INT8, b.HOLA_W_MIXED)
    for H, V in ((64, 8), (128, 700), (256, 4000), (4096, 32000), (4096, 128256), (8192, 128256), (1024, 524288)):
        for rows in (1, 5, 16, 192, 256, 257, 384, 385, 512, 513, 900, 2304, 5000, 40000):
            for wd in (b.HOLA_W_BF16, b.HOLA_W_INT8, b.HOLA_W8A8, b.HOLA_W8A16, b.HOLA_W_MIXED):
                if wd == b.HOLA_W_MIXED and H % 128:
                    continue
                p = b.hola_plan_for_shape(sms, H, V, rows, wd)
                what = (H, V, rows, wd, p)
                cap = 256 if wd in expansion or wd == b.HOLA_W8A16 else 512
                assert 1 <= p["rows_per_pass"] <= cap, what
                assert p["passes"] == -(-rows // p["rows_per_pass"]), what            # no empty pass, every row covered
                assert p["grid"] % 2 == 0 and 2 <= p["grid"] <= sms, what
                assert 2 <= p["stages"] <= 12, what
                assert 16 <= p["tile_v"] <= 256 and p["tile_v"] % 8 == 0, what
                tiles = -(-V // p["tile_v"])
                if p["passes"] > 1 and p["kernels_per_call"] == 2:                      # all passes in one launch
                    assert p["passes"] <= sms // 2, what
                    assert p["grid"] % (2 * p["passes"]) == 0, what
                    groups = p["grid"] // (2 * p["passes"])
                    assert 1 <= groups <= tiles, what                                   # every group has a tile
                else:
                    assert p["kernels_per_call"] == p["passes"] + 1, what
                    assert p["grid"] // 2 <= tiles, what
                if p["passes"] > sms // 2:
                    assert p["kernels_per_call"] == p["passes"] + 1, what               # more passes than pairs: a launch each
    # the shapes the bench runs
    assert b.hola_plan_for_shape(sms, 4096, 128256, 384)["passes"] == 1
    wide = b.hola_plan_for_shape(sms, 8192, 128256, 2304)
    assert wide["passes"] == 6 and wide["rows_per_pass"] == 384 and wide["kernels_per_call"] == 2 and wide["grid"] == 144
    for bad in ((1, 4096, 32000, 5, 0), (sms, 4097, 32000, 5, 0), (sms, 4096, 0, 5, 0), (sms, 4096, 32000, 0, 0),
                (sms, 4096, 32000, 5, 9)):
        with pytest.raises(b.HolaError):
            b.hola_plan_for_shape(*bad)
