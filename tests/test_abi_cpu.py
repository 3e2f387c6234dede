"""The C-ABI library loads without a GPU and exports every symbol include/sp24.h declares; host-side
argument validation answers before any device work."""
import ctypes
import os
import re

from paper_2104_08378_b200 import build

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "sp24.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sp24_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    lib = ctypes.CDLL(build.build_library())
    names = _declared()
    assert "sp24_prune" in names and "sp24_gemm" in names and len(names) >= 11
    for name in names:
        assert hasattr(lib, name), name


def test_binding_lists_the_same_symbols():
    from paper_2104_08378_b200 import binding
    assert sorted(binding.EXPORTS) == _declared()


def test_size_helpers_and_status_strings():
    from paper_2104_08378_b200 import binding as sp
    assert sp.values_bytes("bf16", 49152, 12288) == 603979776          # M * K/2 * 2
    assert sp.meta_bytes("bf16", 49152, 12288, sp.META_CANONICAL) == 75497472
    assert sp.meta_bytes("bf16", 49152, 12288, sp.META_TCGEN05) == 75497472   # already tile-aligned
    assert sp.meta_bytes("i8", 200, 640, sp.META_TCGEN05) == 2 * 3 * 4096     # padded to 256 x 768
    assert sp.values_bytes("f32", 4, 8) == 4 * 4 * 4                     # 1:2 pattern: K/2 fp32 values per row
    assert sp.meta_bytes("f32", 100, 200, sp.META_CANONICAL) == 100 * 50  # one nibble per pair
    assert sp.meta_bytes("f32", 100, 200, sp.META_TCGEN05) == 1 * 2 * 4096
    assert sp.values_bytes("i32", 4, 8) == 0
    assert sp.status_string(0) == "ok" and "shape" in sp.status_string(3)


def test_argument_errors_are_reported_before_touching_a_device():
    from paper_2104_08378_b200 import binding as sp
    lib = sp.lib
    one = ctypes.c_void_p(16)
    assert lib.sp24_prune(sp.F16, 4, 6, one, 6, one, 6, None) == 3            # K % 4
    assert lib.sp24_prune(sp.I32, 4, 8, one, 8, one, 8, None) == 2            # dtype
    assert lib.sp24_prune(sp.F16, 4, 8, None, 8, one, 8, None) == 1           # null
    assert lib.sp24_prune(sp.F16, 4, 8, one, 4, one, 8, None) == 4            # ld < K
    assert lib.sp24_prune(sp.F16, 0, 8, None, 8, None, 8, None) == 0          # empty: nothing to do
    assert lib.sp24_compress(sp.I8, 4, 12, one, 12, one, 6, one, 0, None, None) == 3
    desc = sp.make_desc("bf16", "bf16", 16, 24, 16, 8, 16, 24, 24)            # N % 16
    a, b = ctypes.c_float(1), ctypes.c_float(0)
    assert lib.sp24_gemm(ctypes.byref(desc), ctypes.byref(a), one, one, one, ctypes.byref(b), None, one, one,
                         256, None) == 3
    desc = sp.make_desc("i8", "i32", 32, 32, 32, 16, 32, 32, 32)
    ia, ib = ctypes.c_int32(2), ctypes.c_int32(0)
    assert lib.sp24_gemm(ctypes.byref(desc), ctypes.byref(ia), one, one, one, ctypes.byref(ib), None, one, one,
                         256, None) == 6                                       # int8 alpha != 1
    desc = sp.make_desc("bf16", "f16", 16, 16, 16, 8, 16, 16, 16)
    assert lib.sp24_gemm(ctypes.byref(desc), ctypes.byref(a), one, one, one, ctypes.byref(b), None, one, one,
                         256, None) == 2                                       # cd type mismatch
    desc = sp.make_desc("bf16", "bf16", 16, 16, 16, 8, 16, 16, 16)
    assert lib.sp24_gemm(ctypes.byref(desc), ctypes.byref(a), one, one, one, ctypes.byref(b), None, one, one,
                         8, None) == 7                                         # workspace too small
    assert lib.sp24_gemm(ctypes.byref(desc), ctypes.byref(a), ctypes.c_void_p(24), one, one, ctypes.byref(b),
                         None, one, one, 256, None) == 5                       # misaligned A


def test_tile_plan_and_support_calls_answer_without_a_device():
    """sp24_gemm_plan is host logic: the large and the small shapes do not depend on the SM count, and a
    forced tile shape is reported back; the FP16-accumulate entry point rejects other types on the host."""
    from paper_2104_08378_b200 import binding as sp
    lib = sp.lib
    assert sp.gemm_plan(sp.make_desc("bf16", "bf16", 49152, 8192, 12288, 6144, 12288, 8192, 8192)) == "2x224x2"
    assert sp.gemm_plan(sp.make_desc("f16", "f16", 256, 256, 512, 256, 512, 256, 256)) == "1x128x1"
    c = ctypes.c_int()
    desc = sp.make_desc("bf16", "bf16", 256, 256, 512, 256, 512, 256, 256)
    assert lib.sp24_gemm_plan(ctypes.byref(desc), None, ctypes.byref(c), ctypes.byref(c)) == 1        # null
    bad = sp.make_desc("bf16", "bf16", 256, 256, 0, 256, 512, 256, 256)
    assert lib.sp24_gemm_plan(ctypes.byref(bad), ctypes.byref(c), ctypes.byref(c), ctypes.byref(c)) == 3   # K = 0
    try:
        sp.set_tile_override("2x192x2")
        assert sp.gemm_plan(desc) == "2x192x2"
    finally:
        sp.set_tile_override(None)
    assert sp.gemm_plan(desc) == "1x128x1"
    assert lib.sp24_set_tile_override(-1, 0, 0, 0) == 3
    one = ctypes.c_void_p(16)
    a, b = ctypes.c_float(1), ctypes.c_float(0)
    desc = sp.make_desc("bf16", "bf16", 16, 16, 16, 8, 16, 16, 16)
    assert lib.sp24_gemm_f16acc(ctypes.byref(desc), ctypes.byref(a), one, one, one, ctypes.byref(b), None, one, one,
                                256, None) == 2                                # FP16 operands only
    assert lib.sp24_gemm_status(None, None) == 1
