"""ctypes binding of the sp24 C ABI (include/sp24.h): argument marshalling only.

Every function takes torch CUDA tensors (PyTorch is used for device memory and streams only),
passes their device pointers and the current stream to ``libsp24.so`` and raises
``Sp24Error`` on a non-zero status.  There is no CPU fallback: if the library is missing the
import fails, and every call needs a CUDA device.

16-bit matrices may be torch.float16 / torch.bfloat16 or raw torch.int16 / uint16 bit patterns
(then pass ``dtype=`` explicitly); int8 matrices are torch.int8.
"""
from __future__ import annotations

import ctypes
import os

import torch

from .build import LIB_PATH

OK = 0
F16, BF16, I8, F32, I32, E4M3, E5M2 = 0, 1, 2, 3, 4, 5, 6
META_CANONICAL, META_TCGEN05 = 0, 1
ROW_MAJOR, COL_MAJOR = 0, 1
DTYPE_CODE = {"f16": F16, "bf16": BF16, "i8": I8, "f32": F32, "i32": I32, "e4m3": E4M3, "e5m2": E5M2}
TORCH_DTYPE = {"f16": torch.float16, "bf16": torch.bfloat16, "i8": torch.int8, "f32": torch.float32,
               "i32": torch.int32, "e4m3": torch.float8_e4m3fn, "e5m2": torch.float8_e5m2}
_FROM_TORCH = {torch.float16: "f16", torch.bfloat16: "bf16", torch.int8: "i8", torch.float32: "f32",
               torch.int32: "i32", torch.float8_e4m3fn: "e4m3", torch.float8_e5m2: "e5m2"}

EXPORTS = [
    "sp24_status_string", "sp24_values_bytes", "sp24_meta_bytes", "sp24_prune", "sp24_compress",
    "sp24_decompress", "sp24_prune_compress", "sp24_gemm_workspace_bytes", "sp24_gemm", "sp24_gemm_status",
    "sp24_im2col_nhwc_3x3", "sp24_pipeline_host", "sp24_gemm_static_ws", "sp24_gemm_i8_dequant",
    "sp24_conv3x3_nhwc", "sp24_kept_magnitude", "sp24_apply_mask", "sp24_prune_2d",
    "sp24_gemm_static_ws_status", "sp24_set_tile_override", "sp24_test_set_fault_hooks", "sp24_gemm_f16acc",
    "sp24_gemm_plan",
]


class Sp24Error(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: sp24 status {status} ({status_string(status)})")


class GemmDesc(ctypes.Structure):
    _fields_ = [("ab_type", ctypes.c_int), ("cd_type", ctypes.c_int),
                ("M", ctypes.c_int64), ("N", ctypes.c_int64), ("K", ctypes.c_int64),
                ("lda", ctypes.c_int64), ("ldb", ctypes.c_int64), ("ldc", ctypes.c_int64),
                ("ldd", ctypes.c_int64),
                ("order_b", ctypes.c_int), ("order_c", ctypes.c_int), ("order_d", ctypes.c_int),
                ("a_is_dense", ctypes.c_int)]


def _load() -> ctypes.CDLL:
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: run `python -m paper_2104_08378_b200.build` "
                          "(there is no CPU fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    i64, vp, ci, sz = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
    lib.sp24_status_string.argtypes = [ci]
    lib.sp24_status_string.restype = ctypes.c_char_p
    lib.sp24_values_bytes.argtypes = [ci, i64, i64]
    lib.sp24_values_bytes.restype = sz
    lib.sp24_meta_bytes.argtypes = [ci, i64, i64, ci]
    lib.sp24_meta_bytes.restype = sz
    lib.sp24_prune.argtypes = [ci, i64, i64, vp, i64, vp, i64, vp]
    lib.sp24_compress.argtypes = [ci, i64, i64, vp, i64, vp, i64, vp, ci, vp, vp]
    lib.sp24_decompress.argtypes = [ci, i64, i64, vp, i64, vp, ci, vp, i64, vp]
    lib.sp24_prune_compress.argtypes = [ci, i64, i64, vp, i64, vp, i64, vp, i64, vp, ci, vp, vp]
    lib.sp24_gemm_workspace_bytes.argtypes = [ctypes.POINTER(GemmDesc)]
    lib.sp24_gemm_workspace_bytes.restype = sz
    lib.sp24_gemm.argtypes = [ctypes.POINTER(GemmDesc), vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.sp24_gemm_plan.argtypes = [ctypes.POINTER(GemmDesc), ctypes.POINTER(ci), ctypes.POINTER(ci), ctypes.POINTER(ci)]
    lib.sp24_gemm_plan.restype = ci
    lib.sp24_gemm_f16acc.argtypes = lib.sp24_gemm.argtypes
    lib.sp24_gemm_f16acc.restype = ci
    lib.sp24_gemm_static_ws.argtypes = [ctypes.POINTER(GemmDesc), vp, vp, vp, vp, vp, vp, vp, vp]
    lib.sp24_gemm_static_ws.restype = ci
    lib.sp24_gemm_i8_dequant.argtypes = [ctypes.POINTER(GemmDesc), vp, vp, vp, vp, vp, ci, ctypes.c_float, vp, vp,
                                         sz, vp]
    lib.sp24_gemm_i8_dequant.restype = ci
    lib.sp24_conv3x3_nhwc.argtypes = [ctypes.POINTER(GemmDesc), i64, i64, i64, i64, vp, vp, vp, vp, vp, vp, vp, vp, sz, vp]
    lib.sp24_conv3x3_nhwc.restype = ci
    lib.sp24_kept_magnitude.argtypes = [ci, i64, i64, vp, i64, vp, vp, vp]
    lib.sp24_apply_mask.argtypes = [ci, i64, i64, vp, i64, vp, ci, vp, i64, vp]
    lib.sp24_prune_2d.argtypes = [ci, i64, i64, vp, i64, vp, i64, vp]
    for name in ("sp24_kept_magnitude", "sp24_apply_mask", "sp24_prune_2d"):
        getattr(lib, name).restype = ci
    lib.sp24_gemm_status.argtypes = [vp, vp]
    lib.sp24_gemm_static_ws_status.argtypes = [vp]
    lib.sp24_gemm_static_ws_status.restype = ci
    lib.sp24_set_tile_override.argtypes = [ci, ci, ci, ci]
    lib.sp24_set_tile_override.restype = ci
    lib.sp24_test_set_fault_hooks.argtypes = [ctypes.c_longlong, ci]
    lib.sp24_test_set_fault_hooks.restype = ci
    lib.sp24_im2col_nhwc_3x3.argtypes = [ci, i64, i64, i64, i64, vp, vp, i64, vp]
    lib.sp24_pipeline_host.argtypes = [ctypes.POINTER(GemmDesc)] + [vp] * 13 + [sz, vp]
    for name in ("sp24_prune", "sp24_compress", "sp24_decompress", "sp24_gemm", "sp24_gemm_status",
                 "sp24_im2col_nhwc_3x3", "sp24_pipeline_host"):
        getattr(lib, name).restype = ci
    return lib


lib = _load()


def status_string(status: int) -> str:
    return lib.sp24_status_string(int(status)).decode()


def _check(status: int, where: str):
    if status != OK:
        raise Sp24Error(status, where)


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def _dtype_of(t: torch.Tensor, dtype: str | None) -> str:
    if dtype is not None:
        return dtype
    return _FROM_TORCH[t.dtype]


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def values_bytes(dtype: str, M: int, K: int) -> int:
    return lib.sp24_values_bytes(DTYPE_CODE[dtype], M, K)


def meta_bytes(dtype: str, M: int, K: int, layout: int = META_TCGEN05) -> int:
    return lib.sp24_meta_bytes(DTYPE_CODE[dtype], M, K, layout)


def prune(x: torch.Tensor, out: torch.Tensor | None = None, dtype: str | None = None) -> torch.Tensor:
    """sp24_prune on a 2-D row-major tensor (row stride = leading dimension)."""
    dt = _dtype_of(x, dtype)
    M, K = x.shape
    if out is None:
        out = torch.empty((M, K), dtype=x.dtype, device=x.device)
    assert x.stride(1) == 1 or K <= 1
    _check(lib.sp24_prune(DTYPE_CODE[dt], M, K, _ptr(x), x.stride(0) if M > 1 else K, _ptr(out),
                          out.stride(0) if M > 1 else K, _stream()), "sp24_prune")
    return out


def compress(x: torch.Tensor, layout: int = META_TCGEN05, dtype: str | None = None,
             count_dropped: bool = False):
    """sp24_compress: returns (vals [M, K/2], meta uint8 [meta_bytes], dropped tensor or None)."""
    dt = _dtype_of(x, dtype)
    M, K = x.shape
    vals = torch.empty((M, K // 2), dtype=x.dtype, device=x.device)
    meta = torch.empty(meta_bytes(dt, M, K, layout), dtype=torch.uint8, device=x.device)
    dropped = torch.zeros(1, dtype=torch.int64, device=x.device) if count_dropped else None
    _check(lib.sp24_compress(DTYPE_CODE[dt], M, K, _ptr(x), x.stride(0) if M > 1 else K, _ptr(vals),
                             K // 2, _ptr(meta), layout, _ptr(dropped), _stream()), "sp24_compress")
    return vals, meta, dropped


def compress_into(x, vals, meta, layout: int = META_TCGEN05, dtype: str | None = None, dropped=None):
    dt = _dtype_of(x, dtype)
    M, K = x.shape
    _check(lib.sp24_compress(DTYPE_CODE[dt], M, K, _ptr(x), x.stride(0) if M > 1 else K, _ptr(vals),
                             vals.stride(0) if M > 1 else K // 2, _ptr(meta), layout, _ptr(dropped),
                             _stream()), "sp24_compress")


def prune_compress(x: torch.Tensor, layout: int = META_TCGEN05, dtype: str | None = None, count_dropped: bool = False,
                   pruned: torch.Tensor | None = None, vals: torch.Tensor | None = None,
                   meta: torch.Tensor | None = None):
    """sp24_prune_compress: one pass; returns (pruned [M, K], vals [M, K/2], meta, dropped tensor or None)."""
    dt = _dtype_of(x, dtype)
    M, K = x.shape
    pruned = torch.empty_like(x) if pruned is None else pruned
    vals = torch.empty((M, K // 2), dtype=x.dtype, device=x.device) if vals is None else vals
    meta = torch.empty(meta_bytes(dt, M, K, layout), dtype=torch.uint8, device=x.device) if meta is None else meta
    dropped = torch.zeros(1, dtype=torch.int64, device=x.device) if count_dropped else None
    _check(lib.sp24_prune_compress(DTYPE_CODE[dt], M, K, _ptr(x), x.stride(0) if M > 1 else K, _ptr(pruned),
                                   pruned.stride(0) if M > 1 else K, _ptr(vals), vals.stride(0) if M > 1 else K // 2,
                                   _ptr(meta), layout, _ptr(dropped), _stream()), "sp24_prune_compress")
    return pruned, vals, meta, dropped


def decompress(vals: torch.Tensor, meta: torch.Tensor, layout: int = META_TCGEN05,
               dtype: str | None = None, out: torch.Tensor | None = None) -> torch.Tensor:
    dt = _dtype_of(vals, dtype)
    M, K2 = vals.shape
    y = torch.empty((M, 2 * K2), dtype=vals.dtype, device=vals.device) if out is None else out
    _check(lib.sp24_decompress(DTYPE_CODE[dt], M, 2 * K2, _ptr(vals), vals.stride(0) if M > 1 else K2,
                               _ptr(meta), layout, _ptr(y), y.stride(0) if M > 1 else 2 * K2, _stream()),
           "sp24_decompress")
    return y


def make_desc(ab: str, cd: str, M: int, N: int, K: int, lda: int, ldb: int, ldc: int, ldd: int,
              a_is_dense: bool = False, b_row_major: bool = False, cd_col_major: bool = False) -> GemmDesc:
    cd_order = COL_MAJOR if cd_col_major else ROW_MAJOR
    return GemmDesc(DTYPE_CODE[ab], DTYPE_CODE[cd], M, N, K, lda, ldb, ldc, ldd,
                    ROW_MAJOR if b_row_major else COL_MAJOR, cd_order, cd_order, 1 if a_is_dense else 0)


def _scalar(ab: str, v):
    return ctypes.c_float(float(v)) if ab != "i8" else ctypes.c_int32(int(v))


_workspaces: dict = {}


def workspace(device) -> torch.Tensor:
    key = (torch.device(device).index, torch.cuda.current_stream().cuda_stream)
    if key not in _workspaces:
        _workspaces[key] = torch.zeros(256, dtype=torch.uint8, device=device)
    return _workspaces[key]


def gemm(A: torch.Tensor, meta: torch.Tensor | None, Bt: torch.Tensor, *, alpha=1.0, beta=0.0,
         C: torch.Tensor | None = None, out: torch.Tensor | None = None, cd: str | None = None,
         ab: str | None = None, a_is_dense: bool = False, ws: torch.Tensor | None = None,
         b_row_major: bool = False, cd_col_major: bool = False, acc_f16: bool = False) -> torch.Tensor:
    """sp24_gemm (sp24_gemm_f16acc with acc_f16=True).  A: vals [M, K/2] (or dense [M, K]); Bt: [N, K]
    (K contiguous), or with b_row_major=True the K x N matrix itself, [K, N] (N contiguous); C/D: [M, N],
    or with cd_col_major=True their transposes [N, M] (M contiguous)."""
    ab = _dtype_of(A, ab)
    M = A.shape[0]
    K = A.shape[1] if a_is_dense else 2 * A.shape[1]
    N = Bt.shape[1] if b_row_major else Bt.shape[0]
    assert (Bt.shape[0] if b_row_major else Bt.shape[1]) == K
    cd = cd or ("i32" if ab == "i8" else ("bf16" if ab in ("e4m3", "e5m2") else ab))
    if out is None:
        out = torch.empty((N, M) if cd_col_major else (M, N), dtype=TORCH_DTYPE[cd], device=A.device)
    ws = ws if ws is not None else workspace(A.device)
    desc = make_desc(ab, cd, M, N, K, A.stride(0), Bt.stride(0),
                     C.stride(0) if C is not None else (M if cd_col_major else N), out.stride(0), a_is_dense,
                     b_row_major, cd_col_major)
    a, b = _scalar(ab, alpha), _scalar(ab, beta)
    fn = lib.sp24_gemm_f16acc if acc_f16 else lib.sp24_gemm
    _check(fn(ctypes.byref(desc), ctypes.byref(a), _ptr(A), _ptr(meta), _ptr(Bt),
              ctypes.byref(b), _ptr(C), _ptr(out), _ptr(ws), ws.numel(), _stream()),
           "sp24_gemm_f16acc" if acc_f16 else "sp24_gemm")
    return out


def gemm_plan(desc: GemmDesc) -> str:
    """sp24_gemm_plan: the tile shape the library picks for this problem, as "<ctas>x<block_n>x<mblk>"."""
    c, n, m = ctypes.c_int(), ctypes.c_int(), ctypes.c_int()
    _check(lib.sp24_gemm_plan(ctypes.byref(desc), ctypes.byref(c), ctypes.byref(n), ctypes.byref(m)), "sp24_gemm_plan")
    return f"{c.value}x{n.value}x{m.value}"


def gemm_status(ws: torch.Tensor | None = None, device=None) -> int:
    """sp24_gemm_status: 0, or SP24_ERR_TIMEOUT (9) if a wait expired in any launch on this workspace
    since the last read (the record is then cleared)."""
    ws = ws if ws is not None else workspace(device or "cuda")
    return lib.sp24_gemm_status(_ptr(ws), _stream())


def gemm_static_ws_status() -> int:
    """sp24_gemm_static_ws_status: the same for the library's own workspace array on the current device."""
    return lib.sp24_gemm_static_ws_status(_stream())


def set_tile_override(tile: str | None = None, band: int = 0):
    """sp24_set_tile_override: tile = "<ctas>x<block_n>x<mblk>" forces that tile shape, None restores
    the automatic choice (benchmarks and tests)."""
    c, n, m = (0, 0, 0) if not tile else (list(map(int, tile.split("x"))) + [1])[:3]
    _check(lib.sp24_set_tile_override(c, n, m, band), "sp24_set_tile_override")


def set_fault_hooks(wait_cycles: int = 0, skip_stage: bool = False):
    """sp24_test_set_fault_hooks (failure-path tests only)."""
    _check(lib.sp24_test_set_fault_hooks(int(wait_cycles), 1 if skip_stage else 0), "sp24_test_set_fault_hooks")


def im2col_nhwc_3x3(x: torch.Tensor, dtype: str | None = None, out: torch.Tensor | None = None) -> torch.Tensor:
    dt = _dtype_of(x, dtype)
    Nb, H, W, C = x.shape
    if out is None:
        out = torch.empty((Nb * H * W, 9 * C), dtype=x.dtype, device=x.device)
    _check(lib.sp24_im2col_nhwc_3x3(DTYPE_CODE[dt], Nb, H, W, C, _ptr(x), _ptr(out), out.stride(0), _stream()),
           "sp24_im2col_nhwc_3x3")
    return out


def gemm_static_ws(A: torch.Tensor, meta: torch.Tensor | None, Bt: torch.Tensor, *, alpha=1.0, beta=0.0,
                   C: torch.Tensor | None = None, out: torch.Tensor, cd: str | None = None,
                   ab: str | None = None, a_is_dense: bool = False) -> torch.Tensor:
    """sp24_gemm_static_ws: the GEMM for callers that cannot allocate device memory (the workspace is
    a fixed array inside the library).  `out` must be provided: nothing is allocated here either."""
    ab = _dtype_of(A, ab)
    M = A.shape[0]
    K = A.shape[1] if a_is_dense else 2 * A.shape[1]
    N = Bt.shape[0]
    cd = cd or ("i32" if ab == "i8" else ("bf16" if ab in ("e4m3", "e5m2") else ab))
    desc = make_desc(ab, cd, M, N, K, A.stride(0), Bt.stride(0), C.stride(0) if C is not None else N,
                     out.stride(0), a_is_dense)
    a, b = _scalar(ab, alpha), _scalar(ab, beta)
    _check(lib.sp24_gemm_static_ws(ctypes.byref(desc), ctypes.byref(a), _ptr(A), _ptr(meta), _ptr(Bt),
                                   ctypes.byref(b), _ptr(C), _ptr(out), _stream()), "sp24_gemm_static_ws")
    return out


def gemm_i8_dequant(A: torch.Tensor, meta: torch.Tensor | None, Bt: torch.Tensor, row_scale: torch.Tensor, *,
                    bias: torch.Tensor | None = None, relu: bool = False, out_scale: float = 1.0, cd: str = "bf16",
                    out: torch.Tensor | None = None, a_is_dense: bool = False, ws: torch.Tensor | None = None,
                    b_row_major: bool = False, cd_col_major: bool = False) -> torch.Tensor:
    """sp24_gemm_i8_dequant: int8 sparse GEMM, D = act(row_scale[i] * acc + bias[i]) as cd (bf16/f16/f32/i8)."""
    M = A.shape[0]
    K = A.shape[1] if a_is_dense else 2 * A.shape[1]
    N = Bt.shape[1] if b_row_major else Bt.shape[0]
    if out is None:
        out = torch.empty((N, M) if cd_col_major else (M, N), dtype=TORCH_DTYPE[cd], device=A.device)
    ws = ws if ws is not None else workspace(A.device)
    desc = make_desc("i8", cd, M, N, K, A.stride(0), Bt.stride(0), M if cd_col_major else N, out.stride(0),
                     a_is_dense, b_row_major, cd_col_major)
    _check(lib.sp24_gemm_i8_dequant(ctypes.byref(desc), _ptr(A), _ptr(meta), _ptr(Bt), _ptr(row_scale), _ptr(bias),
                                    1 if relu else 0, ctypes.c_float(out_scale), _ptr(out), _ptr(ws), ws.numel(),
                                    _stream()), "sp24_gemm_i8_dequant")
    return out


def conv3x3_nhwc(A: torch.Tensor, meta: torch.Tensor | None, x: torch.Tensor, *, alpha=1.0, beta=0.0,
                 C: torch.Tensor | None = None, out: torch.Tensor | None = None, cd: str | None = None,
                 ab: str | None = None, a_is_dense: bool = False, ws: torch.Tensor | None = None,
                 nhwc_out: bool = False) -> torch.Tensor:
    """sp24_conv3x3_nhwc: x [Nb, H, W, Cin] -> D [Kout, Nb*H*W] (or NHWC [Nb*H*W, Kout] with nhwc_out)."""
    ab = _dtype_of(A, ab)
    Nb, H, W, Cin = x.shape
    M = A.shape[0]
    K, N = 9 * Cin, Nb * H * W
    cd = cd or ("i32" if ab == "i8" else ("bf16" if ab in ("e4m3", "e5m2") else ab))
    if out is None:
        out = torch.empty((N, M) if nhwc_out else (M, N), dtype=TORCH_DTYPE[cd], device=A.device)
    ws = ws if ws is not None else workspace(A.device)
    desc = make_desc(ab, cd, M, N, K, A.stride(0), K, C.stride(0) if C is not None else (M if nhwc_out else N),
                     out.stride(0), a_is_dense, False, nhwc_out)
    a, b = _scalar(ab, alpha), _scalar(ab, beta)
    _check(lib.sp24_conv3x3_nhwc(ctypes.byref(desc), Nb, H, W, Cin, ctypes.byref(a), _ptr(A), _ptr(meta), _ptr(x),
                                 ctypes.byref(b), _ptr(C), _ptr(out), _ptr(ws), ws.numel(), _stream()),
           "sp24_conv3x3_nhwc")
    return out


def kept_magnitude(x: torch.Tensor, perm: torch.Tensor | None = None, dtype: str | None = None) -> torch.Tensor:
    """sp24_kept_magnitude: total magnitude 2:4 pruning keeps under a column permutation (device double[1])."""
    dt = _dtype_of(x, dtype)
    M, K = x.shape
    res = torch.zeros(1, dtype=torch.float64, device=x.device)
    _check(lib.sp24_kept_magnitude(DTYPE_CODE[dt], M, K, _ptr(x), x.stride(0) if M > 1 else K, _ptr(perm), _ptr(res),
                                   _stream()), "sp24_kept_magnitude")
    return res


def apply_mask(w: torch.Tensor, meta: torch.Tensor, layout: int = META_TCGEN05, out: torch.Tensor | None = None,
               dtype: str | None = None) -> torch.Tensor:
    """sp24_apply_mask: zero every position of w the metadata does not name as kept."""
    dt = _dtype_of(w, dtype)
    M, K = w.shape
    if out is None:
        out = torch.empty_like(w)
    _check(lib.sp24_apply_mask(DTYPE_CODE[dt], M, K, _ptr(w), w.stride(0) if M > 1 else K, _ptr(meta), layout, _ptr(out),
                               out.stride(0) if M > 1 else K, _stream()), "sp24_apply_mask")
    return out


def prune_2d(x: torch.Tensor, out: torch.Tensor | None = None, dtype: str | None = None) -> torch.Tensor:
    """sp24_prune_2d: 2:4 along rows and columns of every 4 x 4 block (exhaustive search)."""
    dt = _dtype_of(x, dtype)
    M, K = x.shape
    if out is None:
        out = torch.empty_like(x)
    _check(lib.sp24_prune_2d(DTYPE_CODE[dt], M, K, _ptr(x), x.stride(0) if M > 1 else K, _ptr(out),
                             out.stride(0) if M > 1 else K, _stream()), "sp24_prune_2d")
    return out
