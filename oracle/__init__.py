"""CPU oracle for the 2:4 structured-sparse path (arXiv 2104.08378).

TEST INFRASTRUCTURE ONLY.  A thin numpy/ctypes front end over ``sp24_oracle.c`` (plain scalar
C, fp64 / int64 arithmetic).  It imports nothing from the CUDA package and the CUDA package
imports nothing from here.  Callers: the tests, the smoke check and the bench's CPU legs.

Array conventions: fp16 and bf16 matrices travel as ``numpy.uint16`` BIT PATTERNS, int8 as
``numpy.int8``, the 8-bit floats as ``numpy.uint8`` bit patterns; ``dtype`` is one of the strings
"f16", "bf16", "i8", "e4m3", "e5m2".  All matrices are 2-D,
C-contiguous (row-major).  B is passed as an ``N x K`` array (K contiguous), i.e. the
transpose of the K x N matrix of Section 3.2.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "sp24_oracle.c")
_LIB = os.path.join(_HERE, "libsp24_oracle.so")

DTYPE_CODE = {"f16": 0, "bf16": 1, "i8": 2, "e4m3": 5, "e5m2": 6}
C_DTYPE_CODE = {"f16": 0, "bf16": 1, "f32": 3, "i32": 4}


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (-O2, OpenMP) next to its source; returns the .so path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = f"{_LIB}.{os.getpid()}.tmp"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c11", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        i64, vp, i32, dbl = ctypes.c_int64, ctypes.c_void_p, ctypes.c_int, ctypes.c_double
        lib.oracle_num_threads.restype = i32
        lib.oracle_prune.argtypes = [i32, i64, i64, vp, i64, vp, i64]
        lib.oracle_prune.restype = None
        lib.oracle_compress.argtypes = [i32, i64, i64, vp, i64, vp, i64, vp]
        lib.oracle_compress.restype = i64
        lib.oracle_decompress.argtypes = [i32, i64, i64, vp, i64, vp, vp, i64]
        lib.oracle_decompress.restype = None
        lib.oracle_meta_operand_bytes.argtypes = [i64, i64]
        lib.oracle_meta_operand_bytes.restype = i64
        lib.oracle_meta_permute.argtypes = [i32, i64, i64, vp, vp, i32]
        lib.oracle_meta_permute.restype = None
        gemm_args = [i32, i64, i64, i64, vp, i64]
        lib.oracle_gemm_sparse.argtypes = gemm_args + [vp, vp, i64, i32, dbl, dbl, i32, vp, i64,
                                                       i64, i64, i64, i64, vp, vp]
        lib.oracle_gemm_sparse.restype = None
        lib.oracle_gemm_dense.argtypes = gemm_args + [vp, i64, i32, dbl, dbl, i32, vp, i64,
                                                      i64, i64, i64, i64, vp, vp]
        lib.oracle_gemm_dense.restype = None
        lib.oracle_gemm_abs.argtypes = [i32, i64, vp, i64, vp, vp, i64, i32, i64, i64, i64, i64, vp]
        lib.oracle_gemm_abs.restype = None
        lib.oracle_prune_1of2.argtypes = [i64, i64, vp, i64, vp, i64]
        lib.oracle_prune_1of2.restype = None
        lib.oracle_compress_1of2.argtypes = [i64, i64, vp, i64, vp, i64, vp]
        lib.oracle_compress_1of2.restype = i64
        lib.oracle_decompress_1of2.argtypes = [i64, i64, vp, i64, vp, vp, i64]
        lib.oracle_decompress_1of2.restype = None
        lib.oracle_gemm_sparse_1of2.argtypes = [i64, vp, i64, vp, vp, i64, dbl, dbl, vp, i64, i64, i64, i64, i64, vp, vp]
        lib.oracle_gemm_sparse_1of2.restype = None
        lib.oracle_meta_operand_bytes_1of2.argtypes = [i64, i64]
        lib.oracle_meta_operand_bytes_1of2.restype = i64
        lib.oracle_meta_permute_1of2.argtypes = [i64, i64, vp, vp, i32]
        lib.oracle_meta_permute_1of2.restype = None
        lib.oracle_kept_magnitude.argtypes = [i32, i64, i64, vp, i64, vp]
        lib.oracle_kept_magnitude.restype = dbl
        lib.oracle_apply_mask.argtypes = [i32, i64, i64, vp, i64, vp, vp, i64]
        lib.oracle_apply_mask.restype = None
        lib.oracle_prune_2d.argtypes = [i32, i64, i64, vp, i64, vp, i64]
        lib.oracle_prune_2d.restype = None
        lib.oracle_dequant.argtypes = [i64, i64, vp, vp, vp, i32, ctypes.c_float, vp, vp]
        lib.oracle_dequant.restype = None
        lib.oracle_to_double.argtypes = [i32, i64, vp, vp]
        lib.oracle_to_double.restype = None
        lib.oracle_im2col_nhwc_3x3.argtypes = [i32, i64, i64, i64, i64, vp, vp, i64]
        lib.oracle_im2col_nhwc_3x3.restype = None
        _lib = lib
    return _lib


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def _np_elem(dtype: str):
    return np.int8 if dtype == "i8" else (np.uint8 if dtype in ("e4m3", "e5m2") else np.uint16)


def _check(a: np.ndarray, dtype: str, name: str) -> np.ndarray:
    if a.dtype != _np_elem(dtype) or a.ndim != 2 or not a.flags.c_contiguous:
        raise ValueError(f"{name}: need a C-contiguous 2-D {_np_elem(dtype).__name__} array")
    return a


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def prune(x: np.ndarray, dtype: str) -> np.ndarray:
    """Keep the two largest-magnitude values of every aligned group of four along a row
    (Section 4.1, step 2); ties keep the lower index; pruned positions become +0."""
    _check(x, dtype, "x")
    M, K = x.shape
    assert K % 4 == 0
    y = np.empty_like(x)
    _load().oracle_prune(DTYPE_CODE[dtype], M, K, _ptr(x), K, _ptr(y), K)
    return y


def compress(x: np.ndarray, dtype: str):
    """Section 3.1 / Figure 1: returns (vals M x K/2, meta M x K/8 uint8 canonical, dropped)."""
    _check(x, dtype, "x")
    M, K = x.shape
    assert K % 8 == 0
    vals = np.empty((M, K // 2), dtype=x.dtype)
    meta = np.empty((M, K // 8), dtype=np.uint8)
    dropped = _load().oracle_compress(DTYPE_CODE[dtype], M, K, _ptr(x), K, _ptr(vals), K // 2,
                                      _ptr(meta))
    return vals, meta, int(dropped)


def decompress(vals: np.ndarray, meta: np.ndarray, dtype: str) -> np.ndarray:
    """Inverse of compress: scatter the kept values to the positions the metadata names."""
    _check(vals, dtype, "vals")
    M, K2 = vals.shape
    K = 2 * K2
    assert meta.dtype == np.uint8 and meta.shape == (M, K // 8) and meta.flags.c_contiguous
    y = np.empty((M, K), dtype=vals.dtype)
    _load().oracle_decompress(DTYPE_CODE[dtype], M, K, _ptr(vals), K2, _ptr(meta), _ptr(y), K)
    return y


def meta_to_operand_order(meta: np.ndarray, dtype: str) -> np.ndarray:
    """Canonical metadata (M x K/8 bytes) -> the padded tensor-core operand order (1-D bytes)."""
    M, K8 = meta.shape
    K = 8 * K8
    out = np.empty(int(_load().oracle_meta_operand_bytes(M, K)), dtype=np.uint8)
    _load().oracle_meta_permute(DTYPE_CODE[dtype], M, K, _ptr(np.ascontiguousarray(meta)),
                                _ptr(out), 0)
    return out


def meta_from_operand_order(buf: np.ndarray, M: int, K: int, dtype: str) -> np.ndarray:
    """Inverse permutation: operand-order bytes -> canonical M x K/8 metadata."""
    assert buf.dtype == np.uint8 and buf.size == int(_load().oracle_meta_operand_bytes(M, K))
    out = np.empty((M, K // 8), dtype=np.uint8)
    _load().oracle_meta_permute(DTYPE_CODE[dtype], M, K, _ptr(np.ascontiguousarray(buf)),
                                _ptr(out), 1)
    return out


def _window(M, N, rows, cols):
    i0, i1 = (0, M) if rows is None else rows
    j0, j1 = (0, N) if cols is None else cols
    assert 0 <= i0 <= i1 <= M and 0 <= j0 <= j1 <= N
    return i0, i1, j0, j1


def _c_args(C, c_dtype, N):
    if C is None:
        return 0, None, 0
    assert C.ndim == 2 and C.flags.c_contiguous
    return C_DTYPE_CODE[c_dtype], _ptr(C), C.shape[1]


def gemm_sparse(vals, meta, Bt, dtype, alpha=1.0, beta=0.0, C=None, c_dtype=None, rows=None,
                cols=None):
    """D = alpha * A_sparse * B + beta * C on a window of the output (Section 3.2, Figure 2).

    ``Bt`` is N x K (K contiguous).  Returns float64 (un-rounded) for fp types, int32 for i8.
    """
    _check(vals, dtype, "vals")
    _check(Bt, dtype, "Bt")
    M, K2 = vals.shape
    K = 2 * K2
    N = Bt.shape[0]
    assert Bt.shape[1] == K and meta.shape == (M, K // 8) and meta.dtype == np.uint8
    i0, i1, j0, j1 = _window(M, N, rows, cols)
    cd, cp, ldc = _c_args(C, c_dtype, N)
    of = np.zeros((i1 - i0, j1 - j0), dtype=np.float64) if dtype != "i8" else None
    oi = np.zeros((i1 - i0, j1 - j0), dtype=np.int32) if dtype == "i8" else None
    _load().oracle_gemm_sparse(DTYPE_CODE[dtype], M, N, K, _ptr(vals), K2,
                               _ptr(np.ascontiguousarray(meta)), _ptr(Bt), K, 1, float(alpha),
                               float(beta), cd, cp, ldc, i0, i1, j0, j1, _ptr(of), _ptr(oi))
    return oi if dtype == "i8" else of


def gemm_dense(A, Bt, dtype, alpha=1.0, beta=0.0, C=None, c_dtype=None, rows=None, cols=None):
    """Textbook D = alpha * A * B + beta * C with a dense A (M x K), same conventions."""
    _check(A, dtype, "A")
    _check(Bt, dtype, "Bt")
    M, K = A.shape
    N = Bt.shape[0]
    assert Bt.shape[1] == K
    i0, i1, j0, j1 = _window(M, N, rows, cols)
    cd, cp, ldc = _c_args(C, c_dtype, N)
    of = np.zeros((i1 - i0, j1 - j0), dtype=np.float64) if dtype != "i8" else None
    oi = np.zeros((i1 - i0, j1 - j0), dtype=np.int32) if dtype == "i8" else None
    _load().oracle_gemm_dense(DTYPE_CODE[dtype], M, N, K, _ptr(A), K, _ptr(Bt), K, 1,
                              float(alpha), float(beta), cd, cp, ldc, i0, i1, j0, j1, _ptr(of),
                              _ptr(oi))
    return oi if dtype == "i8" else of


def gemm_abs(vals, meta, Bt, dtype, rows=None, cols=None) -> np.ndarray:
    """(|A| . |B|)_ij over the kept values in float64: scale of the per-element error bound."""
    M, K2 = vals.shape
    K = 2 * K2
    N = Bt.shape[0]
    i0, i1, j0, j1 = _window(M, N, rows, cols)
    out = np.zeros((i1 - i0, j1 - j0), dtype=np.float64)
    _load().oracle_gemm_abs(DTYPE_CODE[dtype], K, _ptr(vals), K2,
                            _ptr(np.ascontiguousarray(meta)), _ptr(Bt), K, 1, i0, i1, j0, j1,
                            _ptr(out))
    return out


# ---- the 1:2 pattern of the TF32 mode: fp32 matrices travel as numpy.uint32 bit patterns ----
def _check32(a, name):
    if a.dtype != np.uint32 or a.ndim != 2 or not a.flags.c_contiguous:
        raise ValueError(f"{name}: need a C-contiguous 2-D uint32 array (fp32 bit patterns)")
    return a


def prune_1of2(x: np.ndarray) -> np.ndarray:
    """Keep the larger-magnitude value of every aligned pair along a row (ties: the first)."""
    _check32(x, "x")
    M, K = x.shape
    y = np.empty_like(x)
    _load().oracle_prune_1of2(M, K, _ptr(x), K, _ptr(y), K)
    return y


def compress_1of2(x: np.ndarray):
    """Returns (vals M x K/2 uint32, meta M x K/4 uint8 canonical nibbles 0x4 / 0xE, dropped)."""
    _check32(x, "x")
    M, K = x.shape
    assert K % 4 == 0
    vals = np.empty((M, K // 2), dtype=np.uint32)
    meta = np.empty((M, K // 4), dtype=np.uint8)
    dropped = _load().oracle_compress_1of2(M, K, _ptr(x), K, _ptr(vals), K // 2, _ptr(meta))
    return vals, meta, int(dropped)


def decompress_1of2(vals: np.ndarray, meta: np.ndarray) -> np.ndarray:
    _check32(vals, "vals")
    M, K2 = vals.shape
    y = np.empty((M, 2 * K2), dtype=np.uint32)
    _load().oracle_decompress_1of2(M, 2 * K2, _ptr(vals), K2, _ptr(np.ascontiguousarray(meta)), _ptr(y), 2 * K2)
    return y


def gemm_sparse_1of2(vals, meta, Bt, alpha=1.0, beta=0.0, C=None, rows=None, cols=None):
    """(D, |A|.|B|) in float64 on an output window; Bt is N x K uint32 bit patterns, C float32 M x N."""
    _check32(vals, "vals")
    _check32(Bt, "Bt")
    M, K2 = vals.shape
    K, N = 2 * K2, Bt.shape[0]
    assert Bt.shape[1] == K and meta.shape == (M, K // 4)
    i0, i1, j0, j1 = _window(M, N, rows, cols)
    out = np.zeros((i1 - i0, j1 - j0), dtype=np.float64)
    mag = np.zeros_like(out)
    if C is not None:
        assert C.dtype == np.float32 and C.shape == (M, N) and C.flags.c_contiguous
    _load().oracle_gemm_sparse_1of2(K, _ptr(vals), K2, _ptr(np.ascontiguousarray(meta)), _ptr(Bt), K, float(alpha),
                                    float(beta), _ptr(C), N, i0, i1, j0, j1, _ptr(out), _ptr(mag))
    return out, mag


def meta_to_operand_order_1of2(meta: np.ndarray) -> np.ndarray:
    M, K4 = meta.shape
    K = 4 * K4
    out = np.empty(int(_load().oracle_meta_operand_bytes_1of2(M, K)), dtype=np.uint8)
    _load().oracle_meta_permute_1of2(M, K, _ptr(np.ascontiguousarray(meta)), _ptr(out), 0)
    return out


def meta_from_operand_order_1of2(buf: np.ndarray, M: int, K: int) -> np.ndarray:
    out = np.empty((M, K // 4), dtype=np.uint8)
    _load().oracle_meta_permute_1of2(M, K, _ptr(np.ascontiguousarray(buf)), _ptr(out), 1)
    return out


def kept_magnitude(x: np.ndarray, dtype: str, perm=None) -> float:
    """Total magnitude kept by 2:4 pruning of x with its columns permuted by `perm` (Section 4.1)."""
    _check(x, dtype, "x")
    M, K = x.shape
    p = None if perm is None else np.ascontiguousarray(perm, dtype=np.int32)
    return float(_load().oracle_kept_magnitude(DTYPE_CODE[dtype], M, K, _ptr(x), K, _ptr(p)))


def apply_mask(w: np.ndarray, meta: np.ndarray, dtype: str) -> np.ndarray:
    """Keep w where the canonical metadata names the position, +0 elsewhere (Section 4.1 step 3)."""
    _check(w, dtype, "w")
    M, K = w.shape
    y = np.empty_like(w)
    _load().oracle_apply_mask(DTYPE_CODE[dtype], M, K, _ptr(w), K, _ptr(np.ascontiguousarray(meta)), _ptr(y), K)
    return y


def prune_2d(x: np.ndarray, dtype: str) -> np.ndarray:
    """2:4 along rows and columns of every aligned 4 x 4 block, exhaustive search (Section 6)."""
    _check(x, dtype, "x")
    M, K = x.shape
    assert M % 4 == 0 and K % 4 == 0
    y = np.empty_like(x)
    _load().oracle_prune_2d(DTYPE_CODE[dtype], M, K, _ptr(x), K, _ptr(y), K)
    return y


def dequant(acc: np.ndarray, row_scale: np.ndarray, bias=None, relu=False, out_scale=1.0):
    """Dequantising epilogue on an exact int32 accumulator window (rows of `acc` pair with row_scale):
    returns (float64 result, int8 code quantised with fp32 decisions)."""
    assert acc.dtype == np.int32 and acc.ndim == 2 and acc.flags.c_contiguous
    rs = np.ascontiguousarray(row_scale, dtype=np.float32)
    b = None if bias is None else np.ascontiguousarray(bias, dtype=np.float32)
    assert rs.shape == (acc.shape[0],) and (b is None or b.shape == rs.shape)
    f = np.empty(acc.shape, dtype=np.float64)
    q = np.empty(acc.shape, dtype=np.int8)
    _load().oracle_dequant(acc.shape[0], acc.shape[1], _ptr(acc), _ptr(rs), _ptr(b), 1 if relu else 0,
                           ctypes.c_float(out_scale), _ptr(f), _ptr(q))
    return f, q


def im2col_nhwc_3x3(x: np.ndarray, dtype: str) -> np.ndarray:
    """NHWC input (Nb,H,W,C) -> (Nb*H*W) x (9*C) matrix, K index (r*3+s)*C + c, zero padded."""
    assert x.ndim == 4 and x.flags.c_contiguous and x.dtype == _np_elem(dtype)
    Nb, H, W, C = x.shape
    out = np.empty((Nb * H * W, 9 * C), dtype=x.dtype)
    _load().oracle_im2col_nhwc_3x3(DTYPE_CODE[dtype], Nb, H, W, C, _ptr(x), _ptr(out), 9 * C)
    return out


def bits_to_float64(a: np.ndarray, dtype: str) -> np.ndarray:
    """Exact widening of stored values (bit patterns for f16/bf16) to float64, via numpy."""
    if dtype == "i8":
        return a.astype(np.float64)
    if dtype == "f16":
        return a.view(np.float16).astype(np.float64)
    if dtype in ("e4m3", "e5m2"):
        a = np.ascontiguousarray(a)
        out = np.empty(a.shape, dtype=np.float64)
        _load().oracle_to_double(DTYPE_CODE[dtype], a.size, _ptr(a), _ptr(out))
        return out
    return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
