"""Seeded synthetic inputs shaped like the paper's workloads (numpy only, host side).

Holds none of the method's arithmetic: a front end to the stateless counter-based generator in
``csrc/inputs_gen.c`` (plain C, compiled with gcc on first use) and the five benchmark
configurations.  Both the CUDA path and the CPU oracle draw their inputs from here.
Because value (tensor, row, col) depends only on (seed, tensor id, row * ncols + col), any row
range of a matrix can be regenerated on its own, which is how sampled output tiles of the
largest configuration are checked without materialising everything twice.

Storage convention: fp16 / bf16 matrices are numpy.uint16 BIT PATTERNS (round-to-nearest-even
from float64 / float32), int8 matrices are numpy.int8, "tf32" matrices are numpy.uint32 bit
patterns of fp32 values that are exactly representable in TF32 (10 mantissa bits).

The configurations stand in for trained networks the paper evaluates (BERT-base FFN,
GPT-3-scale FFN with hidden size 12288, a ResNet-50 3x3 convolution, an INT8 linear layer as
in the paper's GEMM sweep); only their shapes and value distributions are reproduced.
"""
from __future__ import annotations

import ctypes
from dataclasses import dataclass
import os
import subprocess

import numpy as np

TENSOR_A, TENSOR_B, TENSOR_C, TENSOR_TILES = 0, 1, 2, 3

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "csrc", "inputs_gen.c")
_LIB = os.path.join(_HERE, "libsp24_inputs.so")
_NP_STORAGE = {"i8": np.int8, "tf32": np.uint32, "e4m3": np.uint8, "e5m2": np.uint8}  # else uint16 bit patterns
_DTYPE = {"f16": 0, "bf16": 1, "i8": 2, "tf32": 3, "e4m3": 5, "e5m2": 6}
_lib = None


def build(force: bool = False) -> str:
    """Compile the generator (plain C + OpenMP, gcc) next to the package; returns the .so path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = f"{_LIB}.{os.getpid()}.tmp"
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        u64 = ctypes.c_uint64
        lib.sp24_inputs_raw.argtypes = [u64, u64, u64, u64]
        lib.sp24_inputs_raw.restype = u64
        lib.sp24_inputs_fill.argtypes = [ctypes.c_int, ctypes.c_double, ctypes.c_double,
                                         ctypes.c_int, u64, u64, u64, u64, ctypes.c_void_p]
        lib.sp24_inputs_fill.restype = None
        lib.sp24_inputs_to_fp8.argtypes = [ctypes.c_double, ctypes.c_int]
        lib.sp24_inputs_to_fp8.restype = ctypes.c_uint8
        _lib = lib
    return _lib


def raw_u64(seed: int, tensor_id: int, start: int, count: int) -> np.ndarray:
    """64 random bits for linear indices start .. start+count-1 of one tensor."""
    lib = _load()
    return np.array([lib.sp24_inputs_raw(seed, tensor_id, 0, start + i) for i in range(count)],
                    dtype=np.uint64)


def to_storage(x: np.ndarray, dtype: str) -> np.ndarray:
    """float64 / integer values -> stored representation (uint16 bit patterns or int8), for
    hand-made test matrices; round-to-nearest-even."""
    x = np.asarray(x)
    if dtype == "i8":
        return x.astype(np.int8)
    if dtype == "f16":
        return x.astype(np.float16).view(np.uint16)
    if dtype == "bf16":
        bits = np.ascontiguousarray(x.astype(np.float32)).view(np.uint32)
        rounding = ((bits >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
        return ((bits + rounding) >> np.uint32(16)).astype(np.uint16)
    if dtype in ("e4m3", "e5m2"):
        lib = _load()
        flat = np.asarray(x, dtype=np.float64).ravel()
        out = np.array([lib.sp24_inputs_to_fp8(float(v), 1 if dtype == "e5m2" else 0) for v in flat], dtype=np.uint8)
        return out.reshape(np.shape(x))
    raise ValueError(dtype)


@dataclass(frozen=True)
class Config:
    """One benchmark configuration: D (M x N) = alpha * A (M x K, 2:4 along K) * B (K x N) + beta * C."""
    name: str
    seed: int
    M: int
    N: int
    K: int
    ab_type: str          # "f16" | "bf16" | "i8"
    cd_type: str          # "f16" | "bf16" | "f32" | "i32"
    a_dist: tuple         # ("normal", sigma) | ("int8",)
    b_dist: tuple         # ("normal", sigma) | ("uniform", lo, hi) | ("int8",) | ("im2col",)
    alpha: float = 1.0
    beta: float = 0.0
    c_dist: tuple | None = None
    conv: tuple | None = None   # (batch, H, W, C) of the NHWC input when B is an im2col

    @property
    def dense_equiv_flop(self) -> float:
        return 2.0 * self.M * self.N * self.K


CONFIGS = {
    # Tiny fp16 case: the oracle finishes in well under a second.
    "tiny_f16": Config("tiny_f16", 0, 256, 256, 512, "f16", "f16", ("normal", 1.0),
                       ("uniform", -1.0, 1.0)),
    # BERT-base FFN up-projection: weight 3072 x 768, 32 x 128 tokens.
    "bert_ffn_bf16": Config("bert_ffn_bf16", 1, 3072, 4096, 768, "bf16", "bf16", ("normal", 0.02),
                            ("normal", 1.0)),
    # INT8 linear layer, as in the paper's INT8 sparse-vs-dense GEMM sweep.
    "int8_linear": Config("int8_linear", 2, 4096, 8192, 4096, "i8", "i32", ("int8",), ("int8",)),
    # GPT-3-scale FFN: hidden size 12288, 8192 tokens, beta = 1 with a bf16 C.
    "gpt3_ffn_bf16": Config("gpt3_ffn_bf16", 3, 49152, 8192, 12288, "bf16", "bf16",
                            ("normal", 0.02), ("normal", 1.0), 1.0, 1.0, ("normal", 1.0)),
    # ResNet-50-style 3x3 convolution lowered to a GEMM, K ordered (r, s, c).
    "resnet_conv_f16": Config("resnet_conv_f16", 4, 256, 256 * 14 * 14, 2304, "f16", "f16",
                              ("normal", float(np.sqrt(2.0 / 2304.0))), ("im2col",),
                              conv=(256, 14, 14, 256)),
}
CONFIG_ORDER = ["tiny_f16", "bert_ffn_bf16", "int8_linear", "gpt3_ffn_bf16", "resnet_conv_f16"]


def scaled(cfg: Config, M=None, N=None, K=None, name=None, conv=None) -> Config:
    """Same distributions and dtypes at other dimensions (parity tests at oracle-friendly sizes).

    For the convolution config pass the new NHWC shape as `conv`; N and K follow from it."""
    from dataclasses import replace
    if conv is not None:
        nb, h, w, c = conv
        N, K = nb * h * w, 9 * c
    return replace(cfg, M=M or cfg.M, N=N or cfg.N, K=K or cfg.K,
                   name=name or cfg.name + "_scaled", conv=conv if conv is not None else cfg.conv)


_KIND = {"normal": 0, "uniform": 1, "int8": 2, "relu_normal": 3}


def _matrix(dist, dtype, seed, tensor_id, ncols, row0, row1) -> np.ndarray:
    """Rows row0..row1-1 of a (?, ncols) matrix whose element (r, c) has linear index r*ncols+c."""
    nrows = row1 - row0
    out = np.empty((nrows, ncols), dtype=_NP_STORAGE.get(dtype, np.uint16))
    if nrows == 0 or ncols == 0:
        return out
    p0 = float(dist[1]) if len(dist) > 1 else 0.0
    p1 = float(dist[2]) if len(dist) > 2 else 0.0
    _load().sp24_inputs_fill(_KIND[dist[0]], p0, p1, _DTYPE[dtype], seed, tensor_id,
                             row0 * ncols, nrows * ncols, out.ctypes.data_as(ctypes.c_void_p))
    return out


def gen_A(cfg: Config, rows=None) -> np.ndarray:
    """Dense weight matrix before pruning, rows [r0, r1) (default all): shape (r1-r0, K)."""
    r0, r1 = rows or (0, cfg.M)
    return _matrix(cfg.a_dist, cfg.ab_type, cfg.seed, TENSOR_A, cfg.K, r0, r1)


def gen_conv_input(cfg: Config, images=None) -> np.ndarray:
    """NHWC activation of the convolution config, images [n0, n1): ReLU(N(0,1)) in fp16."""
    nb, h, w, c = cfg.conv
    n0, n1 = images or (0, nb)
    flat = _matrix(("relu_normal", 1.0), cfg.ab_type, cfg.seed, TENSOR_B, h * w * c, n0, n1)
    return flat.reshape(n1 - n0, h, w, c)


def gen_Bt(cfg: Config, cols=None) -> np.ndarray:
    """Activations as an (N, K) array (K contiguous), columns [c0, c1) of the K x N matrix B.

    Not defined for the convolution config, whose B is the im2col of gen_conv_input."""
    if cfg.b_dist[0] == "im2col":
        raise ValueError("B of the convolution config is built by im2col from gen_conv_input")
    c0, c1 = cols or (0, cfg.N)
    return _matrix(cfg.b_dist, cfg.ab_type, cfg.seed, TENSOR_B, cfg.K, c0, c1)


def gen_C(cfg: Config, rows=None) -> np.ndarray | None:
    """C (M x N, row-major) rows [r0, r1), or None when beta == 0."""
    if cfg.c_dist is None:
        return None
    r0, r1 = rows or (0, cfg.M)
    return _matrix(cfg.c_dist, cfg.cd_type, cfg.seed, TENSOR_C, cfg.N, r0, r1)


def sample_tiles(cfg: Config, count: int, tile: int = 128) -> list[tuple[int, int]]:
    """`count` distinct (tile_row, tile_col) indices of the output, seeded, without replacement."""
    tm, tn = cfg.M // tile, cfg.N // tile
    total = tm * tn
    count = min(count, total)
    order = np.argsort(raw_u64(cfg.seed, TENSOR_TILES, 0, total), kind="stable")[:count]
    return [(int(t) // tn, int(t) % tn) for t in order]
