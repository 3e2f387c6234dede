"""Pins for the CPU oracle: what the paper and plain mathematics fix, checked without a GPU.

Each test compares the oracle with something that is not the oracle: a printed example, a
closed form, a brute-force enumeration written independently here, or a library routine
(numpy float64 / int64 matmul) on a case that reduces to it.
"""
import itertools
import os

import numpy as np
import pytest

import oracle
from paper_2104_08378_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
DTYPES = ["f16", "bf16", "i8"]


def _golden(name):
    rows = []
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if line and not line.startswith("#"):
                rows.append(line.split())
    return rows


def _rand(dtype, M, K, seed, dist=None):
    dist = dist or (("int8",) if dtype == "i8" else ("normal", 1.0))
    return inputs._matrix(dist, dtype, seed, 7, K, 0, M)


def _f64(a, dtype):
    return oracle.bits_to_float64(a, dtype)


def _from_float(x, dtype):
    return inputs.to_storage(np.asarray(x, dtype=np.float64), dtype)


def _key(a, dtype):
    return np.abs(a.astype(np.int32)) if dtype == "i8" else (a & 0x7FFF).astype(np.int32)


# ---------------------------------------------------------------------------------------
# the numeric decoders of the oracle agree with numpy on every finite bit pattern
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", ["f16", "bf16"])
def test_decode_all_finite_bit_patterns(dtype):
    bits = np.arange(65536, dtype=np.uint32)
    expo = (bits >> 10) & 0x1F if dtype == "f16" else (bits >> 7) & 0xFF
    finite = bits[expo != (31 if dtype == "f16" else 255)].astype(np.uint16)
    K = 64
    pad = (-len(finite)) % K
    A = np.concatenate([finite, np.zeros(pad, np.uint16)]).reshape(-1, K)
    eye = _from_float(np.eye(K), dtype)
    D = oracle.gemm_dense(A, eye, dtype)          # A . I decodes every element exactly
    assert np.array_equal(D, _f64(A, dtype))


# ---------------------------------------------------------------------------------------
# prune: pattern invariant, kept values untouched, idempotent (Section 3, Section 4.1)
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", DTYPES)
def test_prune_invariants(dtype):
    x = _rand(dtype, 37, 96, 11)
    y = oracle.prune(x, dtype)
    g = y.reshape(37, 24, 4)
    assert ((g == 0).sum(axis=2) >= 2).all()                 # at least two zeros per group
    kept = g != 0
    assert np.array_equal(g[kept], x.reshape(37, 24, 4)[kept])  # kept values bit-identical
    assert np.array_equal(oracle.prune(y, dtype), y)          # idempotent
    # the two kept magnitudes are never smaller than a dropped one
    k = _key(x, dtype).reshape(37, 24, 4)
    kept_pos = np.zeros_like(kept)
    vals, meta, _ = oracle.compress(x, dtype)
    nib = np.stack([meta & 0xF, meta >> 4], axis=2).reshape(37, 24)
    for t in range(2):
        np.put_along_axis(kept_pos, ((nib >> (2 * t)) & 3)[..., None], True, axis=2)
    assert (kept_pos.sum(axis=2) == 2).all()
    min_kept = np.where(kept_pos, k, 1 << 20).min(axis=2)
    max_drop = np.where(~kept_pos, k, -1).max(axis=2)
    assert (min_kept >= max_drop).all()


def _brute_force_keep(keys):
    """Independent definition: over the six keep-patterns take the largest kept-key sum; among
    equals the lexicographically smallest (p0, p1)."""
    best = None
    for p0, p1 in itertools.combinations(range(4), 2):
        s = keys[p0] + keys[p1]
        if best is None or s > best[0]:
            best = (s, p0, p1)
    return best[1], best[2]


@pytest.mark.parametrize("dtype", DTYPES)
def test_prune_matches_brute_force_over_all_patterns(dtype):
    alphabet = [-2.0, -1.0, -0.0, 0.0, 1.0, 2.0, 3.0]
    groups = np.array(list(itertools.product(alphabet, repeat=4)))      # 7^4 groups
    x = _from_float(groups, dtype).reshape(-1, 4)
    if dtype != "i8":
        x[groups.reshape(-1, 4) == 0] = 0
        neg_zero = np.signbit(groups.reshape(-1, 4)) & (groups.reshape(-1, 4) == 0)
        x[neg_zero] = 0x8000                                         # keep -0.0 as a pattern
    rnd = _rand(dtype, 500, 4, 5)
    x = np.concatenate([x, rnd])
    x = np.ascontiguousarray(np.concatenate([x, np.zeros_like(x)], axis=1))  # K = 8: pad group
    vals, meta, _ = oracle.compress(x, dtype)
    y = oracle.prune(x, dtype)
    keys = _key(x, dtype)
    for i in range(x.shape[0]):
        p0, p1 = _brute_force_keep(keys[i, :4])
        assert meta[i, 0] & 0xF == p0 | (p1 << 2), (i, x[i])
        expect = np.zeros(8, dtype=x.dtype)
        expect[p0], expect[p1] = x[i, p0], x[i, p1]
        assert np.array_equal(y[i], expect)
        assert vals[i, 0] == x[i, p0] and vals[i, 1] == x[i, p1]


@pytest.mark.parametrize("dtype", DTYPES)
def test_ties_keep_lower_index(dtype):
    x = _from_float([[1, 1, 1, 1], [2, 1, 1, 1], [1, 2, 2, 2], [-1, 1, -1, 1], [0, 0, 0, 5]], dtype)
    _, meta, _ = oracle.compress(np.ascontiguousarray(np.tile(x, (1, 2))), dtype)
    assert [int(m) & 0xF for m in meta[:, 0]] == [0x4, 0x4, 0x9, 0x4, 0xC]


# ---------------------------------------------------------------------------------------
# compressed format (Section 3.1, Figure 1)
# ---------------------------------------------------------------------------------------
def test_metadata_example_from_the_paper():
    g = dict((r[0], r[1:]) for r in _golden("metadata_example.txt"))
    p = [int(v) for v in g["group0_positions"]] , [int(v) for v in g["group1_positions"]]
    for dtype in DTYPES:
        row = np.zeros((1, 8))
        row[0, p[0][0]], row[0, p[0][1]] = 3.0, -5.0
        row[0, 4 + p[1][0]], row[0, 4 + p[1][1]] = 7.0, 2.0
        x = _from_float(row, dtype)
        vals, meta, dropped = oracle.compress(x, dtype)
        nibbles = [int(meta[0, 0]) & 0xF, int(meta[0, 0]) >> 4]
        decoded = [[n & 3, n >> 2] for n in nibbles]
        assert decoded == [p[0], p[1]]
        assert nibbles == [int(g["nibble0"][0], 16), int(g["nibble1"][0], 16)]
        assert int(meta[0, 0]) == int(g["first_byte"][0], 16)
        assert np.array_equal(_f64(vals, dtype), [[3.0, -5.0, 7.0, 2.0]])
        assert dropped == 0


@pytest.mark.parametrize("dtype", DTYPES)
def test_storage_arithmetic(dtype):
    g = dict((r[0], float(r[1])) for r in _golden("storage_arithmetic.txt"))
    M, K = 16, 64
    x = _rand(dtype, M, K, 3)
    vals, meta, _ = oracle.compress(x, dtype)
    assert vals.shape == (M, K // 2)                               # R x C -> R x C/2
    overhead = meta.nbytes / vals.nbytes
    bits_per_group = (vals.nbytes + meta.nbytes) * 8 / (M * K / 4)
    saving = 1 - (vals.nbytes + meta.nbytes) / x.nbytes
    if dtype == "i8":
        assert overhead == g["meta_overhead_8bit"]
        assert abs(saving - g["saving_8bit_approx"]) < 0.01
    else:
        assert overhead == g["meta_overhead_16bit"]
        assert x.nbytes * 8 / (M * K / 4) == g["dense_bits_per_group_16bit"]
        assert bits_per_group == g["compressed_bits_per_group_16bit"]
        assert abs(saving - g["saving_16bit_approx"]) < 0.01


@pytest.mark.parametrize("dtype", DTYPES)
def test_roundtrip_and_valid_nibbles(dtype):
    x = _rand(dtype, 33, 160, 21)
    vals, meta, dropped = oracle.compress(x, dtype)
    y = oracle.prune(x, dtype)
    assert np.array_equal(oracle.decompress(vals, meta, dtype), y)   # decompress(compress) == prune
    v2, m2, d2 = oracle.compress(y, dtype)
    assert np.array_equal(v2, vals) and np.array_equal(m2, meta) and d2 == 0
    nib = np.concatenate([(meta & 0xF).ravel(), (meta >> 4).ravel()])
    assert set(np.unique(nib).tolist()) <= {0x4, 0x8, 0xC, 0x9, 0xD, 0xE}
    assert dropped == int(((_key(x, dtype) != 0) & (y == 0)).sum())


@pytest.mark.parametrize("dtype", DTYPES)
def test_groups_with_more_than_two_zeros_still_store_two_values(dtype):
    row = np.zeros((3, 8))
    row[1, 2] = 4.0           # one non-zero: positions (0, 2) -> fillers are the lowest zeros
    row[2, 5] = -1.0          # second group, position 1 -> (0, 1)
    x = _from_float(row, dtype)
    vals, meta, dropped = oracle.compress(x, dtype)
    assert vals.shape == (3, 4) and dropped == 0
    assert int(meta[0, 0]) == 0x44                      # all-zero groups: positions 0,1
    assert int(meta[1, 0]) & 0xF == (0 | 2 << 2)
    assert int(meta[2, 0]) >> 4 == (0 | 1 << 2)
    assert np.array_equal(oracle.decompress(vals, meta, dtype), x)


# ---------------------------------------------------------------------------------------
# GEMM (Section 3.2, Figure 2)
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", DTYPES)
def test_sparse_gemm_equals_library_matmul_on_pruned_matrix(dtype):
    M, N, K = 24, 20, 64
    x = _rand(dtype, M, K, 31)
    Bt = _rand(dtype, N, K, 32, ("int8",) if dtype == "i8" else ("uniform", -1.0, 1.0))
    vals, meta, _ = oracle.compress(x, dtype)
    D = oracle.gemm_sparse(vals, meta, Bt, dtype)
    pruned = oracle.decompress(vals, meta, dtype)
    if dtype == "i8":
        ref = pruned.astype(np.int64) @ Bt.astype(np.int64).T
        assert np.array_equal(D, ref.astype(np.int32))
    else:
        ref = _f64(pruned, dtype) @ _f64(Bt, dtype).T
        scale = np.abs(_f64(pruned, dtype)) @ np.abs(_f64(Bt, dtype)).T
        assert np.all(np.abs(D - ref) <= 1e-13 * scale + 1e-300)
        # and exactly the oracle's own dense loop on the pruned matrix (added terms are zeros)
        assert np.array_equal(D, oracle.gemm_dense(oracle.prune(x, dtype), Bt, dtype))
    # a transposed-operand or wrong-index mistake cannot survive a window check either
    sub = oracle.gemm_sparse(vals, meta, Bt, dtype, rows=(5, 9), cols=(3, 17))
    assert np.array_equal(sub, D[5:9, 3:17])


@pytest.mark.parametrize("dtype", ["f16", "bf16", "e4m3", "e5m2"])
def test_gemm_abs_equals_library_matmul_of_magnitudes(dtype):
    """The scale of the per-element error bound, (|A| . |B|)_ij over the kept values: equal to a
    numpy float64 matmul of the magnitudes of the decompressed matrix and of B, in full and on a
    window (an inflated scale -- a sum over the wrong range, a wrong leading dimension -- would
    loosen every floating-point parity test without failing any of them)."""
    M, N, K = 28, 36, 96
    x = _rand(dtype, M, K, 61)
    x[::3, 1::4] = 0                                   # some groups with fillers (zeros that are stored)
    Bt = _rand(dtype, N, K, 62, ("uniform", -1.0, 1.0))
    vals, meta, _ = oracle.compress(x, dtype)
    lib = np.abs(_f64(oracle.decompress(vals, meta, dtype), dtype)) @ np.abs(_f64(Bt, dtype)).T
    got = oracle.gemm_abs(vals, meta, Bt, dtype)
    assert got.shape == (M, N) and np.all(got >= 0)
    assert np.all(np.abs(got - lib) <= 1e-13 * lib + 1e-300)
    sub = oracle.gemm_abs(vals, meta, Bt, dtype, rows=(4, 13), cols=(7, 30))
    assert np.array_equal(sub, got[4:13, 7:30])
    # it bounds the signed product, and meets it when every term has one sign
    D = oracle.gemm_sparse(vals, meta, Bt, dtype)
    assert np.all(np.abs(D) <= got * (1 + 1e-13))
    pos_a, pos_b = x & (0x7F if dtype in ("e4m3", "e5m2") else 0x7FFF), Bt & (0x7F if dtype in ("e4m3", "e5m2") else 0x7FFF)
    vp, mp, _ = oracle.compress(pos_a, dtype)
    assert np.array_equal(oracle.gemm_abs(vp, mp, pos_b, dtype), oracle.gemm_sparse(vp, mp, pos_b, dtype))
    # all ones: K/2 kept products of 1 each
    ones_a, ones_b = _from_float(np.ones((4, K)), dtype), _from_float(-np.ones((6, K)), dtype)
    v1, m1, _ = oracle.compress(ones_a, dtype)
    assert np.all(oracle.gemm_abs(v1, m1, ones_b, dtype) == K // 2)


@pytest.mark.parametrize("dtype", DTYPES)
def test_gemm_closed_forms(dtype):
    K = 32
    x = _rand(dtype, 8, K, 41)
    vals, meta, _ = oracle.compress(x, dtype)
    eye = _from_float(np.eye(K), dtype)
    D = oracle.gemm_sparse(vals, meta, eye, dtype)                   # B = I  =>  D = decompress(A)
    assert np.array_equal(np.asarray(D, dtype=np.float64),
                          _f64(oracle.decompress(vals, meta, dtype), dtype))
    ones_a = _from_float(np.ones((4, K)), dtype)
    ones_b = _from_float(np.ones((6, K)), dtype)
    v1, m1, _ = oracle.compress(ones_a, dtype)
    assert np.all(oracle.gemm_sparse(v1, m1, ones_b, dtype) == K // 2)  # all ones => K/2
    # one non-zero per row selects (a scaled copy of) one row of B
    single = np.zeros((3, K))
    single[0, 5], single[1, 30], single[2, 0] = 2.0, -1.0, 3.0
    vs, ms, _ = oracle.compress(_from_float(single, dtype), dtype)
    Bt = _rand(dtype, 9, K, 43)
    Ds = np.asarray(oracle.gemm_sparse(vs, ms, Bt, dtype), dtype=np.float64)
    Bf = _f64(Bt, dtype)
    assert np.array_equal(Ds, np.stack([2.0 * Bf[:, 5], -1.0 * Bf[:, 30], 3.0 * Bf[:, 0]]))


def test_gemm_alpha_beta():
    dtype = "bf16"
    x, Bt = _rand(dtype, 8, 32, 51), _rand(dtype, 12, 32, 52)
    C = _rand(dtype, 8, 12, 53)
    vals, meta, _ = oracle.compress(x, dtype)
    base = oracle.gemm_sparse(vals, meta, Bt, dtype)
    Cf = _f64(C, dtype)
    assert np.array_equal(oracle.gemm_sparse(vals, meta, Bt, dtype, 0.0, 1.0, C, "bf16"), Cf)
    assert np.array_equal(oracle.gemm_sparse(vals, meta, Bt, dtype, 2.0, 0.0), 2.0 * base)
    got = oracle.gemm_sparse(vals, meta, Bt, dtype, 0.5, -3.0, C, "bf16")
    assert np.array_equal(got, 0.5 * base - 3.0 * Cf)
    C32 = np.ascontiguousarray(Cf.astype(np.float32))
    assert np.array_equal(oracle.gemm_sparse(vals, meta, Bt, dtype, 1.0, 1.0, C32, "f32"), base + Cf)


def test_int8_extremes_closed_form():
    K = 64
    a = np.full((2, K), 127, dtype=np.int8)
    a[1] = -127
    b = np.full((3, K), -127, dtype=np.int8)
    vals, meta, _ = oracle.compress(a, "i8")
    D = oracle.gemm_sparse(vals, meta, b, "i8")
    assert np.array_equal(D, np.array([[-127 * 127 * K // 2] * 3, [127 * 127 * K // 2] * 3]))
    Cm = np.arange(6, dtype=np.int32).reshape(2, 3)
    assert np.array_equal(oracle.gemm_sparse(vals, meta, b, "i8", 1, 1, Cm, "i32"), D + Cm)
    m128 = np.array([[-128, 127, 1, 0] * 2], dtype=np.int8)            # -128 ranks as 128
    _, mm, _ = oracle.compress(m128, "i8")
    assert int(mm[0, 0]) == 0x44


# ---------------------------------------------------------------------------------------
# im2col (Section 4.2: a convolution's reduction dimension is C*R*S)
# ---------------------------------------------------------------------------------------
def test_im2col_gemm_equals_direct_convolution():
    dtype = "f16"
    Nb, H, W, C, Kout = 2, 5, 4, 8, 6
    x = _rand(dtype, Nb * H * W, C, 61).reshape(Nb, H, W, C)
    wgt = _rand(dtype, Kout, 9 * C, 62)                      # (k, (r, s, c))
    cols = oracle.im2col_nhwc_3x3(np.ascontiguousarray(x), dtype)
    out = oracle.gemm_dense(wgt, cols, dtype)                # Kout x (Nb*H*W)
    xf, wf = _f64(x, dtype), _f64(wgt, dtype).reshape(Kout, 3, 3, C)
    direct = np.zeros((Kout, Nb, H, W))
    for k in range(Kout):
        for n in range(Nb):
            for h in range(H):
                for w in range(W):
                    acc = 0.0
                    for r in range(3):
                        for s in range(3):
                            hh, ww = h + r - 1, w + s - 1
                            if 0 <= hh < H and 0 <= ww < W:
                                for c in range(C):
                                    acc += wf[k, r, s, c] * xf[n, hh, ww, c]
                    direct[k, n, h, w] = acc
    assert np.allclose(out, direct.reshape(Kout, -1), rtol=0, atol=1e-12)


# ---------------------------------------------------------------------------------------
# tensor-core operand order of the metadata (a permutation of the canonical nibbles)
# ---------------------------------------------------------------------------------------
@pytest.mark.parametrize("dtype", ["bf16", "i8"])
def test_operand_order_hand_computed_positions(dtype):
    for d, r, q, byte, nib in _golden("operand_order_positions.txt"):
        if d != dtype:
            continue
        r, q, byte, nib = int(r), int(q), int(byte), int(nib)
        meta = np.full((128, 16), 0x44, dtype=np.uint8)
        meta[r, q // 2] = (0x4E if q % 2 == 0 else 0xE4)          # mark one nibble with 0xE
        buf = oracle.meta_to_operand_order(meta, dtype)
        assert buf.size == 4096                                   # K padded to 256 columns
        where = np.flatnonzero(buf != 0x44)
        assert where.tolist() == [byte]
        assert (int(buf[byte]) >> (4 * nib)) & 0xF == 0xE


@pytest.mark.parametrize("dtype", ["f16", "i8"])
def test_operand_order_is_a_padded_bijection(dtype):
    M, K = 200, 640                                               # ragged in M and in K
    x = _rand(dtype, M, K, 71)
    _, meta, _ = oracle.compress(x, dtype)
    buf = oracle.meta_to_operand_order(meta, dtype)
    assert buf.size == 2 * 3 * 4096
    assert np.array_equal(oracle.meta_from_operand_order(buf, M, K, dtype), meta)
    nib = np.concatenate([buf & 0xF, buf >> 4])
    assert set(np.unique(nib).tolist()) <= {0x4, 0x8, 0xC, 0x9, 0xD, 0xE}
    # multiset of nibbles = canonical nibbles + padding nibbles 0x4
    canon = np.bincount(np.concatenate([(meta & 0xF).ravel(), (meta >> 4).ravel()]), minlength=16)
    hw = np.bincount(nib, minlength=16)
    canon[4] += buf.size * 2 - meta.size * 2
    assert np.array_equal(canon, hw)


# ---------------------------------------------------------------------------------------
# dequantising epilogue (Section 4.4, Section 5.1)
# ---------------------------------------------------------------------------------------
def test_dequant_closed_forms_and_numpy_float32():
    rng = np.random.default_rng(3)
    acc = rng.integers(-40_000_000, 40_000_000, size=(6, 50), dtype=np.int64).astype(np.int32)
    acc[0, :8] = [0, 1, -1, 3, -3, 127, -127, 2**24 + 1]
    ones = np.ones(6, np.float32)
    f, q = oracle.dequant(acc, ones)                       # scale 1, no bias: identity / saturation
    assert np.array_equal(f, acc.astype(np.float64))
    assert np.array_equal(q[0, :7], [0, 1, -1, 3, -3, 127, -127]) and q[0, 7] == 127
    f, q = oracle.dequant(acc, ones, relu=True)
    assert np.array_equal(f, np.maximum(acc, 0).astype(np.float64)) and (q >= 0).all()
    # halves round to even: acc * 0.5 with out_scale 1
    half = np.array([[1, 3, 5, -1, -3, 7]], dtype=np.int32)
    _, q = oracle.dequant(half, np.array([0.5], np.float32))
    assert q.tolist() == [[0, 2, 2, 0, -2, 4]]
    # general case against numpy float32 arithmetic (an independent library evaluation)
    rs = rng.uniform(1e-6, 3e-6, size=6).astype(np.float32)
    bias = rng.normal(size=6).astype(np.float32)
    out_scale = np.float32(0.37)
    f, q = oracle.dequant(acc, rs, bias, relu=True, out_scale=float(out_scale))
    want64 = np.maximum(rs.astype(np.float64)[:, None] * acc + bias.astype(np.float64)[:, None], 0)
    assert np.array_equal(f, want64)
    t = acc.astype(np.float32)
    y64 = rs.astype(np.float64)[:, None] * t.astype(np.float64) + bias.astype(np.float64)[:, None]  # exact product+sum
    y = np.maximum(y64.astype(np.float32), np.float32(0))                                          # = one fma rounding
    z = (y * (np.float32(1) / out_scale)).astype(np.float32)
    want_q = np.clip(np.rint(z), -127, 127).astype(np.int8)
    assert np.array_equal(q, want_q)
