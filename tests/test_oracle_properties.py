"""Property tests of the oracle over random shapes and contents (hypothesis): the invariants the
paper fixes must hold for every input, not only for the seeded matrices of the other pin files.

* Section 3 / 4.1: every aligned group of four in prune(x) has at least two zeros, kept values are
  the inputs bit for bit, pruning is idempotent and never keeps a smaller magnitude than it drops.
* Section 3.1: decompress(compress(x)) == prune(x); the values are M x K/2, the metadata K/8 bytes
  per row with valid codes only; the operand-order permutation is a bijection.
* Section 3.2: the sparse GEMM on the compressed operand equals a library matmul on the pruned matrix.
"""
import numpy as np
from hypothesis import given, settings, strategies as st

import oracle

DTYPES = ["f16", "bf16", "i8", "e4m3", "e5m2"]
VALID = {0x4, 0x8, 0x9, 0xC, 0xD, 0xE}


def _storage(dtype):
    return {"i8": np.int8, "e4m3": np.uint8, "e5m2": np.uint8}.get(dtype, np.uint16)


def _finite(x, dtype):
    """Replace NaN / infinity encodings by zeros (the GEMM properties use finite inputs)."""
    if dtype == "i8":
        return x
    with np.errstate(invalid="ignore"):
        v = oracle.bits_to_float64(x, dtype)
    x = x.copy()
    x[~np.isfinite(v)] = 0
    return x


@st.composite
def matrices(draw, max_rows=24, max_groups=12):
    dtype = draw(st.sampled_from(DTYPES))
    M = draw(st.integers(1, max_rows))
    K = 8 * draw(st.integers(1, max_groups))
    seed = draw(st.integers(0, 2 ** 31 - 1))
    rng = np.random.default_rng(seed)
    store = _storage(dtype)
    bits = np.iinfo(store).bits
    x = rng.integers(0, 2 ** bits, size=(M, K), dtype=np.uint64).astype(np.uint16 if bits == 16 else np.uint8).view(store)
    sparsity = draw(st.sampled_from([0.0, 0.3, 0.8]))
    x[rng.random((M, K)) < sparsity] = 0
    if draw(st.booleans()):                      # a small alphabet makes ties frequent
        alphabet = rng.integers(0, 2 ** bits, size=3, dtype=np.uint64).astype(x.view(np.uint16 if bits == 16 else np.uint8).dtype)
        x = alphabet[rng.integers(0, 3, size=(M, K))].view(store)
    return dtype, np.ascontiguousarray(x)


def _keys(x, dtype):
    if dtype == "i8":
        return np.abs(x.astype(np.int32))
    u = x.view(np.uint16 if x.dtype.itemsize == 2 else np.uint8).astype(np.int32)
    return u & (0x7FFF if x.dtype.itemsize == 2 else 0x7F)


@settings(max_examples=60, deadline=None)
@given(matrices())
def test_prune_invariants(case):
    dtype, x = case
    y = oracle.prune(x, dtype)
    kx, ky = _keys(x, dtype).reshape(x.shape[0], -1, 4), _keys(y, dtype).reshape(x.shape[0], -1, 4)
    raw_x, raw_y = x.reshape(x.shape[0], -1, 4), y.reshape(x.shape[0], -1, 4)
    assert ((ky != 0).sum(axis=2) <= 2).all()                         # the 2:4 pattern
    # every output element is the input bit for bit or the all-zero pattern
    assert ((raw_y == raw_x) | (raw_y.view(np.uint8 if x.dtype.itemsize == 1 else np.uint16) == 0)).all()
    # nothing dropped is larger than anything kept: min kept key >= max dropped key in every group
    dropped_max = np.where(ky == 0, kx, 0).max(axis=2)
    kept_keys = np.where(ky != 0, ky, np.iinfo(np.int32).max)
    enough = (ky != 0).sum(axis=2) == 2
    assert (kept_keys.min(axis=2)[enough] >= dropped_max[enough]).all()
    assert np.array_equal(oracle.prune(y, dtype), y)                  # idempotent


@settings(max_examples=60, deadline=None)
@given(matrices())
def test_format_round_trip_and_operand_order(case):
    dtype, x = case
    M, K = x.shape
    vals, meta, dropped = oracle.compress(x, dtype)
    assert vals.shape == (M, K // 2) and meta.shape == (M, K // 8) and meta.dtype == np.uint8
    assert set(np.unique(np.concatenate([(meta & 0xF).ravel(), (meta >> 4).ravel()]))) <= VALID
    pruned = oracle.prune(x, dtype)
    assert np.array_equal(oracle.decompress(vals, meta, dtype), pruned)
    assert dropped == int(((_keys(x, dtype) != 0) & (_keys(pruned, dtype) == 0)).sum())
    assert oracle.compress(pruned, dtype)[2] == 0
    packed = oracle.meta_to_operand_order(meta, dtype)
    assert np.array_equal(oracle.meta_from_operand_order(packed, M, K, dtype), meta)
    # every padding nibble of the operand order is the code of positions (0, 1)
    assert (np.bincount(np.concatenate([packed & 0xF, packed >> 4]), minlength=16)[list(set(range(16)) - VALID)] == 0).all()


@settings(max_examples=40, deadline=None)
@given(matrices(max_rows=12, max_groups=6), st.integers(1, 9))
def test_sparse_gemm_equals_library_matmul_on_the_pruned_matrix(case, N):
    dtype, x = case
    x = _finite(x, dtype)
    rng = np.random.default_rng(N)
    K = x.shape[1]
    bt_vals = rng.integers(-3, 4, size=(N, K))
    Bt = bt_vals.astype(np.int8) if dtype == "i8" else _encode_small_ints(bt_vals, dtype)
    vals, meta, _ = oracle.compress(x, dtype)
    got = oracle.gemm_sparse(vals, meta, Bt, dtype)
    with np.errstate(invalid="ignore"):
        a = oracle.bits_to_float64(oracle.prune(x, dtype), dtype)
    want = a @ bt_vals.astype(np.float64).T
    if dtype == "i8":
        assert np.array_equal(got, want.astype(np.int64).astype(np.int32))
    else:
        # the two sides add in different orders: the bound is relative to the sum of magnitudes
        bound = 1e-13 * (np.abs(a) @ np.abs(bt_vals).astype(np.float64).T) + 1e-300
        assert (np.abs(got - want) <= bound).all()


def _encode_small_ints(v, dtype):
    """Integers -3..3 in a floating-point storage type (exactly representable in all of them)."""
    table = {}
    for n in range(-3, 4):
        if dtype == "f16":
            table[n] = np.float16(n).view(np.uint16)
        elif dtype == "bf16":
            table[n] = np.uint16(np.float32(n).view(np.uint32) >> 16)
        else:
            pats = np.arange(256, dtype=np.uint8)
            dec = oracle.bits_to_float64(pats, dtype)
            cand = pats[(dec == n) & ~np.signbit(dec)] if n >= 0 else pats[dec == n]
            table[n] = cand[0]
    out = np.vectorize(lambda n: table[int(n)])(v)
    return np.ascontiguousarray(out.astype(np.uint16 if dtype in ("f16", "bf16") else np.uint8))
