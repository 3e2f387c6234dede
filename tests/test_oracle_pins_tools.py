"""Pins for the oracle's pruning tools: kept magnitude under permutations (Section 4.1), the fixed
mask of retraining (Section 4.1 step 3) and the row-and-column pattern of Section 6."""
import itertools

import numpy as np
import pytest

import oracle
from paper_2104_08378_b200 import inputs

DTYPES = ["f16", "bf16", "i8"]


def _rand(dtype, M, K, seed):
    return inputs._matrix(("int8",) if dtype == "i8" else ("normal", 1.0), dtype, seed, 3, K, 0, M)


def _mag(x, dtype):
    return np.abs(oracle.bits_to_float64(x, dtype))


@pytest.mark.parametrize("dtype", DTYPES)
def test_kept_magnitude_identity_and_permutation(dtype):
    x = _rand(dtype, 20, 64, 1)
    total = oracle.kept_magnitude(x, dtype)
    assert np.isclose(total, _mag(oracle.prune(x, dtype), dtype).sum(), rtol=1e-13)
    perm = np.random.default_rng(0).permutation(64)
    xp = np.ascontiguousarray(x[:, perm])                       # the permuted matrix, pruned as it stands
    assert np.isclose(oracle.kept_magnitude(x, dtype, perm), _mag(oracle.prune(xp, dtype), dtype).sum(), rtol=1e-13)
    # spreading the large values over the groups keeps more (the effect the paper's Figure 6 shows)
    row = inputs.to_storage(np.array([[9, 8, 7, 6, 0, 0, 0, 0]], dtype=np.float64), dtype)
    assert oracle.kept_magnitude(row, dtype) == 17.0
    assert oracle.kept_magnitude(row, dtype, [0, 1, 4, 5, 2, 3, 6, 7]) == 30.0


@pytest.mark.parametrize("dtype", DTYPES)
def test_apply_mask_keeps_the_pattern_not_the_values(dtype):
    x, w = _rand(dtype, 9, 40, 2), _rand(dtype, 9, 40, 3)
    _, meta, _ = oracle.compress(x, dtype)
    y = oracle.apply_mask(w, meta, dtype)
    kept = oracle.apply_mask(np.full_like(x, 1), meta, dtype) != 0      # the pattern itself
    assert (kept.reshape(9, 10, 4).sum(axis=2) == 2).all()
    assert np.array_equal(y[kept], w[kept]) and (y[~kept] == 0).all()
    assert np.array_equal(oracle.apply_mask(x, meta, dtype), oracle.prune(x, dtype))   # on x itself it is prune


def _valid_patterns():
    pats = []
    for mask in range(1 << 16):
        rows = [(mask >> (4 * i)) & 0xF for i in range(4)]
        if all(bin(r).count("1") == 2 for r in rows) and all(sum((r >> j) & 1 for r in rows) == 2 for j in range(4)):
            pats.append(np.array([[(r >> j) & 1 for j in range(4)] for r in rows], dtype=bool))
    return pats


@pytest.mark.parametrize("dtype", DTYPES)
def test_prune_2d_is_two_per_row_and_column_and_optimal(dtype):
    pats = _valid_patterns()
    assert len(pats) == 90
    x = _rand(dtype, 16, 24, 4)
    y = oracle.prune_2d(x, dtype)
    mag, kept = _mag(x, dtype), None
    for bi, bj in itertools.product(range(4), range(6)):
        blk = y[4 * bi:4 * bi + 4, 4 * bj:4 * bj + 4]
        src = x[4 * bi:4 * bi + 4, 4 * bj:4 * bj + 4]
        m = mag[4 * bi:4 * bi + 4, 4 * bj:4 * bj + 4]
        keep = blk != 0
        zero_src = src == 0
        assert np.array_equal(blk[keep], src[keep])
        # pattern validity (zeros in the source may hide kept positions, so test on the source's support)
        assert ((keep | zero_src).sum(axis=0) >= 2).all() and (keep.sum(axis=0) <= 2).all()
        assert (keep.sum(axis=1) <= 2).all()
        best = max(m[p].sum() for p in pats)                       # brute force over all 90 in float64
        assert m[keep].sum() >= best * (1 - 1e-6)
    # the transposed result is 2:4 along ITS rows as well: pruning it again changes nothing
    assert np.array_equal(oracle.prune(np.ascontiguousarray(y.T), dtype), np.ascontiguousarray(y.T))
    assert np.array_equal(oracle.prune(y, dtype), y)


def test_prune_2d_tie_takes_the_first_pattern():
    ones = inputs.to_storage(np.ones((4, 4)), "bf16")
    y = oracle.prune_2d(ones, "bf16") != 0
    # first candidate in lexicographic order of row pairs: rows 0,1 keep columns (0,1), rows 2,3 keep (2,3)
    assert np.array_equal(y, np.array([[1, 1, 0, 0], [1, 1, 0, 0], [0, 0, 1, 1], [0, 0, 1, 1]], dtype=bool))
