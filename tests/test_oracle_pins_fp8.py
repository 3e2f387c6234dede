"""Pins of the oracle's 8-bit floating-point support against things other than itself: the decoding
against a library conversion, the selection against brute force over keep patterns computed from
the decoded VALUES (the oracle ranks bit patterns), the format invariants of Section 3.1 and the
GEMM against a library matmul on the decoded, pruned matrix."""
import itertools

import numpy as np
import pytest
import torch

import oracle
from paper_2104_08378_b200 import inputs

TORCH_F8 = {"e4m3": torch.float8_e4m3fn, "e5m2": torch.float8_e5m2}


@pytest.mark.parametrize("dtype", ["e4m3", "e5m2"])
def test_decoding_matches_library_conversion_for_all_256_patterns(dtype):
    bits = np.arange(256, dtype=np.uint8)
    mine = oracle.bits_to_float64(bits, dtype)
    lib = torch.from_numpy(bits).view(TORCH_F8[dtype]).to(torch.float64).numpy()
    assert np.array_equal(np.isnan(mine), np.isnan(lib))
    ok = ~np.isnan(lib)
    assert np.array_equal(mine[ok], lib[ok])
    assert np.array_equal(np.signbit(mine[ok]), np.signbit(lib[ok]))


@pytest.mark.parametrize("dtype", ["e4m3", "e5m2"])
def test_input_rounding_matches_library_conversion(dtype):
    rng = np.random.default_rng(0)
    limit = 448.0 if dtype == "e4m3" else 57344.0
    v = np.concatenate([rng.normal(0, 1, 3000), rng.normal(0, 40, 1000), rng.uniform(-2e-2, 2e-2, 2000),
                        [0.0, -0.0, limit, -limit, 2.0 ** -9, 2.0 ** -10, 3 * 2.0 ** -10, 2.0 ** -16, 2.0 ** -17]])
    v = v[np.abs(v) <= limit]
    mine = inputs.to_storage(v, dtype)
    lib = torch.from_numpy(v).to(TORCH_F8[dtype]).view(torch.uint8).numpy()
    assert np.array_equal(mine, lib)


@pytest.mark.parametrize("dtype", ["e4m3", "e5m2"])
def test_selection_equals_brute_force_on_decoded_magnitudes(dtype):
    """Every group over a small alphabet of finite encodings: the kept pair maximises the kept
    |value| sum, ties go to the lexicographically smallest pair of positions (Section 4.1 step 2)."""
    alphabet = np.array([0x00, 0x80, 0x01, 0x81, 0x38, 0xB8, 0x3C, 0x45, 0xC5], dtype=np.uint8)
    groups = np.array(list(itertools.product(alphabet, repeat=4)), dtype=np.uint8)       # 6561 groups
    x = np.ascontiguousarray(np.concatenate([groups, groups], axis=1))                    # K = 8
    mag = np.abs(oracle.bits_to_float64(groups, dtype))
    pruned = oracle.prune(x, dtype)[:, :4]
    for row in range(0, groups.shape[0], 7):
        best, best_pair = -1.0, None
        for pair in itertools.combinations(range(4), 2):
            s = mag[row, pair[0]] + mag[row, pair[1]]
            if s > best:
                best, best_pair = s, pair
        expect = np.zeros(4, dtype=np.uint8)
        expect[list(best_pair)] = groups[row, list(best_pair)]
        assert np.array_equal(pruned[row], expect), (row, groups[row])


@pytest.mark.parametrize("dtype", ["e4m3", "e5m2"])
def test_format_invariants_and_gemm_against_library_matmul(dtype):
    M, N, K = 48, 40, 96
    A = inputs._matrix(("normal", 1.0), dtype, 11, 5, K, 0, M)
    Bt = inputs._matrix(("uniform", -1.0, 1.0), dtype, 12, 6, K, 0, N)
    A[::5, ::3] = 0
    pruned = oracle.prune(A, dtype)
    assert ((pruned.reshape(M, K // 4, 4) & 0x7F) != 0).sum(axis=2).max() <= 2
    assert np.array_equal(oracle.prune(pruned, dtype), pruned)
    vals, meta, dropped = oracle.compress(A, dtype)
    assert vals.shape == (M, K // 2) and meta.shape == (M, K // 8)
    assert set(np.unique(np.concatenate([meta & 0xF, meta >> 4]))) <= {0x4, 0x8, 0x9, 0xC, 0xD, 0xE}
    assert np.array_equal(oracle.decompress(vals, meta, dtype), pruned)
    assert np.array_equal(oracle.compress(pruned, dtype)[0], vals)
    assert dropped == int((((A & 0x7F) != 0) & ((pruned & 0x7F) == 0)).sum())
    # 8-bit types share the operand order of the 8-bit integer row: one row of a 128-column block = 16 bytes
    assert np.array_equal(oracle.meta_to_operand_order(meta, dtype),
                          oracle.meta_to_operand_order(meta, "i8"))
    lib = torch.from_numpy(pruned).view(TORCH_F8[dtype]).to(torch.float64) @ \
        torch.from_numpy(Bt).view(TORCH_F8[dtype]).to(torch.float64).T
    ref = oracle.gemm_sparse(vals, meta, Bt, dtype)
    assert np.allclose(ref, lib.numpy(), rtol=1e-13, atol=1e-13)
    assert np.array_equal(oracle.gemm_dense(pruned, Bt, dtype), ref)
