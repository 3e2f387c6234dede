"""Pins for the oracle's 1:2 functions (the TF32 mode of Section 3.2 / Table 1): brute force over
pairs, round trips, the nibble codes, GEMM against numpy float64 matmul, operand-order bijection."""
import numpy as np

import oracle
from paper_2104_08378_b200 import inputs


def _f32(bits):
    return bits.view(np.float32).astype(np.float64)


def _rand(M, K, seed):
    return inputs._matrix(("normal", 1.0), "tf32", seed, 5, K, 0, M)


def test_inputs_are_tf32_representable():
    x = _rand(8, 64, 1)
    assert x.dtype == np.uint32 and (x & 0x1FFF).max() == 0


def test_pairs_brute_force_and_codes():
    vals = np.array([0.0, -0.0, 1.0, -1.0, 2.0, -2.0, 1e-40, 3.5], dtype=np.float32)
    pairs = np.array([(a, b) for a in vals for b in vals], dtype=np.float32)          # 64 pairs
    x = np.ascontiguousarray(pairs.reshape(8, 16)).view(np.uint32)
    y = oracle.prune_1of2(x)
    v, m, dropped = oracle.compress_1of2(x)
    nib = np.stack([m & 0xF, m >> 4], axis=2).reshape(8, 8)
    xf = np.abs(_f32(x)).reshape(8, 8, 2)
    for i in range(8):
        for g in range(8):
            a, b = xf[i, g]
            second = b > a                                   # tie -> first (independent statement of the rule)
            assert nib[i, g] == (0xE if second else 0x4)
            assert v[i, g] == x[i, 2 * g + int(second)]
            assert y[i, 2 * g + int(not second)] == 0 and y[i, 2 * g + int(second)] == x[i, 2 * g + int(second)]
    assert dropped == int(((x & 0x7FFFFFFF) != 0).sum() - ((y & 0x7FFFFFFF) != 0).sum())
    assert np.array_equal(oracle.decompress_1of2(v, m), y)
    assert np.array_equal(oracle.prune_1of2(y), y)
    assert ((y.reshape(8, 8, 2) != 0).sum(axis=2) <= 1).all()      # at least one zero per pair
    assert v.nbytes == x.nbytes // 2 and m.nbytes * 8 == 4 * v.size  # 4 metadata bits per kept value


def test_gemm_1of2_against_numpy_and_closed_forms():
    M, N, K = 12, 10, 64
    x, Bt = _rand(M, K, 2), _rand(N, K, 3)
    v, m, _ = oracle.compress_1of2(x)
    D, mag = oracle.gemm_sparse_1of2(v, m, Bt)
    pruned = _f32(oracle.decompress_1of2(v, m))
    ref = pruned @ _f32(Bt).T
    assert np.all(np.abs(D - ref) <= 1e-13 * (np.abs(pruned) @ np.abs(_f32(Bt)).T) + 1e-300)
    assert np.allclose(mag, np.abs(pruned) @ np.abs(_f32(Bt)).T, rtol=1e-13)
    eye = np.eye(K, dtype=np.float32).view(np.uint32)
    De, _ = oracle.gemm_sparse_1of2(v, m, np.ascontiguousarray(eye))
    assert np.array_equal(De, pruned)                              # B = I gives decompress(A)
    C = np.arange(M * N, dtype=np.float32).reshape(M, N)
    Dc, _ = oracle.gemm_sparse_1of2(v, m, Bt, alpha=0.5, beta=-2.0, C=C)
    assert np.array_equal(Dc, 0.5 * D - 2.0 * C)
    sub, _ = oracle.gemm_sparse_1of2(v, m, Bt, rows=(3, 7), cols=(2, 9))
    assert np.array_equal(sub, D[3:7, 2:9])


def test_operand_order_1of2_matches_the_16bit_nibble_placement():
    M, K = 200, 320                                                # ragged in M, K padded to 384
    x = _rand(M, K, 4)
    _, m, _ = oracle.compress_1of2(x)
    buf = oracle.meta_to_operand_order_1of2(m)
    assert buf.size == 2 * 6 * 2048
    assert np.array_equal(oracle.meta_from_operand_order_1of2(buf, M, K), m)
    assert set(np.unique(np.concatenate([buf & 0xF, buf >> 4])).tolist()) <= {0x4, 0xE}
    # same placement rule as a 16-bit matrix with twice the columns (a nibble = one pair = one group of four)
    fake = np.ascontiguousarray(m)                                  # M x K/4 bytes == canonical 16-bit meta of M x 2K
    assert np.array_equal(buf, oracle.meta_to_operand_order(fake, "bf16"))
