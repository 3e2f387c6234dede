"""GPU parity of the 1:2 / TF32 path (Section 3.2, Table 1): prune, compress, decompress bit-exact;
sparse and dense kind::tf32 GEMM within the floating-point tolerance of the other GEMM tests."""
import numpy as np
import pytest
import torch

import oracle
from paper_2104_08378_b200 import inputs
from test_gpu_gemm import check_fp

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def sp():
    from paper_2104_08378_b200 import binding
    return binding


def _dev(bits):
    return torch.from_numpy(bits.view(np.int32)).cuda().view(torch.float32)


def _host(t):
    return t.view(torch.int32).cpu().numpy().view(np.uint32)


def _rand(M, K, seed, dist=("normal", 1.0)):
    return inputs._matrix(dist, "tf32", seed, 5, K, 0, M)


@pytest.mark.parametrize("shape", [(128, 128), (200, 328), (37, 96), (1, 8), (513, 1032)])
@pytest.mark.parametrize("layout", [0, 1])
def test_prune_compress_decompress_1of2(sp, shape, layout):
    M, K = shape
    x = _rand(M, K, 1)
    x[::3, ::5] = 0
    x[1::4, 1::2] = x[1::4, 0::2] ^ 0x80000000                     # equal magnitudes, opposite signs: ties
    xd = _dev(x)
    assert np.array_equal(_host(sp.prune(xd)), oracle.prune_1of2(x))
    v_ref, m_ref, d_ref = oracle.compress_1of2(x)
    vals, meta, dropped = sp.compress(xd, layout=layout, count_dropped=True)
    assert np.array_equal(_host(vals), v_ref)
    expect = m_ref.ravel() if layout == 0 else oracle.meta_to_operand_order_1of2(m_ref)
    assert np.array_equal(meta.cpu().numpy(), expect)
    assert int(dropped.item()) == d_ref
    assert np.array_equal(_host(sp.decompress(vals, meta, layout=layout)), oracle.prune_1of2(x))


@pytest.mark.parametrize("dense", [False, True])
@pytest.mark.parametrize("shape", [(128, 128, 64), (16, 16, 16), (144, 272, 208), (384, 640, 1024), (1024, 2240, 512)])
def test_tf32_gemm(sp, dense, shape):
    M, N, K = shape
    A, Bt = _rand(M, K, 7), _rand(N, K, 8, ("uniform", -1.0, 1.0))
    Cm = np.ascontiguousarray(_rand(M, N, 9).view(np.float32))
    v_ref, m_ref, _ = oracle.compress_1of2(A)
    Ad, Btd, Cd = _dev(A), _dev(Bt), torch.from_numpy(Cm).cuda()
    for alpha, beta in ((1.0, 0.0), (0.5, -2.0)):
        if dense:
            D = sp.gemm(sp.prune(Ad), None, Btd, alpha=alpha, beta=beta, C=Cd if beta else None, a_is_dense=True)
        else:
            vals, meta, _ = sp.compress(Ad)
            D = sp.gemm(vals, meta, Btd, alpha=alpha, beta=beta, C=Cd if beta else None)
        torch.cuda.synchronize()
        assert sp.gemm_status(device=D.device) == 0
        rows, cols = (0, min(M, 256)), (max(0, N - 320), N)
        ref, mag = oracle.gemm_sparse_1of2(v_ref, m_ref, Bt, alpha, beta, Cm if beta else None, rows=rows, cols=cols)
        got = D[rows[0]:rows[1], cols[0]:cols[1]].double().cpu().numpy()
        beta_c = abs(beta) * np.abs(Cm[rows[0]:rows[1], cols[0]:cols[1]]) if beta else None
        check_fp(got, ref, abs(alpha) * mag, beta_c)


@pytest.mark.parametrize("dense", [False, True])
@pytest.mark.parametrize("shape", [(128, 128, 64), (144, 272, 208), (512, 1344, 512)])
def test_tf32_b_stored_n_contiguous(sp, dense, shape):
    """order_b = ROW_MAJOR in the TF32 mode: the K x N matrix stored row by row (MN-major operand, which for
    32-bit elements exists only in the 128-byte swizzle with 32-byte units)."""
    M, N, K = shape
    A, Bt = _rand(M, K, 27), _rand(N, K, 28, ("uniform", -1.0, 1.0))
    v_ref, m_ref, _ = oracle.compress_1of2(A)
    Ad, Bkn = _dev(A), _dev(np.ascontiguousarray(Bt.T))          # [K, N], N contiguous
    if dense:
        D = sp.gemm(sp.prune(Ad), None, Bkn, a_is_dense=True, b_row_major=True)
    else:
        vals, meta, _ = sp.compress(Ad)
        D = sp.gemm(vals, meta, Bkn, b_row_major=True)
    torch.cuda.synchronize()
    assert sp.gemm_status(device=D.device) == 0
    ref, mag = oracle.gemm_sparse_1of2(v_ref, m_ref, Bt)
    check_fp(D.double().cpu().numpy(), ref, mag)


def test_tf32_identity_b_is_exact(sp):
    M, K = 256, 192
    A = _rand(M, K, 11)
    eye = np.ascontiguousarray(np.eye(K, dtype=np.float32).view(np.uint32))
    vals, meta, _ = sp.compress(_dev(A))
    D = sp.gemm(vals, meta, _dev(eye))
    torch.cuda.synchronize()
    # every selected index exercised, values exact (compared as numbers: a sum of signed zeros may be -0)
    assert np.array_equal(D.cpu().numpy(), oracle.prune_1of2(A).view(np.float32))
