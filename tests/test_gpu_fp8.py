"""GPU parity of the 8-bit floating-point operand types (e4m3, e5m2).  The paper's Table 1 has no
8-bit floating-point row; the types reuse the 2:4 pattern, the compressed format of the 8-bit
integer row (Section 3.1) and the GEMM of Section 3.2 with FP32 accumulation.  prune / compress /
decompress are compared bit for bit, the GEMM within the floating-point tolerance of the other
GEMM tests."""
import numpy as np
import pytest
import torch

import oracle
from paper_2104_08378_b200 import inputs
from test_gpu_gemm import check_fp

pytestmark = pytest.mark.gpu

TORCH_F8 = {"e4m3": torch.float8_e4m3fn, "e5m2": torch.float8_e5m2}


@pytest.fixture(scope="module")
def sp():
    from paper_2104_08378_b200 import binding
    return binding


def _dev(bits, dtype):
    return torch.from_numpy(bits).cuda().view(TORCH_F8[dtype])


def _host(t):
    return t.view(torch.uint8).cpu().numpy()


def _rand(M, K, dtype, seed, dist=("normal", 1.0), tensor=5):
    return inputs._matrix(dist, dtype, seed, tensor, K, 0, M)


@pytest.mark.parametrize("dtype", ["e4m3", "e5m2"])
@pytest.mark.parametrize("shape", [(128, 256), (200, 336), (37, 96), (1, 8), (513, 1040)])
@pytest.mark.parametrize("layout", [0, 1])
def test_prune_compress_decompress_fp8(sp, dtype, shape, layout):
    M, K = shape
    x = _rand(M, K, dtype, 1)
    x[::3, ::5] = 0
    x[1::4, 1::2] = x[1::4, 0::2] ^ 0x80          # equal magnitudes, opposite signs: ties
    x[2::7, 3::4] = 0x80                           # negative zeros rank as zeros
    xd = _dev(x, dtype)
    assert np.array_equal(_host(sp.prune(xd)), oracle.prune(x, dtype))
    v_ref, m_ref, d_ref = oracle.compress(x, dtype)
    vals, meta, dropped = sp.compress(xd, layout=layout, count_dropped=True)
    assert np.array_equal(_host(vals), v_ref)
    expect = m_ref.ravel() if layout == 0 else oracle.meta_to_operand_order(m_ref, dtype)
    assert np.array_equal(meta.cpu().numpy(), expect)
    assert int(dropped.item()) == d_ref
    assert np.array_equal(_host(sp.decompress(vals, meta, layout=layout)), oracle.prune(x, dtype))


@pytest.mark.parametrize("dtype", ["e4m3", "e5m2"])
def test_every_bit_pattern_and_the_scalar_path(sp, dtype):
    """All 256 encodings (NaN and, for e5m2, infinity patterns included: they rank by their bits) in
    every position of a group, through the vector kernels and -- with an odd leading dimension -- the
    element-wise ones."""
    rng = np.random.default_rng(3)
    x = rng.integers(0, 256, size=(256, 512), dtype=np.uint8)
    x[0, :256] = np.arange(256, dtype=np.uint8)
    for ld in (512, 520 + 3):
        buf = torch.zeros(256, ld, dtype=torch.uint8, device="cuda")
        buf[:, :512] = torch.from_numpy(x).cuda()
        xd = buf.view(TORCH_F8[dtype])[:, :512]
        assert np.array_equal(_host(sp.prune(xd)), oracle.prune(x, dtype))
        v_ref, m_ref, d_ref = oracle.compress(x, dtype)
        vals, meta, dropped = sp.compress(xd, layout=0, count_dropped=True)
        assert np.array_equal(_host(vals), v_ref)
        assert np.array_equal(meta.cpu().numpy(), m_ref.ravel())
        assert int(dropped.item()) == d_ref


@pytest.mark.parametrize("dtype", ["e4m3", "e5m2"])
@pytest.mark.parametrize("dense", [False, True])
@pytest.mark.parametrize("shape", [(128, 128, 256), (32, 32, 32), (160, 288, 416), (384, 640, 2048), (1024, 2240, 512)])
def test_fp8_gemm(sp, dtype, dense, shape):
    M, N, K = shape
    A = _rand(M, K, dtype, 7)
    Bt = _rand(N, K, dtype, 8, ("uniform", -1.0, 1.0), tensor=6)
    Cm = inputs._matrix(("normal", 1.0), "bf16", 9, 7, N, 0, M)
    v_ref, m_ref, _ = oracle.compress(A, dtype)
    scale = oracle.gemm_abs(v_ref, m_ref, Bt, dtype)
    Ad, Btd = _dev(A, dtype), _dev(Bt, dtype)
    Cd = torch.from_numpy(Cm.view(np.int16)).cuda().view(torch.bfloat16)
    for cd, alpha, beta in (("bf16", 1.0, 0.0), ("bf16", 0.5, -2.0), ("f32", 1.0, 0.0), ("f16", 2.0, 0.0)):
        C_arg = Cd if beta else None
        if dense:
            D = sp.gemm(sp.prune(Ad), None, Btd, alpha=alpha, beta=beta, C=C_arg, cd=cd, a_is_dense=True)
        else:
            vals, meta, _ = sp.compress(Ad, layout=sp.META_TCGEN05)
            D = sp.gemm(vals, meta, Btd, alpha=alpha, beta=beta, C=C_arg, cd=cd)
        torch.cuda.synchronize()
        assert sp.gemm_status(device=D.device) == 0
        ref = oracle.gemm_sparse(v_ref, m_ref, Bt, dtype, alpha, beta, Cm if beta else None, "bf16" if beta else None)
        beta_c = abs(beta) * np.abs(oracle.bits_to_float64(Cm, "bf16")) if beta else None
        check_fp(D.to(torch.float64).cpu().numpy(), ref, abs(alpha) * scale, beta_c)


@pytest.mark.parametrize("dtype", ["e4m3", "e5m2"])
@pytest.mark.parametrize("dense", [False, True])
@pytest.mark.parametrize("shape", [(128, 128, 128), (160, 288, 416), (512, 1344, 1024)])
def test_fp8_b_stored_n_contiguous(sp, dtype, dense, shape):
    """order_b = ROW_MAJOR for the 8-bit floats: the K x N matrix stored row by row (MN-major operand)."""
    M, N, K = shape
    A = _rand(M, K, dtype, 17)
    Bt = _rand(N, K, dtype, 18, ("uniform", -1.0, 1.0), tensor=6)
    v_ref, m_ref, _ = oracle.compress(A, dtype)
    Ad = _dev(A, dtype)
    Bkn = _dev(np.ascontiguousarray(Bt.T), dtype)                 # [K, N], N contiguous
    if dense:
        D = sp.gemm(sp.prune(Ad), None, Bkn, cd="f32", a_is_dense=True, b_row_major=True)
    else:
        vals, meta, _ = sp.compress(Ad, layout=sp.META_TCGEN05)
        D = sp.gemm(vals, meta, Bkn, cd="f32", b_row_major=True)
    torch.cuda.synchronize()
    assert sp.gemm_status(device=D.device) == 0
    ref = oracle.gemm_sparse(v_ref, m_ref, Bt, dtype)
    check_fp(D.to(torch.float64).cpu().numpy(), ref, oracle.gemm_abs(v_ref, m_ref, Bt, dtype))


def test_fp8_rejections(sp):
    A = torch.zeros(128, 64, dtype=torch.uint8, device="cuda").view(torch.float8_e4m3fn)
    Bt = torch.zeros(128, 128, dtype=torch.uint8, device="cuda").view(torch.float8_e4m3fn)
    meta = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    with pytest.raises(RuntimeError):      # the accumulator is fp32: no integer output
        sp.gemm(A, meta, Bt, cd="i32")
    with pytest.raises(RuntimeError):      # magnitude sums are defined for the paper's types only
        sp.kept_magnitude(torch.zeros(128, 128, dtype=torch.uint8, device="cuda").view(torch.float8_e4m3fn))
