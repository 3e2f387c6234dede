"""The FP16-accumulation mode of Table 1 (FP16 operands, FP16 accumulator): sp24_gemm_f16acc.

The oracle stays the exact FP64 product.  What changes is the error model: the tensor cores round the
running sum to binary16 after every instruction (32 values of K per sparse instruction, 16 per dense
one), each rounding at most 2^-10 of the magnitude of the sum so far (truncation assumed; round to
nearest would be 2^-11), and no partial sum exceeds (|A|.|B|)_ij.  So
    |err_ij| <= (n_instr + 2) * 2^-10 * (|A|.|B|)_ij,   n_instr = K/32 (sparse) or K/16 (dense),
the +2 covering alpha and the output rounding.  Where every partial sum is a small integer the mode
must be exact, which pins the reading of the 16-bit accumulator cells."""
import numpy as np
import pytest
import torch

import oracle
from paper_2104_08378_b200 import inputs
from gpu_util import to_device, to_host_f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def sp():
    from paper_2104_08378_b200 import binding
    return binding


def _bound(K, dense, scale):
    n_instr = K // (16 if dense else 32)
    return (n_instr + 2) * 2.0 ** -10 * scale + 1e-30


@pytest.mark.parametrize("dense", [False, True])
@pytest.mark.parametrize("tile", [None, "2x224x1", "2x224x2"])
@pytest.mark.parametrize("shape", [(256, 256, 512, "f16"), (528, 720, 2048, "f32")])
def test_f16_accumulate_within_its_error_model(sp, force_tile, dense, tile, shape):
    M, N, K, cd = shape
    cfg = inputs.scaled(inputs.CONFIGS["tiny_f16"], M=M, N=N, K=K)
    A, Bt = inputs.gen_A(cfg), inputs.gen_Bt(cfg)
    Cm = inputs._matrix(("normal", 1.0), cd, 5, 7, N, 0, M) if cd == "f16" else \
        np.random.default_rng(5).standard_normal((M, N)).astype(np.float32)
    v_ref, m_ref, _ = oracle.compress(A, "f16")
    Ad, Btd = to_device(A, "f16"), to_device(Bt, "f16")
    Cd = to_device(Cm, cd)
    vals, meta, _ = sp.compress(Ad)
    pruned = sp.prune(Ad)
    force_tile(tile)
    for alpha, beta in ((1.0, 0.0), (0.5, -1.5)):
        D = sp.gemm(pruned if dense else vals, None if dense else meta, Btd, alpha=alpha, beta=beta,
                    C=Cd if beta else None, cd=cd, a_is_dense=dense, acc_f16=True)
        torch.cuda.synchronize()
        assert sp.gemm_status(device=D.device) == 0
        ref = oracle.gemm_sparse(v_ref, m_ref, Bt, "f16", alpha, beta, Cm if beta else None, cd if beta else None)
        scale = abs(alpha) * oracle.gemm_abs(v_ref, m_ref, Bt, "f16")
        if beta:
            scale = scale + abs(beta) * np.abs(oracle.bits_to_float64(Cm, cd) if cd == "f16" else Cm.astype(np.float64))
        err = np.abs(to_host_f64(D) - ref)
        assert (err <= _bound(K, dense, scale)).all(), float((err / _bound(K, dense, scale)).max())
        # typical size: the roundings add up like a random walk, far below the worst case
        assert np.linalg.norm(err) / np.linalg.norm(ref) <= 2.0 ** -10 * np.sqrt(K / 16 + 2) * 2


def test_f16_accumulate_is_exact_on_small_integers_and_differs_from_fp32_accumulation(sp):
    rng = np.random.default_rng(9)
    M, N, K = 256, 256, 256
    A = inputs.to_storage(rng.integers(-2, 3, size=(M, K)).astype(np.float64), "f16")
    Bt = inputs.to_storage(rng.integers(-2, 3, size=(N, K)).astype(np.float64), "f16")
    v_ref, m_ref, _ = oracle.compress(A, "f16")
    vals, meta, _ = sp.compress(to_device(A, "f16"))
    D = sp.gemm(vals, meta, to_device(Bt, "f16"), cd="f32", acc_f16=True)
    torch.cuda.synchronize()
    # |partial sums| <= 4 * 128: integers that binary16 holds exactly
    assert np.array_equal(to_host_f64(D), oracle.gemm_sparse(v_ref, m_ref, Bt, "f16"))
    # at large K with real-valued inputs the binary16 accumulator is visible in the result
    cfg = inputs.scaled(inputs.CONFIGS["tiny_f16"], M=256, N=256, K=8192)
    A, Bt = inputs.gen_A(cfg), inputs.gen_Bt(cfg)
    vals, meta, _ = sp.compress(to_device(A, "f16"))
    Btd = to_device(Bt, "f16")
    D16 = sp.gemm(vals, meta, Btd, cd="f32", acc_f16=True)
    D32 = sp.gemm(vals, meta, Btd, cd="f32")
    torch.cuda.synchronize()
    assert not torch.equal(D16, D32)
    v_ref, m_ref, _ = oracle.compress(A, "f16")
    ref = oracle.gemm_sparse(v_ref, m_ref, Bt, "f16")
    e16 = np.linalg.norm(to_host_f64(D16) - ref) / np.linalg.norm(ref)
    e32 = np.linalg.norm(to_host_f64(D32) - ref) / np.linalg.norm(ref)
    assert e32 < 1e-5 < e16 < 2.0 ** -10 * np.sqrt(8192 / 32 + 2) * 2


def test_f16_accumulate_rejects_other_types(sp):
    A = torch.zeros(128, 64, dtype=torch.bfloat16, device="cuda")
    Bt = torch.zeros(128, 128, dtype=torch.bfloat16, device="cuda")
    meta = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    with pytest.raises(sp.Sp24Error):
        sp.gemm(A, meta, Bt, acc_f16=True)
