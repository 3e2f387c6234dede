"""Index arithmetic beyond 2^31 elements: the streaming kernels on a matrix of 2.6e9 elements and
the GEMM on an output of 2.2e9 elements, checked against the oracle on row bands / tiles that
include the first and last rows and the rows on both sides of element 2^31.  Inputs are seeded
device-side draws (a host generator pass over gigabytes would dominate the test); the bands the
oracle needs are copied back."""
import numpy as np
import pytest
import torch

import oracle
from test_gpu_gemm import check_fp

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def sp():
    from paper_2104_08378_b200 import binding
    return binding


def test_prune_compress_decompress_past_2_pow_31_elements(sp):
    M, K = 40000, 65536                         # 2.62e9 int8 elements; row 32768 starts at element 2^31
    assert M * K > 2 ** 31
    g = torch.Generator(device="cuda").manual_seed(31)
    x = torch.randint(-127, 128, (M, K), dtype=torch.int8, device="cuda", generator=g)
    x[:, ::7] = 0
    pruned = sp.prune(x)
    vals, meta_c, dropped = sp.compress(x, layout=sp.META_CANONICAL, count_dropped=True)
    _, meta_t, _ = sp.compress(x, layout=sp.META_TCGEN05)
    back = sp.decompress(vals, meta_t, layout=sp.META_TCGEN05)
    torch.cuda.synchronize()
    assert torch.equal(back, pruned)
    meta_c = meta_c.view(M, K // 8)
    total_dropped = 0
    for r0, r1 in ((0, 64), (32704, 32832), (M - 64, M)):
        xb = x[r0:r1].cpu().numpy()
        assert np.array_equal(pruned[r0:r1].cpu().numpy(), oracle.prune(xb, "i8"))
        v_ref, m_ref, _ = oracle.compress(xb, "i8")
        assert np.array_equal(vals[r0:r1].cpu().numpy(), v_ref)
        assert np.array_equal(meta_c[r0:r1].cpu().numpy(), m_ref)
    # the operand-order metadata of whole 128-row blocks (block 255 ends at row 32768, block 256 starts there)
    blk_bytes = (2 * ((K + 255) // 256)) * 2048
    for mb in (0, 255, 256, M // 128 - 1):
        xb = x[mb * 128:(mb + 1) * 128].cpu().numpy()
        m_ref = oracle.compress(xb, "i8")[1]
        got = meta_t[mb * blk_bytes:(mb + 1) * blk_bytes].cpu().numpy()
        assert np.array_equal(got, oracle.meta_to_operand_order(m_ref, "i8"))
    # the dropped count is a property of the whole matrix: non-zeros of x that prune removed
    total_dropped = int(((x != 0) & (pruned == 0)).sum().item())
    assert int(dropped.item()) == total_dropped


@pytest.mark.parametrize("col_major", [False, True])
def test_gemm_output_past_2_pow_31_elements(sp, col_major):
    M, N, K = 65536, 33024, 64                  # 2.16e9 output elements (4.3 GB of bf16), C the same again
    assert M * N > 2 ** 31
    g = torch.Generator(device="cuda").manual_seed(32)
    A = (torch.randn(M, K, device="cuda", generator=g) * 0.5).bfloat16()
    Bt = torch.randn(N, K, device="cuda", generator=g).bfloat16()
    shape = (N, M) if col_major else (M, N)
    C = torch.randn(shape, device="cuda", generator=g, dtype=torch.bfloat16)
    vals, meta, _ = sp.compress(A)
    D = sp.gemm(vals, meta, Bt, alpha=1.0, beta=0.5, C=C, cd_col_major=col_major)
    torch.cuda.synchronize()
    assert sp.gemm_status(device=D.device) == 0
    A_h = A.view(torch.int16).cpu().numpy().view(np.uint16)
    Bt_h = Bt.view(torch.int16).cpu().numpy().view(np.uint16)
    v_ref, m_ref, _ = oracle.compress(A_h, "bf16")
    # the row whose first output element is number 2^31 (row-major: 2^31 / N = 65027.6), corners, middle
    for (r0, c0) in ((0, 0), (65024, 0), (65024, N - 128), (M - 128, N - 128), (M - 128, 0), (32768, 16512)):
        rows, cols = (r0, r0 + 128), (c0, c0 + 128)
        Cw = C[c0:c0 + 128, r0:r0 + 128].t() if col_major else C[r0:r0 + 128, c0:c0 + 128]
        Dw = D[c0:c0 + 128, r0:r0 + 128].t() if col_major else D[r0:r0 + 128, c0:c0 + 128]
        Cw = Cw.to(torch.float64).cpu().numpy()
        ref = oracle.gemm_sparse(v_ref, m_ref, Bt_h, "bf16", rows=rows, cols=cols) + 0.5 * Cw
        scale = oracle.gemm_abs(v_ref, m_ref, Bt_h, "bf16", rows=rows, cols=cols)
        check_fp(Dw.to(torch.float64).cpu().numpy(), ref, scale, 0.5 * np.abs(Cw))
