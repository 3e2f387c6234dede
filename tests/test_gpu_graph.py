"""The whole path (prune -> compress -> GEMM) captured in a CUDA graph and replayed: every entry
point only enqueues work on the caller's stream (tensor maps are encoded on the host and passed by
value), so a captured step must reproduce the eager results bit for bit, also after the input
buffers' contents change between replays."""
import numpy as np
import pytest
import torch

import oracle
from paper_2104_08378_b200 import inputs
from gpu_util import to_device, to_host_bits
from test_gpu_gemm import check_fp

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def sp():
    from paper_2104_08378_b200 import binding
    return binding


@pytest.mark.parametrize("ab", ["bf16", "i8"])
def test_captured_step_replays_bit_exact(sp, ab):
    M, N, K = 640, 704, 512
    cd = "bf16" if ab == "bf16" else "i32"
    dist = ("normal", 1.0) if ab == "bf16" else ("int8",)
    host = [inputs._matrix(dist, ab, 40 + i, 5, K, 0, M) for i in range(3)]
    Bt_h = inputs._matrix(("uniform", -1.0, 1.0) if ab == "bf16" else ("int8",), ab, 50, 6, K, 0, N)
    A = to_device(host[0], ab).clone()
    Bt = to_device(Bt_h, ab)
    pruned = torch.empty_like(A)
    vals = torch.empty((M, K // 2), dtype=A.dtype, device="cuda")
    meta = torch.empty(sp.meta_bytes(ab, M, K, sp.META_TCGEN05), dtype=torch.uint8, device="cuda")
    D = torch.empty((M, N), dtype=sp.TORCH_DTYPE[cd], device="cuda")
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")

    def step():
        sp.prune(A, out=pruned)
        sp.compress_into(pruned, vals, meta, layout=sp.META_TCGEN05)
        sp.gemm(vals, meta, Bt, out=D, cd=cd, ws=ws)

    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        step()                                   # warm-up outside the capture (first-call initialisation)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    for h in host:
        A.copy_(to_device(h, ab))
        graph.replay()
        torch.cuda.synchronize()
        assert sp.gemm_status(ws) == 0
        got_vals, got_meta, got_D = vals.clone(), meta.clone(), D.clone()
        step()                                   # eager, same buffers
        torch.cuda.synchronize()
        assert torch.equal(got_vals.view(torch.uint8), vals.view(torch.uint8))
        assert torch.equal(got_meta, meta)
        assert torch.equal(got_D.view(torch.uint8), D.view(torch.uint8))
        v_ref, m_ref, _ = oracle.compress(h, ab)
        assert np.array_equal(to_host_bits(got_vals), v_ref)
        ref = oracle.gemm_sparse(v_ref, m_ref, Bt_h, ab)
        if ab == "i8":
            assert np.array_equal(got_D.cpu().numpy(), ref)
        else:
            check_fp(got_D.to(torch.float64).cpu().numpy(), ref, oracle.gemm_abs(v_ref, m_ref, Bt_h, ab))
