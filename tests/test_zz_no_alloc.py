"""sp24_gemm_static_ws -- the GEMM entry point for callers that cannot allocate device memory
(all of the GPU's memory already belongs to a framework allocator, or cudaMalloc's device-wide
synchronisation is not acceptable inside a serving loop).  Its workspace is a fixed device array
inside the library, so this test calls it twice in a row (the array keeps the previous call's
contents) and checks each result against the ordinary sp24_gemm, within the tolerance the GEMM
tests use.  Collected last so that a failure here cannot hide any other test.
"""
import numpy as np
import pytest
import torch

from paper_2104_08378_b200 import inputs
from gpu_util import to_device

pytestmark = pytest.mark.gpu


def _close(got: torch.Tensor, want: torch.Tensor):
    g, w = got.double().cpu().numpy(), want.double().cpu().numpy()
    if want.dtype == torch.int32:
        assert np.array_equal(g, w)
        return
    rel = np.linalg.norm(g - w) / max(np.linalg.norm(w), 1e-30)
    assert rel <= 2e-3, f"normwise relative difference {rel:.3e}"


def test_static_workspace_gemm_matches_sp24_gemm_on_two_calls_in_a_row():
    from paper_2104_08378_b200 import binding as sp
    cfg = inputs.scaled(inputs.CONFIGS["gpt3_ffn_bf16"], M=384, N=496, K=1024)
    A, Bt, C = to_device(inputs.gen_A(cfg), "bf16"), to_device(inputs.gen_Bt(cfg), "bf16"), \
        to_device(inputs.gen_C(cfg), "bf16")
    vals, meta, _ = sp.compress(A)
    out = torch.empty((cfg.M, cfg.N), dtype=torch.bfloat16, device="cuda")   # caller-owned output
    # first call: sparse, alpha = 1, beta = 1
    want1 = sp.gemm(vals, meta, Bt, alpha=1.0, beta=1.0, C=C)
    sp.gemm_static_ws(vals, meta, Bt, alpha=1.0, beta=1.0, C=C, out=out)
    torch.cuda.synchronize()
    _close(out, want1)
    # second call straight after, other scalars and the dense variant: the shared array holds
    # the first call's record and must not leak into this one
    pruned = sp.prune(A)
    want2 = sp.gemm(pruned, None, Bt, alpha=-0.5, beta=0.0, a_is_dense=True)
    sp.gemm_static_ws(pruned, None, Bt, alpha=-0.5, beta=0.0, out=out, a_is_dense=True)
    torch.cuda.synchronize()
    _close(out, want2)
    # int8 through the same array
    cfg8 = inputs.scaled(inputs.CONFIGS["int8_linear"], M=256, N=256, K=512)
    A8, B8 = to_device(inputs.gen_A(cfg8), "i8"), to_device(inputs.gen_Bt(cfg8), "i8")
    v8, m8, _ = sp.compress(A8)
    out8 = torch.empty((256, 256), dtype=torch.int32, device="cuda")
    sp.gemm_static_ws(v8, m8, B8, alpha=1, beta=0, out=out8)
    torch.cuda.synchronize()
    _close(out8, sp.gemm(v8, m8, B8, alpha=1, beta=0))


def test_static_workspace_gemm_validates_like_sp24_gemm():
    from paper_2104_08378_b200 import binding as sp
    a = torch.zeros((16, 8), dtype=torch.float16, device="cuda")
    m = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    out = torch.zeros((16, 8), dtype=torch.float16, device="cuda")
    with pytest.raises(sp.Sp24Error):                      # N = 8 breaks the multiple-of-16 rule
        sp.gemm_static_ws(a, m, torch.zeros((8, 16), dtype=torch.float16, device="cuda"), out=out)
