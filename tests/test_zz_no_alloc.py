"""sp24_gemm_static_ws -- the GEMM entry point for callers that cannot allocate device memory
(all of the GPU's memory already belongs to a framework allocator, or cudaMalloc's device-wide
synchronisation is not acceptable inside a serving loop).  Its workspace is a fixed device array
inside the library, shared by every call.  The test calls it twice in a row (the array keeps
whatever the previous call left there) and checks each result bit for bit against the ordinary
sp24_gemm -- both run the same deterministic kernel -- and once against the CPU oracle; it checks
that the calls leave the amount of free device memory unchanged, and that an expired device-side
wait is observable through sp24_gemm_static_ws_status.  Collected last so that a failure here
cannot hide any other test.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2104_08378_b200 import inputs
from gpu_util import to_device, to_host_f64

pytestmark = pytest.mark.gpu
ERR_TIMEOUT = 9


def _same_bits(got: torch.Tensor, want: torch.Tensor):
    assert got.dtype == want.dtype and got.shape == want.shape
    assert torch.equal(got.contiguous().view(torch.uint8), want.contiguous().view(torch.uint8))


def test_static_workspace_gemm_matches_sp24_gemm_on_two_calls_in_a_row():
    from paper_2104_08378_b200 import binding as sp
    cfg = inputs.scaled(inputs.CONFIGS["gpt3_ffn_bf16"], M=384, N=496, K=1024)
    A_h, Bt_h, C_h = inputs.gen_A(cfg), inputs.gen_Bt(cfg), inputs.gen_C(cfg)
    A, Bt, C = to_device(A_h, "bf16"), to_device(Bt_h, "bf16"), to_device(C_h, "bf16")
    vals, meta, _ = sp.compress(A)
    pruned = sp.prune(A)
    out = torch.empty((cfg.M, cfg.N), dtype=torch.bfloat16, device="cuda")   # caller-owned output
    want1 = sp.gemm(vals, meta, Bt, alpha=1.0, beta=1.0, C=C)
    want2 = sp.gemm(pruned, None, Bt, alpha=-0.5, beta=0.0, a_is_dense=True)
    assert sp.gemm_static_ws_status() == 0            # also the set-up call: resolves the array's address
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    reserved_before = torch.cuda.memory_reserved()
    # first call: sparse, alpha = 1, beta = 1
    sp.gemm_static_ws(vals, meta, Bt, alpha=1.0, beta=1.0, C=C, out=out)
    torch.cuda.synchronize()
    _same_bits(out, want1)
    got1 = to_host_f64(out)
    # second call straight after, other scalars and the dense variant, through the same array
    sp.gemm_static_ws(pruned, None, Bt, alpha=-0.5, beta=0.0, out=out, a_is_dense=True)
    torch.cuda.synchronize()
    _same_bits(out, want2)
    assert sp.gemm_static_ws_status() == 0
    # nothing was allocated on the device by either call
    assert torch.cuda.mem_get_info()[0] == free_before
    assert torch.cuda.memory_reserved() == reserved_before
    # and the first result against the oracle, with the tolerance of the GEMM tests
    vals_ref, meta_ref, _ = oracle.compress(A_h, "bf16")
    ref = oracle.gemm_sparse(vals_ref, meta_ref, Bt_h, "bf16", 1.0, 1.0, C_h, "bf16")
    bound = 1e-2 * (oracle.gemm_abs(vals_ref, meta_ref, Bt_h, "bf16") + np.abs(oracle.bits_to_float64(C_h, "bf16")))
    err = np.abs(got1 - ref)
    assert np.linalg.norm(err) / np.linalg.norm(ref) <= 2e-3
    assert (err <= bound + 1e-30).all()
    # int8 through the same array
    cfg8 = inputs.scaled(inputs.CONFIGS["int8_linear"], M=256, N=256, K=512)
    A8, B8 = to_device(inputs.gen_A(cfg8), "i8"), to_device(inputs.gen_Bt(cfg8), "i8")
    v8, m8, _ = sp.compress(A8)
    out8 = torch.empty((256, 256), dtype=torch.int32, device="cuda")
    sp.gemm_static_ws(v8, m8, B8, alpha=1, beta=0, out=out8)
    torch.cuda.synchronize()
    _same_bits(out8, sp.gemm(v8, m8, B8, alpha=1, beta=0))


def test_static_workspace_reports_an_expired_wait():
    """The bounded-wait failure path through the shared array: a test hook makes a wait expire after
    about ten milliseconds (nothing faults or hangs); the status reader of this entry point must
    report it once, and the next call must work."""
    from paper_2104_08378_b200 import binding as sp
    torch.manual_seed(7)
    A = (torch.randn(256, 1024, device="cuda") * 0.1).bfloat16()
    Bt = torch.randn(256, 1024, device="cuda").bfloat16()
    vals, meta, _ = sp.compress(A)
    out = torch.empty((256, 256), dtype=torch.bfloat16, device="cuda")
    want = sp.gemm(vals, meta, Bt)
    assert sp.gemm_static_ws_status() == 0
    try:
        sp.set_fault_hooks(20000000, True)
        sp.gemm_static_ws(vals, meta, Bt, out=out)
        torch.cuda.synchronize()
    finally:
        sp.set_fault_hooks(0, False)
    assert sp.gemm_static_ws_status() == ERR_TIMEOUT
    assert sp.gemm_static_ws_status() == 0
    sp.gemm_static_ws(vals, meta, Bt, out=out)
    torch.cuda.synchronize()
    assert sp.gemm_static_ws_status() == 0
    _same_bits(out, want)


def test_static_workspace_gemm_validates_like_sp24_gemm():
    from paper_2104_08378_b200 import binding as sp
    a = torch.zeros((16, 8), dtype=torch.float16, device="cuda")
    m = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    out = torch.zeros((16, 8), dtype=torch.float16, device="cuda")
    with pytest.raises(sp.Sp24Error):                      # N = 8 breaks the multiple-of-16 rule
        sp.gemm_static_ws(a, m, torch.zeros((8, 16), dtype=torch.float16, device="cuda"), out=out)
