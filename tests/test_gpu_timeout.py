"""The failure path of the GEMM kernel, exercised without faulting or hanging anything: a test hook
makes the TMA producers leave out one k-block, so the MMA issuer's wait for it can never be satisfied.
Every device-side wait is bounded (here shortened to about ten milliseconds): the roles must give
up, record which wait expired, free tensor memory and return; the host must then read
SP24_ERR_TIMEOUT from the workspace, and the very next launch on the same context must work.
The status record is sticky: good launches after the failed one do not erase it; reading it does."""
import pytest
import torch

pytestmark = pytest.mark.gpu

ERR_TIMEOUT = 9


@pytest.fixture(scope="module")
def sp():
    from paper_2104_08378_b200 import binding
    return binding


@pytest.fixture
def fault_hooks(sp):
    yield sp.set_fault_hooks
    sp.set_fault_hooks(0, False)


@pytest.mark.parametrize("tile", ["1x128x1", "2x224x1", "2x224x2"])
def test_expired_wait_is_reported_and_the_context_stays_usable(sp, force_tile, fault_hooks, tile):
    torch.manual_seed(3)
    M, N, K = 512, 448, 1024
    A = (torch.randn(M, K, device="cuda") * 0.1).bfloat16()
    Bt = torch.randn(N, K, device="cuda").bfloat16()
    vals, meta, _ = sp.compress(A)
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    force_tile(tile)
    good = sp.gemm(vals, meta, Bt, ws=ws).clone()
    torch.cuda.synchronize()
    assert sp.gemm_status(ws) == 0

    fault_hooks(20000000, True)                                   # ~10 ms of SM clock per wait; one k-block left out
    sp.gemm(vals, meta, Bt, ws=ws)
    torch.cuda.synchronize()                                      # returns: nothing hangs
    fault_hooks(0, False)
    # two good launches on the same workspace do not erase the record of the failed one
    again = sp.gemm(vals, meta, Bt, ws=ws)
    sp.gemm(vals, meta, Bt, ws=ws)
    torch.cuda.synchronize()
    assert torch.equal(again.view(torch.int16), good.view(torch.int16))
    words = ws.view(torch.int32)[:2].tolist()
    assert words[0] in (1, 2, 3, 4, 5)                            # which role's wait expired first
    assert words[1] >= 1                                          # how many waits expired
    assert sp.gemm_status(ws) == ERR_TIMEOUT                      # reported ...
    assert sp.gemm_status(ws) == 0                                # ... once: reading clears the record
    assert ws.view(torch.int32)[:4].tolist() == [0, 0, 0, 0]
