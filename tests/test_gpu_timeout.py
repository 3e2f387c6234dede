"""The failure path of the GEMM kernel, exercised without faulting or hanging anything: a test hook
makes the TMA producers leave out one k-block, so the MMA issuer's wait for it can never be satisfied.
Every device-side wait is bounded (here shortened to about ten milliseconds): the roles must give
up, record which wait expired, free tensor memory and return; the host must then read
SP24_ERR_TIMEOUT from the workspace, and the very next launch on the same context must work."""
import pytest
import torch

pytestmark = pytest.mark.gpu

ERR_TIMEOUT = 9


@pytest.fixture(scope="module")
def sp():
    from paper_2104_08378_b200 import binding
    return binding


@pytest.mark.parametrize("tile", ["1x128x1", "2x224x1", "2x224x2"])
def test_expired_wait_is_reported_and_the_context_stays_usable(sp, monkeypatch, tile):
    torch.manual_seed(3)
    M, N, K = 512, 448, 1024
    A = (torch.randn(M, K, device="cuda") * 0.1).bfloat16()
    Bt = torch.randn(N, K, device="cuda").bfloat16()
    vals, meta, _ = sp.compress(A)
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    monkeypatch.setenv("SP24_TILE", tile)
    good = sp.gemm(vals, meta, Bt, ws=ws).clone()
    torch.cuda.synchronize()
    assert sp.gemm_status(ws) == 0

    monkeypatch.setenv("SP24_TEST_WAIT_CYCLES", "20000000")      # ~10 ms of SM clock per wait
    monkeypatch.setenv("SP24_TEST_SKIP_STAGE", "1")
    sp.gemm(vals, meta, Bt, ws=ws)
    torch.cuda.synchronize()                                      # returns: nothing hangs
    assert sp.gemm_status(ws) == ERR_TIMEOUT
    code = int(ws.view(torch.int32)[0].item())
    assert code in (1, 2, 3, 4, 5)                                # which role's wait expired first

    monkeypatch.delenv("SP24_TEST_SKIP_STAGE")
    monkeypatch.delenv("SP24_TEST_WAIT_CYCLES")
    again = sp.gemm(vals, meta, Bt, ws=ws)
    torch.cuda.synchronize()
    assert sp.gemm_status(ws) == 0
    assert torch.equal(again.view(torch.int16), good.view(torch.int16))
