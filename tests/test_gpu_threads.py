"""Host-side thread safety: several Python threads (ctypes releases the GIL) call the library at the
same time, each on its own stream and with its own workspace; every result equals the one computed
alone."""
import threading

import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def sp():
    from paper_2104_08378_b200 import binding
    return binding


def test_concurrent_callers_on_separate_streams(sp):
    torch.manual_seed(5)
    M, N, K = 768, 896, 1024
    A = (torch.randn(M, K, device="cuda") * 0.1).bfloat16()
    Bt = torch.randn(N, K, device="cuda").bfloat16()
    pruned0, vals0, meta0, _ = sp.prune_compress(A)
    want = sp.gemm(vals0, meta0, Bt)
    torch.cuda.synchronize()
    results, errors = [None] * 6, []

    def worker(i):
        try:
            stream = torch.cuda.Stream()
            ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
            with torch.cuda.stream(stream):
                for _ in range(20):
                    pruned, vals, meta, _ = sp.prune_compress(A)
                    out = sp.gemm(vals, meta, Bt, ws=ws)
                stream.synchronize()
                assert sp.gemm_status(ws) == 0
                results[i] = (pruned, vals, meta, out)
        except Exception as e:  # noqa: BLE001
            errors.append(e)

    threads = [threading.Thread(target=worker, args=(i,)) for i in range(6)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    for pruned, vals, meta, out in results:
        assert torch.equal(pruned.view(torch.int16), pruned0.view(torch.int16))
        assert torch.equal(vals.view(torch.int16), vals0.view(torch.int16)) and torch.equal(meta, meta0)
        assert torch.equal(out.view(torch.int16), want.view(torch.int16))
