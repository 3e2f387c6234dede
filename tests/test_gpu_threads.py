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


def test_concurrent_host_buffer_pipelines_in_bands(sp):
    """Two host threads run the banded form of sp24_pipeline_host (M >= 16384: copy-out on the library's
    second stream) on the same device at once, each on its own stream with its own buffers; the events
    that order a band's copy-out behind its GEMM belong to the call, so neither thread can make the
    other's copy start early."""
    import ctypes
    M, N, K = 16384, 256, 256
    gen = torch.Generator().manual_seed(11)
    hosts, wants = [], []
    for i in range(2):
        hA = (torch.randn(M, K, generator=gen) * 0.1).bfloat16().pin_memory()
        hB = torch.randn(N, K, generator=gen).bfloat16().pin_memory()
        hosts.append((hA, hB))
        vals, meta, _ = sp.compress(hA.cuda())
        wants.append(sp.gemm(vals, meta, hB.cuda()).cpu())
    torch.cuda.synchronize()
    errors, outs = [], [None, None]

    def worker(i):
        try:
            hA, hB = hosts[i]
            stream = torch.cuda.Stream()
            with torch.cuda.stream(stream):
                dA = torch.empty((M, K), dtype=torch.bfloat16, device="cuda")
                dV = torch.empty((M, K // 2), dtype=torch.bfloat16, device="cuda")
                dM = torch.empty(sp.meta_bytes("bf16", M, K), dtype=torch.uint8, device="cuda")
                dB = torch.empty((N, K), dtype=torch.bfloat16, device="cuda")
                dD = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
                ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
                hD = torch.empty((M, N), dtype=torch.bfloat16).pin_memory()
                desc = sp.make_desc("bf16", "bf16", M, N, K, K // 2, K, N, N)
                al, be = ctypes.c_float(1.0), ctypes.c_float(0.0)
                vp = lambda t: ctypes.c_void_p(t.data_ptr()) if t is not None else None  # noqa: E731
                for _ in range(10):
                    hD.zero_()
                    st = sp.lib.sp24_pipeline_host(ctypes.byref(desc), ctypes.byref(al), vp(hA), vp(hB), ctypes.byref(be),
                                                   None, vp(hD), vp(dA), vp(dV), vp(dM), vp(dB), None, vp(dD), vp(ws),
                                                   ws.numel(), stream.cuda_stream)
                    assert st == 0
                    stream.synchronize()            # the caller's stream ends behind the second stream's copies
                    assert torch.equal(hD.view(torch.int16), wants[i].view(torch.int16))
                assert sp.gemm_status(ws) == 0
            outs[i] = True
        except Exception as e:  # noqa: BLE001
            errors.append(e)

    threads = [threading.Thread(target=worker, args=(i,)) for i in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    assert all(outs)
