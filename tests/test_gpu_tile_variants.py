"""Every tile shape the GEMM is built in, for every operand kind, against the oracle.

The library picks the tile shape from the problem size, so at sizes the oracle finishes in seconds
only the small shapes would run; sp24_set_tile_override(<CTAs>, <BLOCK_N>, <m-blocks>)
forces each one.  Sizes span several tiles with ragged tails in M and N."""
import numpy as np
import pytest
import torch

import oracle
from paper_2104_08378_b200 import inputs
from gpu_util import to_device
from test_gpu_gemm import check_fp

pytestmark = pytest.mark.gpu

TORCH_F8 = {"e4m3": torch.float8_e4m3fn, "e5m2": torch.float8_e5m2}
TILES = ["1x128x1", "2x224x1", "2x224x2", "2x192x2", "2x256x1", "2x240x1", "2x256x2"]
DENSE_ONLY = {"2x256x2"}          # two 256-column accumulators fill tensor memory: no room for metadata columns
NO_192 = [t for t in TILES if t not in ("2x192x2", "2x240x1")]
BUILT = {"bf16": TILES, "f16": TILES, "i8": [t for t in TILES if t != "2x240x1"], "tf32": NO_192[:4], "e4m3": NO_192,
         "e5m2": NO_192}


@pytest.fixture(scope="module")
def sp():
    from paper_2104_08378_b200 import binding
    return binding


def _dev(a, kind):
    if kind in TORCH_F8:
        return torch.from_numpy(a).cuda().view(TORCH_F8[kind])
    if kind == "tf32":
        return torch.from_numpy(a.view(np.int32)).cuda().view(torch.float32)
    return to_device(a, kind)


@pytest.mark.parametrize("dense", [False, True])
@pytest.mark.parametrize("tile", TILES)
@pytest.mark.parametrize("kind", ["bf16", "f16", "i8", "tf32", "e4m3", "e5m2"])
def test_forced_tile_shape(sp, force_tile, kind, tile, dense):
    if tile not in BUILT[kind] or (tile in DENSE_ONLY and not dense):
        pytest.skip("shape not built for this kind")
    M, N, K = 1184, 736, 640          # 2.3 tiles of 512 rows, 3.3 of 224 columns, 5 k-blocks of 128
    A = inputs._matrix(("int8",) if kind == "i8" else ("normal", 1.0), kind, 21, 5, K, 0, M)
    Bt = inputs._matrix(("int8",) if kind == "i8" else ("uniform", -1.0, 1.0), kind, 22, 6, K, 0, N)
    Ad, Btd = _dev(A, kind), _dev(Bt, kind)
    force_tile(tile)
    if kind == "i8":
        Cm = inputs._matrix(("int8",), "i8", 23, 7, N, 0, M).astype(np.int32)
        Cd, alpha, beta, cd = torch.from_numpy(Cm).cuda(), 1, 1, "i32"
    elif kind == "tf32":
        Cm = np.ascontiguousarray(inputs._matrix(("normal", 1.0), "tf32", 23, 7, N, 0, M).view(np.float32))
        Cd, alpha, beta, cd = torch.from_numpy(Cm).cuda(), 0.5, -1.5, "f32"
    else:
        cd = "f16" if kind == "f16" else "bf16"
        Cm = inputs._matrix(("normal", 1.0), cd, 23, 7, N, 0, M)
        Cd, alpha, beta = to_device(Cm, cd), 0.5, -1.5
    if dense:
        D = sp.gemm(sp.prune(Ad), None, Btd, alpha=alpha, beta=beta, C=Cd, cd=cd, a_is_dense=True)
    else:
        vals, meta, _ = sp.compress(Ad, layout=sp.META_TCGEN05)
        D = sp.gemm(vals, meta, Btd, alpha=alpha, beta=beta, C=Cd, cd=cd)
    torch.cuda.synchronize()
    assert sp.gemm_status(device=D.device) == 0
    if kind == "tf32":
        v_ref, m_ref, _ = oracle.compress_1of2(A)
        ref, scale = oracle.gemm_sparse_1of2(v_ref, m_ref, Bt, alpha, beta, Cm)
        check_fp(D.to(torch.float64).cpu().numpy(), ref, abs(alpha) * scale, abs(beta) * np.abs(Cm.astype(np.float64)))
        return
    v_ref, m_ref, _ = oracle.compress(A, kind)
    ref = oracle.gemm_sparse(v_ref, m_ref, Bt, kind, alpha, beta, Cm, cd)
    if kind == "i8":
        assert np.array_equal(D.cpu().numpy(), ref)
    else:
        scale = oracle.gemm_abs(v_ref, m_ref, Bt, kind)
        check_fp(D.to(torch.float64).cpu().numpy(), ref, abs(alpha) * scale,
                 abs(beta) * np.abs(oracle.bits_to_float64(Cm, cd)))
