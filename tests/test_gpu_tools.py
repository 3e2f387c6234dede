"""GPU parity of the pruning tools: kept magnitude (double sum, relative 1e-12), apply_mask and
prune_2d bit-exact against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2104_08378_b200 import inputs
from gpu_util import to_device, to_host_bits

pytestmark = pytest.mark.gpu
DTYPES = ["f16", "bf16", "i8"]


@pytest.fixture(scope="module")
def sp():
    from paper_2104_08378_b200 import binding
    return binding


def _rand(dtype, M, K, seed):
    return inputs._matrix(("int8",) if dtype == "i8" else ("normal", 1.0), dtype, seed, 3, K, 0, M)


@pytest.mark.parametrize("dtype", DTYPES)
def test_kept_magnitude(sp, dtype):
    x = _rand(dtype, 300, 520, 1)
    xd = to_device(x, dtype)
    got = float(sp.kept_magnitude(xd).item())
    assert abs(got - oracle.kept_magnitude(x, dtype)) <= 1e-12 * got
    perm = np.random.default_rng(1).permutation(520).astype(np.int32)
    got_p = float(sp.kept_magnitude(xd, torch.from_numpy(perm).cuda()).item())
    assert abs(got_p - oracle.kept_magnitude(x, dtype, perm)) <= 1e-12 * got_p
    assert sp.kept_magnitude(xd[:0]).item() == 0.0


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("layout", [0, 1])
def test_apply_mask(sp, dtype, layout):
    x, w = _rand(dtype, 200, 656, 2), _rand(dtype, 200, 656, 3)
    _, meta_ref, _ = oracle.compress(x, dtype)
    _, meta, _ = sp.compress(to_device(x, dtype), layout=layout)
    wd = to_device(w, dtype)
    assert np.array_equal(to_host_bits(sp.apply_mask(wd, meta, layout=layout)), oracle.apply_mask(w, meta_ref, dtype))
    sp.apply_mask(wd, meta, layout=layout, out=wd)                       # in place
    assert np.array_equal(to_host_bits(wd), oracle.apply_mask(w, meta_ref, dtype))


@pytest.mark.parametrize("dtype", DTYPES)
def test_prune_2d(sp, dtype):
    x = _rand(dtype, 132, 260, 4)
    x[::5, ::3] = 0
    x[8:12, 8:12] = x[8, 8]                                              # a block of equal magnitudes: ties
    y = sp.prune_2d(to_device(x, dtype))
    assert np.array_equal(to_host_bits(y), oracle.prune_2d(x, dtype))
    with pytest.raises(sp.Sp24Error):
        sp.prune_2d(to_device(x[:130], dtype))                           # M % 4 != 0


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("shape", [(64, 512), (37, 4096), (5, 32768), (130, 264)])
def test_kept_magnitude_vector_and_scalar_paths(sp, dtype, shape):
    """Rows that take the 16-byte-vector kernels, rows too long for the shared-memory gather of the
    permuted form (32768 16-bit columns), and an unaligned view that takes the element-wise kernel."""
    M, K = shape
    x = _rand(dtype, M, K, 6)
    x[::2, ::3] = 0
    perm = np.random.default_rng(2).permutation(K).astype(np.int32)
    permd = torch.from_numpy(perm).cuda()
    want, want_p = oracle.kept_magnitude(x, dtype), oracle.kept_magnitude(x, dtype, perm)
    xd = to_device(x, dtype)
    assert abs(float(sp.kept_magnitude(xd).item()) - want) <= 1e-12 * want
    assert abs(float(sp.kept_magnitude(xd, permd).item()) - want_p) <= 1e-12 * want_p
    wide = torch.zeros(M, K + 3, dtype=xd.dtype, device="cuda")           # odd leading dimension
    wide[:, :K] = xd
    view = wide[:, :K]
    assert abs(float(sp.kept_magnitude(view).item()) - want) <= 1e-12 * want
    assert abs(float(sp.kept_magnitude(view, permd).item()) - want_p) <= 1e-12 * want_p


@pytest.mark.parametrize("dtype", DTYPES)
def test_apply_mask_and_prune_2d_on_unaligned_views(sp, dtype):
    M, K = 68, 264
    x, w = _rand(dtype, M, K, 7), _rand(dtype, M, K, 8)
    _, meta_ref, _ = oracle.compress(x, dtype)
    _, meta, _ = sp.compress(to_device(x, dtype), layout=0)
    wide = torch.zeros(M, K + 5, dtype=to_device(w, dtype).dtype, device="cuda")
    wide[:, :K] = to_device(w, dtype)
    view = wide[:, :K]
    assert np.array_equal(to_host_bits(sp.apply_mask(view, meta, layout=0).contiguous()), oracle.apply_mask(w, meta_ref, dtype))
    assert np.array_equal(to_host_bits(sp.prune_2d(view).contiguous()), oracle.prune_2d(w, dtype))
    big = _rand(dtype, 512, 2048, 9)
    assert np.array_equal(to_host_bits(sp.prune_2d(to_device(big, dtype))), oracle.prune_2d(big, dtype))
