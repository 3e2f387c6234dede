"""GPU parity for prune / compress / decompress / im2col: bit-exact against the CPU oracle,
called through the C ABI (ctypes binding)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2104_08378_b200 import inputs
from gpu_util import to_device, to_host_bits

pytestmark = pytest.mark.gpu

DTYPES = ["f16", "bf16", "i8"]
SHAPES = [(256, 512), (200, 656), (37, 96), (129, 272), (1, 16), (513, 2064)]


@pytest.fixture(scope="module")
def sp():
    from paper_2104_08378_b200 import binding
    return binding


def _rand(dtype, M, K, seed):
    dist = ("int8",) if dtype == "i8" else ("normal", 1.0)
    return inputs._matrix(dist, dtype, seed, 9, K, 0, M)


def _adversarial(dtype, M, K, seed):
    """Few distinct magnitudes (many ties), zeros of both signs, denormals, -128 for int8."""
    rng = np.random.default_rng(seed)
    if dtype == "i8":
        pool = np.array([-128, -127, -2, -1, 0, 0, 1, 2, 127], dtype=np.int8)
    elif dtype == "f16":
        pool = np.array([0x0000, 0x8000, 0x0001, 0x8001, 0x3C00, 0xBC00, 0x4000, 0xC000, 0x7BFF, 0x03FF],
                        dtype=np.uint16)
    else:
        pool = np.array([0x0000, 0x8000, 0x0001, 0x8001, 0x3F80, 0xBF80, 0x4000, 0xC000, 0x7F7F, 0x007F],
                        dtype=np.uint16)
    return np.ascontiguousarray(pool[rng.integers(0, len(pool), size=(M, K))])


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("shape", SHAPES)
def test_prune_bit_exact(sp, dtype, shape):
    M, K = shape
    for x in (_rand(dtype, M, K, 1), _adversarial(dtype, M, K, 2)):
        y = sp.prune(to_device(x, dtype))
        assert np.array_equal(to_host_bits(y), oracle.prune(x, dtype))


@pytest.mark.parametrize("dtype", DTYPES)
def test_prune_in_place_and_strided(sp, dtype):
    M, K, ld = 70, 144, 176
    x = _rand(dtype, M, ld, 3)
    xd = to_device(x, dtype)
    view = xd[:, :K]                                   # leading dimension 176 > K
    sp.prune(view, out=view)                           # y aliases x
    got = to_host_bits(xd)
    assert np.array_equal(got[:, :K], oracle.prune(np.ascontiguousarray(x[:, :K]), dtype))
    assert np.array_equal(got[:, K:], x[:, K:])        # columns past K untouched
    # misaligned start (scalar path): drop the first 4 columns
    x2 = _rand(dtype, M, ld, 4)
    xd2 = to_device(x2, dtype)
    y2 = sp.prune(xd2[:, 4:4 + 100])
    assert np.array_equal(to_host_bits(y2), oracle.prune(np.ascontiguousarray(x2[:, 4:104]), dtype))


@pytest.mark.parametrize("dtype", DTYPES)
@pytest.mark.parametrize("shape", SHAPES + [(64, 40)])
@pytest.mark.parametrize("layout", [0, 1])
def test_compress_decompress_bit_exact(sp, dtype, shape, layout):
    M, K = shape
    for x in (_rand(dtype, M, K, 5), _adversarial(dtype, M, K, 6)):
        vals_ref, meta_ref, dropped_ref = oracle.compress(x, dtype)
        vals, meta, dropped = sp.compress(to_device(x, dtype), layout=layout, count_dropped=True)
        assert np.array_equal(to_host_bits(vals), vals_ref)
        meta_h = meta.cpu().numpy()
        expect = meta_ref.ravel() if layout == 0 else oracle.meta_to_operand_order(meta_ref, dtype)
        assert meta_h.size == expect.size
        assert np.array_equal(meta_h, expect)
        assert int(dropped.item()) == dropped_ref
        back = sp.decompress(vals, meta, layout=layout)
        assert np.array_equal(to_host_bits(back), oracle.prune(x, dtype))


def test_compress_of_pruned_input_drops_nothing(sp):
    x = _rand("bf16", 128, 256, 7)
    y = sp.prune(to_device(x, "bf16"))
    v1, m1, d1 = sp.compress(y, count_dropped=True)
    v0, m0, _ = sp.compress(to_device(x, "bf16"))
    assert int(d1.item()) == 0
    assert torch.equal(v1.view(torch.int16), v0.view(torch.int16)) and torch.equal(m1, m0)


def test_empty_and_bad_arguments(sp):
    e = torch.empty((0, 64), dtype=torch.float16, device="cuda")
    assert sp.prune(e).shape == (0, 64)
    x = torch.zeros((4, 6), dtype=torch.float16, device="cuda")
    with pytest.raises(sp.Sp24Error) as err:
        sp.prune(x)                                     # K % 4 != 0
    assert err.value.status == 3
    with pytest.raises(sp.Sp24Error):
        sp.compress(torch.zeros((4, 12), dtype=torch.int8, device="cuda"))   # K % 8 != 0
    with pytest.raises(sp.Sp24Error):
        sp.prune(torch.zeros((4, 8), dtype=torch.int32, device="cuda"), dtype="i32")


@pytest.mark.parametrize("dtype", ["f16", "i8"])
def test_im2col_bit_exact(sp, dtype):
    cfg = inputs.scaled(inputs.CONFIGS["resnet_conv_f16"], conv=(3, 14, 14, 32))
    x = inputs._matrix(("relu_normal", 1.0) if dtype != "i8" else ("int8",), dtype, 4, 1, 14 * 14 * 32, 0, 3)
    x = x.reshape(3, 14, 14, 32)
    got = sp.im2col_nhwc_3x3(to_device(x, dtype))
    assert np.array_equal(to_host_bits(got), oracle.im2col_nhwc_3x3(x, dtype))
    assert got.shape == (cfg.N, cfg.K)


@pytest.mark.parametrize("dtype", ["f16", "bf16", "i8"])
@pytest.mark.parametrize("shape", [(128, 256), (200, 336), (37, 96), (513, 1040), (1024, 4096)])
@pytest.mark.parametrize("layout", [0, 1])
def test_fused_prune_compress_equals_the_two_passes(sp, dtype, shape, layout):
    """sp24_prune_compress: one pass over x gives prune(x) and compress(x) bit for bit (oracle on both),
    also in place (y = x) and with the dropped count."""
    M, K = shape
    cfg = inputs.scaled(inputs.CONFIGS["int8_linear" if dtype == "i8" else "tiny_f16"], M=M, N=32, K=K)
    x = inputs._matrix(cfg.a_dist, dtype, 77, inputs.TENSOR_A, K, 0, M)
    x[::3, ::5] = 0
    xd = to_device(x, dtype)
    pruned, vals, meta, dropped = sp.prune_compress(xd, layout=layout, count_dropped=True)
    v_ref, m_ref, d_ref = oracle.compress(x, dtype)
    assert np.array_equal(to_host_bits(pruned), oracle.prune(x, dtype))
    assert np.array_equal(to_host_bits(vals), v_ref)
    expect = m_ref.ravel() if layout == 0 else oracle.meta_to_operand_order(m_ref, dtype)
    assert np.array_equal(meta.cpu().numpy(), expect)
    assert int(dropped.item()) == d_ref
    inplace = xd.clone()
    p2, v2, m2, _ = sp.prune_compress(inplace, layout=layout, pruned=inplace)
    assert p2.data_ptr() == inplace.data_ptr()
    assert torch.equal(inplace.view(torch.uint8), pruned.view(torch.uint8))
    assert torch.equal(v2.view(torch.uint8), vals.view(torch.uint8)) and torch.equal(m2, meta)


def test_fused_prune_compress_falls_back_for_unaligned_operands(sp):
    """An odd leading dimension takes the element-wise kernels (two passes) with the same result."""
    M, K, ld = 64, 96, 99
    x = inputs._matrix(("normal", 1.0), "bf16", 78, inputs.TENSOR_A, K, 0, M)
    buf = torch.zeros(M, ld, dtype=torch.bfloat16, device="cuda")
    buf[:, :K] = to_device(x, "bf16")
    xd = buf[:, :K]
    out = torch.zeros(M, ld, dtype=torch.bfloat16, device="cuda")[:, :K]
    pruned, vals, meta, _ = sp.prune_compress(xd, layout=0, pruned=out)
    v_ref, m_ref, _ = oracle.compress(x, "bf16")
    assert np.array_equal(to_host_bits(pruned.contiguous()), oracle.prune(x, "bf16"))
    assert np.array_equal(to_host_bits(vals), v_ref)
    assert np.array_equal(meta.cpu().numpy(), m_ref.ravel())


@pytest.mark.parametrize("dtype", ["f16", "bf16", "i8"])
def test_every_bit_pattern_in_every_position(sp, dtype):
    """All 65536 (256 for int8) encodings -- zeros of both signs, subnormals, infinities and NaN
    patterns, -128 -- meet random partners in every position of a group: prune, compress (both
    layouts) and the fused pass against the oracle, bit for bit."""
    rng = np.random.default_rng(5)
    n = 256 if dtype == "i8" else 65536
    store = np.int8 if dtype == "i8" else np.uint16
    allv = np.arange(n, dtype=np.uint8 if dtype == "i8" else np.uint16).view(store)
    M, K = 4 * n // 256, 1024                       # every pattern once in each of the four positions
    x = rng.integers(0, n, size=(M, K)).astype(np.uint16 if dtype != "i8" else np.uint8).view(store)
    x = np.ascontiguousarray(x)
    groups = x.reshape(-1, 4)
    for pos in range(4):
        groups[pos * n:(pos + 1) * n, pos] = allv      # group pos*n + v holds pattern v at position pos
    # near-ties: copy the pattern into a second position with the sign flipped in a quarter of the groups
    flip = np.uint16(0x8000) if dtype != "i8" else None
    if flip is not None:
        g16 = groups.view(np.uint16)
        g16[::4, 3] = g16[::4, 0] ^ flip
    x = groups.reshape(M, K)
    xd = to_device(x, dtype)
    assert np.array_equal(to_host_bits(sp.prune(xd)), oracle.prune(x, dtype))
    v_ref, m_ref, d_ref = oracle.compress(x, dtype)
    for layout in (0, 1):
        vals, meta, dropped = sp.compress(xd, layout=layout, count_dropped=True)
        assert np.array_equal(to_host_bits(vals), v_ref)
        expect = m_ref.ravel() if layout == 0 else oracle.meta_to_operand_order(m_ref, dtype)
        assert np.array_equal(meta.cpu().numpy(), expect)
        assert int(dropped.item()) == d_ref
    pruned, vals, meta, _ = sp.prune_compress(xd, layout=1)
    assert np.array_equal(to_host_bits(pruned), oracle.prune(x, dtype))
    assert np.array_equal(to_host_bits(vals), v_ref)
