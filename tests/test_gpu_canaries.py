"""No kernel writes outside its outputs: every output lives between two guard bands filled with a
canary byte (and, for strided outputs, has canaries in the row padding); after each call the bands
must be untouched.  Shapes have ragged tails in every dimension the kernels tile."""
import numpy as np
import pytest
import torch

pytestmark = pytest.mark.gpu
CANARY = 0xA5
GUARD = 4096


@pytest.fixture(scope="module")
def sp():
    from paper_2104_08378_b200 import binding
    return binding


class Guarded:
    """A 2-D tensor of `dtype` with `rows` x `cols` elements and leading dimension `ld`, carved out of a
    byte buffer that starts and ends with guard bands."""

    def __init__(self, rows, cols, dtype, ld=None):
        self.es = torch.empty(0, dtype=dtype).element_size()
        self.rows, self.cols, self.ld = rows, cols, ld or cols
        self.nbytes = rows * self.ld * self.es
        self.buf = torch.full((GUARD + self.nbytes + GUARD,), CANARY, dtype=torch.uint8, device="cuda")
        body = self.buf[GUARD:GUARD + self.nbytes].view(dtype).view(rows, self.ld)
        self.t = body[:, :cols]

    def check(self, what):
        assert bool((self.buf[:GUARD] == CANARY).all()), f"{what}: wrote before the buffer"
        assert bool((self.buf[GUARD + self.nbytes:] == CANARY).all()), f"{what}: wrote past the buffer"
        if self.ld > self.cols:
            pad = self.buf[GUARD:GUARD + self.nbytes].view(self.rows, self.ld * self.es)[:, self.cols * self.es:]
            assert bool((pad == CANARY).all()), f"{what}: wrote into the row padding"


@pytest.mark.parametrize("dtype", [torch.bfloat16, torch.int8, torch.float8_e4m3fn, torch.float32])
@pytest.mark.parametrize("shape", [(130, 264), (257, 1040), (1, 16), (384, 4096)])
def test_streaming_kernels_stay_inside_their_outputs(sp, dtype, shape):
    M, K = shape
    if dtype == torch.int8:
        x = torch.randint(-127, 128, (M, K), dtype=torch.int8, device="cuda")
    else:
        x = torch.randn(M, K, device="cuda").to(dtype)
    name = sp._FROM_TORCH[dtype]
    for ld_extra in (0, 16):                          # packed and padded rows (vector kernels both times)
        y = Guarded(M, K, dtype, K + ld_extra)
        sp.prune(x, out=y.t)
        torch.cuda.synchronize()
        y.check("prune")
        for layout in (sp.META_CANONICAL, sp.META_TCGEN05):
            vals = Guarded(M, K // 2, dtype, K // 2 + ld_extra)
            meta = Guarded(1, sp.meta_bytes(name, M, K, layout), torch.uint8)
            sp.compress_into(x, vals.t, meta.t.view(-1), layout=layout)
            torch.cuda.synchronize()
            vals.check("compress values")
            meta.check("compress metadata")
            back = Guarded(M, K, dtype, K + ld_extra)
            sp.decompress(vals.t, meta.t.view(-1), layout=layout, out=back.t)
            torch.cuda.synchronize()
            back.check("decompress")
            if name != "f32":
                p2, v2, m2 = Guarded(M, K, dtype, K + ld_extra), Guarded(M, K // 2, dtype), Guarded(1, meta.cols, torch.uint8)
                sp.prune_compress(x, layout=layout, pruned=p2.t, vals=v2.t, meta=m2.t.view(-1))
                torch.cuda.synchronize()
                p2.check("fused pruned"), v2.check("fused values"), m2.check("fused metadata")


@pytest.mark.parametrize("kind", ["bf16", "i8", "e4m3", "tf32"])
@pytest.mark.parametrize("tile", ["1x128x1", "2x224x1", "2x224x2", "2x240x1"])
def test_gemm_stays_inside_d(sp, force_tile, kind, tile):
    if tile == "2x240x1" and kind != "bf16":
        pytest.skip("240-column tiles are built for the 16-bit kinds")
    M, N, K = 1184, 736, 640
    if kind == "i8":
        A = torch.randint(-127, 128, (M, K), dtype=torch.int8, device="cuda")
        Bt = torch.randint(-127, 128, (N, K), dtype=torch.int8, device="cuda")
        cd, cdt = "i32", torch.int32
    elif kind == "tf32":
        A, Bt, cd, cdt = torch.randn(M, K, device="cuda"), torch.randn(N, K, device="cuda"), "f32", torch.float32
    elif kind == "e4m3":
        A, Bt = torch.randn(M, K, device="cuda").to(torch.float8_e4m3fn), torch.randn(N, K, device="cuda").to(torch.float8_e4m3fn)
        cd, cdt = "bf16", torch.bfloat16
    else:
        A, Bt, cd, cdt = torch.randn(M, K, device="cuda").bfloat16(), torch.randn(N, K, device="cuda").bfloat16(), "bf16", torch.bfloat16
    vals, meta, _ = sp.compress(A)
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    force_tile(tile)
    for ld_extra in (0, 32):
        D = Guarded(M, N, cdt, N + ld_extra)
        sp.gemm(vals, meta, Bt, out=D.t, cd=cd, ws=ws)
        torch.cuda.synchronize()
        assert sp.gemm_status(ws) == 0
        D.check(f"gemm {kind} {tile}")
    if kind in ("bf16", "i8") and tile != "2x240x1":   # (240 columns: row-major outputs only)
        Dt = Guarded(N, M, cdt, M + 32)              # column-major D (M contiguous)
        sp.gemm(vals, meta, Bt, out=Dt.t, cd=cd, cd_col_major=True, ws=ws)
        torch.cuda.synchronize()
        Dt.check(f"gemm {kind} {tile} column-major")


@pytest.mark.parametrize("dtype", [torch.float16, torch.int8])
@pytest.mark.parametrize("shape", [(3, 5, 7, 64), (2, 14, 14, 256), (1, 1, 1, 16)])
def test_im2col_stays_inside_its_output(sp, dtype, shape):
    Nb, H, W, C = shape
    x = torch.randint(-100, 100, shape, device="cuda").to(dtype)
    for ld_extra in (0, 16):
        out = Guarded(Nb * H * W, 9 * C, dtype, 9 * C + ld_extra)
        sp.im2col_nhwc_3x3(x, out=out.t)
        torch.cuda.synchronize()
        out.check("im2col")
        assert torch.equal(out.t.contiguous(), sp.im2col_nhwc_3x3(x))
