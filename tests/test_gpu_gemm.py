"""GPU parity for the sparse GEMM and its dense variant against the CPU oracle, through the C ABI.

Tolerances (floating point): normwise ||D_gpu - D_ref||_F / ||D_ref||_F <= 2e-3 and per element
|err| <= 1e-2 * (|alpha| (|A|.|B|)_ij + |beta| |C_ij|); the reference is the oracle's un-rounded
float64 result.  int8 -> int32 must match bit for bit.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2104_08378_b200 import inputs
from gpu_util import to_device, to_host_f64

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def sp():
    from paper_2104_08378_b200 import binding
    return binding


def _problem(cfg, with_c=None):
    A = inputs.gen_A(cfg)
    Bt = inputs.gen_Bt(cfg)
    Cm = inputs.gen_C(cfg) if with_c is None else with_c
    return A, Bt, Cm


def check_fp(D_gpu, ref, scale, beta_c=None):
    err = np.abs(D_gpu - ref)
    denom = np.linalg.norm(ref)
    rel = np.linalg.norm(err) / denom if denom > 0 else np.linalg.norm(err)
    bound = 1e-2 * (scale + (0 if beta_c is None else beta_c)) + 1e-30
    worst = float((err / bound).max()) if err.size else 0.0
    assert rel <= 2e-3, f"normwise relative error {rel:.3e}"
    assert worst <= 1.0, f"per-element error reaches {worst:.3f} of its bound"


def run_case(sp, cfg, dense=False, cd=None, rows=None, cols=None, alpha=None, beta=None):
    ab = cfg.ab_type
    cd = cd or cfg.cd_type
    alpha = cfg.alpha if alpha is None else alpha
    beta = cfg.beta if beta is None else beta
    A, Bt, Cm = _problem(cfg)
    Cm = None
    vals_ref, meta_ref, _ = oracle.compress(A, ab)
    Ad, Btd = to_device(A, ab), to_device(Bt, ab)
    Cd = None
    if beta != 0:
        if ab == "i8":
            Cm = inputs._matrix(("int8",), "i8", cfg.seed, inputs.TENSOR_C, cfg.N, 0, cfg.M).astype(np.int32)
        else:
            store = cd if cd != "f32" else "bf16"          # fp32 C: bf16-representable values, widened
            Cm = inputs._matrix(("normal", 1.0), store, cfg.seed, inputs.TENSOR_C, cfg.N, 0, cfg.M)
            if cd == "f32":
                Cm = np.ascontiguousarray(oracle.bits_to_float64(Cm, store).astype(np.float32))
        Cd = to_device(Cm, "i32" if ab == "i8" else cd)
    if dense:
        pruned = sp.prune(Ad)
        D = sp.gemm(pruned, None, Btd, alpha=alpha, beta=beta, C=Cd, cd=cd, a_is_dense=True)
    else:
        vals, meta, _ = sp.compress(Ad, layout=sp.META_TCGEN05)
        D = sp.gemm(vals, meta, Btd, alpha=alpha, beta=beta, C=Cd, cd=cd)
    torch.cuda.synchronize()
    assert sp.gemm_status(device=D.device) == 0
    c_dtype = None if Cm is None else ("i32" if ab == "i8" else cd)
    ref = oracle.gemm_sparse(vals_ref, meta_ref, Bt, ab, alpha, beta, Cm if beta != 0 else None, c_dtype,
                             rows=rows, cols=cols)
    r0, r1 = rows or (0, cfg.M)
    c0, c1 = cols or (0, cfg.N)
    got = to_host_f64(D[r0:r1, c0:c1])
    if ab == "i8":
        assert np.array_equal(got, ref)
    else:
        scale = abs(alpha) * oracle.gemm_abs(vals_ref, meta_ref, Bt, ab, rows=rows, cols=cols)
        beta_c = None
        if beta != 0:
            csub = np.ascontiguousarray(Cm[r0:r1, c0:c1])
            beta_c = abs(beta) * np.abs(oracle.bits_to_float64(csub, cd) if cd != "f32" else csub)
        check_fp(got, ref, scale, beta_c)
    return D


TINY = inputs.CONFIGS["tiny_f16"]


@pytest.mark.parametrize("dense", [False, True])
def test_tiny_f16_config(sp, dense):
    run_case(sp, TINY, dense=dense)
    run_case(sp, TINY, dense=dense, cd="f32")


@pytest.mark.parametrize("dense", [False, True])
@pytest.mark.parametrize("shape", [(128, 128, 128), (128, 128, 32), (16, 16, 16), (144, 272, 400),
                                   (384, 640, 1024), (256, 128, 4096)])
def test_bf16_shapes_tiles_and_ragged_tails(sp, dense, shape):
    M, N, K = shape
    cfg = inputs.scaled(inputs.CONFIGS["bert_ffn_bf16"], M=M, N=N, K=K)
    run_case(sp, cfg, dense=dense)


@pytest.mark.parametrize("dense", [False, True])
@pytest.mark.parametrize("shape", [(128, 128, 256), (32, 32, 32), (160, 288, 416), (384, 512, 2048)])
def test_int8_bit_exact(sp, dense, shape):
    M, N, K = shape
    cfg = inputs.scaled(inputs.CONFIGS["int8_linear"], M=M, N=N, K=K)
    run_case(sp, cfg, dense=dense)
    run_case(sp, cfg, dense=dense, beta=1)


def test_alpha_beta_with_c(sp):
    cfg = inputs.scaled(inputs.CONFIGS["gpt3_ffn_bf16"], M=256, N=384, K=512)
    run_case(sp, cfg)                                  # alpha = 1, beta = 1, C bf16
    run_case(sp, cfg, alpha=0.5, beta=-2.0)
    run_case(sp, cfg, alpha=2.0, beta=0.0)
    run_case(sp, cfg, cd="f32", alpha=1.0, beta=1.0)


@pytest.mark.parametrize("dense", [False, True])
@pytest.mark.parametrize("case", [("bf16", 128, 128, 128), ("f16", 144, 272, 400), ("bf16", 512, 672, 1024),
                                  ("bf16", 1024, 9472, 256), ("i8", 160, 288, 416), ("i8", 512, 1344, 1024)])
def test_b_stored_n_contiguous(sp, dense, case):
    """order_b = ROW_MAJOR: the K x N matrix stored row by row (MN-major tensor-core operand)."""
    ab, M, N, K = case
    base = inputs.CONFIGS["int8_linear" if ab == "i8" else ("tiny_f16" if ab == "f16" else "bert_ffn_bf16")]
    cfg = inputs.scaled(base, M=M, N=N, K=K)
    A, Bt = inputs.gen_A(cfg), inputs.gen_Bt(cfg)
    vals_ref, meta_ref, _ = oracle.compress(A, ab)
    Ad = to_device(A, ab)
    Bkn = to_device(np.ascontiguousarray(Bt.T), ab)          # [K, N], N contiguous
    cd = "i32" if ab == "i8" else "f32"
    if dense:
        D = sp.gemm(sp.prune(Ad), None, Bkn, cd=cd, a_is_dense=True, b_row_major=True)
    else:
        vals, meta, _ = sp.compress(Ad)
        D = sp.gemm(vals, meta, Bkn, cd=cd, b_row_major=True)
    torch.cuda.synchronize()
    assert sp.gemm_status(device=D.device) == 0
    rows, cols = (0, min(M, 256)), (max(0, N - 320), N)      # a window keeps the oracle quick
    ref = oracle.gemm_sparse(vals_ref, meta_ref, Bt, ab, rows=rows, cols=cols)
    got = to_host_f64(D[rows[0]:rows[1], cols[0]:cols[1]])
    if ab == "i8":
        assert np.array_equal(got, ref)
    else:
        check_fp(got, ref, oracle.gemm_abs(vals_ref, meta_ref, Bt, ab, rows=rows, cols=cols))


@pytest.mark.parametrize("case", [("bf16", "bf16", 272, 464, 528, 1.0), ("f16", "f32", 128, 160, 256, -0.5),
                                  ("i8", "i32", 288, 352, 512, 1), ("bf16", "bf16", 1024, 9472, 256, 0.0)])
def test_c_and_d_stored_m_contiguous(sp, case):
    """order_c = order_d = COL_MAJOR: D^T ([N, M], the [tokens, out_features] layout)."""
    ab, cd, M, N, K, beta = case
    base = inputs.CONFIGS["int8_linear" if ab == "i8" else "bert_ffn_bf16"]
    cfg = inputs.scaled(base, M=M, N=N, K=K)
    if ab == "f16":
        cfg = inputs.scaled(inputs.CONFIGS["tiny_f16"], M=M, N=N, K=K)
    A, Bt = inputs.gen_A(cfg), inputs.gen_Bt(cfg)
    vals_ref, meta_ref, _ = oracle.compress(A, ab)
    Cm = Cd = None
    if beta != 0:
        if ab == "i8":
            Cm = inputs._matrix(("int8",), "i8", 5, inputs.TENSOR_C, N, 0, M).astype(np.int32)
        else:
            Cm = inputs._matrix(("normal", 1.0), "bf16", 5, inputs.TENSOR_C, N, 0, M)
            if cd == "f32":
                Cm = np.ascontiguousarray(oracle.bits_to_float64(Cm, "bf16").astype(np.float32))
        Cd = to_device(np.ascontiguousarray(Cm.T), cd)           # [N, M]
    vals, meta, _ = sp.compress(to_device(A, ab))
    Dt = sp.gemm(vals, meta, to_device(Bt, ab), alpha=1 if ab == "i8" else 2.0, beta=beta, C=Cd, cd=cd,
                 cd_col_major=True)
    torch.cuda.synchronize()
    assert Dt.shape == (N, M)
    alpha = 1 if ab == "i8" else 2.0
    rows, cols = (0, min(M, 288)), (max(0, N - 352), N)
    ref = oracle.gemm_sparse(vals_ref, meta_ref, Bt, ab, alpha, beta, Cm, cd if Cm is not None else None,
                             rows=rows, cols=cols)
    got = to_host_f64(Dt.t()[rows[0]:rows[1], cols[0]:cols[1]])
    if ab == "i8":
        assert np.array_equal(got, ref)
    else:
        scale = abs(alpha) * oracle.gemm_abs(vals_ref, meta_ref, Bt, ab, rows=rows, cols=cols)
        beta_c = None
        if Cm is not None:
            csub = np.ascontiguousarray(Cm[rows[0]:rows[1], cols[0]:cols[1]])
            beta_c = abs(beta) * np.abs(oracle.bits_to_float64(csub, cd) if cd != "f32" else csub)
        check_fp(got, ref, scale, beta_c)


@pytest.mark.parametrize("cd", ["bf16", "f16", "f32", "i8"])
@pytest.mark.parametrize("layout", ["row", "col"])
def test_int8_dequant_epilogue(sp, cd, layout):
    """sp24_gemm_i8_dequant: float outputs within tolerance of the fp64 oracle, int8 codes bit-exact."""
    cfg = inputs.scaled(inputs.CONFIGS["int8_linear"], M=416, N=608, K=1024)
    M, N, K = cfg.M, cfg.N, cfg.K
    A, Bt = inputs.gen_A(cfg), inputs.gen_Bt(cfg)
    vals_ref, meta_ref, _ = oracle.compress(A, "i8")
    acc = oracle.gemm_sparse(vals_ref, meta_ref, Bt, "i8")
    rng = np.random.default_rng(17)
    rs = (rng.uniform(0.5, 2.0, size=M) / (127.0 * 127.0 * np.sqrt(K / 2) / 3)).astype(np.float32)
    bias = rng.normal(scale=0.5, size=M).astype(np.float32)
    out_scale = 2.5 / 127.0
    vals, meta, _ = sp.compress(to_device(A, "i8"))
    for relu in (False, True):
        D = sp.gemm_i8_dequant(vals, meta, to_device(Bt, "i8"), torch.from_numpy(rs).cuda(),
                               bias=torch.from_numpy(bias).cuda(), relu=relu, out_scale=out_scale, cd=cd,
                               cd_col_major=(layout == "col"))
        torch.cuda.synchronize()
        got = D.t() if layout == "col" else D
        f_ref, q_ref = oracle.dequant(acc, rs, bias, relu=relu, out_scale=out_scale)
        if cd == "i8":
            assert np.array_equal(got.cpu().numpy(), q_ref)
        else:
            err = np.abs(to_host_f64(got) - f_ref)
            tol = {"bf16": 2.0 ** -8, "f16": 2.0 ** -11, "f32": 2.0 ** -22}[cd]
            bound = tol * (np.abs(rs.astype(np.float64))[:, None] * np.abs(acc) + np.abs(bias)[:, None]) + 1e-30
            assert (err <= bound).all(), float((err / bound).max())
    # no bias, fp32 out, scale 1: the integer accumulator itself while it is exactly representable
    D = sp.gemm_i8_dequant(vals, meta, to_device(Bt, "i8"), torch.ones(M, device="cuda"), cd="f32")
    torch.cuda.synchronize()
    assert np.array_equal(to_host_f64(D), acc.astype(np.float32).astype(np.float64))


@pytest.mark.parametrize("case", [("f16", 8, 14, 14, 128, 256), ("bf16", 5, 8, 20, 256, 144), ("i8", 8, 14, 14, 256, 288),
                                  ("f16", 40, 14, 14, 128, 512)])
@pytest.mark.parametrize("dense", [False, True])
def test_implicit_conv3x3_matches_im2col_gemm(sp, case, dense):
    """sp24_conv3x3_nhwc reads the activation through im2col-mode TMA: same result as the oracle's
    explicit im2col followed by its sparse GEMM; NHWC output checked too."""
    ab, Nb, H, W, Cin, Kout = case
    dist = ("int8",) if ab == "i8" else ("relu_normal", 1.0)
    x = inputs._matrix(dist, ab, 21, 1, H * W * Cin, 0, Nb).reshape(Nb, H, W, Cin)
    wdist = ("int8",) if ab == "i8" else ("normal", float(np.sqrt(2.0 / (9 * Cin))))
    A = inputs._matrix(wdist, ab, 21, 0, 9 * Cin, 0, Kout)
    Bt = oracle.im2col_nhwc_3x3(np.ascontiguousarray(x), ab)
    vals_ref, meta_ref, _ = oracle.compress(A, ab)
    N = Nb * H * W
    cols = (max(0, N - 400), N)
    rows = (0, min(Kout, 160))
    ref = oracle.gemm_sparse(vals_ref, meta_ref, Bt, ab, rows=rows, cols=cols)
    ref0 = oracle.gemm_sparse(vals_ref, meta_ref, Bt, ab, rows=rows, cols=(0, 300))
    Ad, xd = to_device(A, ab), to_device(x, ab)
    cd = "i32" if ab == "i8" else "f32"
    for nhwc in (False, True):
        if dense:
            D = sp.conv3x3_nhwc(sp.prune(Ad), None, xd, cd=cd, a_is_dense=True, nhwc_out=nhwc)
        else:
            vals, meta, _ = sp.compress(Ad)
            D = sp.conv3x3_nhwc(vals, meta, xd, cd=cd, nhwc_out=nhwc)
        torch.cuda.synchronize()
        assert sp.gemm_status(device=D.device) == 0
        Dm = D.t() if nhwc else D
        for (c0, c1), want in ((cols, ref), ((0, 300), ref0)):
            got = to_host_f64(Dm[rows[0]:rows[1], c0:c1])
            if ab == "i8":
                assert np.array_equal(got, want)
            else:
                check_fp(got, want, oracle.gemm_abs(vals_ref, meta_ref, Bt, ab, rows=rows, cols=(c0, c1)))


@pytest.mark.parametrize("dims", [(384, 448, 512), (20000, 288, 128)])
def test_pipeline_host_entry_point(sp, dims):
    """sp24_pipeline_host: host buffers in, compress + GEMM on the device, D back in a host buffer.
    The second case is large enough for the row-band pipeline (two bands, the last one ragged); it
    runs twice in a row so that the second call's copies follow the first call's on both streams."""
    import ctypes
    cfg = inputs.scaled(inputs.CONFIGS["gpt3_ffn_bf16"], M=dims[0], N=dims[1], K=dims[2])
    M, N, K = cfg.M, cfg.N, cfg.K
    A, Bt, Cm = inputs.gen_A(cfg), inputs.gen_Bt(cfg), inputs.gen_C(cfg)
    hA, hB, hC = (torch.from_numpy(a.view(np.int16)).pin_memory() for a in (A, Bt, Cm))
    hD = torch.empty((M, N), dtype=torch.int16).pin_memory()
    dA = torch.empty((M, K), dtype=torch.bfloat16, device="cuda")
    dV = torch.empty((M, K // 2), dtype=torch.bfloat16, device="cuda")
    dM = torch.empty(sp.meta_bytes("bf16", M, K), dtype=torch.uint8, device="cuda")
    dB = torch.empty((N, K), dtype=torch.bfloat16, device="cuda")
    dC = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    dD = torch.empty((M, N), dtype=torch.bfloat16, device="cuda")
    ws = torch.zeros(256, dtype=torch.uint8, device="cuda")
    desc = sp.make_desc("bf16", "bf16", M, N, K, K // 2, K, N, N)
    al, be = ctypes.c_float(1.0), ctypes.c_float(1.0)
    vp = lambda t: ctypes.c_void_p(t.data_ptr())  # noqa: E731
    for _ in range(2):
        st = sp.lib.sp24_pipeline_host(ctypes.byref(desc), ctypes.byref(al), vp(hA), vp(hB), ctypes.byref(be), vp(hC),
                                       vp(hD), vp(dA), vp(dV), vp(dM), vp(dB), vp(dC), vp(dD), vp(ws), 256,
                                       torch.cuda.current_stream().cuda_stream)
        assert st == 0
    torch.cuda.synchronize()
    assert sp.gemm_status(ws) == 0
    vals_ref, meta_ref, _ = oracle.compress(A, "bf16")
    ref = oracle.gemm_sparse(vals_ref, meta_ref, Bt, "bf16", 1.0, 1.0, Cm, "bf16")
    got = oracle.bits_to_float64(hD.numpy().view(np.uint16), "bf16")
    check_fp(got, ref, oracle.gemm_abs(vals_ref, meta_ref, Bt, "bf16"), np.abs(oracle.bits_to_float64(Cm, "bf16")))


def test_leading_dimensions_larger_than_the_matrices(sp):
    """Every operand as a window of a wider allocation (lda, ldb, ldc, ldd > logical width)."""
    cfg = inputs.scaled(inputs.CONFIGS["gpt3_ffn_bf16"], M=272, N=464, K=528)
    M, N, K = cfg.M, cfg.N, cfg.K
    A, Bt, Cm = inputs.gen_A(cfg), inputs.gen_Bt(cfg), inputs.gen_C(cfg)
    vals_ref, meta_ref, _ = oracle.compress(A, "bf16")
    vals_t, meta, _ = sp.compress(to_device(A, "bf16"))
    pad = lambda t, extra: torch.nn.functional.pad(t.view(torch.int16), (0, extra)).view(t.dtype)  # noqa: E731
    vals_w = pad(vals_t, 24)[:, :K // 2]                      # lda = K/2 + 24
    Bt_w = pad(to_device(Bt, "bf16"), 40)[:, :K]              # ldb = K + 40
    C_w = pad(to_device(Cm, "bf16"), 16)[:, :N]               # ldc = N + 16
    D_full = torch.full((M, N + 48), 7.0, dtype=torch.bfloat16, device="cuda")
    D_w = D_full[:, :N]                                       # ldd = N + 48
    sp.gemm(vals_w, meta, Bt_w, alpha=1.0, beta=1.0, C=C_w, out=D_w)
    torch.cuda.synchronize()
    ref = oracle.gemm_sparse(vals_ref, meta_ref, Bt, "bf16", 1.0, 1.0, Cm, "bf16")
    scale = oracle.gemm_abs(vals_ref, meta_ref, Bt, "bf16")
    check_fp(to_host_f64(D_w), ref, scale, np.abs(oracle.bits_to_float64(Cm, "bf16")))
    assert torch.all(D_full[:, N:] == 7.0)                    # nothing written past column N
    # C aliasing D (in-place accumulate)
    D2 = to_device(Cm, "bf16").clone()
    sp.gemm(vals_t, meta, to_device(Bt, "bf16"), alpha=1.0, beta=1.0, C=D2, out=D2)
    torch.cuda.synchronize()
    check_fp(to_host_f64(D2), ref, scale, np.abs(oracle.bits_to_float64(Cm, "bf16")))


def test_identity_b_returns_decompressed_a(sp):
    """B = I: the sparse GEMM must reproduce prune(A) exactly (every selected index is exercised)."""
    for ab, K in (("f16", 256), ("bf16", 384), ("i8", 512)):
        M = 256
        A = inputs._matrix(("int8",) if ab == "i8" else ("normal", 1.0), ab, 11, 0, K, 0, M)
        if ab == "i8":
            A = np.clip(A, -127, 127)
        eye = inputs.to_storage(np.eye(K), ab)
        vals, meta, _ = sp.compress(to_device(A, ab))
        D = sp.gemm(vals, meta, to_device(eye, ab), cd="i32" if ab == "i8" else "f32")
        torch.cuda.synchronize()
        expect = oracle.bits_to_float64(oracle.prune(A, ab), ab)
        assert np.array_equal(to_host_f64(D), expect)


def test_rejects_bad_arguments(sp):
    a = torch.zeros((16, 8), dtype=torch.float16, device="cuda")
    m = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    bt = torch.zeros((16, 16), dtype=torch.float16, device="cuda")
    with pytest.raises(sp.Sp24Error):                   # N not a multiple of 16
        sp.gemm(a, m, torch.zeros((8, 16), dtype=torch.float16, device="cuda"))
    with pytest.raises(sp.Sp24Error):                   # int8 alpha != 1
        sp.gemm(torch.zeros((32, 16), dtype=torch.int8, device="cuda"), m,
                torch.zeros((32, 32), dtype=torch.int8, device="cuda"), alpha=2)
    with pytest.raises(sp.Sp24Error):                   # beta != 0 without C
        sp.gemm(a, m, bt, beta=1.0)
    out = sp.gemm(torch.zeros((0, 8), dtype=torch.float16, device="cuda"), m, bt)
    assert out.shape == (0, 16)


@pytest.mark.parametrize("ab", ["bf16", "i8"])
def test_shards_of_tokens_or_rows_give_the_bits_of_the_full_product(sp, ab):
    """Splitting N (tokens, the multi-GPU sharding) or M (the row bands of the host pipeline) must not
    change a single bit of the result, although the shards run on other tile shapes than the full
    problem: every output element is accumulated over K in the same order whatever tile computes it."""
    M, N, K = 2048, 4096, 1024
    cfg = inputs.scaled(inputs.CONFIGS["int8_linear" if ab == "i8" else "bert_ffn_bf16"], M=M, N=N, K=K)
    A, Bt = to_device(inputs.gen_A(cfg), ab), to_device(inputs.gen_Bt(cfg), ab)
    vals, meta, _ = sp.compress(A)
    cd = "i32" if ab == "i8" else "bf16"
    full = sp.gemm(vals, meta, Bt, cd=cd)
    desc = sp.make_desc(ab, cd, M, N, K, K // 2, K, N, N)
    plans = {sp.gemm_plan(desc)}
    for n0, n1 in ((0, 256), (256, 1280), (1280, N)):                      # token shards of unequal size
        part = sp.gemm(vals, meta, Bt[n0:n1], cd=cd)
        plans.add(sp.gemm_plan(sp.make_desc(ab, cd, M, n1 - n0, K, K // 2, K, n1 - n0, n1 - n0)))
        assert torch.equal(part.view(torch.uint8), full[:, n0:n1].contiguous().view(torch.uint8))
    for m0, m1 in ((0, 128), (128, 1152), (1152, M)):                       # row bands (128-row metadata blocks)
        mv, mm, _ = sp.compress(A[m0:m1])
        part = sp.gemm(mv, mm, Bt, cd=cd)
        assert torch.equal(part.view(torch.uint8), full[m0:m1].view(torch.uint8))
    torch.cuda.synchronize()
    assert len(plans) > 1                                                   # the shards did take other tile shapes
