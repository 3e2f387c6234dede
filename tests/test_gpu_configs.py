"""The five benchmark configurations at full size, in the launch configuration bench.py times.

prune / compress / metadata are compared with the oracle in full (bit-exact).  The GEMM is
compared on every element for configurations 1, 2, 3 and 5 (seconds to tens of seconds of oracle
time); for configuration 4 on 64 seeded 128 x 128 output tiles plus the four corner tiles, each
computed by the oracle one by one.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2104_08378_b200 import inputs
from gpu_util import to_device, to_host_bits, to_host_f64
from test_gpu_gemm import check_fp

pytestmark = pytest.mark.gpu
TILE = 128


@pytest.fixture(scope="module")
def sp():
    from paper_2104_08378_b200 import binding
    return binding


def _tiles(cfg, count):
    tm, tn = cfg.M // TILE, cfg.N // TILE
    tiles = inputs.sample_tiles(cfg, count, TILE)
    for corner in [(0, 0), (0, tn - 1), (tm - 1, 0), (tm - 1, tn - 1)]:
        if corner not in tiles:
            tiles.append(corner)
    return tiles


def _check_tiles(cfg, D, vals_ref, meta_ref, Bt, Cm, tiles):
    """tiles: (tm, tn) = one 128 x 128 output tile, or (tm, None) = the whole 128-row band."""
    ab, cd = cfg.ab_type, cfg.cd_type
    for (tm, tn) in tiles:
        rows = (tm * TILE, min(cfg.M, (tm + 1) * TILE))
        cols = (0, cfg.N) if tn is None else (tn * TILE, (tn + 1) * TILE)
        ref = oracle.gemm_sparse(vals_ref, meta_ref, Bt, ab, cfg.alpha, cfg.beta,
                                 Cm if cfg.beta != 0 else None, cd if cfg.beta != 0 else None, rows=rows, cols=cols)
        got = to_host_f64(D[rows[0]:rows[1], cols[0]:cols[1]])
        if ab == "i8":
            assert np.array_equal(got, ref), f"tile {(tm, tn)}"
        else:
            scale = abs(cfg.alpha) * oracle.gemm_abs(vals_ref, meta_ref, Bt, ab, rows=rows, cols=cols)
            beta_c = None
            if cfg.beta != 0:
                beta_c = abs(cfg.beta) * np.abs(oracle.bits_to_float64(
                    np.ascontiguousarray(Cm[rows[0]:rows[1], cols[0]:cols[1]]), cd))
            check_fp(got, ref, scale, beta_c)


def _run_config(sp, cfg, Bt, full_gemm):
    ab, cd = cfg.ab_type, cfg.cd_type
    A = inputs.gen_A(cfg)
    Cm = inputs.gen_C(cfg)
    Ad, Btd = to_device(A, ab), to_device(Bt, ab)
    Cd = to_device(Cm, cd) if Cm is not None else None
    # prune, compress, metadata: bit-exact, in full
    pruned = sp.prune(Ad)
    vals, meta, dropped = sp.compress(pruned, layout=sp.META_TCGEN05, count_dropped=True)
    vals_ref, meta_ref, dropped_ref = oracle.compress(A, ab)
    assert np.array_equal(to_host_bits(pruned), oracle.prune(A, ab))
    assert np.array_equal(to_host_bits(vals), vals_ref)
    assert np.array_equal(meta.cpu().numpy(), oracle.meta_to_operand_order(meta_ref, ab))
    assert int(dropped.item()) == 0
    # the same three outputs from the one-pass entry point (what the benchmark's step launches)
    pruned_f, vals_f, meta_f, dropped_f = sp.prune_compress(Ad, layout=sp.META_TCGEN05, count_dropped=True)
    assert torch.equal(pruned_f.view(torch.uint8), pruned.view(torch.uint8))
    assert torch.equal(vals_f.view(torch.uint8), vals.view(torch.uint8)) and torch.equal(meta_f, meta)
    assert int(dropped_f.item()) == dropped_ref
    del Ad, pruned_f, vals_f, meta_f
    for dense in (False, True):
        if dense:
            D = sp.gemm(pruned, None, Btd, alpha=cfg.alpha, beta=cfg.beta, C=Cd, cd=cd, a_is_dense=True)
        else:
            D = sp.gemm(vals, meta, Btd, alpha=cfg.alpha, beta=cfg.beta, C=Cd, cd=cd)
        torch.cuda.synchronize()
        assert sp.gemm_status(device=D.device) == 0
        if full_gemm:
            tiles = [(i, None) for i in range((cfg.M + TILE - 1) // TILE)]       # every element
        else:
            tiles = _tiles(cfg, 64)
        _check_tiles(cfg, D, vals_ref, meta_ref, Bt, Cm, tiles)
        del D


def test_config1_tiny_f16(sp):
    cfg = inputs.CONFIGS["tiny_f16"]
    _run_config(sp, cfg, inputs.gen_Bt(cfg), full_gemm=True)


def test_config2_bert_ffn_bf16(sp):
    cfg = inputs.CONFIGS["bert_ffn_bf16"]
    _run_config(sp, cfg, inputs.gen_Bt(cfg), full_gemm=True)


def test_config3_int8_linear(sp):
    cfg = inputs.CONFIGS["int8_linear"]
    _run_config(sp, cfg, inputs.gen_Bt(cfg), full_gemm=True)


def test_config4_gpt3_ffn_bf16(sp):
    cfg = inputs.CONFIGS["gpt3_ffn_bf16"]
    _run_config(sp, cfg, inputs.gen_Bt(cfg), full_gemm=False)


def test_config5_resnet_conv_f16(sp):
    cfg = inputs.CONFIGS["resnet_conv_f16"]
    x = inputs.gen_conv_input(cfg)
    Btd = sp.im2col_nhwc_3x3(to_device(x, cfg.ab_type))          # on-device lowering
    Bt = oracle.im2col_nhwc_3x3(x, cfg.ab_type)
    assert np.array_equal(to_host_bits(Btd), Bt)
    del Btd
    _run_config(sp, cfg, Bt, full_gemm=True)
    # the same layer as an implicit GEMM (activation read through im2col-mode TMA, B never built)
    A = inputs.gen_A(cfg)
    vals_ref, meta_ref, _ = oracle.compress(A, cfg.ab_type)
    vals, meta, _ = sp.compress(to_device(A, cfg.ab_type))
    D = sp.conv3x3_nhwc(vals, meta, to_device(x, cfg.ab_type), cd=cfg.cd_type)
    torch.cuda.synchronize()
    assert sp.gemm_status(device=D.device) == 0
    _check_tiles(cfg, D, vals_ref, meta_ref, Bt, None, _tiles(cfg, 64))
