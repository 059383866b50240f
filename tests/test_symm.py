"""GPU parity of the symmetric forms (CG_FLAG_A_SYMMETRIC, CG_FLAG_B_SYMMETRIC) against the CPU oracle.  The oracle takes the upper
triangle as the matrix; the kernel gets a symmetric operand in which everything it promises not to read -- below the
diagonal, outside the 256 x 256 squares on it -- is a NaN, so a single stray read fails the comparison.
Integer-valued operands with a linear epilogue must match bit for bit; the rest within the bf16 tolerance
|D_gpu - D_ref| <= 1e-2 (|D_ref| + 1), relative Frobenius error <= 5e-3."""
import dataclasses

import numpy as np
import pytest

from cg_inputs import workloads as W

import parity_util as PU

pytestmark = pytest.mark.gpu

SI = ("smallint", 1.0)


@pytest.fixture(scope="module")
def ctx():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    import paper_2604_01489_b200 as cg
    c = cg.Context(0)
    yield c
    c.close()


def poisoned(p):
    if p.act & W.FLAG_B_SYMMETRIC:
        return dataclasses.replace(p, B=W.poison_below_blocks(p.B, 256))
    return dataclasses.replace(p, A=W.poison_below_blocks(p.A, 256))


def check(ctx, oracle, p, exact=False, rows=None, **tuning):
    ctx.set_tuning(reset=True)
    if tuning:
        ctx.set_tuning(**tuning)
    d = PU.run_gpu_ex(ctx, poisoned(p))
    r64, rout = PU.oracle_ex(oracle, p, rows=rows)
    if rows is not None:
        d = d.reshape(p.batch * p.M, p.N)[rows]
    c = PU.compare_ex(d, r64, rout, p.out_dtype)
    assert c["finite"], "an output element was not written, or something below the diagonal was read"
    assert c["ok"], c
    if exact:
        assert c["bit_equal"], c
    return ctx.last_plan()


PLANS = [dict(tile_n=128, cta_group=1), dict(tile_n=256, cta_group=1), dict(tile_n=256, cta_group=2), dict()]
SIZES = [(136, 72, 1), (520, 264, 2), (904, 136, 1), (1024, 512, 1)]       # (M = K, N, batch)


@pytest.mark.parametrize("colmajor", [False, True], ids=["Brow", "Bcol"])
@pytest.mark.parametrize("plan", PLANS, ids=lambda d: "auto" if not d else f"bn{d['tile_n']}cg{d['cta_group']}")
@pytest.mark.parametrize("size", SIZES, ids=lambda s: "x".join(map(str, s)))
def test_integer_operands_bit_exact(ctx, oracle, size, plan, colmajor):
    m, n, batch = size
    act = W.ACT_RELU | W.FLAG_A_SYMMETRIC | (W.FLAG_B_COLMAJOR if colmajor else 0)
    p = W.make(m, n, m, batch, seed=m + n, act=act, alpha=1.0, beta=1.0, A=SI, B=SI, bias=SI, R=SI)
    pl = check(ctx, oracle, p, exact=True, **plan)
    assert pl["latency_kernel"] == 0


@pytest.mark.parametrize("plan", PLANS, ids=lambda d: "auto" if not d else f"bn{d['tile_n']}cg{d['cta_group']}")
def test_normal_operands_with_activation(ctx, oracle, plan):
    p = W.make(776, 392, 776, 2, seed=5, act=W.ACT_SILU | W.FLAG_A_SYMMETRIC | W.FLAG_BIAS_BF16, A=("normal", 1.0),
               B=("normal", 0.05), bias=("normal", 0.5, "bf16"))
    check(ctx, oracle, p, **plan)


@pytest.mark.parametrize("tuning", [dict(tile_n=128, cluster_split=2), dict(tile_n=256, cluster_split=4),
                                    dict(tile_n=128, cta_group=1, num_units=24, dp_units=0),
                                    dict(tile_n=256, cta_group=2, num_units=7, dp_units=2)],
                         ids=["cluster2", "cluster4", "splitk", "streamk-pairs"])
def test_split_plans(ctx, oracle, tuning):
    """K ranges that start anywhere: mirrored and plain blocks inside one unit, units that hold only one kind."""
    p = W.make(1024, 256, 1024, 1, seed=6, act=W.ACT_NONE | W.FLAG_A_SYMMETRIC | W.FLAG_B_COLMAJOR, alpha=0.5, A=SI, B=SI)
    check(ctx, oracle, p, exact=True, **tuning)


def test_skinny_memory_bound_shape_sampled_rows(ctx, oracle):
    """The shape the flag is for: a large symmetric A streamed once against a narrow B."""
    m, n = 4096, 128
    p = W.make(m, n, m, 1, seed=7, act=W.ACT_GELU_TANH | W.FLAG_A_SYMMETRIC | W.FLAG_B_COLMAJOR, A=("normal", 1.0),
               B=("normal", 1.0 / 64.0), bias=("normal", 0.1))
    rows = np.array([0, 1, 127, 128, 255, 256, 1000, 2047, 2048, 3333, 4095], dtype=np.int64)
    pl = check(ctx, oracle, p, rows=rows)
    assert pl["num_units"] >= 32


def test_extensions_combine_with_the_flag(ctx, oracle):
    p = W.make(520, 264, 520, 1, seed=8, act=W.ACT_NONE | W.FLAG_A_SYMMETRIC | W.FLAG_BIAS_PER_ROW, alpha=2.0, A=SI, B=SI,
               bias=SI, row_scale=("pow2",), col_scale=("pow2",), clamp=(-64.0, 64.0), out_dtype=W.OUT_F32)
    check(ctx, oracle, p, exact=True)


def test_row_reduction_with_the_flag(ctx, oracle):
    import torch
    p = W.make(520, 264, 520, 1, seed=9, act=W.ACT_NONE | W.FLAG_A_SYMMETRIC, A=SI, B=SI)
    dev = PU.to_device_ex(poisoned(p))
    out = torch.full((520,), float("nan"), device="cuda")
    ctx.set_tuning(reset=True)
    ctx.gemm_epilogue_ex(dev["A"], dev["B"], None, None, None, 520, 264, 520, 1, 1.0, 0.0, p.act, row_reduce=1, row_out=out)
    ctx.check()
    ref = oracle.gemm_epilogue_reduce(p.A, p.B, None, None, 520, 264, 520, 1, 1.0, 0.0, p.act, 1)[-1]
    assert np.array_equal(out.cpu().numpy().astype(np.float64), ref)          # integers: exact in fp32


def test_error_codes(ctx):
    import paper_2604_01489_b200 as cg
    p = W.make(128, 64, 128, seed=1)
    dev = PU.to_device(p)
    h = ctx.handle
    ctx.set_tuning(reset=True)
    call = lambda M=128, K=128, act=cg.CG_FLAG_A_SYMMETRIC: cg.cg_gemm_epilogue_ex(h, dev["A"], dev["B"], None, None, dev["D"], M, 64, K,
                                                                                 1, 1.0, 0.0, act)
    assert call() == cg.CG_OK
    assert call(M=64) == cg.CG_ERR_INVALID_ARG                                        # not square
    assert call(act=cg.CG_FLAG_A_SYMMETRIC | cg.CG_FLAG_IN_F32 | cg.CG_FLAG_B_COLMAJOR) == cg.CG_ERR_UNSUPPORTED
    assert cg.cg_gemm_epilogue(h, dev["A"], dev["B"], None, None, dev["D"], 128, 64, 128, 1, 1.0, 0.0,
                               cg.CG_FLAG_A_SYMMETRIC) == cg.CG_ERR_INVALID_ARG       # an extended flag
    ctx.set_tuning(tile_n=512, cta_group=2)
    assert call() == cg.CG_ERR_INVALID_ARG                                            # no symmetric form of that tile
    ctx.set_tuning(reset=True)
    ctx.check()


# ---------------------------------------------------------------- symmetric B

SIZES_B = [(72, 136, 1), (264, 520, 2), (136, 904, 1), (512, 1024, 1)]       # (M, N = K, batch)


@pytest.mark.parametrize("colmajor", [False, True], ids=["Brow", "Bcol"])
@pytest.mark.parametrize("plan", PLANS, ids=lambda d: "auto" if not d else f"bn{d['tile_n']}cg{d['cta_group']}")
@pytest.mark.parametrize("size", SIZES_B, ids=lambda s: "x".join(map(str, s)))
def test_symmetric_b_integer_operands_bit_exact(ctx, oracle, size, plan, colmajor):
    m, n, batch = size
    act = W.ACT_RELU | W.FLAG_B_SYMMETRIC | (W.FLAG_B_COLMAJOR if colmajor else 0)
    p = W.make(m, n, n, batch, seed=m + n, act=act, alpha=1.0, beta=1.0, A=SI, B=SI, bias=SI, R=SI)
    pl = check(ctx, oracle, p, exact=True, **plan)
    assert pl["latency_kernel"] == 0


@pytest.mark.parametrize("plan", PLANS, ids=lambda d: "auto" if not d else f"bn{d['tile_n']}cg{d['cta_group']}")
def test_symmetric_b_normal_operands_with_activation(ctx, oracle, plan):
    p = W.make(392, 776, 776, 2, seed=15, act=W.ACT_GELU_TANH | W.FLAG_B_SYMMETRIC | W.FLAG_B_BROADCAST, A=("normal", 1.0),
               B=("normal", 0.05), bias=("normal", 0.5))
    check(ctx, oracle, p, **plan)


@pytest.mark.parametrize("tuning", [dict(tile_n=128, cluster_split=2), dict(tile_n=256, cluster_split=4),
                                    dict(tile_n=128, cta_group=1, num_units=24, dp_units=0),
                                    dict(tile_n=256, cta_group=2, num_units=7, dp_units=2)],
                         ids=["cluster2", "cluster4", "splitk", "streamk-pairs"])
def test_symmetric_b_split_plans(ctx, oracle, tuning):
    p = W.make(256, 1024, 1024, 1, seed=16, act=W.ACT_NONE | W.FLAG_B_SYMMETRIC, alpha=0.5, A=SI, B=SI)
    check(ctx, oracle, p, exact=True, **tuning)


def test_symmetric_b_skinny_memory_bound_shape_sampled_rows(ctx, oracle):
    """The shape the flag pays on: few rows of A against a large symmetric B."""
    m, n = 128, 4096
    p = W.make(m, n, n, 1, seed=17, act=W.ACT_SILU | W.FLAG_B_SYMMETRIC, A=("normal", 1.0), B=("normal", 1.0 / 64.0),
               bias=("normal", 0.1))
    rows = np.array([0, 1, 31, 32, 63, 64, 100, 127], dtype=np.int64)
    pl = check(ctx, oracle, p, rows=rows)
    assert pl["num_units"] > pl["num_tiles"]            # K is split


def test_symmetric_b_error_codes(ctx):
    import paper_2604_01489_b200 as cg
    p = W.make(64, 128, 128, seed=1)
    dev = PU.to_device(p)
    h = ctx.handle
    ctx.set_tuning(reset=True)
    call = lambda N=128, K=128, act=cg.CG_FLAG_B_SYMMETRIC: cg.cg_gemm_epilogue_ex(h, dev["A"], dev["B"], None, None, dev["D"], 64, N, K,
                                                                                 1, 1.0, 0.0, act)
    assert call() == cg.CG_OK
    assert call(N=64) == cg.CG_ERR_INVALID_ARG                                        # not square
    assert call(act=cg.CG_FLAG_B_SYMMETRIC | cg.CG_FLAG_IN_F32 | cg.CG_FLAG_B_COLMAJOR) == cg.CG_ERR_UNSUPPORTED
    assert call(act=cg.CG_FLAG_B_SYMMETRIC | cg.CG_FLAG_A_SYMMETRIC) == cg.CG_ERR_INVALID_ARG     # (64 x 128 A is not square)
    ctx.check()
