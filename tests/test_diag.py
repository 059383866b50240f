"""Structured matmul C = diag(d) @ B: pins for the oracle (CPU) and GPU parity through the C ABI."""
import numpy as np
import pytest

from cg_inputs import gen, workloads as W


def f64(b):
    return gen.bf16_bits_to_f32(b).astype(np.float64)


# ---------------------------------------------------------------- oracle pins (no GPU)

def test_oracle_diag_identity_powers_of_two_and_numpy(oracle):
    M, N = 37, 24
    B = gen.tensor(3, gen.TENSOR_B, (M, N), "normal", 1.0)
    c64, c16 = oracle.diag_matmul(np.ones(M, dtype=np.float32), B)
    assert np.array_equal(c16, B) and np.array_equal(c64, f64(B))                       # diag(1) = I
    d = np.exp2(np.arange(M) % 7 - 3).astype(np.float32)
    c64, c16 = oracle.diag_matmul(d, B)
    assert np.array_equal(c64, f64(B) * d[:, None].astype(np.float64))                  # exact scaling, row by row
    assert np.array_equal(gen.bf16_bits_to_f32(c16), gen.bf16_bits_to_f32(B) * d[:, None])
    d = gen.tensor(4, gen.TENSOR_ROW_SCALE, (M,), "normal", 1.0, dtype="f32")
    c64, _ = oracle.diag_matmul(d, B)
    assert np.array_equal(c64, np.einsum("i,ij->ij", d.astype(np.float64), f64(B)))
    Bf = gen.tensor(5, gen.TENSOR_B, (M, N), "normal", 1.0, dtype="f32")
    c64, c32 = oracle.diag_matmul(d, Bf, out_dtype=W.OUT_F32)
    assert np.array_equal(c32, d[:, None] * Bf)                                         # fp32 x fp32, one rounding = numpy's
    assert np.array_equal(c64, d.astype(np.float64)[:, None] * Bf.astype(np.float64))


def test_oracle_diag_equals_the_dense_product_with_diag_matrix(oracle):
    """The definition: the (pinned) GEMM oracle fed A = diag(d) gives the same matrix."""
    M, N = 29, 16
    d16 = gen.tensor(6, gen.TENSOR_ROW_SCALE, (M,), "normal", 1.0)                      # bf16 bits, so that diag(d) is a bf16 matrix
    d = gen.bf16_bits_to_f32(d16)
    B = gen.tensor(7, gen.TENSOR_B, (M, N), "normal", 1.0)
    A = np.zeros((1, M, M), dtype=np.uint16)
    A[0, np.arange(M), np.arange(M)] = d16
    g64, g16 = oracle.gemm_epilogue(A, B.reshape(1, M, N), None, None, M, N, M, 1, 1.0, 0.0, W.ACT_NONE)
    c64, c16 = oracle.diag_matmul(d, B)
    assert np.array_equal(g64[0], c64) and np.array_equal(g16[0], c16)


# ---------------------------------------------------------------- GPU parity

@pytest.fixture(scope="module")
def ctx():
    import torch
    if not torch.cuda.is_available():
        pytest.fail("GPU tests need a CUDA device")
    import paper_2604_01489_b200 as cg
    c = cg.Context(0)
    yield c
    c.close()


@pytest.mark.gpu
@pytest.mark.parametrize("shape", [(1, 8), (37, 24), (1000, 4104), (4096, 2048), (70000, 8)], ids=lambda s: "x".join(map(str, s)))
@pytest.mark.parametrize("dtype", [W.OUT_BF16, W.OUT_F32], ids=["bf16", "f32"])
def test_gpu_diag_matmul(ctx, oracle, shape, dtype):
    import torch
    M, N = shape
    d = gen.tensor(M, gen.TENSOR_ROW_SCALE, (M,), "normal", 1.0, dtype="f32")
    if dtype == W.OUT_F32:
        B = gen.tensor(N, gen.TENSOR_B, (M, N), "normal", 1.0, dtype="f32")
        Bd = torch.from_numpy(B).cuda()
    else:
        B = gen.tensor(N, gen.TENSOR_B, (M, N), "normal", 1.0)
        Bd = torch.from_numpy(B.view(np.int16)).cuda().view(torch.bfloat16)
    Cd = torch.full_like(Bd, float("nan"))
    ctx.diag_matmul(torch.from_numpy(d).cuda(), Bd, Cd, M, N, dtype)
    ctx.check()
    c64, cout = oracle.diag_matmul(d, B, out_dtype=dtype)
    if dtype == W.OUT_F32:
        assert np.array_equal(Cd.cpu().numpy(), cout)                                   # one IEEE rounding on both sides
    else:
        got = Cd.view(torch.int16).cpu().numpy().view(np.uint16)
        # fp32 product, then bf16: a double rounding that can differ from the oracle's single one by one bf16 ulp
        diff = np.abs(got.astype(np.int32) - cout.astype(np.int32))
        assert diff.max() <= 1 and np.mean(diff != 0) < 1e-3
        assert np.all(np.abs(gen.bf16_bits_to_f32(got).astype(np.float64) - c64) <= 1e-2 * (np.abs(c64) + 1.0))
        d2 = gen.bf16_bits_to_f32(gen.f32_to_bf16_bits(d))                              # bf16-representable scales: exact products
        ctx.diag_matmul(torch.from_numpy(d2).cuda(), Bd, Cd, M, N, dtype)
        _, c2 = oracle.diag_matmul(d2, B, out_dtype=dtype)
        assert np.array_equal(Cd.view(torch.int16).cpu().numpy().view(np.uint16), c2)


@pytest.mark.gpu
def test_gpu_diag_in_place_and_error_codes(ctx, oracle):
    import torch
    import paper_2604_01489_b200 as cg
    M, N = 300, 264
    d = gen.tensor(1, gen.TENSOR_ROW_SCALE, (M,), "normal", 1.0, dtype="f32")
    B = gen.tensor(2, gen.TENSOR_B, (M, N), "normal", 1.0, dtype="f32")
    Bd = torch.from_numpy(B).cuda()
    dd = torch.from_numpy(d).cuda()
    ctx.diag_matmul(dd, Bd, Bd, M, N, W.OUT_F32)                                        # C aliases B
    ctx.check()
    assert np.array_equal(Bd.cpu().numpy(), oracle.diag_matmul(d, B, out_dtype=W.OUT_F32)[1])
    h = ctx.handle
    assert cg.cg_diag_matmul(h, None, Bd, Bd, M, N, W.OUT_F32) == cg.CG_ERR_INVALID_ARG
    assert cg.cg_diag_matmul(h, dd, Bd, Bd, 0, N, W.OUT_F32) == cg.CG_ERR_INVALID_ARG
    assert cg.cg_diag_matmul(h, dd, Bd, Bd, M, N, W.OUT_F16) == cg.CG_ERR_INVALID_ARG
    assert cg.cg_diag_matmul(h, dd, Bd, Bd, M, 262, W.OUT_F32) == cg.CG_ERR_UNSUPPORTED    # not whole 16-byte vectors
    assert cg.cg_diag_matmul(h, dd, Bd.data_ptr() + 4, Bd, M, N, W.OUT_F32) == cg.CG_ERR_UNSUPPORTED
