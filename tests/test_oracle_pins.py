"""Pins for the CPU oracle: every check compares it with something other than itself --
closed forms, exact integer cases, a pure-Python triple loop, numpy/torch fp64 library
routines, invariants.  The paper prints no worked numerical example for this path, so no
pin is a printed value."""
import os

import numpy as np
import pytest
import torch

from cg_inputs import gen, workloads as W

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def bits(x):
    """float array (values exactly representable in bf16) -> uint16 bf16 bits."""
    b = gen.f32_to_bf16_bits(np.asarray(x, dtype=np.float32))
    assert np.array_equal(gen.bf16_bits_to_f32(b), np.asarray(x, dtype=np.float32))
    return b


def f64(b):
    return gen.bf16_bits_to_f32(b).astype(np.float64)


def run(oracle, p, **kw):
    return oracle.gemm_epilogue(p.A, p.B, p.bias, p.R, p.M, p.N, p.K, p.batch, p.alpha, p.beta, p.act, **kw)


# ---------------------------------------------------------------- contraction

def test_identity_operands(oracle):
    n = 48
    eye = bits(np.eye(n)).reshape(1, n, n)
    x = gen.tensor(7, gen.TENSOR_B, (1, n, n), "normal", 1.0)
    d64, d16 = oracle.gemm_epilogue(eye, x, None, None, n, n, n, 1, 1.0, 0.0, W.ACT_NONE)
    assert np.array_equal(d64[0], f64(x[0])) and np.array_equal(d16, x)      # I @ B = B
    d64, d16 = oracle.gemm_epilogue(x, eye, None, None, n, n, n, 1, 1.0, 0.0, W.ACT_NONE)
    assert np.array_equal(d64[0], f64(x[0])) and np.array_equal(d16, x)      # A @ I = A


@pytest.mark.parametrize("K", [8, 256, 1024, 4096])
def test_all_ones_gives_K(oracle, K):
    M, N = 5, 16
    ones_a = bits(np.ones((1, M, K)))
    ones_b = bits(np.ones((1, K, N)))
    d64, d16 = oracle.gemm_epilogue(ones_a, ones_b, None, None, M, N, K, 1, 1.0, 0.0, W.ACT_NONE)
    assert np.all(d64 == float(K))
    assert np.all(f64(d16) == float(K))        # these K are exactly representable in bf16


@pytest.mark.parametrize("colmajor", [False, True])
def test_small_integers_exact_vs_int64(oracle, colmajor):
    M, N, K, batch = 37, 24, 200, 3
    act = W.ACT_NONE | (W.FLAG_B_COLMAJOR if colmajor else 0)
    p = W.make(M, N, K, batch, seed=11, act=act, A=("smallint", 1.0), B=("smallint", 1.0))
    a = f64(p.A).astype(np.int64)
    b = f64(p.B).astype(np.int64)
    if colmajor:
        b = np.swapaxes(b, 1, 2)               # stored [batch,N,K] -> logical [batch,K,N]
    want = np.einsum("bmk,bkn->bmn", a, b)
    d64, _ = run(oracle, p)
    assert np.array_equal(d64, want.astype(np.float64))


def naive(p):
    """The definition as a pure-Python m-n-k loop in fp64, libm activations via math."""
    import math
    a, b = f64(p.A), f64(p.B)
    if p.act & W.FLAG_B_COLMAJOR:
        b = np.swapaxes(b, 1, 2)
    bias = None if p.bias is None else (f64(p.bias) if p.act & W.FLAG_BIAS_BF16 else p.bias.astype(np.float64))
    r = None if p.R is None else f64(p.R)
    out = np.zeros((p.batch, p.M, p.N))
    for bb in range(p.batch):
        for m in range(p.M):
            for n in range(p.N):
                s = 0.0
                for k in range(p.K):
                    s += float(a[bb, m, k]) * float(b[bb, k, n])
                t = p.alpha * s + (float(bias[n]) if bias is not None else 0.0)
                kind = p.act & 0xFF
                if kind == W.ACT_RELU:
                    u = t if t > 0 else 0.0
                elif kind == W.ACT_SILU:
                    u = t / (1.0 + math.exp(-t))
                elif kind == W.ACT_GELU_TANH:
                    u = 0.5 * t * (1.0 + math.tanh(math.sqrt(2.0 / math.pi) * (t + 0.044715 * t ** 3)))
                else:
                    u = t
                out[bb, m, n] = u + (p.beta * float(r[bb, m, n]) if p.beta != 0 else 0.0)
    return out


@pytest.mark.parametrize("act", [W.ACT_NONE, W.ACT_RELU, W.ACT_SILU | W.FLAG_B_COLMAJOR,
                                 W.ACT_GELU_TANH | W.FLAG_BIAS_BF16])
def test_tiny_vs_python_triple_loop(oracle, act):
    p = W.make(13, 8, 29, 3, seed=5, act=act, alpha=0.75, beta=-1.5, A=("normal", 1.0), B=("uniform", 1.0),
               bias=("normal", 1.0), R=("normal", 1.0))
    d64, _ = run(oracle, p)
    want = naive(p)
    # same operation order => bit-equal for the linear part; libm vs math.* share the C library
    assert np.allclose(d64, want, rtol=1e-14, atol=1e-15)
    if (act & 0xFF) in (W.ACT_NONE, W.ACT_RELU):
        assert np.array_equal(d64, want)


def test_vs_numpy_fp64_matmul(oracle):
    p = W.make(70, 96, 333 - 5, 2, seed=9, A=("normal", 1.0), B=("normal", 0.05))   # K = 328
    d64, _ = run(oracle, p)
    want = np.matmul(f64(p.A), f64(p.B))
    assert np.allclose(d64, want, rtol=1e-12, atol=1e-12)


def test_vs_torch_fp64_fused_reference(oracle):
    """Library special case: torch CPU float64 matmul + its own gelu(tanh)/silu/relu."""
    for act, fn in ((W.ACT_GELU_TANH, lambda t: torch.nn.functional.gelu(t, approximate="tanh")),
                    (W.ACT_SILU, torch.nn.functional.silu), (W.ACT_RELU, torch.relu),
                    (W.ACT_GELU_ERF, torch.nn.functional.gelu), (W.ACT_SIGMOID, torch.sigmoid), (W.ACT_TANH, torch.tanh),
                    (W.ACT_LEAKY_RELU, lambda t: torch.nn.functional.leaky_relu(t, 0.01))):
        p = W.make(33, 40, 64, 2, seed=21, act=act, alpha=1.25, beta=0.5, A=("normal", 1.0),
                   B=("normal", 0.2), bias=("normal", 1.0), R=("normal", 1.0))
        a, b, r = (torch.from_numpy(f64(x)) for x in (p.A, p.B, p.R))
        t = p.alpha * torch.matmul(a, b) + torch.from_numpy(p.bias.astype(np.float64))
        want = fn(t) + p.beta * r
        d64, _ = run(oracle, p)
        assert np.allclose(d64, want.numpy(), rtol=1e-12, atol=1e-13)


# ---------------------------------------------------------------- indexing / layout

def test_index_valued_inputs_name_their_source(oracle):
    M, N, K = 9, 16, 24
    for k0 in (0, 7, K - 1):
        a = np.zeros((1, M, K)); a[0, :, k0] = 1.0                     # picks row k0 of B
        b = (np.arange(K)[:, None] * 2 + np.arange(N)[None, :] % 2).reshape(1, K, N).astype(np.float64)
        d64, _ = oracle.gemm_epilogue(bits(a), bits(b), None, None, M, N, K, 1, 1.0, 0.0, W.ACT_NONE)
        assert np.array_equal(d64[0], np.broadcast_to(b[0, k0], (M, N)))
    a = np.zeros((1, M, K)); a[0, np.arange(M), np.arange(M)] = np.arange(1, M + 1)   # row m scales B[m]
    d64, _ = oracle.gemm_epilogue(bits(a), bits(b), None, None, M, N, K, 1, 1.0, 0.0, W.ACT_NONE)
    assert np.array_equal(d64[0], b[0, :M] * np.arange(1, M + 1)[:, None])


def test_colmajor_equals_transposed_rowmajor(oracle):
    p = W.make(17, 24, 40, 2, seed=3, act=W.ACT_SILU | W.FLAG_B_COLMAJOR, bias=("normal", 1.0))
    d_col, _ = run(oracle, p)
    b_row = np.ascontiguousarray(np.swapaxes(p.B, 1, 2))
    d_row, _ = oracle.gemm_epilogue(p.A, b_row, p.bias, None, p.M, p.N, p.K, p.batch, p.alpha, p.beta, W.ACT_SILU)
    assert np.array_equal(d_col, d_row)
    # and the generator gives the same LOGICAL values in either storage order
    q = W.make(17, 24, 40, 2, seed=3, act=W.ACT_SILU, bias=("normal", 1.0))
    assert np.array_equal(q.B, b_row)


def test_batch_entries_are_independent(oracle):
    p = W.make(10, 16, 32, 4, seed=8, act=W.ACT_RELU, beta=2.0, bias=("normal", 1.0), R=("normal", 1.0))
    full, _ = run(oracle, p)
    for b in range(p.batch):
        one, _ = oracle.gemm_epilogue(p.A[b:b + 1].copy(), p.B[b:b + 1].copy(), p.bias, p.R[b:b + 1].copy(),
                                      p.M, p.N, p.K, 1, p.alpha, p.beta, p.act)
        assert np.array_equal(one[0], full[b])


def test_rows_and_points_match_full(oracle):
    p = W.make(21, 32, 48, 3, seed=13, act=W.ACT_GELU_TANH | W.FLAG_B_COLMAJOR, alpha=0.5, beta=1.0,
               bias=("normal", 1.0), R=("normal", 1.0))
    full, full16 = run(oracle, p)
    rows = np.array([0, 5, 21, 62], dtype=np.int64)
    r64, r16 = oracle.gemm_epilogue_rows(p.A, p.B, p.bias, p.R, rows, p.M, p.N, p.K, p.batch, p.alpha, p.beta, p.act)
    assert np.array_equal(r64, full.reshape(-1, p.N)[rows]) and np.array_equal(r16, full16.reshape(-1, p.N)[rows])
    idx = np.array([0, 17, 999, p.batch * p.M * p.N - 1], dtype=np.int64)
    p64, p16 = oracle.gemm_epilogue_points(p.A, p.B, p.bias, p.R, idx, p.M, p.N, p.K, p.batch, p.alpha, p.beta, p.act)
    assert np.array_equal(p64, full.reshape(-1)[idx]) and np.array_equal(p16, full16.reshape(-1)[idx])


# ---------------------------------------------------------------- alpha, bias, beta*R

def test_zero_A_leaves_act_of_bias_plus_beta_R(oracle):
    M, N, K = 6, 16, 8
    p = W.make(M, N, K, 1, seed=2, act=W.ACT_RELU, beta=-0.5, bias=("normal", 1.0), R=("normal", 1.0))
    p.A[:] = 0
    d64, _ = run(oracle, p)
    want = np.maximum(p.bias.astype(np.float64), 0.0)[None, :] + (-0.5) * f64(p.R)[0]
    assert np.array_equal(d64[0], want)


def test_bias_not_scaled_by_alpha_and_R_only_by_beta(oracle):
    p = W.make(8, 16, 16, 1, seed=4, A=("smallint", 1.0), B=("smallint", 1.0), bias=("smallint", 1.0),
               R=("smallint", 1.0), alpha=2.0, beta=4.0)
    d64, _ = run(oracle, p)
    ab = np.matmul(f64(p.A), f64(p.B))[0]
    assert np.array_equal(d64[0], 2.0 * ab + p.bias.astype(np.float64)[None, :] + 4.0 * f64(p.R)[0])
    # alpha -> 2*alpha equals doubling A (exact: power of two)
    p2 = W.make(8, 16, 16, 1, seed=4, A=("smallint", 1.0), B=("smallint", 1.0), alpha=4.0)
    p3 = W.make(8, 16, 16, 1, seed=4, A=("smallint", 1.0), B=("smallint", 1.0), alpha=2.0)
    p3.A = bits(2.0 * f64(p3.A))
    assert np.array_equal(run(oracle, p2)[0], run(oracle, p3)[0])


def test_beta_zero_never_reads_R(oracle):
    p = W.make(4, 8, 8, 1, seed=6, R=("normal", 1.0), beta=0.0)
    base, _ = run(oracle, p)
    p.R[:] = 0x7FC0                              # NaNs everywhere
    again, _ = run(oracle, p)
    assert np.array_equal(base, again)
    none, _ = oracle.gemm_epilogue(p.A, p.B, None, None, p.M, p.N, p.K, 1, 1.0, 0.0, p.act)
    assert np.array_equal(base, none)
    with pytest.raises(ValueError):
        oracle.gemm_epilogue(p.A, p.B, None, None, p.M, p.N, p.K, 1, 1.0, 1.0, p.act)


def test_bf16_bias_flag(oracle):
    p = W.make(4, 16, 8, 1, seed=6, act=W.ACT_NONE | W.FLAG_BIAS_BF16, bias=("normal", 1.0))
    assert p.bias.dtype == np.uint16
    d_bf, _ = run(oracle, p)
    d_f32, _ = oracle.gemm_epilogue(p.A, p.B, gen.bf16_bits_to_f32(p.bias), None, p.M, p.N, p.K, 1, 1.0, 0.0, W.ACT_NONE)
    assert np.array_equal(d_bf, d_f32)


# ---------------------------------------------------------------- activations

def test_activation_closed_forms(oracle):
    kinds = {"silu": W.ACT_SILU, "gelu_tanh": W.ACT_GELU_TANH, "gelu_erf": W.ACT_GELU_ERF, "sigmoid": W.ACT_SIGMOID,
             "tanh": W.ACT_TANH, "leaky_relu": W.ACT_LEAKY_RELU}
    n = 0
    with open(os.path.join(GOLDEN, "activation_closed_forms.txt")) as f:
        for line in f:
            if line.startswith("#"):
                continue
            name, x, want = line.split()
            got = oracle.activation(kinds[name], float(x))
            assert abs(got - float(want)) <= 1e-14 * abs(float(want)) + 1e-17, (name, x, got, want)
            n += 1
    assert n == 66
    assert oracle.activation(W.ACT_RELU, -1.0) == 0.0 and oracle.activation(W.ACT_RELU, 2.0) == 2.0
    assert oracle.activation(W.ACT_NONE, -3.25) == -3.25


def test_activation_identities(oracle):
    import math
    for x in np.linspace(-8, 8, 161):
        x = float(x)
        assert abs(oracle.activation(W.ACT_SILU, x) - oracle.activation(W.ACT_SILU, -x) - x) < 1e-14
        assert abs(oracle.activation(W.ACT_GELU_TANH, x) - oracle.activation(W.ACT_GELU_TANH, -x) - x) < 1e-14
        # 1/2 (1 + tanh z) = sigmoid(2 z): GELU-tanh written through one exponential
        z = math.sqrt(2.0 / math.pi) * (x + 0.044715 * x ** 3)
        assert abs(oracle.activation(W.ACT_GELU_TANH, x) - x / (1.0 + math.exp(-2.0 * z))) < 1e-14 * max(1.0, abs(x))
        assert oracle.activation(W.ACT_RELU, x) == max(x, 0.0)
        assert abs(oracle.activation(W.ACT_GELU_ERF, x) - oracle.activation(W.ACT_GELU_ERF, -x) - x) < 1e-14
        assert abs(oracle.activation(W.ACT_SIGMOID, x) + oracle.activation(W.ACT_SIGMOID, -x) - 1.0) < 1e-15
        assert oracle.activation(W.ACT_TANH, x) == -oracle.activation(W.ACT_TANH, -x)
        assert abs(oracle.activation(W.ACT_SILU, x) - x * oracle.activation(W.ACT_SIGMOID, x)) < 1e-14 * max(1.0, abs(x))
        assert abs(2.0 * oracle.activation(W.ACT_SIGMOID, 2.0 * x) - 1.0 - oracle.activation(W.ACT_TANH, x)) < 1e-14
        assert oracle.activation(W.ACT_LEAKY_RELU, x) == (x if x > 0 else 0.01 * x)


# ---------------------------------------------------------------- bf16 rounding

def test_bf16_roundtrip_exhaustive(oracle):
    for h in range(0x10000):
        exp = (h >> 7) & 0xFF
        if exp == 0xFF and (h & 0x7F):          # NaN payloads are not preserved
            continue
        v = oracle.bf16_to_f64(h)
        assert oracle.f64_to_bf16(v) == h, hex(h)
    v = oracle.bf16_to_f64(0x3F80)
    assert v == 1.0 and oracle.bf16_to_f64(0xC000) == -2.0 and oracle.bf16_to_f64(0x0001) == 2.0 ** -133


def test_bf16_ties_to_even_and_neighbours(oracle):
    ulp = 2.0 ** -7                                   # spacing in [1, 2)
    assert oracle.f64_to_bf16(1.0 + ulp / 2) == 0x3F80           # tie -> even (1.0)
    assert oracle.f64_to_bf16(1.0 + 3 * ulp / 2) == 0x3F82       # tie -> even (1 + 2 ulp)
    assert oracle.f64_to_bf16(1.0 + ulp / 2 + 2.0 ** -40) == 0x3F81   # just above the tie
    assert oracle.f64_to_bf16(1.0 + ulp / 2 - 2.0 ** -40) == 0x3F80   # just below
    assert oracle.f64_to_bf16(-(1.0 + ulp / 2)) == 0xBF80
    assert oracle.f64_to_bf16(1.0 + ulp / 2 + 2.0 ** -30) == 0x3F81   # a value fp32 would round to the tie first
    assert oracle.f64_to_bf16(3.5e38) == 0x7F80 and oracle.f64_to_bf16(-3.5e38) == 0xFF80
    big = (2.0 - 2.0 ** -7) * 2.0 ** 127                        # largest finite bf16
    assert oracle.f64_to_bf16(big) == 0x7F7F
    assert oracle.f64_to_bf16(big + 2.0 ** 119) == 0x7F80       # tie at the top rounds to even = inf
    assert oracle.f64_to_bf16(big + 2.0 ** 118) == 0x7F7F
    assert oracle.f64_to_bf16(2.0 ** -134) == 0x0000            # half the smallest subnormal -> even (0)
    assert oracle.f64_to_bf16(2.0 ** -134 * 1.0001) == 0x0001
    assert oracle.f64_to_bf16(0.0) == 0x0000 and oracle.f64_to_bf16(-0.0) == 0x8000


def test_bf16_rounding_vs_torch_on_fp32_values(oracle):
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.normal(size=4000), rng.normal(size=1000) * 1e-30, rng.normal(size=1000) * 1e30,
                        rng.normal(size=500) * 1e-39]).astype(np.float32)
    want = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    got = np.array([oracle.f64_to_bf16(float(v)) for v in x], dtype=np.uint16)
    assert np.array_equal(got, want)


def test_output_bf16_is_rne_of_fp64_result(oracle):
    p = W.make(16, 32, 64, 1, seed=17, act=W.ACT_SILU, bias=("normal", 1.0))
    d64, d16 = run(oracle, p)
    got = np.array([oracle.f64_to_bf16(float(v)) for v in d64.reshape(-1)], dtype=np.uint16)
    assert np.array_equal(got, d16.reshape(-1))
    err = np.abs(f64(d16) - d64)
    assert np.all(err <= 2.0 ** -8 * np.abs(d64) + 1e-300)      # half an ulp, relative 2^-8


def test_rejects_bad_arguments(oracle):
    a = np.zeros((1, 8, 8), dtype=np.uint16)
    with pytest.raises(ValueError):
        oracle.gemm_epilogue(a, a, None, None, 8, 8, 8, 1, 1.0, 0.0, 8)          # unknown activation
    with pytest.raises(ValueError):
        oracle.gemm_epilogue(a, a, None, None, 8, 8, 4, 1, 1.0, 0.0, 0)          # size mismatch
