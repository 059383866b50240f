"""The five seeded workloads (shapes, layouts, value distributions, epilogues) and a helper for
ad-hoc test problems.  Pure data: no arithmetic of the method lives here.

Activation / flag encoding of the ``act`` argument (shared by the C ABI and the oracle's C ABI):
low byte = activation (0 none, 1 ReLU, 2 GELU-tanh, 3 SiLU, 4 GELU-erf, 5 sigmoid, 6 tanh,
7 leaky ReLU with slope 0.01); bit 8 = B stored column-major
([batch,N,K]); bit 9 = bias is bf16 instead of fp32.  Extended entry point only: bit 10 = the bias
is per output row (length M); bit 11 = one B shared by all batch entries; bit 12 = clamp the
activation's result to [clamp_lo, clamp_hi]; bit 13 = A and B are float32 and multiplied as TF32.  Output dtype codes: 0 bf16, 1 fp16, 2 fp32.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field
from typing import Optional

import numpy as np

from . import gen

ACT_NONE, ACT_RELU, ACT_GELU_TANH, ACT_SILU = 0, 1, 2, 3
ACT_GELU_ERF, ACT_SIGMOID, ACT_TANH, ACT_LEAKY_RELU = 4, 5, 6, 7
FLAG_B_COLMAJOR = 1 << 8
FLAG_BIAS_BF16 = 1 << 9
FLAG_BIAS_PER_ROW = 1 << 10
FLAG_B_BROADCAST = 1 << 11
FLAG_CLAMP = 1 << 12
FLAG_IN_F32 = 1 << 13
FLAG_A_SYMMETRIC = 1 << 14
FLAG_B_SYMMETRIC = 1 << 15
OUT_BF16, OUT_F16, OUT_F32 = 0, 1, 2


@dataclass
class Problem:
    name: str
    M: int
    N: int
    K: int
    batch: int
    alpha: float
    beta: float
    act: int                      # activation | flags
    A: np.ndarray                 # uint16 bf16 bits [batch, M, K] (float32 with FLAG_IN_F32, also B)
    B: np.ndarray                 # uint16 bf16 bits [batch, K, N] or [batch, N, K] (column-major flag)
    bias: Optional[np.ndarray]    # float32 [N] / uint16 bf16 bits [N] / None
    R: Optional[np.ndarray]       # uint16 bf16 bits [batch, M, N] / None
    seed: int = 0
    meta: dict = field(default_factory=dict)
    # extended consumer family (cg_gemm_epilogue_ex); all off by default
    row_scale: Optional[np.ndarray] = None   # float32 [M]
    col_scale: Optional[np.ndarray] = None   # float32 [N]
    clamp_lo: float = 0.0
    clamp_hi: float = 0.0
    out_dtype: int = OUT_BF16

    @property
    def extended(self) -> bool:
        return bool(self.act & (FLAG_BIAS_PER_ROW | FLAG_B_BROADCAST | FLAG_CLAMP | FLAG_IN_F32 | FLAG_A_SYMMETRIC | FLAG_B_SYMMETRIC)) or self.row_scale is not None \
            or self.col_scale is not None or self.out_dtype != OUT_BF16

    @property
    def flops(self) -> float:
        return 2.0 * self.M * self.N * self.K * self.batch

    @property
    def algorithmic_bytes(self) -> int:
        """Each operand read once, D written once."""
        out_bytes = 4 if self.out_dtype == OUT_F32 else 2
        b_entries = 1 if self.act & FLAG_B_BROADCAST else self.batch
        in_bytes = 4 if self.act & FLAG_IN_F32 else 2
        b = in_bytes * (self.batch * self.M * self.K + b_entries * self.K * self.N) + out_bytes * self.batch * self.M * self.N
        for v in (self.row_scale, self.col_scale):
            if v is not None:
                b += v.nbytes
        if self.bias is not None:
            b += self.bias.nbytes
        if self.R is not None and self.beta != 0.0:
            b += self.R.nbytes
        return b


# name -> spec.  dist entries: (distribution, scale[, dtype])
CONFIGS = {
    "cfg1_256_relu": dict(M=256, N=256, K=256, batch=1, seed=0, act=ACT_RELU, alpha=1.0, beta=0.0,
                          A=("uniform", 1.0), B=("uniform", 1.0), bias=("normal", 1.0, "f32"), R=None),
    "cfg2_4096_gelu": dict(M=4096, N=4096, K=4096, batch=1, seed=1, act=ACT_GELU_TANH | FLAG_BIAS_BF16,
                           alpha=1.0, beta=0.0, A=("normal", 1.0 / 64.0), B=("normal", 1.0 / 64.0),
                           bias=("normal", 0.1, "bf16"), R=None),
    "cfg3_skinny_silu": dict(M=128, N=8192, K=8192, batch=1, seed=2, act=ACT_SILU | FLAG_B_COLMAJOR,
                             alpha=1.0, beta=0.0, A=("normal", 1.0), B=("normal", 1.0 / math.sqrt(8192.0)),
                             bias=("zeros", 0.0, "f32"), R=None),
    "cfg4_batched_residual": dict(M=1024, N=1024, K=1024, batch=32, seed=3, act=ACT_NONE, alpha=0.5,
                                  beta=1.0, A=("uniform", 1.0), B=("uniform", 1.0), bias=None,
                                  R=("normal", 1.0)),
    "cfg5_8192_silu": dict(M=8192, N=8192, K=8192, batch=1, seed=4, act=ACT_SILU, alpha=1.0, beta=0.0,
                           A=("normal", 1.0 / math.sqrt(8192.0)), B=("normal", 1.0 / math.sqrt(8192.0)),
                           bias=("normal", 0.02, "f32"), R=None),
}
CONFIG_ORDER = list(CONFIGS)


def make(M, N, K, batch=1, seed=0, act=ACT_NONE, alpha=1.0, beta=0.0, A=("uniform", 1.0),
         B=("uniform", 1.0), bias=None, R=None, name="adhoc", row_scale=None, col_scale=None, clamp=None,
         out_dtype=OUT_BF16) -> Problem:
    """Build a problem from distribution specs (see CONFIGS for the format).  ``row_scale`` /
    ``col_scale``: distribution specs of fp32 vectors ("pow2" draws exact powers of two 2^-2..2^2);
    ``clamp``: (lo, hi), sets FLAG_CLAMP.  With FLAG_A_SYMMETRIC A is made symmetric by mirroring its upper
    triangle (see also ``poison_below_blocks``)."""
    colmajor = bool(act & FLAG_B_COLMAJOR)
    in_dtype = "f32" if act & FLAG_IN_F32 else "bf16"
    a = gen.tensor(seed, gen.TENSOR_A, (batch, M, K), A[0], A[1], dtype=in_dtype)
    if act & FLAG_A_SYMMETRIC:
        if M != K:
            raise ValueError("a symmetric A is square")
        iu = np.triu_indices(M, 1)
        a[:, iu[1], iu[0]] = a[:, iu[0], iu[1]]
    b = gen.tensor(seed, gen.TENSOR_B, (1 if act & FLAG_B_BROADCAST else batch, K, N), B[0], B[1], dtype=in_dtype,
                   colmajor_last2=colmajor)
    if act & FLAG_B_SYMMETRIC:
        if N != K:
            raise ValueError("a symmetric B is square")
        iu = np.triu_indices(N, 1)
        b[:, iu[1], iu[0]] = b[:, iu[0], iu[1]]
    bias_arr = None
    if bias is not None:
        want = "bf16" if act & FLAG_BIAS_BF16 else "f32"
        dtype = bias[2] if len(bias) > 2 else want
        if dtype != want:
            raise ValueError("bias dtype does not match FLAG_BIAS_BF16")
        bias_arr = gen.tensor(seed, gen.TENSOR_BIAS, (M if act & FLAG_BIAS_PER_ROW else N,), bias[0], bias[1], dtype=dtype)
    r = None
    if R is not None:
        r = gen.tensor(seed, gen.TENSOR_R, (batch, M, N), R[0], R[1])

    def scale_vec(spec, tensor_id, n):
        if spec is None:
            return None
        if spec[0] == "pow2":          # exact powers of two: scaling by them commutes with every rounding
            u = gen.tensor(seed, tensor_id, (n,), "uniform", 1.0, dtype="f32")
            return np.exp2(np.floor((u + 1.0) * 2.5) - 2.0).astype(np.float32)
        return gen.tensor(seed, tensor_id, (n,), spec[0], spec[1], dtype="f32")

    lo, hi = clamp if clamp is not None else (0.0, 0.0)
    if clamp is not None:
        act |= FLAG_CLAMP
    return Problem(name=name, M=M, N=N, K=K, batch=batch, alpha=alpha, beta=beta, act=act, A=a, B=b,
                   bias=bias_arr, R=r, seed=seed, row_scale=scale_vec(row_scale, gen.TENSOR_ROW_SCALE, M),
                   col_scale=scale_vec(col_scale, gen.TENSOR_COL_SCALE, N), clamp_lo=float(lo), clamp_hi=float(hi),
                   out_dtype=out_dtype)


def poison_below_blocks(a: np.ndarray, block: int, bits: int = 0x7FC0) -> np.ndarray:
    """Copy of the square matrices ``a`` [batch, M, M] (bf16 bits) in which every element below the diagonal and
    outside the block x block squares on the diagonal is a NaN: what a kernel that honours the symmetric flag
    at that block size never reads."""
    out = a.copy()
    m = a.shape[-1]
    i, k = np.meshgrid(np.arange(m), np.arange(m), indexing="ij")
    out[:, (i // block) > (k // block)] = bits
    return out


def config(name: str) -> Problem:
    spec = dict(CONFIGS[name])
    return make(name=name, **spec)


def sample_rows(p: Problem, count: int, seed: int = 12345) -> np.ndarray:
    """``count`` distinct seeded row ids (b*M + m), always including the first and last row."""
    total = p.batch * p.M
    count = min(count, total)
    rng = np.random.default_rng(seed)
    rows = set([0, total - 1])
    while len(rows) < count:
        rows.add(int(rng.integers(0, total)))
    return np.array(sorted(rows), dtype=np.int64)
