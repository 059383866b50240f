"""The five seeded workloads (shapes, layouts, value distributions, epilogues) and a helper for
ad-hoc test problems.  Pure data: no arithmetic of the method lives here.

Activation / flag encoding of the ``act`` argument (shared by the C ABI and the oracle's C ABI):
low byte = activation (0 none, 1 ReLU, 2 GELU-tanh, 3 SiLU, 4 GELU-erf, 5 sigmoid, 6 tanh,
7 leaky ReLU with slope 0.01); bit 8 = B stored column-major
([batch,N,K]); bit 9 = bias is bf16 instead of fp32.
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
    A: np.ndarray                 # uint16 bf16 bits [batch, M, K]
    B: np.ndarray                 # uint16 bf16 bits [batch, K, N] or [batch, N, K] (column-major flag)
    bias: Optional[np.ndarray]    # float32 [N] / uint16 bf16 bits [N] / None
    R: Optional[np.ndarray]       # uint16 bf16 bits [batch, M, N] / None
    seed: int = 0
    meta: dict = field(default_factory=dict)

    @property
    def flops(self) -> float:
        return 2.0 * self.M * self.N * self.K * self.batch

    @property
    def algorithmic_bytes(self) -> int:
        """Each operand read once, D written once."""
        b = 2 * self.batch * (self.M * self.K + self.K * self.N + self.M * self.N)
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
         B=("uniform", 1.0), bias=None, R=None, name="adhoc") -> Problem:
    """Build a problem from distribution specs (see CONFIGS for the format)."""
    colmajor = bool(act & FLAG_B_COLMAJOR)
    a = gen.tensor(seed, gen.TENSOR_A, (batch, M, K), A[0], A[1])
    b = gen.tensor(seed, gen.TENSOR_B, (batch, K, N), B[0], B[1], colmajor_last2=colmajor)
    bias_arr = None
    if bias is not None:
        want = "bf16" if act & FLAG_BIAS_BF16 else "f32"
        dtype = bias[2] if len(bias) > 2 else want
        if dtype != want:
            raise ValueError("bias dtype does not match FLAG_BIAS_BF16")
        bias_arr = gen.tensor(seed, gen.TENSOR_BIAS, (N,), bias[0], bias[1], dtype=dtype)
    r = None
    if R is not None:
        r = gen.tensor(seed, gen.TENSOR_R, (batch, M, N), R[0], R[1])
    return Problem(name=name, M=M, N=N, K=K, batch=batch, alpha=alpha, beta=beta, act=act, A=a, B=b,
                   bias=bias_arr, R=r, seed=seed)


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
