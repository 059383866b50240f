"""The seeded generator: frozen first values, distribution moments, index purity."""
import os

import numpy as np

from cg_inputs import gen, workloads as W

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def test_first8_frozen():
    seen = 0
    with open(os.path.join(GOLDEN, "generator_first8.txt")) as f:
        for line in f:
            if line.startswith("#"):
                continue
            name, tname, dtype, *hexes = line.split()
            spec = W.CONFIGS[name]
            d = spec[tname]
            tid = {"A": gen.TENSOR_A, "B": gen.TENSOR_B, "bias": gen.TENSOR_BIAS, "R": gen.TENSOR_R}[tname]
            v = gen.tensor(spec["seed"], tid, (8,), d[0], d[1], dtype=dtype)
            bits = v.view(np.uint32) if dtype == "f32" else v
            assert [int(x) for x in bits] == [int(h, 16) for h in hexes], (name, tname)
            seen += 1
    assert seen == 15


def test_moments():
    n = 1_000_000
    idx = np.arange(n, dtype=np.uint64)
    u = gen.values_f64(1, gen.TENSOR_A, idx, "uniform")
    assert u.min() >= -1.0 and u.max() < 1.0
    assert abs(u.mean()) < 3 * (1 / np.sqrt(3)) / np.sqrt(n)
    assert abs(u.std() - 1 / np.sqrt(3)) < 2e-3
    g = gen.values_f64(1, gen.TENSOR_B, idx, "normal", 0.25)
    assert abs(g.mean()) < 3 * 0.25 / np.sqrt(n)
    assert abs(g.std() - 0.25) < 3 * 0.25 / np.sqrt(2 * n) * 1.5
    assert abs(np.mean(g ** 4) / 0.25 ** 4 - 3.0) < 0.05             # Gaussian kurtosis
    s = gen.values_f64(1, gen.TENSOR_A, idx, "smallint")
    assert set(np.unique(s)) == set(float(i) for i in range(-4, 5))


def test_index_purity_and_tensor_independence():
    idx = np.array([5, 1 << 20, (1 << 33) + 7], dtype=np.uint64)
    whole = gen.values_f64(3, gen.TENSOR_A, np.arange(8, dtype=np.uint64), "normal", 1.0)
    assert gen.values_f64(3, gen.TENSOR_A, idx, "normal", 1.0)[0] == whole[5]
    a = gen.values_f64(3, gen.TENSOR_A, idx, "uniform")
    assert not np.array_equal(a, gen.values_f64(3, gen.TENSOR_B, idx, "uniform"))
    assert not np.array_equal(a, gen.values_f64(4, gen.TENSOR_A, idx, "uniform"))
    # chunked, threaded generation equals one-shot generation
    t = gen.tensor(9, gen.TENSOR_R, (3, 700, 1001), "normal", 2.0)
    v = gen.values_f64(9, gen.TENSOR_R, np.arange(t.size, dtype=np.uint64), "normal", 2.0)
    assert np.array_equal(t.reshape(-1), gen.f32_to_bf16_bits(v.astype(np.float32)))


def test_bf16_bits_helpers_roundtrip():
    h = np.arange(0x10000, dtype=np.uint32).astype(np.uint16)
    finite = ((h >> 7) & 0xFF) != 0xFF
    assert np.array_equal(gen.f32_to_bf16_bits(gen.bf16_bits_to_f32(h[finite])), h[finite])


def test_config_shapes():
    p = W.config("cfg1_256_relu")
    assert p.A.shape == (1, 256, 256) and p.bias.dtype == np.float32 and p.R is None
    assert p.flops == 2 * 256 ** 3 and p.algorithmic_bytes == 3 * 256 * 256 * 2 + 1024
    spec = W.CONFIGS["cfg3_skinny_silu"]
    assert spec["act"] & W.FLAG_B_COLMAJOR and spec["M"] == 128
    q = W.make(8, 16, 24, 2, act=W.FLAG_B_COLMAJOR)
    assert q.B.shape == (2, 16, 24)
    rows = W.sample_rows(W.make(8, 8, 8, 3), 5)
    assert rows[0] == 0 and rows[-1] == 23 and len(set(rows.tolist())) == 5
