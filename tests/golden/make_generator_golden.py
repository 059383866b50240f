"""Writes generator_first8.txt: the first 8 values (as stored bit patterns) of every tensor of
the five workloads, from cg_inputs only.  Freezes the input recipe; calls neither the oracle
nor the CUDA path."""
import os
import sys

import numpy as np

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__)))))
from cg_inputs import gen, workloads as W  # noqa: E402

here = os.path.dirname(os.path.abspath(__file__))
with open(os.path.join(here, "generator_first8.txt"), "w") as f:
    f.write("# config tensor dtype first-8 stored values in hex (logical row-major indices 0..7)\n")
    for name, spec in W.CONFIGS.items():
        seed = spec["seed"]
        for tname, tid in (("A", gen.TENSOR_A), ("B", gen.TENSOR_B), ("bias", gen.TENSOR_BIAS), ("R", gen.TENSOR_R)):
            d = spec[tname]
            if d is None:
                continue
            dtype = d[2] if len(d) > 2 else "bf16"
            v = gen.tensor(seed, tid, (8,), d[0], d[1], dtype=dtype)
            bits = v.view(np.uint32) if dtype == "f32" else v
            f.write(f"{name} {tname} {dtype} " + " ".join(f"{int(x):x}" for x in bits) + "\n")
