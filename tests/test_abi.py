"""Host-side checks that need no GPU: the C-ABI library builds, loads and exports every symbol
that include/cg.h declares; the binding's constants match the header."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "cg.h")).read()
    return sorted(set(re.findall(r"CG_API\s+int\s+(cg_\w+)\s*\(", text)))


def header_enum(name):
    text = open(os.path.join(ROOT, "include", "cg.h")).read()
    m = re.search(rf"\b{name}\s*=\s*([^,/}}\n]+)", text)
    assert m, name
    return eval(m.group(1).strip())   # plain integer expressions such as `1 << 8`


@pytest.fixture(scope="module")
def lib():
    import paper_2604_01489_b200 as cg
    return cg.load()


def test_library_exports_every_declared_symbol(lib):
    names = declared_functions()
    assert len(names) >= 7 and "cg_create" in names and "cg_gemm_epilogue" in names and "cg_destroy" in names
    for name in names:
        assert hasattr(lib, name), f"libcg.so does not export {name}"


def test_binding_lists_the_same_entry_points():
    from paper_2604_01489_b200 import binding
    assert sorted(binding.EXPORTS) == declared_functions()


def test_constants_match_header():
    from paper_2604_01489_b200 import binding
    for name in ("CG_OK", "CG_ERR_INVALID_ARG", "CG_ERR_UNSUPPORTED", "CG_ERR_ARCH", "CG_ERR_CUDA", "CG_ERR_WORKSPACE",
                 "CG_ERR_TIMEOUT", "CG_ACT_NONE", "CG_ACT_RELU", "CG_ACT_GELU_TANH", "CG_ACT_SILU",
                 "CG_ACT_GELU_ERF", "CG_ACT_SIGMOID", "CG_ACT_TANH", "CG_ACT_LEAKY_RELU",
                 "CG_FLAG_B_COLMAJOR", "CG_FLAG_BIAS_BF16"):
        assert getattr(binding, name) == header_enum(name), name
    from cg_inputs import workloads as W
    from oracle import ref
    for mod in (W, ref):                       # the input module and the oracle use the same encoding
        assert mod.ACT_RELU == binding.CG_ACT_RELU and mod.ACT_GELU_TANH == binding.CG_ACT_GELU_TANH
        assert mod.ACT_SILU == binding.CG_ACT_SILU and mod.FLAG_B_COLMAJOR == binding.CG_FLAG_B_COLMAJOR
        assert mod.FLAG_BIAS_BF16 == binding.CG_FLAG_BIAS_BF16
        assert (mod.ACT_GELU_ERF, mod.ACT_SIGMOID, mod.ACT_TANH, mod.ACT_LEAKY_RELU) == (
            binding.CG_ACT_GELU_ERF, binding.CG_ACT_SIGMOID, binding.CG_ACT_TANH, binding.CG_ACT_LEAKY_RELU)


def test_struct_layouts_match_header():
    from paper_2604_01489_b200 import binding
    text = open(os.path.join(ROOT, "include", "cg.h")).read()
    tuning = re.search(r"typedef struct cg_tuning \{(.*?)\} cg_tuning_t;", text, re.S).group(1)
    fields = re.findall(r"int\s+(\w+);", tuning)
    assert [f for f, _ in binding.cg_tuning_t._fields_] == fields
    plan = re.search(r"typedef struct cg_plan_info \{(.*?)\} cg_plan_info_t;", text, re.S).group(1)
    names = []
    for decl in re.findall(r"int\s+([^;]+);", plan):
        names += [n.strip() for n in decl.split(",")]
    assert [f for f, _ in binding.cg_plan_info_t._fields_] == names


def test_null_handle_is_rejected_without_a_gpu(lib):
    assert lib.cg_destroy(None) == 1
    assert lib.cg_set_tuning(None, None) == 1
    assert lib.cg_gemm_epilogue(None, None, None, None, None, None, 8, 8, 8, 1, 1.0, 0.0, 0, None) == 1
    assert lib.cg_create(None, 0, 0) == 1


def test_product_package_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2604_01489_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text, f"{f} mentions the oracle"
