"""CPU-only checks of the library's host side: it loads, exports every declared symbol, its registry agrees
with the paper's tables and with the oracle's independently typed registry, and argument errors are reported."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
from helpers import read_table

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def mm():
    from paper_2511_10909_b200.build import build
    build()
    from paper_2511_10909_b200 import mmasim
    return mmasim


def test_library_exports_every_declared_symbol(mm):
    header = open(os.path.join(ROOT, "include", "mmasim.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    names = set(re.findall(r"\b(mmasim_[a-z_0-9]+)\s*\(", header))
    assert {"mmasim_create_model", "mmasim_gemm", "mmasim_dot_batch", "mmasim_gemm_ex", "mmasim_gemm_host"} <= names
    lib = ctypes.CDLL(mm.library_path())
    for n in names:
        assert hasattr(lib, n), n


def test_registry_matches_paper_tables_and_oracle(mm):
    rows = read_table("registry_tables.txt")
    keys = set()
    for arch, in_fmt, acc, family, L, F, F2, rho_name, P, G, kb in rows:
        num = lambda s: 0 if s == "-" else int(s)
        model = mm.Model(arch, in_fmt, acc)
        assert (model.family, model.l_max, model.F, model.F2, model.P, model.G, model.k_block) == \
               (family, num(L), num(F), num(F2), num(P), num(G), num(kb)), (arch, in_fmt, acc)
        assert model.rho == ("" if rho_name == "-" or family == "e" else rho_name)
        keys.add((arch, in_fmt, acc))
    assert keys == set(mm.model_keys()) == set(oracle.REGISTRY)


def test_unsupported_triples_and_overrides(mm):
    for bad in (("volta", "bf16", "fp32"), ("turing", "tf32", "fp32"), ("hopper", "e2m1", "fp32"),
                ("ada", "mxe4m3", "fp32"), ("cdna1", "fp64", "fp64"), ("cdna3", "fp16", "fp16"),
                ("hopper", "bf16", "fp16"), ("cdna2", "e4m3", "fp32"), ("blackwell", "fp32", "fp32")):
        with pytest.raises(mm.MmasimError):
            mm.Model(*bad)
    assert mm.Model("blackwell", "e4m3", "fp32", b_fmt="e2m1").family == "t"
    with pytest.raises(mm.MmasimError):
        mm.Model("hopper", "e4m3", "fp32", b_fmt="e2m1")
    with pytest.raises(mm.MmasimError):
        mm.Model("hopper", "fp16", "fp32", b_fmt="bf16")
    m = mm.Model("cdna3", "fp16", "fp32", inner_round=1, F=20)
    assert (m.inner_round, m.F) == (1, 20)
    with pytest.raises(mm.MmasimError):
        mm.Model("cdna2", "fp16", "fp32", F=20)


def test_argument_errors_without_a_gpu(mm):
    lib, p = mm._lib, ctypes.c_void_p
    model = mm.Model("hopper", "fp16", "fp32")
    buf = np.zeros(4096, dtype=np.uint8)
    ptr = p(buf.ctypes.data + (-buf.ctypes.data % 16))
    assert lib.mmasim_gemm(None, 4, 4, 16, ptr, ptr, None, ptr, None) == 1
    assert lib.mmasim_gemm(model._h, 4, 4, 16, None, ptr, None, ptr, None) == 1
    assert lib.mmasim_gemm(model._h, 0, 4, 16, ptr, ptr, None, ptr, None) == 3
    assert lib.mmasim_gemm(model._h, 4, 4, 24, ptr, ptr, None, ptr, None) == 3          # 24 % 16 != 0
    assert b"multiple" in lib.mmasim_last_error()
    assert lib.mmasim_gemm(model._h, 4, 4, 8, ptr, ptr, None, ptr, None) != 3           # L = min(K, L_max) = 8
    assert lib.mmasim_gemm(model._h, 4, 4, 16, p(ptr.value + 2), ptr, None, ptr, None) == 4
    assert lib.mmasim_dot_batch(mm.Model("blackwell", "mxe4m3", "fp32")._h, 4, 32, ptr, ptr, None, ptr, None) == 2
    o = mm._make_opts(k_chunk=24)
    assert lib.mmasim_gemm_ex(model._h, 4, 4, 64, ptr, ptr, None, ptr, ctypes.byref(o), None) == 3
    o = mm._make_opts(k_chunk=32)
    assert lib.mmasim_gemm_ex(mm.Model("cdna2", "fp16", "fp32")._h, 4, 4, 64, ptr, ptr, None, ptr, ctypes.byref(o), None) == 2
    # scale factors required / refused
    assert lib.mmasim_gemm(mm.Model("blackwell", "nvf4", "fp32")._h, 4, 4, 64, ptr, ptr, None, ptr, None) == 1
    # a host pointer is either rejected as such (GPU machine) or the CUDA runtime reports that there is no device
    assert lib.mmasim_gemm(model._h, 4, 4, 16, ptr, ptr, None, ptr, None) in (1, 5)


def test_binding_refuses_cpu_tensors(mm):
    import torch
    model = mm.Model("hopper", "fp16", "fp32")
    with pytest.raises(mm.MmasimError):
        mm.gemm(model, torch.zeros((4, 16), dtype=torch.int16), torch.zeros((4, 16), dtype=torch.int16))


def test_product_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2511_10909_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cpp", ".h", ".cuh")):
                text = open(os.path.join(dirpath, f)).read()
                assert not re.search(r"^\s*(from|import)\s+oracle\b", text, flags=re.M), f
                assert "oracle/" not in text and "oracle." not in text, f
    for f in os.listdir(os.path.join(ROOT, "oracle")):
        if f.endswith(".py"):
            assert "paper_2511_10909_b200" not in open(os.path.join(ROOT, "oracle", f)).read()
