"""The probing framework of Section 3.1 (Steps 2 and 3) run against the CPU oracle as a black box: it must recover the
parameters of Tables 4-7 from input / output behaviour alone.  (The same probes run against the CUDA library in
tests/test_gpu_clfp.py.)"""
import numpy as np
import pytest

import oracle
from paper_2511_10909_b200 import clfp


def oracle_target(key):
    m = oracle.lookup(*key)
    return clfp.Target(m.elem, key[2], lambda A, B, C: oracle.phi_dot_batch(m, A, B, C))


def test_encode_decode_roundtrip():
    for fmt, vals in (("fp16", [1.0, -1.5, 2.0 ** -24, 65504.0, 0.0]), ("bf16", [1.5, 2.0 ** 100, -2.0 ** -133]),
                      ("tf32", [1.0 + 2.0 ** -10, 2.0 ** -149 * 2 ** 13]), ("e4m3", [448.0, 2.0 ** -9, -1.5]),
                      ("e5m2", [57344.0, 2.0 ** -16, 1.5]), ("fp32", [2.0 ** -149, 3.0]), ("fp64", [1e300, -2.0 ** -1074])):
        f = oracle.FORMATS[{"bf16_1k": "bf16"}.get(fmt, fmt)]
        for v in vals:
            w = clfp.encode(fmt, v)
            d = oracle.decode(f, w)
            assert d.cls == oracle.FINITE and (-1) ** d.sign * d.sig * 2.0 ** (d.exp - f.mbits) == v, (fmt, v)
    with pytest.raises(ValueError):
        clfp.encode("e4m3", 1.0 + 2.0 ** -4)
    with pytest.raises(ValueError):
        clfp.encode("fp16", 2.0 ** 16)


def test_predicted_matrices_are_the_tables_of_figure_2():
    from helpers import read_table
    exp = {}
    for row in read_table("fig2_trees.txt"):
        for off, v in enumerate(int(x) for x in row[2:]):
            exp.setdefault(row[0], {})[(int(row[1]), int(row[1]) + 1 + off)] = v
    trees = {name + str(sorted(par.items())): t for name, par, t in clfp.candidate_trees(4)}
    assert clfp.predict_matrix(trees["chain[]"], 4) == exp["a"]
    assert clfp.predict_matrix(trees["pairwise[('P', 4)]"], 4) == exp["b"]
    assert clfp.predict_matrix(trees["fused[('L', 2), ('swamped', False)]"], 4) == exp["c"]
    assert clfp.predict_matrix(trees["fused[('L', 4), ('swamped', True)]"], 4) == exp["d"]


@pytest.mark.parametrize("key,K,want", [
    (("cdna1", "fp32", "fp32"), 4, ("chain", {})),
    (("ampere", "fp64", "fp64"), 4, ("chain", {})),
    (("cdna2", "bf16", "fp32"), 8, ("pairwise", {"P": 2})),
    (("cdna2", "fp16", "fp32"), 8, ("pairwise", {"P": 4})),
    (("cdna1", "bf16", "fp32"), 4, ("fused", {"L": 2, "swamped": False})),
    (("cdna1", "fp16", "fp32"), 8, ("fused", {"L": 4, "swamped": False})),
    (("volta", "fp16", "fp32"), 8, ("fused", {"L": 4, "swamped": True})),
    (("ampere", "tf32", "fp32"), 8, ("fused", {"L": 4, "swamped": True})),
    (("hopper", "bf16", "fp32"), 32, ("fused", {"L": 16, "swamped": True})),
    (("cdna3", "fp16", "fp32"), 16, ("fused", {"L": 8, "swamped": True})),
])
def test_step2_recovers_the_summation_tree(key, K, want):
    t = oracle_target(key)
    trees = clfp.infer_tree(clfp.swamp_matrix(t, K), K)
    assert trees and trees[0] == want, (key, trees)


@pytest.mark.parametrize("key,L,F,rho", [
    (("volta", "fp16", "fp32"), 4, 23, (23, "exact")),
    (("turing", "fp16", "fp16"), 8, 24, (10, "RNE")),
    (("ampere", "bf16", "fp32"), 8, 24, (23, "undetermined")),
    (("hopper", "tf32", "fp32"), 8, 25, (23, "RZ")),
    (("hopper", "fp16", "fp16"), 16, 25, (10, "RNE")),
    (("hopper", "e4m3", "fp32"), 32, 13, (13, "exact")),
    (("ada", "e5m2", "fp16"), 16, 13, (10, "RNE")),
    (("blackwell", "e4m3", "fp32"), 32, 25, (23, "RZ")),
])
def test_step3_recovers_table_4(key, L, F, rho):
    """L_max, F and the conversion rho of the T-FDPA rows, from probes alone."""
    t = oracle_target(key)
    got = clfp.characterise(t, 2 * L)
    assert got["trees"][0] == ("fused", {"L": L, "swamped": True})
    assert got["F"] == F and got["term_rounding"] == "RZ" and got["rho"] == rho, got


def test_exact_fused_sum_has_no_precision_limit():
    t = oracle_target(("cdna1", "fp16", "fp32"))
    assert clfp.fused_precision(t, 4) is None
