"""Workaround and design-space exploration (Sections 6.3 and 7): hypothetical (L_max, F, rho) models are bit-exact
against the oracle run with the same parameters, and the sweeps show the trends the paper argues from."""
import dataclasses

import numpy as np
import pytest
import torch

import oracle
from paper_2511_10909_b200 import workloads as wl

pytestmark = pytest.mark.gpu

gu = pytest.importorskip("gpu_util") if torch.cuda.is_available() else None


@pytest.mark.parametrize("key, ov", [
    (("hopper", "e4m3", "fp32"), dict(l_max=8, F=17, rho="RZ-FP32")),
    (("hopper", "e4m3", "fp32"), dict(l_max=64, F=13)),
    (("hopper", "fp16", "fp32"), dict(l_max=32, F=30, rho="RNE-FP32")),
    (("blackwell", "bf16", "fp32"), dict(F=20)),
    (("ampere", "tf32", "fp32"), dict(l_max=2, rho="RNE-FP32")),
    (("cdna3", "fp16", "fp32"), dict(F=20, F2=27)),
])
def test_hypothetical_models_match_the_oracle(key, ov):
    from paper_2511_10909_b200 import mmasim
    M, N, K = 96, 80, 192
    inp = wl.normal_inputs(key[1], key[2], M, N, K, seed=71)
    model = mmasim.Model(*key, **ov)
    D = mmasim.gemm(model, gu.dev(inp["A"]), gu.dev(inp["B"]), gu.dev(inp["C"]))
    torch.cuda.synchronize()
    names = {"l_max": "L", "F": "F", "F2": "F2", "rho": "rho"}
    m = dataclasses.replace(oracle.lookup(*key), **{names[k]: v for k, v in ov.items()})
    pairs = wl.sample_pairs(M, N, 300, seed=72)
    want = oracle.phi_gemm_sampled(m, inp["A"], inp["B"], inp["C"], pairs)
    gu.assert_samples_equal(gu.host_words(D), want, pairs, f"{key} {ov}")


def test_design_sweep_precision_and_block_length():
    """More fractional bits help until the output format's own 24 bits dominate; L_max alone changes little."""
    from paper_2511_10909_b200 import explore
    A, B, C, _, _ = wl.cfg3(512)
    dA, dB, dC = gu.dev(A), gu.dev(B), gu.dev(C)
    rows = explore.design_sweep("hopper", "e4m3", "fp32", dA, dB, dC, F=(None, 17, 21, 25), rho=(None, "RZ-FP32"))
    by = {(r["F"], r["rho"]): r for r in rows}
    assert set(by) == {(F, rho) for F in (13, 17, 21, 25) for rho in ("RZ-E8M13", "RZ-FP32")}
    assert all(r["count"] == 512 * 512 for r in rows)
    err = [by[(F, "RZ-FP32")]["mean_abs"] for F in (13, 17, 21, 25)]
    assert err[0] > 8 * err[1] > 64 * err[2]
    assert err[3] <= err[2]
    # with 13-bit outputs the output conversion dominates, so a more precise sum buys little
    assert by[(25, "RZ-E8M13")]["mean_abs"] > 0.2 * by[(13, "RZ-E8M13")]["mean_abs"]
    rows_l = explore.design_sweep("hopper", "e4m3", "fp32", dA, dB, dC, l_max=(8, 32, 64))
    e = [r["mean_abs"] for r in rows_l]
    assert max(e) < 4 * min(e)


def test_chunk_sweep_promotion_recovers_accuracy():
    """Promotion to FP32 every k_chunk elements: shorter chunks leave fewer low-precision additions in a row."""
    from paper_2511_10909_b200 import explore, mmasim
    A, B, C, sa, sb = wl.cfg3(1024)
    rows = explore.chunk_sweep(mmasim.Model("hopper", "e4m3", "fp32"), gu.dev(A), gu.dev(B), chunks=(0, 32, 128, 512),
                               row_scale=gu.dev(sa), col_scale=gu.dev(sb))
    e = {r["k_chunk"]: r["mean_abs"] for r in rows}
    assert e[32] < e[128] < e[512] < e[0]
    assert e[0] > 2 * e[128]


def test_fp8_through_the_fp16_instruction():
    """The FP16 row of the same architecture sums with F = 25 and writes 24-bit results: far closer to the real result."""
    from paper_2511_10909_b200 import explore
    A, B, C, _, _ = wl.cfg3(512)
    r = explore.fp8_via_fp16("hopper", "e4m3", gu.dev(A), gu.dev(B), gu.dev(C))
    assert r["native"]["count"] == r["via_fp16"]["count"] == 512 * 512
    assert r["native"]["mean_abs"] > 100 * r["via_fp16"]["mean_abs"]
    w = explore.widen_fp8_to_fp16("e4m3", gu.dev(A)).cpu().numpy().view(np.float16).astype(np.float64)
    np.testing.assert_array_equal(w, torch.from_numpy(A).view(torch.float8_e4m3fn).double().numpy())


@pytest.mark.parametrize("key", [("ampere", "fp16", "fp32"), ("blackwell", "mxe4m3", "fp32"), ("blackwell", "nvf4", "fp32"),
                                 ("cdna3", "bf16", "fp32"), ("cdna3", "e4m3", "fp32")], ids=lambda k: "-".join(k))
def test_printed_form_override_matches_the_oracle_and_differs_on_zero_heavy_inputs(key):
    """The `literal_emax` override (maximum exponent over every term, as Algorithms 7-11 print it) against the oracle's
    printed form on inputs with many zero elements and zero or tiny accumulators; the row itself (reading R2, decided by
    the B200) differs from it on some of these outputs, and not at all on inputs without zeros."""
    import oracle
    from paper_2511_10909_b200 import explore, mmasim
    g = wl.rng(77)
    M, N, K = 96, 64, 128
    inp = wl.normal_inputs(key[1], key[2], M, N, K, seed=78)
    A, B = inp["A"].copy(), inp["B"].copy()
    packed = key[1] in ("mxf4", "nvf4")
    zero = g.random(A.shape) < (0.35 if packed else 0.6)
    A[zero] = 0
    A[::3] = 0                                               # whole rows of zeros: blocks without any nonzero product
    # small values beside the zeros, so that a zero term's exponent can exceed every nonzero product's
    if not packed and A.dtype.itemsize == 2:
        A[~zero] = wl.cast((g.standard_normal(A.shape) * 2.0 ** -12).astype(np.float32), key[1])[~zero]
    C = (g.standard_normal((M, N)) * 2.0 ** g.integers(-60, -20, (M, N))).astype(np.float32).view(np.uint32)
    C[g.random((M, N)) < 0.5] = 0
    kw = {k: gu.dev(inp[k]) for k in ("sfa", "sfb") if k in inp}
    r = explore.printed_form_difference(*key, gu.dev(A), gu.dev(B), gu.dev(C), **kw)
    assert mmasim.last_kernel() == "generic"
    lit = gu.host_words(r["printed"])
    pairs = wl.sample_pairs(M, N, 500, seed=79)
    Au, Bu = (gu.unpack_fp4(A), gu.unpack_fp4(B)) if packed else (A, B)
    want = oracle.phi_gemm_sampled(oracle.printed(oracle.lookup(*key)), Au, Bu, C, pairs, SFA=inp.get("sfa"), SFB=inp.get("sfb"))
    gu.assert_samples_equal(lit, want, pairs, f"printed form of {key}")
    if oracle.lookup(*key).family in ("t", "st", "gst"):     # (a block of zero products keeps a tiny accumulator under R2 and
        assert r["differing"] > 0, key                       # truncates it away when the zero products count)
    dense = wl.normal_inputs(key[1], key[2], M, N, K, seed=80)
    if not packed:                                           # no zero elements, nonzero accumulators: nothing changes
        kw = {k: gu.dev(dense[k]) for k in ("sfa", "sfb") if k in dense}
        r2 = explore.printed_form_difference(*key, gu.dev(dense["A"]), gu.dev(dense["B"]), gu.dev(dense["C"]), **kw)
        zeros_in = int((dense["A"].astype(np.int64) << 1 == 0).sum() + (dense["B"].astype(np.int64) << 1 == 0).sum())
        if zeros_in == 0:
            assert r2["differing"] == 0, key
