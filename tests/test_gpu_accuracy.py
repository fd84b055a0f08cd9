"""Accuracy analysis of Section 6 at GEMM scale: the asymmetric rounding of the CDNA3 models (Section 6.2.4, Figure 3)
and the reduced summation precision of the Hopper FP8 row (Section 6.2.2), measured with the library's own FP64
reference and error-statistics reduction."""
import numpy as np
import pytest
import torch

from paper_2511_10909_b200 import workloads as wl

pytestmark = pytest.mark.gpu

gu = pytest.importorskip("gpu_util") if torch.cuda.is_available() else None


def test_error_stats_against_numpy():
    from paper_2511_10909_b200 import mmasim
    g = wl.rng(61)
    d = g.standard_normal(100003).astype(np.float32)
    d[::1000] = np.inf
    ref = d.astype(np.float64) + 1e-3 * g.standard_normal(d.size)
    ref[5::997] = np.nan
    s = mmasim.error_stats("fp32", torch.from_numpy(d.view(np.int32)).cuda(), torch.from_numpy(ref).cuda()).cpu().numpy()
    delta = d.astype(np.float64) - ref
    ok = np.isfinite(delta)
    dl = delta[ok]
    want = [ok.sum(), dl.sum(), np.abs(dl).sum(), (dl * dl).sum(), (dl < 0).sum(), (dl > 0).sum(), np.abs(dl).max(),
            (np.abs(dl) / np.abs(ref[ok])).sum()]
    assert s[0] == want[0] and s[4] == want[4] and s[5] == want[5] and s[6] == want[6]
    np.testing.assert_allclose(s[[1, 2, 3, 7]], np.array(want)[[1, 2, 3, 7]], rtol=1e-9, atol=1e-12)


def test_reference_is_the_real_result():
    from paper_2511_10909_b200 import accuracy
    g = wl.rng(62)
    a = g.standard_normal((64, 96)).astype(np.float16)
    b = g.standard_normal((48, 96)).astype(np.float16)
    c = g.standard_normal((64, 48)).astype(np.float32)
    ref = accuracy.reference_fp64("fp16", "fp32", gu.dev(a.view(np.uint16)), gu.dev(b.view(np.uint16)), gu.dev(c.view(np.uint32)))
    want = a.astype(np.float64) @ b.astype(np.float64).T + c
    np.testing.assert_allclose(ref.cpu().numpy(), want, rtol=1e-13, atol=1e-13)


def test_round_down_bias_of_the_cdna3_model():
    """delta_RD leans to the negative side, delta_RZ is symmetric (Figure 3)."""
    from paper_2511_10909_b200 import accuracy
    r = accuracy.bias_experiment()
    rd, rz = r["RD"], r["RZ"]
    assert rd["count"] == rz["count"] == 1024 * 1024
    assert rd["mean"] < 0 and rd["negative"] > 0.55 and rd["negative"] > rd["positive"] + 0.1
    assert abs(rz["negative"] - rz["positive"]) < 0.01
    assert abs(rz["mean"]) < 0.05 * abs(rd["mean"])
    assert rz["rms"] <= rd["rms"]


def test_hopper_fp8_summation_precision_is_the_bottleneck():
    """F = 13 (Hopper FP8) against F = 25 (Blackwell FP8) on the inputs of config 3 at 1024^3: the mean relative error
    grows by orders of magnitude (Section 6.2.2)."""
    from paper_2511_10909_b200 import accuracy, mmasim
    A, B, C, _, _ = wl.cfg3(1024)
    dA, dB, dC = gu.dev(A), gu.dev(B), gu.dev(C)
    ref = accuracy.reference_fp64("e4m3", "fp32", dA, dB, dC)
    hopper = accuracy.deviation_stats(mmasim.Model("hopper", "e4m3", "fp32"), dA, dB, dC, ref)
    blackwell = accuracy.deviation_stats(mmasim.Model("blackwell", "e4m3", "fp32"), dA, dB, dC, ref)
    assert hopper["mean_abs"] > 100 * blackwell["mean_abs"]
    assert hopper["mean"] != 0.0


def test_risky_designs_at_gemm_scale():
    """Table 10, row by row: each design named there shows as a larger (or one-sided) deviation from the real result than
    the nearest row without it, on the same inputs."""
    from paper_2511_10909_b200 import accuracy
    r = accuracy.risky_designs()
    ftz = r["input_ftz"]
    assert ftz["cdna2"]["mean_abs"] > 100 * ftz["cdna1"]["mean_abs"]           # flushed FP16 subnormals
    assert r["small_F"]["F13"]["mean_abs"] > 100 * r["small_F"]["F25"]["mean_abs"]
    assert r["rz_e8m13"]["RZ-E8M13"]["mean_abs"] > 100 * r["rz_e8m13"]["RZ-FP32"]["mean_abs"]
    assert r["rne_fp16"]["fp16_out"]["mean_abs"] > 100 * r["rne_fp16"]["fp32_out"]["mean_abs"]
    asym = r["asymmetry"]
    assert asym["hopper-fp16"]["asymmetric"] == 0
    for k in ("cdna3-fp16", "cdna3-bf16", "cdna3-e4m3"):
        assert asym[k]["asymmetric"] > 0.05 * asym[k]["count"], (k, asym[k])
        assert asym[k]["mean_sum"] < 0                                          # round-down: both signs lean the same way
