"""The Blackwell rows of the registry against the B200's fifth-generation matrix instruction (Section 3.1, Step 4;
Table 3's UTC*MMA instruction classes): tcgen05.mma, run through mmasim_hw_umma, must agree bit for bit with the model
evaluated by the CUDA path (every output) and by the CPU oracle (sampled outputs).  FP16 / BF16 / TF32 use the input
classes of config 4 plus zero-heavy rows; FP8 / FP6 / FP4 use normal values, random codes (NaN and infinity included),
zero-heavy rows and cancelling pairs.  The give-up path of the kernel's one wait is tested with a barrier nobody
arrives at."""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_10909_b200 import workloads as wl
pytestmark = pytest.mark.gpu

gu = pytest.importorskip("gpu_util") if torch.cuda.is_available() else None


def _needs_b200():
    if torch.cuda.get_device_capability(0)[0] != 10:
        pytest.skip("the hardware comparison is about the B200 (compute capability 10.x)")


# kind -> (A element format, B element format, K of one instruction)
KINDS = {"f16_f32": ("fp16", "fp16", 16), "bf16_f32": ("bf16", "bf16", 16), "tf32_f32": ("tf32", "tf32", 8),
         "e4m3_f32": ("e4m3", "e4m3", 32), "e5m2_f32": ("e5m2", "e5m2", 32), "e4m3_e5m2_f32": ("e4m3", "e5m2", 32),
         "e2m3_f32": ("e2m3", "e2m3", 32), "e3m2_f32": ("e3m2", "e3m2", 32), "e2m1_f32": ("e2m1", "e2m1", 32)}


def _run(kind, A, B, C):
    from paper_2511_10909_b200 import mmasim
    return gu.host_words(mmasim.hw_umma(kind, gu.dev(A), gu.dev(B), gu.dev(C)))


def _tiles(fa, fb, K, M):
    if fa in ("fp16", "bf16", "tf32"):
        return wl.hw_tiles(fa, "fp32", K, M, nb=16)
    return wl.hw_tiles8(fa, K, M, nb=16, b_fmt=fb)


def test_operand_layouts_with_exact_integers():
    """Small integers make every product and sum exact: D must be the integer matrix product, whatever the model."""
    _needs_b200()
    g = wl.rng(93)
    for kind, (fa, fb, k) in KINDS.items():
        for K, M in ((k, 128), (4 * k, 256)):
            lim = 2 if "e2m1" in (fa, fb) else 3
            a = g.integers(-lim, lim + 1, (M, K)); b = g.integers(-lim, lim + 1, (16, K)); c = g.integers(-50, 51, (M, 16))
            D = _run(kind, wl.cast(a.astype(np.float32), fa), wl.cast(b.astype(np.float32), fb), c.astype(np.float32).view(np.uint32))
            assert np.array_equal(D.view(np.float32).astype(np.int64), a @ b.T + c), (kind, K)


@pytest.mark.parametrize("kind", list(KINDS))
@pytest.mark.parametrize("chain", [1, 3])
def test_blackwell_model_matches_tcgen05(kind, chain):
    from paper_2511_10909_b200 import mmasim
    _needs_b200()
    fa, fb, k = KINDS[kind]
    K, M = k * chain, 1 << 13
    A, B, C = _tiles(fa, fb, K, M)
    hw = _run(kind, A, B, C)
    key = ("blackwell", fa, "fp32")
    model = mmasim.Model(*key, b_fmt=fb)
    D = gu.host_words(mmasim.gemm(model, gu.dev(A), gu.dev(B), gu.dev(C)))
    bad = np.argwhere(hw != D)
    assert bad.size == 0, (kind, K, len(bad), [(tuple(x), hex(int(hw[tuple(x)])), hex(int(D[tuple(x)]))) for x in bad[:6]])
    if fa == fb:
        pairs = wl.sample_pairs(M, 16, 768, seed=94)
        want = gu.oracle_samples(key, {"A": A, "B": B, "C": C}, pairs)
        gu.assert_samples_equal(hw, want, pairs, f"hardware tcgen05 {kind} K={K} against the oracle")


def test_the_comparison_discriminates():
    """The same FP8 inputs under the Hopper row (F = 13, RZ-E8M13) differ from the hardware: the harness is not vacuous."""
    from paper_2511_10909_b200 import mmasim
    _needs_b200()
    A, B, C = _tiles("e4m3", "e4m3", 32, 1 << 12)
    hw = _run("e4m3_f32", A, B, C)
    D = gu.host_words(mmasim.gemm(mmasim.Model("hopper", "e4m3", "fp32"), gu.dev(A), gu.dev(B), gu.dev(C)))
    assert (hw != D).sum() > 100


def test_bounded_wait_gives_up_and_the_context_stays_usable():
    """A barrier nobody arrives at: the kernel's wait runs out, the status word says so, the kernel returns (its tensor
    memory released), and the next launch on the same context works."""
    from paper_2511_10909_b200 import mmasim
    _needs_b200()
    A = torch.zeros((256, 32), dtype=torch.uint8, device="cuda")
    B = torch.zeros((16, 32), dtype=torch.uint8, device="cuda")
    out = torch.full((256, 16), 0x5A5A5A5A, dtype=torch.int32, device="cuda")
    with pytest.raises(mmasim.MmasimError) as e:
        mmasim.hw_umma("selftest_timeout", A, B, out=out)
    assert e.value.status == 6
    assert bool((out == 0x5A5A5A5A).all())                               # nothing was stored
    torch.cuda.synchronize()
    D = mmasim.hw_umma("e4m3_f32", A, B)                                 # the context is alive, tensor memory is free again
    assert bool((D == 0).all())


def test_hw_umma_rejects_bad_arguments():
    from paper_2511_10909_b200 import mmasim
    A = torch.zeros((64, 32), dtype=torch.uint8, device="cuda")
    B = torch.zeros((16, 32), dtype=torch.uint8, device="cuda")
    with pytest.raises(mmasim.MmasimError):
        mmasim.hw_umma("e4m3_f32", A, B)                                 # 64 rows: not a multiple of 128
    A = torch.zeros((128, 48), dtype=torch.uint8, device="cuda")
    with pytest.raises(mmasim.MmasimError):
        mmasim.hw_umma("e4m3_f32", A, torch.zeros((16, 48), dtype=torch.uint8, device="cuda"))   # K = 48: not a multiple of 32


# ---- block-scaled kinds: ST-FDPA (Algorithm 8) and GST-FDPA (Algorithm 9) against the instruction ----------------------
SCALED = {"mxe4m3": ("e4m3", 32, 32), "mxe5m2": ("e5m2", 32, 32), "mxe2m3": ("e2m3", 32, 32), "mxe3m2": ("e3m2", 32, 32),
          "mxe2m1": ("e2m1", 32, 32), "mxf4": ("e2m1", 64, 32), "nvf4": ("e2m1", 64, 16)}      # element, K of one instruction, k_block


def _scaled_inputs(kind, K, M, wide):
    elem, k, kb = SCALED[kind]
    A, B, C = wl.hw_tiles8(elem, K, M, nb=16, seed=29)
    g = wl.rng(95, stream=K + len(kind))
    nsf = K // kb
    if kind == "nvf4":                                   # UE4M3 codes: any 7-bit code (0x7F is the NaN), some zeros
        sfa = g.integers(0, 127, (M, nsf)).astype(np.uint8)
        sfb = g.integers(0, 127, (16, nsf)).astype(np.uint8)
        if wide:
            sfa[g.random((M, nsf)) < 0.02] = 0x7F
            sfa[g.random((M, nsf)) < 0.05] = 0
    else:                                                # E8M0: a band around 1 or, wide, the whole range with NaN codes
        lo, hi = (0, 255) if wide else (127 - 12, 127 + 12)
        sfa = g.integers(lo, hi + 1, (M, nsf)).astype(np.uint8)
        sfb = g.integers(lo, hi + 1, (16, nsf)).astype(np.uint8)
        if wide:
            sfb[g.random((16, nsf)) < 0.9] = 127          # keep most products inside the FP32 range
    if kind in ("mxf4", "nvf4"):
        A, B = wl.pack_fp4(A), wl.pack_fp4(B)
    return A, B, C, sfa, sfb


@pytest.mark.parametrize("kind", list(SCALED))
@pytest.mark.parametrize("chain,wide", [(1, False), (2, False), (2, True)])
def test_block_scaled_models_match_tcgen05(kind, chain, wide):
    from paper_2511_10909_b200 import mmasim
    _needs_b200()
    elem, k, kb = SCALED[kind]
    K, M = k * chain, 1 << 12
    A, B, C, sfa, sfb = _scaled_inputs(kind, K, M, wide)
    hw = gu.host_words(mmasim.hw_umma(kind, gu.dev(A), gu.dev(B), gu.dev(C), sfa=gu.dev(sfa), sfb=gu.dev(sfb), K=K))
    key = ("blackwell", kind, "fp32")
    inp = {"A": A, "B": B, "C": C, "sfa": sfa, "sfb": sfb}
    D = gu.run_gemm(key, inp, K=K)
    bad = np.argwhere(hw != D)
    assert bad.size == 0, (kind, K, wide, len(bad), [(tuple(x), hex(int(hw[tuple(x)])), hex(int(D[tuple(x)]))) for x in bad[:6]])
    pairs = wl.sample_pairs(M, 16, 512, seed=96)
    gu.assert_samples_equal(hw, gu.oracle_samples(key, inp, pairs), pairs, f"hardware tcgen05 {kind} K={K} against the oracle")


# FP16 accumulators: kind -> (element format, K of one instruction)
KINDS16 = {"f16_f16": ("fp16", 16), "e4m3_f16": ("e4m3", 32), "e5m2_f16": ("e5m2", 32), "e2m1_f16": ("e2m1", 32)}


def _tiles16(fa, K, M):
    if fa == "fp16":
        return wl.hw_tiles(fa, "fp16", K, M, nb=16)
    A, B, C32 = wl.hw_tiles8(fa, K, M, nb=16)
    # FP16 accumulator words: the FP32 values that fit, cast; everything else an arbitrary 16-bit pattern
    c = C32.view(np.float32)
    with np.errstate(over="ignore", invalid="ignore"):
        fits = np.isfinite(c) & (np.abs(c) < 6.0e4)
        C = np.where(fits, c.astype(np.float16).view(np.uint16), (C32 >> 16).astype(np.uint16))
    return A, B, np.ascontiguousarray(C.astype(np.uint16))


def test_fp16_accumulator_layout_with_exact_integers():
    _needs_b200()
    g = wl.rng(97)
    for kind, (fa, k) in KINDS16.items():
        for K, M in ((k, 128), (4 * k, 256)):
            lim = 2 if fa == "e2m1" else 3
            a = g.integers(-lim, lim + 1, (M, K)); b = g.integers(-lim, lim + 1, (16, K)); c = g.integers(-50, 51, (M, 16))
            D = _run(kind, wl.cast(a.astype(np.float32), fa), wl.cast(b.astype(np.float32), fa), c.astype(np.float16).view(np.uint16))
            assert np.array_equal(D.view(np.float16).astype(np.int64), a @ b.T + c), (kind, K)


@pytest.mark.parametrize("kind", list(KINDS16))
@pytest.mark.parametrize("chain", [1, 3])
def test_blackwell_fp16_accumulator_rows_match_tcgen05(kind, chain):
    """The FP16-accumulator rows of the Blackwell column (T-FDPA with rho = RNE-FP16 after every instruction)."""
    from paper_2511_10909_b200 import mmasim
    _needs_b200()
    fa, k = KINDS16[kind]
    K, M = k * chain, 1 << 13
    A, B, C = _tiles16(fa, K, M)
    hw = _run(kind, A, B, C)
    key = ("blackwell", fa, "fp16")
    D = gu.host_words(mmasim.gemm(mmasim.Model(*key), gu.dev(A), gu.dev(B), gu.dev(C)))
    bad = np.argwhere(hw != D)
    assert bad.size == 0, (kind, K, len(bad), [(tuple(x), hex(int(hw[tuple(x)])), hex(int(D[tuple(x)]))) for x in bad[:6]])
    pairs = wl.sample_pairs(M, 16, 768, seed=98)
    want = gu.oracle_samples(key, {"A": A, "B": B, "C": C}, pairs)
    gu.assert_samples_equal(hw, want, pairs, f"hardware tcgen05 {kind} K={K} against the oracle")
