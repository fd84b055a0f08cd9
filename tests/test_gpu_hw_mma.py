"""The Blackwell rows of the registry against the hardware they describe (Section 3.1, Step 4): the B200's own
mma.sync instruction, run through mmasim_hw_mma, must agree bit for bit with the model evaluated by the CUDA path
(every output) and by the CPU oracle (sampled outputs), on the input classes of config 4 plus zero-heavy rows.
These runs also pin two readings of the paper: zero terms take no part in e_max, and rho overflows to infinity.
The warp-level FP8 instruction, which no registry row describes, is compared with the composition of models that the
probes of clfp.py point to."""
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


# kind -> (element format, accumulator format, K of one instruction)
KINDS = {"f16_f32": ("fp16", "fp32", 16), "f16_f16": ("fp16", "fp16", 16), "bf16_f32": ("bf16", "fp32", 16),
         "tf32_f32": ("tf32", "fp32", 8), "f16_f32_k8": ("fp16", "fp32", 8), "tf32_f32_k4": ("tf32", "fp32", 4)}


def _run(kind, A, B, C):
    from paper_2511_10909_b200 import mmasim
    return gu.host_words(mmasim.hw_mma(kind, gu.dev(A), gu.dev(B), gu.dev(C)))


def test_fragment_layouts_with_exact_integers():
    """Small integers make every product and sum exact: D must be the integer matrix product, whatever the model."""
    _needs_b200()
    g = wl.rng(90)
    M = 64
    for kind, (fmt, acc, k) in list(KINDS.items()) + [("e4m3_f32", ("e4m3", "fp32", 32)), ("e5m2_f32", ("e5m2", "fp32", 32)),
                                                       ("e4m3_f16", ("e4m3", "fp16", 32)), ("e5m2_f16", ("e5m2", "fp16", 32)),
                                                       ("e4m3_e5m2_f32", ("e4m3", "fp32", 32)), ("e4m3_f32_k16", ("e4m3", "fp32", 16)),
                                                       ("f64", ("fp64", "fp64", 4))]:
        for K in (k, 3 * k):
            a = g.integers(-2, 3, (M, K)); b = g.integers(-2, 3, (8, K)); c = g.integers(-8, 9, (M, 8))
            if fmt == "fp64":
                A, B, C = (x.astype(np.float64).view(np.uint64) for x in (a, b, c))
            else:
                A, B = wl.cast(a.astype(np.float32), fmt), wl.cast(b.astype(np.float32), "e5m2" if kind == "e4m3_e5m2_f32" else fmt)
                C = c.astype(np.float32).view(np.uint32) if acc == "fp32" else c.astype(np.float16).view(np.uint16)
            D = _run(kind, A, B, C)
            want = a @ b.T + c
            got = D.view({2: np.float16, 4: np.float32, 8: np.float64}[D.dtype.itemsize]).astype(np.int64)
            assert np.array_equal(got, want), (kind, K)


@pytest.mark.parametrize("kind", list(KINDS))
@pytest.mark.parametrize("chain", [1, 4])
def test_blackwell_model_matches_mma_sync(kind, chain):
    from paper_2511_10909_b200 import mmasim
    _needs_b200()
    fmt, acc, k = KINDS[kind]
    if chain > 1 and kind in ("f16_f32_k8", "tf32_f32_k4"):
        pytest.skip("a chain of the short instructions is a chain of shorter blocks than the registry row's L")
    K, M = k * chain, 1 << 13
    A, B, C = wl.hw_tiles(fmt, acc, K, M)
    hw = _run(kind, A, B, C)
    key = ("blackwell", fmt, acc)
    D = gu.host_words(mmasim.gemm(mmasim.Model(*key), gu.dev(A), gu.dev(B), gu.dev(C)))
    bad = np.argwhere(hw != D)
    assert bad.size == 0, (kind, K, len(bad), [(tuple(x), hex(int(hw[tuple(x)])), hex(int(D[tuple(x)]))) for x in bad[:4]])
    pairs = wl.sample_pairs(M, 8, 768, seed=91)
    want = gu.oracle_samples(key, {"A": A, "B": B, "C": C}, pairs)
    gu.assert_samples_equal(hw, want, pairs, f"hardware {kind} K={K} against the oracle")


@pytest.mark.parametrize("K", [4, 16])
def test_fp64_mma_is_a_chain_of_fmas(K):
    from paper_2511_10909_b200 import mmasim
    _needs_b200()
    A, B, C = wl.hw_tiles("fp64", "fp64", K, 1 << 12)
    hw = _run("f64", A, B, C)
    key = ("blackwell", "fp64", "fp64")
    D = gu.host_words(mmasim.gemm(mmasim.Model(*key), gu.dev(A), gu.dev(B), gu.dev(C)))
    assert np.array_equal(hw, D)
    pairs = wl.sample_pairs(1 << 12, 8, 512, seed=92)
    gu.assert_samples_equal(hw, gu.oracle_samples(key, {"A": A, "B": B, "C": C}, pairs), pairs, "FP64 mma against the oracle")


def test_the_comparison_discriminates():
    """The same inputs under the Ampere row (L = 8, F = 24) do differ from the hardware: the harness is not vacuous."""
    from paper_2511_10909_b200 import mmasim
    _needs_b200()
    A, B, C = wl.hw_tiles("fp16", "fp32", 16, 1 << 12)
    hw = _run("f16_f32", A, B, C)
    D = gu.host_words(mmasim.gemm(mmasim.Model("ampere", "fp16", "fp32"), gu.dev(A), gu.dev(B), gu.dev(C)))
    assert (hw != D).sum() > 100


def test_hw_mma_rejects_bad_shapes():
    from paper_2511_10909_b200 import mmasim
    A = torch.zeros((24, 16), dtype=torch.int16, device="cuda")
    B = torch.zeros((8, 16), dtype=torch.int16, device="cuda")
    with pytest.raises(mmasim.MmasimError):
        mmasim.hw_mma("f16_f32", A, B)                                   # 24 rows: not a multiple of 16
    with pytest.raises(mmasim.MmasimError):
        mmasim.hw_mma("f16_f32", A[:16, :8].contiguous(), B[:, :8].contiguous())   # K = 8 with a k16 instruction


@pytest.mark.parametrize("fmt", ["e4m3", "e5m2"])
@pytest.mark.parametrize("K", [32, 96])
def test_fp8_mma_sync_is_the_fp16_row_in_two_blocks_plus_an_fp32_addition(fmt, K):
    """The warp-level FP8 instruction of the B200 matches none of the registry's FP8 rows (those describe the newer
    interface); the probes of clfp.py show two fused blocks of 16 (the elements k = 0, 1 mod 4, then k = 2, 3 mod 4
    with the first result as accumulator) and the accumulator added outside them.  With the Blackwell FP16 row for the
    blocks and an IEEE FP32 addition for C - the FP32-promotion workaround with chunks of 32 - the composition agrees
    with the hardware bit for bit, special values, zeros and chains of instructions included."""
    from paper_2511_10909_b200 import explore, mmasim
    _needs_b200()
    M = 1 << 12
    order = [32 * q + k for q in range(K // 32) for half in ((0, 1), (2, 3)) for k in range(32) if k % 4 in half]
    for mode in ("normal", "bits", "zeros"):
        g = wl.rng(95 + K + len(mode))
        inp = wl.normal_inputs(fmt, "fp32", M, 8, K, seed=96)
        A, B, C = inp["A"].copy(), inp["B"].copy(), inp["C"].copy()
        if mode == "bits":                                    # NaN, infinities, subnormals, any accumulator
            A = g.integers(0, 256, A.shape, dtype=np.uint8)
            B = g.integers(0, 256, B.shape, dtype=np.uint8)
            C = g.integers(0, 1 << 32, C.shape, dtype=np.uint64).astype(np.uint32)
        if mode == "zeros":
            A[g.random(A.shape) < 0.5] = 0
            A[g.random(A.shape) < 0.1] = 0x80
            C[g.random(C.shape) < 0.3] = 0x80000000
        hw = _run(fmt + "_f32", A, B, C)
        D = gu.host_words(explore.b200_fp8_mma_sync(fmt, gu.dev(A), gu.dev(B), gu.dev(C)))
        bad = np.argwhere(hw != D)
        assert bad.size == 0, (fmt, K, mode, len(bad), [(tuple(x), hex(int(hw[tuple(x)])), hex(int(D[tuple(x)]))) for x in bad[:4]])
        # the same composition through the oracle: FP8 values as FP16 words, reordered, chunks of 32
        wide = lambda X: gu.host_words(explore.widen_fp8_to_fp16(fmt, gu.dev(X)))[:, order]
        pairs = wl.sample_pairs(M, 8, 400, seed=97)
        want = oracle.phi_gemm_sampled(oracle.lookup("blackwell", "fp16", "fp32"), wide(A), wide(B), C, pairs, k_chunk=32)
        gu.assert_samples_equal(hw, want, pairs, f"hardware {fmt} K={K} {mode} against the oracle's composition")


def test_fp8_mma_sync_with_mixed_operand_types():
    """A in E4M3, B in E5M2: the same composition."""
    from paper_2511_10909_b200 import explore
    _needs_b200()
    g = wl.rng(98)
    M, K = 1 << 12, 64
    for mode in ("normal", "bits"):
        A = wl.normal_inputs("e4m3", "fp32", M, 8, K, seed=99)["A"]
        B = wl.normal_inputs("e5m2", "fp32", M, 8, K, seed=100)["B"]
        C = wl.normal_inputs("e4m3", "fp32", M, 8, K, seed=101)["C"]
        if mode == "bits":
            A = g.integers(0, 256, A.shape, dtype=np.uint8)
            B = g.integers(0, 256, B.shape, dtype=np.uint8)
            C = g.integers(0, 1 << 32, C.shape, dtype=np.uint64).astype(np.uint32)
        hw = _run("e4m3_e5m2_f32", A, B, C)
        D = gu.host_words(explore.b200_fp8_mma_sync("e4m3", gu.dev(A), gu.dev(B), gu.dev(C), b_fmt="e5m2"))
        assert np.array_equal(hw, D), (mode, int((hw != D).sum()))


@pytest.mark.parametrize("fmt", ["e4m3", "e5m2"])
def test_fp8_mma_sync_with_fp16_accumulator(fmt):
    """FP8 inputs, FP16 accumulator: the two blocks of 16 run through the Blackwell FP16 -> FP16 row (RNE-FP16 after each
    block) from a +0 accumulator, and C is added by an IEEE FP16 addition (NaN as 0x7FFF)."""
    from paper_2511_10909_b200 import explore, mmasim
    _needs_b200()
    g = wl.rng(102)
    M, K = 1 << 12, 32
    i1 = [k for k in range(32) if k % 4 in (0, 1)]
    i2 = [k for k in range(32) if k % 4 in (2, 3)]
    model = mmasim.Model("blackwell", "fp16", "fp16")
    for mode in ("normal", "bits"):
        A = wl.normal_inputs(fmt, "fp32", M, 8, K, seed=103)["A"]
        B = wl.normal_inputs(fmt, "fp32", M, 8, K, seed=104)["B"]
        C = (g.standard_normal((M, 8)) * 2.0 ** g.integers(-6, 6, (M, 8))).astype(np.float16).view(np.uint16)
        if mode == "bits":
            A = g.integers(0, 256, A.shape, dtype=np.uint8)
            B = g.integers(0, 256, B.shape, dtype=np.uint8)
            C = g.integers(0, 1 << 16, C.shape).astype(np.uint16)
        hw = _run(fmt + "_f16", A, B, C)
        A16, B16 = explore.widen_fp8_to_fp16(fmt, gu.dev(A)), explore.widen_fp8_to_fp16(fmt, gu.dev(B))
        zero = torch.zeros((M, 8), dtype=torch.int16, device="cuda")
        t1 = mmasim.gemm(model, A16[:, i1].contiguous(), B16[:, i1].contiguous(), zero)
        t2 = mmasim.gemm(model, A16[:, i2].contiguous(), B16[:, i2].contiguous(), t1)
        d = t2.view(torch.float16) + gu.dev(C).view(torch.float16)
        D = gu.host_words(d.view(torch.int16)).copy()
        D[np.isnan(D.view(np.float16))] = 0x7FFF
        assert np.array_equal(hw, D), (fmt, mode, int((hw != D).sum()))


@pytest.mark.parametrize("K", [16, 48])
def test_fp8_k16_mma_sync_is_two_blocks_of_eight(K):
    """m16n8k16 on E4M3: the same scheme with the halves of one operand register per row - two fused blocks of 8 (the
    Blackwell FP16 row with L = 8: the FP16 instruction of that length) chained from +0, then the FP32 addition of C."""
    from paper_2511_10909_b200 import explore, mmasim
    _needs_b200()
    g = wl.rng(105 + K)
    M = 1 << 12
    order = [16 * q + k for q in range(K // 16) for half in ((0, 1), (2, 3)) for k in range(16) if k % 4 in half]
    p = torch.tensor(order, device="cuda")
    model = mmasim.Model("blackwell", "fp16", "fp32", l_max=8)
    for mode in ("normal", "bits"):
        inp = wl.normal_inputs("e4m3", "fp32", M, 8, K, seed=106)
        A, B, C = inp["A"], inp["B"], inp["C"]
        if mode == "bits":
            A = g.integers(0, 256, A.shape, dtype=np.uint8)
            B = g.integers(0, 256, B.shape, dtype=np.uint8)
            C = g.integers(0, 1 << 32, C.shape, dtype=np.uint64).astype(np.uint32)
        hw = _run("e4m3_f32_k16", A, B, C)
        A16 = explore.widen_fp8_to_fp16("e4m3", gu.dev(A))[:, p].contiguous()
        B16 = explore.widen_fp8_to_fp16("e4m3", gu.dev(B))[:, p].contiguous()
        D = gu.host_words(mmasim.gemm(model, A16, B16, gu.dev(C), k_chunk=16))
        assert np.array_equal(hw, D), (K, mode, int((hw != D).sum()))
