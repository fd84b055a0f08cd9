"""The tuned kernels against the oracle (sampled) and against the generic kernels (every output), bit for bit,
on ragged shapes, random bit streams (NaN, infinities, subnormals, wide exponent spreads) and extreme accumulators."""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_10909_b200 import workloads as wl

pytestmark = pytest.mark.gpu
gu = pytest.importorskip("gpu_util") if torch.cuda.is_available() else None

FAST8 = [("ada", "e4m3", "fp32"), ("ada", "e5m2", "fp16"), ("hopper", "e4m3", "fp32"), ("hopper", "e5m2", "fp32"),
         ("hopper", "e4m3", "fp16"), ("hopper", "e5m2", "fp16"), ("blackwell", "e4m3", "fp32"), ("blackwell", "e5m2", "fp32"),
         ("blackwell", "e3m2", "fp32"), ("blackwell", "e2m3", "fp32"), ("blackwell", "e2m1", "fp32"),
         ("blackwell", "e4m3", "fp16"), ("rtx_blackwell", "e2m3", "fp16")]


FAST16 = [("volta", "fp16", "fp32"), ("volta", "fp16", "fp16"), ("turing", "fp16", "fp32"), ("ampere", "fp16", "fp16"),
          ("hopper", "fp16", "fp32"), ("blackwell", "fp16", "fp16"), ("ampere", "bf16", "fp32"), ("hopper", "bf16", "fp32"),
          ("ampere", "tf32", "fp32"), ("hopper", "tf32", "fp32")]
KERNEL16 = {"fp16": "tfdpa_f16", "bf16": "tfdpa_bf16", "tf32": "tfdpa_tf32"}


def _check(key, inp, nsample=600, expect_kernel=None, **kw):
    from paper_2511_10909_b200 import mmasim
    D = gu.run_gemm(key, inp, **kw)
    if expect_kernel:
        assert mmasim.last_kernel() == expect_kernel
    G = gu.run_gemm(key, inp, force_generic=True, **kw)
    assert mmasim.last_kernel() == "generic"
    bad = np.argwhere(D != G)
    assert bad.size == 0, (key, len(bad), bad[:4], [hex(int(D[tuple(b)])) for b in bad[:4]], [hex(int(G[tuple(b)])) for b in bad[:4]])
    M, N = D.shape
    pairs = wl.sample_pairs(M, N, nsample, seed=M + N)
    okw = {}
    if "k_chunk" in kw:
        okw["k_chunk"] = kw["k_chunk"]
    if "row_scale" in kw:
        okw["row_scale"] = gu.host_words(kw["row_scale"])
        okw["col_scale"] = gu.host_words(kw["col_scale"])
    gu.assert_samples_equal(D, gu.oracle_samples(key, inp, pairs, **okw), pairs, str(key))
    return D


@pytest.mark.parametrize("key", FAST8, ids=lambda k: "-".join(k))
def test_fp8_normal_inputs_ragged_shape(key):
    inp = wl.normal_inputs(key[1], key[2], 200, 100, 256, seed=21)
    _check(key, inp, expect_kernel="tfdpa_lut8")


@pytest.mark.parametrize("key", FAST8, ids=lambda k: "-".join(k))
def test_fp8_random_bit_stream(key):
    g = wl.rng(22)
    M, N, K = 150, 70, 128
    m = oracle.lookup(*key)
    bits = 1 + oracle.FORMATS[m.elem].ebits + oracle.FORMATS[m.elem].mbits
    A = g.integers(0, 1 << bits, (M, K), dtype=np.uint8)
    B = g.integers(0, 1 << bits, (N, K), dtype=np.uint8)
    if key[2] == "fp16":
        C = g.integers(0, 1 << 16, (M, N), dtype=np.uint16)
    else:
        C = g.integers(0, 1 << 32, (M, N), dtype=np.uint32)
    _check(key, {"A": A, "B": B, "C": C}, expect_kernel="tfdpa_lut8")


@pytest.mark.parametrize("key", [("hopper", "e4m3", "fp32"), ("blackwell", "e5m2", "fp32"), ("blackwell", "e4m3", "fp16")],
                         ids=lambda k: "-".join(k))
def test_fp8_extreme_accumulators(key):
    # accumulators around the subnormal boundary, around the overflow boundary, and products that cancel exactly
    g = wl.rng(23)
    M, N, K = 128, 64, 64
    inp = wl.normal_inputs(key[1], key[2], M, N, K, seed=24)
    A = inp["A"].copy()
    A[:, 1::2] = inp["A"][:, 0::2] ^ 0x80                  # exact cancellation of neighbouring terms in half the rows
    Bm = inp["B"].copy()
    Bm[:, 1::2] = inp["B"][:, 0::2]
    A[M // 2:], Bm[N // 2:] = inp["A"][M // 2:], inp["B"][N // 2:]
    if key[2] == "fp16":
        C = ((g.integers(0, 2, (M, N)) << 15) | (g.choice([0, 1, 2, 29, 30], (M, N)) << 10) | g.integers(0, 1024, (M, N))).astype(np.uint16)
    else:
        C = ((g.integers(0, 2, (M, N)) << 31) | (g.choice([0, 1, 2, 3, 252, 253, 254], (M, N)) << 23) | g.integers(0, 1 << 23, (M, N))).astype(np.uint32)
    _check(key, {"A": A, "B": Bm, "C": C}, expect_kernel="tfdpa_lut8")


@pytest.mark.parametrize("key", [("hopper", "e4m3", "fp32"), ("ada", "e4m3", "fp32"), ("hopper", "e5m2", "fp32"), ("hopper", "e4m3", "fp16")],
                         ids=lambda k: "-".join(k))
def test_fp8_no_nonzero_product_and_register_limits(key):
    # rows of A that are all +-0 (the result is rho of the accumulator alone, whatever its size; +0 for c = -0), beside
    # ordinary rows, with accumulators of every exponent: far below the products, around the largest exponent the
    # FP32 sum register can hold, and up to the largest finite value
    g = wl.rng(29)
    M, N, K = 128, 64, 96
    inp = wl.normal_inputs(key[1], key[2], M, N, K, seed=30)
    A = inp["A"].copy()
    A[0::4] = (g.integers(0, 2, (M // 4, K)) << 7).astype(np.uint8)
    A[1::4, : K // 3] = 0                                      # one block without products, then ordinary blocks
    if key[2] == "fp16":
        C = g.integers(0, 1 << 16, (M, N)).astype(np.uint16)
        C[(C & 0x7C00) == 0x7C00] = 0x8000
    else:
        field = g.choice(np.r_[0:8, 100:120, 236:255], (M, N))
        C = ((g.integers(0, 2, (M, N)) << 31) | (field << 23) | g.integers(0, 1 << 23, (M, N))).astype(np.uint32)
        C[g.random((M, N)) < 0.1] = 0x80000000
    _check(key, {"A": A, "B": inp["B"], "C": C}, expect_kernel="tfdpa_lut8")


def test_fp8_promotion_and_dequant_ragged():
    key = ("hopper", "e4m3", "fp32")
    g = wl.rng(25)
    inp = wl.normal_inputs("e4m3", "fp32", 130, 66, 512, seed=26)
    inp["A"][3, 7] = 0x7F                                       # one NaN
    rs = gu.dev(g.standard_normal(130).astype(np.float32))
    cs = gu.dev(g.standard_normal(66).astype(np.float32))
    _check(key, inp, expect_kernel="tfdpa_lut8", k_chunk=128, row_scale=rs, col_scale=cs)
    _check(key, inp, expect_kernel="tfdpa_lut8", k_chunk=32)
    _check(key, inp, expect_kernel="tfdpa_lut8", row_scale=rs, col_scale=cs)


def test_mixed_fp8_types():
    from paper_2511_10909_b200 import mmasim
    g = wl.rng(27)
    M, N, K = 64, 64, 64
    A = g.integers(0, 256, (M, K), dtype=np.uint8)
    B = g.integers(0, 256, (N, K), dtype=np.uint8)
    C = g.standard_normal((M, N)).astype(np.float32).view(np.uint32)
    model = mmasim.Model("blackwell", "e4m3", "fp32", b_fmt="e5m2")
    D = gu.host_words(mmasim.gemm(model, gu.dev(A), gu.dev(B), gu.dev(C)))
    assert mmasim.last_kernel() == "tfdpa_lut8"
    F = oracle.FORMATS
    for i, j in [(0, 0), (5, 9), (63, 63), (17, 40), (33, 2)] + [tuple(p) for p in wl.sample_pairs(M, N, 100, 5)]:
        d = int(C[i, j])
        for k in range(0, K, 32):
            d = oracle.t_fdpa(A[i, k:k + 32].tolist(), B[j, k:k + 32].tolist(), d, F["e4m3"], F["e5m2"], F["fp32"], 25, "RZ-FP32")
        assert int(D[i, j]) == d, (i, j)


@pytest.mark.parametrize("key", FAST16, ids=lambda k: "-".join(k))
def test_16bit_normal_inputs_ragged_shape(key):
    inp = wl.normal_inputs(key[1], key[2], 200, 100, 256, seed=31)
    _check(key, inp, expect_kernel=KERNEL16[key[1]])


@pytest.mark.parametrize("key", FAST16, ids=lambda k: "-".join(k))
def test_16bit_random_bit_stream(key):
    g = wl.rng(32)
    M, N, K = 150, 70, 128
    wbits = 32 if key[1] == "tf32" else 16
    dt = np.uint32 if wbits == 32 else np.uint16
    A = g.integers(0, 1 << wbits, (M, K), dtype=np.uint64).astype(dt)
    B = g.integers(0, 1 << wbits, (N, K), dtype=np.uint64).astype(dt)
    if key[2] == "fp16":
        C = g.integers(0, 1 << 16, (M, N), dtype=np.uint16)
    else:
        C = g.integers(0, 1 << 32, (M, N), dtype=np.uint32)
    _check(key, {"A": A, "B": B, "C": C}, expect_kernel=KERNEL16[key[1]])


@pytest.mark.parametrize("key", FAST16, ids=lambda k: "-".join(k))
def test_16bit_config4_classes_as_gemm(key):
    # the adversarial classes of the probe batch (subnormals, cancellation, outliers, inf / NaN, bit streams) as GEMM operands
    m = oracle.lookup(*key)
    A, B, C = wl.cfg4(m.elem, 32, n=1 << 12)
    A, B = A[:192].reshape(192, 32), B[192:192 + 96].reshape(96, 32)
    A = np.ascontiguousarray(np.tile(A, (1, 4)))
    B = np.ascontiguousarray(np.tile(B, (1, 4)))
    Cm = np.resize(C, (192, 96)).copy()
    if key[2] == "fp16":
        Cm = (Cm >> 16).astype(np.uint16)
    _check(key, {"A": A, "B": B, "C": Cm}, expect_kernel=KERNEL16[key[1]])


def test_bf16_wide_exponents_and_extreme_accumulators():
    key = ("hopper", "bf16", "fp32")
    g = wl.rng(33)
    M, N, K = 128, 64, 64
    def mat(rows):
        sign = g.integers(0, 2, (rows, K), dtype=np.uint16)
        exp = g.integers(1, 255, (rows, K)).astype(np.uint16)          # the whole exponent range
        man = g.integers(0, 128, (rows, K), dtype=np.uint16)
        return ((sign << 15) | (exp << 7) | man).astype(np.uint16)
    C = ((g.integers(0, 2, (M, N)) << 31) | (g.choice([0, 1, 2, 100, 127, 150, 253, 254], (M, N)) << 23) | g.integers(0, 1 << 23, (M, N))).astype(np.uint32)
    _check(key, {"A": mat(M), "B": mat(N), "C": C}, expect_kernel="tfdpa_bf16")


def test_16bit_promotion():
    key = ("hopper", "fp16", "fp32")
    inp = wl.normal_inputs("fp16", "fp32", 130, 66, 256, seed=34)
    _check(key, inp, expect_kernel="tfdpa_f16", k_chunk=64)


ST_KEYS = [("blackwell", "mxe4m3", "fp32"), ("blackwell", "mxe5m2", "fp32"), ("rtx_blackwell", "mxe3m2", "fp32"),
           ("blackwell", "mxe2m3", "fp32"), ("rtx_blackwell", "mxe2m1", "fp32")]


@pytest.mark.parametrize("key", ST_KEYS, ids=lambda k: "-".join(k))
def test_st_fdpa_block_scaled(key):
    inp = wl.normal_inputs(key[1], key[2], 200, 100, 256, seed=41)
    _check(key, inp, expect_kernel="tfdpa_lut8")
    # random element bytes, scale factors over the whole E8M0 range including NaN (0xFF), random accumulators
    g = wl.rng(42)
    m = oracle.lookup(*key)
    bits = 1 + oracle.FORMATS[m.elem].ebits + oracle.FORMATS[m.elem].mbits
    M, N, K = 150, 70, 128
    inp = {"A": g.integers(0, 1 << bits, (M, K), dtype=np.uint8), "B": g.integers(0, 1 << bits, (N, K), dtype=np.uint8),
           "C": g.integers(0, 1 << 32, (M, N), dtype=np.uint32),
           "sfa": g.integers(0, 256, (M, K // 32), dtype=np.uint8), "sfb": g.integers(0, 256, (N, K // 32), dtype=np.uint8)}
    _check(key, inp, expect_kernel="tfdpa_lut8")
    # moderate scales (results in the normal range) with a few NaN scale factors
    inp["sfa"] = g.integers(100, 150, (M, K // 32), dtype=np.uint8)
    inp["sfb"] = g.integers(100, 150, (N, K // 32), dtype=np.uint8)
    inp["sfa"][5, 1] = 255
    inp["sfb"][9, 3] = 255
    inp["C"] = g.standard_normal((M, N)).astype(np.float32).view(np.uint32)
    _check(key, inp, expect_kernel="tfdpa_lut8")


TR_KEYS = [("cdna3", "fp16", "fp32"), ("cdna3", "bf16", "fp32"), ("cdna3", "tf32", "fp32"), ("cdna3", "e4m3", "fp32"),
           ("cdna3", "e5m2", "fp32")]


def _tr_kernel(key):
    return "gtrfdpa" if key[1] in ("e4m3", "e5m2") else "trfdpa"


@pytest.mark.parametrize("key", TR_KEYS, ids=lambda k: "-".join(k))
def test_tr_gtr_normal_inputs_and_bias_case(key):
    inp = wl.normal_inputs(key[1], key[2], 200, 100, 256, seed=51)
    _check(key, inp, expect_kernel=_tr_kernel(key))
    # the regime of the paper's bias experiment (Section 6.2.4): large A, B and a small accumulator of either sign
    g = wl.rng(52)
    scale = 1000.0 if key[1] not in ("e4m3", "e5m2") else 16.0
    A = wl.cast(g.standard_normal((130, 128)).astype(np.float32) * scale, key[1])
    B = wl.cast(g.standard_normal((70, 128)).astype(np.float32) * scale, key[1])
    C = g.standard_normal((130, 70)).astype(np.float32).view(np.uint32)
    _check(key, {"A": A, "B": B, "C": C}, expect_kernel=_tr_kernel(key))


@pytest.mark.parametrize("key", TR_KEYS, ids=lambda k: "-".join(k))
def test_tr_gtr_random_bit_stream(key):
    g = wl.rng(53)
    M, N, K = 150, 70, 128
    m = oracle.lookup(*key)
    if key[1] in ("e4m3", "e5m2"):
        A = g.integers(0, 256, (M, K), dtype=np.uint8)
        B = g.integers(0, 256, (N, K), dtype=np.uint8)
    else:
        wbits = 32 if key[1] == "tf32" else 16
        dt = np.uint32 if wbits == 32 else np.uint16
        A = g.integers(0, 1 << wbits, (M, K), dtype=np.uint64).astype(dt)
        B = g.integers(0, 1 << wbits, (N, K), dtype=np.uint64).astype(dt)
    C = g.integers(0, 1 << 32, (M, N), dtype=np.uint32)
    _check(key, {"A": A, "B": B, "C": C}, expect_kernel=_tr_kernel(key))
    # products near 2^128 (overflow to infinity) and accumulators at both ends of the exponent range
    if key[1] in ("bf16", "tf32"):
        low = 13 if key[1] == "tf32" else 0
        dt = np.uint32 if key[1] == "tf32" else np.uint16
        mb = 10 if key[1] == "tf32" else 7
        def mat(rows):
            sign = g.integers(0, 2, (rows, K), dtype=np.uint64)
            exp = g.choice([1, 60, 127, 186, 190, 191, 192, 254], (rows, K)).astype(np.uint64)
            man = g.integers(0, 1 << mb, (rows, K), dtype=np.uint64)
            return ((((sign << 8) | exp) << mb | man) << low).astype(dt)
        C = ((g.integers(0, 2, (M, N)) << 31) | (g.choice([0, 1, 2, 127, 253, 254], (M, N)) << 23) | g.integers(0, 1 << 23, (M, N))).astype(np.uint32)
        _check(key, {"A": mat(M), "B": mat(N), "C": C}, expect_kernel=_tr_kernel(key))


@pytest.mark.parametrize("key", TR_KEYS, ids=lambda k: "-".join(k))
def test_tr_gtr_config4_classes_as_gemm(key):
    m = oracle.lookup(*key)
    if key[1] in ("e4m3", "e5m2"):
        g = wl.rng(54)
        A = g.integers(0, 256, (192, 128), dtype=np.uint8)
        A[:, 1::2] = A[:, 0::2] ^ 0x80                       # neighbouring terms cancel: the even / odd groups matter
        B = g.integers(0, 256, (96, 128), dtype=np.uint8)
        B[:, 1::2] = B[:, 0::2]
        C = g.standard_normal((192, 96)).astype(np.float32).view(np.uint32)
    else:
        A, B, C = wl.cfg4(m.elem, 32, n=1 << 12)
        A, B = A[:192].reshape(192, 32), B[192:192 + 96].reshape(96, 32)
        A = np.ascontiguousarray(np.tile(A, (1, 4)))
        B = np.ascontiguousarray(np.tile(B, (1, 4)))
        C = np.resize(C, (192, 96)).copy()
    _check(key, {"A": A, "B": B, "C": C}, expect_kernel=_tr_kernel(key))


FP_KEYS = [("cdna3", "fp32", "fp32"), ("cdna1", "fp32", "fp32"), ("hopper", "fp64", "fp64"), ("cdna2", "fp64", "fp64"),
           ("cdna2", "fp16", "fp32"), ("cdna2", "bf16", "fp32"), ("cdna2", "bf16_1k", "fp32")]
FP_KERNEL = {"fp32": "fma_f32", "fp64": "fma_f64", "fp16": "ftz_addmul", "bf16": "ftz_addmul", "bf16_1k": "ftz_addmul"}


@pytest.mark.parametrize("key", FP_KEYS, ids=lambda k: "-".join(k))
def test_fp_pipe_models(key):
    inp = wl.normal_inputs(key[1], key[2], 200, 100, 128, seed=61)
    _check(key, inp, nsample=300, expect_kernel=FP_KERNEL[key[1]])
    # random bit streams: NaN, infinities, subnormals, huge exponent spread
    g = wl.rng(62)
    m = oracle.lookup(*key)
    wbits = oracle.FORMATS[m.elem].storage_bits
    M, N, K = 100, 70, 64
    A = g.integers(0, 1 << 63, (M, K), dtype=np.uint64).astype(wl.word_dtype(m.elem)) if wbits < 64 else g.integers(0, 1 << 63, (M, K), dtype=np.uint64) * 2 + g.integers(0, 2, (M, K), dtype=np.uint64)
    B = g.integers(0, 1 << 63, (N, K), dtype=np.uint64).astype(wl.word_dtype(m.elem)) if wbits < 64 else g.integers(0, 1 << 63, (N, K), dtype=np.uint64) * 2 + g.integers(0, 2, (N, K), dtype=np.uint64)
    cbits = 64 if key[2] == "fp64" else 32
    C = (g.integers(0, 1 << 63, (M, N), dtype=np.uint64) * 2).astype(np.uint64 if cbits == 64 else np.uint32)
    _check(key, {"A": A, "B": B, "C": C}, nsample=300, expect_kernel=FP_KERNEL[key[1]])


@pytest.mark.parametrize("key", [("cdna2", "fp16", "fp32"), ("cdna2", "bf16", "fp32"), ("cdna2", "bf16_1k", "fp32")], ids=lambda k: "-".join(k))
def test_ftz_flush_boundary(key):
    # operands whose products and sums sit around 2^-126: the hardware flush mode must agree with "round, then flush"
    g = wl.rng(63)
    M, N, K = 128, 64, 64
    if key[1] == "fp16":
        A = ((g.integers(0, 2, (M, K)) << 15) | (g.integers(0, 4, (M, K)) << 10) | g.integers(0, 1024, (M, K))).astype(np.uint16)
        B = ((g.integers(0, 2, (N, K)) << 15) | (g.integers(0, 4, (N, K)) << 10) | g.integers(0, 1024, (N, K))).astype(np.uint16)
    else:
        A = ((g.integers(0, 2, (M, K)) << 15) | (g.integers(0, 70, (M, K)) << 7) | g.integers(0, 128, (M, K))).astype(np.uint16)
        B = ((g.integers(0, 2, (N, K)) << 15) | (g.integers(58, 130, (N, K)) << 7) | g.integers(0, 128, (N, K))).astype(np.uint16)
    C = ((g.integers(0, 2, (M, N)) << 31) | (g.integers(0, 4, (M, N)) << 23) | g.integers(0, 1 << 23, (M, N))).astype(np.uint32)
    _check(key, {"A": A, "B": B, "C": C}, nsample=400, expect_kernel="ftz_addmul")


GST_KEYS = [("blackwell", "mxf4", "fp32"), ("blackwell", "nvf4", "fp32"), ("rtx_blackwell", "nvf4", "fp32")]


@pytest.mark.parametrize("key", GST_KEYS, ids=lambda k: "-".join(k))
def test_gst_fdpa_group_scaled(key):
    inp = wl.normal_inputs(key[1], key[2], 200, 100, 256, seed=71)
    _check(key, inp, expect_kernel="gstfdpa")
    # random nibbles, scale factors over the whole code range (zero, subnormal, NaN scales), random accumulators
    g = wl.rng(72)
    M, N, K = 150, 70, 192
    kb = 16 if key[1] == "nvf4" else 32
    inp = {"A": g.integers(0, 256, (M, K // 2), dtype=np.uint8), "B": g.integers(0, 256, (N, K // 2), dtype=np.uint8),
           "C": g.integers(0, 1 << 32, (M, N), dtype=np.uint32),
           "sfa": g.integers(0, 256, (M, K // kb), dtype=np.uint8), "sfb": g.integers(0, 256, (N, K // kb), dtype=np.uint8)}
    _check(key, inp, expect_kernel="gstfdpa")
    # moderate scales and accumulators so that most results are ordinary numbers, with a few NaN scales
    lo, hi = (0x20, 0x50) if key[1] == "nvf4" else (110, 140)
    inp["sfa"] = g.integers(lo, hi, (M, K // kb), dtype=np.uint8)
    inp["sfb"] = g.integers(lo, hi, (N, K // kb), dtype=np.uint8)
    inp["sfa"][7, 2] = 0xFF
    inp["sfb"][3, 0] = 0x7F if key[1] == "nvf4" else 0xFF
    inp["C"] = g.standard_normal((M, N)).astype(np.float32).view(np.uint32)
    _check(key, inp, expect_kernel="gstfdpa")


@pytest.mark.parametrize("key", [("cdna1", "fp16", "fp32"), ("cdna1", "bf16", "fp32")], ids=lambda k: "-".join(k))
def test_e_fdpa_exact_sum(key):
    # the exact sum in FP64 where the block fits its window, by the book elsewhere: ordinary values (ragged shape),
    # random bit streams (NaN, infinities, subnormals, any exponent spread), zeros and cancelling products, and
    # accumulators from the subnormal range to the overflow boundary
    g = wl.rng(41)
    inp = wl.normal_inputs(key[1], key[2], 130, 70, 96, seed=42)
    _check(key, inp, expect_kernel="efdpa")
    M, N, K = 96, 64, 64
    A = g.integers(0, 1 << 16, (M, K), dtype=np.uint16)
    B = g.integers(0, 1 << 16, (N, K), dtype=np.uint16)
    C = g.integers(0, 1 << 32, (M, N), dtype=np.uint32)
    _check(key, {"A": A, "B": B, "C": C}, expect_kernel="efdpa")
    inp = wl.normal_inputs(key[1], key[2], M, N, K, seed=43)
    A = inp["A"].copy()
    A[:, 1::2] = inp["A"][:, 0::2] ^ 0x8000                # exact cancellation of neighbouring products in half the rows
    Bm = inp["B"].copy()
    Bm[:, 1::2] = inp["B"][:, 0::2]
    A[M // 2:], Bm[N // 2:] = inp["A"][M // 2:], inp["B"][N // 2:]
    A[g.random((M, K)) < 0.05] = 0                         # zeros: +0 and -0
    A[g.random((M, K)) < 0.02] = 0x8000
    field = g.choice(np.r_[0:4, 100:150, 250:255], (M, N)).astype(np.uint32)
    C = ((g.integers(0, 2, (M, N)).astype(np.uint32) << 31) | (field << 23) | g.integers(0, 1 << 23, (M, N)).astype(np.uint32)).astype(np.uint32)
    C[g.random((M, N)) < 0.1] = 0x80000000
    _check(key, {"A": A, "B": Bm, "C": C}, expect_kernel="efdpa")


@pytest.mark.parametrize("key", GST_KEYS, ids=lambda k: "-".join(k))
def test_gst_fdpa_sparse_groups(key):
    # mostly zero codes (+0 and -0), so that groups with and without a nonzero product mix inside every micro-tile and the
    # per-element nonzero masks decide e_max; scale factors over a wide band, zero scale bytes for NVFP4; small
    # accumulators, so that a group counted or not counted in e_max changes the result
    g = wl.rng(73)
    M, N, K = 140, 90, 256
    kb = 16 if key[1] == "nvf4" else 32

    def sparse(rows):
        codes = g.integers(0, 16, (rows, K)).astype(np.uint8)
        codes[g.random((rows, K)) < 0.8] = 0
        codes[g.random((rows, K)) < 0.05] = 8                       # -0
        codes[: rows // 4] = g.integers(0, 16, (rows // 4, K))          # a dense quarter
        return (codes[:, 0::2] | (codes[:, 1::2] << 4)).astype(np.uint8)

    lo, hi = (0x08, 0x68) if key[1] == "nvf4" else (90, 160)
    sfa = g.integers(lo, hi, (M, K // kb), dtype=np.uint8)
    sfb = g.integers(lo, hi, (N, K // kb), dtype=np.uint8)
    if key[1] == "nvf4":
        sfa[g.random(sfa.shape) < 0.05] = 0
        sfb[g.random(sfb.shape) < 0.05] = 0x80
    C = (g.standard_normal((M, N)) * 2.0 ** g.integers(-40, 10, (M, N))).astype(np.float32).view(np.uint32)
    C[g.random((M, N)) < 0.2] = 0
    inp = {"A": sparse(M), "B": sparse(N), "C": C, "sfa": sfa, "sfb": sfb}
    _check(key, inp, expect_kernel="gstfdpa")


def test_no_bulk_copy_wait_gave_up():
    # the tuned kernels count CTAs whose bounded wait on a bulk copy ran out (such a CTA stores nothing): after real work
    # on this device the counter is still zero
    from paper_2511_10909_b200 import mmasim
    for key in (("hopper", "e4m3", "fp32"), ("hopper", "fp16", "fp32"), ("cdna3", "bf16", "fp32"), ("cdna1", "fp16", "fp32")):
        inp = wl.normal_inputs(key[1], key[2], 256, 192, 128, seed=81)
        gu.run_gemm(key, inp)
    assert mmasim.copy_timeouts() == 0
