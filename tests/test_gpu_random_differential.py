"""Randomised differential test of the tuned kernels: seeded random shapes (ragged tiles), value mixes (random bit
streams with NaN / infinities / subnormals, ordinary values, many zeros and exactly cancelling products) and
accumulators of every exponent, every output compared with the generic kernel (which `test_gpu_parity.py` checks
against the oracle) and a sample of outputs with the oracle itself."""
import numpy as np
import pytest
import torch

from paper_2511_10909_b200 import workloads as wl

pytestmark = pytest.mark.gpu

gu = pytest.importorskip("gpu_util") if torch.cuda.is_available() else None

CASES = [
    # (arch, A type, accumulator, B type or None, kernel name)
    ("hopper", "e4m3", "fp32", None, "tfdpa_lut8"), ("hopper", "e5m2", "fp32", None, "tfdpa_lut8"),
    ("hopper", "e4m3", "fp32", "e5m2", "tfdpa_lut8"), ("ada", "e5m2", "fp16", "e4m3", "tfdpa_lut8"),
    ("ada", "e4m3", "fp32", None, "tfdpa_lut8"), ("hopper", "e4m3", "fp16", None, "tfdpa_lut8"),
    ("blackwell", "e4m3", "fp32", None, "tfdpa_lut8"), ("hopper", "fp16", "fp32", None, "tfdpa_f16"),
    ("ampere", "bf16", "fp32", None, "tfdpa_bf16"), ("ampere", "tf32", "fp32", None, "tfdpa_tf32"),
    ("cdna3", "fp16", "fp32", None, "trfdpa"), ("cdna3", "tf32", "fp32", None, "trfdpa"),
    ("cdna3", "e4m3", "fp32", None, "gtrfdpa"), ("cdna1", "fp16", "fp32", None, "efdpa"), ("cdna1", "bf16", "fp32", None, "efdpa"),
]


def _words(g, fmt, rows, K, mode, seed):
    bits = {"e4m3": 8, "e5m2": 8, "fp16": 16, "bf16": 16, "tf32": 32}[fmt]
    dt = {8: np.uint8, 16: np.uint16, 32: np.uint32}[bits]
    if mode == 0:
        return g.integers(0, 1 << bits, (rows, K), dtype=np.uint64).astype(dt)
    X = wl.normal_inputs(fmt, "fp32", rows, rows, K, seed=seed)["A"].copy()
    if mode == 2:
        X[g.random((rows, K)) < 0.1] = 0
        X[g.random((rows, K)) < 0.03] = dt(1 << (bits - 1))           # -0
    return X


@pytest.mark.parametrize("case", CASES, ids=lambda c: "-".join(x for x in c[:4] if x))
@pytest.mark.parametrize("seed", range(3))
def test_tuned_kernel_equals_generic_kernel_and_oracle(case, seed):
    import oracle
    from paper_2511_10909_b200 import mmasim
    arch, fa, acc, fb, kernel = case
    fb = fb or fa
    g = wl.rng(3100 + 17 * seed + CASES.index(case))
    mode = seed % 3
    M, N, K = int(g.integers(1, 330)), int(g.integers(1, 330)), 32 * int(g.integers(1, 5))
    A, B = _words(g, fa, M, K, mode, 2 * seed), _words(g, fb, N, K, mode, 2 * seed + 1)
    if mode == 2:                                                     # products that cancel exactly in some rows
        sign = A.dtype.type(1 << (8 * A.dtype.itemsize - 1))
        rows = np.arange(0, M, 3)
        A[rows, 1::2] = A[rows, 0::2] ^ sign
        if fa == fb:
            B[:, 1::2] = B[:, 0::2]
    if acc == "fp16":
        C = g.integers(0, 1 << 16, (M, N)).astype(np.uint16)
    else:
        field = g.choice(np.r_[0:6, 90:170, 236:256], (M, N)).astype(np.uint32)
        C = ((g.integers(0, 2, (M, N)).astype(np.uint32) << 31) | (field << 23) |
             g.integers(0, 1 << 23, (M, N)).astype(np.uint32)).astype(np.uint32)
        C[g.random((M, N)) < 0.1] = 0x80000000 if mode == 2 else 0
    model = mmasim.Model(arch, fa, acc, b_fmt=fb)
    dA, dB, dC = gu.dev(A), gu.dev(B), gu.dev(C)
    D = mmasim.gemm(model, dA, dB, dC)
    assert mmasim.last_kernel() == kernel
    G = mmasim.gemm(model, dA, dB, dC, force_generic=True)
    assert mmasim.last_kernel() == "generic"
    torch.cuda.synchronize()
    diff = (D != G).nonzero()
    assert diff.shape[0] == 0, (case, (M, N, K), mode, diff.shape[0], diff[:4].tolist())
    if fa == fb:                                                      # the oracle's registry holds equal-type rows
        pairs = wl.sample_pairs(M, N, 60, seed=seed)
        want = oracle.phi_gemm_sampled(oracle.lookup(arch, fa, acc), A, B, C, pairs)
        gu.assert_samples_equal(gu.host_words(D), want, pairs, str(case))
