"""Every registry row on seeded random shapes: the kernel the dispatcher picks against the generic kernels on every output
word, and against the oracle on sampled outputs.  Two inputs per row: N(0,1) values in the row's format (with zero
elements and zero accumulators mixed in), and raw random bit patterns for A, B, C and the scale factors (NaN, infinity,
subnormals, any exponent spread).  Shapes are ragged against every tile size; K is a multiple of the row's block."""
import zlib

import numpy as np
import pytest
import torch

from paper_2511_10909_b200 import workloads as wl

pytestmark = pytest.mark.gpu

gu = pytest.importorskip("gpu_util") if torch.cuda.is_available() else None


def _keys():
    if not torch.cuda.is_available():
        return []
    from paper_2511_10909_b200 import mmasim
    return list(mmasim.model_keys())


def _word_dtype(nbytes):
    return {1: np.uint8, 2: np.uint16, 4: np.uint32, 8: np.uint64}[nbytes]


@pytest.mark.parametrize("key", _keys(), ids=lambda k: "-".join(k))
def test_row_on_random_shapes(key):
    from paper_2511_10909_b200 import mmasim
    g = wl.rng(zlib.crc32("-".join(key).encode()))
    model = mmasim.Model(*key)
    kmul = 64 if key[1] in ("mxf4", "nvf4") else 32
    M, N, K = int(g.integers(1, 300)), int(g.integers(1, 200)), kmul * int(g.integers(1, 6))
    # ---- ordinary values with zeros mixed in ----
    inp = wl.normal_inputs(key[1], key[2], M, N, K, seed=int(g.integers(1, 1 << 30)))
    A, B, C = inp["A"].copy(), inp["B"].copy(), inp["C"].copy()
    A[g.random(A.shape) < 0.1] = 0
    B[g.random(B.shape) < 0.05] = 0
    C[g.random(C.shape) < 0.2] = 0
    inp.update(A=A, B=B, C=C)
    D = gu.run_gemm(key, inp)
    kernel = mmasim.last_kernel()
    G = gu.run_gemm(key, inp, force_generic=True)
    assert mmasim.last_kernel() == "generic"
    bad = np.argwhere(D != G)
    assert bad.size == 0, (key, kernel, (M, N, K), len(bad), bad[:4])
    pairs = wl.sample_pairs(M, N, 64, seed=M * 1000 + N)
    gu.assert_samples_equal(D, gu.oracle_samples(key, inp, pairs), pairs, f"{key} {kernel} {(M, N, K)}")
    # ---- raw bit patterns ----
    wild = {"A": g.integers(0, 256, A.shape, dtype=np.uint8) if A.dtype.itemsize == 1
            else g.integers(0, 1 << (8 * A.dtype.itemsize - 1), A.shape, dtype=np.uint64).astype(_word_dtype(A.dtype.itemsize)) * 2
            + g.integers(0, 2, A.shape).astype(_word_dtype(A.dtype.itemsize))}
    wild["B"] = (g.integers(0, 256, B.shape, dtype=np.uint8) if B.dtype.itemsize == 1
                 else g.integers(0, 1 << (8 * B.dtype.itemsize - 1), B.shape, dtype=np.uint64).astype(_word_dtype(B.dtype.itemsize)) * 2
                 + g.integers(0, 2, B.shape).astype(_word_dtype(B.dtype.itemsize)))
    wild["C"] = (g.integers(0, 1 << (8 * C.dtype.itemsize - 1), C.shape, dtype=np.uint64).astype(_word_dtype(C.dtype.itemsize)) * 2
                 + g.integers(0, 2, C.shape).astype(_word_dtype(C.dtype.itemsize)))
    if key[1] not in ("mxf4", "nvf4") and A.dtype.itemsize == 1:
        # one element per byte in the low bits: keep the codes inside the format's width
        bits = model.a_bits if model.a_bits < 8 else 8
        width = {"e4m3": 8, "e5m2": 8, "e3m2": 6, "e2m3": 6, "e2m1": 4}.get(key[1].replace("mx", ""), bits)
        wild["A"] &= np.uint8((1 << width) - 1)
        wild["B"] &= np.uint8((1 << width) - 1)
    if "sfa" in inp:
        wild["sfa"] = g.integers(0, 256, inp["sfa"].shape, dtype=np.uint8)
        wild["sfb"] = g.integers(0, 256, inp["sfb"].shape, dtype=np.uint8)
    D = gu.run_gemm(key, wild)
    kernel = mmasim.last_kernel()
    G = gu.run_gemm(key, wild, force_generic=True)
    bad = np.argwhere(D != G)
    assert bad.size == 0, (key, kernel, (M, N, K), "bit patterns", len(bad), bad[:4])
    gu.assert_samples_equal(D, gu.oracle_samples(key, wild, pairs), pairs, f"{key} {kernel} {(M, N, K)} bit patterns")


def _raw_words(g, shape, itemsize):
    if itemsize == 1:
        return g.integers(0, 256, shape, dtype=np.uint8)
    return (g.integers(0, 1 << (8 * itemsize - 1), shape, dtype=np.uint64).astype(_word_dtype(itemsize)) * 2
            + g.integers(0, 2, shape).astype(_word_dtype(itemsize)))


_SMALL_WIDTH = {"e4m3": 8, "e5m2": 8, "e3m2": 6, "e2m3": 6, "e2m1": 4}


@pytest.mark.parametrize("seed", range(int(__import__("os").environ.get("MMASIM_PARITY_SEEDS", "3"))))
def test_rows_on_more_seeds_and_magnitudes(seed):
    """Every registry row again on further seeded shapes, the dispatcher's kernel against the generic kernels on every
    output word and against the oracle on 16 sampled outputs, with four inputs each: ordinary values with zeros, raw bit patterns, and the bit patterns with the top
    exponent bit of every word cleared (tiny products: zero and subnormal results) or set (huge ones: overflow, infinities
    and NaNs).  MMASIM_PARITY_SEEDS sets the number of seeds (default 3; 240 ran clean)."""
    from paper_2511_10909_b200 import mmasim
    for key in mmasim.model_keys():
        g = wl.rng(zlib.crc32(("-".join(key) + f"#{seed}").encode()))
        packed4 = key[1] in ("mxf4", "nvf4")
        kmul = 64 if packed4 else 32
        M, N, K = int(g.integers(1, 400)), int(g.integers(1, 300)), kmul * int(g.integers(1, 9))
        inp = wl.normal_inputs(key[1], key[2], M, N, K, seed=int(g.integers(1, 1 << 30)))
        A, B, C = inp["A"].copy(), inp["B"].copy(), inp["C"].copy()
        A[g.random(A.shape) < 0.1] = 0
        B[g.random(B.shape) < 0.05] = 0
        C[g.random(C.shape) < 0.2] = 0
        inp.update(A=A, B=B, C=C)
        cases = [("values", inp)]
        wild = {k: _raw_words(g, inp[k].shape, inp[k].dtype.itemsize) for k in ("A", "B", "C")}
        width = 8 * A.dtype.itemsize
        if not packed4 and A.dtype.itemsize == 1:
            width = _SMALL_WIDTH.get(key[1].replace("mx", ""), 8)
            wild["A"] &= np.uint8((1 << width) - 1)
            wild["B"] &= np.uint8((1 << width) - 1)
        if "sfa" in inp:
            wild["sfa"] = g.integers(0, 256, inp["sfa"].shape, dtype=np.uint8)
            wild["sfb"] = g.integers(0, 256, inp["sfb"].shape, dtype=np.uint8)
        cases.append(("bit patterns", wild))
        for name, setbit in (("small magnitudes", False), ("large magnitudes", True)):
            v = {k: x.copy() for k, x in wild.items()}
            for k in ("A", "B", "C"):
                if packed4 and k != "C":
                    continue
                top = v[k].dtype.type(1 << ((8 * C.dtype.itemsize if k == "C" else width) - 2))
                v[k] = (v[k] | top) if setbit else (v[k] & ~top)
            cases.append((name, v))
        for name, x in cases:
            D = gu.run_gemm(key, x)
            kernel = mmasim.last_kernel()
            G = gu.run_gemm(key, x, force_generic=True)
            bad = np.argwhere(D != G)
            assert bad.size == 0, (key, kernel, (M, N, K), name, len(bad), bad[:4])
            pairs = wl.sample_pairs(M, N, 16, seed=M * 1000 + N + seed)
            gu.assert_samples_equal(D, gu.oracle_samples(key, x, pairs), pairs, f"{key} {kernel} {(M, N, K)} {name}")
