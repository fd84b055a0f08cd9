"""Leading dimensions and out-of-bounds stores: the bounds evidence of the GEMM entry points.

Every matrix sits inside a larger buffer filled with sentinel words: A, B (packed FP4 included), the scale-factor
matrices and C are surrounded by words that would poison the result if a kernel consumed them (NaN patterns where the
format has one), and D by canary words that must be intact afterwards.  Shapes are ragged against every tile size
(128 x 128, 128 x 64, 64 x 128, 16 x 16).  Row strides come in two kinds: a multiple of 16 bytes, which the tuned
kernels accept, and an odd one, which only the generic kernels take; ldc differs from ldd.  Every output word is
compared with the oracle.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_10909_b200 import workloads as wl

pytestmark = pytest.mark.gpu

gu = pytest.importorskip("gpu_util") if torch.cuda.is_available() else None

# one model per kernel template
KEYS = [("hopper", "e4m3", "fp32"), ("hopper", "e4m3", "fp16"), ("hopper", "e5m2", "fp32"), ("ada", "e4m3", "fp32"),
        ("hopper", "fp16", "fp32"), ("volta", "fp16", "fp16"), ("ampere", "bf16", "fp32"), ("hopper", "tf32", "fp32"),
        ("blackwell", "e4m3", "fp32"), ("blackwell", "e2m1", "fp16"), ("blackwell", "mxe4m3", "fp32"),
        ("blackwell", "mxf4", "fp32"), ("blackwell", "nvf4", "fp32"),
        ("cdna3", "bf16", "fp32"), ("cdna3", "tf32", "fp32"), ("cdna3", "e4m3", "fp32"),
        ("cdna1", "fp16", "fp32"), ("cdna1", "bf16", "fp32"), ("cdna2", "fp16", "fp32"), ("cdna2", "bf16", "fp32"),
        ("cdna1", "fp32", "fp32"), ("hopper", "fp64", "fp64")]
SHAPES = [(129, 65), (1, 127), (255, 1), (130, 129)]
CANARY = 0xA5


def _embed(x, ld_words, pre_words, fill):
    """Places the 2-D array x (storage words) into a flat sentinel-filled buffer with the given row stride, `pre_words`
    words before the first row and as many behind the last; returns (device buffer, device view of x)."""
    rows, cols = x.shape
    total = pre_words + (rows - 1) * ld_words + cols + pre_words
    buf = np.full(total, fill, dtype=x.dtype)
    view = np.lib.stride_tricks.as_strided(buf[pre_words:], shape=(rows, cols), strides=(ld_words * x.itemsize, x.itemsize))
    view[...] = x
    t = gu.dev(buf)
    return t, t[pre_words:].as_strided((rows, cols), (ld_words, 1))


def _poison(dtype):
    return np.array(-1).astype(np.int64).astype(dtype)                 # all ones: NaN in every format that has one


@pytest.mark.parametrize("aligned", [True, False], ids=["ld16", "ldodd"])
@pytest.mark.parametrize("shape", SHAPES, ids=lambda s: f"{s[0]}x{s[1]}")
@pytest.mark.parametrize("key", KEYS, ids=lambda k: "-".join(k))
def test_padded_strides_and_canaries(key, shape, aligned):
    from paper_2511_10909_b200 import mmasim
    M, N = shape
    K = 64
    m = oracle.lookup(*key)
    inp = wl.normal_inputs(key[1], key[2], M, N, K, seed=21)
    model = mmasim.Model(*key)
    packed = key[1] in ("mxf4", "nvf4")
    A, B, C = inp["A"], inp["B"], inp["C"]
    wa = A.dtype.itemsize
    # leading dimensions in storage words: +16 bytes keeps the 16-byte row starts of the tuned kernels, +3 words (one
    # byte for packed FP4, whose leading dimension in elements must stay even) does not
    pad_in = 16 // wa if aligned else (1 if packed else 3)
    lda, ldb = A.shape[1] + pad_in, B.shape[1] + 2 * pad_in
    ldc, ldd = N + 5, N + 12
    align_words = lambda x: 64 // x.dtype.itemsize                     # keeps every base pointer 16-byte aligned
    bufA, vA = _embed(A, lda, align_words(A), _poison(A.dtype))
    bufB, vB = _embed(B, ldb, align_words(B), _poison(B.dtype))
    bufC, vC = _embed(C, ldc, align_words(C), _poison(C.dtype))
    canary = np.frombuffer(bytes([CANARY]) * C.dtype.itemsize, dtype=C.dtype)[0]
    bufD, vD = _embed(np.full((M, N), canary, dtype=C.dtype), ldd, align_words(C), canary)
    kw = {}
    if "sfa" in inp:
        # scale matrices are packed (one row stride = scales per row); sentinel rows before and behind them
        bufSA, vSA = _embed(inp["sfa"], inp["sfa"].shape[1], 64, np.uint8(0xFF))
        bufSB, vSB = _embed(inp["sfb"], inp["sfb"].shape[1], 64, np.uint8(0xFF))
        kw = dict(sfa=vSA, sfb=vSB)
    D = mmasim.gemm(model, vA, vB, vC, out=vD, K=K, **kw)
    torch.cuda.synchronize()
    kernel = mmasim.last_kernel()
    if aligned:
        assert kernel != "generic", kernel                             # every model of KEYS has a tuned kernel
    else:
        assert kernel == "generic", kernel
    got = gu.host_words(D)
    want = gu.oracle_samples(key, inp, np.stack(np.meshgrid(np.arange(M), np.arange(N), indexing="ij"), -1).reshape(-1, 2))
    assert np.array_equal(got.astype(np.uint64).reshape(-1), want), (key, shape, kernel)
    # canaries: everything in D's buffer outside the M x N view is untouched
    whole = gu.host_words(bufD).copy()
    pre = align_words(C)
    mask = np.ones(whole.shape, dtype=bool)
    idx = pre + (np.arange(M)[:, None] * ldd + np.arange(N)[None, :])
    mask[idx.reshape(-1)] = False
    assert (whole[mask] == canary).all(), (key, shape, kernel, int((whole[mask] != canary).sum()))
    # the inputs are untouched too
    for buf, view, src in ((bufA, vA, A), (bufB, vB, B), (bufC, vC, C)):
        assert np.array_equal(gu.host_words(view.contiguous()), src)


@pytest.mark.parametrize("key", [("hopper", "e4m3", "fp32"), ("blackwell", "nvf4", "fp32"), ("cdna3", "bf16", "fp32")],
                         ids=lambda k: "-".join(k))
def test_host_entry_point_with_leading_dimensions(key):
    # the same call on host buffers: strided numpy views go through mmasim_gemm_host with their strides
    from paper_2511_10909_b200 import mmasim
    M, N, K = 70, 45, 128
    inp = wl.normal_inputs(key[1], key[2], M, N, K, seed=22)
    want = gu.run_gemm(key, inp)

    def strided(x, extra):
        buf = np.full((x.shape[0], x.shape[1] + extra), 0xFF, dtype=x.dtype)
        buf[:, :x.shape[1]] = x
        return buf[:, :x.shape[1]]

    out_buf = np.full((M, N + 7), 0xA5A5A5A5, dtype=np.uint32)
    got = mmasim.gemm_host(mmasim.Model(*key), strided(inp["A"], 16), strided(inp["B"], 32), strided(inp["C"], 3),
                           K=K, sfa=inp.get("sfa"), sfb=inp.get("sfb"), out=out_buf[:, :N])
    assert np.array_equal(got, want)
    assert (out_buf[:, N:] == 0xA5A5A5A5).all()


def test_chunk_promotion_and_dequant_with_leading_dimensions():
    # the FP32-promotion variant of the tuned F = 13 kernel and its dequantisation epilogue on strided operands
    from paper_2511_10909_b200 import mmasim
    key = ("hopper", "e4m3", "fp32")
    M, N, K = 131, 67, 256
    inp = wl.normal_inputs(key[1], key[2], M, N, K, seed=23)
    g = wl.rng(24)
    sa, sb = g.standard_normal(M).astype(np.float32), g.standard_normal(N).astype(np.float32)
    _, vA = _embed(inp["A"], K + 16, 64, np.uint8(0xFF))
    _, vB = _embed(inp["B"], K + 48, 64, np.uint8(0xFF))
    _, vC = _embed(inp["C"], N + 1, 16, np.uint32(0xFFFFFFFF))
    bufD, vD = _embed(np.full((M, N), 0xA5A5A5A5, dtype=np.uint32), N + 9, 16, np.uint32(0xA5A5A5A5))
    model = mmasim.Model(*key)
    mmasim.gemm(model, vA, vB, vC, out=vD, k_chunk=128, row_scale=gu.dev(sa), col_scale=gu.dev(sb))
    torch.cuda.synchronize()
    assert mmasim.last_kernel() == "tfdpa_lut8"
    pairs = np.stack(np.meshgrid(np.arange(M), np.arange(N), indexing="ij"), -1).reshape(-1, 2)
    want = gu.oracle_samples(key, inp, pairs, k_chunk=128, row_scale=sa.view(np.uint32), col_scale=sb.view(np.uint32))
    assert np.array_equal(gu.host_words(vD.contiguous()).astype(np.uint64).reshape(-1), want)
    whole = gu.host_words(bufD)
    assert int((whole == 0xA5A5A5A5).sum()) == whole.size - M * N
