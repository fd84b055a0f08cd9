"""GPU parity: the CUDA library against the CPU oracle, bit for bit, through the C ABI.

Small cases compare every output; the full-size configurations compare seeded samples of outputs that the oracle
computes one by one.  Integer / bit-pattern work: the bar is exact equality of every output word.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2511_10909_b200 import workloads as wl

pytestmark = pytest.mark.gpu

gu = pytest.importorskip("gpu_util") if torch.cuda.is_available() else None


def _all_pairs(M, N):
    return np.stack(np.meshgrid(np.arange(M), np.arange(N), indexing="ij"), axis=-1).reshape(-1, 2)


# ---- config 1: FP16 256^3 under the Volta FP16 -> FP32 model, every output -------------------------------
def test_cfg1_every_output():
    A, B, C = wl.cfg1()
    inp = {"A": A, "B": B, "C": C}
    key = ("volta", "fp16", "fp32")
    D = gu.run_gemm(key, inp)
    pairs = _all_pairs(256, 256)
    gu.assert_samples_equal(D, gu.oracle_samples(key, inp, pairs), pairs, "cfg1")
    # C = NULL means +0
    D2 = gu.run_gemm(key, {"A": A, "B": B})
    assert np.array_equal(D, D2)


# ---- every registry row on a small ragged shape, every output sampled densely -----------------------------
ALL_KEYS = sorted(oracle.REGISTRY)


@pytest.mark.parametrize("key", ALL_KEYS, ids=lambda k: "-".join(k))
def test_every_model_small(key):
    m = oracle.lookup(*key)
    M, N = 37, 29                                        # not multiples of any tile
    K = 192 if m.family != "fma" else 67
    inp = wl.normal_inputs(key[1], key[2], M, N, K, seed=11)
    D = gu.run_gemm(key, inp)
    pairs = _all_pairs(M, N)[::3]
    gu.assert_samples_equal(D, gu.oracle_samples(key, inp, pairs), pairs, str(key))


# ---- adversarial words for every unscaled model through dot_batch (classes of config 4 at reduced n) -------
DOT_MODELS = [("cdna2", "fp16", "fp32"), ("cdna2", "bf16", "fp32"), ("cdna2", "bf16_1k", "fp32"),
              ("hopper", "fp16", "fp32"), ("hopper", "bf16", "fp32"), ("hopper", "tf32", "fp32"),
              ("hopper", "fp16", "fp16"), ("volta", "fp16", "fp32"), ("ampere", "tf32", "fp32"),
              ("cdna3", "fp16", "fp32"), ("cdna3", "bf16", "fp32"), ("cdna3", "tf32", "fp32"),
              ("cdna1", "fp16", "fp32"), ("cdna1", "bf16", "fp32")]


def _dot_case(key, K, n):
    from paper_2511_10909_b200 import mmasim
    m = oracle.lookup(*key)
    A, B, C = wl.cfg4(m.elem, K, n=n)
    if key[2] == "fp16":
        C = (C >> 16).astype(np.uint16)                  # top half of the FP32 word: an arbitrary FP16 word
    model = mmasim.Model(*key)
    D = gu.host_words(mmasim.dot_batch(model, gu.dev(A), gu.dev(B), gu.dev(C)))
    return m, A, B, C, D


@pytest.mark.parametrize("key", DOT_MODELS, ids=lambda k: "-".join(k))
@pytest.mark.parametrize("K", [4, 8, 16, 32])
def test_cfg4_classes_every_dot(key, K):
    n = 1 << 13
    m, A, B, C, D = _dot_case(key, K, n)
    want = oracle.phi_dot_batch(m, A, B, C)
    bad = np.flatnonzero(D.astype(np.uint64) != want)
    assert bad.size == 0, (key, K, bad[:5], [hex(int(D[i])) for i in bad[:5]], [hex(int(want[i])) for i in bad[:5]])


# ---- ragged dot batches: a last tile that is not full (odd row counts for 8-byte rows), row lengths that are staged
# through shared memory (8..128 bytes) and row lengths that are read directly (48, 96, 256 bytes, ...) -----------------
@pytest.mark.parametrize("key,K,n", [
    (("volta", "fp16", "fp32"), 4, 777), (("volta", "fp16", "fp32"), 4, 1), (("volta", "fp16", "fp16"), 12, 515),
    (("hopper", "fp16", "fp32"), 32, 1283), (("hopper", "fp16", "fp32"), 64, 300), (("hopper", "fp16", "fp32"), 48, 300),
    (("hopper", "fp16", "fp16"), 128, 259), (("hopper", "bf16", "fp32"), 16, 257), (("hopper", "bf16", "fp32"), 80, 255),
    (("hopper", "tf32", "fp32"), 32, 511), (("hopper", "tf32", "fp32"), 24, 513), (("ampere", "tf32", "fp32"), 4, 130),
    (("cdna2", "fp16", "fp32"), 4, 1001), (("cdna2", "fp16", "fp32"), 64, 258), (("cdna2", "fp16", "fp32"), 20, 258),
    (("cdna2", "bf16", "fp32"), 8, 3), (("cdna2", "bf16_1k", "fp32"), 24, 600), (("cdna2", "bf16", "fp32"), 256, 70),
], ids=str)
def test_dot_batch_ragged(key, K, n):
    from paper_2511_10909_b200 import mmasim
    m, A, B, C, D = _dot_case(key, K, n)
    assert mmasim.last_kernel() in ("dot_tfdpa", "dot_ftz")
    want = oracle.phi_dot_batch(m, A, B, C)
    bad = np.flatnonzero(D.astype(np.uint64) != want)
    assert bad.size == 0, (key, K, n, bad[:5], [hex(int(D[i])) for i in bad[:5]], [hex(int(want[i])) for i in bad[:5]])


# ---- config 4 at full size: 2^20 dots, EVERY dot checked (all eight classes), the CDNA2 models and an NVIDIA model in
# each of the three formats, K = 4, 8, 16, 32 ----
CFG4_FULL = [("cdna2", "fp16", "fp32"), ("cdna2", "bf16", "fp32"), ("cdna2", "bf16_1k", "fp32"),
             ("hopper", "fp16", "fp32"), ("hopper", "bf16", "fp32"), ("hopper", "tf32", "fp32")]


@pytest.mark.parametrize("K", [4, 8, 16, 32])
@pytest.mark.parametrize("key", CFG4_FULL, ids=lambda k: "-".join(k))
def test_cfg4_full_size_every_dot(key, K):
    from paper_2511_10909_b200 import mmasim
    n = 1 << 20
    m, A, B, C, D = _dot_case(key, K, n)
    assert mmasim.last_kernel() in ("dot_tfdpa", "dot_ftz")
    want = oracle.phi_dot_batch(m, A, B, C)
    bad = np.flatnonzero(D.astype(np.uint64) != want)
    assert bad.size == 0, (key, K, bad.size, bad[:5], [hex(int(D[i])) for i in bad[:5]], [hex(int(want[i])) for i in bad[:5]])


# ---- config 2: BF16 2048^3 under the Ampere model; 65 536 sampled outputs and four full lines (two rows, two columns) -----------------------
def test_cfg2_sampled():
    A, B, C = wl.cfg2()
    inp = {"A": A, "B": B, "C": C}
    key = ("ampere", "bf16", "fp32")
    D = gu.run_gemm(key, inp)
    pairs = np.concatenate([wl.sample_pairs(2048, 2048, 65536, seed=2),
                            np.stack([np.full(2048, 5), np.arange(2048)], 1),
                            np.stack([np.full(2048, 2047), np.arange(2048)], 1),
                            np.stack([np.arange(2048), np.full(2048, 0)], 1),
                            np.stack([np.arange(2048), np.full(2048, 2047)], 1)])
    gu.assert_samples_equal(D, gu.oracle_samples(key, inp, pairs), pairs, "cfg2")


# ---- config 3: E4M3 4096^3 under the Hopper FP8 model, plain and with FP32 promotion every 128 -------------
@pytest.fixture(scope="module")
def cfg3_inputs():
    A, B, C, sa, sb = wl.cfg3()
    return {"A": A, "B": B, "C": C, "sa": sa, "sb": sb}


def test_cfg3_plain_sampled(cfg3_inputs):
    key = ("hopper", "e4m3", "fp32")
    inp = cfg3_inputs
    D = gu.run_gemm(key, inp)
    pairs = wl.sample_pairs(4096, 4096, 16384, seed=3)
    gu.assert_samples_equal(D, gu.oracle_samples(key, inp, pairs), pairs, "cfg3")


def test_cfg3_chunk128_promotion_and_dequant(cfg3_inputs):
    key = ("hopper", "e4m3", "fp32")
    inp = cfg3_inputs
    D = gu.run_gemm(key, inp, k_chunk=128, row_scale=gu.dev(inp["sa"]), col_scale=gu.dev(inp["sb"]))
    pairs = wl.sample_pairs(4096, 4096, 16384, seed=33)
    want = gu.oracle_samples(key, inp, pairs, k_chunk=128, row_scale=inp["sa"].view(np.uint32),
                             col_scale=inp["sb"].view(np.uint32))
    gu.assert_samples_equal(D, want, pairs, "cfg3 chunk 128")


# ---- interface properties ------------------------------------------------------------------------------
def test_independence_of_outputs():
    # Section 3.1, Step 1: replicated rows and columns give bitwise identical outputs everywhere
    from paper_2511_10909_b200 import mmasim
    g = wl.rng(9)
    K = 64
    a = wl.cast(g.standard_normal(K), "fp16")
    b = wl.cast(g.standard_normal(K), "fp16")
    A, B = np.tile(a, (50, 1)), np.tile(b, (70, 1))
    C = np.full((50, 70), 0x3E000000, dtype=np.uint32)
    for key in (("hopper", "fp16", "fp32"), ("cdna3", "fp16", "fp32"), ("cdna2", "fp16", "fp32")):
        D = gu.run_gemm(key, {"A": A, "B": B, "C": C})
        assert (D == D[0, 0]).all()


def test_c_aliases_d():
    from paper_2511_10909_b200 import mmasim
    inp = wl.normal_inputs("bf16", "fp32", 40, 24, 64, seed=12)
    key = ("hopper", "bf16", "fp32")
    want = gu.run_gemm(key, inp)
    model = mmasim.Model(*key)
    CD = gu.dev(inp["C"])
    mmasim.gemm(model, gu.dev(inp["A"]), gu.dev(inp["B"]), CD, out=CD)
    assert np.array_equal(gu.host_words(CD), want)


def test_host_entry_point_matches_device_entry_point():
    from paper_2511_10909_b200 import mmasim
    inp = wl.normal_inputs("mxe4m3", "fp32", 33, 17, 128, seed=13)
    key = ("blackwell", "mxe4m3", "fp32")
    want = gu.run_gemm(key, inp)
    got = mmasim.gemm_host(mmasim.Model(*key), inp["A"], inp["B"], inp["C"], sfa=inp["sfa"], sfb=inp["sfb"])
    assert np.array_equal(got, want)


@pytest.mark.parametrize("key, K", [(("hopper", "e4m3", "fp32"), 1024), (("blackwell", "mxe4m3", "fp32"), 512),
                                    (("blackwell", "nvf4", "fp32"), 512), (("hopper", "fp16", "fp16"), 512)],
                         ids=lambda k: "-".join(k) if isinstance(k, tuple) else str(k))
def test_host_entry_point_in_row_panels(key, K):
    # large enough for the panel pipeline of the host entry point (>= 1024 rows, >= 32 MiB), ragged last panel
    from paper_2511_10909_b200 import mmasim
    M, N = 4000 + 72, 3072
    inp = wl.normal_inputs(key[1], key[2], M, N, K, seed=14)
    model = mmasim.Model(*key)
    kw = {}
    if key[1] == "e4m3":
        g = wl.rng(15)
        kw = dict(k_chunk=128, row_scale=g.standard_normal(M).astype(np.float32), col_scale=g.standard_normal(N).astype(np.float32))
    dkw = {k: (gu.dev(v) if isinstance(v, np.ndarray) else v) for k, v in kw.items()}
    want = gu.run_gemm(key, inp, **dkw)
    got = mmasim.gemm_host(model, inp["A"], inp["B"], inp["C"], sfa=inp.get("sfa"), sfb=inp.get("sfb"), **kw)
    assert np.array_equal(got.view(want.dtype), want)


def test_device_errors():
    from paper_2511_10909_b200 import mmasim
    model = mmasim.Model("hopper", "fp16", "fp32")
    A = torch.zeros((4, 16), dtype=torch.int16, device="cuda")
    with pytest.raises(mmasim.MmasimError) as e:
        mmasim.gemm(model, A, A, K=24, M=2, N=2)                                     # K not a multiple of L
    assert e.value.status == 3
    import ctypes
    host = np.zeros((4, 16), dtype=np.uint16)
    st = mmasim._lib.mmasim_gemm(model._h, 4, 4, 16, ctypes.c_void_p(host.ctypes.data), ctypes.c_void_p(A.data_ptr()),
                                 None, ctypes.c_void_p(A.data_ptr()), None)
    assert st == 1                                                               # host pointer rejected
