"""Self-probing through the C ABI: the probes of Section 3.1 (Steps 2 and 3) run against mmasim_dot_batch as a black
box and must recover the summation trees of Figure 2 and the (L_max, F, rho) rows of Table 4 from outputs alone."""
import numpy as np
import pytest
import torch

from paper_2511_10909_b200 import clfp

pytestmark = pytest.mark.gpu

gu = pytest.importorskip("gpu_util") if torch.cuda.is_available() else None


def library_target(key):
    from paper_2511_10909_b200 import mmasim
    model = mmasim.Model(*key)
    in_fmt = {"bf16_1k": "bf16"}.get(key[1], key[1])

    def dot(A, B, C):
        return gu.host_words(mmasim.dot_batch(model, gu.dev(A), gu.dev(B), gu.dev(C)))
    return clfp.Target(in_fmt, key[2], dot)


@pytest.mark.parametrize("key,K,want", [
    (("cdna1", "fp32", "fp32"), 4, ("chain", {})),
    (("hopper", "fp64", "fp64"), 8, ("chain", {})),
    (("cdna2", "bf16", "fp32"), 8, ("pairwise", {"P": 2})),
    (("cdna2", "bf16_1k", "fp32"), 8, ("pairwise", {"P": 4})),
    (("cdna2", "fp16", "fp32"), 16, ("pairwise", {"P": 4})),
    (("cdna1", "bf16", "fp32"), 4, ("fused", {"L": 2, "swamped": False})),
    (("cdna1", "fp16", "fp32"), 8, ("fused", {"L": 4, "swamped": False})),
    (("cdna3", "bf16", "fp32"), 16, ("fused", {"L": 8, "swamped": True})),
    (("cdna3", "e5m2", "fp32"), 32, ("fused", {"L": 16, "swamped": True})),
])
def test_summation_trees_from_the_black_box(key, K, want):
    t = library_target(key)
    trees = clfp.infer_tree(clfp.swamp_matrix(t, K), K)
    assert trees and trees[0] == want, (key, trees)


@pytest.mark.parametrize("key,L,F,rho", [
    (("volta", "fp16", "fp32"), 4, 23, (23, "exact")),
    (("volta", "fp16", "fp16"), 4, 23, (10, "RNE")),
    (("turing", "fp16", "fp32"), 8, 24, (23, "undetermined")),
    (("ampere", "tf32", "fp32"), 4, 24, (23, "undetermined")),
    (("ampere", "bf16", "fp32"), 8, 24, (23, "undetermined")),
    (("ada", "e4m3", "fp32"), 16, 13, (13, "exact")),
    (("ada", "e5m2", "fp16"), 16, 13, (10, "RNE")),
    (("hopper", "tf32", "fp32"), 8, 25, (23, "RZ")),
    (("hopper", "bf16", "fp32"), 16, 25, (23, "RZ")),
    (("hopper", "fp16", "fp32"), 16, 25, (23, "RZ")),
    (("hopper", "fp16", "fp16"), 16, 25, (10, "RNE")),
    (("hopper", "e4m3", "fp32"), 32, 13, (13, "exact")),
    (("hopper", "e5m2", "fp16"), 32, 13, (10, "RNE")),
    (("blackwell", "e4m3", "fp32"), 32, 25, (23, "RZ")),
    (("blackwell", "e5m2", "fp16"), 32, 25, (10, "RNE")),
    (("rtx_blackwell", "bf16", "fp32"), 16, 25, (23, "RZ")),
])
def test_table_4_from_the_black_box(key, L, F, rho):
    t = library_target(key)
    got = clfp.characterise(t, 2 * L)
    assert got["trees"][0] == ("fused", {"L": L, "swamped": True}), got
    assert got["F"] == F and got["term_rounding"] == "RZ" and got["rho"] == rho, got


def test_probing_the_hardware_itself():
    """The same probes against the B200's mma.sync (one instruction = one dot product of 16 per output): a swamped fused
    summation of 16 products and the accumulator with 25 fractional bits, truncated terms, RZ to FP32 - the Blackwell
    row of Table 4, recovered from the machine."""
    from paper_2511_10909_b200 import mmasim
    if torch.cuda.get_device_capability(0)[0] != 10:
        pytest.skip("the hardware probe is about the B200")

    def dot(A, B, C):
        # n independent dots -> one 16-row tile each: row 0 of A holds a, the eight rows of B all hold b, c in column 0
        n, K = A.shape
        out = np.empty(n, dtype=np.uint32)
        for s in range(0, n, 512):
            a, b, c = A[s:s + 512], B[s:s + 512], C[s:s + 512]
            m = len(a)
            At = np.zeros((m * 16, K), dtype=A.dtype); At[0::16] = a
            Ct = np.zeros((m * 16, 8), dtype=np.uint32); Ct[0::16, 0] = c
            for t in range(m):              # B differs per dot: one launch per dot keeps the harness interface simple
                Bt = np.repeat(b[t:t + 1], 8, axis=0)
                D = gu.host_words(mmasim.hw_mma("f16_f32", gu.dev(At[16 * t:16 * t + 16]), gu.dev(Bt), gu.dev(Ct[16 * t:16 * t + 16])))
                out[s + t] = D[0, 0]
        return out

    t = clfp.Target("fp16", "fp32", dot)
    assert clfp.infer_tree(clfp.swamp_matrix(t, 16), 16)[0] == ("fused", {"L": 16, "swamped": True})
    assert clfp.fused_precision(t, 16) == 25
    assert clfp.term_rounding(t, 16, 25) == "RZ"
    assert clfp.output_conversion(t, 16, 25) == (23, "RZ")
