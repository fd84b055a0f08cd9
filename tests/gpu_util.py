"""Shared plumbing of the GPU parity tests: upload words, run the library, run the oracle, compare bit for bit."""
import numpy as np
import torch

import oracle
from paper_2511_10909_b200 import mmasim, workloads as wl

_SIGNED = {np.dtype(np.uint8): np.uint8, np.dtype(np.uint16): np.int16, np.dtype(np.uint32): np.int32,
           np.dtype(np.uint64): np.int64}
_UNSIGNED = {1: np.uint8, 2: np.uint16, 4: np.uint32, 8: np.uint64}


def dev(x):
    if x is None:
        return None
    x = np.ascontiguousarray(x)
    return torch.from_numpy(x.view(_SIGNED.get(x.dtype, x.dtype))).cuda()


def host_words(t):
    a = t.cpu().numpy()
    return a.view(_UNSIGNED[a.dtype.itemsize])


def unpack_fp4(packed):
    out = np.empty(packed.shape[:-1] + (packed.shape[-1] * 2,), dtype=np.uint8)
    out[..., 0::2] = packed & 0xF
    out[..., 1::2] = packed >> 4
    return out


def run_gemm(key, inp, **kw):
    """inp: dict with A, B, C (+ sfa, sfb).  Returns the M x N output words (numpy, unsigned)."""
    model = mmasim.Model(*key)
    D = mmasim.gemm(model, dev(inp["A"]), dev(inp["B"]), dev(inp.get("C")),
                    sfa=dev(inp.get("sfa")), sfb=dev(inp.get("sfb")), **kw)
    torch.cuda.synchronize()
    return host_words(D)


def oracle_samples(key, inp, pairs, **kw):
    m = oracle.lookup(*key)
    A, B = inp["A"], inp["B"]
    if key[1] in ("mxf4", "nvf4"):
        A, B = unpack_fp4(A), unpack_fp4(B)
    return oracle.phi_gemm_sampled(m, A, B, inp.get("C"), pairs, SFA=inp.get("sfa"), SFB=inp.get("sfb"), **kw)


def assert_samples_equal(D, want, pairs, what=""):
    got = D[pairs[:, 0], pairs[:, 1]].astype(np.uint64)
    bad = np.flatnonzero(got != want)
    assert bad.size == 0, (f"{what}: {bad.size} of {len(want)} sampled outputs differ; first at "
                           f"{tuple(pairs[bad[0]])}: got {int(got[bad[0]]):#x}, oracle {int(want[bad[0]]):#x}")
