"""Config 5 at full size: models of every family at 8192 x 8192 x 8192 with A, B ~ N(0,1) in each format and
C ~ N(0,1); seeded sampled outputs are compared bit for bit with the oracle.  The default run covers one model per
family / element kind; MMASIM_FULL_SWEEP=1 covers all 86 registry rows (several minutes)."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2511_10909_b200 import workloads as wl

pytestmark = pytest.mark.gpu
gu = pytest.importorskip("gpu_util") if torch.cuda.is_available() else None

SIZE = 8192
SUBSET = [("hopper", "e4m3", "fp32"), ("blackwell", "fp16", "fp16"), ("volta", "fp16", "fp32"), ("ampere", "bf16", "fp32"),
          ("hopper", "tf32", "fp32"), ("blackwell", "mxe4m3", "fp32"), ("blackwell", "nvf4", "fp32"), ("cdna3", "fp16", "fp32"),
          ("cdna3", "e5m2", "fp32"), ("cdna2", "fp16", "fp32"), ("cdna1", "fp16", "fp32"), ("cdna3", "fp32", "fp32")]
KEYS = sorted(oracle.REGISTRY) if os.environ.get("MMASIM_FULL_SWEEP") == "1" else SUBSET
_cache = {}


def _inputs(in_fmt, acc):
    ck = (in_fmt, acc)
    if ck not in _cache:
        _cache.clear()                                   # one 8192^2 input set in host memory at a time
        _cache[ck] = wl.normal_inputs(in_fmt, acc, SIZE, SIZE, SIZE, seed=5)
    return _cache[ck]


@pytest.mark.parametrize("key", sorted(KEYS, key=lambda k: (k[1], k[2], k[0])), ids=lambda k: "-".join(k))
def test_cfg5_sampled_outputs(key):
    inp = _inputs(key[1], key[2])
    D = gu.run_gemm(key, inp)
    n = 1024 if oracle.lookup(*key).family != "fma" else 256          # the FMA chain oracle is the slowest per MAC
    pairs = wl.sample_pairs(SIZE, SIZE, n, seed=55)
    gu.assert_samples_equal(D, gu.oracle_samples(key, inp, pairs), pairs, "-".join(key))
