"""Closed-loop feature probing (Section 3.1) of an MMA interface given as a black box.

The paper derives its models by probing hardware: Step 2 infers the summation tree from the outputs d(i,j) of inputs
that hold one huge product +U, one -U and otherwise a tiny product v (extended FPRev); Step 3 probes precision and
rounding of the fused summations.  This module runs those probes against any `dot(A, B, C) -> D` callable on raw
words (n x K, n x K, n -> n numpy arrays) - in this repository `mmasim_dot_batch`, so that the library can be asked
to re-derive the parameters of Tables 4-7 from its own behaviour - and against nothing else: it holds no model
arithmetic, only probe construction, the symbolic swamping rules of Figure 2 and the read-out of the results.

Limits: FP6 / FP4 element types are not probed (their exponent range cannot hold a swamping pair for F = 25), and the
tree search enumerates the families of Figure 2 (binary chain, fused blocks with the accumulator inside - swamped or
not -, pairwise groups), which is the paper's "enumerate and check" route, not FPRev's general construction.
"""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import Callable, Optional

import numpy as np

# name -> (exponent bits, mantissa bits, bias, storage bits, ignored low bits, has infinity)
_FMT = {
    "fp64": (11, 52, 1023, 64, 0, True), "fp32": (8, 23, 127, 32, 0, True), "tf32": (8, 10, 127, 32, 13, True),
    "bf16": (8, 7, 127, 16, 0, True), "bf16_1k": (8, 7, 127, 16, 0, True), "fp16": (5, 10, 15, 16, 0, True),
    "e5m2": (5, 2, 15, 8, 0, True), "e4m3": (4, 3, 7, 8, 0, False),
}
_DTYPE = {8: np.uint8, 16: np.uint16, 32: np.uint32, 64: np.uint64}


def word_dtype(fmt: str):
    return _DTYPE[_FMT[fmt][3]]


def encode(fmt: str, x: float) -> int:
    """The word of `fmt` whose value is exactly x (a ValueError if x is not representable)."""
    ebits, mbits, bias, bits, low, has_inf = _FMT[fmt]
    sign = 1 if math.copysign(1.0, x) < 0 else 0
    mag = abs(x)
    if mag == 0.0:
        return sign << (bits - 1)
    m, e = math.frexp(mag)                      # mag = m * 2**e, 0.5 <= m < 1
    exp = e - 1                                 # floor(log2 mag)
    emin = 1 - bias
    q = max(exp, emin) - mbits                  # exponent of the last kept bit
    n = mag / 2.0 ** q
    if n != int(n):
        raise ValueError(f"{x} is not a {fmt} value")
    n = int(n)
    top = (1 << ebits) - 1
    field = exp + bias if n >> mbits else 0
    if field >= top + (0 if has_inf else 1):
        raise ValueError(f"{x} overflows {fmt}")
    return ((sign << (ebits + mbits)) | (field << mbits) | (n & ((1 << mbits) - 1))) << low


def decode(fmt: str, w: int) -> float:
    """Value of an accumulator word (FP64 / FP32 / FP16)."""
    if fmt == "fp64":
        return float(np.array([w], dtype=np.uint64).view(np.float64)[0])
    if fmt == "fp32":
        return float(np.array([w], dtype=np.uint32).view(np.float32)[0])
    return float(np.array([w], dtype=np.uint16).view(np.float16)[0])


@dataclass
class Target:
    """An MMA interface under test: element format of A and B, accumulator format, and the dot callable."""
    in_fmt: str
    acc_fmt: str
    dot: Callable[[np.ndarray, np.ndarray, np.ndarray], np.ndarray]

    # exponents (eu, ev) of the swamping pair U = 2**eu, v = 2**ev, and the split of a product exponent over a and b
    def scales(self):
        ebits, mbits, bias, *_ = _FMT[self.in_fmt]
        emax, emin = (1 << ebits) - 2 - bias, 1 - bias
        if not _FMT[self.in_fmt][5]:
            emax += 1                           # E4M3: the top exponent field holds finite numbers
        hi, lo = 2 * min(emax, 50), 2 * max(emin, -50)
        if hi - lo < 40:                        # E4M3: only subnormal factors put v far enough below U (Equation 5)
            lo = 2 * (emin - mbits)
        if self.acc_fmt == "fp16":
            hi, lo = 15, -24
        return hi, lo, emin - mbits, emax

    def split(self, e: int):
        """(ea, eb) with ea + eb = e, both exponents of representable powers of two (subnormals included)."""
        _, _, lo_e, emax = self.scales()
        ea = max(min(e // 2, emax), lo_e)
        eb = e - ea
        if not lo_e <= eb <= emax:
            ea = e - max(min(eb, emax), lo_e)
            eb = e - ea
        if not (lo_e <= ea <= emax and lo_e <= eb <= emax):
            raise ValueError(f"2**{e} is not a product of two {self.in_fmt} values")
        return ea, eb

    def run(self, rows):
        """rows: list of (products, c); a product is (mantissa in {0, +-1, +-1.5}, exponent) or None (zero)."""
        K = len(rows[0][0])
        A = np.zeros((len(rows), K), dtype=word_dtype(self.in_fmt))
        B = np.zeros_like(A)
        C = np.zeros(len(rows), dtype=word_dtype(self.acc_fmt))
        for t, (prods, c) in enumerate(rows):
            for k, p in enumerate(prods):
                if p is None:
                    continue
                m, e = p
                ea, eb = self.split(e)
                A[t, k] = encode(self.in_fmt, m * 2.0 ** ea)
                B[t, k] = encode(self.in_fmt, 2.0 ** eb)
            if c is not None:
                C[t] = encode(self.acc_fmt, c[0] * 2.0 ** c[1])
        D = np.asarray(self.dot(A, B, C))
        return [decode(self.acc_fmt, int(w)) for w in D]


# ---------------------------------------------------------------------------------------------------------------------
# Step 2: summation order and arity
# ---------------------------------------------------------------------------------------------------------------------
def swamp_matrix(target: Target, K: int) -> dict:
    """d(i,j) / v for all 0 <= i < j <= K (index K is the accumulator): Section 3.1, Step 2."""
    eu, ev, _, _ = target.scales()
    rows, index = [], []
    for i in range(K + 1):
        for j in range(i + 1, K + 1):
            p = [(1.0, ev)] * (K + 1)
            p[i], p[j] = (1.0, eu), (-1.0, eu)
            rows.append((p[:K], p[K]))
            index.append((i, j))
    out = target.run(rows)
    v = 2.0 ** ev
    res = {}
    for ij, d in zip(index, out):
        n = d / v
        if n != int(n):
            raise ValueError(f"d{ij} = {d} is not a multiple of v: the swamping condition (Equation 5) does not hold")
        res[ij] = int(n)
    return res


def candidate_trees(K: int):
    """(name, parameters, tree) for the tree families of Figure 2.  A tree is ('leaf', k), ('bin', l, r) or
    ('fused', children, swamped)."""
    c = ("leaf", K)
    out = []
    t = c
    for k in range(K):
        t = ("bin", t, ("leaf", k))
    out.append(("chain", {}, t))
    for P in (2, 4):
        if K % P:
            continue
        t = c
        for g in range(0, K, P):
            grp = ("bin", ("leaf", g), ("leaf", g + 1))
            if P == 4:
                grp = ("bin", grp, ("bin", ("leaf", g + 2), ("leaf", g + 3)))
            t = ("bin", t, grp)
        out.append(("pairwise", {"P": P}, t))
    for L in range(2, K + 1):
        if K % L:
            continue
        for swamped in (True, False):
            t = c
            for g in range(0, K, L):
                t = ("fused", [t] + [("leaf", k) for k in range(g, g + L)], swamped)
            out.append(("fused", {"L": L, "swamped": swamped}, t))
    return out


def _evaluate(tree, leaves):
    """Symbolic value (coefficient of U, count of v) under the swamping rules of Section 3.1, Step 2."""
    kind = tree[0]
    if kind == "leaf":
        return leaves[tree[1]]
    if kind == "bin":
        vals = [_evaluate(tree[1], leaves), _evaluate(tree[2], leaves)]
        swamped = True
    else:
        vals = [_evaluate(ch, leaves) for ch in tree[1]]
        swamped = tree[2]
    u = sum(x[0] for x in vals)
    big = any(x[0] for x in vals)
    if swamped:
        return (u, 0) if big else (0, sum(x[1] for x in vals))     # any +-U in the operation swamps the small summands
    return (u, 0) if u else (0, sum(x[1] for x in vals))           # exact fused sum: v survives once +U and -U cancel


def predict_matrix(tree, K: int) -> dict:
    res = {}
    for i in range(K + 1):
        for j in range(i + 1, K + 1):
            leaves = [(0, 1)] * (K + 1)
            leaves[i], leaves[j] = (1, 0), (-1, 0)
            res[(i, j)] = _evaluate(tree, leaves)[1]
    return res


def infer_tree(matrix: dict, K: int):
    """Every tree of the enumerated families that reproduces the matrix, simplest first."""
    return [(name, par) for name, par, tree in candidate_trees(K) if predict_matrix(tree, K) == matrix]


# ---------------------------------------------------------------------------------------------------------------------
# Step 3: precision and rounding of a fused summation (products 0 .. L-1 and the accumulator in one operation)
# ---------------------------------------------------------------------------------------------------------------------
def fused_precision(target: Target, K: int, limit: int = 40) -> Optional[int]:
    """FusedSum(U, -U, eps): halve eps until the output is no longer eps.  Returns the number F of fractional bits
    (relative to the exponent of U) that the fused summation keeps, or None if eps never got lost down to
    U * 2**-limit (an exact summation, as far as the formats allow the test)."""
    eu, _, lo_e, _ = target.scales()
    rows, ts = [], []
    for t in range(0, limit + 1):
        e = eu - t
        try:
            target.split(e)
        except ValueError:
            break
        rows.append(([(1.0, eu), (-1.0, eu), (1.0, e)] + [None] * (K - 3), None))
        ts.append(t)
    out = target.run(rows)
    for t, d in zip(ts, out):
        if d != 2.0 ** (eu - t):
            return t - 1
    return None


def term_rounding(target: Target, K: int, F: int) -> str:
    """Rounding of one aligned term inside the fused summation: +-1.5 eps and +-0.5 eps next to U - U, eps half a
    unit of the summation grid."""
    eu, *_ = target.scales()
    e = eu - F - 1                                                 # eps = 2**e, the grid unit is 2 eps
    probes = [(1.5, e), (1.0, e - 1), (-1.5, e), (-1.0, e - 1)]
    rows = [([(1.0, eu), (-1.0, eu), p] + [None] * (K - 3), None) for p in probes]
    got = tuple(round(d / 2.0 ** (e + 1)) for d in target.run(rows))
    table = {(0, 0, 0, 0): "RZ", (0, 0, -1, -1): "RD", (1, 1, 0, 0): "RU", (1, 1, -1, -1): "RA", (1, 0, -1, 0): "RN"}
    return table.get(got, f"unknown{got}")


def output_conversion(target: Target, K: int, F: int):
    """(mantissa bits, rounding) of the conversion of the fused sum to the output (rho, Table 2): U + eps with eps
    halved until it is lost gives the bits; U + 0.75 ulp and U + 0.25 ulp (both signs) give the direction where the
    fused sum has bits to spare (F above the output's mantissa)."""
    eu, *_ = target.scales()
    rows = [([(1.0, eu), (1.0, eu - t)] + [None] * (K - 2), None) for t in range(1, F + 1)]
    out = target.run(rows)
    mbits = 0
    for t, d in zip(range(1, F + 1), out):
        if d != 2.0 ** eu + 2.0 ** (eu - t):
            break
        mbits = t
    if F < mbits + 2:
        return mbits, "exact" if F <= mbits else "undetermined"
    ulp = eu - mbits
    probes = [(1.0, 1.5, ulp - 1), (1.0, 1.0, ulp - 2), (-1.0, -1.5, ulp - 1), (-1.0, -1.0, ulp - 2)]   # +-0.75, +-0.25 ulp
    rows = [([(s, eu), (m, e)] + [None] * (K - 2), None) for s, m, e in probes]
    got = tuple(round((d - s * 2.0 ** eu) / 2.0 ** ulp) for d, (s, _, _) in zip(target.run(rows), probes))
    table = {(0, 0, 0, 0): "RZ", (0, 0, -1, -1): "RD", (1, 1, 0, 0): "RU", (1, 1, -1, -1): "RA", (1, 0, -1, 0): "RN"}
    mode = table.get(got, f"unknown{got}")
    if mode == "RN" and F >= mbits + 1:
        # ties: U + 0.5 ulp and U + 1.5 ulp
        rows = [([(1.0, eu), (1.0, ulp - 1)] + [None] * (K - 2), None), ([(1.0, eu), (1.5, ulp)] + [None] * (K - 2), None)]
        a, b = (round((d - 2.0 ** eu) / 2.0 ** ulp) for d in target.run(rows))
        mode = {(0, 2): "RNE", (1, 2): "RNA/RNU", (0, 1): "RNZ/RND", (1, 1): "RNO"}.get((a, b), f"RN?{(a, b)}")
    return mbits, mode


def characterise(target: Target, K: int) -> dict:
    """Steps 2 and 3 in one go: the summation tree of a K-element dot product and, for fused blocks, F, the term
    rounding and the output conversion."""
    trees = infer_tree(swamp_matrix(target, K), K)
    res = {"trees": trees}
    if trees and trees[0][0] == "fused" and trees[0][1]["swamped"]:
        L = trees[0][1]["L"]
        F = fused_precision(target, L)
        res.update(L=L, F=F)
        if F is not None:
            res["term_rounding"] = term_rounding(target, L, F)
            res["rho"] = output_conversion(target, L, F)
    return res
