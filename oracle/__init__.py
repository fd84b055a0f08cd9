"""CPU oracle for the bit-accurate MMA arithmetic models (TEST INFRASTRUCTURE).

This package is a plain, slow, arbitrary-precision restatement of the paper's
Algorithms 1-11 and Tables 2-7, written to be checked against the paper by eye.
It exists only so that tests, the smoke check and the benchmark's CPU-baseline
leg have something independent to compare the CUDA path with.  The product
(the CUDA library and its Python binding) never imports it, and it never
imports the product.

All arithmetic is done on Python ``int`` values (unbounded), every intermediate
value being a dyadic rational ``m * 2**e``; nothing here uses floating point.

Parity status: every function is pinned by ``tests/test_oracle_*.py`` against
values the paper prints (its worked-example table and summation-tree tables),
closed forms and library routines, except where the paper is silent and a
reading had to be chosen; those readings are listed in the header of
``oracle/ops.py`` and are "parity unpinned" against real hardware.
"""
from .formats import FORMATS, decode, Dec, FINITE, INF, NAN  # noqa: F401
from .rounding import round_dyadic, RHO  # noqa: F401
from .ops import (  # noqa: F401
    ftz_add, ftz_mul, flush_subnormal, fma, e_fdpa, t_fdpa, st_fdpa, gst_fdpa,
    tr_fdpa, gtr_fdpa, ieee_add_f32, ieee_mul_f32,
)
from .models import (  # noqa: F401
    Model, REGISTRY, lookup, printed, phi_dot, phi_gemm, phi_gemm_sampled, phi_dot_batch,
    ARCHS, chunk_promote_dot,
)
