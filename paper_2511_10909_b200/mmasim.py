"""ctypes binding of libmmasim.so: argument marshalling only, every step of the path runs in the CUDA kernels.

PyTorch is used for device memory and streams.  There is no CPU fallback: if the shared library is missing the
import fails, and every compute call needs CUDA tensors.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import c_int, c_int32, c_int64, c_void_p, c_char_p, POINTER, Structure, byref

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libmmasim.so")

ARCH = {n: i for i, n in enumerate(
    ["volta", "turing", "ampere", "ada", "hopper", "blackwell", "rtx_blackwell", "cdna1", "cdna2", "cdna3"])}
FMT = {n: i for i, n in enumerate(
    ["fp64", "fp32", "tf32", "bf16", "bf16_1k", "fp16", "e4m3", "e5m2", "e3m2", "e2m3", "e2m1",
     "mxe4m3", "mxe5m2", "mxe3m2", "mxe2m3", "mxe2m1", "mxf4", "nvf4"])}
ACC = {"fp32": 0, "fp16": 1, "fp64": 2}
FAMILY = ["fma", "ftz", "e", "t", "st", "gst", "tr", "gtr"]
RHO = ["", "RZ-FP32", "RZ-E8M13", "RNE-FP32", "RNE-FP16"]
FORCE_GENERIC = 1


class MmasimError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"mmasim status {status}: {message}")
        self.status = status


class _Info(Structure):
    _fields_ = [(n, c_int32) for n in ("family", "l_max", "F", "F2", "rho", "P", "G", "k_block", "a_bits", "b_bits",
                                       "acc_bytes", "inner_round")]


class _Overrides(Structure):
    _fields_ = [(n, c_int32) for n in ("l_max", "F", "F2", "rho", "inner_round", "literal_emax")]


class _GemmOpts(Structure):
    _fields_ = [("lda", c_int64), ("ldb", c_int64), ("ldc", c_int64), ("ldd", c_int64),
                ("sfa", c_void_p), ("sfb", c_void_p), ("k_chunk", c_int64),
                ("row_scale", c_void_p), ("col_scale", c_void_p), ("flags", c_int32)]


def _load():
    if not os.path.exists(_LIB_PATH):
        raise ImportError(f"{_LIB_PATH} is missing: build it with `python -m paper_2511_10909_b200.build` "
                          "(there is no CPU fallback)")
    lib = ctypes.CDLL(_LIB_PATH)
    lib.mmasim_create_model.restype = c_void_p
    lib.mmasim_create_model.argtypes = [c_int, c_int, c_int]
    lib.mmasim_create_model_ex.restype = c_void_p
    lib.mmasim_create_model_ex.argtypes = [c_int, c_int, c_int, c_int, POINTER(_Overrides)]
    lib.mmasim_destroy_model.restype = None
    lib.mmasim_destroy_model.argtypes = [c_void_p]
    lib.mmasim_model_info.restype = c_int
    lib.mmasim_model_info.argtypes = [c_void_p, POINTER(_Info)]
    lib.mmasim_gemm.restype = c_int
    lib.mmasim_gemm.argtypes = [c_void_p, c_int64, c_int64, c_int64, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]
    lib.mmasim_gemm_ex.restype = c_int
    lib.mmasim_gemm_ex.argtypes = [c_void_p, c_int64, c_int64, c_int64, c_void_p, c_void_p, c_void_p, c_void_p,
                                   POINTER(_GemmOpts), c_void_p]
    lib.mmasim_gemm_noalloc.restype = c_int
    lib.mmasim_gemm_noalloc.argtypes = [c_void_p, c_int64, c_int64, c_int64, c_void_p, c_void_p, c_void_p, c_void_p,
                                        POINTER(_GemmOpts), c_void_p]
    lib.mmasim_dot_batch.restype = c_int
    lib.mmasim_dot_batch.argtypes = [c_void_p, c_int64, c_int64, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]
    lib.mmasim_gemm_host.restype = c_int
    lib.mmasim_gemm_host.argtypes = [c_void_p, c_int64, c_int64, c_int64, c_void_p, c_void_p, c_void_p, c_void_p,
                                     POINTER(_GemmOpts)]
    lib.mmasim_int_peak.restype = c_int
    lib.mmasim_int_peak.argtypes = [c_int, c_int64, c_int64, c_void_p, POINTER(c_int32), c_void_p]
    lib.mmasim_hw_mma.restype = c_int
    lib.mmasim_hw_mma.argtypes = [c_int, c_int64, c_int64, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]
    lib.mmasim_hw_umma.restype = c_int
    lib.mmasim_hw_umma.argtypes = [c_int, c_int64, c_int64, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p, c_void_p]
    lib.mmasim_error_stats.restype = c_int
    lib.mmasim_error_stats.argtypes = [c_int, c_int64, c_void_p, c_void_p, c_void_p, c_void_p]
    lib.mmasim_host_release.restype = c_int
    lib.mmasim_host_release.argtypes = []
    lib.mmasim_last_kernel.restype = c_char_p
    lib.mmasim_last_error.restype = c_char_p
    return lib


_lib = _load()


def library_path() -> str:
    return _LIB_PATH


def _check(status: int):
    if status != 0:
        raise MmasimError(status, _lib.mmasim_last_error().decode())


def last_kernel() -> str:
    return _lib.mmasim_last_kernel().decode()


class Model:
    """Handle of one (architecture, input type, accumulator type) model of the paper's Tables 3-7."""

    def __init__(self, arch: str, in_fmt: str, acc: str, b_fmt: str | None = None, **overrides):
        self.arch, self.in_fmt, self.acc, self.b_fmt = arch, in_fmt, acc, b_fmt or in_fmt
        ov = None
        if overrides:
            vals = {k: -1 for k in ("l_max", "F", "F2", "rho", "inner_round", "literal_emax")}
            for k, v in overrides.items():
                if k not in vals:
                    raise TypeError(f"unknown override {k}")
                vals[k] = RHO.index(v) if k == "rho" and isinstance(v, str) else int(v)
            ov = byref(_Overrides(**vals))
        h = _lib.mmasim_create_model_ex(ARCH[arch], FMT[in_fmt], FMT[self.b_fmt], ACC[acc], ov)
        if not h:
            raise MmasimError(2, _lib.mmasim_last_error().decode())
        self._h = c_void_p(h)
        info = _Info()
        _check(_lib.mmasim_model_info(self._h, byref(info)))
        self.family = FAMILY[info.family]
        self.l_max, self.F, self.F2, self.rho = info.l_max, info.F, info.F2, RHO[info.rho]
        self.P, self.G, self.k_block = info.P, info.G, info.k_block
        self.a_bits, self.b_bits, self.acc_bytes = info.a_bits, info.b_bits, info.acc_bytes
        self.inner_round = info.inner_round

    def __del__(self):
        h = getattr(self, "_h", None)
        if h and _lib is not None:
            _lib.mmasim_destroy_model(h)
            self._h = None

    def __repr__(self):
        return f"Model({self.arch}, {self.in_fmt}, {self.acc}: {self.family} L={self.l_max} F={self.F} {self.rho})"


def create_model(arch: str, in_fmt: str, acc: str, **kw) -> Model:
    return Model(arch, in_fmt, acc, **kw)


def model_keys():
    """Every (arch, in_fmt, acc) triple the library accepts with equal A and B types."""
    keys = []
    for a in ARCH:
        for f in FMT:
            for c in ACC:
                h = _lib.mmasim_create_model(ARCH[a], FMT[f], ACC[c])
                if h:
                    _lib.mmasim_destroy_model(c_void_p(h))
                    keys.append((a, f, c))
    return keys


def _ptr(t):
    return None if t is None else c_void_p(t.data_ptr())


def _stream(stream):
    import torch
    s = stream if stream is not None else torch.cuda.current_stream()
    return c_void_p(s.cuda_stream)


def _acc_dtype(model: Model):
    import torch
    return {8: torch.int64, 4: torch.int32, 2: torch.int16}[model.acc_bytes]


def _make_opts(sfa=None, sfb=None, k_chunk=0, row_scale=None, col_scale=None, force_generic=False,
               lda=0, ldb=0, ldc=0, ldd=0):
    o = _GemmOpts()
    o.lda, o.ldb, o.ldc, o.ldd = lda, ldb, ldc, ldd
    o.sfa, o.sfb = sfa, sfb
    o.k_chunk = k_chunk
    o.row_scale, o.col_scale = row_scale, col_scale
    o.flags = FORCE_GENERIC if force_generic else 0
    return o


def _matrix(t, name, rows, cols, bits, device):
    """Checks one matrix argument (CUDA tensor, element width, shape, unit inner stride) and returns its leading
    dimension in storage words; `cols` is the number of storage words per row that the call reads or writes."""
    if t is None:
        return 0
    if not t.is_cuda or t.device != device:
        raise MmasimError(1, f"{name} must be a CUDA tensor on {device} (no CPU fallback)")
    if t.element_size() * 8 != bits:
        raise MmasimError(1, f"{name} has {t.element_size() * 8}-bit elements, the model needs {bits}-bit words")
    if t.dim() != 2 or t.shape[0] < rows or t.shape[1] < cols:
        raise MmasimError(3, f"{name} has shape {tuple(t.shape)}, the call needs at least {rows} x {cols}")
    if t.shape[1] > 1 and t.stride(1) != 1:
        raise MmasimError(3, f"{name} must be contiguous along its rows (stride {t.stride(1)})")
    ld = t.stride(0) if t.shape[0] > 1 else max(t.stride(0), t.shape[1])
    if ld < cols:
        raise MmasimError(3, f"{name}: row stride {ld} is smaller than the row length {cols}")
    return ld


def _vector(t, name, n, bytes_per, device):
    if t is None:
        return
    if not t.is_cuda or t.device != device:
        raise MmasimError(1, f"{name} must be a CUDA tensor on {device}")
    if not t.is_contiguous() or t.element_size() != bytes_per or t.numel() < n:
        raise MmasimError(3, f"{name} must be a contiguous tensor of at least {n} {bytes_per}-byte elements")


def gemm(model: Model, A, B, C=None, out=None, *, M=None, N=None, K=None, sfa=None, sfb=None, k_chunk=0,
         row_scale=None, col_scale=None, force_generic=False, stream=None):
    """D = Phi(A, B, C) on CUDA tensors of raw words.

    A: M x K, B: N x K (each row is one column of the paper's K x N matrix), C/D: M x N words of the accumulator
    type (integer tensors of the element width; FP4 of the GST models packed two per byte, so A is M x K/2 uint8).
    Row-strided views are accepted (the row stride becomes the leading dimension lda / ldb / ldc / ldd of
    mmasim_gemm_ex); the inner dimension must be contiguous.  Returns D (allocated with torch if ``out`` is None).
    """
    import torch
    if not A.is_cuda:
        raise MmasimError(1, "mmasim.gemm needs CUDA tensors (no CPU fallback); use gemm_host for host buffers")
    per_word = 2 if model.a_bits == 4 else 1                 # elements per storage word
    M = A.shape[0] if M is None else M
    N = B.shape[0] if N is None else N
    if K is None:
        K = A.shape[1] * per_word
    if out is None:
        out = torch.empty((M, N), dtype=_acc_dtype(model), device=A.device)
    dev = A.device
    kw = -(-K // per_word)
    lda = _matrix(A, "A", M, kw, max(model.a_bits, 8), dev) * per_word
    ldb = _matrix(B, "B", N, kw, max(model.b_bits, 8), dev) * per_word
    ldc = _matrix(C, "C", M, N, model.acc_bytes * 8, dev)
    ldd = _matrix(out, "out", M, N, model.acc_bytes * 8, dev)
    if model.k_block:
        nsf = -(-K // model.k_block)
        for t, name, rows in ((sfa, "sfa", M), (sfb, "sfb", N)):
            if t is not None and (_matrix(t, name, rows, nsf, 8, dev) != nsf):
                raise MmasimError(3, f"{name} must be a packed {rows} x {nsf} byte matrix")
    _vector(row_scale, "row_scale", M, 4, dev)
    _vector(col_scale, "col_scale", N, 4, dev)
    strided = (lda, ldb) != (K, K) or (C is not None and ldc != N) or ldd != N
    plain = sfa is None and not k_chunk and row_scale is None and not force_generic and not strided
    if plain:
        _check(_lib.mmasim_gemm(model._h, M, N, K, _ptr(A), _ptr(B), _ptr(C), _ptr(out), _stream(stream)))
    else:
        o = _make_opts(_ptr(sfa), _ptr(sfb), k_chunk, _ptr(row_scale), _ptr(col_scale), force_generic,
                       lda, ldb, ldc, ldd)
        _check(_lib.mmasim_gemm_ex(model._h, M, N, K, _ptr(A), _ptr(B), _ptr(C), _ptr(out), byref(o), _stream(stream)))
    return out


def gemm_noalloc(model: Model, A, B, C, out, *, k_chunk=0, row_scale=None, col_scale=None, stream=None):
    """D = Phi(A, B, C) into the caller's ``out`` through mmasim_gemm_noalloc: no device memory is allocated or freed
    by the call (the scratch of the kernel is a fixed array inside the library), for callers that must not touch the
    allocator when they call.  FP8 models with F = 13 only; contiguous CUDA tensors; ``out`` is required, since
    creating it here would allocate.  Calls share the scratch: keep them ordered on one stream."""
    if not A.is_cuda:
        raise MmasimError(1, "mmasim.gemm_noalloc needs CUDA tensors (no CPU fallback)")
    dev = A.device
    M, N, K = A.shape[0], B.shape[0], A.shape[1]
    lda = _matrix(A, "A", M, K, 8, dev)
    ldb = _matrix(B, "B", N, K, 8, dev)
    ldc = _matrix(C, "C", M, N, model.acc_bytes * 8, dev)
    ldd = _matrix(out, "out", M, N, model.acc_bytes * 8, dev)
    _vector(row_scale, "row_scale", M, 4, dev)
    _vector(col_scale, "col_scale", N, 4, dev)
    o = _make_opts(None, None, k_chunk, _ptr(row_scale), _ptr(col_scale), False, lda, ldb, ldc, ldd)
    _check(_lib.mmasim_gemm_noalloc(model._h, M, N, K, _ptr(A), _ptr(B), _ptr(C), _ptr(out), byref(o), _stream(stream)))
    return out


def dot_batch(model: Model, A, B, C=None, out=None, *, stream=None):
    """d_t = Phi(a_t, b_t, c_t) for the n rows of A and B (contiguous n x K CUDA tensors of raw words)."""
    import torch
    if not A.is_cuda:
        raise MmasimError(1, "mmasim.dot_batch needs CUDA tensors (no CPU fallback)")
    n, K = A.shape
    if out is None:
        out = torch.empty((n,), dtype=_acc_dtype(model), device=A.device)
    dev = A.device
    for t, name, bits in ((A, "A", model.a_bits), (B, "B", model.b_bits)):
        if _matrix(t, name, n, K, max(bits, 8), dev) != K and n > 1:
            raise MmasimError(3, f"{name} must be a packed n x K matrix")
    _vector(C, "C", n, model.acc_bytes, dev)
    _vector(out, "out", n, model.acc_bytes, dev)
    _check(_lib.mmasim_dot_batch(model._h, n, K, _ptr(A), _ptr(B), _ptr(C), _ptr(out), _stream(stream)))
    return out


def gemm_host(model: Model, A, B, C=None, *, K=None, sfa=None, sfb=None, k_chunk=0, row_scale=None, col_scale=None,
              out=None):
    """As gemm, on host buffers (numpy arrays or CPU tensors): the library copies to the device and back.
    Row-strided numpy views of A, B, C and ``out`` are passed with their strides as leading dimensions."""
    import numpy as np

    def as_np(x, keep_rows=False):
        if x is None:
            return None
        if hasattr(x, "numpy"):
            x = x.numpy()
        if keep_rows and x.ndim == 2 and (x.shape[1] == 1 or x.strides[1] == x.itemsize) and x.strides[0] >= x.shape[1] * x.itemsize \
                and x.strides[0] % x.itemsize == 0:
            return x
        return np.ascontiguousarray(x)

    A, B, C, out = (as_np(x, True) for x in (A, B, C, out))
    sfa, sfb, row_scale, col_scale = map(as_np, (sfa, sfb, row_scale, col_scale))
    per_word = 2 if model.a_bits == 4 else 1
    M, N = A.shape[0], B.shape[0]
    if K is None:
        K = A.shape[1] * per_word
    if out is None:
        out = np.empty((M, N), dtype={8: np.uint64, 4: np.uint32, 2: np.uint16}[model.acc_bytes])
    ld = lambda x: 0 if x is None else x.strides[0] // x.itemsize
    p = lambda x: None if x is None else c_void_p(x.ctypes.data)
    o = _make_opts(p(sfa), p(sfb), k_chunk, p(row_scale), p(col_scale), False,
                   ld(A) * per_word, ld(B) * per_word, ld(C), ld(out))
    _check(_lib.mmasim_gemm_host(model._h, M, N, K, p(A), p(B), p(C), p(out), byref(o)))
    return out


def copy_timeouts() -> int:
    """CTAs of the tuned kernels whose bounded wait on a bulk copy ran out (they store nothing); synchronises the device."""
    from ctypes import c_uint64
    n = c_uint64(0)
    _check(_lib.mmasim_copy_timeouts(byref(n)))
    return int(n.value)


def host_release():
    """Destroys the device memory pools that gemm_host keeps between calls."""
    _check(_lib.mmasim_host_release())


STAT_NAMES = ["count", "sum", "sum_abs", "sum_sq", "negative", "positive", "max_abs", "sum_rel"]


def error_stats(acc: str, D, ref, stats=None, *, stream=None):
    """Accumulate the deviation statistics of the output words D against the FP64 reference `ref` (CUDA tensors) into
    `stats` (8 doubles on the device, created zeroed if not given); returns `stats`."""
    import torch
    if not D.is_cuda or not ref.is_cuda or ref.dtype != torch.float64:
        raise MmasimError(1, "mmasim.error_stats needs CUDA tensors and an FP64 reference")
    if stats is None:
        stats = torch.zeros(8, dtype=torch.float64, device=D.device)
    _check(_lib.mmasim_error_stats(ACC[acc], D.numel(), _ptr(D), _ptr(ref), _ptr(stats), _stream(stream)))
    return stats


HW_KINDS = ["f16_f32", "f16_f16", "bf16_f32", "tf32_f32", "e4m3_f32", "e5m2_f32", "f64", "f16_f32_k8", "tf32_f32_k4",
            "e4m3_f16", "e5m2_f16", "e4m3_e5m2_f32", "e4m3_f32_k16"]
_HW_ACC_BYTES = {"f16_f16": 2, "f64": 8, "e4m3_f16": 2, "e5m2_f16": 2}


def hw_mma(kind: str, A, B, C=None, out=None, *, stream=None):
    """The B200's own `mma.sync` of the given kind on every 16-row tile of A (8 rows for "f64") against the 8 rows
    of B: D (M x 8) = A (M x K) * B^T + C, CUDA tensors of raw words."""
    import torch
    if not A.is_cuda:
        raise MmasimError(1, "mmasim.hw_mma needs CUDA tensors")
    M, K = A.shape
    if out is None:
        dt = {2: torch.int16, 4: torch.int32, 8: torch.int64}[_HW_ACC_BYTES.get(kind, 4)]
        out = torch.empty((M, 8), dtype=dt, device=A.device)
    _check(_lib.mmasim_hw_mma(HW_KINDS.index(kind), M, K, _ptr(A), _ptr(B), _ptr(C), _ptr(out), _stream(stream)))
    return out


UMMA_KINDS = ["f16_f32", "bf16_f32", "tf32_f32", "e4m3_f32", "e5m2_f32", "e4m3_e5m2_f32", "e2m3_f32", "e3m2_f32", "e2m1_f32",
              "selftest_timeout", "mxe4m3", "mxe5m2", "mxe2m3", "mxe3m2", "mxe2m1", "mxf4", "nvf4",
              "f16_f16", "e4m3_f16", "e5m2_f16", "e2m1_f16"]


def hw_umma(kind: str, A, B, C=None, out=None, *, sfa=None, sfb=None, K=None, stream=None):
    """The B200's `tcgen05.mma` of the given kind on every 128-row tile of A against the 16 rows of B:
    D (M x 16) = A (M x K) * B^T + C, CUDA tensors of raw words; FP32 accumulator words, 16-bit FP16 words for the `*_f16` kinds.  Raises MmasimError(6) if the
    kernel's bounded wait for the instruction ran out (the call synchronises to read the status word)."""
    import torch
    if not A.is_cuda:
        raise MmasimError(1, "mmasim.hw_umma needs CUDA tensors")
    M = A.shape[0]
    if K is None:
        K = A.shape[1] * (2 if kind in ("mxf4", "nvf4") else 1)      # packed FP4: two elements per byte
    if out is None:
        out = torch.empty((M, 16), dtype=torch.int16 if kind.endswith("_f16") else torch.int32, device=A.device)
    status = torch.zeros(1, dtype=torch.int32, device=A.device)
    _check(_lib.mmasim_hw_umma(UMMA_KINDS.index(kind), M, K, _ptr(A), _ptr(B), _ptr(C), _ptr(out), _ptr(sfa), _ptr(sfb),
                               _ptr(status), _stream(stream)))
    code = int(status.item())
    if code:
        raise MmasimError(code, "mmasim_hw_umma: the bounded wait for the instruction ran out; nothing was stored")
    return out


PEAK_KINDS = ["iadd3", "lop3", "shf", "imad", "macmix", "viaddmax", "viaddmax16x2", "f2i", "fmul", "popc",
              "imad+alu", "fmul+alu", "imad.wide", "mac_d1", "mac_d2", "dp4a", "dfma", "dfma+alu", "ffma.rm", "ffma2.rm",
              "ffma.rn.x16", "ffma.rn.x32", "ffma.rm.x16", "ffma2.rm.x16", "dfma.rn.x16", "dfma.rn.x32", "dfma.rm.x16", "dmma.rm.k4", "dmma.rm.k16",
              "cvt.f32.f64", "cvt.s32.f64", "dadd.rm.x16", "ffma2.rm.x16+alu"]


def int_peak(kind: str, blocks: int, iters: int, sink, stream=None) -> int:
    """Launch one issue-rate micro-benchmark; returns the number of counted operations of the launch."""
    opr = c_int32(0)
    _check(_lib.mmasim_int_peak(PEAK_KINDS.index(kind), blocks, iters, _ptr(sink), byref(opr), _stream(stream)))
    iters = (iters + 7) // 8 * 8
    return blocks * 256 * iters * 8 * opr.value
