"""ctypes front end of the CPU oracle (``dq_oracle.c``).

TEST INFRASTRUCTURE ONLY: tests, the smoke check and the benchmark's CPU
baseline use it; the CUDA library never does.  Arrays are numpy, C-contiguous.
The shared object is compiled on first use with gcc.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "dq_oracle.c")
_HDR = os.path.join(_HERE, "dq_oracle.h")
_SO = os.path.join(_HERE, "libdq_oracle.so")
_lock = threading.Lock()
_lib = None

CFLAGS = ["-O2", "-ffp-contract=off", "-frounding-math", "-fopenmp", "-shared", "-fPIC", "-std=c11", "-Wall"]


def build(force: bool = False) -> str:
    """Compile the oracle if the shared object is missing or stale."""
    newest = max(os.path.getmtime(_SRC), os.path.getmtime(_HDR))
    if force or not os.path.exists(_SO) or os.path.getmtime(_SO) < newest:
        tmp = _SO + ".tmp.%d" % os.getpid()
        subprocess.run(["gcc", *CFLAGS, "-o", tmp, _SRC, "-lm"], check=True, cwd=_HERE)
        os.replace(tmp, _SO)
    return _SO


_i64p = np.ctypeslib.ndpointer(np.int64, flags="C_CONTIGUOUS")
_f32p = np.ctypeslib.ndpointer(np.float32, flags="C_CONTIGUOUS")
_f64p = np.ctypeslib.ndpointer(np.float64, flags="C_CONTIGUOUS")
_u32p = np.ctypeslib.ndpointer(np.uint32, flags="C_CONTIGUOUS")


def lib():
    global _lib
    with _lock:
        if _lib is None:
            L = C.CDLL(build())
            seg = [_i64p, C.c_int32, C.c_int32]
            L.oracle_padded_elems.restype = C.c_int64
            L.oracle_padded_elems.argtypes = [_i64p, C.c_int32]
            L.oracle_num_buckets.restype = C.c_int64
            L.oracle_num_buckets.argtypes = seg
            L.oracle_seg_offsets.restype = None
            L.oracle_seg_offsets.argtypes = [_i64p, C.c_int32, _i64p]
            L.oracle_bucket_table.restype = None
            L.oracle_bucket_table.argtypes = seg + [_i64p, _i64p]
            L.oracle_bucket_norms.restype = None
            L.oracle_bucket_norms.argtypes = [C.c_void_p, C.c_int64, C.c_int32] + seg + [_f32p]
            L.oracle_bucket_norms_p.restype = None
            L.oracle_bucket_norms_p.argtypes = [C.c_void_p, C.c_int64, C.c_int32] + seg + [C.c_int32, _f32p]
            L.oracle_choose_bits.restype = C.c_int32
            L.oracle_choose_bits.argtypes = [_f32p, C.c_int64, C.c_int32, C.c_int32, C.c_int32,
                                             C.c_double, C.c_double, C.c_int32, C.c_int32, C.c_int32,
                                             C.POINTER(C.c_int32), C.POINTER(C.c_double)]
            L.oracle_philox4x32_10.restype = None
            L.oracle_philox4x32_10.argtypes = [_u32p, _u32p, _u32p]
            L.oracle_quantize.restype = None
            L.oracle_quantize.argtypes = ([C.c_void_p, C.c_int64, C.c_int32] + seg +
                                          [_f32p, C.c_int32, C.c_uint64, C.c_uint32,
                                           _u32p, C.c_void_p, C.c_void_p])
            L.oracle_pack.restype = None
            L.oracle_pack.argtypes = [_u32p, C.c_int64, C.c_int32, _u32p]
            L.oracle_unpack.restype = None
            L.oracle_unpack.argtypes = [_u32p, C.c_int64, C.c_int32, _u32p]
            L.oracle_quantize_pack.restype = None
            L.oracle_quantize_pack.argtypes = ([C.c_void_p, C.c_int64, C.c_int32] + seg +
                                               [_f32p, C.c_int32, C.c_uint64, C.c_uint32,
                                                _u32p, C.c_int64])
            L.oracle_dequantize.restype = None
            L.oracle_dequantize.argtypes = [_u32p, _f32p] + seg + [C.c_int32, _f64p]
            L.oracle_unpack_dequant_average.restype = None
            L.oracle_unpack_dequant_average.argtypes = ([_u32p, C.c_int64, _f32p, C.c_int32, C.c_int32]
                                                        + seg + [_f32p])
            L.oracle_unpack_average_update.restype = None
            L.oracle_unpack_average_update.argtypes = ([_u32p, C.c_int64, _f32p, C.c_int32, C.c_int32]
                                                       + seg + [C.c_double, _f32p])
            L.oracle_set_threads.restype = None
            L.oracle_set_threads.argtypes = [C.c_int32]
            L.oracle_get_threads.restype = C.c_int32
            L.oracle_get_threads.argtypes = []
            _lib = L
    return _lib


def set_threads(n: int) -> None:
    lib().oracle_set_threads(int(n))


def get_threads() -> int:
    return int(lib().oracle_get_threads())


def _seg(seg_elems):
    a = np.ascontiguousarray(np.asarray(seg_elems, dtype=np.int64))
    assert a.ndim == 1
    return a


class Layout:
    """Bucketed layout of a list of tensors (sizes ``seg_elems``), bucket size ``bucket``."""

    def __init__(self, seg_elems, bucket: int):
        assert bucket % 32 == 0 and bucket >= 32
        self.seg = _seg(seg_elems)
        self.n_seg = int(self.seg.size)
        self.bucket = int(bucket)
        L = lib()
        self.D32 = int(L.oracle_padded_elems(self.seg, self.n_seg))
        self.nb = int(L.oracle_num_buckets(self.seg, self.n_seg, self.bucket))
        self.offsets = np.zeros(self.n_seg, np.int64)
        L.oracle_seg_offsets(self.seg, self.n_seg, self.offsets)
        self.bucket_start = np.zeros(max(self.nb, 1), np.int64)
        self.bucket_len = np.zeros(max(self.nb, 1), np.int64)
        L.oracle_bucket_table(self.seg, self.n_seg, self.bucket, self.bucket_start, self.bucket_len)
        self.bucket_start = self.bucket_start[: self.nb]
        self.bucket_len = self.bucket_len[: self.nb]

    def packed_words(self, b: int) -> int:
        return b * self.D32 // 32

    def _args(self):
        return (self.seg, self.n_seg, self.bucket)


def _check_grads(lay: Layout, grads: np.ndarray):
    assert grads.dtype == np.float32 and grads.ndim == 2 and grads.shape[1] >= lay.D32
    assert grads.strides[1] == 4 and grads.strides[0] % 4 == 0
    return grads.ctypes.data, grads.strides[0] // 4, grads.shape[0]


NORM_L2, NORM_LINF = 2, 0


def whole_tensor_bucket(seg_elems) -> int:
    """Bucket size that gives every tensor a single bucket (the paper's own normalisation, Eq. 5)."""
    return max(32, (int(max(seg_elems)) + 31) // 32 * 32)


def bucket_norms(lay: Layout, grads: np.ndarray, p: int = NORM_L2) -> np.ndarray:
    """Per-bucket norms; ``p`` = NORM_L2 (default) or NORM_LINF."""
    assert p in (NORM_L2, NORM_LINF)
    ptr, stride, M = _check_grads(lay, grads)
    norms = np.zeros((M, lay.nb), np.float32)
    if p == NORM_L2:
        lib().oracle_bucket_norms(ptr, stride, M, *lay._args(), norms)
    else:
        lib().oracle_bucket_norms_p(ptr, stride, M, *lay._args(), p, norms)
    return norms


def choose_bits(norms: np.ndarray, T: int, t: int, eps_hat: float, alpha: float,
                b_min: int = 2, b_max: int = 16, fixed_b: int = 0):
    """Returns (b, s, x) with x the real-valued argument of Eq. 17: b* = log2(x+1)+1."""
    norms = np.ascontiguousarray(norms, np.float32)
    M, nb = norms.shape
    s = C.c_int32(0)
    x = C.c_double(0.0)
    b = lib().oracle_choose_bits(norms, nb, M, T, t, eps_hat, alpha, b_min, b_max, fixed_b,
                                 C.byref(s), C.byref(x))
    return int(b), int(s.value), float(x.value)


def philox4x32_10(ctr, key) -> np.ndarray:
    c = np.ascontiguousarray(ctr, np.uint32)
    k = np.ascontiguousarray(key, np.uint32)
    out = np.zeros(4, np.uint32)
    lib().oracle_philox4x32_10(c, k, out)
    return out


def quantize(lay: Layout, grads: np.ndarray, norms: np.ndarray, b: int, seed: int, step: int,
             want_x_v: bool = False):
    """Codes [M, D32]; with want_x_v also x (signed position on the level grid) and v (uniform)."""
    ptr, stride, M = _check_grads(lay, grads)
    norms = np.ascontiguousarray(norms, np.float32)
    assert norms.shape == (M, lay.nb)
    codes = np.zeros((M, lay.D32), np.uint32)
    if want_x_v:
        frac = np.zeros((M, lay.D32), np.float32)
        u = np.zeros((M, lay.D32), np.float32)
        lib().oracle_quantize(ptr, stride, M, *lay._args(), norms, b, seed, step, codes,
                              frac.ctypes.data, u.ctypes.data)
        return codes, frac, u
    lib().oracle_quantize(ptr, stride, M, *lay._args(), norms, b, seed, step, codes, None, None)
    return codes


def pack(codes: np.ndarray, b: int) -> np.ndarray:
    codes = np.ascontiguousarray(codes, np.uint32).ravel()
    n = codes.size
    assert n % 32 == 0
    words = np.zeros(n // 32 * b, np.uint32)
    lib().oracle_pack(codes, n, b, words)
    return words


def unpack(words: np.ndarray, n: int, b: int) -> np.ndarray:
    words = np.ascontiguousarray(words, np.uint32).ravel()
    assert n % 32 == 0 and words.size >= n // 32 * b
    codes = np.zeros(n, np.uint32)
    lib().oracle_unpack(words, n, b, codes)
    return codes


def quantize_pack(lay: Layout, grads: np.ndarray, norms: np.ndarray, b: int, seed: int, step: int,
                  packed_stride: int | None = None) -> np.ndarray:
    ptr, stride, M = _check_grads(lay, grads)
    norms = np.ascontiguousarray(norms, np.float32)
    assert norms.shape == (M, lay.nb)
    if packed_stride is None:
        packed_stride = lay.packed_words(b)
    assert packed_stride >= lay.packed_words(b)
    packed = np.zeros((M, packed_stride), np.uint32)
    lib().oracle_quantize_pack(ptr, stride, M, *lay._args(), norms, b, seed, step, packed, packed_stride)
    return packed


def dequantize(lay: Layout, codes: np.ndarray, norms: np.ndarray, b: int) -> np.ndarray:
    """One worker: fp64 values of Eq. 5 for codes [D32] and norms [nb]."""
    codes = np.ascontiguousarray(codes, np.uint32)
    norms = np.ascontiguousarray(norms, np.float32)
    assert codes.shape == (lay.D32,) and norms.shape == (lay.nb,)
    vals = np.zeros(lay.D32, np.float64)
    lib().oracle_dequantize(codes, norms, *lay._args(), b, vals)
    return vals


def unpack_dequant_average(lay: Layout, packed: np.ndarray, norms: np.ndarray, b: int) -> np.ndarray:
    packed = np.ascontiguousarray(packed, np.uint32)
    norms = np.ascontiguousarray(norms, np.float32)
    M = packed.shape[0]
    assert norms.shape == (M, lay.nb) and packed.shape[1] >= lay.packed_words(b)
    out = np.zeros(lay.D32, np.float32)
    lib().oracle_unpack_dequant_average(packed, packed.shape[1], norms, M, b, *lay._args(), out)
    return out


def unpack_average_update(lay: Layout, packed: np.ndarray, norms: np.ndarray, b: int, eta: float,
                          x: np.ndarray) -> np.ndarray:
    """x - eta * average (Eq. 2); returns a new fp32 array [D32], padding copied from ``x``."""
    packed = np.ascontiguousarray(packed, np.uint32)
    norms = np.ascontiguousarray(norms, np.float32)
    M = packed.shape[0]
    assert norms.shape == (M, lay.nb) and packed.shape[1] >= lay.packed_words(b)
    out = np.array(x, dtype=np.float32, copy=True)
    assert out.shape == (lay.D32,)
    lib().oracle_unpack_average_update(packed, packed.shape[1], norms, M, b, *lay._args(), float(eta), out)
    return out
