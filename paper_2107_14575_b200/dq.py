"""Thin ctypes binding of the C-ABI CUDA library (``include/dq.h``).

Argument marshalling only: every step of the path runs in the library's
kernels.  Tensors are torch CUDA tensors (device memory and streams are
torch's); the functions have the names and the argument order of the C calls.
There is no fallback: a missing ``libdq.so`` raises.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Optional, Sequence

_PKG = os.path.dirname(os.path.abspath(__file__))
# DQ_LIBRARY selects another build of the same library (the bounds-checked one, libdq_checked.so)
LIB_PATH = os.environ.get("DQ_LIBRARY") or os.path.join(_PKG, "libdq.so")

OK, ERR_ARG, ERR_ALIGN, ERR_RANGE, ERR_CUDA, ERR_STATE, ERR_TOO_LARGE = 0, -1, -2, -3, -4, -5, -6
STAT_NONFINITE, STAT_BAD_BITS, STAT_CAPACITY, STAT_WAIT, STAT_INTERNAL = 1, 2, 4, 8, 16
NORM_L2, NORM_LINF = 2, 0          # DQ_NORM_*: member of the l_p family of Eq. 5
BUCKET_WHOLE_TENSOR = 0            # DQ_BUCKET_WHOLE_TENSOR: one norm per tensor

# every symbol include/dq.h declares
SYMBOLS = [
    "dq_layout_create", "dq_layout_create_ex", "dq_layout_norm", "dq_layout_whole_tensor", "dq_layout_destroy", "dq_layout_num_segments", "dq_layout_padded_elems",
    "dq_layout_seg_offset", "dq_layout_num_buckets", "dq_layout_packed_words", "dq_layout_bucket",
    "dq_layout_shard_bounds", "dq_layout_slice", "dq_layout_table_bytes", "dq_layout_bind_device_table",
    "dq_bucket_norms", "dq_tensor_norms_scratch_bytes", "dq_tensor_norms", "dq_choose_bits_scratch_bytes", "dq_choose_bits",
    "dq_choose_bits_noalloc_max_norms", "dq_choose_bits_noalloc",
    "dq_quantize_pack", "dq_quantize_pack_worker", "dq_norms_quantize_pack", "dq_norms_quantize_pack_worker", "dq_unpack_dequant_average",
    "dq_unpack_average_update", "dq_status_string", "dq_debug_set_wait_limits",
]


class DQError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} ({code})")


class Rule(C.Structure):
    """``dq_rule_t``: parameters of the bit rule, Eq. 17."""
    _fields_ = [("T", C.c_int32), ("t", C.c_int32), ("eps_hat", C.c_double), ("alpha", C.c_double),
                ("b_min", C.c_int32), ("b_max", C.c_int32), ("fixed_b", C.c_int32)]

    @classmethod
    def dynamic(cls, T: int, t: int, eps_hat: float, alpha: float, b_min: int = 2, b_max: int = 16):
        return cls(T, t, eps_hat, alpha, b_min, b_max, 0)

    @classmethod
    def fixed(cls, b: int):
        return cls(1, 0, 1.0, 1.0, 1, 16, b)


_lib = None


def lib():
    """Loads ``libdq.so`` (built by ``python -m paper_2107_14575_b200.build``)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2107_14575_b200.build` "
                "(there is no fallback implementation)")
        L = C.CDLL(LIB_PATH)
        vp, i32, i64, u32, u64, sz = C.c_void_p, C.c_int32, C.c_int64, C.c_uint32, C.c_uint64, C.c_size_t
        L.dq_layout_create.restype = C.c_int
        L.dq_layout_create.argtypes = [C.POINTER(i64), i32, i32, C.POINTER(vp)]
        L.dq_layout_create_ex.restype = C.c_int
        L.dq_layout_create_ex.argtypes = [C.POINTER(i64), i32, i32, i32, C.POINTER(vp)]
        L.dq_layout_norm.restype = i32
        L.dq_layout_norm.argtypes = [vp]
        L.dq_layout_whole_tensor.restype = i32
        L.dq_layout_whole_tensor.argtypes = [vp]
        L.dq_layout_destroy.restype = None
        L.dq_layout_destroy.argtypes = [vp]
        L.dq_layout_num_segments.restype = i32
        L.dq_layout_num_segments.argtypes = [vp]
        L.dq_layout_padded_elems.restype = i64
        L.dq_layout_padded_elems.argtypes = [vp]
        L.dq_layout_seg_offset.restype = i64
        L.dq_layout_seg_offset.argtypes = [vp, i32]
        L.dq_layout_num_buckets.restype = i64
        L.dq_layout_num_buckets.argtypes = [vp]
        L.dq_layout_packed_words.restype = i64
        L.dq_layout_packed_words.argtypes = [vp, i32]
        L.dq_layout_bucket.restype = C.c_int
        L.dq_layout_bucket.argtypes = [vp, i64, C.POINTER(i64), C.POINTER(i64)]
        L.dq_layout_shard_bounds.restype = C.c_int
        L.dq_layout_shard_bounds.argtypes = [vp, i32, C.POINTER(i64)]
        L.dq_layout_slice.restype = C.c_int
        L.dq_layout_slice.argtypes = [vp, i64, i64, C.POINTER(vp), C.POINTER(i64)]
        L.dq_layout_table_bytes.restype = sz
        L.dq_layout_table_bytes.argtypes = [vp]
        L.dq_layout_bind_device_table.restype = C.c_int
        L.dq_layout_bind_device_table.argtypes = [vp, vp, sz, vp]
        L.dq_bucket_norms.restype = C.c_int
        L.dq_bucket_norms.argtypes = [vp, vp, i64, i32, vp, vp, vp]
        L.dq_tensor_norms_scratch_bytes.restype = sz
        L.dq_tensor_norms_scratch_bytes.argtypes = [vp, i32]
        L.dq_tensor_norms.restype = C.c_int
        L.dq_tensor_norms.argtypes = [vp, vp, i64, i32, vp, vp, sz, vp, vp]
        L.dq_choose_bits_scratch_bytes.restype = sz
        L.dq_choose_bits_scratch_bytes.argtypes = [vp, i32]
        L.dq_choose_bits.restype = C.c_int
        L.dq_choose_bits.argtypes = [vp, vp, i32, C.POINTER(Rule), vp, vp, sz, vp, vp]
        L.dq_choose_bits_noalloc_max_norms.restype = i64
        L.dq_choose_bits_noalloc_max_norms.argtypes = []
        L.dq_choose_bits_noalloc.restype = C.c_int
        L.dq_choose_bits_noalloc.argtypes = [vp, vp, i32, C.POINTER(Rule), vp, vp, vp]
        L.dq_quantize_pack.restype = C.c_int
        L.dq_quantize_pack.argtypes = [vp, vp, i64, i32, vp, vp, u64, u32, vp, i64, vp, vp]
        L.dq_quantize_pack_worker.restype = C.c_int
        L.dq_quantize_pack_worker.argtypes = [vp, vp, i64, i32, vp, vp, u64, u32, u32, vp, i64, vp, vp]
        L.dq_norms_quantize_pack_worker.restype = C.c_int
        L.dq_norms_quantize_pack_worker.argtypes = [vp, vp, i64, i32, vp, u64, u32, u32, vp, vp, i64, vp, vp]
        L.dq_norms_quantize_pack.restype = C.c_int
        L.dq_norms_quantize_pack.argtypes = [vp, vp, i64, i32, vp, u64, u32, vp, vp, i64, vp, vp]
        L.dq_unpack_dequant_average.restype = C.c_int
        L.dq_unpack_dequant_average.argtypes = [vp, vp, i64, vp, i32, vp, vp, vp, vp]
        L.dq_unpack_average_update.restype = C.c_int
        L.dq_unpack_average_update.argtypes = [vp, vp, i64, vp, i32, vp, C.c_float, vp, vp, vp]
        L.dq_status_string.restype = C.c_char_p
        L.dq_status_string.argtypes = [C.c_int]
        L.dq_debug_set_wait_limits.restype = None
        L.dq_debug_set_wait_limits.argtypes = [u64, i32]
        _lib = L
    return _lib


def status_string(code: int) -> str:
    return lib().dq_status_string(int(code)).decode()


def debug_set_wait_limits(limit_ns: int = 0, lose_first_wait: bool = False) -> None:
    """``dq_debug_set_wait_limits`` (test hook); the defaults restore normal operation."""
    lib().dq_debug_set_wait_limits(int(limit_ns), 1 if lose_first_wait else 0)


def _check(rc: int, where: str) -> None:
    if rc != OK:
        raise DQError(rc, where)


def _ptr(t) -> int:
    """Device (or host) address of a torch tensor, or an int passed through."""
    if t is None:
        return 0
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream) -> int:
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    if isinstance(stream, int):
        return stream
    return stream.cuda_stream


class Layout:
    """``dq_layout_t``: the padded, bucketed layout of a list of tensors.

    ``bucket = BUCKET_WHOLE_TENSOR`` gives one norm per tensor (Eq. 5 as written);
    ``norm`` picks the member of the l_p family the norm calls compute."""

    def __init__(self, seg_elems: Sequence[int], bucket: int, norm: int = NORM_L2, _handle=None):
        h = C.c_void_p()
        if _handle is not None:
            h = _handle                     # a layout the library created (dq_layout_slice)
        elif norm == NORM_L2 and bucket != BUCKET_WHOLE_TENSOR:
            arr = (C.c_int64 * len(seg_elems))(*[int(x) for x in seg_elems])
            _check(lib().dq_layout_create(arr, len(seg_elems), int(bucket), C.byref(h)), "dq_layout_create")
        else:
            arr = (C.c_int64 * len(seg_elems))(*[int(x) for x in seg_elems])
            _check(lib().dq_layout_create_ex(arr, len(seg_elems), int(bucket), int(norm), C.byref(h)),
                   "dq_layout_create_ex")
        self._h = h
        self.bucket = int(bucket)
        self.norm = int(lib().dq_layout_norm(h))
        self.whole_tensor = bool(lib().dq_layout_whole_tensor(h))
        self.n_seg = int(lib().dq_layout_num_segments(h))
        self.D32 = int(lib().dq_layout_padded_elems(h))
        self.nb = int(lib().dq_layout_num_buckets(h))
        self.offsets = [int(lib().dq_layout_seg_offset(h, i)) for i in range(self.n_seg)]
        self._table = None          # keeps the bound device table alive

    def __del__(self):
        h, self._h = getattr(self, "_h", None), None
        if h is not None and _lib is not None:
            _lib.dq_layout_destroy(h)

    @property
    def handle(self):
        return self._h

    def packed_words(self, b: int) -> int:
        return int(lib().dq_layout_packed_words(self._h, int(b)))

    def bucket_range(self, k: int):
        s, n = C.c_int64(), C.c_int64()
        _check(lib().dq_layout_bucket(self._h, int(k), C.byref(s), C.byref(n)), "dq_layout_bucket")
        return int(s.value), int(n.value)

    def table_bytes(self) -> int:
        return int(lib().dq_layout_table_bytes(self._h))

    def shard_bounds(self, n_shards: int):
        """First bucket of each of ``n_shards`` contiguous ranges, plus ``nb`` (``dq_layout_shard_bounds``)."""
        out = (C.c_int64 * (int(n_shards) + 1))()
        _check(lib().dq_layout_shard_bounds(self._h, int(n_shards), out), "dq_layout_shard_bounds")
        return [int(x) for x in out]

    def slice(self, k0: int, k1: int):
        """Buckets [k0, k1) as a layout of their own and where it starts in this padded buffer
        (``dq_layout_slice``); returns (Layout, first_elem)."""
        h, first = C.c_void_p(), C.c_int64()
        _check(lib().dq_layout_slice(self._h, int(k0), int(k1), C.byref(h), C.byref(first)), "dq_layout_slice")
        return Layout(None, self.bucket, self.norm, _handle=h), int(first.value)

    def bind_device_table(self, dev_buf, nbytes: Optional[int] = None, stream=None) -> None:
        """dev_buf: a torch uint8/int32 CUDA tensor (kept alive by this object) or a raw address."""
        if nbytes is None:
            nbytes = dev_buf.numel() * dev_buf.element_size()
        _check(lib().dq_layout_bind_device_table(self._h, _ptr(dev_buf), int(nbytes), _stream(stream)),
               "dq_layout_bind_device_table")
        self._table = dev_buf

    def bind(self, device="cuda", stream=None) -> "Layout":
        """Allocates the device table with torch (if the layout needs one) and binds it."""
        need = self.table_bytes()
        if need:
            import torch
            self.bind_device_table(torch.empty(need, dtype=torch.uint8, device=device), need, stream)
        return self


def bucket_norms(layout: Layout, grads, worker_stride_elems: int, M: int, norms, status, stream=None) -> None:
    _check(lib().dq_bucket_norms(layout.handle, _ptr(grads), int(worker_stride_elems), int(M), _ptr(norms),
                                 _ptr(status), _stream(stream)), "dq_bucket_norms")


def tensor_norms_scratch_bytes(layout: Layout, M: int) -> int:
    return int(lib().dq_tensor_norms_scratch_bytes(layout.handle, int(M)))


def tensor_norms(layout: Layout, grads, worker_stride_elems: int, M: int, norms, scratch, scratch_bytes: int, status,
                 stream=None) -> None:
    """One norm per tensor of a whole-tensor layout (``dq_tensor_norms``)."""
    _check(lib().dq_tensor_norms(layout.handle, _ptr(grads), int(worker_stride_elems), int(M), _ptr(norms),
                                 _ptr(scratch), int(scratch_bytes), _ptr(status), _stream(stream)), "dq_tensor_norms")


def choose_bits_scratch_bytes(layout: Layout, M: int) -> int:
    return int(lib().dq_choose_bits_scratch_bytes(layout.handle, int(M)))


def choose_bits(layout: Layout, norms, M: int, rule: Rule, dev_b, scratch, scratch_bytes: int, status,
                stream=None) -> None:
    _check(lib().dq_choose_bits(layout.handle, _ptr(norms), int(M), C.byref(rule), _ptr(dev_b), _ptr(scratch),
                                int(scratch_bytes), _ptr(status), _stream(stream)), "dq_choose_bits")


def choose_bits_noalloc(layout: Layout, norms, M: int, rule: Rule, dev_b, status, stream=None) -> None:
    """``dq_choose_bits`` for callers that cannot provide scratch memory: the reduction's
    scratch is a 64 KB array inside the library (see ``include/dq.h`` for the limit and
    the sharing rules)."""
    _check(lib().dq_choose_bits_noalloc(layout.handle, _ptr(norms), int(M), C.byref(rule), _ptr(dev_b),
                                        _ptr(status), _stream(stream)), "dq_choose_bits_noalloc")


def quantize_pack(layout: Layout, grads, worker_stride_elems: int, M: int, norms, dev_b, seed: int, step: int,
                  packed, packed_stride_words: int, status, stream=None) -> None:
    _check(lib().dq_quantize_pack(layout.handle, _ptr(grads), int(worker_stride_elems), int(M), _ptr(norms),
                                  _ptr(dev_b), int(seed) & (2 ** 64 - 1), int(step) & 0xFFFFFFFF, _ptr(packed),
                                  int(packed_stride_words), _ptr(status), _stream(stream)), "dq_quantize_pack")


def quantize_pack_worker(layout: Layout, grads, worker_stride_elems: int, M: int, norms, dev_b, seed: int, step: int,
                         first_worker: int, packed, packed_stride_words: int, status, stream=None) -> None:
    _check(lib().dq_quantize_pack_worker(layout.handle, _ptr(grads), int(worker_stride_elems), int(M), _ptr(norms),
                                         _ptr(dev_b), int(seed) & (2 ** 64 - 1), int(step) & 0xFFFFFFFF,
                                         int(first_worker) & 0xFFFFFFFF, _ptr(packed), int(packed_stride_words),
                                         _ptr(status), _stream(stream)), "dq_quantize_pack_worker")


def norms_quantize_pack_worker(layout: Layout, grads, worker_stride_elems: int, M: int, dev_b, seed: int, step: int,
                               first_worker: int, norms, packed, packed_stride_words: int, status,
                               stream=None) -> None:
    _check(lib().dq_norms_quantize_pack_worker(layout.handle, _ptr(grads), int(worker_stride_elems), int(M),
                                               _ptr(dev_b), int(seed) & (2 ** 64 - 1), int(step) & 0xFFFFFFFF,
                                               int(first_worker) & 0xFFFFFFFF, _ptr(norms), _ptr(packed),
                                               int(packed_stride_words), _ptr(status), _stream(stream)),
           "dq_norms_quantize_pack_worker")


def norms_quantize_pack(layout: Layout, grads, worker_stride_elems: int, M: int, dev_b, seed: int, step: int,
                        norms, packed, packed_stride_words: int, status, stream=None) -> None:
    _check(lib().dq_norms_quantize_pack(layout.handle, _ptr(grads), int(worker_stride_elems), int(M), _ptr(dev_b),
                                        int(seed) & (2 ** 64 - 1), int(step) & 0xFFFFFFFF, _ptr(norms), _ptr(packed),
                                        int(packed_stride_words), _ptr(status), _stream(stream)),
           "dq_norms_quantize_pack")


def unpack_dequant_average(layout: Layout, packed, packed_stride_words: int, norms, M: int, dev_b, out, status,
                           stream=None) -> None:
    _check(lib().dq_unpack_dequant_average(layout.handle, _ptr(packed), int(packed_stride_words), _ptr(norms),
                                           int(M), _ptr(dev_b), _ptr(out), _ptr(status), _stream(stream)),
           "dq_unpack_dequant_average")


def unpack_average_update(layout: Layout, packed, packed_stride_words: int, norms, M: int, dev_b, lr: float, params,
                          status, stream=None) -> None:
    """``params <- params - lr * average`` (Eq. 2), the average formed on the fly."""
    _check(lib().dq_unpack_average_update(layout.handle, _ptr(packed), int(packed_stride_words), _ptr(norms),
                                          int(M), _ptr(dev_b), float(lr), _ptr(params), _ptr(status),
                                          _stream(stream)), "dq_unpack_average_update")
