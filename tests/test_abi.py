"""CPU-only checks of the C-ABI library: it loads, exports what the header
declares, its host-side layout agrees with the oracle's, and argument errors
are reported before anything is launched."""
import ctypes as C
import os
import re

import numpy as np
import pytest

import oracle
from paper_2107_14575_b200 import workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    txt = open(os.path.join(ROOT, "include", "dq.h")).read()
    txt = re.sub(r"/\*.*?\*/", "", txt, flags=re.S)
    return sorted(set(re.findall(r"\b(dq_[a-z_0-9]+)\s*\(", txt)))


def test_library_exports_every_declared_symbol(dqlib):
    names = _declared_functions()
    assert len(names) >= 16
    assert sorted(dqlib.SYMBOLS) == names
    raw = C.CDLL(dqlib.LIB_PATH)
    for n in names:
        assert getattr(raw, n) is not None


def test_no_fallback_without_library(monkeypatch, dqlib):
    monkeypatch.setattr(dqlib, "_lib", None)
    monkeypatch.setattr(dqlib, "LIB_PATH", "/nonexistent/libdq.so")
    with pytest.raises(RuntimeError, match="no fallback"):
        dqlib.lib()


LAYOUTS = [
    ([70, 32, 1, 100], 64),
    ([0, 5, 0], 32),
    ([1 << 20], 512),
    (W.resnet18_cifar_segments(), 512),
    (W.vgg16_cifar_segments(), 2048),
    (W.text_classifier_segments(), 1024),
    ([33, 4097, 31, 0, 64], 4096),
]


@pytest.mark.parametrize("segs,bucket", LAYOUTS)
def test_layout_matches_oracle(dqlib, segs, bucket):
    lay = dqlib.Layout(segs, bucket)
    ref = oracle.Layout(segs, bucket)
    assert lay.D32 == ref.D32 and lay.nb == ref.nb and lay.n_seg == ref.n_seg
    assert lay.offsets == ref.offsets.tolist()
    ks = sorted(set([0, 1, ref.nb // 3, ref.nb // 2, ref.nb - 2, ref.nb - 1]) & set(range(ref.nb)))
    if ref.nb <= 4096:
        ks = range(ref.nb)
    for k in ks:
        assert lay.bucket_range(k) == (int(ref.bucket_start[k]), int(ref.bucket_len[k]))
    for b in (1, 3, 16):
        assert lay.packed_words(b) == ref.packed_words(b)
    assert lay.table_bytes() == (0 if len(segs) == 1 else 12 * (len(segs) + 1))


def test_layout_errors(dqlib):
    for segs, bucket, code in [([10], 48, dqlib.ERR_RANGE), ([10], 16, dqlib.ERR_RANGE),
                               ([10], 8192, dqlib.ERR_RANGE), ([-1], 32, dqlib.ERR_RANGE),
                               ([0, 0], 32, dqlib.ERR_RANGE), ([1 << 31], 32, dqlib.ERR_RANGE),
                               ([1 << 30, 1 << 30], 32, dqlib.ERR_RANGE)]:
        with pytest.raises(dqlib.DQError) as e:
            dqlib.Layout(segs, bucket)
        assert e.value.code == code
    with pytest.raises(dqlib.DQError) as e:
        dqlib.Layout([], 32)
    assert e.value.code == dqlib.ERR_ARG
    lay = dqlib.Layout([100], 32)
    with pytest.raises(dqlib.DQError):
        lay.bucket_range(4)
    assert dqlib.status_string(dqlib.ERR_ALIGN).startswith("misaligned")


def test_argument_errors_need_no_gpu(dqlib):
    """Host-side validation returns before any CUDA call, so it runs on a CPU-only box.
    The addresses are fabricated and never dereferenced."""
    lay = dqlib.Layout([1000], 64)
    A = 0x7f0000001000            # "aligned" fake address
    L = dqlib.lib()
    h = lay.handle
    rule = dqlib.Rule.fixed(4)
    # NULL pointers
    assert L.dq_bucket_norms(h, 0, 1024, 1, A, A, 0) == dqlib.ERR_ARG
    assert L.dq_bucket_norms(h, A, 1024, 0, A, A, 0) == dqlib.ERR_ARG
    assert L.dq_quantize_pack(h, A, 1024, 1, A, 0, 0, 0, A, 1024, A, 0) == dqlib.ERR_ARG
    assert L.dq_unpack_dequant_average(h, A, 1024, A, 1, A, 0, A, 0) == dqlib.ERR_ARG
    assert L.dq_choose_bits(h, A, 1, C.byref(rule), A, 0, 256, A, 0) == dqlib.ERR_ARG
    # alignment: pointer, fp32 stride (multiple of 32), packed stride (multiple of 4)
    assert L.dq_bucket_norms(h, A + 4, 1024, 1, A, A, 0) == dqlib.ERR_ALIGN
    assert L.dq_bucket_norms(h, A, 1000, 2, A, A, 0) == dqlib.ERR_ALIGN
    assert L.dq_quantize_pack(h, A, 1024, 1, A, A, 0, 0, A, 1022, A, 0) == dqlib.ERR_ALIGN
    assert L.dq_unpack_dequant_average(h, A + 8, 1024, A, 1, A, A, A, 0) == dqlib.ERR_ALIGN
    # ranges: worker stride shorter than the layout, too many workers, capacity below b = 1, rule fields
    assert L.dq_bucket_norms(h, A, 512, 2, A, A, 0) == dqlib.ERR_RANGE
    assert L.dq_bucket_norms(h, A, 1024, 5000, A, A, 0) == dqlib.ERR_RANGE
    assert L.dq_quantize_pack(h, A, 1024, 1, A, A, 0, 0, A, 16, A, 0) == dqlib.ERR_RANGE
    bad = dqlib.Rule(10, 10, 1.0, 0.9, 2, 16, 0)           # t must be < T
    assert L.dq_choose_bits(h, A, 1, C.byref(bad), A, A, 256, A, 0) == dqlib.ERR_RANGE
    bad = dqlib.Rule(10, 0, 0.0, 0.9, 2, 16, 0)            # eps_hat must be > 0
    assert L.dq_choose_bits(h, A, 1, C.byref(bad), A, A, 256, A, 0) == dqlib.ERR_RANGE
    bad = dqlib.Rule(10, 0, 1.0, 0.9, 2, 16, 17)
    assert L.dq_choose_bits(h, A, 1, C.byref(bad), A, A, 256, A, 0) == dqlib.ERR_RANGE
    assert L.dq_choose_bits(h, A, 1, C.byref(rule), A, A, 0, A, 0) == dqlib.ERR_RANGE    # scratch too small
    # a layout with several tensors must have its device table bound first
    multi = dqlib.Layout([100, 100], 32)
    assert L.dq_bucket_norms(multi.handle, A, 256, 1, A, A, 0) == dqlib.ERR_STATE
    assert multi.table_bytes() == 36
    assert dqlib.choose_bits_scratch_bytes(lay, 4) == 256


def test_norm_family_layouts(dqlib):
    """Whole-tensor layouts agree with the oracle's (a bucket as large as the largest tensor), the
    norm kind is remembered, and the host checks of the new calls need no GPU."""
    segs = [1000, 33, 0, 5000, 1]
    lay = dqlib.Layout(segs, dqlib.BUCKET_WHOLE_TENSOR, dqlib.NORM_LINF)
    ref = oracle.Layout(segs, oracle.whole_tensor_bucket(segs))
    assert lay.whole_tensor and lay.norm == dqlib.NORM_LINF
    assert lay.D32 == ref.D32 and lay.nb == ref.nb == 4 and lay.offsets == ref.offsets.tolist()
    for k in range(ref.nb):
        assert lay.bucket_range(k) == (int(ref.bucket_start[k]), int(ref.bucket_len[k]))
    assert lay.table_bytes() == 24 * (len(segs) + 1)         # bucket table and 4096-element piece table
    # pieces: ceil(1000/4096) + ceil(33/4096) + 0 + ceil(5000/4096) + 1 = 5 per worker
    assert dqlib.tensor_norms_scratch_bytes(lay, 3) == 3 * 5 * 4
    plain = dqlib.Layout(segs, 64)
    assert not plain.whole_tensor and plain.norm == dqlib.NORM_L2
    assert dqlib.tensor_norms_scratch_bytes(plain, 3) == 0
    assert dqlib.Layout(segs, 64, dqlib.NORM_LINF).norm == dqlib.NORM_LINF

    L = dqlib.lib()
    arr = (C.c_int64 * 1)(100)
    h = C.c_void_p()
    assert L.dq_layout_create_ex(arr, 1, 32, 7, C.byref(h)) == dqlib.ERR_ARG          # unknown norm
    assert L.dq_layout_create(arr, 1, 0, C.byref(h)) == dqlib.ERR_RANGE               # whole tensor only via _ex
    big = (C.c_int64 * 1)((1 << 30) + 1)
    assert L.dq_layout_create_ex(big, 1, 0, dqlib.NORM_L2, C.byref(h)) == dqlib.ERR_RANGE

    A = 0x7f0000001000
    one = dqlib.Layout([10000], dqlib.BUCKET_WHOLE_TENSOR)
    assert one.nb == 1 and one.table_bytes() == 0
    need = dqlib.tensor_norms_scratch_bytes(one, 2)
    assert need == 2 * 3 * 4
    # the bucketed calls refuse a whole-tensor layout and the other way round
    assert L.dq_bucket_norms(one.handle, A, 10016, 2, A, A, 0) == dqlib.ERR_RANGE
    assert L.dq_norms_quantize_pack(one.handle, A, 10016, 2, A, 0, 0, A, A, 10016, A, 0) == dqlib.ERR_RANGE
    flat = dqlib.Layout([10000], 512)
    assert L.dq_tensor_norms(flat.handle, A, 10016, 2, A, A, 1 << 20, A, 0) == dqlib.ERR_RANGE
    assert L.dq_tensor_norms(one.handle, A, 10016, 2, A, 0, need, A, 0) == dqlib.ERR_ARG
    assert L.dq_tensor_norms(one.handle, A, 10016, 2, A, A + 4, need, A, 0) == dqlib.ERR_ALIGN
    assert L.dq_tensor_norms(one.handle, A, 10016, 2, A, A, need - 1, A, 0) == dqlib.ERR_RANGE


def test_worker_offset_calls_check_their_arguments(dqlib):
    lay = dqlib.Layout([1000], 64)
    A = 0x7f0000001000
    L = dqlib.lib()
    h = lay.handle
    assert L.dq_quantize_pack_worker(h, A, 1024, 1, A, 0, 0, 0, 3, A, 1024, A, 0) == dqlib.ERR_ARG
    assert L.dq_quantize_pack_worker(h, A, 1024, 1, A, A, 0, 0, 3, A, 1022, A, 0) == dqlib.ERR_ALIGN
    assert L.dq_norms_quantize_pack_worker(h, A, 1024, 1, 0, 0, 0, 3, A, A, 1024, A, 0) == dqlib.ERR_ARG
    assert L.dq_norms_quantize_pack_worker(h, A, 1024, 1, A, 0, 0, 3, A, A, 16, A, 0) == dqlib.ERR_RANGE
