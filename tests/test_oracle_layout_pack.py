"""Pins for the oracle's layout and its pack/unpack (CPU only).

Each check compares the oracle with something fixed outside it: hand-worked
offsets and words, an independent bit-string construction with numpy, and the
cost ratios the paper prints in Table 2.
"""
import numpy as np
import pytest

import oracle
from conftest import read_golden
from paper_2107_14575_b200 import workloads as W


def test_layout_hand_worked():
    # tensors of 70, 32, 1 and 100 elements, buckets of 64
    lay = oracle.Layout([70, 32, 1, 100], 64)
    assert lay.offsets.tolist() == [0, 96, 128, 160]
    assert lay.D32 == 96 + 32 + 32 + 128
    # 70 -> buckets (0,64) (64,6); 32 -> (96,32); 1 -> (128,1); 100 -> (160,64) (224,36)
    assert lay.nb == 6
    assert lay.bucket_start.tolist() == [0, 64, 96, 128, 160, 224]
    assert lay.bucket_len.tolist() == [64, 6, 32, 1, 64, 36]
    assert lay.packed_words(3) == 3 * lay.D32 // 32


def test_layout_empty_tensor_and_single():
    lay = oracle.Layout([0, 5, 0], 32)
    assert lay.D32 == 32 and lay.nb == 1
    assert lay.offsets.tolist() == [0, 0, 32]
    assert lay.bucket_start.tolist() == [0] and lay.bucket_len.tolist() == [5]


def test_resnet18_size_matches_paper_cost():
    # Table 2: vanilla SGD on CIFAR-10 costs 1998.06 (GiB) with W = 8 workers,
    # 6000 iterations (Table 1), 32-bit values -> d = cost * 2^30 / (8*6000*4)
    rows = {r[0]: r for r in read_golden("table2_costs.txt")}
    cost = float(rows["vanilla"][3])
    d_from_paper = cost * 2 ** 30 / (8 * 6000 * 4)
    d = sum(W.resnet18_cifar_segments(10))
    assert d == 11173962
    assert abs(d - d_from_paper) / d < 5e-6      # the table has 6 significant digits


def test_cost_model_matches_table2():
    # a fixed b-bit scheme costs b/32 of vanilla SGD: the packed stream must
    # hold exactly b bits per (padded) element and nothing else
    rows = read_golden("table2_costs.txt")
    vanilla = [float(x) for x in rows[0][2:5]]
    lay = oracle.Layout([1 << 12], 512)
    for r in rows[1:]:
        b = int(r[1])
        ratio = lay.packed_words(b) * 32 / (lay.D32 * 32)
        for cost, van in zip(r[2:5], vanilla):
            assert abs(float(cost) / van - ratio) < 2e-4, (r[0], cost, van)


def _numpy_pack(codes, b):
    """Independent construction: little-endian bit matrix -> bit string -> words."""
    bits = ((codes[:, None] >> np.arange(b, dtype=np.uint32)[None, :]) & 1).astype(np.uint8)
    stream = bits.reshape(-1)                                 # element-major, LSB first
    by = np.packbits(stream, bitorder="little")
    return by.view("<u4").copy()


@pytest.mark.parametrize("b", list(range(1, 17)))
@pytest.mark.parametrize("n", [32, 64, 992, 1024, (1 << 16) + 32])
def test_pack_roundtrip_and_bitstring(b, n):
    codes = W.random_codes(n, b, seed=1000 * b + n % 997)
    words = oracle.pack(codes, b)
    assert words.size == b * n // 32
    assert np.array_equal(words, _numpy_pack(codes, b))
    assert np.array_equal(oracle.unpack(words, n, b), codes)


@pytest.mark.parametrize("b", [1, 2, 3, 7, 16])
def test_pack_extreme_codes(b):
    for val in (0, (1 << b) - 1, 1 << (b - 1)):
        codes = np.full(96, val, np.uint32)
        words = oracle.pack(codes, b)
        assert np.array_equal(oracle.unpack(words, 96, b), codes)
        assert int(np.unpackbits(words.view(np.uint8)).sum()) == 96 * bin(val).count("1")


def test_pack_golden_words():
    for row in read_golden("pack_words.txt"):
        txt = " ".join(row).split("|")
        b = int(txt[0])
        codes = np.array([int(x) for x in txt[1].split()], np.uint32)
        want = np.array([int(x, 16) for x in txt[2].split()], np.uint32)
        assert codes.size == 32 and want.size == b
        got = oracle.pack(codes, b)
        assert [hex(x) for x in got] == [hex(x) for x in want]
        assert np.array_equal(oracle.unpack(want, 32, b), codes)


def test_groups_are_independent():
    # group g (32 codes) maps to words [b*g, b*g + b): changing one group
    # leaves all other words alone
    b, n = 5, 32 * 7
    codes = W.random_codes(n, b, seed=3)
    w0 = oracle.pack(codes, b)
    codes2 = codes.copy()
    codes2[32 * 3: 32 * 4] ^= np.uint32(0x1F)
    w1 = oracle.pack(codes2, b)
    diff = np.nonzero(w0 != w1)[0]
    assert diff.min() >= 3 * b and diff.max() < 4 * b
