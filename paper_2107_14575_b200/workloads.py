"""Seeded synthetic gradient workloads.

Only shapes and random values live here: tensor-size lists in the shape of the
networks the paper trains (ResNet-18 on CIFAR-10, a VGG-16, an LSTM text
classifier), value distributions, and the placement of tensors at given
offsets.  None of the quantizer's arithmetic is in this module; the padded
offsets are always supplied by the caller (the CPU checker or the CUDA
library each compute their own).

The paper's datasets and trained models are not used; these arrays stand in
for the gradients of those networks.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Callable, List, Optional, Sequence

import numpy as np


# --------------------------------------------------------------------------
# tensor-size lists
# --------------------------------------------------------------------------

def resnet18_cifar_segments(num_classes: int = 10) -> List[int]:
    """Parameter tensors of a CIFAR-style ResNet-18 (3x3 stem), forward order.

    62 tensors, 11,173,962 elements for 10 classes.
    """
    segs: List[int] = []

    def conv_bn(cin, cout, k):
        segs.append(cout * cin * k * k)
        segs.extend([cout, cout])          # batch-norm weight, bias

    conv_bn(3, 64, 3)
    cin = 64
    for cout, stride in ((64, 1), (128, 2), (256, 2), (512, 2)):
        for blk in range(2):
            first = blk == 0
            conv_bn(cin if first else cout, cout, 3)
            conv_bn(cout, cout, 3)
            if first and (stride != 1 or cin != cout):
                conv_bn(cin, cout, 1)      # projection shortcut
        cin = cout
    segs.append(num_classes * 512)
    segs.append(num_classes)
    return segs


def vgg16_cifar_segments(num_classes: int = 100) -> List[int]:
    """Weight tensors of a VGG-16 for 32x32x3 inputs: 13 conv + 3 FC, 15,285,952 elements."""
    cfg = [64, 64, 128, 128, 256, 256, 256, 512, 512, 512, 512, 512, 512]
    segs, cin = [], 3
    for c in cfg:
        segs.append(c * cin * 9)
        cin = c
    segs += [512 * 512, 512 * 512, num_classes * 512]
    return segs


def text_classifier_segments() -> List[int]:
    """Embedding 30,000x300, 2-layer LSTM (hidden 256), 4-class head: 10,098,756 elements."""
    H, E = 256, 300
    return [30000 * E,
            4 * H * E, 4 * H * H, 4 * H, 4 * H,
            4 * H * H, 4 * H * H, 4 * H, 4 * H,
            4 * H, 4]


# --------------------------------------------------------------------------
# workload descriptions
# --------------------------------------------------------------------------

@dataclass
class Workload:
    name: str
    segments: List[int]
    M: int
    bucket: int
    T: int = 1                       # steps of the schedule (1 = single round trip)
    fixed_b: Sequence[int] = ()      # non-empty -> fixed bit widths to run
    alpha: float = 1.0               # alpha of the bit rule
    x0: float = 6.0                  # eps_hat is calibrated so that x(t=0) = x0
    seed: int = 0
    # fills out[M, n] (float32) for tensor index `seg`, step t
    fill: Optional[Callable[["Workload", np.random.Generator, int, int, np.ndarray], None]] = None
    notes: str = ""
    extra: dict = field(default_factory=dict)

    @property
    def d(self) -> int:
        return int(sum(self.segments))


def _rng(w: Workload, step: int, m: int, seg: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([w.seed, step, m, seg])))


def _fill_normal(sigma: float):
    def f(w, rng, seg, step, out):
        out[...] = rng.standard_normal(out.shape, dtype=np.float32) * np.float32(sigma)
    return f


def _fill_resnet(w, rng, seg, step, out):
    nseg = len(w.segments)
    scale = 1e-2 * 10.0 ** (-seg / max(nseg - 1, 1)) * (0.98 ** step)
    out[...] = rng.laplace(0.0, scale, out.shape).astype(np.float32)


def _fill_vgg(w, rng, seg, step, out):
    base = rng.standard_normal(out.shape, dtype=np.float32) * np.float32(1e-2)
    mask = rng.random(out.shape, dtype=np.float32) < np.float32(0.01)
    out[...] = np.where(mask, base * np.float32(100.0), base)


def _fill_text(w, rng, seg, step, out):
    if seg == 0:                                        # embedding: 3% of rows non-zero
        rows, cols = 30000, 300
        out[...] = 0.0
        hot = rng.choice(rows, size=900, replace=False)
        v = out.reshape(rows, cols)
        v[hot, :] = rng.standard_normal((900, cols), dtype=np.float32) * np.float32(1e-2)
    else:
        out[...] = rng.standard_normal(out.shape, dtype=np.float32) * np.float32(1e-2)


def config_flat(d: int = 1 << 20, M: int = 4, bucket: int = 512, sigma: float = 0.1,
                fixed_b: Sequence[int] = (2, 4, 8), seed: int = 0, name: str = "flat") -> Workload:
    """One flat tensor, i.i.d. normal values of standard deviation ``sigma``."""
    return Workload(name=name, segments=[d], M=M, bucket=bucket, fixed_b=tuple(fixed_b),
                    seed=seed, fill=_fill_normal(sigma))


def config_resnet18(M: int = 8, bucket: int = 512, T: int = 100, seed: int = 0) -> Workload:
    """Per-layer Laplace values, scale falling 10x from first to last tensor, x0.98 per step."""
    return Workload(name="resnet18", segments=resnet18_cifar_segments(10), M=M, bucket=bucket, T=T,
                    alpha=(2.4e-3) ** (1.0 / T), seed=seed, fill=_fill_resnet)


def config_vgg16(M: int = 16, bucket: int = 2048, T: int = 200, seed: int = 0) -> Workload:
    """Gaussian values with 1% of entries scaled x100."""
    return Workload(name="vgg16", segments=vgg16_cifar_segments(100), M=M, bucket=bucket, T=T,
                    alpha=(2.4e-3) ** (1.0 / T), seed=seed, fill=_fill_vgg)


def config_text(M: int = 16, bucket: int = 1024, T: int = 100, seed: int = 0) -> Workload:
    """Embedding gradient with 97% of rows exactly zero, dense LSTM and head tensors."""
    return Workload(name="text", segments=text_classifier_segments(), M=M, bucket=bucket, T=T,
                    alpha=(2.4e-3) ** (1.0 / T), seed=seed, fill=_fill_text)


def scaled_down(w: Workload, factor: int, M: Optional[int] = None) -> Workload:
    """Same tensor list with every size divided by ``factor`` (at least 1 element each):
    keeps the ragged multi-tensor structure at a size a CPU check finishes quickly."""
    segs = [max(1, n // factor) for n in w.segments]
    out = Workload(**{**w.__dict__})
    out.segments = segs
    out.name = f"{w.name}/{factor}"
    if M is not None:
        out.M = M
    if w.name == "text":
        out.fill = _fill_normal(1e-2)
    return out


# --------------------------------------------------------------------------
# materialisation
# --------------------------------------------------------------------------

def make_grads(w: Workload, offsets: Sequence[int], padded_elems: int, step: int = 0,
               pad_value: float = 0.0, row_stride: Optional[int] = None) -> np.ndarray:
    """float32 array [M, row_stride]; tensor i of worker m sits at offsets[i].

    Elements outside every tensor (padding) are set to ``pad_value``.
    """
    stride = padded_elems if row_stride is None else row_stride
    assert stride >= padded_elems
    g = np.full((w.M, stride), pad_value, dtype=np.float32)
    for m in range(w.M):
        for i, n in enumerate(w.segments):
            if n == 0:
                continue
            w.fill(w, _rng(w, step, m, i), i, step, g[m, offsets[i]: offsets[i] + n])
    return g


def random_codes(n: int, b: int, seed: int) -> np.ndarray:
    """n uniformly random b-bit codes (uint32)."""
    rng = np.random.Generator(np.random.PCG64(seed))
    return rng.integers(0, 1 << b, size=n, dtype=np.uint32)
