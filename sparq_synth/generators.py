"""Seeded numpy generators and workload shape tables (no SPARQ arithmetic)."""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass
from typing import List, Sequence, Tuple

import numpy as np

_CHUNK = 1 << 24


def _rng(seed: int, stream: int, chunk: int = 0) -> np.random.Generator:
    """Counter-based generator keyed by (seed, stream, chunk): a chunk's values
    do not depend on how many threads fill the tensor."""
    return np.random.Generator(np.random.Philox(key=[int(seed), (int(stream) << 40) | int(chunk)]))


def activations(seed: int, shape: Sequence[int], zero_frac: float, stream: int = 0) -> np.ndarray:
    """uint8 tensor: zeros with probability ``zero_frac``, else a discrete
    half-normal ``clip(round(|z| * 40), 1, 255)`` with z ~ N(0, 1)."""
    total = int(np.prod(shape, dtype=np.int64)) if len(shape) else 1
    out = np.empty(total, dtype=np.uint8)

    def fill(chunk: int) -> None:
        lo = chunk * _CHUNK
        hi = min(total, lo + _CHUNK)
        rng = _rng(seed, stream, chunk)
        z = rng.standard_normal(hi - lo, dtype=np.float32)
        v = np.clip(np.rint(np.abs(z) * np.float32(40.0)), 1, 255).astype(np.uint8)
        if zero_frac > 0.0:
            u = rng.random(hi - lo, dtype=np.float32)
            v[u < np.float32(zero_frac)] = 0
        out[lo:hi] = v

    nchunks = (total + _CHUNK - 1) // _CHUNK
    if nchunks <= 1:
        if total:
            fill(0)
    else:
        with ThreadPoolExecutor(max_workers=min(nchunks, os.cpu_count() or 1)) as pool:
            list(pool.map(fill, range(nchunks)))
    return out.reshape(tuple(shape))


def weights(seed: int, shape: Sequence[int], stream: int = 1) -> np.ndarray:
    """int8 tensor ``clip(round(z * 30), -127, 127)`` with z ~ N(0, 1)."""
    rng = _rng(seed, stream)
    z = rng.standard_normal(tuple(shape), dtype=np.float32)
    return np.clip(np.rint(z * np.float32(30.0)), -127, 127).astype(np.int8)


def scales(seed: int, n: int, stream: int = 2) -> np.ndarray:
    """float32 per-output-channel scale drawn from U(0.001, 0.01)."""
    rng = _rng(seed, stream)
    u = rng.random(int(n), dtype=np.float32)
    return (np.float32(0.001) + np.float32(0.009) * u).astype(np.float32)


def bias(seed: int, n: int, stream: int = 3) -> np.ndarray:
    """float32 per-output-channel bias drawn from U(-1, 1)."""
    rng = _rng(seed, stream)
    u = rng.random(int(n), dtype=np.float32)
    return (np.float32(2.0) * u - np.float32(1.0)).astype(np.float32)


@dataclass(frozen=True)
class ConvShape:
    """One convolution layer of a workload (NHWC input, [cout][r][s][cin] weights)."""

    name: str
    h: int
    w: int
    cin: int
    cout: int
    r: int
    s: int
    stride: int
    pad: int
    count: int = 1  # how many times this exact shape occurs in the network

    def out_hw(self) -> Tuple[int, int]:
        return conv_out_hw(self.h, self.w, self.r, self.s, self.stride, self.pad)

    def gemm_mnk(self, batch: int) -> Tuple[int, int, int]:
        ho, wo = self.out_hw()
        return batch * ho * wo, self.cout, self.r * self.s * self.cin

    def ops(self, batch: int) -> int:
        m, n, k = self.gemm_mnk(batch)
        return 2 * m * n * k


def conv_out_hw(h: int, w: int, r: int, s: int, stride: int, pad: int) -> Tuple[int, int]:
    return (h + 2 * pad - r) // stride + 1, (w + 2 * pad - s) // stride + 1


def resnet50_conv_layers() -> List[ConvShape]:
    """Every convolution of a standard ResNet-50 bottleneck stack except the
    7x7 stem (the paper leaves the first convolution un-quantized, Section 5).
    Stride 2 sits on the 3x3 of the first block of stages 3-5; the projection
    shortcuts are included.  Identical shapes are merged with a count."""
    seq: List[ConvShape] = []
    hw = 56
    cin = 64
    for stage, (mid, blocks) in enumerate([(64, 3), (128, 4), (256, 6), (512, 3)], start=2):
        cout = mid * 4
        for b in range(blocks):
            stride = 2 if (b == 0 and stage > 2) else 1
            seq.append(ConvShape(f"s{stage}.1x1a", hw, hw, cin, mid, 1, 1, 1, 0))
            seq.append(ConvShape(f"s{stage}.3x3", hw, hw, mid, mid, 3, 3, stride, 1))
            if b == 0:
                seq.append(ConvShape(f"s{stage}.proj", hw, hw, cin, cout, 1, 1, stride, 0))
            hw = hw // stride
            seq.append(ConvShape(f"s{stage}.1x1b", hw, hw, mid, cout, 1, 1, 1, 0))
            cin = cout
    merged: List[ConvShape] = []
    index = {}
    for c in seq:
        key = (c.h, c.w, c.cin, c.cout, c.r, c.s, c.stride, c.pad)
        if key in index:
            i = index[key]
            m = merged[i]
            merged[i] = ConvShape(m.name, m.h, m.w, m.cin, m.cout, m.r, m.s, m.stride, m.pad, m.count + 1)
        else:
            index[key] = len(merged)
            merged.append(c)
    return merged


def inv_out_scale(k: int, zero_frac: float = 0.5) -> float:
    """A fixed requantization multiplier for a layer with reduction length ``k``.

    With the value recipe above an accumulator has a standard deviation of about
    ``sqrt(k * (1 - zero_frac) * 1600 * 900)`` and the mean per-channel scale is
    0.0055; the multiplier maps one standard deviation of the dequantized output
    to 40 on the next layer's uint8 grid (the activations' own half-normal)."""
    sigma_acc = (k * (1.0 - zero_frac) * 1600.0 * 900.0) ** 0.5
    return float(np.float32(40.0 / (sigma_acc * 0.0055)))


def sparse24_weights(seed: int, n_out: int, k: int, stream: int = 1):
    """2:4 structured-sparse weights in compressed form: (vals (n_out, k/2) int8, pos (n_out,
    k/2) uint8).  In every group of four reduction indices two coordinates are kept,
    uniformly among the six choices, in increasing order; values as `weights`."""
    assert k % 4 == 0
    vals = weights(seed, (n_out, k // 2))
    rng = _rng(seed, stream + 16)
    combos = np.array([(0, 1), (0, 2), (0, 3), (1, 2), (1, 3), (2, 3)], dtype=np.uint8)
    pick = rng.integers(0, 6, size=(n_out, k // 4))
    pos = combos[pick].reshape(n_out, k // 2)
    return vals, np.ascontiguousarray(pos)


def sparse24_dense(vals: np.ndarray, pos: np.ndarray) -> np.ndarray:
    """The dense (n_out, k) int8 matrix that the compressed form stands for (data movement only)."""
    n_out, half = vals.shape
    dense = np.zeros((n_out, half * 2), dtype=np.int8)
    cols = (np.arange(half) // 2 * 4)[None, :] + pos.astype(np.int64)
    np.put_along_axis(dense, cols, vals, axis=1)
    return dense
