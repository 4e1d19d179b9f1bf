"""Seeded synthetic weight sets shaped like the paper's workloads.

This module only draws numbers and lists shapes. It holds none of the C-step's
arithmetic (no u, no norms, no thresholds), so both the CPU oracle's tests and
the CUDA path can consume the same host buffers without sharing any method code.

The paper trains VGG-19 and ResNet-56 on CIFAR-10, a VGG-style CNN on ImageNet
and a 2-layer LSTM language model on WikiText-2 (Evaluation section, tasks 1-3).
Trained weights and datasets are not available offline, so every tensor here is
random with the same shapes and the usual initialisation statistics:

* Kaiming-normal (fan_in, gain sqrt(2)) for conv / fc weights,
* uniform(-0.1, 0.1) for the LSTM language model,
* lambda ~ N(0, sigma^2) with sigma = 1e-2 where a configuration asks for a
  non-zero multiplier, zeros otherwise (first L-C iteration).

Random numbers are counter based: element ``i`` of tensor ``t`` in stream ``r``
(0 = w, 1 = lambda) is a pure function of ``(seed, r, t, i)``, so a buffer can be
filled in any order and by any number of threads and is reproducible anywhere.
"""
from __future__ import annotations

import math
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field
from typing import List, Optional, Sequence, Tuple

import numpy as np

_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)
_GOLD = 0x9E3779B97F4A7C15
_MASK64 = (1 << 64) - 1


def _mix64_scalar(z: int) -> int:
    """splitmix64 output function on a Python int (Steele, Lea, Flood 2014)."""
    z &= _MASK64
    z ^= z >> 30
    z = (z * 0xBF58476D1CE4E5B9) & _MASK64
    z ^= z >> 27
    z = (z * 0x94D049BB133111EB) & _MASK64
    z ^= z >> 31
    return z


def _mix64(z: np.ndarray) -> np.ndarray:
    """Vectorised splitmix64 output function, in place on a uint64 array."""
    z ^= z >> np.uint64(30)
    z *= _M1
    z ^= z >> np.uint64(27)
    z *= _M2
    z ^= z >> np.uint64(31)
    return z


def _stream_key(seed: int, stream: int, tensor: int) -> int:
    base = _mix64_scalar((seed + _GOLD) & _MASK64)
    return base ^ ((stream & 0xFF) << 56) ^ ((tensor & 0xFFFF) << 40)


def _bits(seed: int, stream: int, tensor: int, start: int, count: int) -> np.ndarray:
    z = np.arange(start, start + count, dtype=np.uint64)
    z ^= np.uint64(_stream_key(seed, stream, tensor))
    return _mix64(z)


def _uniform01(h: np.ndarray) -> np.ndarray:
    """32-bit integers -> doubles strictly inside (0, 1)."""
    return (h.astype(np.float64) + 0.5) * (1.0 / 4294967296.0)


def _fill_chunk(out: np.ndarray, kind: str, scale: float, seed: int, stream: int,
                tensor: int, start: int) -> None:
    n = out.shape[0]
    z = _bits(seed, stream, tensor, start, n)
    hi = (z >> np.uint64(32)).astype(np.uint32)
    if kind == "uniform":
        u = _uniform01(hi)
        out[:] = ((2.0 * u - 1.0) * scale).astype(np.float32)
    elif kind == "normal":
        lo = (z & np.uint64(0xFFFFFFFF)).astype(np.uint32)
        u1 = _uniform01(hi)
        u2 = _uniform01(lo)
        r = np.sqrt(-2.0 * np.log(u1))
        out[:] = (r * np.cos((2.0 * math.pi) * u2) * scale).astype(np.float32)
    else:  # pragma: no cover
        raise ValueError(kind)


_CHUNK = 1 << 21


def draw(n: int, kind: str, scale: float, seed: int, stream: int, tensor: int,
         threads: int = 8) -> np.ndarray:
    """``n`` float32 values; ``kind`` is 'normal' (sigma=scale), 'uniform'
    (on (-scale, scale)) or 'zeros'."""
    out = np.zeros(n, dtype=np.float32)
    if kind == "zeros" or n == 0:
        return out
    jobs = [(s, min(s + _CHUNK, n)) for s in range(0, n, _CHUNK)]

    def run(job):
        a, b = job
        _fill_chunk(out[a:b], kind, scale, seed, stream, tensor, a)

    if len(jobs) == 1 or threads <= 1:
        for j in jobs:
            run(j)
    else:
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(run, jobs))
    return out


@dataclass
class WeightSet:
    """A list of host tensors plus the call the configuration makes on them."""
    name: str
    shapes: List[Tuple[int, ...]]
    w: List[np.ndarray]
    lam: List[np.ndarray]
    mu: float
    op: str                      # 'prune' | 'filter' | 'block'
    sparsity: float
    fuse: Tuple[str, ...]        # subset of ('fp16', 'lambda', 'penalty')
    block: Tuple[int, int] = (4, 4)
    seed: int = 0
    notes: str = ""
    names: List[str] = field(default_factory=list)

    @property
    def numel(self) -> int:
        return int(sum(int(np.prod(s)) for s in self.shapes))


def _kaiming_sigma(shape: Sequence[int]) -> float:
    fan_in = int(np.prod(shape[1:])) if len(shape) > 1 else int(shape[0])
    return math.sqrt(2.0 / fan_in)


def resnet56_shapes() -> List[Tuple[int, ...]]:
    """CIFAR ResNet-56: conv1, 3 stages x 9 basic blocks (two 3x3 convs each),
    1x1 projection shortcuts at the two stage changes, fc. 58 tensors."""
    shapes: List[Tuple[int, ...]] = [(16, 3, 3, 3)]
    cin = 16
    for cout in (16, 32, 64):
        for b in range(9):
            shapes.append((cout, cin if b == 0 else cout, 3, 3))
            shapes.append((cout, cout, 3, 3))
            if b == 0 and cin != cout:
                shapes.append((cout, cin, 1, 1))
        cin = cout
    shapes.append((10, 64))
    return shapes


def vgg19_shapes() -> List[Tuple[int, ...]]:
    """CIFAR VGG-19: sixteen 3x3 convs and a 10-way classifier."""
    plan = [(3, 64), (64, 64), (64, 128), (128, 128), (128, 256), (256, 256),
            (256, 256), (256, 256), (256, 512)] + [(512, 512)] * 7
    return [(co, ci, 3, 3) for ci, co in plan] + [(10, 512)]


def alexnet_shapes() -> List[Tuple[int, ...]]:
    return [(96, 3, 11, 11), (256, 96, 5, 5), (384, 256, 3, 3), (384, 384, 3, 3),
            (256, 384, 3, 3), (4096, 9216), (4096, 4096), (1000, 4096)]


def lstm_lm_shapes(tied: bool = False, vocab: int = 33278, hidden: int = 1500
                   ) -> List[Tuple[int, ...]]:
    shapes: List[Tuple[int, ...]] = [(vocab, hidden)]
    for _ in range(2):
        shapes += [(4 * hidden, hidden), (4 * hidden, hidden), (4 * hidden,), (4 * hidden,)]
    if not tied:
        shapes.append((vocab, hidden))
    return shapes


def _build(name, shapes, w_kind, w_scale, lam_sigma, mu, op, sparsity, fuse, seed,
           notes="", threads=8) -> WeightSet:
    ws, lams = [], []
    for t, shp in enumerate(shapes):
        n = int(np.prod(shp))
        if w_kind == "kaiming":
            w = draw(n, "normal", _kaiming_sigma(shp), seed, 0, t, threads)
        elif w_kind == "normal":
            w = draw(n, "normal", w_scale, seed, 0, t, threads)
        else:
            w = draw(n, "uniform", w_scale, seed, 0, t, threads)
        lam = draw(n, "normal" if lam_sigma > 0 else "zeros", lam_sigma, seed, 1, t, threads)
        ws.append(w.reshape(shp))
        lams.append(lam.reshape(shp))
    return WeightSet(name=name, shapes=[tuple(s) for s in shapes], w=ws, lam=lams, mu=mu,
                     op=op, sparsity=sparsity, fuse=tuple(fuse), seed=seed, notes=notes)


def config(which, scale: float = 1.0, threads: int = 8) -> WeightSet:
    """The five benchmark configurations ('1'..'5', plus '5t' with the decoder
    tied to the embedding). ``scale`` < 1 shrinks every dimension except kernel
    sizes, for quick parity runs that keep the structure (many tensors, ragged
    block edges, mixed filter lengths)."""
    which = str(which)

    def sc(shapes):
        if scale == 1.0:
            return shapes
        out = []
        for s in shapes:
            if len(s) == 4:
                out.append((max(2, int(round(s[0] * scale))), max(1, int(round(s[1] * scale))),
                            s[2], s[3]))
            else:
                out.append(tuple(max(3, int(round(d * scale))) for d in s))
        return out

    if which == "1":
        n = max(16, int(round(1048576 * scale)))
        return _build("cfg1-single-1M", [(n,)], "normal", 0.05, 0.0, 1e-3, "prune", 0.9,
                      ("fp16", "lambda"), 0, "single tensor, P+Q", threads)
    if which == "2":
        return _build("cfg2-resnet56", sc(resnet56_shapes()), "kaiming", 0.0, 1e-2, 1e-2,
                      "prune", 0.95, ("lambda",), 1, "58 tensors", threads)
    if which == "3":
        return _build("cfg3-vgg19", sc(vgg19_shapes()), "kaiming", 0.0, 0.0, 1e-3,
                      "filter", 0.8, ("lambda",), 2, "filter pruning", threads)
    if which == "4":
        return _build("cfg4-alexnet", sc(alexnet_shapes()), "kaiming", 0.0, 1e-2, 1e-3,
                      "prune", 0.98, ("fp16", "lambda", "penalty"), 3, "P+Q + penalty", threads)
    if which in ("5", "5t"):
        shapes = lstm_lm_shapes(tied=(which == "5t"))
        if scale != 1.0:
            v = max(6, int(round(33278 * scale)) | 2)      # keep vocab % 4 == 2 (ragged rows)
            h = max(4, (int(round(1500 * scale)) // 4) * 4)
            shapes = lstm_lm_shapes(tied=(which == "5t"), vocab=v, hidden=h)
        return _build("cfg%s-lstm-lm" % which, shapes, "uniform", 0.1, 0.0, 1e-3,
                      "block", 0.9, ("lambda",), 4, "4x4 block pruning", threads)
    raise ValueError("unknown configuration %r" % (which,))


def config_numel(which) -> int:
    """Parameters of a configuration at full size, without drawing it."""
    which = str(which)
    if which == "1":
        return 1048576
    shapes = {"2": resnet56_shapes, "3": vgg19_shapes, "4": alexnet_shapes,
              "5": lstm_lm_shapes, "5t": lambda: lstm_lm_shapes(tied=True)}[which]()
    return int(sum(int(np.prod(s)) for s in shapes))


def random_set(shapes: Sequence[Sequence[int]], seed: int, kind: str = "normal",
               scale: float = 1.0, lam_sigma: float = 0.0, mu: float = 1e-3,
               op: str = "prune", sparsity: float = 0.5,
               fuse: Sequence[str] = ("lambda",)) -> WeightSet:
    """Small ad-hoc weight set for tests."""
    return _build("random", [tuple(s) for s in shapes], kind, scale, lam_sigma, mu, op,
                  sparsity, fuse, seed, threads=1)
