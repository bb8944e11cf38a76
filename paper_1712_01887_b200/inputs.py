"""Seeded synthetic gradient sets with the shapes of the paper's workloads.

This module serves both the CUDA path and the CPU oracle with *identical
bits*: every gradient is generated once, on the host, by a counter-based
generator (numpy's Philox keyed by (seed + worker, workload, iteration)) and
handed to both sides.  It holds none of the method's arithmetic: no clipping,
no momentum, no selection, no top-k counts.

The paper trains on ImageNet, Penn Treebank and LibriSpeech; none of that data
is used.  Each workload below takes its tensor *shapes* from the model the
paper names (Sec. 4.1-4.4) and fills them with a stated value distribution.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Sequence, Tuple

import numpy as np

BASE_SEED = 171201887


# --------------------------------------------------------------------------- shapes

def resnet50_shapes() -> List[Tuple[int, ...]]:
    """The 161 conv / batch-norm / fc parameter tensors of a standard ResNet-50
    (Table 3 workload: 25,557,032 fp32 values = 97.49 MiB)."""
    shapes: List[Tuple[int, ...]] = [(64, 3, 7, 7), (64,), (64,)]
    inplanes = 64
    for planes, blocks in ((64, 3), (128, 4), (256, 6), (512, 3)):
        for b in range(blocks):
            shapes += [(planes, inplanes, 1, 1), (planes,), (planes,)]
            shapes += [(planes, planes, 3, 3), (planes,), (planes,)]
            shapes += [(planes * 4, planes, 1, 1), (planes * 4,), (planes * 4,)]
            if b == 0:
                shapes += [(planes * 4, inplanes, 1, 1), (planes * 4,), (planes * 4,)]
            inplanes = planes * 4
    shapes += [(1000, 2048), (1000,)]
    return shapes


def lstm_lm_shapes(vocab: int = 10000, hidden: int = 1500) -> List[Tuple[int, ...]]:
    """2-layer LSTM language model (Sec. 4.3), untied embedding and softmax: 11 tensors."""
    shapes: List[Tuple[int, ...]] = [(vocab, hidden)]
    for _ in range(2):
        shapes += [(4 * hidden, hidden), (4 * hidden, hidden), (4 * hidden,), (4 * hidden,)]
    shapes += [(vocab, hidden), (vocab,)]
    return shapes


def deepspeech_shapes(hidden: int = 1024, scale_div: int = 1) -> List[Tuple[int, ...]]:
    """DeepSpeech-shaped set (Sec. 4.4): 2 conv layers, 7 bidirectional GRU layers,
    fc to 29 classes: 62 tensors, 122,096,829 values at hidden=1024.
    scale_div > 1 shrinks the hidden size for small parity cases."""
    h = hidden // scale_div
    first_in = 352 // scale_div if scale_div > 1 else 352
    shapes: List[Tuple[int, ...]] = [(32, 1, 41, 11), (32,), (32, 32, 21, 11), (32,)]
    for layer in range(7):
        inp = first_in if layer == 0 else 2 * h
        for _direction in range(2):
            shapes += [(3 * h, inp), (3 * h, h), (3 * h,), (3 * h,)]
    shapes += [(29, 2 * h), (29,)]
    return shapes


def numel_of(shapes: Sequence[Tuple[int, ...]]) -> List[int]:
    return [int(np.prod(s)) for s in shapes]


# --------------------------------------------------------------------------- workloads

@dataclass
class Workload:
    """One benchmark / parity configuration."""
    name: str
    shapes: List[Tuple[int, ...]]
    num_workers: int
    momentum: float
    clip_threshold: float          # thr_G before the N^-1/2 scaling; <= 0: off
    sparsity: float
    iterations: int
    kind: str                      # value recipe, see fill()
    sample_ratio: float = 0.01
    sigma: np.ndarray = field(default=None, repr=False)   # per-tensor scale (resnet50)

    @property
    def numel(self) -> List[int]:
        return numel_of(self.shapes)

    @property
    def total(self) -> int:
        return int(sum(self.numel))


def _rng(tag: int, worker: int, iteration: int, seed: int = BASE_SEED) -> np.random.Generator:
    key = [np.uint64(seed + worker), np.uint64((tag << 32) | (iteration & 0xFFFFFFFF))]
    return np.random.Generator(np.random.Philox(key=key))


_TAGS = {"outlier": 1, "resnet50": 2, "lstm": 3, "deepspeech": 4, "normal": 5}


def workload(name: str, **kw) -> Workload:
    """The five configurations.  `name` in
    cfg1 | resnet50 | lstm | deepspeech | deepspeech_small | sweep (needs n=...)."""
    if name == "cfg1":
        return Workload("cfg1", [(1 << 20,)], 4, 0.9, 1.0, 0.999, 5, "outlier")
    if name == "resnet50":
        shapes = resnet50_shapes()
        g = np.random.Generator(np.random.Philox(key=[np.uint64(BASE_SEED), np.uint64(0x5157)]))
        sigma = (10.0 ** (-5.0 + 3.0 * g.random(len(shapes)))).astype(np.float32)
        return Workload("resnet50", shapes, 8, 0.9, 0.0, 0.999, 10, "resnet50", sigma=sigma)
    if name == "lstm":
        return Workload("lstm", lstm_lm_shapes(), 4, 0.9, 1.0, 0.999, 10, "lstm")
    if name == "lstm_small":
        return Workload("lstm_small", lstm_lm_shapes(vocab=1000, hidden=150), 4, 0.9, 1.0, 0.999,
                        10, "lstm")
    if name == "deepspeech":
        return Workload("deepspeech", deepspeech_shapes(), 4, 0.9, 1.0, 0.75, 100, "deepspeech")
    if name == "deepspeech_small":
        return Workload("deepspeech_small", deepspeech_shapes(scale_div=4), 4, 0.9, 1.0, 0.75, 100,
                        "deepspeech")
    if name == "sweep":
        n = int(kw["n"])
        return Workload(f"sweep_{n}", [(n,)], 1, 0.9, 0.0, float(kw.get("sparsity", 0.999)), 3,
                        "normal")
    raise ValueError(name)


def fill(wl: Workload, arena: np.ndarray, offset: Sequence[int], worker: int, iteration: int,
         seed: int = BASE_SEED) -> None:
    """Write worker `worker`'s gradient of iteration `iteration` into `arena`
    (float32), tensor j at arena[offset[j] : offset[j] + numel[j]].  Slots
    between tensors are left untouched."""
    assert arena.dtype == np.float32
    rng = _rng(_TAGS[wl.kind], worker, iteration, seed)
    numel = wl.numel
    for j, n in enumerate(numel):
        dst = arena[offset[j]: offset[j] + n]
        if wl.kind == "outlier":
            # N(0, 1e-3) with 1% of entries replaced by Laplace(0, 1e-2) outliers
            x = rng.standard_normal(n, dtype=np.float32) * np.float32(1e-3)
            pick = rng.random(n, dtype=np.float32) < np.float32(0.01)
            lap = rng.laplace(0.0, 1e-2, size=int(pick.sum())).astype(np.float32)
            x[pick] = lap
            dst[:] = x
        elif wl.kind == "resnet50":
            dst[:] = rng.standard_normal(n, dtype=np.float32) * wl.sigma[j]
        elif wl.kind == "lstm":
            x = rng.standard_normal(n, dtype=np.float32) * np.float32(1e-3)
            if j == 0:
                # embedding gradient: about 2% of the rows non-zero, the others exactly +0
                rows, cols = wl.shapes[0]
                live = rng.random(rows) < 0.02
                x = x.reshape(rows, cols)
                x[~live, :] = 0.0
                x = x.reshape(-1)
            dst[:] = x
        elif wl.kind == "deepspeech":
            # Student-t(nu=3) * 1e-4 = Z / sqrt(chi2_3 / 3) * 1e-4, built in float32
            z = rng.standard_normal(n, dtype=np.float32)
            c = rng.standard_normal(n, dtype=np.float32) ** 2
            c += rng.standard_normal(n, dtype=np.float32) ** 2
            c += rng.standard_normal(n, dtype=np.float32) ** 2
            c /= np.float32(3.0)
            np.sqrt(c, out=c)
            z /= c
            z *= np.float32(1e-4)
            dst[:] = z
        elif wl.kind == "normal":
            dst[:] = rng.standard_normal(n, dtype=np.float32)
        else:
            raise ValueError(wl.kind)


def packed_layout(numel: Sequence[int], align: int = 1) -> Tuple[np.ndarray, int]:
    """Tensor start offsets for tensors laid back to back, each start rounded up
    to `align` elements; returns (offsets, arena_len)."""
    off = []
    pos = 0
    for n in numel:
        pos = -(-pos // align) * align
        off.append(pos)
        pos += int(n)
    arena_len = -(-pos // align) * align
    return np.asarray(off, dtype=np.int64), int(arena_len)


def warmup_stage_of(iteration: int, iters_per_stage: int = 20) -> int:
    """Stage index 0..4 of the warm-up schedule for an iteration counter
    (DeepSpeech-shaped workload: 5 stages of 20 iterations)."""
    return min(iteration // iters_per_stage, 4)
