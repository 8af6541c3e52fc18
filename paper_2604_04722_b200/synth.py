"""Seeded synthetic inputs for the adaptive KV-cache quantization hot path.

This module only draws random numbers and shapes them; it holds none of the
method's arithmetic (no controller, no quantizer, no attention).  The CPU
oracle and the CUDA path are both fed from here, so neither needs the other's
random number generator.

The workloads follow the shapes of the SmolLM backbones the paper evaluates
(Table 1: 30/32/24 layers, 9/15/32 heads) with head_dim 64 and grouped KV
heads, and stand in for the benchmark contexts the paper runs through those
models (Section 4.1), which are not available offline.

Recipe (all draws use numpy's PCG64 via ``default_rng`` with a key made of the
seed and the coordinates of the block being drawn, so any block can be
regenerated alone):

* K, V rows: N(0,1) in fp32; four "outlier" channels per (layer, KV head),
  drawn without replacement and independently for K and for V, are multiplied
  by 8; the result is rounded once to fp16.
* Q rows: N(0,1) rounded to fp16.
* bit-widths, i.i.d. mode: classes drawn from a 4-way categorical mix.
* bit-widths, run mode: contiguous runs, length ~ Geometric(1/mean_run),
  class of each run drawn from the mix.
* controller features (Eq. 17 gives the vector; the order used here is
  frequency, quality score, attention variance, entropy):
  col 0 truncated Zipf(1.1) rank over a 49152-word vocabulary, normalised to
  [0,1]; col 1 U(0,1); col 2 LogNormal(-2,1); col 3 U(0, ln 49152).
* controller weights (Eq. 19-21 shapes): Kaiming-uniform,
  W ~ U(+-sqrt(6/fan_in)), b ~ U(+-1/sqrt(fan_in)), fp32, row-major [out][in].
"""
from __future__ import annotations

import math
import os
from dataclasses import dataclass, field
from typing import Dict, Optional, Tuple

import numpy as np

VOCAB = 49152
BIT_CHOICES = np.array([2, 4, 8, 16], dtype=np.uint8)

# tags that separate the random streams
_TAG_K, _TAG_V, _TAG_Q, _TAG_BITS, _TAG_FEAT, _TAG_MLP, _TAG_OUTLIER = range(1, 8)


@dataclass(frozen=True)
class Workload:
    """One benchmark configuration (shapes + how its bit-widths are chosen)."""

    name: str
    layers: int
    batch: int
    q_heads: int
    kv_heads: int
    head_dim: int
    context: int                # tokens cached before the first decode step
    decode_steps: int           # decode steps, each appending one token per sequence
    bits_mode: str              # "iid" | "runs" | "controller"
    mix: Tuple[float, float, float, float] = (0.25, 0.25, 0.25, 0.25)
    mean_run: int = 16
    hidden: int = 32            # controller width used by this workload
    seed: int = 0               # data seed
    mlp_seed: int = 0           # controller-weight seed (picked so that all four classes occur)
    note: str = ""

    @property
    def max_ctx(self) -> int:
        return self.context + self.decode_steps


CONFIGS: Dict[str, Workload] = {
    "cfg1": Workload("cfg1", 1, 1, 9, 3, 64, 512, 0, "iid",
                     (0.40, 0.35, 0.20, 0.05), seed=0,
                     note="SmolLM-135M-shaped single layer, one decode step"),
    "cfg2": Workload("cfg2", 30, 1, 9, 3, 64, 2048, 64, "controller",
                     seed=0, mlp_seed=322,
                     note="SmolLM-135M-shaped full cache, controller bits"),
    "cfg3": Workload("cfg3", 32, 8, 15, 5, 64, 4096, 128, "controller",
                     seed=1, mlp_seed=98,
                     note="SmolLM-360M-shaped, batch 8"),
    "cfg4": Workload("cfg4", 24, 16, 32, 32, 64, 8192, 0, "runs",
                     (0.25, 0.40, 0.25, 0.10), mean_run=16, seed=0,
                     note="SmolLM-1.7B-shaped, geometric runs"),
    "cfg5": Workload("cfg5", 1, 16, 32, 32, 64, 32768, 0, "iid",
                     (0.50, 0.30, 0.15, 0.05), seed=0, mlp_seed=167,
                     note="stress: one SmolLM-1.7B-shaped layer, context 32768"),
}


def _rng(*key: int) -> np.random.Generator:
    return np.random.default_rng([int(k) & 0xFFFFFFFF for k in key])


def outlier_channels(seed: int, layer: int, kv_heads: int, head_dim: int,
                     tag: int) -> np.ndarray:
    """[kv_heads][4] channel indices that carry the x8 outliers."""
    rng = _rng(seed, _TAG_OUTLIER, tag, layer)
    return np.stack([rng.choice(head_dim, size=4, replace=False)
                     for _ in range(kv_heads)]).astype(np.int64)


def _rows(seed: int, tag: int, layer: int, b: int, t0: int, n: int,
          kv_heads: int, head_dim: int) -> np.ndarray:
    rng = _rng(seed, tag, layer, b, t0)
    x = rng.standard_normal((n, kv_heads, head_dim), dtype=np.float32)
    ch = outlier_channels(seed, layer, kv_heads, head_dim, tag)
    scale = np.ones((kv_heads, head_dim), dtype=np.float32)
    for h in range(kv_heads):
        scale[h, ch[h]] = 8.0
    x *= scale[None]
    return x.astype(np.float16)


def kv_rows(seed: int, layer: int, b: int, t0: int, n: int, kv_heads: int,
            head_dim: int = 64) -> Tuple[np.ndarray, np.ndarray]:
    """K and V rows of tokens [t0, t0+n) of sequence b: fp16 [n][kv_heads][head_dim].

    The stream is keyed by (seed, layer, b, t0): callers must cut a sequence
    into the same segments on both sides of a comparison.
    """
    return (_rows(seed, _TAG_K, layer, b, t0, n, kv_heads, head_dim),
            _rows(seed, _TAG_V, layer, b, t0, n, kv_heads, head_dim))


def kv_batch(seed: int, layer: int, batch: int, t0: int, n: int, kv_heads: int,
             head_dim: int = 64) -> Tuple[np.ndarray, np.ndarray]:
    """fp16 [batch][n][kv_heads][head_dim] for K and V.

    Blocks are independent streams, so large batches are drawn by a thread pool
    (numpy's generators release the GIL); the values do not depend on it.
    """
    K = np.empty((batch, n, kv_heads, head_dim), dtype=np.float16)
    V = np.empty_like(K)

    def fill(job):
        b, tag, out = job
        out[b] = _rows(seed, tag, layer, b, t0, n, kv_heads, head_dim)

    jobs = [(b, tag, out) for b in range(batch) for tag, out in ((_TAG_K, K), (_TAG_V, V))]
    if batch * n * kv_heads * head_dim < (1 << 22):
        for j in jobs:
            fill(j)
    else:
        from concurrent.futures import ThreadPoolExecutor
        with ThreadPoolExecutor(max_workers=min(len(jobs), os.cpu_count() or 1)) as ex:
            list(ex.map(fill, jobs))
    return K, V


def queries(seed: int, layer: int, step: int, batch: int, q_heads: int,
            head_dim: int = 64) -> np.ndarray:
    """fp16 [batch][q_heads][head_dim] ~ N(0,1)."""
    rng = _rng(seed, _TAG_Q, layer, step)
    return rng.standard_normal((batch, q_heads, head_dim),
                               dtype=np.float32).astype(np.float16)


def bits_iid(seed: int, b: int, t0: int, n: int, mix) -> np.ndarray:
    """uint8 [n] with values in {2,4,8,16}, i.i.d. from the 4-way mix."""
    rng = _rng(seed, _TAG_BITS, b, t0)
    p = np.asarray(mix, dtype=np.float64)
    cls = rng.choice(4, size=n, p=p / p.sum())
    return BIT_CHOICES[cls]


def bits_runs(seed: int, b: int, t0: int, n: int, mix, mean_run: int = 16) -> np.ndarray:
    """uint8 [n]: contiguous runs, length ~ Geometric(1/mean_run), class from the mix."""
    rng = _rng(seed, _TAG_BITS, b, t0, 1)
    p = np.asarray(mix, dtype=np.float64)
    out = np.empty(n, dtype=np.uint8)
    pos = 0
    while pos < n:
        # draw a batch of runs at a time
        m = max(16, (n - pos) // mean_run + 16)
        lens = rng.geometric(1.0 / mean_run, size=m)
        cls = rng.choice(4, size=m, p=p / p.sum())
        for ln, c in zip(lens, cls):
            if pos >= n:
                break
            end = min(n, pos + int(ln))
            out[pos:end] = BIT_CHOICES[c]
            pos = end
    return out


def bits_uniform(n: int, bits: int) -> np.ndarray:
    """uint8 [n] all equal to ``bits`` (the static uniform-precision baselines)."""
    return np.full(n, bits, dtype=np.uint8)


_ZIPF_CDF: Optional[np.ndarray] = None


def _zipf_cdf() -> np.ndarray:
    global _ZIPF_CDF
    if _ZIPF_CDF is None:
        r = np.arange(1, VOCAB + 1, dtype=np.float64)
        pmf = r ** -1.1
        _ZIPF_CDF = np.cumsum(pmf / pmf.sum())
    return _ZIPF_CDF


def features(seed: int, b: int, t0: int, n: int) -> np.ndarray:
    """float32 [n][4]: frequency, quality score, attention variance, entropy."""
    rng = _rng(seed, _TAG_FEAT, b, t0)
    cdf = _zipf_cdf()
    rank = np.searchsorted(cdf, rng.random(n), side="left") + 1     # 1..VOCAB
    rank = np.minimum(rank, VOCAB)
    f = np.empty((n, 4), dtype=np.float32)
    f[:, 0] = ((rank - 1) / float(VOCAB - 1)).astype(np.float32)
    f[:, 1] = rng.random(n).astype(np.float32)
    f[:, 2] = rng.lognormal(-2.0, 1.0, size=n).astype(np.float32)
    f[:, 3] = (rng.random(n) * math.log(VOCAB)).astype(np.float32)
    return f


def features_batch(seed: int, batch: int, t0: int, n: int) -> np.ndarray:
    """float32 [batch][n][4]."""
    return np.stack([features(seed, b, t0, n) for b in range(batch)])


@dataclass
class ControllerWeights:
    hidden: int
    W1: np.ndarray   # [hidden][4]
    b1: np.ndarray   # [hidden]
    W2: np.ndarray   # [hidden][hidden]
    b2: np.ndarray   # [hidden]
    W3: np.ndarray   # [4][hidden]
    b3: np.ndarray   # [4]

    def as_tuple(self):
        return (self.W1, self.b1, self.W2, self.b2, self.W3, self.b3)


def controller_weights(seed: int, hidden: int = 32) -> ControllerWeights:
    """Seeded Kaiming-uniform 4 -> hidden -> hidden -> 4 MLP parameters (fp32)."""
    rng = _rng(seed, _TAG_MLP, hidden)

    def lin(fan_out: int, fan_in: int):
        wb = math.sqrt(6.0 / fan_in)
        bb = 1.0 / math.sqrt(fan_in)
        W = rng.uniform(-wb, wb, size=(fan_out, fan_in)).astype(np.float32)
        b = rng.uniform(-bb, bb, size=(fan_out,)).astype(np.float32)
        return np.ascontiguousarray(W), np.ascontiguousarray(b)

    W1, b1 = lin(hidden, 4)
    W2, b2 = lin(hidden, hidden)
    W3, b3 = lin(4, hidden)
    return ControllerWeights(hidden, W1, b1, W2, b2, W3, b3)


def workload_bits(wl: Workload, b: int, t0: int, n: int) -> Optional[np.ndarray]:
    """Bit-widths of tokens [t0, t0+n) of sequence b for "iid"/"runs" workloads.

    Returns None for "controller" workloads, whose bit-widths are the method's
    own output (computed from ``features`` by whoever runs the controller).
    """
    if wl.bits_mode == "iid":
        return bits_iid(wl.seed, b, t0, n, wl.mix)
    if wl.bits_mode == "runs":
        return bits_runs(wl.seed, b, t0, n, wl.mix, wl.mean_run)
    return None
