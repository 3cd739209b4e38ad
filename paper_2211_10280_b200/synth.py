"""Seeded synthetic inputs for the SGNS / DASGD hot path.

This module only *generates inputs* (token streams, unigram counts, initial
embedding tables, drift permutations) and names the workload presets.  It holds
none of the method's arithmetic: no Philox-based negative sampling, no alias
table, no gradient maths.  Both the CUDA path and the CPU oracle are fed the
arrays produced here; neither is imported from here.

The token streams stand in for the word stream of a natural-language corpus:
unigram frequencies of text are Zipf-like, so tokens are drawn i.i.d. from
Zipf(s) over the vocabulary ranks (rank r has probability proportional to
(r+1)^-s), optionally relabelled by a rank -> token permutation to emulate a
concept drift.
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import List, Optional, Sequence

import numpy as np


@dataclass(frozen=True)
class Workload:
    """One named workload: model shape, batch shape, replicas and stream law."""

    name: str
    V: int            # vocabulary size
    d: int            # embedding dimension
    window: int       # symmetric context window w
    k: int            # negatives per pair
    batch: int        # centre tokens per mini-batch (B)
    W: int            # logical model replicas
    batches: int      # mini-batches per replica
    zipf_s: float     # Zipf exponent of the token stream
    stream_seeds: tuple  # one seed per replica substream
    max_delay: int = 0    # message delivery delay bound, in whole steps
    drift_every: int = 0  # re-draw the rank->token permutation every this many batches (0 = never)
    lr: float = 0.025
    seed: int = 0         # library seed (negative sampler, delays)
    reduction: int = 0    # 0: batch loss = sum of the pair losses; 1: their mean
    max_grad_buffer: int = 1  # a replica sends after every this many of its batches
    routed: int = 0       # 1: the replicas share replica 0's batches, each training the centre words routed to it

    @property
    def pairs_per_batch(self) -> int:
        return n_pairs(self.batch, self.window)


def n_pairs(n: int, w: int) -> int:
    """Number of (centre, context) pairs of a batch of n tokens, window clipped to the batch."""
    return sum(min(q, w) + min(n - 1 - q, w) for q in range(n)) if n < 2 * w + 2 else 2 * w * n - w * (w + 1)


TINY = Workload("sgns_tiny", V=10_000, d=64, window=2, k=5, batch=512, W=1, batches=200,
                zipf_s=1.0, stream_seeds=(0,), seed=0)
MID = Workload("sgns_mid", V=100_000, d=128, window=5, k=5, batch=4096, W=1, batches=2000,
               zipf_s=1.0, stream_seeds=(1,), seed=1, reduction=1)
LARGE_DASGD = Workload("sgns_large_dasgd", V=1_000_000, d=300, window=5, k=15, batch=8192, W=4,
                       batches=500, zipf_s=1.0, stream_seeds=(2, 3, 4, 5), max_delay=2, seed=2, reduction=1)
LARGE_DRIFT = Workload("sgns_large_drift", V=1_000_000, d=300, window=5, k=15, batch=16384, W=8,
                       batches=1000, zipf_s=1.1, stream_seeds=tuple(range(6, 14)), max_delay=2,
                       drift_every=100, seed=6, reduction=1)


def sweep_point(d: int, batch: int, k: int) -> Workload:
    """One point of the throughput sweep (V = 1M, one replica, window 5, 100 batches)."""
    return Workload(f"sgns_sweep_d{d}_B{batch}_k{k}", V=1_000_000, d=d, window=5, k=k, batch=batch,
                    W=1, batches=100, zipf_s=1.0, stream_seeds=(14,), seed=14, reduction=1)


SWEEP = [sweep_point(d, b, k) for d in (64, 128, 300, 512) for b in (256, 2048, 16384, 65536)
         for k in (5, 15)]

WORKLOADS = {w.name: w for w in [TINY, MID, LARGE_DASGD, LARGE_DRIFT] + SWEEP}


def scaled(w: Workload, **kw) -> Workload:
    """A copy of a workload with some fields replaced (used for reduced-size test cases)."""
    return replace(w, **kw)


def _rng(seed: int, stream: int = 0) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[int(seed), int(stream)]))


def zipf_cdf(V: int, s: float) -> np.ndarray:
    w = np.arange(1, V + 1, dtype=np.float64) ** (-float(s))
    cdf = np.cumsum(w)
    cdf /= cdf[-1]
    return cdf


def zipf_ranks(V: int, s: float, n: int, seed: int, cdf: Optional[np.ndarray] = None) -> np.ndarray:
    """n i.i.d. Zipf(s) ranks in [0, V) by inverse-CDF lookup of seeded uniforms."""
    if cdf is None:
        cdf = zipf_cdf(V, s)
    u = _rng(seed, 1).random(n)
    r = np.searchsorted(cdf, u, side="right")
    return np.minimum(r, V - 1).astype(np.int32)


def drift_permutation(V: int, seed: int, epoch: int) -> np.ndarray:
    """Rank -> token permutation of drift epoch `epoch` (epoch 0 is also a random permutation)."""
    return _rng(seed, 1000 + epoch).permutation(V).astype(np.int32)


def token_stream(w: Workload, replica: int, batches: Optional[int] = None) -> np.ndarray:
    """The replica's substream as an int32 array [batches, batch] of token ids.

    Without drift the rank -> token map is the identity (a frequency-sorted
    vocabulary).  With drift the map is re-drawn every `drift_every` batches,
    the same for all replicas.
    """
    nb = w.batches if batches is None else batches
    ranks = zipf_ranks(w.V, w.zipf_s, nb * w.batch, w.stream_seeds[replica]).reshape(nb, w.batch)
    if not w.drift_every:
        return ranks
    out = np.empty_like(ranks)
    for e in range((nb + w.drift_every - 1) // w.drift_every):
        perm = drift_permutation(w.V, w.seed, e)
        sl = slice(e * w.drift_every, min(nb, (e + 1) * w.drift_every))
        out[sl] = perm[ranks[sl]]
    return out


def stream_counts(streams: Sequence[np.ndarray], V: int) -> np.ndarray:
    """Unigram counts of the given streams plus one (so that no count is zero), as uint64[V]."""
    c = np.ones(V, dtype=np.uint64)
    for s in streams:
        c += np.bincount(np.asarray(s).ravel(), minlength=V).astype(np.uint64)
    return c


def init_tables(V: int, d: int, seed: int):
    """Initial tables: input rows ~ U(-0.5/d, 0.5/d) in fp32, output rows zero."""
    u = _rng(seed, 2).random((V, d), dtype=np.float32)
    w_in = ((u - np.float32(0.5)) / np.float32(d)).astype(np.float32)
    w_out = np.zeros((V, d), dtype=np.float32)
    return w_in, w_out


def random_tables(V: int, d: int, seed: int, scale: float = 0.5):
    """Both tables random (for tests that need non-zero output rows)."""
    g = _rng(seed, 3)
    w_in = ((g.random((V, d), dtype=np.float32) - np.float32(0.5)) * np.float32(2 * scale)).astype(np.float32)
    w_out = ((g.random((V, d), dtype=np.float32) - np.float32(0.5)) * np.float32(2 * scale)).astype(np.float32)
    return w_in, w_out


def all_streams(w: Workload, batches: Optional[int] = None) -> List[np.ndarray]:
    return [token_stream(w, r, batches) for r in range(w.W)]
