"""Seeded synthetic multi-path token streams.

These streams stand in for sampled reasoning traces of one prompt: several
paths drawn from the same model share sub-steps (here: segments from a common
pool) in different order, separated by private tokens.  The module only draws
random tokens and log-probabilities; it contains none of the draft-construction
arithmetic, so the CPU oracle and the CUDA library can both be fed from it.

Random numbers come from splitmix64 (Steele, Lea, Flood 2014) used as a
counter-based generator: draw ``n`` of stream ``seed`` is
``mix(seed + (n + 1) * GOLDEN)``.
"""
from __future__ import annotations

import dataclasses
import numpy as np

_GOLDEN = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)

BASE_SEED = 20250305 * 16


def splitmix64(seed: int, start: int, count: int) -> np.ndarray:
    """Outputs ``start .. start+count-1`` of the splitmix64 stream ``seed``."""
    with np.errstate(over="ignore"):
        n = np.arange(start + 1, start + count + 1, dtype=np.uint64)
        z = np.uint64(seed & 0xFFFFFFFFFFFFFFFF) + n * _GOLDEN
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
        return z ^ (z >> np.uint64(31))


class Stream:
    """Sequential reader of uniforms in [0, 1) from one splitmix64 stream."""

    def __init__(self, seed: int, block: int = 1 << 14):
        self.seed = seed
        self.block = block
        self.pos = 0
        self.buf = np.empty(0)
        self.off = 0

    def uniform(self, n: int) -> np.ndarray:
        out = np.empty(n, dtype=np.float64)
        filled = 0
        while filled < n:
            if self.off == len(self.buf):
                raw = splitmix64(self.seed, self.pos, self.block)
                self.pos += self.block
                self.buf = (raw >> np.uint64(11)).astype(np.float64) * (1.0 / (1 << 53))
                self.off = 0
            take = min(n - filled, len(self.buf) - self.off)
            out[filled:filled + take] = self.buf[self.off:self.off + take]
            self.off += take
            filled += take
        return out

    def one(self) -> float:
        return float(self.uniform(1)[0])


@dataclasses.dataclass(frozen=True)
class Workload:
    """One benchmark configuration (shapes and the stream recipe)."""

    name: str
    G: int                 # independent prompts (groups)
    N: int                 # paths per prompt
    L: int                 # history capacity per path
    V: int                 # vocabulary size
    k_max: int             # largest query suffix length
    D: int                 # maximum draft length
    steps: int             # decode steps (upper bound)
    segments: int          # shared segments per prompt
    seg_len: tuple         # inclusive segment length range
    zipf: float            # Zipf exponent of token ids inside segments
    overlap: float         # probability that the next run is a shared segment
    lp_mean: float         # logprob ~ -Exponential(mean)
    seg_zipf: float = 0.0  # > 0: segments drawn Zipf(seg_zipf) instead of uniformly
    index: int = 0

    @property
    def P(self) -> int:
        return self.G * self.N


WORKLOADS = {
    1: Workload("cfg1_n4_l256", 1, 4, 256, 32000, 3, 4, 50, 20, (8, 32), 1.1, 0.70, 0.5, index=1),
    2: Workload("cfg2_n16_l1024", 1, 16, 1024, 128256, 4, 8, 500, 60, (8, 64), 1.1, 0.40, 0.5, index=2),
    3: Workload("cfg3_n64_l2048", 1, 64, 2048, 128256, 4, 8, 1000, 120, (8, 64), 1.1, 0.25, 0.5, index=3),
    4: Workload("cfg4_32x16_l4096", 32, 16, 4096, 151936, 5, 12, 2000, 100, (16, 96), 1.2, 0.35, 0.4, index=4),
    5: Workload("cfg5_n256_l8192", 1, 256, 8192, 151936, 8, 16, 500, 200, (8, 64), 1.1, 0.10, 1.0,
                seg_zipf=1.0, index=5),
}


def _zipf_cdf(n: int, s: float) -> np.ndarray:
    w = np.arange(1, n + 1, dtype=np.float64) ** (-s)
    c = np.cumsum(w)
    return c / c[-1]


def _lengths(u: np.ndarray, lo: int, hi: int) -> np.ndarray:
    return lo + np.minimum((u * (hi - lo + 1)).astype(np.int64), hi - lo)


def make_streams(w: Workload, seed: int | None = None):
    """Full-length streams for every path of ``w``.

    Returns ``(tokens int32 [P, L], logprobs float32 [P, L])``.  Group ``g`` of
    a multi-prompt workload uses seed ``seed + 1000 * g`` for its own pool.
    """
    if seed is None:
        seed = BASE_SEED + w.index
    tokens = np.empty((w.P, w.L), dtype=np.int32)
    logprobs = np.empty((w.P, w.L), dtype=np.float32)
    tok_cdf = _zipf_cdf(w.V, w.zipf)
    seg_cdf = _zipf_cdf(w.segments, w.seg_zipf) if w.seg_zipf > 0 else None
    lo, hi = w.seg_len
    for g in range(w.G):
        gseed = seed + 1000 * g
        pool_rng = Stream(gseed * 7919 + 1)
        seg_lens = _lengths(pool_rng.uniform(w.segments), lo, hi)
        pool = [np.searchsorted(tok_cdf, pool_rng.uniform(int(n)), side="right").astype(np.int32)
                for n in seg_lens]
        pool = [np.minimum(p, w.V - 1) for p in pool]
        for n in range(w.N):
            p = g * w.N + n
            rng = Stream(gseed * 7919 + 1000003 * (n + 1))
            filled = 0
            while filled < w.L:
                if rng.one() < w.overlap:
                    u = rng.one()
                    if seg_cdf is None:
                        s = min(int(u * w.segments), w.segments - 1)
                    else:
                        s = min(int(np.searchsorted(seg_cdf, u, side="right")), w.segments - 1)
                    run = pool[s]
                else:
                    length = int(_lengths(rng.uniform(1), lo, hi)[0])
                    run = np.minimum((rng.uniform(length) * w.V).astype(np.int32), w.V - 1)
                take = min(len(run), w.L - filled)
                tokens[p, filled:filled + take] = run[:take]
                filled += take
            u = rng.uniform(w.L)
            logprobs[p] = (w.lp_mean * np.log1p(-u)).astype(np.float32)
    return tokens, logprobs


def small_random(P: int, L: int, V: int, seed: int, lp_mean: float = 0.5):
    """Dense tiny case: i.i.d. uniform tokens over a small vocabulary."""
    rng = Stream(seed * 31 + 17)
    tokens = np.minimum((rng.uniform(P * L) * V).astype(np.int32), V - 1).reshape(P, L)
    logprobs = (lp_mean * np.log1p(-rng.uniform(P * L))).astype(np.float32).reshape(P, L)
    return tokens, logprobs


def sampled_window(tokens: np.ndarray, logprobs: np.ndarray, lens: np.ndarray, width: int):
    """The next ``width`` stream entries of every path after position ``lens``.

    Positions past the end of the stream hold token -1 and logprob 0.
    """
    P, L = tokens.shape
    idx = lens[:, None].astype(np.int64) + np.arange(width)[None, :]
    ok = idx < L
    idx = np.minimum(idx, L - 1)
    rows = np.arange(P)[:, None]
    t = np.where(ok, tokens[rows, idx], -1).astype(np.int32)
    lp = np.where(ok, logprobs[rows, idx], 0.0).astype(np.float32)
    return t, lp
