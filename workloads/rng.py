"""Seeded random numbers for the synthetic workloads.

One splitmix64 stream per (config, purpose); bulk Gaussian draws (logits) come
from a numpy generator keyed by a value drawn from such a stream.  Nothing here
knows about grammars or parsing.
"""
from __future__ import annotations

import numpy as np

BASE_SEED = 250601151
_M64 = (1 << 64) - 1


class SplitMix64:
    """The splitmix64 generator (Steele, Lea, Flood 2014), 64-bit state."""

    def __init__(self, seed: int):
        self.state = seed & _M64

    def next_u64(self) -> int:
        self.state = (self.state + 0x9E3779B97F4A7C15) & _M64
        z = self.state
        z = ((z ^ (z >> 30)) * 0xBF58476D1CE4E5B9) & _M64
        z = ((z ^ (z >> 27)) * 0x94D049BB133111EB) & _M64
        return z ^ (z >> 31)

    def below(self, n: int) -> int:
        """Uniform integer in [0, n)."""
        return self.next_u64() % n

    def between(self, lo: int, hi: int) -> int:
        """Uniform integer in [lo, hi]."""
        return lo + self.next_u64() % (hi - lo + 1)

    def unit(self) -> float:
        return (self.next_u64() >> 11) * (1.0 / (1 << 53))

    def chance(self, p: float) -> bool:
        return self.unit() < p

    def pick(self, seq):
        return seq[self.below(len(seq))]

    def geometric(self, mean: float) -> int:
        """Geometric on {0,1,2,...} with the given mean."""
        p = 1.0 / (1.0 + mean)
        k = 0
        while not self.chance(p):
            k += 1
            if k > 10_000:
                break
        return k


def stream(config: int, purpose: str) -> SplitMix64:
    """Independent stream for one purpose of one config."""
    h = BASE_SEED * 10 + config
    for ch in purpose.encode():
        h = (h * 0x100000001B3 + ch) & _M64
    return SplitMix64(h)


def numpy_generator(config: int, purpose: str) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(stream(config, purpose).next_u64()))
