"""Shared helpers of the GPU parity tests: drive the CUDA library and the CPU oracle side by
side on the same seeded workload and compare bit for bit."""
from __future__ import annotations

import numpy as np

import oracle
import workloads


def torch_mod():
    import torch

    return torch


class OracleBatch:
    """One full-chart oracle sequence per row."""

    def __init__(self, w: workloads.Workload, pruned: bool = False):
        self.w = w
        self.g = oracle.Grammar(w.ebnf, w.start)
        self.vocab = oracle.Vocab(w.vocab, w.eos)
        self.pruned = pruned
        self.seqs = [oracle.Sequence_(self.g, pruned=pruned) for _ in range(w.batch)]
        self.finished = [False] * w.batch

    def reset(self, b: int):
        self.seqs[b] = oracle.Sequence_(self.g, pruned=self.pruned)
        self.finished[b] = False

    def advance(self, b: int, tok: int) -> int:
        """Returns the status the library must report for this row."""
        from paper_2506_01151_b200 import ERR_FINISHED, ERR_INVALID_ARG, ERR_TOKEN_REJECTED, FMT_OK

        if tok == -1:
            return FMT_OK
        if self.finished[b]:
            return ERR_FINISHED
        if tok < 0 or tok >= self.w.V:
            return ERR_INVALID_ARG
        if tok == self.w.eos:
            if self.seqs[b].accepting:
                self.finished[b] = True
                return FMT_OK
            return ERR_TOKEN_REJECTED
        data = self.w.vocab[tok]
        if not data:
            return ERR_TOKEN_REJECTED
        return FMT_OK if self.seqs[b].advance(data) else ERR_TOKEN_REJECTED

    def mask(self, b: int) -> np.ndarray:
        words = (self.w.V + 31) // 32
        if self.finished[b]:
            m = np.zeros(words, dtype=np.uint32)
            m[self.w.eos >> 5] = np.uint32(1 << (self.w.eos & 31))
            return m
        return self.seqs[b].mask(self.vocab)


def describe_diff(w, got: np.ndarray, want: np.ndarray, limit: int = 8) -> str:
    g, e = oracle.bits(got, w.V), oracle.bits(want, w.V)
    bad = np.nonzero(g != e)[0]
    parts = ["%d differing tokens" % len(bad)]
    for t in bad[:limit]:
        parts.append("tok %d %r gpu=%d oracle=%d" % (t, w.vocab[t], g[t], e[t]))
    return "; ".join(parts)
