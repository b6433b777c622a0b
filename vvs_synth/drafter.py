"""Synthetic stand-in for the drafter of the decoding loop (inputs only, no arithmetic of the method).

The paper's drafter (an EAGLE-2 style model with trained weights) is not available; the loop tests
and the loop benchmark need something that proposes, per iteration, K drafted tokens with their
distributions and a small candidate tree given as token paths.  Everything here is a pure function
of (seed, iteration): it never looks at the target model, so the oracle loop and the library loop
can be fed the same proposals."""
from __future__ import annotations

import numpy as np

from . import gen


class SyntheticDrafter:
    """propose(it) -> dict(drafts int32 [K] codebook indices, q float32 [K, V], paths int32
    [n_paths, depth] codebook indices (path 0 starts with the drafts; the others share a stem of
    random length with it and continue with random codes), path_len int32 [n_paths], u_select in
    (0, 1)).  `n_sets` draft sets are drawn once and cycled (the distributions are large)."""

    def __init__(self, seed: int, vocab: int, k: int, n_paths: int = 12, depth: int = 5, n_sets: int = 16,
                 logit_std: float = 1.0, ragged: bool = False):
        self.seed, self.vocab, self.k, self.n_paths, self.depth, self.n_sets = seed, vocab, k, n_paths, depth, n_sets
        self.ragged = ragged
        self.q, self.d = gen.independent_draft(seed, 0, n_sets, k, vocab, logit_std)

    def first_token(self) -> int:
        return int(gen.rng_for(self.seed, "loop.first").integers(0, self.vocab))

    def propose(self, it: int) -> dict:
        g = gen.rng_for(self.seed, f"loop.it.{it}")
        s = it % self.n_sets
        drafts = self.d[s].astype(np.int32)
        depth = self.depth
        stem = int(g.integers(1, depth + 1))
        head = np.resize(drafts, depth).astype(np.int32)
        paths = np.tile(head[None, :], (self.n_paths, 1)).astype(np.int32)
        noise = g.integers(0, self.vocab, size=(self.n_paths, depth))
        paths[1:, stem:] = noise[1:, stem:]
        path_len = np.full(self.n_paths, depth, np.int32)
        if self.ragged:
            path_len = g.integers(1, depth + 1, size=self.n_paths).astype(np.int32)
        u = float((np.floor(g.random() * (1 << 24)) + 0.5) / (1 << 24))
        return dict(drafts=drafts, q=self.q[s], paths=paths, path_len=path_len, u_select=u)
