"""Shared helpers for the tests: tiny context-dependent models and sample-path logits.
Holds none of the verification arithmetic."""
from __future__ import annotations

import itertools
from fractions import Fraction

import numpy as np


class TreeModel:
    """A context-dependent model on a tiny vocabulary: one distribution per prefix."""

    def __init__(self, table):
        self.table = table

    def __call__(self, prefix):
        return self.table[tuple(prefix)]


def random_tree(rng, V, depth, exact=False, zero_prob=0.0, denom=12):
    """Random distributions for every prefix of length 0..depth.

    exact=True draws rationals with small denominators (as Fractions); otherwise
    float64 Dirichlet-like vectors.  zero_prob > 0 plants exact zeros.
    """
    table = {}
    for L in range(depth + 1):
        for pre in itertools.product(range(V), repeat=L):
            if exact:
                w = [int(rng.integers(1, denom)) for _ in range(V)]
                if zero_prob > 0:
                    w = [0 if rng.random() < zero_prob else x for x in w]
                    if sum(w) == 0:
                        w[0] = 1
                tot = sum(w)
                table[pre] = [Fraction(x, tot) for x in w]
            else:
                w = rng.gamma(0.7, size=V) + 1e-3
                table[pre] = list(w / w.sum())
    return TreeModel(table)


def path_logits(P, Q, blocks, gamma, V):
    """Log-probability rows along each block's sample path, as float64 arrays
    target [B, gamma+1, V] and draft [B, gamma, V] (log 0 = -inf)."""
    B = len(blocks)
    tgt = np.empty((B, gamma + 1, V))
    drf = np.empty((B, gamma, V))
    with np.errstate(divide="ignore"):
        for b, blk in enumerate(blocks):
            for r in range(gamma + 1):
                tgt[b, r] = np.log(np.array([float(x) for x in P(blk[:r])]))
                if r < gamma:
                    drf[b, r] = np.log(np.array([float(x) for x in Q(blk[:r])]))
    return tgt, drf


def all_blocks(V, gamma):
    return list(itertools.product(range(V), repeat=gamma))


def read_golden(path):
    """Parse tests/golden/toy_example.txt into a dict of tokens per key."""
    out = {"bv": {}, "gv": {}}
    with open(path) as f:
        for line in f:
            line = line.split("#")[0].split()
            if not line:
                continue
            if line[0] in ("bv", "gv"):
                out[line[0]][line[1]] = line[2:]
            else:
                out[line[0]] = line[1:]
    return out
