"""TEST INFRASTRUCTURE -- not part of the product path.

Exact laws of Token Verification (Algorithm 1), Block Verification
(Algorithm 2) and Greedy Block Verification (Algorithm 4, with the distribution
modification of Algorithm 5) of arXiv 2403.10444 on tiny vocabularies, with the algorithm's
own randomness (eta_1..eta_gamma and the draw of Y) integrated out
analytically.  Works in any exact or floating number type: pass probabilities
as ``fractions.Fraction`` for exact rational results.

A model is a callable ``M(prefix: tuple[int, ...]) -> sequence of probabilities``
(one per token), so context-dependent models are allowed.  ``P`` is the target
model M_b and ``Q`` the draft model M_s.

This module is independent of ``verify_oracle.c``: the tests use it (a) to
check itself against what the paper proves -- Theorem 1 / Eq.
"output_block_distribution", Lemma 3, Theorem 2 and the worked two-token
example -- and (b) to pin the C oracle's intermediates and its use of the
uniforms.
"""
from __future__ import annotations

import itertools
from typing import Callable, Dict, List, Sequence, Tuple

Model = Callable[[Tuple[int, ...]], Sequence]


def joint(M: Model, seq: Tuple[int, ...], prefix: Tuple[int, ...] = ()):
    """M^l(seq | prefix) = prod_i M(seq_i | prefix, seq^{i-1})."""
    pr = 1
    for i, x in enumerate(seq):
        pr = pr * M(prefix + seq[:i])[x]
    return pr


def block_quantities(P: Model, Q: Model, block: Tuple[int, ...]):
    """p_i (Eq. "def_as"), S_i and h_i (Eq. "pacc_block") for one drafted block.

    Returns (p[0..gamma], S[0..gamma-1], h[0..gamma]) with h[0] = 1.
    """
    g = len(block)
    p = [1]
    for i in range(1, g + 1):
        ctx = block[: i - 1]
        x = block[i - 1]
        v = p[i - 1] * P(ctx)[x] / Q(ctx)[x]
        p.append(v if v < 1 else 1)
    S = []
    for i in range(g):
        Pi, Qi = P(block[:i]), Q(block[:i])
        S.append(sum(max(p[i] * a - b, 0) for a, b in zip(Pi, Qi)))
    h = [1]
    for i in range(1, g):
        h.append(S[i] / (S[i] + 1 - p[i]) if S[i] > 0 else 0)
    h.append(p[g])
    return p, S, h


def greedy_quantities(P: Model, Q: Model, block: Tuple[int, ...]):
    """Algorithm 4 for one drafted block: the unclipped products
    pt_i = pt_{i-1} M_b(X_i|.)/M_s(X_i|.), the two sums of its step "Set h_i"
    (num_i = sum_x max(pt_i M_b - M_s, 0), den_i = sum_x max(M_s - pt_i M_b, 0)) and the
    probabilities min(h_i, 1) with which position i passes its test (h_gamma = pt_gamma;
    0 when num_i = 0, the reading taken for an empty residual).

    Returns (pt[0..gamma], num[0..gamma-1], den[0..gamma-1], a[0..gamma]) with a[0] = 1.
    """
    g = len(block)
    pt = [1]
    for i in range(1, g + 1):
        ctx = block[: i - 1]
        x = block[i - 1]
        pt.append(pt[i - 1] * P(ctx)[x] / Q(ctx)[x])
    num, den = [], []
    for i in range(g):
        Pi, Qi = P(block[:i]), Q(block[:i])
        num.append(sum(max(pt[i] * a - b, 0) for a, b in zip(Pi, Qi)))
        den.append(sum(max(b - pt[i] * a, 0) for a, b in zip(Pi, Qi)))
    acc = [1]
    for i in range(1, g):
        if num[i] == 0:
            acc.append(0)
        elif den[i] == 0 or num[i] >= den[i]:
            acc.append(1)
        else:
            acc.append(num[i] / den[i])
    acc.append(pt[g] if pt[g] < 1 else 1)
    return pt, num, den, acc


def token_quantities(P: Model, Q: Model, block: Tuple[int, ...]):
    """h_i^token = min(M_b(X_i|.)/M_s(X_i|.), 1) (Eq. "accept_probability"), h[0] = 1."""
    h = [1]
    for i in range(1, len(block) + 1):
        ctx = block[: i - 1]
        x = block[i - 1]
        r = P(ctx)[x] / Q(ctx)[x]
        h.append(r if r < 1 else 1)
    return h


def tau_law_block(h: Sequence) -> List:
    """Pr(tau = i | block), i = 0..gamma, for tau = max{i : eta_i <= h_i} (0 if none)."""
    g = len(h) - 1
    law = []
    for i in range(g + 1):
        pr = h[i]
        for j in range(i + 1, g + 1):
            pr = pr * (1 - h[j])
        law.append(pr)
    return law


def tau_law_token(h: Sequence) -> List:
    """Pr(tau = i | block) when tau is the length of the initial run of acceptances."""
    g = len(h) - 1
    law, run = [], 1
    for i in range(g + 1):
        if i > 0:
            run = run * h[i]
        law.append(run * (1 - h[i + 1]) if i < g else run)
    return law


def residual(P: Model, Q: Model, block: Tuple[int, ...], i: int, p_i) -> List:
    """Distribution of Y given tau = i: Eq. "pres-block" (p_i = 1: Eq. "pres-token");
    at i = gamma it is the target distribution M_b(. | c, X^gamma)."""
    g = len(block)
    Pi = P(block[:i])
    if i == g:
        return list(Pi)
    Qi = Q(block[:i])
    w = [max(p_i * a - b, 0) for a, b in zip(Pi, Qi)]
    tot = sum(w)
    if tot == 0:
        return [0 for _ in w]
    return [x / tot for x in w]


def _blocks(V: int, g: int):
    return itertools.product(range(V), repeat=g)


def verify_law(P: Model, Q: Model, V: int, gamma: int, algo: str):
    """Joint law of (block, tau, Y): dict {(block, tau, y): probability}."""
    out: Dict[Tuple[Tuple[int, ...], int, int], object] = {}
    for block in _blocks(V, gamma):
        qb = joint(Q, block)
        if qb == 0:
            continue
        if algo == "block":
            p, _, h = block_quantities(P, Q, block)
            tl = tau_law_block(h)
        elif algo == "greedy":
            # tau = the last position whose test passes, as in Algorithm 2; the residual of
            # Eq. "pres_greedy" is Eq. "pres-block" with the unclipped product
            p, _, _, acc = greedy_quantities(P, Q, block)
            tl = tau_law_block(acc)
        else:
            h = token_quantities(P, Q, block)
            tl = tau_law_token(h)
            p = [1] * (gamma + 1)
        for i, pt in enumerate(tl):
            if pt == 0:
                continue
            for y, py in enumerate(residual(P, Q, block, i, p[i])):
                if py != 0:
                    out[(block, i, y)] = qb * pt * py
    return out


def output_law(P: Model, Q: Model, V: int, gamma: int, algo: str, ell: int):
    """Law of O^ell where O = (X^tau, Y, Z^{gamma-tau}), Z ~ M_b^{gamma-tau}(. | c, X^tau, Y)
    (Lemma 2, Eq. "verify_goal"); ell <= gamma + 1."""
    law: Dict[Tuple[int, ...], object] = {}
    for (block, i, y), pr in verify_law(P, Q, V, gamma, algo).items():
        head = block[:i] + (y,)
        if len(head) >= ell:
            key = head[:ell]
            law[key] = law.get(key, 0) + pr
        else:
            for z in _blocks(V, ell - len(head)):
                pz = joint(P, z, head)
                if pz != 0:
                    key = head + z
                    law[key] = law.get(key, 0) + pr * pz
    return law


def modified_model(P: Model, Q: Model, head: Tuple[int, ...], n_mod: int) -> Model:
    """Algorithm 5 (distribution modification) after Algorithm 4 returned ``head`` = (X^tau, Y):
    for the next n_mod = gamma - tau - 1 positions the next-token law is proportional to
    max(M_b(c, head, x^i) - M_s(c, head, x^i), 0) in the JOINT probabilities (Eq. "model_new");
    after that it is M_b again.  Returns a model over continuations of ``head``."""

    def M(pre: Tuple[int, ...]):
        if len(pre) >= n_mod:
            return P(head + pre)
        seq = head + pre
        Pn, Qn = P(seq), Q(seq)
        jp, jq = joint(P, seq), joint(Q, seq)
        w = [max(jp * a - jq * b, 0) for a, b in zip(Pn, Qn)]
        tot = sum(w)
        if tot == 0:  # a prefix the modified model itself cannot produce
            return [0 for _ in w]
        return [x / tot for x in w]

    return M


def output_law_greedy(P: Model, Q: Model, V: int, gamma: int, ell: int, modify: bool = True):
    """Law of the first ell <= gamma tokens of (X^tau, Y, Z) for Algorithm 4, where Z follows the
    modified model of Algorithm 5 (modify=True; Lemma "greedy_block_identical" says the result is
    M_b^ell) or plain M_b (modify=False; the paper shows this breaks the guarantee)."""
    law: Dict[Tuple[int, ...], object] = {}
    for (block, i, y), pr in verify_law(P, Q, V, gamma, "greedy").items():
        head = block[:i] + (y,)
        if len(head) >= ell:
            key = head[:ell]
            law[key] = law.get(key, 0) + pr
            continue
        M = modified_model(P, Q, head, gamma - i - 1) if modify else (lambda pre: P(head + pre))
        for z in _blocks(V, ell - len(head)):
            pz = joint(M, z)
            if pz != 0:
                key = head + z
                law[key] = law.get(key, 0) + pr * pz
    return law


def expected_tau(P: Model, Q: Model, V: int, gamma: int, algo: str):
    """E[tau]: expected number of accepted draft tokens in one iteration."""
    return sum(pr * i for (_, i, _), pr in verify_law(P, Q, V, gamma, algo).items())


def prob_tau_ge(P: Model, Q: Model, V: int, gamma: int, algo: str, prefix: Tuple[int, ...]):
    """Pr(tau >= len(prefix) | X^i = prefix)."""
    i = len(prefix)
    num = den = 0
    for (block, t, _), pr in verify_law(P, Q, V, gamma, algo).items():
        if block[:i] == prefix:
            den = den + pr
            if t >= i:
                num = num + pr
    return num / den
