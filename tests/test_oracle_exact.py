"""Pins for oracle/exact.py against what the paper prints and proves (CPU only)."""
import itertools
import os
from fractions import Fraction as F

import numpy as np
import pytest

from oracle import exact
from helpers import random_tree, read_golden, all_blocks

GOLD = read_golden(os.path.join(os.path.dirname(__file__), "golden", "toy_example.txt"))


def toy_models():
    tgt = [F(x) for x in GOLD["target"]]
    drf = [F(x) for x in GOLD["draft"]]
    return (lambda pre: tgt), (lambda pre: drf), int(GOLD["gamma"][0])


def test_toy_expected_accepted_lengths():
    # Section "A Motivating Example": 10/9 for token verification, 11/9 for block verification
    P, Q, g = toy_models()
    assert exact.expected_tau(P, Q, 2, g, "token") == F(GOLD["E_tau_token"][0])
    assert exact.expected_tau(P, Q, 2, g, "block") == F(GOLD["E_tau_block"][0])
    assert F(GOLD["E_tau_block"][0]) < F(GOLD["E_tau_ideal"][0])


def test_toy_token_acceptance():
    P, Q, g = toy_models()
    assert exact.token_quantities(P, Q, (0, 0))[1] == F(GOLD["tv_accept_a"][0])
    assert exact.token_quantities(P, Q, (1, 1))[1] == F(GOLD["tv_accept_b"][0])


@pytest.mark.parametrize("name", ["aa", "ab", "ba", "bb"])
def test_toy_block_behaviour(name):
    # per-block acceptance behaviour described in the paragraph
    # "Verification with partial information"
    P, Q, g = toy_models()
    blk = tuple("ab".index(c) for c in name)
    row = GOLD["bv"][name]
    p, S, h = exact.block_quantities(P, Q, blk)
    law = exact.tau_law_block(h)
    assert law[2] == F(row[0]) and law[1] == F(row[1]) and law[0] == F(row[2])
    if row[3] != "-":
        y = "ab".index(row[3])
        for i in range(g):
            if law[i] != 0:
                res = exact.residual(P, Q, blk, i, p[i])
                assert res[y] == 1


def test_toy_ideal_is_joint_min():
    # the "ideal algorithm with full information": 2 * sum_x min(M_b(x^2), M_s(x^2)) = 12/9
    P, Q, g = toy_models()
    tot = sum(min(exact.joint(P, b), exact.joint(Q, b)) for b in all_blocks(2, 2))
    assert 2 * tot == F(GOLD["E_tau_ideal"][0])


@pytest.mark.parametrize("algo", ["block", "token"])
@pytest.mark.parametrize("V,gamma,seed", [(2, 3, 0), (3, 2, 1), (3, 3, 2), (4, 2, 3)])
def test_lossless_exact_rationals(algo, V, gamma, seed):
    # Theorem 1 via Lemma 2 / Eq. "output_block_distribution":
    # Pr(O^l = x^l) = M_b^l(x^l) for every l <= gamma+1, with exact arithmetic
    rng = np.random.default_rng(seed)
    P = random_tree(rng, V, gamma, exact=True, zero_prob=0.15)
    Q = random_tree(rng, V, gamma, exact=True)
    for ell in range(1, gamma + 2):
        law = exact.output_law(P, Q, V, gamma, algo, ell)
        for seq in itertools.product(range(V), repeat=ell):
            assert law.get(seq, 0) == exact.joint(P, seq), (ell, seq)


@pytest.mark.parametrize("V,gamma,seed", [(8, 2, 5), (5, 3, 6), (8, 3, 7)])
def test_lossless_float_trees(V, gamma, seed):
    rng = np.random.default_rng(seed)
    P = random_tree(rng, V, gamma)
    Q = random_tree(rng, V, gamma)
    for ell in (1, 2, gamma + 1) if V < 8 or gamma < 3 else (1, 2):
        law = exact.output_law(P, Q, V, gamma, "block", ell)
        for seq in itertools.product(range(V), repeat=ell):
            assert abs(law.get(seq, 0.0) - exact.joint(P, seq)) < 1e-12


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_lemma3_prefix_keep_probability(seed):
    # Lemma 3: Pr(tau >= i | X^i = x^i) = p_i(x^i); and Pr(tau = i | X^i) = S_i
    rng = np.random.default_rng(seed)
    V, g = 3, 3
    P = random_tree(rng, V, g, exact=True)
    Q = random_tree(rng, V, g, exact=True)
    for i in range(g + 1):
        for pre in itertools.product(range(V), repeat=i):
            blk = pre + (0,) * (g - i)
            p, S, _ = exact.block_quantities(P, Q, blk)
            ge = exact.prob_tau_ge(P, Q, V, g, "block", pre)
            assert ge == p[i]
            if i < g:
                # Pr(tau = i | X^i) = p_i - sum_x Q(x) p_{i+1}(x^i, x) = S_i
                nxt = sum(Q(pre)[x] * exact.block_quantities(P, Q, (pre + (x,) + (0,) * g)[:g])[0][i + 1]
                          for x in range(V))
                assert p[i] - nxt == S[i]


@pytest.mark.parametrize("seed", range(6))
def test_theorem2_block_never_below_token(seed):
    rng = np.random.default_rng(100 + seed)
    V, g = 3, 3
    P = random_tree(rng, V, g, exact=True)
    Q = random_tree(rng, V, g, exact=True)
    eb = exact.expected_tau(P, Q, V, g, "block")
    et = exact.expected_tau(P, Q, V, g, "token")
    assert eb >= et
    # E_BV[tau] = sum_i sum_{x^i} M_s(x^i) p_i(x^i)   (Lemma 3 summed over prefixes)
    tot = 0
    for i in range(1, g + 1):
        for pre in itertools.product(range(V), repeat=i):
            blk = pre + (0,) * (g - i)
            tot += exact.joint(Q, pre) * exact.block_quantities(P, Q, blk)[0][i]
    assert tot == eb


def test_token_closed_form_context_free():
    # E_TV[tau] = sum_{k=1..gamma} (1 - d_TV)^k for context-independent models
    rng = np.random.default_rng(9)
    V, g = 4, 3
    P = random_tree(rng, V, 0, exact=True)
    Q = random_tree(rng, V, 0, exact=True)
    Pc, Qc = (lambda pre: P(())), (lambda pre: Q(()))
    dtv = sum(abs(a - b) for a, b in zip(P(()), Q(()))) / 2
    assert exact.expected_tau(Pc, Qc, V, g, "token") == sum((1 - dtv) ** k for k in range(1, g + 1))


def test_gamma1_laws_coincide():
    rng = np.random.default_rng(11)
    V = 4
    P = random_tree(rng, V, 1, exact=True)
    Q = random_tree(rng, V, 1, exact=True)
    assert exact.verify_law(P, Q, V, 1, "block") == exact.verify_law(P, Q, V, 1, "token")
