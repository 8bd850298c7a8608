"""Pins of the oracle's probability-domain procedures (oracle_verify_probs), CPU only.

What fixes them, other than themselves: the exact laws of ``oracle/exact.py`` in rationals
(Eq. "def_as", "pacc_block", the law of tau, the residual distributions), the paper's two-token
worked example (10/9 and 11/9 accepted tokens), Theorem 1 by enumeration over every drafted block
and a grid of uniforms, explicit cumulative sums for the sampler, and the logit-domain procedures
(pinned on their own) on inputs whose softmax is the given distribution.
"""
import itertools
from fractions import Fraction as F

import numpy as np
import pytest

import oracle
from oracle import exact
from helpers import random_tree, all_blocks, path_logits

ALGOS = {"block": oracle.BLOCK_VERIFY, "token": oracle.TOKEN_VERIFY}


def path_probs(P, Q, blocks, gamma, V):
    tgt = np.empty((len(blocks), gamma + 1, V))
    drf = np.empty((len(blocks), gamma, V))
    for b, blk in enumerate(blocks):
        for r in range(gamma + 1):
            tgt[b, r] = [float(x) for x in P(blk[:r])]
            if r < gamma:
                drf[b, r] = [float(x) for x in Q(blk[:r])]
    return tgt, drf


def toy():
    # the two-token example of the paper's introduction: M_b = (1/3, 2/3), M_s = (2/3, 1/3), context-free
    return (lambda pre: [F(1, 3), F(2, 3)]), (lambda pre: [F(2, 3), F(1, 3)])


@pytest.mark.parametrize("V,gamma,seed", [(3, 2, 0), (4, 3, 1), (5, 4, 2)])
def test_intermediates_equal_the_exact_rationals(V, gamma, seed):
    rng = np.random.default_rng(seed)
    P = random_tree(rng, V, gamma, exact=True)
    Q = random_tree(rng, V, gamma, exact=True)
    blocks = all_blocks(V, gamma)
    tgt, drf = path_probs(P, Q, blocks, gamma, V)
    tok = np.array(blocks, dtype=np.int32)
    uni = rng.random((len(blocks), gamma + 2)).astype(np.float32)
    rb = oracle.verify_probs(oracle.BLOCK_VERIFY, tgt, drf, tok, uni)
    rt = oracle.verify_probs(oracle.TOKEN_VERIFY, tgt, drf, tok, uni)
    for b, blk in enumerate(blocks):
        p, S, h = exact.block_quantities(P, Q, blk)
        assert np.allclose(rb.p[b], [float(x) for x in p], rtol=1e-13, atol=0)
        assert np.allclose(rb.S[b], [float(x) for x in S], rtol=1e-12, atol=1e-15)
        assert np.allclose(rb.h[b], [float(x) for x in h], rtol=1e-12, atol=1e-15)
        # tau from the definition, with the oracle's own uniforms
        eta = uni[b].astype(np.float64)
        tau = max([i for i in range(1, gamma + 1) if float(h[i]) > 0 and eta[i - 1] <= float(h[i])], default=0)
        if min(abs(eta[i - 1] - float(h[i])) for i in range(1, gamma + 1)) > 1e-9:
            assert rb.out_len[b] == tau + 1
        ht = exact.token_quantities(P, Q, blk)
        tt = 0
        for i in range(1, gamma + 1):
            if float(ht[i]) > 0 and eta[i - 1] <= float(ht[i]):
                tt = i
            else:
                break
        if min(abs(eta[i - 1] - float(ht[i])) for i in range(1, gamma + 1)) > 1e-9:
            assert rt.out_len[b] == tt + 1
            made = min(tt + 1, gamma)
            assert np.allclose(rt.h[b, 1 : made + 1], [float(x) for x in ht[1 : made + 1]], rtol=1e-13)


@pytest.mark.parametrize("algo", ["block", "token"])
def test_sampled_token_follows_the_explicit_cumulative_sums(algo):
    rng = np.random.default_rng(7)
    V, gamma = 6, 3
    P = random_tree(rng, V, gamma)
    Q = random_tree(rng, V, gamma)
    blocks = all_blocks(V, gamma)
    tgt, drf = path_probs(P, Q, blocks, gamma, V)
    tok = np.array(blocks, dtype=np.int32)
    uni = rng.random((len(blocks), gamma + 2)).astype(np.float32)
    r = oracle.verify_probs(ALGOS[algo], tgt, drf, tok, uni)
    for b, blk in enumerate(blocks):
        tau = int(r.out_len[b]) - 1
        p_tau = 1.0 if algo == "token" else float(exact.block_quantities(P, Q, blk)[0][tau])
        if tau == gamma:
            w = tgt[b, gamma]
            u = float(uni[b, gamma + 1])
        else:
            w = np.maximum(p_tau * tgt[b, tau] - drf[b, tau], 0.0)
            u = float(uni[b, gamma])
        c = np.cumsum(w)
        if r.margin_smp[b] > 1e-9:
            assert r.out_tokens[b, tau] == int(np.searchsorted(c, u * c[-1], side="right"))
        assert list(r.out_tokens[b, :tau]) == list(blk[:tau])
        assert (r.out_tokens[b, tau + 1 :] == -1).all()


def test_worked_example_accepted_lengths():
    # 10/9 accepted tokens under Algorithm 1 and 11/9 under Algorithm 2 with two drafted tokens: the mean
    # of tau over the drafted blocks (weights M_s^2) and a fine midpoint grid of the two uniforms
    P, Q = toy()
    V, gamma, n = 2, 2, 180
    grid = (np.arange(n) + 0.5) / n
    blocks = all_blocks(V, gamma)
    for algo, want in (("token", F(10, 9)), ("block", F(11, 9))):
        mean = 0.0
        for blk in blocks:
            e1, e2 = np.meshgrid(grid, grid, indexing="ij")
            uni = np.stack([e1.ravel(), e2.ravel(), np.full(n * n, 0.5), np.full(n * n, 0.5)], 1).astype(np.float32)
            tgt, drf = path_probs(P, Q, [blk] * (n * n), gamma, V)
            r = oracle.verify_probs(ALGOS[algo], tgt, drf, np.array([blk] * (n * n), np.int32), uni)
            mean += float(exact.joint(Q, blk)) * float((r.out_len - 1).mean())
        # (the acceptance weights of this example are multiples of 1/4 and 1/5... of the grid step: exact)
        assert abs(mean - float(want)) < 1e-3


@pytest.mark.parametrize("algo", ["block", "token"])
def test_output_law_is_the_target_law(algo):
    # Theorem 1 on a tiny context-dependent pair of models: the law of the first emitted token, with the
    # uniforms on a midpoint grid, against M_b(. | c)
    rng = np.random.default_rng(11)
    V, gamma, n = 3, 2, 24
    P = random_tree(rng, V, gamma, exact=True)
    Q = random_tree(rng, V, gamma, exact=True)
    grid = (np.arange(n) + 0.5) / n
    e = np.stack([x.ravel() for x in np.meshgrid(grid, grid, grid, indexing="ij")], 1)
    law = np.zeros(V)
    for blk in all_blocks(V, gamma):
        uni = np.concatenate([e, e[:, 2:3]], 1).astype(np.float32)    # one grid serves both sampling uniforms
        tgt, drf = path_probs(P, Q, [blk] * len(e), gamma, V)
        r = oracle.verify_probs(ALGOS[algo], tgt, drf, np.array([blk] * len(e), np.int32), uni)
        first = r.out_tokens[:, 0]
        for x in range(V):
            law[x] += float(exact.joint(Q, blk)) * float((first == x).mean())
    assert np.allclose(law, [float(x) for x in P(())], atol=2.5 / n)


@pytest.mark.parametrize("algo", ["block", "token"])
def test_agrees_with_the_logit_procedures_on_log_probabilities(algo):
    rng = np.random.default_rng(3)
    V, gamma = 7, 4
    P = random_tree(rng, V, gamma)
    Q = random_tree(rng, V, gamma)
    blocks = [tuple(rng.integers(0, V, gamma)) for _ in range(200)]
    tgt, drf = path_probs(P, Q, blocks, gamma, V)
    ltgt, ldrf = path_logits(P, Q, blocks, gamma, V)
    tok = np.array(blocks, dtype=np.int32)
    uni = rng.random((len(blocks), gamma + 2)).astype(np.float32)
    a = oracle.verify_probs(ALGOS[algo], tgt, drf, tok, uni)
    b = oracle.verify(ALGOS[algo], ltgt, ldrf, tok, uni, 1.0)
    safe = (np.minimum(b.margin_eta, b.margin_smp) > 1e-9)
    assert safe.sum() > 150
    assert np.array_equal(a.out_len[safe], b.out_len[safe])
    assert np.array_equal(a.out_tokens[safe], b.out_tokens[safe])
    if algo == "block":
        assert np.allclose(a.p, b.p, rtol=1e-12) and np.allclose(a.S, b.S, rtol=1e-10, atol=1e-14)
        assert np.allclose(a.h, b.h, rtol=1e-10, atol=1e-14)


def test_rows_are_used_as_stored_and_faults_are_per_sequence():
    V, gamma = 4, 2
    tgt = np.full((3, gamma + 1, V), 0.25)
    drf = np.full((3, gamma, V), 0.25)
    tok = np.zeros((3, gamma), np.int32)
    uni = np.full((3, gamma + 2), 0.5, np.float32)
    drf[1, 0, 0] = 0.0            # a token the draft model cannot have produced
    tok[2, 1] = V                 # a token outside the vocabulary
    tgt[0] *= 0.5                 # rows that do not sum to one are not renormalised: ratio 1/2 at both tests
    for algo in ALGOS.values():
        r = oracle.verify_probs(algo, tgt, drf, tok, uni)
        assert r.out_len[1] == -1 and r.out_len[2] == -1 and (r.out_tokens[1:] == -1).all()
    r = oracle.verify_probs(oracle.BLOCK_VERIFY, tgt, drf, tok, uni)
    assert np.allclose(r.p[0], [1.0, 0.5, 0.25])
    # S_1 = sum max(0.5 * 0.125 - 0.25, 0) = 0: h_1 = 0, h_2 = p_2 = 0.25 < 0.5: tau = 0, residual max(0.125 - 0.25, 0) empty
    assert r.out_len[0] == -1
    r = oracle.verify_probs(oracle.TOKEN_VERIFY, tgt, drf, tok, np.full((3, gamma + 2), 0.4, np.float32))
    # both tests pass (0.4 <= 1/2): tau = 2, and Y from P_2 = (1/8, 1/8, 1/8, 1/8) divided by its own sum: 0.4 falls in cell 1
    assert r.out_len[0] == 3 and list(r.out_tokens[0]) == [0, 0, 1]


def test_bf16_and_f32_storage_are_widened_exactly():
    rng = np.random.default_rng(5)
    V, gamma, B = 16, 3, 32
    t = rng.dirichlet(np.ones(V), (B, gamma + 1)).astype(np.float32)
    d = rng.dirichlet(np.ones(V), (B, gamma)).astype(np.float32)
    tb = (t.view(np.uint32) >> 16).astype(np.uint16)      # truncated to bf16 bit patterns
    db = (d.view(np.uint32) >> 16).astype(np.uint16)
    tok = rng.integers(0, V, (B, gamma)).astype(np.int32)
    uni = rng.random((B, gamma + 2)).astype(np.float32)
    wide_t = (tb.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    wide_d = (db.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    for algo in ALGOS.values():
        a = oracle.verify_probs(algo, tb, db, tok, uni)
        b = oracle.verify_probs(algo, wide_t, wide_d, tok, uni)
        assert np.array_equal(a.out_tokens, b.out_tokens) and np.array_equal(a.out_len, b.out_len)
        c = oracle.verify_probs(algo, t, d, tok, uni)
        e = oracle.verify_probs(algo, t.astype(np.float64), d.astype(np.float64), tok, uni)
        assert np.array_equal(c.out_tokens, e.out_tokens) and np.array_equal(c.out_len, e.out_len)
