"""Pins for the C oracle (oracle/verify_oracle.c): CPU only.

The oracle is pinned to things other than itself: the paper's worked example,
brute-force enumeration over every drafted block and a grid of uniforms (the
lossless guarantee), the exact laws of oracle/exact.py (themselves pinned to
the paper's theorems), scipy's logsumexp, and explicit cumulative sums.
"""
import itertools
import os
from fractions import Fraction as F

import numpy as np
import pytest
from scipy.special import logsumexp
from scipy.stats import chi2

import oracle
from oracle import exact
from helpers import random_tree, path_logits, all_blocks, read_golden

GOLD = read_golden(os.path.join(os.path.dirname(__file__), "golden", "toy_example.txt"))


def midgrid(n):
    return ((np.arange(n) + 0.5) / n).astype(np.float32)


def run_grid(P, Q, V, gamma, algo, n_eta, n_u):
    """Every block x every eta on an n_eta^gamma mid-point grid x every sampling
    uniform on an n_u mid-point grid.  Returns (blocks, result, shape)."""
    blocks = all_blocks(V, gamma)
    tgt1, drf1 = path_logits(P, Q, blocks, gamma, V)
    etas = np.array(list(itertools.product(midgrid(n_eta), repeat=gamma)), np.float32)
    us = midgrid(n_u)
    nE, nU, nB = len(etas), len(us), len(blocks)
    uni = np.empty((nB, nE, nU, gamma + 2), np.float32)
    uni[..., :gamma] = etas[None, :, None, :]
    uni[..., gamma] = us[None, None, :]
    uni[..., gamma + 1] = us[None, None, :]
    rep = nE * nU
    tgt = np.repeat(tgt1, rep, axis=0)
    drf = np.repeat(drf1, rep, axis=0)
    tok = np.repeat(np.array(blocks, np.int32), rep, axis=0)
    res = oracle.verify(algo, tgt, drf, tok, uni.reshape(-1, gamma + 2))
    return blocks, res, (nB, nE, nU)


def toy():
    tgt = [F(x) for x in GOLD["target"]]
    drf = [F(x) for x in GOLD["draft"]]
    return (lambda pre: tgt), (lambda pre: drf)


@pytest.mark.parametrize("algo,key", [(oracle.BLOCK_VERIFY, "E_tau_block"),
                                      (oracle.TOKEN_VERIFY, "E_tau_token")])
def test_toy_example_through_uniform_grid(algo, key):
    # all thresholds of the toy example are multiples of 1/4, so a mid-point grid
    # with n divisible by 4 integrates the uniforms exactly
    P, Q = toy()
    n = 8
    blocks, res, (nB, nE, nU) = run_grid(P, Q, 2, 2, algo, n, 6)
    tau = (res.out_len - 1).reshape(nB, nE, nU)
    qb = np.array([float(exact.joint(Q, b)) for b in blocks])
    e_tau = float((tau.mean(axis=(1, 2)) * qb).sum())
    assert abs(e_tau - float(F(GOLD[key][0]))) < 1e-12
    # marginals of the first two output tokens equal the target model's
    # (O_2 is the continuation Z ~ M_b when tau = 0, integrated analytically)
    out = res.out_tokens.reshape(nB, nE, nU, 3)
    law1 = np.zeros(2)
    law12 = np.zeros((2, 2))
    Pv = np.array([float(x) for x in P(())])
    for b in range(nB):
        for o1 in range(2):
            m1 = out[b, :, :, 0] == o1
            law1[o1] += qb[b] * m1.mean()
            for o2 in range(2):
                have2 = (tau[b] >= 1) & m1 & (out[b, :, :, 1] == o2)
                cont = (tau[b] == 0) & m1
                law12[o1, o2] += qb[b] * (have2.mean() + cont.mean() * Pv[o2])
    assert np.allclose(law1, Pv, atol=1e-12)
    assert np.allclose(law12, np.outer(Pv, Pv), atol=1e-12)


@pytest.mark.parametrize("seed", [0, 1, 2, 3])
def test_intermediates_match_exact_on_every_block(seed):
    rng = np.random.default_rng(seed)
    V, g = (3, 3) if seed % 2 else (8, 2)
    P = random_tree(rng, V, g)
    Q = random_tree(rng, V, g)
    blocks = all_blocks(V, g)
    tgt, drf = path_logits(P, Q, blocks, g, V)
    uni = rng.random((len(blocks), g + 2), dtype=np.float32)
    res = oracle.block_verify(tgt, drf, np.array(blocks, np.int32), uni)
    rtv = oracle.token_verify(tgt, drf, np.array(blocks, np.int32), uni)
    for b, blk in enumerate(blocks):
        p, S, h = exact.block_quantities(P, Q, blk)
        assert np.allclose(res.p[b], p, rtol=1e-12, atol=1e-15)
        assert np.allclose(res.S[b], S, rtol=1e-11, atol=1e-15)
        assert np.allclose(res.h[b], h, rtol=1e-11, atol=1e-15)
        ht = exact.token_quantities(P, Q, blk)
        k = int(rtv.out_len[b])  # tau + 1: h_1..h_{tau+1} were formed (h_{tau+1} only if tau < g)
        upto = min(k, g)
        assert np.allclose(rtv.h[b, : upto + 1], ht[: upto + 1], rtol=1e-12)


@pytest.mark.parametrize("algo,name", [(oracle.BLOCK_VERIFY, "block"), (oracle.TOKEN_VERIFY, "token")])
def test_lossless_by_brute_force_over_blocks_and_uniforms(algo, name):
    # enumerate every drafted block; the uniforms are integrated on a mid-point
    # grid, whose error per decision is at most 1/n
    rng = np.random.default_rng(42)
    V, g, n_eta, n_u = 3, 2, 48, 96
    P = random_tree(rng, V, g)
    Q = random_tree(rng, V, g)
    blocks, res, (nB, nE, nU) = run_grid(P, Q, V, g, algo, n_eta, n_u)
    tau = (res.out_len - 1).reshape(nB, nE, nU)
    Y = np.take_along_axis(res.out_tokens.reshape(nB, nE, nU, g + 1),
                           tau[..., None].astype(np.int64), axis=-1)[..., 0]
    law = exact.verify_law(P, Q, V, g, name)
    for b, blk in enumerate(blocks):
        qb = float(exact.joint(Q, blk))
        for i in range(g + 1):
            for y in range(V):
                emp = ((tau[b] == i) & (Y[b] == y)).mean()
                want = float(law.get((blk, i, y), 0.0)) / qb
                assert abs(emp - want) < (g + 1) / n_eta + 1.0 / n_u + 1e-9
    o1 = res.out_tokens.reshape(nB, nE, nU, g + 1)[..., 0]
    m = np.zeros(V)
    for b, blk in enumerate(blocks):
        for x in range(V):
            m[x] += float(exact.joint(Q, blk)) * (o1[b] == x).mean()
    assert np.allclose(m, [float(x) for x in P(())], atol=3.0 / n_eta + 1.0 / n_u)


def test_monte_carlo_output_law_matches_target():
    # chi-square of O_1 and (O_1, O_2) with blocks drawn from the draft tree
    rng = np.random.default_rng(7)
    V, g, N = 6, 3, 200_000
    P = random_tree(rng, V, g)
    Q = random_tree(rng, V, g)
    blocks = all_blocks(V, g)
    qb = np.array([float(exact.joint(Q, b)) for b in blocks])
    idx = rng.choice(len(blocks), size=N, p=qb / qb.sum())
    tgt1, drf1 = path_logits(P, Q, blocks, g, V)
    tok = np.array(blocks, np.int32)[idx]
    uni = rng.random((N, g + 2), dtype=np.float32)
    for algo in (oracle.BLOCK_VERIFY, oracle.TOKEN_VERIFY):
        res = oracle.verify(algo, tgt1[idx], drf1[idx], tok, uni)
        o1 = res.out_tokens[:, 0]
        cnt = np.bincount(o1, minlength=V).astype(float)
        expct = N * np.array([float(x) for x in P(())])
        stat = ((cnt - expct) ** 2 / expct).sum()
        assert stat < chi2.ppf(1 - 1e-6, V - 1)
        # second token: the verifier's own where it emitted two, else a fresh target draw
        o2 = res.out_tokens[:, 1].copy()
        need = res.out_len < 2
        cdfs = np.array([np.cumsum(np.array(P((a,)), float)) for a in range(V)])
        r = rng.random(int(need.sum()))
        o2[need] = [min(int(np.searchsorted(cdfs[a], x, side="right")), V - 1)
                    for a, x in zip(o1[need], r)]
        pair = np.zeros((V, V))
        np.add.at(pair, (o1, o2), 1.0)
        want = N * np.array([[float(exact.joint(P, (a, b))) for b in range(V)] for a in range(V)])
        stat2 = ((pair - want) ** 2 / want).sum()
        assert stat2 < chi2.ppf(1 - 1e-6, V * V - 1)


@pytest.mark.parametrize("dtype", [np.float64, np.float32, "bf16"])
def test_normalisers_reduce_to_scipy_logsumexp(dtype):
    rng = np.random.default_rng(3)
    B, g, V, T = 3, 2, 257, np.float32(0.8)
    t = rng.normal(0, 3, (B, g + 1, V))
    d = t[:, :g] + rng.normal(0, 1, (B, g, V))
    if dtype == "bf16":
        tb = (t.astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
        db = (d.astype(np.float32).view(np.uint32) >> 16).astype(np.uint16)
        t64 = (tb.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
        d64 = (db.astype(np.uint32) << 16).view(np.float32).astype(np.float64)
        ta, da = tb, db
    else:
        ta, da = t.astype(dtype), d.astype(dtype)
        t64, d64 = ta.astype(np.float64), da.astype(np.float64)
    tok = rng.integers(0, V, (B, g)).astype(np.int32)
    uni = rng.random((B, g + 2), dtype=np.float32)
    res = oracle.block_verify(ta, da, tok, uni, temperature=T)
    assert np.allclose(res.lse_t, logsumexp(t64 / float(T), axis=-1), rtol=0, atol=1e-12)
    assert np.allclose(res.lse_d, logsumexp(d64 / float(T), axis=-1), rtol=0, atol=1e-12)


def test_residual_mass_identity_and_bounds():
    # S_i = p_i - sum_x min(p_i P_i(x), Q_i(x)); 0 <= S_i <= p_i; p_i = 1 => S_i = d_TV
    rng = np.random.default_rng(5)
    B, g, V = 16, 4, 300
    t = rng.normal(0, 2, (B, g + 1, V))
    d = t[:, :g] + rng.normal(0, 0.7, (B, g, V))
    tok = rng.integers(0, V, (B, g)).astype(np.int32)
    uni = rng.random((B, g + 2), dtype=np.float32)
    res = oracle.block_verify(t, d, tok, uni)
    Pm = np.exp(t - logsumexp(t, axis=-1, keepdims=True))
    Qm = np.exp(d - logsumexp(d, axis=-1, keepdims=True))
    for b in range(B):
        for i in range(g):
            p = res.p[b, i]
            ident = p - np.minimum(p * Pm[b, i], Qm[b, i]).sum()
            assert abs(res.S[b, i] - ident) < 1e-12
            assert -1e-15 <= res.S[b, i] <= p + 1e-15
            if p == 1.0:
                assert abs(res.S[b, i] - 0.5 * np.abs(Pm[b, i] - Qm[b, i]).sum()) < 1e-12
        assert np.all((res.h[b] >= 0) & (res.h[b] <= 1 + 1e-15))
        q = 1.0
        for i in range(1, g + 1):
            x = tok[b, i - 1]
            q = min(q * Pm[b, i - 1, x] / Qm[b, i - 1, x], 1.0)
            assert abs(res.p[b, i] - q) < 1e-12 * max(q, 1e-300) + 1e-15
        assert res.h[b, g] == res.p[b, g]


def test_sampler_against_explicit_cumulative_sums():
    rng = np.random.default_rng(8)
    B, g, V = 400, 1, 37
    t = rng.normal(0, 2, (B, g + 1, V))
    d = t[:, :g] + rng.normal(0, 1.0, (B, g, V))
    d[:, 0, 0] = 50.0                    # drafted token 0 is certain for the draft model
    t[:, 0, 0] = -50.0                   # and the target rejects it: tau = 0 always
    tok = np.zeros((B, g), np.int32)
    uni = rng.random((B, g + 2), dtype=np.float32)
    res = oracle.block_verify(t, d, tok, uni)
    assert np.all(res.out_len == 1)
    Pm = np.exp(t - logsumexp(t, axis=-1, keepdims=True))
    Qm = np.exp(d - logsumexp(d, axis=-1, keepdims=True))
    w = np.maximum(Pm[:, 0] - Qm[:, 0], 0)
    c = np.cumsum(w, axis=-1)
    for b in range(B):
        want = int(np.searchsorted(c[b], float(uni[b, g]) * c[b, -1], side="right"))
        assert res.out_tokens[b, 0] == want
        assert w[b, want] > 0
    uni0 = uni.copy(); uni0[:, g] = 0.0
    r0 = oracle.block_verify(t, d, tok, uni0)
    assert np.all(r0.out_tokens[:, 0] == np.argmax(w > 0, axis=-1))


def test_gamma1_bit_identical_outputs():
    rng = np.random.default_rng(12)
    B, V = 500, 50
    t = rng.normal(0, 2, (B, 2, V)).astype(np.float32)
    d = (t[:, :1] + rng.normal(0, 1, (B, 1, V))).astype(np.float32)
    tok = rng.integers(0, V, (B, 1)).astype(np.int32)
    uni = rng.random((B, 3), dtype=np.float32)
    a = oracle.block_verify(t, d, tok, uni)
    c = oracle.token_verify(t, d, tok, uni)
    assert np.array_equal(a.out_tokens, c.out_tokens) and np.array_equal(a.out_len, c.out_len)


def test_draft_equals_target_accepts_everything():
    rng = np.random.default_rng(13)
    B, g, V = 20, 5, 64
    t = rng.normal(0, 2, (B, g + 1, V)).astype(np.float32)
    d = t[:, :g].copy()
    tok = rng.integers(0, V, (B, g)).astype(np.int32)
    uni = rng.random((B, g + 2), dtype=np.float32)
    for algo in (oracle.BLOCK_VERIFY, oracle.TOKEN_VERIFY):
        r = oracle.verify(algo, t, d, tok, uni)
        assert np.all(r.out_len == g + 1)
        assert np.array_equal(r.out_tokens[:, :g], tok)
    r = oracle.block_verify(t, d, tok, uni)
    assert np.all(r.S == 0) and np.all(r.p == 1) and np.all(r.h[:, 1:g] == 0)


@pytest.mark.parametrize("algo", [oracle.BLOCK_VERIFY, oracle.TOKEN_VERIFY, oracle.GREEDY_BLOCK_VERIFY])
def test_a_position_with_an_empty_residual_is_never_the_selected_one(algo):
    # Where P_i and Q_i coincide, Eqs. "pres-token" / "pres-block" have nothing to sample from (0/0).
    # The algorithms never get there: the ratio of the next drafted token is then 1, so test i + 1
    # passes whatever its uniform (Algorithm 1 does not stop at i; in Algorithms 2 and 4 p_{i+1} = p_i
    # and a later position is selected, Lemma 3).  Checked for every block and every eta on a grid,
    # with the coinciding position planted at every i, the other rows random.
    rng = np.random.default_rng(77)
    V, g, n = 4, 3, 6
    grid = midgrid(n)
    for same in range(g):
        t = rng.normal(0, 1.5, (1, g + 1, V))
        d = t[:, :g] + rng.normal(0, 1.0, (1, g, V))
        d[0, same] = t[0, same]
        blocks = all_blocks(V, g)
        etas = list(itertools.product(grid, repeat=g))
        B = len(blocks) * len(etas)
        tgt = np.repeat(t, B, axis=0).astype(np.float32)
        drf = np.repeat(d, B, axis=0).astype(np.float32)
        tok = np.repeat(np.array(blocks, np.int32), len(etas), axis=0)
        uni = np.empty((B, g + 2), np.float32)
        uni[:, :g] = np.tile(np.array(etas, np.float32), (len(blocks), 1))
        uni[:, g:] = 0.5
        r = oracle.verify(algo, tgt, drf, tok, uni)
        assert np.all(r.out_len >= 1)                  # no domain error anywhere ...
        assert not np.any(r.out_len - 1 == same)       # ... and tau is never the planted position


def test_sampling_from_nothing_is_a_domain_error():
    # The sampler itself, given weights that sum to nothing, has no token to return: the sequence
    # ends as a domain error.  Reached here through the drafting step on a row of -inf logits
    # (the verification procedures cannot reach it, see the test above).
    row = np.full((1, 8), -np.inf, np.float32)
    tok, lse, _ = oracle.sample_rows(row, np.array([0.3], np.float32), 1.0)
    assert tok[0] == -1 and np.isnan(lse[0])


def test_temperature_scales_with_logits():
    rng = np.random.default_rng(14)
    B, g, V = 30, 3, 40
    t = rng.normal(0, 2, (B, g + 1, V)).astype(np.float32)
    d = (t[:, :g] + rng.normal(0, 1, (B, g, V))).astype(np.float32)
    tok = rng.integers(0, V, (B, g)).astype(np.int32)
    uni = rng.random((B, g + 2), dtype=np.float32)
    a = oracle.block_verify(t, d, tok, uni, temperature=0.5)
    c = oracle.block_verify(t * 4, d * 4, tok, uni, temperature=2.0)  # powers of two: exact
    assert np.array_equal(a.out_tokens, c.out_tokens)
    assert np.array_equal(a.S, c.S) and np.array_equal(a.h, c.h)


def test_bf16_bits_equal_widened_floats():
    rng = np.random.default_rng(15)
    B, g, V = 10, 3, 100
    t32 = rng.normal(0, 2, (B, g + 1, V)).astype(np.float32)
    d32 = (t32[:, :g] + rng.normal(0, 1, (B, g, V))).astype(np.float32)
    tb = (t32.view(np.uint32) >> 16).astype(np.uint16)
    db = (d32.view(np.uint32) >> 16).astype(np.uint16)
    tw = (tb.astype(np.uint32) << 16).view(np.float32)
    dw = (db.astype(np.uint32) << 16).view(np.float32)
    tok = rng.integers(0, V, (B, g)).astype(np.int32)
    uni = rng.random((B, g + 2), dtype=np.float32)
    a = oracle.block_verify(tb, db, tok, uni)
    c = oracle.block_verify(tw, dw, tok, uni)
    assert np.array_equal(a.out_tokens, c.out_tokens) and np.array_equal(a.S, c.S)


def test_domain_errors_are_per_sequence():
    rng = np.random.default_rng(16)
    B, g, V = 6, 2, 16
    t = rng.normal(0, 1, (B, g + 1, V)).astype(np.float32)
    d = (t[:, :g] + rng.normal(0, 1, (B, g, V))).astype(np.float32)
    tok = rng.integers(0, V, (B, g)).astype(np.int32)
    uni = rng.random((B, g + 2), dtype=np.float32)
    t[1, 0, 3] = np.nan
    tok[2, 1] = V
    d[3, 0, tok[3, 0]] = -np.inf
    t[4, 1, :] = -np.inf
    t[5, 2, 7] = -np.inf      # legal: probability 0
    r = oracle.block_verify(t, d, tok, uni)
    assert list(r.out_len[1:5]) == [-1, -1, -1, -1]
    assert np.all(r.out_tokens[1:5] == -1)
    assert r.out_len[0] >= 1 and r.out_len[5] >= 1
    with pytest.raises(ValueError):
        oracle.block_verify(t, d, tok, uni, temperature=0.0)


# ---------------- the drafting step of Algorithm 3 (oracle_sample_rows) ----------------
def test_draft_sampler_frequencies_are_the_softmax():
    # a mid-point grid of n uniforms integrates the sampler exactly up to 1/n per token:
    # Pr(X = x) must be softmax(z / T)(x), written out here with numpy
    rng = np.random.default_rng(5)
    V, n, T = 7, 4000, 0.7
    z = rng.normal(size=V) * 2
    z[3] = -np.inf                                   # a token of probability zero
    p = np.exp(z / np.float32(T) - np.max(z / np.float32(T)))
    p /= p.sum()
    u = midgrid(n)
    tok, lse, _ = oracle.sample_rows(np.tile(z, (n, 1)), u, T)
    freq = np.bincount(tok, minlength=V) / n
    assert np.all(np.abs(freq - p) <= 1.0 / n + 1e-12)
    assert freq[3] == 0
    assert np.allclose(lse, logsumexp(z / np.float32(T)), rtol=1e-14)
    # index order: the token is non-decreasing in the uniform, u = 0 gives the first token
    assert np.all(np.diff(tok) >= 0) and tok[0] == 0


def test_draft_sampler_matches_searchsorted_and_storage_types():
    rng = np.random.default_rng(6)
    rows, V = 64, 1000
    z32 = (rng.normal(size=(rows, V)) * 3).astype(np.float32)
    u = rng.random(rows, dtype=np.float32)
    tok, lse, margin = oracle.sample_rows(z32, u, 1.0)
    for r in range(rows):
        w = np.exp(z32[r].astype(np.float64) - lse[r])
        C = np.cumsum(w)
        k = int(np.searchsorted(C, float(u[r]) * C[-1], side="right"))
        if margin[r] > 1e-12:
            assert tok[r] == min(k, V - 1)
    # bf16 bits and float64 holding the same values give the same tokens
    bits = (z32.view(np.uint32) >> 16).astype(np.uint16)
    widened = (bits.astype(np.uint32) << 16).view(np.float32)
    t16, l16, _ = oracle.sample_rows(bits, u, 1.0)
    t64, l64, _ = oracle.sample_rows(widened.astype(np.float64), u, 1.0)
    assert np.array_equal(t16, t64) and np.array_equal(l16, l64)


def test_draft_sampler_domain_errors():
    z = np.zeros((3, 5), np.float32)
    z[0, 2] = np.nan
    z[1, :] = -np.inf
    tok, lse, _ = oracle.sample_rows(z, np.full(3, 0.5, np.float32), 1.0)
    assert tok[0] == -1 and tok[1] == -1 and tok[2] == 2
    assert np.isnan(lse[0]) and np.isnan(lse[1]) and abs(lse[2] - np.log(5)) < 1e-15


# ---------------- supplied draft normalisers (oracle_verify_lse) ----------------
@pytest.mark.parametrize("algo", [oracle.BLOCK_VERIFY, oracle.TOKEN_VERIFY])
def test_supplied_draft_normalisers(algo):
    rng = np.random.default_rng(8)
    B, g, V = 6, 4, 300
    tgt = rng.normal(size=(B, g + 1, V)) * 2
    drf = tgt[:, :g] + rng.normal(size=(B, g, V)) * 0.7
    tok = rng.integers(0, V, size=(B, g)).astype(np.int32)
    uni = rng.random((B, g + 2), dtype=np.float32)
    base = oracle.verify(algo, tgt, drf, tok, uni, 0.9)
    # (a) the normalisers the oracle computes itself, rounded to float32, change nothing beyond
    #     that rounding (2e-6 absolute in lse, hence 2e-6 relative in Q)
    own = logsumexp(drf / np.float32(0.9), axis=-1).astype(np.float32)
    res = oracle.verify(algo, tgt, drf, tok, uni, 0.9, draft_lse=own)
    m = ~np.isnan(base.lse_d)
    assert np.array_equal(res.lse_d[m], own.astype(np.float64)[m])
    if algo == oracle.BLOCK_VERIFY:
        assert np.allclose(res.p, base.p, rtol=2e-5) and np.allclose(res.S, base.S, rtol=0, atol=1e-5)
    # (b) the supplied value is really what is used: shifting row r's normaliser by d multiplies
    #     Q_r by exp(-d), so the ratio P_r(X)/Q_r(X) grows by exp(d): written out for p_1
    shifted = own.copy()
    shifted[:, 0] += np.float32(0.25)
    res2 = oracle.verify(algo, tgt, drf, tok, uni, 0.9, draft_lse=shifted)
    if algo == oracle.BLOCK_VERIFY:
        x = tok[:, 0]
        lp = tgt[np.arange(B), 0, x] / np.float32(0.9) - logsumexp(tgt[:, 0] / np.float32(0.9), axis=-1)
        lq = drf[np.arange(B), 0, x] / np.float32(0.9) - shifted[:, 0].astype(np.float64)
        assert np.allclose(res2.p[:, 1], np.minimum(np.exp(lp - lq), 1.0), rtol=1e-12)
        # and S_0 = sum max(P_0 - Q_0 e^{-d}, 0) with the shifted normaliser
        P0 = np.exp(tgt[:, 0] / np.float32(0.9) - logsumexp(tgt[:, 0] / np.float32(0.9), axis=-1)[:, None])
        Q0 = np.exp(drf[:, 0] / np.float32(0.9) - shifted[:, 0].astype(np.float64)[:, None])
        assert np.allclose(res2.S[:, 0], np.maximum(P0 - Q0, 0).sum(-1), rtol=1e-11)
    # (c) a supplied value that is not finite is a domain error of that sequence only
    broken = own.copy()
    broken[2, 1] = np.nan
    res3 = oracle.verify(algo, tgt, drf, tok, uni, 0.9, draft_lse=broken)
    if algo == oracle.BLOCK_VERIFY:
        assert res3.out_len[2] == -1 and (res3.out_len[[0, 1, 3, 4, 5]] > 0).all()
