"""Statistical checks of the CUDA path on a tiny vocabulary (GPU).

Theorem 1: the emitted tokens, continued by sampling from the target model, follow the target
model's law M_b.  With seeded trials through the C-ABI entry points, the first emitted token and
the first two (the second drawn from the target when only one was emitted) are compared with
M_b by a chi-square test, and the mean number of accepted tokens with the exact expectation
(Theorem 2 orders the two algorithms).
"""
import itertools

import numpy as np
import pytest
import torch
from scipy import stats

import oracle
from oracle import exact
from helpers import random_tree

pytestmark = pytest.mark.gpu


def sample_rows(rng, table, prefixes, V):
    """One draw per trial from table[prefix of that trial] by inverse CDF."""
    cdf = np.cumsum(table[prefixes], axis=1)
    u = rng.random(len(prefixes))[:, None] * cdf[:, -1:]
    return np.minimum((cdf <= u).sum(axis=1), V - 1)


def tree_tables(M, V, depth):
    """Per depth an array [V**L, V] of the tree's distributions, prefix in base-V order."""
    return [np.array([[float(x) for x in M(pre)] for pre in itertools.product(range(V), repeat=L)])
            for L in range(depth + 1)]


def draw_trials(P, Q, V, g, N, seed, dtype):
    rng = np.random.default_rng(seed)
    tp, tq = tree_tables(P, V, g), tree_tables(Q, V, g)
    code = np.zeros(N, dtype=np.int64)
    tok = np.empty((N, g), dtype=np.int32)
    tgt = np.empty((N, g + 1, V), dtype=np.float32)
    drf = np.empty((N, g, V), dtype=np.float32)
    shift = rng.normal(size=(N, 2 * g + 1)).astype(np.float32) * 3      # logits are defined up to a shift
    with np.errstate(divide="ignore"):
        for i in range(g + 1):
            tgt[:, i] = np.log(tp[i][code]).astype(np.float32) + shift[:, i:i + 1]
            if i < g:
                drf[:, i] = np.log(tq[i][code]).astype(np.float32) + shift[:, g + 1 + i:g + 2 + i]
                tok[:, i] = sample_rows(rng, tq[i], code, V)
                code = code * V + tok[:, i]
    uni = rng.random((N, g + 2), dtype=np.float32)
    t, d = torch.from_numpy(tgt), torch.from_numpy(drf)
    if dtype == "bf16":
        t, d = t.bfloat16(), d.bfloat16()
    return t, d, torch.from_numpy(tok), torch.from_numpy(uni), rng


@pytest.mark.parametrize("algo", ["block", "token"])
@pytest.mark.parametrize("V,g,seed", [(8, 2, 0), (4, 3, 1), (16, 2, 2)])
def test_emitted_tokens_follow_the_target_law(V, g, seed, algo):
    import paper_2403_10444_b200 as bv
    N = 400_000
    rng0 = np.random.default_rng(1000 + seed)
    P = random_tree(rng0, V, g)
    Q = random_tree(rng0, V, g)
    t, d, tok, uni, rng = draw_trials(P, Q, V, g, N, seed, "f32")
    fn = bv.bv_verify if algo == "block" else bv.tv_verify
    ot, ol = fn(t.cuda(), d.cuda(), tok.cuda(), uni.cuda(), 1.0)
    ot, ol = ot.cpu().numpy(), ol.cpu().numpy()
    assert (ol >= 1).all() and (ol <= g + 1).all()
    # the accepted prefix is the drafted one
    for i in range(g):
        m = ol > i + 1
        assert np.array_equal(ot[m, i], tok.numpy()[m, i])

    # the stored fp32 log-probabilities define the laws actually verified
    Pf = lambda pre: np.exp(np.log(np.array([float(x) for x in P(pre)])).astype(np.float32).astype(np.float64))
    p1 = Pf(()); p1 = p1 / p1.sum()
    o1 = ot[:, 0]
    cnt1 = np.bincount(o1, minlength=V)
    chi1 = ((cnt1 - N * p1) ** 2 / (N * p1)).sum()
    assert chi1 < stats.chi2.isf(1e-6, V - 1), (chi1, cnt1 / N, p1)

    # (O_1, O_2): continue with a target draw where only one token was emitted
    tp1 = np.stack([Pf((x,)) for x in range(V)])
    tp1 = tp1 / tp1.sum(axis=1, keepdims=True)
    o2 = np.where(ol >= 2, ot[:, 1], sample_rows(rng, tp1, o1, V))
    cnt2 = np.bincount(o1 * V + o2, minlength=V * V).astype(np.float64)
    e2 = (N * p1[:, None] * tp1).ravel()
    chi2 = ((cnt2 - e2) ** 2 / e2).sum()
    assert chi2 < stats.chi2.isf(1e-6, V * V - 1), chi2

    # mean accepted length against the exact expectation of this algorithm
    want = float(exact.expected_tau(P, Q, V, g, algo))
    tau = ol - 1
    se = tau.std() / np.sqrt(N)
    assert abs(tau.mean() - want) < 5 * se + 1e-4, (tau.mean(), want, se)


def test_block_accepts_more_than_token_on_the_same_trials():
    import paper_2403_10444_b200 as bv
    V, g, N = 8, 3, 200_000
    rng0 = np.random.default_rng(77)
    P, Q = random_tree(rng0, V, g), random_tree(rng0, V, g)
    t, d, tok, uni, _ = draw_trials(P, Q, V, g, N, 5, "bf16")
    a = [x.cuda() for x in (t, d, tok, uni)]
    lb = bv.bv_verify(*a, 1.0)[1].float().mean().item()
    lt = bv.tv_verify(*a, 1.0)[1].float().mean().item()
    eb = float(exact.expected_tau(P, Q, V, g, "block"))
    et = float(exact.expected_tau(P, Q, V, g, "token"))
    assert eb > et
    # bf16 storage perturbs the laws a little; the ordering (Theorem 2) must survive clearly
    assert lb - lt > 0.5 * (eb - et)
