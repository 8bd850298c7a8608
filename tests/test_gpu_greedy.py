"""Greedy Block Verification (Algorithm 4) on the GPU: gbv_verify / gbv_verify_ex through the
C-ABI against the CPU oracle on the same seeded bits, and the statistical properties the paper
proves for one iteration (GPU)."""
import numpy as np
import pytest
import torch
from scipy import stats

import oracle
from oracle import exact
from helpers import random_tree
from paper_2403_10444_b200 import workloads as wl
from parity import run_oracle, run_cuda, compare, assert_parity
from test_gpu_parity import random_inputs
from test_gpu_distribution import draw_trials

pytestmark = pytest.mark.gpu

G = oracle.GREEDY_BLOCK_VERIFY


def parity_case(inp, check_diag=True):
    ref = run_oracle(G, inp)
    ot, ol, diag = run_cuda(G, inp)
    rep = compare(G, ref, ot, ol, diag, inp)
    print(rep)
    assert_parity(rep, check_diag)
    ot2, ol2 = run_cuda(G, inp, diagnostics=False)[:2]
    rep2 = compare(G, ref, ot2, ol2, None, inp)
    assert_parity(rep2, False)
    # the call without diagnostics leaves out sweeps that cannot matter: same tokens, bit for bit
    assert torch.equal(ot, ot2) and torch.equal(ol, ol2)
    return ref


@pytest.mark.parametrize("name", ["c1", "c2"])
def test_small_configs(name):
    parity_case(wl.make_inputs(wl.CONFIGS[name], "cpu"))


@pytest.mark.parametrize("name", ["c3", "c4"])
def test_full_size_configs(name):
    ref = parity_case(wl.make_inputs(wl.CONFIGS[name], "cuda"))
    assert (ref.p[:, 1:] > 1.0).any()        # the unclipped product does leave [0, 1] on these inputs


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("V", [8, 16, 1000, 4104, 20000])
def test_vocabularies_and_block_lengths(V, dtype):
    for gamma, B in ((1, 5), (2, 37), (5, 9), (16, 4)):
        parity_case(random_inputs(B, gamma, V, dtype, seed=V * 3 + gamma))


@pytest.mark.parametrize("sigma_d", [0.05, 0.5, 2.0])
def test_acceptance_levels(sigma_d):
    for seed in range(2):
        parity_case(random_inputs(48, 6, 12000, "bf16", seed=200 + seed, T=0.9, sigma_d=sigma_d))


def test_longest_block():
    parity_case(random_inputs(6, 64, 2048, "bf16", seed=64, sigma_d=0.3))


@pytest.mark.parametrize("cell", [(1, 2, 0.1), (16, 16, 1.0), (64, 4, 3.0)])
def test_sweep_cells(cell):
    parity_case(wl.make_inputs(wl.sweep_cell(*cell), "cuda"))


def test_gamma1_equals_block_verification_bitwise():
    inp = random_inputs(300, 1, 776, "f32", seed=21)
    a = run_cuda(G, inp, diagnostics=False)
    b = run_cuda(oracle.BLOCK_VERIFY, inp, diagnostics=False)
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])


def test_same_as_block_verification_while_the_product_stays_below_one():
    inp = random_inputs(256, 4, 4096, "bf16", seed=33, sigma_d=1.5)
    ot, ol, diag = run_cuda(G, inp)
    bt, bl, _ = run_cuda(oracle.BLOCK_VERIFY, inp)
    below = (diag["p"][:, 1:] < 1.0).all(dim=1)
    assert 10 < int(below.sum()) < 256
    assert torch.equal(ot[below], bt[below]) and torch.equal(ol[below], bl[below])
    assert not (torch.equal(ot[~below], bt[~below]) and torch.equal(ol[~below], bl[~below]))


def test_draft_equals_target_and_domain_errors():
    inp = random_inputs(16, 6, 4096, "bf16", seed=22)
    inp["draft_logits"] = inp["target_logits"][:, :6].clone()
    ot, ol, diag = run_cuda(G, inp)
    assert torch.all(ol == 7) and torch.all(diag["S"] == 0) and torch.all(diag["p"] == 1)
    parity_case(inp)
    inp = random_inputs(8, 3, 640, "f32", seed=23)
    inp["target_logits"][1, 0, 3] = float("nan")
    inp["draft_tokens"][2, 1] = 640
    inp["target_logits"][4, 1, :] = -float("inf")
    ref = run_oracle(G, inp)
    ot, ol, _ = run_cuda(G, inp)
    assert list(ol.cpu().numpy()[[1, 2, 4]]) == [-1] * 3
    assert np.array_equal(ol.cpu().numpy(), ref.out_len) and np.array_equal(ot.cpu().numpy(), ref.out_tokens)


def test_refusal_of_rows_that_are_not_whole_vectors():
    import paper_2403_10444_b200 as bv
    inp = wl.make_inputs(wl.scaled(wl.CONFIGS["c1"], V=1027), "cuda")
    with pytest.raises(bv.BVError):
        bv.gbv_verify(inp["target_logits"], inp["draft_logits"], inp["draft_tokens"], inp["uniforms"], 1.0)


@pytest.mark.parametrize("V,g,seed", [(8, 2, 0), (4, 3, 1), (16, 2, 2)])
def test_one_iteration_statistics(V, g, seed):
    # Lemma "block-accept" summed over blocks gives E[tau] = sum_l sum_{x^l} min(M_b, M_s), which
    # Theorem "greedy_one_iter" states is never below Block Verification's; and the first emitted
    # token follows the target model (the part of the guarantee that needs no modified continuation).
    import paper_2403_10444_b200 as bv
    N = 400_000
    rng0 = np.random.default_rng(2000 + seed)
    P, Q = random_tree(rng0, V, g), random_tree(rng0, V, g)
    t, d, tok, uni, _ = draw_trials(P, Q, V, g, N, seed, "f32")
    a = [x.cuda() for x in (t, d, tok, uni)]
    ot, ol = bv.gbv_verify(*a, 1.0)
    bl = bv.bv_verify(*a, 1.0)[1]
    ot, ol, bl = ot.cpu().numpy(), ol.cpu().numpy(), bl.cpu().numpy()
    assert (ol >= 1).all() and (ol <= g + 1).all()
    p1 = np.exp(np.log(np.array([float(x) for x in P(())])).astype(np.float32).astype(np.float64))
    p1 = p1 / p1.sum()
    cnt1 = np.bincount(ot[:, 0], minlength=V)
    chi1 = ((cnt1 - N * p1) ** 2 / (N * p1)).sum()
    assert chi1 < stats.chi2.isf(1e-6, V - 1), (chi1, cnt1 / N, p1)
    want = float(exact.expected_tau(P, Q, V, g, "greedy"))
    tau = ol - 1
    se = tau.std() / np.sqrt(N)
    assert abs(tau.mean() - want) < 5 * se + 1e-4, (tau.mean(), want, se)
    assert want >= float(exact.expected_tau(P, Q, V, g, "block"))
    assert tau.mean() >= (bl - 1).mean() - 5 * se
