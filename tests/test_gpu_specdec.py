"""The decoding loop of Algorithm 3 around the library (paper_2403_10444_b200/specdec.py) on
synthetic last-token models (GPU).

  - the same loop written with the CPU oracle's drafting and verification steps, on the same
    uniforms, must generate the same tokens;
  - the paper's two-token example run through many iterations: 20/9 tokens per iteration with
    Block Verification, 19/9 with Token Verification (accepted tokens 11/9 and 10/9 plus the
    correction token);
  - Theorem 1 across iterations: the first tokens generated follow the target chain's law.
"""
import os
from fractions import Fraction as F

import numpy as np
import pytest
import torch
from scipy import stats

import oracle
from helpers import read_golden
from paper_2403_10444_b200 import specdec, workloads as wl
from parity import to_numpy_logits

pytestmark = pytest.mark.gpu
GOLD = read_golden(os.path.join(os.path.dirname(__file__), "golden", "toy_example.txt"))


def oracle_loop(tt, dt, first, u_draft, u_verify, gamma, T, algo, supply_lse):
    """Algorithm 3 with the oracle's steps: draft gamma tokens one after the other from the draft
    model's rows, score the path with the target model's rows, verify, extend the sequence."""
    tt_np, dt_np = to_numpy_logits(tt), to_numpy_logits(dt)
    N, B = u_draft.shape[0], first.shape[0]
    cur = first.numpy().astype(np.int64)
    out_seq = [[] for _ in range(B)]
    for n in range(N):
        toks = np.empty((B, gamma), np.int32)
        lse = np.empty((B, gamma), np.float32)
        last = cur
        for i in range(gamma):
            tok, l, _ = oracle.sample_rows(dt_np[last], u_draft[n, i].numpy(), T)
            toks[:, i], lse[:, i], last = tok, l.astype(np.float32), tok.astype(np.int64)
        path = np.concatenate([cur[:, None], toks.astype(np.int64)], axis=1)
        res = oracle.verify(algo, tt_np[path], dt_np[path[:, :gamma]], toks, u_verify[n].numpy(), T,
                            draft_lse=lse if supply_lse else None)
        for b in range(B):
            k = int(res.out_len[b])
            out_seq[b] += [int(x) for x in res.out_tokens[b, :k]]
        cur = np.array([s[-1] for s in out_seq], np.int64)
    return out_seq


@pytest.mark.parametrize("algo,oalgo,lse", [("block", oracle.BLOCK_VERIFY, False),
                                            ("token", oracle.TOKEN_VERIFY, False),
                                            ("block_lse", oracle.BLOCK_VERIFY, True),
                                            ("token_lse", oracle.TOKEN_VERIFY, True)])
def test_loop_matches_the_oracle_loop(algo, oalgo, lse):
    V, B, gamma, N, T = 2048, 12, 4, 6, 0.9
    tt, dt = wl.markov_models(V, "bf16", 5, 2.0, 0.8, 1.1, "cpu")
    first = torch.arange(B, dtype=torch.int32)
    ud, uv = wl.loop_uniforms(N, B, gamma, 6, "cpu")
    want = oracle_loop(tt, dt, first, ud, uv, gamma, T, oalgo, lse)
    res = specdec.run(tt.cuda(), dt.cuda(), first.cuda(), ud.cuda(), uv.cuda(), gamma, T, algo)
    toks, lens = res["tokens"].cpu().numpy(), res["lengths"].cpu().numpy()
    if lse:
        # the supplied normalisers are each side's own float32 values, which may differ in the last
        # bit; a sequence may then part ways at a near-tie, so only agreement of most is asked
        same = sum(list(toks[b, : lens[b]]) == want[b] for b in range(B))
        assert same >= B - 1
    else:
        for b in range(B):
            assert list(toks[b, : lens[b]]) == want[b], b
    assert (toks[np.arange(toks.shape[1])[None, :] >= lens[:, None]] == -1).all()
    assert N <= lens.min() and lens.max() <= N * (gamma + 1)


def toy_tables(V=8):
    """The paper's context-free two-token example as [V, V] tables (tokens 2.. masked out)."""
    p = torch.full((V,), -float("inf"))
    q = p.clone()
    p[:2] = torch.log(torch.tensor([float(F(x)) for x in GOLD["target"]]))
    q[:2] = torch.log(torch.tensor([float(F(x)) for x in GOLD["draft"]]))
    return p.repeat(V, 1).contiguous(), q.repeat(V, 1).contiguous()


@pytest.mark.parametrize("algo,key", [("block", "E_tau_block"), ("block_lse", "E_tau_block"), ("token", "E_tau_token")])
def test_toy_example_block_efficiency(algo, key):
    tt, dt = toy_tables()
    B, N, gamma = 20000, 8, 2
    ud, uv = wl.loop_uniforms(N, B, gamma, 11, "cuda")
    res = specdec.run(tt.cuda(), dt.cuda(), torch.zeros(B, dtype=torch.int32, device="cuda"), ud, uv, gamma, 1.0, algo)
    tau = res["tau"].float().cpu().numpy().ravel()
    want = float(F(GOLD[key][0]))
    se = tau.std() / np.sqrt(tau.size)
    assert abs(tau.mean() - want) < 5 * se, (tau.mean(), want)
    assert abs(specdec.block_efficiency(res) - (want + 1.0)) < 5 * se
    # every generated token is a or b, and their frequencies are the target model's
    toks = res["tokens"].cpu().numpy()
    gen = toks[toks >= 0]
    assert gen.max() <= 1
    pa = float(F(GOLD["target"][0]))
    assert abs((gen == 0).mean() - pa) < 5 * np.sqrt(pa * (1 - pa) / gen.size)


@pytest.mark.parametrize("algo", ["block_lse", "token"])
def test_generated_tokens_follow_the_target_chain(algo):
    # the first three generated tokens, which come from one, two or three iterations depending on
    # what was accepted, against the target chain's law (chi-square over V^3 cells)
    V, B, N, gamma, T = 8, 300_000, 3, 2, 1.0
    tt, dt = wl.markov_models(V, "f32", 21, 1.2, 0.9, 0.0, "cuda")
    ud, uv = wl.loop_uniforms(N, B, gamma, 22, "cuda")
    res = specdec.run(tt, dt, torch.full((B,), 3, dtype=torch.int32, device="cuda"), ud, uv, gamma, T, algo)
    toks = res["tokens"][:, :3].cpu().numpy().astype(np.int64)
    assert (toks >= 0).all()
    P = torch.softmax(tt.double().cpu() / T, dim=-1).numpy()
    expect = (P[3][:, None, None] * P[:, :, None] * P[None, :, :]).ravel() * B
    cnt = np.bincount(toks[:, 0] * V * V + toks[:, 1] * V + toks[:, 2], minlength=V ** 3)
    chi = ((cnt - expect) ** 2 / expect).sum()
    assert chi < stats.chi2.isf(1e-6, V ** 3 - 1), chi


def test_block_verification_generates_more_per_iteration():
    V, B, N, gamma = 4096, 256, 12, 6
    tt, dt = wl.markov_models(V, "bf16", 31, 2.0, 1.0, 1.1, "cuda")
    ud, uv = wl.loop_uniforms(N, B, gamma, 32, "cuda")
    first = torch.zeros(B, dtype=torch.int32, device="cuda")
    be = {a: specdec.block_efficiency(specdec.run(tt, dt, first, ud, uv, gamma, 1.0, a)) for a in specdec.ALGOS}
    assert be["block"] > be["token"] and be["block_lse"] > be["token"]


@pytest.mark.parametrize("B", [48, 12])        # the flow kernel; the small-batch kernel (a cooperative launch) for block / token
@pytest.mark.parametrize("algo", ["block_lse", "block", "token"])
def test_graph_replay_generates_the_same_tokens(algo, B):
    V, N, gamma = 4096, 9, 5
    tt, dt = wl.markov_models(V, "bf16", 41, 2.0, 1.0, 1.1, "cuda")
    ud, uv = wl.loop_uniforms(N, B, gamma, 42, "cuda")
    first = torch.arange(B, dtype=torch.int32, device="cuda")
    a = specdec.run(tt, dt, first, ud, uv, gamma, 0.9, algo)
    b = specdec.run(tt, dt, first, ud, uv, gamma, 0.9, algo, graph=True)
    for k in ("tokens", "lengths", "tau", "drafted"):
        assert torch.equal(a[k], b[k]), k


@pytest.mark.parametrize("algo,oalgo", [("block", oracle.BLOCK_VERIFY), ("token", oracle.TOKEN_VERIFY)])
def test_nucleus_masked_rows_through_the_loop(algo, oalgo):
    # top-p masked rows (-inf outside each row's nucleus, the two models' nuclei differ): tokens the
    # target model excludes are never emitted, and the loop still equals the oracle's
    V, B, gamma, N, T = 1024, 10, 4, 5, 0.8
    tt, dt = wl.markov_models(V, "f32", 51, 2.0, 1.0, 1.1, "cpu")
    tt, dt = wl.top_p_mask(tt, 0.9, T), wl.top_p_mask(dt, 0.9, T)
    assert 0.02 < torch.isfinite(tt).float().mean() < 0.9
    first = torch.arange(B, dtype=torch.int32)
    ud, uv = wl.loop_uniforms(N, B, gamma, 52, "cpu")
    want = oracle_loop(tt, dt, first, ud, uv, gamma, T, oalgo, False)
    res = specdec.run(tt.cuda(), dt.cuda(), first.cuda(), ud.cuda(), uv.cuda(), gamma, T, algo)
    toks, lens = res["tokens"].cpu().numpy(), res["lengths"].cpu().numpy()
    for b in range(B):
        got = list(toks[b, : lens[b]])
        assert got == want[b], b
        prev = int(first[b])
        for x in got:
            assert torch.isfinite(tt[prev, x]), "a token outside the target model's nucleus was emitted"
            prev = x


@pytest.mark.parametrize("dtype,V,B,gamma,T", [("bf16", 4096, 40, 6, 0.9), ("f32", 1024, 7, 3, 1.3), ("bf16", 32768, 300, 8, 0.8), ("f32", 8, 5, 10, 1.0)])
def test_draft_chain_equals_the_sampler_called_step_by_step(dtype, V, B, gamma, T):
    # one launch for the whole chain against gamma calls of bv_sample_draft with the look-ups in between
    # (bit for bit), and against the oracle's drafting step applied step by step
    import paper_2403_10444_b200 as bv
    tt, dt = wl.markov_models(V, dtype, 61, 2.0, 1.0, 1.1 if V > 8 else 0.0, "cuda")
    g = torch.Generator(device="cuda").manual_seed(62)
    first = torch.randint(0, V, (B,), generator=g, device="cuda", dtype=torch.int32)
    u = torch.rand((gamma, B), generator=g, device="cuda")
    tok, lse = bv.bv_draft_chain(dt, first, u, T)
    last = first.to(torch.int64)
    dt_np = to_numpy_logits(dt.cpu())
    last_np = first.cpu().numpy().astype(np.int64)
    safe = np.ones(B, bool)
    for i in range(gamma):
        t_i, l_i = bv.bv_sample_draft(dt.index_select(0, last), u[i].contiguous(), T)
        assert torch.equal(t_i, tok[:, i]) and torch.equal(l_i.view(torch.int32), lse[:, i].contiguous().view(torch.int32))
        want, want_lse, margin = oracle.sample_rows(dt_np[last_np], u[i].cpu().numpy(), T)
        safe &= margin > 1e-6                      # (a sequence that parts ways at a near-tie is not followed further)
        got = tok[:, i].cpu().numpy()
        assert (got[safe] == want[safe]).all()
        assert np.abs(lse[:, i].cpu().numpy()[safe] - want_lse[safe]).max() < 3e-6
        last, last_np = t_i.to(torch.int64), got.astype(np.int64)
    assert safe.sum() >= 0.8 * B       # (a uniform within 1e-6 of an edge of its cell: about 1 % of the draws at V = 32768)


def test_draft_chain_ends_a_sequence_at_a_token_it_cannot_follow():
    import paper_2403_10444_b200 as bv
    V, B, gamma = 16, 4, 5
    dt = torch.zeros((V, V), device="cuda")
    dt[3, :] = float("-inf")                       # nothing can follow token 3
    dt[:, 3] += 50.0                               # ... which every other row produces almost surely
    first = torch.tensor([0, 3, V, 5], dtype=torch.int32, device="cuda")     # sequence 2 starts outside the vocabulary
    u = torch.full((gamma, B), 0.5, device="cuda")
    tok, lse = bv.bv_draft_chain(dt, first, u, 1.0)
    tok, lse = tok.cpu(), lse.cpu()
    assert tok[0].tolist() == [3, -1, -1, -1, -1] and torch.isnan(lse[0, 1:]).all() and not torch.isnan(lse[0, 0])
    assert tok[1].tolist() == [-1] * 5 and tok[2].tolist() == [-1] * 5 and torch.isnan(lse[1:3]).all()
    assert tok[3].tolist() == [3, -1, -1, -1, -1]


@pytest.mark.parametrize("algo", ["block_lse", "token"])
def test_loop_with_and_without_the_chain_kernel_generates_the_same_tokens(algo):
    V, B, N, gamma = 4096, 24, 7, 5
    tt, dt = wl.markov_models(V, "bf16", 71, 2.0, 1.0, 1.1, "cuda")
    ud, uv = wl.loop_uniforms(N, B, gamma, 72, "cuda")
    first = torch.arange(B, dtype=torch.int32, device="cuda")
    a = specdec.run(tt, dt, first, ud, uv, gamma, 0.9, algo, chain=True)
    b = specdec.run(tt, dt, first, ud, uv, gamma, 0.9, algo, chain=False)
    for k in ("tokens", "lengths", "tau", "drafted"):
        assert torch.equal(a[k], b[k]), k
