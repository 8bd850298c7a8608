"""Block Verification with supplied draft normalisers (bv_verify_lse) against the oracle that is
given the same normalisers, and the two-call pipeline sampler -> verification (GPU)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2403_10444_b200 import workloads as wl
from parity import compare, assert_parity, to_numpy_logits

pytestmark = pytest.mark.gpu


def run_case(inp, lse_f32, algo=oracle.BLOCK_VERIFY):
    import paper_2403_10444_b200 as bv
    fn = bv.bv_verify_lse if algo == oracle.BLOCK_VERIFY else bv.tv_verify_lse
    ref = oracle.verify(algo, to_numpy_logits(inp["target_logits"]), to_numpy_logits(inp["draft_logits"]),
                        inp["draft_tokens"].numpy(), inp["uniforms"].numpy(), inp["temperature"], draft_lse=lse_f32.numpy())
    d = {k: (v.cuda() if torch.is_tensor(v) else v) for k, v in inp.items()}
    a = (d["target_logits"], d["draft_logits"], d["draft_tokens"], d["uniforms"], lse_f32.cuda(), d["temperature"])
    ot, ol, diag = fn(*a, diagnostics=True)
    torch.cuda.synchronize()
    rep = compare(algo, ref, ot, ol, diag, inp)
    print(rep)
    assert_parity(rep, True)
    ot2, ol2 = fn(*a)
    rep2 = compare(algo, ref, ot2, ol2, None, inp)
    assert_parity(rep2, False)
    assert torch.equal(ot, ot2) and torch.equal(ol, ol2)
    return ref


def own_lse(inp):
    z = inp["draft_logits"].double() / np.float32(inp["temperature"])
    return torch.logsumexp(z, dim=-1).float()


@pytest.mark.parametrize("algo", [oracle.BLOCK_VERIFY, oracle.TOKEN_VERIFY])
@pytest.mark.parametrize("name,B", [("c2", 8), ("c3", 24), ("c4", 40), ("c3", 300)])
def test_supplied_normalisers_match_the_oracle(name, B, algo):
    w = wl.scaled(wl.CONFIGS[name], B=B) if B < 100 else wl.scaled(wl.CONFIGS[name], B=B, V=16384)
    inp = wl.make_inputs(w, "cpu")
    run_case(inp, own_lse(inp), algo)


@pytest.mark.parametrize("algo", [oracle.BLOCK_VERIFY, oracle.TOKEN_VERIFY])
def test_supplied_value_is_what_is_used_and_faults_are_per_sequence(algo):
    inp = wl.make_inputs(wl.scaled(wl.CONFIGS["c2"], B=6, V=4096, gamma=4), "cpu")
    lse = own_lse(inp)
    lse[:, 1] += 0.3          # a wrong normaliser is used as given: the oracle gets the same one
    lse[2, 0] = float("nan")
    ref = run_case(inp, lse, algo)
    assert ref.out_len[2] == -1 and (np.delete(ref.out_len, 2) > 0).all()


def test_sampler_then_verification_pipeline():
    # the drafting step leaves tokens and normalisers; the verification takes both as they are
    import paper_2403_10444_b200 as bv
    w = wl.scaled(wl.CONFIGS["c3"], B=16, gamma=5)
    inp = wl.make_inputs(w, "cuda")
    g = torch.Generator(device="cuda").manual_seed(3)
    u_draft = torch.rand((w.B * w.gamma,), generator=g, device="cuda")
    tok, lse = bv.bv_sample_draft(inp["draft_logits"].view(-1, w.V), u_draft, w.temperature)
    tok, lse = tok.view(w.B, w.gamma), lse.view(w.B, w.gamma).contiguous()
    ot, ol = bv.bv_verify_lse(inp["target_logits"], inp["draft_logits"], tok.contiguous(), inp["uniforms"], lse, w.temperature)
    ref = oracle.verify(oracle.BLOCK_VERIFY, to_numpy_logits(inp["target_logits"]), to_numpy_logits(inp["draft_logits"]),
                        tok.cpu().numpy(), inp["uniforms"].cpu().numpy(), w.temperature, draft_lse=lse.cpu().numpy())
    cpu_inp = {k: (v.cpu() if torch.is_tensor(v) else v) for k, v in inp.items()}
    rep = compare(oracle.BLOCK_VERIFY, ref, ot, ol, None, cpu_inp)
    assert_parity(rep, False)
    assert (ol.cpu() >= 1).all()


def test_refusals():
    import paper_2403_10444_b200 as bv
    inp = wl.make_inputs(wl.scaled(wl.CONFIGS["c1"], V=1027), "cuda")     # rows that are not 16-byte vectors
    lse = torch.zeros((1, 4), device="cuda")
    with pytest.raises(bv.BVError):
        bv.bv_verify_lse(inp["target_logits"], inp["draft_logits"], inp["draft_tokens"], inp["uniforms"], lse, 1.0)
