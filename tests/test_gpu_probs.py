"""Algorithms 2 and 1 on given probabilities (bv_verify_probs, tv_verify_probs) against the oracle's
procedures on the same stored numbers (GPU)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2403_10444_b200 import workloads as wl
from parity import compare, assert_parity, record, to_numpy_logits

pytestmark = pytest.mark.gpu

ALGOS = {"block": oracle.BLOCK_VERIFY, "token": oracle.TOKEN_VERIFY}


def probs_inputs(w, dev="cpu"):
    """The workload's distributions softmax(logits / T) in fp64, stored in the workload's dtype (so
    the rows sum to one only up to the storage rounding), with its drafted tokens and uniforms."""
    inp = wl.make_inputs(w, "cpu")
    T = float(np.float32(inp["temperature"]))
    out = dict(inp)
    for k in ("target_logits", "draft_logits"):
        out[k] = torch.softmax(inp[k].double() / T, -1).to(inp[k].dtype).contiguous()
    out["temperature"] = 1.0
    return out


def run_case(algo_name, inp, label):
    import paper_2403_10444_b200 as bv
    algo = ALGOS[algo_name]
    ref = oracle.verify_probs(algo, to_numpy_logits(inp["target_logits"]), to_numpy_logits(inp["draft_logits"]),
                              inp["draft_tokens"].numpy(), inp["uniforms"].numpy())
    fn = bv.bv_verify_probs if algo_name == "block" else bv.tv_verify_probs
    a = tuple(inp[k].cuda() for k in ("target_logits", "draft_logits", "draft_tokens", "uniforms"))
    ot, ol, diag = fn(*a, diagnostics=True)
    torch.cuda.synchronize()
    rep = compare(algo, ref, ot, ol, diag, inp, probs=True)
    print(rep)
    record(rep, label + " diagnostics")
    assert_parity(rep, True)
    ot2, ol2 = fn(*a)
    torch.cuda.synchronize()
    rep2 = compare(algo, ref, ot2, ol2, None, inp, probs=True)
    record(rep2, label + " plain")
    assert_parity(rep2, False)
    return ref, (ot2, ol2)


@pytest.mark.parametrize("algo", ["block", "token"])
@pytest.mark.parametrize("name,B,gamma", [("c2", 8, 8), ("c3", 64, 8), ("c4", 40, 8), ("c3", 300, 4), ("c2", 3, 33)])
def test_probabilities_match_the_oracle(algo, name, B, gamma):
    w = wl.scaled(wl.CONFIGS[name], B=B, gamma=gamma)
    run_case(algo, probs_inputs(w), "probs %s B=%d gamma=%d %s" % (name, B, gamma, algo))


@pytest.mark.parametrize("kernel", [1, 4])         # the flow kernel, the small-batch kernel
@pytest.mark.parametrize("algo", ["block", "token"])
@pytest.mark.parametrize("V", [8, 24, 1000, 4104, 33000, (1 << 21) + 8])
def test_ragged_vocabularies(algo, V, kernel, bv_options):
    import paper_2403_10444_b200 as bv
    bv_options("kernel", kernel)
    w = wl.scaled(wl.CONFIGS["c3"], B=17 if V < (1 << 20) else 3, gamma=3, V=V)
    run_case(algo, probs_inputs(w), "probs ragged V=%d %s kernel %d" % (V, algo, kernel))
    assert bv.bv_last_kernel() == kernel


@pytest.mark.parametrize("algo", ["block", "token"])
def test_high_acceptance_reaches_the_last_row(algo):
    w = wl.scaled(wl.sweep_cell(48, 6, 0.1), V=32768)
    ref, _ = run_case(algo, probs_inputs(w), "probs high acceptance %s" % algo)
    assert (ref.out_len == 7).sum() > 5


@pytest.mark.parametrize("kernel", [1, 4])
@pytest.mark.parametrize("algo", ["block", "token"])
def test_faults_are_per_sequence_and_rows_are_used_as_stored(algo, kernel, bv_options):
    bv_options("kernel", kernel)
    w = wl.scaled(wl.CONFIGS["c2"], B=6, gamma=4, V=4096)
    inp = probs_inputs(w)
    tok = inp["draft_tokens"]
    inp["draft_logits"][1, 0, tok[1, 0]] = 0.0            # a token the draft model cannot have produced
    inp["draft_tokens"][2, 0] = w.V                       # outside the vocabulary
    inp["target_logits"][3, 0, tok[3, 0]] = float("nan")
    inp["target_logits"][4] *= 0.5                        # not renormalised
    ref, (ot, ol) = run_case(algo, inp, "probs faults %s" % algo)
    assert list(ref.out_len[1:4]) == [-1, -1, -1] and ref.out_len[0] > 0 and ref.out_len[5] > 0
    assert list(ol.cpu().numpy()[1:4]) == [-1, -1, -1]


def test_rows_that_are_not_whole_vectors_are_refused():
    import paper_2403_10444_b200 as bv
    w = wl.scaled(wl.CONFIGS["c1"], V=1022)
    inp = probs_inputs(w)
    a = tuple(inp[k].cuda() for k in ("target_logits", "draft_logits", "draft_tokens", "uniforms"))
    with pytest.raises(bv.BVError) as e:
        bv.bv_verify_probs(*a)
    assert e.value.status == -2


@pytest.mark.parametrize("kernel", [1, 4])
def test_only_the_needed_rows_are_read(kernel, bv_options):
    bv_options("kernel", kernel)
    # rows that neither algorithm reads may hold anything: here NaN everywhere except the entries of
    # the drafted tokens, in the positions that cannot be the selected one
    import paper_2403_10444_b200 as bv
    w = wl.scaled(wl.CONFIGS["c4"], B=32, gamma=8, V=8192)
    inp = probs_inputs(w)
    ref = oracle.verify_probs(oracle.BLOCK_VERIFY, to_numpy_logits(inp["target_logits"]), to_numpy_logits(inp["draft_logits"]),
                              inp["draft_tokens"].numpy(), inp["uniforms"].numpy())
    g = w.gamma
    eta = inp["uniforms"].numpy().astype(np.float64)
    poisoned = 0
    for b in range(w.B):
        for i in range(1, g):
            if eta[b, i - 1] > ref.p[b, i] * (1 + 1e-3):          # cannot be the selected position: never swept
                keep_t = inp["target_logits"][b, i, inp["draft_tokens"][b, i]].clone()
                keep_d = inp["draft_logits"][b, i, inp["draft_tokens"][b, i]].clone()
                inp["target_logits"][b, i] = float("nan")
                inp["draft_logits"][b, i] = float("nan")
                inp["target_logits"][b, i, inp["draft_tokens"][b, i]] = keep_t
                inp["draft_logits"][b, i, inp["draft_tokens"][b, i]] = keep_d
                poisoned += 1
    assert poisoned > 20
    a = tuple(inp[k].cuda() for k in ("target_logits", "draft_logits", "draft_tokens", "uniforms"))
    ot, ol = bv.bv_verify_probs(*a)
    rep = compare(oracle.BLOCK_VERIFY, ref, ot, ol, None, inp, probs=True)
    assert rep.hard_mismatches == 0 and rep.mismatches <= 1, str(rep)
