"""Do the oracle's pins notice a wrong oracle?  (CPU only.)

Each case plants one plausible mistake in a copy of oracle/verify_oracle.c (a dropped term, a
wrong row, a wrong sign, a transposed operand, an off-by-one), compiles the copy and runs the
pins of test_oracle_c.py against it.  A mistake that no pin catches would mean that the parity
of the CUDA path with the oracle proves less than it claims.  The real oracle is never touched.
"""
import contextlib
import ctypes
import os
import subprocess

import numpy as np
import pytest

import oracle
import test_oracle_c as pins
import test_oracle_greedy as gpins
import test_oracle_probs as ppins

SRC = open(os.path.join(os.path.dirname(oracle.__file__), "verify_oracle.c")).read()
# the procedures on given probabilities follow the ones on logits in the file and repeat some of
# their lines: a mutation is planted in one part only
PROBS_MARK = "/* ================= the same procedures on given probabilities"
assert SRC.count(PROBS_MARK) == 1
HEAD, TAIL = SRC.split(PROBS_MARK)
TAIL = PROBS_MARK + TAIL

# (name, text in the oracle, what replaces it)
MUTATIONS = [
    ("ratio uses the row of position i instead of i-1",
     "double zq = logit_at(s->drf, s->dtype, s->doff + (size_t)(i - 1) * V + (size_t)x);",
     "double zq = logit_at(s->drf, s->dtype, s->doff + (size_t)(i < s->gamma ? i : i - 1) * V + (size_t)x);"),
    ("ratio upside down",
     "*lr = (zp / s->T - lse_t) - (zq / s->T - lse_d);",
     "*lr = (zq / s->T - lse_d) - (zp / s->T - lse_t);"),
    ("ratio without the normalisers",
     "*lr = (zp / s->T - lse_t) - (zq / s->T - lse_d);",
     "*lr = (zp / s->T) - (zq / s->T);"),
    ("p_i not clipped at 1",
     "p[i] = v < 1.0 ? v : 1.0;",
     "p[i] = v;"),
    ("p_i forgets p_{i-1}",
     "double v = p[i - 1] * exp(lr);",
     "double v = exp(lr);"),
    ("h_i without the 1 - p_i term",
     "h[i] = S[i] > 0.0 ? S[i] / (S[i] + 1.0 - p[i]) : 0.0;",
     "h[i] = S[i] > 0.0 ? S[i] / (S[i] + 1.0) : 0.0;"),
    ("h_i with the sign of p_i flipped",
     "h[i] = S[i] > 0.0 ? S[i] / (S[i] + 1.0 - p[i]) : 0.0;",
     "h[i] = S[i] > 0.0 ? S[i] / (S[i] + 1.0 + p[i]) : 0.0;"),
    ("h_gamma taken from the residual formula",
     "h[g] = p[g];",
     "h[g] = p[g] / (2.0 - p[g]);"),
    ("token verification keeps going after a rejection",
     "            tau = i;\n        else\n            break;",
     "            tau = i;\n        else\n            continue;"),
    ("block verification takes the first position that passes instead of the last",
     "        if (h[i] > 0.0 && eta <= h[i])\n            tau = i;\n    }",
     "        if (h[i] > 0.0 && eta <= h[i] && tau == 0)\n            tau = i;\n    }"),
    ("residual not clipped at zero",
     "return w > 0.0 ? w : 0.0;",
     "return w;"),
    ("residual with the two models swapped",
     "double w = p * P - Q;",
     "double w = Q - p * P;"),
    ("residual forgets p_i",
     "double w = p * P - Q;",
     "double w = P - Q;"),
    ("sampler returns the token after the one whose cell holds u",
     "            *margin = lo < hi ? lo : hi;\n            return x;",
     "            *margin = lo < hi ? lo : hi;\n            return x + 1 < V ? x + 1 : x;"),
    ("block verification samples the residual of position tau+1",
     "int Y = sample_index_order(s->tgt, s->toff + (size_t)tau * V, lse_t[tau],\n"
     "                                   s->drf, s->doff + (size_t)tau * V, lse_d[tau],\n"
     "                                   have_draft, s->dtype, s->V, s->T, p[tau], u, &W, &m_smp);",
     "int t2 = tau + 1 < g ? tau + 1 : tau;\n"
     "        int Y = sample_index_order(s->tgt, s->toff + (size_t)t2 * V, lse_t[t2],\n"
     "                                   s->drf, s->doff + (size_t)t2 * V, lse_d[t2],\n"
     "                                   have_draft, s->dtype, s->V, s->T, p[t2], u, &W, &m_smp);"),
    ("normaliser without the maximum added back",
     "*lse_out = m + log(s);",
     "*lse_out = log(s);"),
    ("supplied draft normaliser ignored",
     "    if (s->given_lse_d) {\n        double v = (double)s->given_lse_d[r];",
     "    if (0 && s->given_lse_d) {\n        double v = (double)s->given_lse_d[r];"),
    ("supplied draft normaliser of the wrong row",
     "double v = (double)s->given_lse_d[r];",
     "double v = (double)s->given_lse_d[r > 0 ? r - 1 : r];"),
    ("drafting step samples with the verification's other uniform convention (token after)",
     "1.0, (double)uniforms[r], &W, &m);",
     "1.0, 1.0 - (double)uniforms[r], &W, &m);"),
    ("greedy block verification clips its running product",
     "pt[i] = pt[i - 1] * exp(lr);",
     "pt[i] = pt[i - 1] * exp(lr) < 1.0 ? pt[i - 1] * exp(lr) : 1.0;"),
    ("greedy block verification: denominator sum gathers the wrong side",
     "            else\n                c += -w;",
     "            else\n                c += Q;"),
    ("greedy block verification: h_i upside down",
     "h[i] = c > 0.0 ? a / c : (a > 0.0 ? INFINITY : 0.0);",
     "h[i] = a > 0.0 ? c / a : 0.0;"),
    ("greedy block verification: last test against the clipped weight of Algorithm 2's form",
     "    if ((double)s->u[g - 1] <= pt[g])\n        tau = g;",
     "    if ((double)s->u[g - 1] <= pt[g] / (1.0 + pt[g]))\n        tau = g;"),
    ("greedy block verification: residual with a product clipped at one",
     "have_draft, s->dtype, s->V, s->T, pt[tau], u, &W, &m_smp);",
     "have_draft, s->dtype, s->V, s->T, pt[tau] < 1.0 ? pt[tau] : 1.0, u, &W, &m_smp);"),
    ("token verification without the min with 1",
     "double h = ratio < 1.0 ? ratio : 1.0;       /* h_i^token = min(ratio, 1) */",
     "double h = ratio;"),
]


def _find_selection_mutations():
    """Mutations of the parts of the file not quoted above are located by search, so that the
    test fails loudly (rather than silently testing nothing) if the oracle's text changes."""
    extra = []
    if "acc += weight_at(s->tgt, s->toff + (size_t)i * V, lse_t[i]," in HEAD:
        extra.append(("S_i from the rows of position i+1",
                      "acc += weight_at(s->tgt, s->toff + (size_t)i * V, lse_t[i],\n"
                      "                             s->drf, s->doff + (size_t)i * V, lse_d[i], 1,",
                      "acc += weight_at(s->tgt, s->toff + (size_t)(i + 1 < g ? i + 1 : i) * V, lse_t[i + 1 < g ? i + 1 : i],\n"
                      "                             s->drf, s->doff + (size_t)(i + 1 < g ? i + 1 : i) * V, lse_d[i + 1 < g ? i + 1 : i], 1,"))
    return extra


MUTATIONS += _find_selection_mutations()


def _compile(text, tmp_path, tag):
    c = tmp_path / ("oracle_%s.c" % tag)
    so = tmp_path / ("liboracle_%s.so" % tag)
    c.write_text(text)
    subprocess.check_call(["gcc", "-O1", "-fopenmp", "-shared", "-fPIC", "-o", str(so), str(c), "-lm"])
    lib = ctypes.CDLL(str(so))
    vp, ip = ctypes.c_void_p, ctypes.c_int
    lib.oracle_verify.restype = ctypes.c_int
    lib.oracle_verify.argtypes = [ip, vp, vp, vp, vp, ip, ip, ip, ip, ctypes.c_double,
                                  vp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.oracle_verify_lse.restype = ctypes.c_int
    lib.oracle_verify_lse.argtypes = [ip, vp, vp, vp, vp, vp, ip, ip, ip, ip, ctypes.c_double,
                                      vp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.oracle_sample_rows.restype = ctypes.c_int
    lib.oracle_sample_rows.argtypes = [vp, vp, ip, ip, ip, ctypes.c_double, vp, vp, vp]
    lib.oracle_verify_probs.restype = ctypes.c_int
    lib.oracle_verify_probs.argtypes = [ip, vp, vp, vp, vp, ip, ip, ip, ip, vp, vp, vp, vp, vp, vp, vp]
    lib.oracle_threads.restype = ctypes.c_int
    return lib


@contextlib.contextmanager
def _installed(lib):
    oracle._load()
    saved = oracle._lib
    oracle._lib = lib
    try:
        yield
    finally:
        oracle._lib = saved


def _pins():
    """A quick subset of the pins: the paper's worked example, the exact intermediates on
    every block, explicit normalisers and cumulative sums."""
    yield lambda: pins.test_toy_example_through_uniform_grid(oracle.BLOCK_VERIFY, "E_tau_block")
    yield lambda: pins.test_toy_example_through_uniform_grid(oracle.TOKEN_VERIFY, "E_tau_token")
    yield lambda: pins.test_intermediates_match_exact_on_every_block(0)
    yield lambda: pins.test_intermediates_match_exact_on_every_block(1)
    yield lambda: pins.test_residual_mass_identity_and_bounds()
    yield lambda: pins.test_sampler_against_explicit_cumulative_sums()
    yield lambda: pins.test_gamma1_bit_identical_outputs()
    yield lambda: pins.test_normalisers_reduce_to_scipy_logsumexp(np.float32)
    yield lambda: pins.test_lossless_by_brute_force_over_blocks_and_uniforms(oracle.BLOCK_VERIFY, "block")
    yield lambda: pins.test_supplied_draft_normalisers(oracle.BLOCK_VERIFY)
    yield lambda: pins.test_draft_sampler_frequencies_are_the_softmax()
    yield lambda: gpins.test_c_oracle_toy_example_through_uniform_grid()
    yield lambda: gpins.test_c_oracle_intermediates_match_exact(0)
    yield lambda: gpins.test_c_oracle_intermediates_match_exact(1)
    yield lambda: gpins.test_c_oracle_law_by_brute_force_over_blocks_and_uniforms()
    yield lambda: gpins.test_c_oracle_sample_follows_the_residual_with_the_unclipped_product()


def _probs_pins():
    """The pins of the procedures on given probabilities."""
    yield lambda: ppins.test_worked_example_accepted_lengths()
    yield lambda: ppins.test_intermediates_equal_the_exact_rationals(3, 2, 0)
    yield lambda: ppins.test_intermediates_equal_the_exact_rationals(4, 3, 1)
    yield lambda: ppins.test_sampled_token_follows_the_explicit_cumulative_sums("block")
    yield lambda: ppins.test_sampled_token_follows_the_explicit_cumulative_sums("token")
    yield lambda: ppins.test_output_law_is_the_target_law("block")
    yield lambda: ppins.test_agrees_with_the_logit_procedures_on_log_probabilities("token")


def _caught(pin_set=_pins):
    for pin in pin_set():
        try:
            pin()
        except AssertionError:
            return True
    return False


def test_the_pins_pass_on_the_real_oracle_compiled_the_same_way(tmp_path):
    with _installed(_compile(SRC, tmp_path, "clean")):
        assert not _caught()
        assert not _caught(_probs_pins)


@pytest.mark.parametrize("idx", range(len(MUTATIONS)))
def test_a_planted_mistake_is_caught(idx, tmp_path):
    name, old, new = MUTATIONS[idx]
    assert HEAD.count(old) == 1, "the oracle's text changed: update the mutation '%s'" % name
    with _installed(_compile(HEAD.replace(old, new) + TAIL, tmp_path, "m%d" % idx)):
        assert _caught(), "no pin noticed: " + name


# the same kinds of mistake in the procedures on given probabilities
PROBS_MUTATIONS = [
    ("ratio upside down", "*ratio = P / Q;", "*ratio = Q / P;"),
    ("ratio from the row of position i", "double P = stored_prob(s, 1, i - 1, x), Q = stored_prob(s, 0, i - 1, x);",
     "double P = stored_prob(s, 1, i < s->gamma ? i : i - 1, x), Q = stored_prob(s, 0, i < s->gamma ? i : i - 1, x);"),
    ("p_i not clipped at 1", "p[i] = v < 1.0 ? v : 1.0;", "p[i] = v;"),
    ("p_i forgets p_{i-1}", "double v = p[i - 1] * ratio;", "double v = ratio;"),
    ("h_i without the 1 - p_i term", "h[i] = S[i] > 0.0 ? S[i] / (S[i] + 1.0 - p[i]) : 0.0;",
     "h[i] = S[i] > 0.0 ? S[i] / (S[i] + 1.0) : 0.0;"),
    ("residual with the two models swapped", "double w = p * P - stored_prob(s, 0, i, x);",
     "double w = stored_prob(s, 0, i, x) - p * P;"),
    ("residual forgets p_i", "double w = p * P - stored_prob(s, 0, i, x);", "double w = P - stored_prob(s, 0, i, x);"),
    ("token verification keeps going after a rejection", "            tau = i;\n        else\n            break;",
     "            tau = i;\n        else\n            continue;"),
    ("token verification without the min with 1", "double h = ratio < 1.0 ? ratio : 1.0;", "double h = ratio;"),
    ("block verification samples with p of the wrong position", "int Y = sample_probs(s, tau, p[tau],",
     "int Y = sample_probs(s, tau, p[tau > 0 ? tau - 1 : tau],"),
]


@pytest.mark.parametrize("idx", range(len(PROBS_MUTATIONS)))
def test_a_planted_mistake_in_the_probability_procedures_is_caught(idx, tmp_path):
    name, old, new = PROBS_MUTATIONS[idx]
    assert TAIL.count(old) == 1, "the oracle's text changed: update the mutation '%s'" % name
    with _installed(_compile(HEAD + TAIL.replace(old, new), tmp_path, "p%d" % idx)):
        assert _caught(_probs_pins), "no pin noticed: " + name
