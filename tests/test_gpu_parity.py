"""GPU parity: the CUDA library against the CPU oracle on the same seeded bits,
element by element, through the C-ABI (via the ctypes binding)."""
import os

import numpy as np
import pytest
import torch

import oracle
from paper_2403_10444_b200 import workloads as wl
from parity import run_oracle, run_cuda, compare, assert_parity, record

pytestmark = pytest.mark.gpu

ALGOS = [oracle.BLOCK_VERIFY, oracle.TOKEN_VERIFY]
KERNELS = {"flow": 1, "cluster": 2, "stream": 3, "small": 4}     # values of the library's "kernel" option


def parity_case(inp, algo, check_diag=True):
    ref = run_oracle(algo, inp)
    ot, ol, diag = run_cuda(algo, inp)
    rep = compare(algo, ref, ot, ol, diag, inp)
    print(rep)
    record(rep, os.environ.get("PYTEST_CURRENT_TEST", "") + " diagnostics")
    assert_parity(rep, check_diag)
    # the entry points without diagnostic outputs are the ones a server calls (and the bench times);
    # for Algorithm 2 they leave out the second sweep of positions that cannot be selected, so
    # their tokens are checked against the oracle on their own
    ot2, ol2 = run_cuda(algo, inp, diagnostics=False)[:2]
    rep2 = compare(algo, ref, ot2, ol2, None, inp)
    print(rep2)
    record(rep2, os.environ.get("PYTEST_CURRENT_TEST", "") + " plain")
    assert_parity(rep2, False)
    return rep


def random_inputs(B, gamma, V, dtype, seed, T=1.0, sigma_t=2.0, sigma_d=1.0):
    w = wl.Workload("t", B, gamma, V, dtype, T, seed, sigma_t, 0.0, 0, 0.0, sigma_d)
    return wl.make_inputs(w, "cpu")


@pytest.mark.parametrize("algo", ALGOS)
@pytest.mark.parametrize("name", ["c1", "c2"])
def test_small_configs(name, algo):
    parity_case(wl.make_inputs(wl.CONFIGS[name], "cpu"), algo)


@pytest.mark.parametrize("algo", ALGOS)
@pytest.mark.parametrize("name", ["c3", "c4"])
def test_full_size_configs(name, algo):
    # generated on the GPU (fast), the same bits copied to the oracle
    inp = wl.make_inputs(wl.CONFIGS[name], "cuda")
    parity_case(inp, algo)


@pytest.mark.parametrize("algo", ALGOS)
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("V", [1, 2, 3, 8, 17, 1000, 1027, 4104, 20000])
def test_ragged_vocabularies(V, dtype, algo):
    # V = 1..17 and odd V take the element-wise path; multiples of 16 bytes the 128-bit path
    for gamma, B in ((1, 5), (2, 37), (5, 9)):
        parity_case(random_inputs(B, gamma, V, dtype, seed=V * 7 + gamma), algo)


@pytest.mark.parametrize("algo", ALGOS)
@pytest.mark.parametrize("cluster", [1, 2, 4, 8])
def test_every_cluster_width(cluster, algo, bv_options):
    bv_options("cluster", cluster)
    bv_options("kernel", KERNELS["cluster"])
    parity_case(random_inputs(19, 4, 24000, "bf16", seed=cluster, T=0.8), algo)
    parity_case(random_inputs(7, 3, 5000, "f32", seed=cluster + 10), algo)


@pytest.mark.parametrize("algo", ALGOS)
@pytest.mark.parametrize("kernel", ["flow", "cluster", "stream", "small"])
def test_every_kernel(kernel, algo, bv_options):
    # the library has several kernels for each algorithm; each must match the oracle
    bv_options("kernel", KERNELS[kernel])
    parity_case(random_inputs(32 if kernel == "small" else 40, 5, 24000, "bf16", seed=77, T=0.8), algo)
    parity_case(random_inputs(9, 3, 4096, "f32", seed=78), algo)
    parity_case(wl.make_inputs(wl.scaled(wl.CONFIGS["c4"], B=6), "cuda"), algo)


@pytest.mark.parametrize("chunks", [1, 3, 8])
def test_flow_chunk_counts(chunks, bv_options):
    bv_options("kernel", KERNELS["flow"])
    bv_options("flow_chunks", chunks)
    parity_case(random_inputs(21, 4, 16384, "bf16", seed=chunks), oracle.BLOCK_VERIFY)
    bv_options("flow_ctas", 3)     # far fewer CTAs than items
    parity_case(random_inputs(21, 4, 16384, "bf16", seed=chunks + 1), oracle.BLOCK_VERIFY)


@pytest.mark.parametrize("fine", [1, 5, 100])
def test_flow_finer_chunks_for_the_last_sequences(fine, bv_options):
    bv_options("kernel", KERNELS["flow"])
    bv_options("flow_fine", fine)
    parity_case(random_inputs(21, 4, 65536, "bf16", seed=fine), oracle.BLOCK_VERIFY)
    parity_case(wl.make_inputs(wl.scaled(wl.CONFIGS["c4"], B=12), "cuda"), oracle.BLOCK_VERIFY)
    bv_options("flow_ctas", 3)
    parity_case(random_inputs(9, 6, 131072, "f32", seed=fine + 1), oracle.BLOCK_VERIFY)


@pytest.mark.parametrize("algo", ALGOS)
@pytest.mark.parametrize("kernel", ["flow", "small", "default"])
@pytest.mark.parametrize("dtype,V", [("f32", 1 << 21), ("bf16", (1 << 21) + 8), ("bf16", (1 << 21) + 1)])
def test_very_large_vocabularies(dtype, V, kernel, algo, bv_options):
    # two million logits a row: chunk, piece and segment ranges far beyond the benchmark's sizes; the odd V
    # takes the element-wise path
    if kernel != "default":
        if V % 8:
            pytest.skip("the flow and small-batch kernels take rows of whole 16-byte vectors")
        bv_options("kernel", KERNELS[kernel])
    parity_case(random_inputs(3, 2, V, dtype, seed=V % 97, T=0.9), algo)


@pytest.mark.parametrize("algo", ALGOS)
def test_many_short_sequences(algo, bv_options):
    # far more sequences than CTAs, rows of a few vectors: every counter and queue index of the flow kernel
    bv_options("kernel", KERNELS["flow"])
    parity_case(random_inputs(6000, 3, 64, "bf16", seed=5, sigma_d=0.5), algo)
    parity_case(random_inputs(3000, 1, 16, "f32", seed=6), algo)


@pytest.mark.parametrize("algo", ALGOS)
def test_more_sequences_than_resident_clusters(algo):
    parity_case(random_inputs(700, 3, 512, "f32", seed=3), algo)


@pytest.mark.parametrize("kernel", ["flow", "small"])
@pytest.mark.parametrize("algo", ALGOS)
@pytest.mark.parametrize("gamma", [1, 16, 64])
def test_block_lengths(gamma, algo, kernel, bv_options):
    bv_options("kernel", KERNELS[kernel])
    parity_case(random_inputs(6, gamma, 2048, "bf16", seed=gamma, sigma_d=0.3), algo)


@pytest.mark.parametrize("kernel", ["flow", "small"])
@pytest.mark.parametrize("T", [0.2, 0.6, 1.0, 2.5])
def test_temperatures(T, kernel, bv_options):
    bv_options("kernel", KERNELS[kernel])
    for algo in ALGOS:
        parity_case(random_inputs(12, 4, 8192, "f32", seed=5, T=T), algo)


@pytest.mark.parametrize("algo", ALGOS)
@pytest.mark.parametrize("B,gamma,V,dtype", [(1, 8, 152064, "bf16"), (16, 8, 152064, "bf16"), (2, 2, 1024, "f32"),
                                             (32, 15, 4096, "bf16"), (5, 33, 640, "f32"), (3, 1, 8, "bf16"), (8, 60, 2048, "bf16")])
def test_small_batch_kernel(B, gamma, V, dtype, algo, bv_options):
    # the kernel of the latency regime, forced for every shape it admits (chunks and pieces of every count)
    bv_options("kernel", KERNELS["small"])
    parity_case(random_inputs(B, gamma, V, dtype, seed=B + gamma, T=0.9, sigma_d=0.4), algo)
    bv_options("kernel", 0)
    bv_options("small_bytes", 1)       # ... and the default choice with the small-batch kernel all but switched off
    parity_case(random_inputs(B, gamma, V, dtype, seed=B + gamma + 1, T=0.9, sigma_d=0.4), algo)


def test_gamma1_block_equals_token_bitwise():
    inp = random_inputs(300, 1, 777, "f32", seed=21)
    a = run_cuda(oracle.BLOCK_VERIFY, inp, diagnostics=False)
    b = run_cuda(oracle.TOKEN_VERIFY, inp, diagnostics=False)
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])


@pytest.mark.parametrize("kernel", ["flow", "small"])
def test_draft_equals_target(kernel, bv_options):
    bv_options("kernel", KERNELS[kernel])
    inp = random_inputs(16, 6, 4096, "bf16", seed=22)
    inp["draft_logits"] = inp["target_logits"][:, :6].clone()
    for algo in ALGOS:
        ot, ol, diag = run_cuda(algo, inp)
        assert torch.all(ol == 7)
        assert torch.equal(ot[:, :6].cpu(), inp["draft_tokens"])
        parity_case(inp, algo)
    _, _, diag = run_cuda(oracle.BLOCK_VERIFY, inp)
    assert torch.all(diag["S"] == 0) and torch.all(diag["p"] == 1)


@pytest.mark.parametrize("kernel", ["flow", "small"])
def test_masked_logits_and_domain_errors(kernel, bv_options):
    bv_options("kernel", KERNELS[kernel])
    inp = random_inputs(8, 3, 640, "f32", seed=23)
    t, d, tok = inp["target_logits"], inp["draft_logits"], inp["draft_tokens"]
    # top-k style masking: legal
    t[0, :, 100:] = -float("inf")
    d[0, :, 200:] = -float("inf")
    q = torch.softmax(d[0], dim=-1)
    tok[0] = torch.multinomial(q, 1).squeeze(1).to(torch.int32)
    t[1, 0, 3] = float("nan")
    tok[2, 1] = 640
    d[3, 0, tok[3, 0]] = -float("inf")
    t[4, 1, :] = -float("inf")
    t[5, 2, 7] = float("inf")
    tok[6, 0] = -1
    ref = run_oracle(oracle.BLOCK_VERIFY, inp)
    ot, ol, _ = run_cuda(oracle.BLOCK_VERIFY, inp)
    assert list(ol.cpu().numpy()[[1, 2, 3, 4, 5, 6]]) == [-1] * 6
    assert torch.all(ot[[1, 2, 3, 4, 5, 6]] == -1)
    assert np.array_equal(ol.cpu().numpy(), ref.out_len)
    assert np.array_equal(ot.cpu().numpy(), ref.out_tokens)
    # Algorithm 1 reads rows 0..tau only: same inputs, compare with its oracle
    ref = run_oracle(oracle.TOKEN_VERIFY, inp)
    ot, ol, _ = run_cuda(oracle.TOKEN_VERIFY, inp)
    assert np.array_equal(ol.cpu().numpy(), ref.out_len)
    assert np.array_equal(ot.cpu().numpy(), ref.out_tokens)


def test_deterministic_bits():
    inp = wl.make_inputs(wl.scaled(wl.CONFIGS["c3"], B=8), "cuda")
    a = run_cuda(oracle.BLOCK_VERIFY, inp)
    b = run_cuda(oracle.BLOCK_VERIFY, inp)
    assert torch.equal(a[0], b[0]) and torch.equal(a[1], b[1])
    for k in a[2]:
        assert torch.equal(a[2][k].view(torch.int32), b[2][k].view(torch.int32))


@pytest.mark.parametrize("cell", [(1, 2, 0.1), (16, 16, 1.0), (64, 4, 3.0), (512, 2, 1.0)])
def test_sweep_cells(cell):
    inp = wl.make_inputs(wl.sweep_cell(*cell), "cuda")
    for algo in ALGOS:
        parity_case(inp, algo)


def test_host_buffer_entry_matches_device_entry():
    import paper_2403_10444_b200 as bv
    inp = random_inputs(33, 4, 3000, "bf16", seed=31)
    pinned = {k: (v.pin_memory() if torch.is_tensor(v) else v) for k, v in inp.items()}
    for host_fn, algo in ((bv.bv_verify_host, oracle.BLOCK_VERIFY), (bv.tv_verify_host, oracle.TOKEN_VERIFY)):
        ot, ol = host_fn(pinned["target_logits"], pinned["draft_logits"], pinned["draft_tokens"],
                         pinned["uniforms"], pinned["temperature"])
        dt, dl = run_cuda(algo, inp, diagnostics=False)
        assert torch.equal(ot, dt.cpu()) and torch.equal(ol, dl.cpu())


def test_launch_count_and_nonblocking_stream():
    import paper_2403_10444_b200 as bv
    inp = {k: (v.cuda() if torch.is_tensor(v) else v) for k, v in random_inputs(5, 2, 1024, "f32", 1).items()}
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        ot, ol = bv.bv_verify(inp["target_logits"], inp["draft_logits"], inp["draft_tokens"],
                              inp["uniforms"], 1.0, stream=s)
    s.synchronize()
    assert bv.bv_last_launch_count() == 1
    ref = run_oracle(oracle.BLOCK_VERIFY, inp)
    assert np.array_equal(ol.cpu().numpy(), ref.out_len)


@pytest.mark.parametrize("sigma_d", [0.05, 0.5, 2.0])
def test_skipped_second_sweeps_change_nothing(sigma_d):
    # Without diagnostic outputs Algorithm 2's second sweep runs only for positions with
    # eta_i <= p_i (h_i <= p_i always), from the top down, until one is selected.  The emitted
    # tokens must be bit for bit those of the call that computes every position, at every
    # acceptance level: nearly all positions wanted (small noise) or nearly none (large).
    for seed in range(3):
        inp = random_inputs(48, 6, 12000, "bf16", seed=100 + seed, T=0.9, sigma_d=sigma_d)
        full = run_cuda(oracle.BLOCK_VERIFY, inp, diagnostics=True)
        fast = run_cuda(oracle.BLOCK_VERIFY, inp, diagnostics=False)
        assert torch.equal(full[0], fast[0]) and torch.equal(full[1], fast[1])


def test_calls_on_several_streams_at_once():
    # every stream has a workspace of its own: calls in flight together on different streams, of shapes
    # that the flow kernel and the small-batch kernel serve, give what the same calls give one by one
    import paper_2403_10444_b200 as bv
    shapes = [(48, 5, 16384, "bf16"), (6, 4, 8192, "f32"), (80, 3, 4096, "bf16"), (2, 8, 32000, "bf16")]
    cases = []
    for i, (B, g, V, dt) in enumerate(shapes):
        inp = {k: (v.cuda() if torch.is_tensor(v) else v) for k, v in random_inputs(B, g, V, dt, seed=500 + i).items()}
        a = (inp["target_logits"], inp["draft_logits"], inp["draft_tokens"], inp["uniforms"], inp["temperature"])
        cases.append((a, bv.bv_verify(*a), bv.tv_verify(*a)))
    torch.cuda.synchronize()
    streams = [torch.cuda.Stream() for _ in cases]
    for rep in range(3):
        outs = []
        for (a, _, _), s in zip(cases, streams):
            with torch.cuda.stream(s):
                outs.append((bv.bv_verify(*a, stream=s), bv.tv_verify(*a, stream=s)))
        for s in streams:
            s.synchronize()
            assert bv.bv_stream_status(s) == 0
        for (a, want_b, want_t), (got_b, got_t) in zip(cases, outs):
            assert torch.equal(got_b[0], want_b[0]) and torch.equal(got_b[1], want_b[1])
            assert torch.equal(got_t[0], want_t[0]) and torch.equal(got_t[1], want_t[1])
