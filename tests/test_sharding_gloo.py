"""The multi-GPU path's host logic on CPU: two gloo ranks split one batch (no GPU needed).

The verification function handed to the sharding code here is the CPU oracle (tests may use
it); on GPUs the same code is given the CUDA entry points.
"""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from paper_2403_10444_b200 import sharding
from paper_2403_10444_b200 import workloads as wl


def test_shard_bounds_cover_the_batch():
    for B in (0, 1, 2, 7, 8, 255, 256):
        for ws in (1, 2, 3, 8):
            cuts = [sharding.shard_bounds(B, r, ws) for r in range(ws)]
            assert cuts[0][0] == 0 and cuts[-1][1] == B
            assert all(a[1] == b[0] for a, b in zip(cuts, cuts[1:]))
            sizes = [hi - lo for lo, hi in cuts]
            assert max(sizes) - min(sizes) <= 1 and sizes == sorted(sizes, reverse=True)
    with pytest.raises(ValueError):
        sharding.shard_bounds(4, 2, 2)


def test_single_rank_without_process_group():
    assert sharding.world() == (0, 1)
    assert sharding.max_over_ranks(3.5) == 3.5
    assert sharding.whole_job_rate(2048, 2.0) == 2048 / 2e-3


def _oracle_fn(algo):
    import oracle
    from parity import to_numpy_logits

    def fn(t, d, tok, uni, T):
        r = oracle.verify(algo, to_numpy_logits(t), to_numpy_logits(d), tok.numpy(), uni.numpy(), T)
        return torch.from_numpy(r.out_tokens.astype(np.int32)), torch.from_numpy(r.out_len.astype(np.int32))
    return fn


def _rank_main(rank, ws, port, B, q):
    import sys
    sys.path.insert(0, os.path.dirname(__file__))
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=ws)
    try:
        import oracle
        w = wl.scaled(wl.CONFIGS["c2"], B=B, V=2000, gamma=5)
        inp = wl.make_inputs(w, "cpu")                      # every rank draws the same batch
        res = {}
        for name, algo in (("block", oracle.BLOCK_VERIFY), ("token", oracle.TOKEN_VERIFY)):
            fn = _oracle_fn(algo)
            ot, ol = sharding.verify_sharded(fn, inp)
            lo, hi = sharding.shard_bounds(B, rank, ws)
            lt, ll = sharding.verify_sharded(fn, inp, gather=False)
            assert lt.shape[0] == hi - lo and torch.equal(lt, ot[lo:hi]) and torch.equal(ll, ol[lo:hi])
            res[name] = (ot.numpy(), ol.numpy())
        slow = sharding.max_over_ranks(10.0 + rank)
        rate = sharding.whole_job_rate(100, 2.0)
        q.put((rank, res, slow, rate))
    finally:
        dist.destroy_process_group()


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


@pytest.mark.parametrize("B", [5, 1])
def test_two_gloo_ranks_reproduce_the_unsharded_result(B):
    import oracle
    ws = 2
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = _free_port()
    procs = [ctx.Process(target=_rank_main, args=(r, ws, port, B, q)) for r in range(ws)]
    for p in procs:
        p.start()
    got = [q.get(timeout=120) for _ in range(ws)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    w = wl.scaled(wl.CONFIGS["c2"], B=B, V=2000, gamma=5)
    inp = wl.make_inputs(w, "cpu")
    for name, algo in (("block", oracle.BLOCK_VERIFY), ("token", oracle.TOKEN_VERIFY)):
        want = _oracle_fn(algo)(inp["target_logits"], inp["draft_logits"], inp["draft_tokens"],
                                inp["uniforms"], inp["temperature"])
        for rank, res, slow, rate in got:
            assert np.array_equal(res[name][0], want[0].numpy()), (name, rank)
            assert np.array_equal(res[name][1], want[1].numpy()), (name, rank)
    for rank, res, slow, rate in got:
        assert slow == 11.0                      # the maximum over the two ranks
        assert rate == 2 * 100 / 2e-3            # whole-job units per second


def test_rank_command_is_the_documented_launch():
    cmd = sharding.rank_command("bench.py", ["--gpus", "4", "--steps", "2"], 4, port=29517)
    assert cmd[1:] == ["-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node", "4", "--master-addr",
                       "127.0.0.1", "--master-port", "29517", "bench.py", "--gpus", "4", "--steps", "2"]
    with pytest.raises(ValueError):
        sharding.rank_command("bench.py", [], 0)


def test_bench_starts_its_own_ranks_when_not_under_a_launcher():
    """`bench.py --gpus 2` run as a plain program starts two ranks of itself; shown on the CPU with the
    reference arm (the oracle), where rank 0 alone works and prints the one line."""
    import json
    import os
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    env = {k: v for k, v in os.environ.items()
           if k not in ("RANK", "WORLD_SIZE", "LOCAL_RANK", "MASTER_ADDR", "MASTER_PORT")}
    r = subprocess.run([sys.executable, os.path.join(root, "bench.py"), "--impl", "reference", "--gpus", "2",
                        "--workload", "c1", "--steps", "2", "--warmup", "1"],
                       env=env, capture_output=True, text=True, timeout=300)
    assert r.returncode == 0, r.stderr[-2000:]
    lines = [json.loads(l) for l in r.stdout.splitlines() if l.startswith("{")]
    assert len(lines) == 1                                  # rank 0 alone reports
    line = lines[0]
    assert line["impl"] == "reference" and line["n_gpus"] == 2 and line["steps"] == 2
    assert line["value"] > 0 and line["cpu_baseline"]["kind"] == "oracle"
