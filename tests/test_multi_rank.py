"""The N > 1 path on CPU: two gloo ranks shard a batch, each checks its own shard with the oracle, and the
timing reduction / result gather behave as bench.py relies on (no GPU needed)."""
import os
import subprocess
import sys

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

import workloads as W
from oracle import head as OH
from oracle import verify as OV
from paper_2609_27396_b200 import dist_util as DU

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def test_shard_requests_partition_and_balance():
    lens = W.workload(3).attn.ctx_lens
    for world in (1, 2, 4, 8):
        parts = DU.shard_requests(lens, world)
        assert sorted(i for p in parts for i in p) == list(range(len(lens)))
        loads = [sum(lens[i] for i in p) for p in parts]
        assert max(loads) - min(loads) <= max(lens)
    assert DU.shard_requests([5, 1], 4) == [[0], [1], [], []]
    assert DU.rank_seed(7, 0) == 7 and DU.rank_seed(7, 3) != DU.rank_seed(7, 2)


def _worker(rank, world, port, q):
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sh = W.VerifyShape(6, 5, 300, 2, 8, "greedy", 0.7, 1.0)
    v = W.make_verify_inputs(sh, 11)                       # same global batch on both ranks
    lens = [40, 10, 30, 20, 50, 60]
    mine = DU.shard_requests(lens, world)[rank]
    res = OV.verify_greedy(v.target[mine], v.draft_tokens[mine], v.reps[mine])
    a, b = DU.gather_results(res["accept_len"].tolist(), res["bonus"].tolist())
    t = DU.max_over_ranks(1.0 + rank)
    # the head loop shards the same way: each request's chain depends on its own rows and bonus only
    hin = W.make_head_inputs(W.HeadShape(6, 3, 16, 64, 8), 13)
    toks = OH.draft_head_greedy(hin.sel_reps[mine], hin.w_lm, hin.ar_w, hin.ar_e, hin.bonus[mine])
    q.put((rank, mine, a, b, t, toks.tolist()))
    dist.destroy_process_group()


def test_two_gloo_ranks_shard_and_reduce():
    world, port = 2, 29511 + (os.getpid() % 200)
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, world, port, q)) for r in range(world)]
    for p in procs:
        p.start()
    got = [q.get(timeout=120) for _ in range(world)]
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    sh = W.VerifyShape(6, 5, 300, 2, 8, "greedy", 0.7, 1.0)
    v = W.make_verify_inputs(sh, 11)
    full = OV.verify_greedy(v.target, v.draft_tokens, v.reps)
    hin = W.make_head_inputs(W.HeadShape(6, 3, 16, 64, 8), 13)
    htoks = OH.draft_head_greedy(hin.sel_reps, hin.w_lm, hin.ar_w, hin.ar_e, hin.bonus)
    for rank, mine, a, b, t, toks in got:
        assert t == 2.0                                    # max over ranks of (1 + rank)
        assert toks == htoks[mine].tolist()                # a shard's head tokens = the same rows of the whole batch
        parts = DU.shard_requests([40, 10, 30, 20, 50, 60], world)
        for r in range(world):                             # every rank sees every shard's outcome
            assert a[r] == full["accept_len"][parts[r]].tolist() and b[r] == full["bonus"][parts[r]].tolist()


def test_reference_arm_nonzero_rank_is_silent():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2", LOCAL_RANK="1")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2", "--steps", "1",
                        "--warmup", "0"], env=env, capture_output=True, text=True, timeout=120)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_launcher_builds_one_environment_per_gpu():
    envs = DU.rank_environments(4, 29400, base={"PATH": "/bin", "RANK": "9"})
    assert [e["RANK"] for e in envs] == ["0", "1", "2", "3"] and [e["LOCAL_RANK"] for e in envs] == ["0", "1", "2", "3"]
    assert all(e["WORLD_SIZE"] == "4" and e["MASTER_ADDR"] == "127.0.0.1" and e["MASTER_PORT"] == "29400" for e in envs)
    assert all(e["PATH"] == "/bin" for e in envs)
    p = DU.free_port()
    assert 1024 <= p < 65536


def test_launcher_starts_n_ranks_that_rendezvous(tmp_path):
    """launch_ranks starts N children with a consistent rendezvous: each child joins a gloo group of the size it
    was told and writes its rank; rank 0's stdout is the launcher's."""
    script = tmp_path / "child.py"
    script.write_text(
        "import os, sys, torch.distributed as dist\n"
        "dist.init_process_group('gloo')\n"
        "assert dist.get_world_size() == int(os.environ['WORLD_SIZE']) == 3\n"
        "open(os.path.join(sys.argv[1], 'rank%d' % dist.get_rank()), 'w').write(os.environ['LOCAL_RANK'])\n"
        "dist.barrier(); dist.destroy_process_group()\n")
    assert DU.launch_ranks([str(script), str(tmp_path)], 3, timeout=120) == 0
    assert sorted(f for f in os.listdir(tmp_path) if f.startswith("rank")) == ["rank0", "rank1", "rank2"]
    assert (tmp_path / "rank2").read_text() == "2"
    failing = tmp_path / "bad.py"
    failing.write_text("import os, sys\nsys.exit(3 if os.environ['RANK'] == '1' else 0)\n")
    assert DU.launch_ranks([str(failing)], 2, timeout=60) == 3
