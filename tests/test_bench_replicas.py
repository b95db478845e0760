"""The N > 1 path of bench.py is "replicas only": no data-path collective, the job's figures are the
slowest rank's time and the sum of the ranks' tokens.  Checked here with two gloo ranks on CPU."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from helpers import ROOT


def _worker(rank, world, port, q):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    sys.path.insert(0, ROOT)
    import bench
    ms, tokens = bench.reduce_over_ranks(10.0 + 5.0 * rank, 100 + rank, "cpu")
    q.put((rank, ms, tokens, bench.shard_of_rank(rank)["prompt_seed_offset"]))
    dist.barrier()
    dist.destroy_process_group()


def test_two_replicas_over_gloo():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, 29641, q)) for r in range(2)]
    for p in procs:
        p.start()
    got = sorted(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [g[1] for g in got] == [15.0, 15.0]          # max over ranks
    assert [g[2] for g in got] == [201, 201]            # whole-job tokens
    assert got[0][3] != got[1][3]                       # different prompts per replica


def test_without_process_group_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.reduce_over_ranks(3.5, 7, "cpu") == (3.5, 7)


def test_reference_arm_runs_on_rank_zero_only():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    r = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--steps", "1"],
                       capture_output=True, text=True, env=env, timeout=300)
    assert r.returncode == 0 and r.stdout.strip() == ""


def test_step_bytes_matches_hand_count():
    sys.path.insert(0, ROOT)
    import bench
    from paper_2403_09919_b200 import synth
    sb = bench.step_bytes(synth.CONFIGS["7b"], 900)
    assert abs(sb["llm"] / 1e9 - 13.21) < 0.01 and abs(sb["drafter"] / 1e9 - 4.23) < 0.01
    assert abs(sb["kv"] / 900 / 1e6 - 0.524) < 0.001
