"""The N > 1 logic of bench.py on CPU: two gloo ranks, max-over-ranks timing, per-rank prompts, whole-job value."""
import os
import subprocess
import sys
import textwrap

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import torch, torch.distributed as dist
    import bench
    from workloads import CONFIGS, make_prompt
    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo", rank=rank, world_size=world)
    # every rank measured something else: the slowest rank defines the time
    got = bench.max_over_ranks([10.0 + rank, 5.0 - rank, 1.0], "cpu", world)
    cfg = bench.rank_config(CONFIGS["tiny"], rank)
    p = make_prompt(cfg, 0, "cpu")
    digest = int(p.q.view(torch.int16).to(torch.int64).sum().item())
    gathered = [None] * world
    dist.all_gather_object(gathered, (cfg.lengths, cfg.seed, digest))
    dist.barrier()
    if rank == 0:
        print(json.dumps({"max": got, "ranks": gathered, "value": bench.whole_job_value(2048, 10, world, got[0])}))
    dist.destroy_process_group()
""") % ROOT


def test_two_gloo_ranks_share_nothing_but_the_clock():
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29541", WORLD_SIZE="2")
    procs = [subprocess.Popen([sys.executable, "-c", WORKER], env=dict(env, RANK=str(r)), stdout=subprocess.PIPE,
                              stderr=subprocess.PIPE, text=True) for r in range(2)]
    outs = [p.communicate(timeout=120) for p in procs]
    assert all(p.returncode == 0 for p in procs), outs
    import json
    line = json.loads(outs[0][0].strip().splitlines()[-1])
    assert line["max"] == [11.0, 5.0, 1.0]
    (len0, seed0, dig0), (len1, seed1, dig1) = line["ranks"]
    assert len0 == len1 and seed0 != seed1 and dig0 != dig1          # same shapes, different prompts
    assert abs(line["value"] - 2 * 2048 * 10 / 11e-3) < 1e-6          # tokens of both ranks over the slowest rank's time
    assert outs[1][0].strip() == ""                                    # only rank 0 prints


def test_reference_arm_is_silent_on_other_ranks():
    env = dict(os.environ, RANK="1", WORLD_SIZE="2")
    out = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--gpus", "2"], env=env,
                         capture_output=True, text=True, timeout=120)
    assert out.returncode == 0 and out.stdout.strip() == ""
