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


KEYS_WORKER = r"""
import argparse, json, os, sys
sys.path.insert(0, %r)
import numpy as np, torch
import bench, oracle
from workloads import bf16_bits, small_config
from paper_2603_02631_b200.sharded import ShardOps

class OracleOps(ShardOps):
    def shard_lse(self, sh):
        return torch.from_numpy(oracle.token_importance(bf16_bits(sh.q), [bf16_bits(k) for k in sh.k_layers])[1])
    def shard_importance(self, sh, lse_all):
        own = self.shard_lse(sh).double().numpy(); allr = lse_all.double().numpy()
        with np.errstate(divide="ignore"):
            extra = allr + np.log(-np.expm1(np.minimum(own - allr, 0.0)))
        return torch.from_numpy(oracle.token_importance(bf16_bits(sh.q), [bf16_bits(k) for k in sh.k_layers], extra_lse=extra)[0])
    def smooth(self, padded, w):
        return torch.from_numpy(oracle.avg_pool(padded.double().numpy(), w))
    def chunk_means(self, x, c):
        return torch.from_numpy(oracle.chunk_means(x.double().numpy(), c))
    def select_topk(self, scores, k):
        return torch.from_numpy(oracle.select_topk(scores.double().numpy(), k))
    def compact(self, kept, c, sh):
        out = oracle.compact(kept.numpy(), c, sh.hi - sh.lo, sh.token_ids.numpy().astype(np.int64),
                             sh.char_start.numpy().astype(np.int64), sh.char_end.numpy().astype(np.int64))
        return tuple(torch.from_numpy(np.asarray(x, dtype=np.int64)) for x in out)

cfg = small_config("keys", n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=64, n_lookahead=4, lengths=(1000,), chunk=32,
                   keep=(0.2,), rank=4, n_needles=2, n_strong=1, seed=3)
args = argparse.Namespace(steps=2, warmup=1, workload="keys")
bench.run_keys(args, ops=OracleOps(), device="cpu", backend="gloo", cfg=cfg)
"""


def test_bench_key_sharded_mode_runs_on_two_gloo_ranks():
    """bench.py --parallelism keys: the same driver code on two CPU ranks (gloo), the oracle standing in for the kernels;
    rank 0 prints the JSON line with the key-sharded configuration and the selection's size."""
    import json
    import subprocess
    import sys
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT="29561", WORLD_SIZE="2")
    procs = [subprocess.Popen([sys.executable, "-c", KEYS_WORKER % ROOT], env=dict(env, RANK=str(r)), stdout=subprocess.PIPE,
                              stderr=subprocess.PIPE, text=True) for r in range(2)]
    outs = [p.communicate(timeout=300) for p in procs]
    assert all(p.returncode == 0 for p in procs), [o[1][-2000:] for o in outs]
    line = json.loads(outs[0][0].strip().splitlines()[-1])
    assert line["config"]["parallelism"] == "keys x2" and line["scaling"] == "strong" and line["n_gpus"] == 2
    assert line["config"]["keys_per_rank"] == [512, 488] and line["value"] > 0
    assert line["kept_chunks"] == 7 and line["kept_tokens"] > 0 and line["spans"] >= 1
    assert outs[1][0].strip() == ""                       # only rank 0 prints
