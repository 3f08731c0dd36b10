"""One long prompt over several ranks (key-sharded), on CPU: gloo ranks run the collectives and the stitching of
paper_2603_02631_b200.sharded with the oracle standing in for the kernels, and every rank must end with exactly the
selection the oracle gives for the whole prompt in one process."""
import json
import os
import subprocess
import sys
import textwrap

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = textwrap.dedent("""
    import os, sys, json
    sys.path.insert(0, %r)
    import numpy as np, torch, torch.distributed as dist
    import oracle
    from workloads import bf16_bits, make_prompt, small_config
    from paper_2603_02631_b200.sharded import Shard, ShardOps, shard_bounds, sharded_select

    class OracleOps(ShardOps):
        # the oracle as the per-rank arithmetic: a shard's rows see the other ranks' keys as an extra denominator term
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

    rank, world = int(os.environ["RANK"]), int(os.environ["WORLD_SIZE"])
    dist.init_process_group("gloo", rank=rank, world_size=world)
    results = []
    for (n, chunk, keep, w) in json.loads(os.environ["CASES"]):
        cfg = small_config("shard", n_layers=2, n_q_heads=4, n_kv_heads=2, head_dim=64, n_lookahead=4, lengths=(n,), chunk=chunk,
                           rank=4, n_needles=2 if n >= 200 else 0, n_strong=1, needle_len=(4, 16), seed=n + chunk)
        p = make_prompt(cfg, 0, "cpu")                       # the same bytes on every rank (seeded)
        lo, hi = shard_bounds(n, world, chunk)[rank]
        sh = Shard(lo, hi, p.q, [k[:, lo:hi].contiguous() for k in p.k], p.token_ids[lo:hi], p.char_start[lo:hi], p.char_end[lo:hi])
        k = oracle.keep_count((n + chunk - 1) // chunk, keep)
        got = sharded_select(sh, n, k, OracleOps(), chunk=chunk, pool_kernel=w)
        ref = oracle.compress(bf16_bits(p.q), [bf16_bits(x) for x in p.k], p.token_ids.numpy(), p.char_start.numpy(),
                              p.char_end.numpy(), chunk=chunk, keep=keep, pool_kernel=w)
        imp_err = float(np.abs(got.importance_local.double().numpy() - ref["importance"][lo:hi]).max()) if hi > lo else 0.0
        results.append(dict(kept=got.kept.tolist() == ref["kept"].tolist(), ids=got.ids.tolist() == ref["ids"].tolist(),
                            pos=got.pos.tolist() == ref["pos"].tolist(), tok=got.tok_spans.tolist() == ref["tok_spans"].tolist(),
                            ch=got.char_spans.tolist() == ref["char_spans"].tolist(), imp_err=imp_err,
                            lse_err=float(np.abs(got.lse_all.double().numpy() - ref["lse"]).max()), bounds=[lo, hi]))
    dist.barrier()
    print(json.dumps(results))
    dist.destroy_process_group()
""") % ROOT

CASES = [
    (1000, 32, 0.2, 13),     # ordinary: boundaries inside the prompt, kept chunks on both sides of them
    (997, 32, 0.9, 13),      # almost everything kept: spans run across rank boundaries and must merge; partial last chunk
    (20, 2, 0.5, 13),        # ranks shorter than the pooling half-width: halos come from several neighbours
    (5, 4, 1.0, 13),         # fewer chunks than ranks can fill: some ranks hold nothing
    (300, 8, 0.1, 1),        # no smoothing
]


@pytest.mark.parametrize("world,port", [(2, 29551), (3, 29552), (4, 29553)])
def test_key_sharded_selection_equals_the_single_process_oracle(world, port):
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), WORLD_SIZE=str(world), CASES=json.dumps(CASES))
    procs = [subprocess.Popen([sys.executable, "-c", WORKER], env=dict(env, RANK=str(r)), stdout=subprocess.PIPE,
                              stderr=subprocess.PIPE, text=True) for r in range(world)]
    outs = [p.communicate(timeout=300) for p in procs]
    assert all(p.returncode == 0 for p in procs), [o[1][-2000:] for o in outs]
    for r, (out, _) in enumerate(outs):
        for case, res in zip(CASES, json.loads(out.strip().splitlines()[-1])):
            assert res["kept"] and res["ids"] and res["pos"] and res["tok"] and res["ch"], (world, r, case, res)
            # the exchange runs in fp32 (what the devices hold): values agree to fp32 rounding, the selection exactly
            assert res["imp_err"] < 1e-6 and res["lse_err"] < 1e-5, (world, r, case, res)


def test_shard_bounds_are_chunk_aligned_and_cover_the_prompt():
    from paper_2603_02631_b200.sharded import shard_bounds
    for n, world, chunk in [(1000, 3, 32), (131072, 8, 32), (5, 4, 4), (64, 2, 64), (1, 3, 32)]:
        b = shard_bounds(n, world, chunk)
        assert b[0][0] == 0 and b[-1][1] == n and all(x[1] == y[0] for x, y in zip(b, b[1:]))
        assert all(lo % chunk == 0 or lo == n for lo, _ in b)
