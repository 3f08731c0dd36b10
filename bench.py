#!/usr/bin/env python
"""Throughput of the speculative-prefill scoring + selection path on synthetic long-context prompts.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl ours|reference] [--workload NAME]

One step = one pass of the whole path (score -> chunk pool -> top-k -> span compaction) over one batch
of the workload, inputs resident in HBM.  Prints ONE JSON line (rank 0).  With N > 1 (torchrun) every
rank runs the same workload shape on its own prompts: prompts are independent, so there is no
collective on the data path and the scaling is weak.

`--impl reference` times the CPU oracle (plain NumPy fp64, as it stands) on the host cores instead.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "prompt tokens scored+selected per second"
UNIT = "tokens/s"
DEFAULT_WORKLOAD = "long128k"          # N = 131072, the configuration the metric is quoted on
FALLBACK_HBM_GBS = 6650.0


# DRAM read + write bytes of one scoring launch, from the ncu capture summarised in profiles/.  Each entry names
# the SHA-256 of the kernel source it was taken from: once the source changes, the figure is reported as null.
NCU_TRAFFIC = {
    ("long128k", "fused"): {"bytes": 4 * (538341120 + 6759680), "source": "paper_2603_02631_b200/csrc/score_fused.cu",
                            "sha256": "97f49fa8be69ccf6ba8df7c7e8e1053a340d517c09eb1a11f3c31d6407593490",
                            "note": "captured on long128k_l4 (4 of 16 layers), scaled x4"},
}


def ncu_traffic(workload, path):
    import hashlib
    entry = NCU_TRAFFIC.get((workload, path))
    if entry is None:
        return None
    try:
        with open(os.path.join(ROOT, entry["source"]), "rb") as f:
            if hashlib.sha256(f.read()).hexdigest() != entry["sha256"]:
                return None
    except OSError:
        return None
    return entry["bytes"]


def parse_args():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=300)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD)
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--sustained-seconds", type=float, default=1.5,
                    help="length of the back-to-back spf_score loop behind the `sustained` record (0: skip)")
    ap.add_argument("--no-secondary", action="store_true", help="skip the scoring fractions of the other workloads")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--parallelism", default="prompts", choices=["prompts", "keys"],
                    help="prompts: every rank scores its own prompts (no collective); keys: ONE prompt's keys are split over "
                         "the ranks in chunk-aligned ranges and the ranks exchange row log-sum-exps, pooling halos, chunk "
                         "scores and selections")
    ap.add_argument("--score-path", default="auto", choices=["auto", "general", "fused"],
                    help="kernels behind spf_score: fused single-kernel path, general two-sweep path, or automatic")
    return ap.parse_args()


def hbm_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


# ----------------------------------------------------------------------------------------------- clocks
class ClockSampler:
    """nvidia-smi polled every 10 ms into a file; mark() remembers a position, stats(lo, hi) summarises a span."""
    FIELDS = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
              "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
              "clocks_event_reasons.sw_power_cap")
    NAMES = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.path = None

    def start(self):
        """Starts the sampling and waits (up to 5 s) for its first line."""
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(
                ["nvidia-smi", f"--query-gpu={self.FIELDS}", "--format=csv,noheader,nounits", "-lms", "10",
                 "-i", str(self.index)], stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
            deadline = time.time() + 5.0
            while time.time() < deadline and os.path.getsize(self.path) == 0:
                time.sleep(0.02)
        except Exception:
            self.proc = None

    def mark(self) -> int:
        """Number of samples written so far."""
        if self.proc is None:
            return 0
        try:
            return sum(1 for _ in open(self.path))
        except OSError:
            return 0

    def stop(self):
        if self.proc is None:
            return
        time.sleep(0.03)                                   # let the sample that covers the last launches land
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()

    def stats(self, lo: int = 0, hi: int = None):
        """Median SM clock, maximum clock and the throttle reasons seen in samples lo..hi (one before lo is included:
        it covers the start of the span)."""
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0, "power_w": None}
        if self.path is None:
            return out
        sm, mx, pw, reasons = [], [], [], set()
        try:
            lines = list(open(self.path))
        except OSError:
            return out
        for line in lines[max(lo - 1, 0):hi]:
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
                pw.append(float(parts[2]))
            except ValueError:
                continue
            for name, val in zip(self.NAMES, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(mx), reasons=sorted(reasons), samples=len(sm),
                       power_w=statistics.median(pw))
        return out

    def close(self):
        try:
            os.unlink(self.path)
        except Exception:
            pass


# ----------------------------------------------------------------------------------------------- oracle leg
def pick_sample_layers(cfg, prompt, budget_s=15.0):
    """How many layers the oracle can score in about `budget_s` seconds (times layer 0 to find out)."""
    import oracle
    from workloads import bf16_bits
    t0 = time.perf_counter()
    oracle.token_importance(bf16_bits(prompt.q[:1]), [bf16_bits(prompt.k[0])])
    per_layer = time.perf_counter() - t0
    return max(1, min(cfg.n_layers, int(budget_s / max(per_layer, 1e-3))))


def oracle_sample(cfg, prompt, keep, sample_layers):
    """Times the oracle on `sample_layers` of the prompt's layers (all keys) plus the full selection and
    scales the scoring time to all layers.  Returns (tokens/s, seconds of CPU work, description)."""
    import numpy as np
    import oracle
    from workloads import bf16_bits

    q = bf16_bits(prompt.q[:sample_layers])
    k = [bf16_bits(x) for x in prompt.k[:sample_layers]]
    ids, cs, ce = (t.cpu().numpy() for t in (prompt.token_ids, prompt.char_start, prompt.char_end))
    t0 = time.perf_counter()
    imp, _ = oracle.token_importance(q, k)
    t1 = time.perf_counter()
    scores = oracle.chunk_means(oracle.avg_pool(imp, cfg.pool_kernel), cfg.chunk)
    kept = oracle.select_topk(scores, oracle.keep_count(len(scores), keep))
    oracle.compact(kept, cfg.chunk, prompt.n_tokens, ids, cs, ce)
    t2 = time.perf_counter()
    t_full = (t1 - t0) * cfg.n_layers / sample_layers + (t2 - t1)
    desc = (f"oracle on layers 0..{sample_layers - 1} of {cfg.n_layers} (all {prompt.n_tokens} keys, all heads), "
            f"scoring time scaled x{cfg.n_layers / sample_layers:g}, plus the full selection")
    return prompt.n_tokens / t_full, t2 - t0, desc


def blas_threads():
    try:
        from threadpoolctl import threadpool_info
        return max([p.get("num_threads", 1) for p in threadpool_info()] or [1])
    except Exception:
        return os.cpu_count() or 1


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    import torch
    from workloads import CONFIGS, make_prompt
    cfg = CONFIGS[args.workload]
    prompt = make_prompt(cfg, 0, "cuda" if torch.cuda.is_available() else "cpu").to("cpu")
    keep = cfg.keep[0]
    steps = max(1, min(args.steps, 4))              # each step is seconds of CPU work
    sample_layers = pick_sample_layers(cfg, prompt, budget_s=60.0 / steps)
    vals, secs, desc = [], 0.0, ""
    for _ in range(steps):
        v, s, desc = oracle_sample(cfg, prompt, keep, sample_layers)
        vals.append(v)
        secs += s
    value = len(vals) / sum(1.0 / v for v in vals)
    cores = blas_threads()
    line = {
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": steps,
        "warmup": 1, "ms_per_step": 1e3 * cfg.lengths[0] / value, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name, "n_tokens": cfg.lengths[0], "n_layers": cfg.n_layers,
                   "n_q_heads": cfg.n_q_heads, "n_kv_heads": cfg.n_kv_heads, "head_dim": cfg.head_dim,
                   "n_lookahead": cfg.n_lookahead, "chunk": cfg.chunk, "keep": keep},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": cores, "kind": "oracle", "sample": desc},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }
    print(json.dumps(line), flush=True)


# ----------------------------------------------------------------------------------------------- multi-rank helpers
def rank_config(cfg, rank):
    """Weak scaling: every rank gets the same shapes and its own prompts (a different seed per rank)."""
    import dataclasses
    return cfg if rank == 0 else dataclasses.replace(cfg, seed=cfg.seed + 1000 * rank)


def max_over_ranks(values, device, world):
    """Element-wise maximum over all ranks of a list of floats (identity for a single process)."""
    if world <= 1:
        return list(values)
    import torch
    import torch.distributed as dist
    t = torch.tensor(list(values), device=device, dtype=torch.float64)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return t.tolist()


def whole_job_value(tokens_per_rank_step, steps, world, ms_total_max):
    """Aggregate tokens per second of all ranks: every rank processed the same number of tokens."""
    return world * tokens_per_rank_step * steps / (ms_total_max * 1e-3)


# ----------------------------------------------------------------------------------------------- our arm
def score_bytes(cfg):
    """Algorithmic bytes of one spf_score pass over the workload: K read once, Q, importance and lse written."""
    n_prompts = len(cfg.lengths)
    rows = cfg.n_layers * cfg.n_q_heads * cfg.n_lookahead
    return cfg.k_bytes() + n_prompts * rows * cfg.head_dim * 2 + 4 * sum(cfg.lengths) + n_prompts * rows * 4


def time_score_launches(spf, sel, prompts, launches, stream):
    """Average CUDA-event duration of `launches` passes of spf_score over `prompts` (one event pair around all)."""
    import torch
    bufs = [spf.binding.PromptBuffers(p.q, p.k, sel.importance[:p.n_tokens], sel.lse) for p in prompts]
    ws = sel._workspace(max(bufs, key=lambda b: b.importance.numel()))
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    for _ in range(launches):
        for bf in bufs:
            spf.spf_score([bf], ws, 0.0, sel.dev_status)
    b.record(stream)
    torch.cuda.synchronize()
    return a.elapsed_time(b) / launches


def fp8_workload(spf, dev, peak, stream, name="long128k"):
    """The long-context workload with its key cache in 8 bits (spf_score_fp8 on the path the library picks, and pinned to
    the general two-sweep kernels for comparison): the algorithmic bytes are the E4M3 cache read once, the scales, Q,
    importance and lse."""
    import torch
    from workloads import CONFIGS, make_prompt, quantize_keys_e4m3
    cfg = CONFIGS[name]
    try:
        prompt = make_prompt(cfg, 0, dev)
        k8, scales = quantize_keys_e4m3(prompt.k)
        q = prompt.q
        n = prompt.n_tokens
        del prompt
        torch.cuda.empty_cache()
        sel = spf.Selector(cfg.n_layers, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.n_lookahead, n, chunk=cfg.chunk,
                           pool_kernel=cfg.pool_kernel, device=dev)
        bufs = spf.Fp8PromptBuffers(q, k8, scales, sel.importance[:n], sel.lse)
        ws = torch.empty(spf.spf_score_fp8_workspace_bytes([bufs]), dtype=torch.uint8, device=dev)

        def timed(path):
            previous = spf.spf_set_score_path(path)
            try:
                sel.dev_status.zero_()
                for _ in range(3):
                    spf.spf_score_fp8([bufs], ws, 0.0, sel.dev_status)
                a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                a.record(stream)
                for _ in range(20):
                    spf.spf_score_fp8([bufs], ws, 0.0, sel.dev_status)
                b.record(stream)
                torch.cuda.synchronize()
            finally:
                spf.spf_set_score_path(previous)
            return a.elapsed_time(b) / 20, int(sel.dev_status.item())

        ms, status = timed(0)
        ms_general, _ = timed(1)
        rows = cfg.n_layers * cfg.n_q_heads * cfg.n_lookahead
        nbytes = cfg.k_bytes() // 2 + 4 * cfg.n_layers * cfg.n_kv_heads + rows * cfg.head_dim * 2 + 4 * n + 4 * rows
        gbs = nbytes / (ms * 1e-3) / 1e9
        return {"workload": name + "_fp8", "kernels": "path picked by the library (fused where the shape allows)", "ms_per_launch": ms,
                "achieved": gbs, "frac": gbs / peak, "algorithmic_bytes": nbytes, "tokens": n, "dev_status": status,
                "ms_per_launch_general_path": ms_general}
    except Exception as err:
        return {"workload": name + "_fp8", "error": str(err)[:200]}


def secondary_workloads(spf, dev, peak, stream, names=("small32k", "wide64k", "ragged8")):
    """Scoring fraction of the HBM rate on the other workload configurations (20 launches each after 3 warm-ups)."""
    import torch
    from workloads import CONFIGS, make_prompt
    out = [fp8_workload(spf, dev, peak, stream)]
    for name in names:
        cfg = CONFIGS[name]
        try:
            prompts = [make_prompt(cfg, i, dev) for i in range(len(cfg.lengths))]
            sel = spf.Selector(cfg.n_layers, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.n_lookahead, max(cfg.lengths),
                               chunk=cfg.chunk, pool_kernel=cfg.pool_kernel, device=dev)
            time_score_launches(spf, sel, prompts, 3, stream)
            ms = time_score_launches(spf, sel, prompts, 20, stream)
            status = int(sel.dev_status.item())
            gbs = score_bytes(cfg) / (ms * 1e-3) / 1e9
            out.append({"workload": name, "ms_per_launch": ms, "achieved": gbs, "frac": gbs / peak, "dev_status": status,
                        "tokens": sum(cfg.lengths)})
            del prompts, sel
            torch.cuda.empty_cache()
        except Exception as err:                           # e.g. not enough free memory for the 36 GB batch
            out.append({"workload": name, "error": str(err)[:200]})
    return out


def run_ours(args):
    import torch
    import torch.distributed as dist

    import paper_2603_02631_b200 as spf
    from workloads import CONFIGS, make_prompt

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    dev = f"cuda:{local_rank}"
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device(dev))

    cfg = CONFIGS[args.workload]
    keep = cfg.keep[0]
    n_prompts = len(cfg.lengths)
    # weak scaling: every rank gets the same shapes, its own prompts (distinct seeds via the prompt index)
    prompts = [make_prompt(rank_config(cfg, rank), i, dev) for i in range(n_prompts)]
    max_n = max(cfg.lengths)
    sel = spf.Selector(cfg.n_layers, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.n_lookahead, max_n,
                       chunk=cfg.chunk, pool_kernel=cfg.pool_kernel, device=dev)
    tokens_per_step = sum(cfg.lengths)
    stream = torch.cuda.current_stream()
    # which scoring kernels run: probe the fused path once on the first prompt (it refuses shapes it does not cover)
    want = {"auto": 0, "general": 1, "fused": 2}[args.score_path]
    fused = False
    if want != 1:
        spf.spf_set_score_path(2)
        try:
            p0 = prompts[0]
            sel.run(p0.q, p0.k, p0.token_ids, p0.char_start, p0.char_end, keep)
            fused = True
        except spf.SpfError:
            if want == 2:
                raise
    spf.spf_set_score_path(2 if fused else 1)
    # kernels per step: scoring per prompt (fused: score_fused; general: pack_q, score_lse, merge_lse, score_max), then
    # chunk_pool and select_compact (top-k + compaction) per prompt, or the three batched calls once per batch
    score_launches = 1 if fused else 4
    score_kernels = "score_fused_kernel" if fused else "pack_q + score_lse + merge_lse + score_max"
    if n_prompts > 1:
        bsel = spf.BatchSelector(cfg.n_layers, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.n_lookahead, cfg.lengths,
                                 chunk=cfg.chunk, pool_kernel=cfg.pool_kernel, device=dev)
        launches_per_step = score_launches * n_prompts + 3

        def step():
            bsel.run(prompts, keep)
    else:
        bsel = None
        launches_per_step = score_launches + 2           # chunk_pool, then top-k and compaction in one launch

        def step():
            p = prompts[0]
            sel.run(p.q, p.k, p.token_ids, p.char_start, p.char_end, keep)

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3)):
        step()
    barrier()

    # --- device-resident throughput ------------------------------------------------------------
    sampler = ClockSampler(local_rank)
    sampler.start()
    t_start, t_end = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    m0 = sampler.mark()
    t_start.record(stream)
    for _ in range(args.steps):
        step()
    t_end.record(stream)
    barrier()
    ms_total = t_start.elapsed_time(t_end)
    status = int((bsel or sel).dev_status.item())
    if status != 0:
        raise RuntimeError(f"device status {status} ({spf.spf_status_string(status)}) after the timed region")

    # --- the scoring call on its own (same launches, events around spf_score only) --------------------
    bufs = [spf.binding.PromptBuffers(p.q, p.k, sel.importance[:p.n_tokens], sel.lse) for p in prompts]
    ws = sel._workspace(bufs[cfg.lengths.index(max_n)])
    events = []
    for it in range(args.steps):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record(stream)
        for bf in bufs:
            spf.spf_score([bf], ws, 0.0, sel.dev_status)
        b.record(stream)
        events.append((a, b))
    torch.cuda.synchronize()
    m1 = sampler.mark()
    score_ms = [a.elapsed_time(b) for a, b in events]
    score_ms_avg = sum(score_ms) / len(score_ms)

    # --- sustained: the scoring call back to back for a second or more (the power-capped steady state) ------------
    sustained = None
    if args.sustained_seconds > 0:
        launches = max(10, int(args.sustained_seconds * 1e3 / score_ms_avg))
        m2 = sampler.mark()
        ms = time_score_launches(spf, sel, prompts, launches, stream)
        m3 = sampler.mark()
        sustained = {"launches": launches, "ms_per_launch": ms}
    sampler.stop()
    clocks = sampler.stats(m0, m1)
    if sustained:
        c = sampler.stats(m2, m3)
        sustained.update(sm_mhz=c["sm_mhz"], power_w=c["power_w"], reasons=c["reasons"], samples=c["samples"],
                         ms_x_mhz=(sustained["ms_per_launch"] * c["sm_mhz"]) if c["sm_mhz"] else None)
    sampler.close()

    # --- end to end: host buffers through the C entry point spf_compress_host ---------------------------------------
    e2e = None
    if args.e2e_steps > 0:
        host = []
        h2d = 0
        for p in prompts:
            hp = dict(q=p.q.cpu().pin_memory(), k=[x.cpu().pin_memory() for x in p.k],
                      ids=p.token_ids.cpu().pin_memory(), cs=p.char_start.cpu().pin_memory(),
                      ce=p.char_end.cpu().pin_memory())
            h2d += hp["q"].numel() * 2 + sum(x.numel() * 2 for x in hp["k"]) + 3 * 4 * p.n_tokens
            host.append(hp)
        del prompts, bufs, bsel
        torch.cuda.empty_cache()

        def e2e_step():
            d2h = 0
            for hp in host:
                out = sel.run_host(hp["q"], hp["k"], hp["ids"], hp["cs"], hp["ce"], keep)
                d2h += 16 + 4 + sum(v.nbytes for v in out.values())
            return d2h

        e2e_step()
        barrier()
        t0 = time.perf_counter()
        d2h = 0
        for _ in range(args.e2e_steps):
            d2h = e2e_step()
        barrier()
        e2e_s = time.perf_counter() - t0
        e2e = {"seconds": e2e_s, "h2d": h2d, "d2h": d2h}
        del host
        sel._arena = None
        torch.cuda.empty_cache()

    # --- reduce over ranks --------------------------------------------------------------------------
    ms_total, e2e_s_max, score_ms_avg = max_over_ranks([ms_total, e2e["seconds"] if e2e else 0.0, score_ms_avg], dev, world)
    if e2e:
        e2e["seconds"] = e2e_s_max
    if rank != 0:
        if world > 1:
            dist.destroy_process_group()
        return

    value = whole_job_value(tokens_per_step, args.steps, world, ms_total)
    peak, peak_kind = hbm_peak()
    k_bytes = cfg.k_bytes()
    sbytes = score_bytes(cfg)
    achieved = sbytes / (score_ms_avg * 1e-3) / 1e9
    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_total / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "bf16 in, f32 accumulate/softmax", "data": "synthetic",
        "config": {"workload": cfg.name, "n_prompts_per_gpu": n_prompts, "n_tokens": list(cfg.lengths),
                   "n_layers": cfg.n_layers, "n_q_heads": cfg.n_q_heads, "n_kv_heads": cfg.n_kv_heads,
                   "head_dim": cfg.head_dim, "n_lookahead": cfg.n_lookahead, "chunk": cfg.chunk, "keep": keep,
                   "pool_kernel": cfg.pool_kernel, "k_cache_bytes": k_bytes,
                   "l2": "inputs larger than L2 (key cache streamed every step)", "parallelism": f"prompts x{world}"},
        "clocks": {"sm_mhz": clocks["sm_mhz"], "sm_max_mhz": clocks["sm_max_mhz"], "reasons": clocks["reasons"],
                   "samples": clocks["samples"], "span": "timed steps + the spf_score-only launches, 10 ms period"},
        "gpu_launches": launches_per_step * args.steps,
        "roofline": {"bound": "hbm", "kernel": f"spf_score ({score_kernels})",
                     "achieved": achieved, "peak": peak, "peak_kind": f"of {peak_kind}", "unit": "GB/s",
                     "frac": achieved / peak, "traffic": ncu_traffic(cfg.name, "fused" if fused else "general"), "ms_per_launch": score_ms_avg,
                     "algorithmic_bytes": sbytes},
    }
    if sustained:
        gbs = sbytes / (sustained["ms_per_launch"] * 1e-3) / 1e9
        sustained.update(achieved=gbs, frac=gbs / peak)
        line["sustained"] = sustained
    if e2e:
        line["e2e"] = {"value": world * tokens_per_step * args.e2e_steps / e2e["seconds"], "unit": UNIT,
                       "h2d_bytes_per_step": e2e["h2d"], "d2h_bytes_per_step": e2e["d2h"], "steps": args.e2e_steps,
                       "api": "spf_compress_host (C ABI, pinned host buffers, device arena reused between calls)"}
    if world == 1 and not args.no_secondary and cfg.name == DEFAULT_WORKLOAD:
        line["secondary"] = secondary_workloads(spf, dev, peak, stream)
    if world == 1 and not args.no_cpu_baseline:
        cpu_prompt = make_prompt(cfg, 0, dev).to("cpu")
        v, secs, desc = oracle_sample(cfg, cpu_prompt, keep, pick_sample_layers(cfg, cpu_prompt))
        line["cpu_baseline"] = {"value": v, "unit": UNIT, "cores": blas_threads(), "kind": "oracle", "sample": desc,
                                "cpu_seconds": secs}
    print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


# ----------------------------------------------------------------------------------------------- one prompt over N ranks
def run_keys(args, ops=None, device=None, backend="nccl", cfg=None):
    """One prompt whose keys are split over the ranks (paper_2603_02631_b200.sharded): a step is sharded_select on every
    rank, i.e. shard log-sum-exps -> all-reduce -> shard importance -> halo / chunk-score / selection all-gathers.  The
    total work is fixed as the ranks grow ("strong" scaling).  `ops`, `device`, `backend` and `cfg` exist so that the same
    code can be driven on CPU ranks (gloo) with a stand-in for the kernels; the defaults are the CUDA library over NCCL."""
    import torch
    import torch.distributed as dist
    from paper_2603_02631_b200.sharded import LibraryOps, Shard, shard_bounds, sharded_select
    from workloads import CONFIGS, make_prompt

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    on_gpu = device is None
    if on_gpu:
        torch.cuda.set_device(local_rank)
        device = f"cuda:{local_rank}"
    own_group = not dist.is_initialized()
    if own_group:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")     # a bare `python bench.py --parallelism keys` is a one-rank group
        os.environ.setdefault("MASTER_PORT", "29577")
        if on_gpu:
            dist.init_process_group(backend, rank=rank, world_size=world, device_id=torch.device(device))
        else:
            dist.init_process_group(backend, rank=rank, world_size=world)
    cfg = cfg or CONFIGS[args.workload]
    if len(cfg.lengths) != 1:
        raise SystemExit("--parallelism keys splits ONE prompt: pick a single-prompt workload")
    keep = cfg.keep[0]
    prompt = make_prompt(cfg, 0, device)                    # the same seeded bytes on every rank; each keeps its range
    n = prompt.n_tokens
    lo, hi = shard_bounds(n, world, cfg.chunk)[rank]
    shard = Shard(lo, hi, prompt.q, [k[:, lo:hi].contiguous() for k in prompt.k], prompt.token_ids[lo:hi].contiguous(),
                  prompt.char_start[lo:hi].contiguous(), prompt.char_end[lo:hi].contiguous())
    del prompt
    if on_gpu:
        torch.cuda.empty_cache()
    if ops is None:
        import paper_2603_02631_b200 as spf
        ops = LibraryOps()
        k_count = spf.spf_keep_count((n + cfg.chunk - 1) // cfg.chunk, keep)
    else:
        import math
        n_chunks = (n + cfg.chunk - 1) // cfg.chunk
        k_count = max(1, min(n_chunks, math.ceil(keep * n_chunks - 1e-9)))

    def step():
        return sharded_select(shard, n, k_count, ops, chunk=cfg.chunk, pool_kernel=cfg.pool_kernel)

    def barrier():
        dist.barrier()
        if on_gpu:
            torch.cuda.synchronize()

    for _ in range(max(args.warmup, 3) if on_gpu else args.warmup):
        step()
    barrier()
    if on_gpu:
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
    t0 = time.perf_counter()
    last = None
    for _ in range(args.steps):
        last = step()
    if on_gpu:
        b.record()
    barrier()
    ms_total = a.elapsed_time(b) if on_gpu else (time.perf_counter() - t0) * 1e3
    (ms_total,) = max_over_ranks([ms_total], device, world)
    line = None
    if rank == 0:
        line = {
            "metric": METRIC, "value": n * args.steps / (ms_total * 1e-3), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms_total / args.steps, "higher_is_better": True, "scaling": "strong",
            "vs_baseline": None, "dtype": "bf16 in, f32 accumulate/softmax", "data": "synthetic",
            "config": {"workload": cfg.name, "n_tokens": [n], "n_layers": cfg.n_layers, "n_q_heads": cfg.n_q_heads,
                       "n_kv_heads": cfg.n_kv_heads, "head_dim": cfg.head_dim, "n_lookahead": cfg.n_lookahead, "chunk": cfg.chunk,
                       "keep": keep, "pool_kernel": cfg.pool_kernel, "parallelism": f"keys x{world}",
                       "keys_per_rank": [hi_ - lo_ for lo_, hi_ in shard_bounds(n, world, cfg.chunk)],
                       "exchange": "max + sum all-reduce of L*Hq*m floats, all-gathers of pooling halos, chunk scores, selections",
                       "kernels": "spf_score_shard_lse_ex + spf_score_shard_apply_ex (the fused kernel, one visit per call, where the shape allows)" if on_gpu else "stand-in"},
            "kept_chunks": int(last.kept.numel()), "kept_tokens": int(last.ids.numel()), "spans": int(last.tok_spans.shape[0]),
            "gpu_launches": (9 * args.steps) if on_gpu else 0,
        }
        print(json.dumps(line), flush=True)
    if own_group:
        dist.destroy_process_group()
    return line


def run_fp8_line(args):
    """`--workload <name>_fp8`: the whole path on one prompt of <name> whose key cache is held as E4M3 bytes
    (Selector.run_fp8: spf_score_fp8 -> spf_chunk_pool -> spf_select_compact), device-resident, one GPU.  The roofline's
    bytes are this format's own: the 8-bit cache read once + scales + Q + importance + lse."""
    import torch
    import paper_2603_02631_b200 as spf
    from workloads import CONFIGS, make_prompt, quantize_keys_e4m3
    torch.cuda.set_device(0)
    dev = "cuda:0"
    cfg = CONFIGS[args.workload[:-len("_fp8")]]
    keep = cfg.keep[0]
    prompt = make_prompt(cfg, 0, dev)
    k8, scales = quantize_keys_e4m3(prompt.k)
    q, ids, cs, ce, n = prompt.q, prompt.token_ids, prompt.char_start, prompt.char_end, prompt.n_tokens
    del prompt
    torch.cuda.empty_cache()
    sel = spf.Selector(cfg.n_layers, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.n_lookahead, n, chunk=cfg.chunk,
                       pool_kernel=cfg.pool_kernel, device=dev)
    spf.spf_set_score_path({"auto": 0, "general": 1, "fused": 2}[args.score_path])
    stream = torch.cuda.current_stream()
    for _ in range(max(args.warmup, 3)):
        sel.run_fp8(q, k8, scales, ids, cs, ce, keep)
    torch.cuda.synchronize()
    sampler = ClockSampler(0)
    sampler.start()
    m0 = sampler.mark()
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record(stream)
    for _ in range(args.steps):
        sel.run_fp8(q, k8, scales, ids, cs, ce, keep)
    b.record(stream)
    torch.cuda.synchronize()
    ms_step = a.elapsed_time(b) / args.steps
    bufs = spf.Fp8PromptBuffers(q, k8, scales, sel.importance[:n], sel.lse)
    a.record(stream)
    for _ in range(args.steps):
        spf.spf_score_fp8([bufs], sel.workspace, 0.0, sel.dev_status)
    b.record(stream)
    torch.cuda.synchronize()
    m1 = sampler.mark()
    sampler.stop()
    clocks = sampler.stats(m0, m1)
    sampler.close()
    status = int(sel.dev_status.item())
    if status != 0:
        raise RuntimeError(f"device status {status} ({spf.spf_status_string(status)})")
    ms_score = a.elapsed_time(b) / args.steps
    rows = cfg.n_layers * cfg.n_q_heads * cfg.n_lookahead
    nbytes = cfg.k_bytes() // 2 + 4 * cfg.n_layers * cfg.n_kv_heads + rows * cfg.head_dim * 2 + 4 * n + 4 * rows
    peak, peak_kind = hbm_peak()
    gbs = nbytes / (ms_score * 1e-3) / 1e9
    print(json.dumps({
        "metric": METRIC, "value": n / (ms_step * 1e-3), "unit": UNIT, "n_gpus": 1, "steps": args.steps,
        "warmup": max(args.warmup, 3), "ms_per_step": ms_step, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
        "dtype": "e4m3 keys, two-term e4m3 queries (bf16 in), f32 accumulate/softmax", "data": "synthetic",
        "config": {"workload": args.workload, "n_tokens": [n], "n_layers": cfg.n_layers, "n_q_heads": cfg.n_q_heads,
                   "n_kv_heads": cfg.n_kv_heads, "head_dim": cfg.head_dim, "n_lookahead": cfg.n_lookahead, "chunk": cfg.chunk,
                   "keep": keep, "k_cache_bytes": cfg.k_bytes() // 2, "score_path": args.score_path,
                   "l2": "inputs larger than L2 (key cache streamed every step)"},
        "clocks": {"sm_mhz": clocks["sm_mhz"], "sm_max_mhz": clocks["sm_max_mhz"], "reasons": clocks["reasons"],
                   "samples": clocks["samples"]},
        "gpu_launches": 4 * args.steps, "e2e": None,
        "roofline": {"bound": "hbm", "kernel": "spf_score_fp8", "achieved": gbs, "peak": peak, "peak_kind": f"of {peak_kind}",
                     "unit": "GB/s", "frac": gbs / peak, "traffic": None, "ms_per_launch": ms_score, "algorithmic_bytes": nbytes},
    }), flush=True)


def main():
    args = parse_args()
    if args.impl == "reference":
        run_reference(args)
    elif args.workload.endswith("_fp8"):
        run_fp8_line(args)
    elif args.parallelism == "keys":
        run_keys(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
