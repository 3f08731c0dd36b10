"""One long prompt over several ranks: each rank holds a contiguous, chunk-aligned range of the prompt's keys.

Host-side orchestration only (torch.distributed collectives between the library's calls).  Exchanges per prompt:
one max and one sum all-reduce of L*Hq*m floats (row log-sum-exps), one all-gather of the pooling halos
(pool_kernel - 1 floats per rank), one all-gather of the chunk scores, one all-gather of the per-rank selections.
The arithmetic sits behind a small `ShardOps` interface: `LibraryOps` calls the CUDA library, the CPU tests plug
in a stand-in so that the collectives and the stitching can be exercised with the gloo backend.
"""
from __future__ import annotations

import dataclasses
from typing import List, Optional, Sequence, Tuple

import torch
import torch.distributed as dist


@dataclasses.dataclass
class Shard:
    """What one rank holds of the prompt: keys [lo, hi) of every layer, and the token arrays of the same range."""
    lo: int
    hi: int
    q: torch.Tensor                      # [L, Hq, m, d], the same on every rank
    k_layers: Sequence[torch.Tensor]     # L tensors [Hkv, hi - lo, d]
    token_ids: torch.Tensor              # int32 [hi - lo]
    char_start: torch.Tensor             # int32 [hi - lo], character offsets in the whole prompt
    char_end: torch.Tensor


def shard_bounds(n_tokens: int, world: int, chunk: int) -> List[Tuple[int, int]]:
    """Contiguous key ranges, one per rank, every boundary a multiple of the chunk size (only the last range may end
    inside a chunk); ranks beyond the number of chunks get empty ranges."""
    n_chunks = (n_tokens + chunk - 1) // chunk
    per, extra = divmod(n_chunks, world)
    out, c0 = [], 0
    for r in range(world):
        c1 = c0 + per + (1 if r < extra else 0)
        out.append((min(c0 * chunk, n_tokens), min(c1 * chunk, n_tokens)))
        c0 = c1
    return out


class ShardOps:
    """The per-rank arithmetic.  All tensors live on the rank's device."""

    def shard_lse(self, shard: Shard) -> torch.Tensor:              # fp32 [L, Hq, m]: log-sum-exp over the shard's keys
        raise NotImplementedError

    def shard_importance(self, shard: Shard, lse_all: torch.Tensor) -> torch.Tensor:   # fp32 [hi - lo]
        raise NotImplementedError

    def smooth(self, padded: torch.Tensor, pool_kernel: int) -> torch.Tensor:          # zero-padded average pool, same length
        raise NotImplementedError

    def chunk_means(self, smoothed: torch.Tensor, chunk: int) -> torch.Tensor:
        raise NotImplementedError

    def select_topk(self, scores: torch.Tensor, k: int) -> torch.Tensor:               # int64 ascending chunk indices
        raise NotImplementedError

    def compact(self, kept_local: torch.Tensor, chunk: int, shard: Shard):
        """-> (ids int64 [n_kept], pos int64 [n_kept] local, tok_spans int64 [s, 2] local, char_spans int64 [s, 2])."""
        raise NotImplementedError


class LibraryOps(ShardOps):
    """ShardOps on the CUDA library (one GPU per rank)."""

    def __init__(self, softmax_scale: float = 0.0):
        from . import binding
        self.b = binding
        self.scale = softmax_scale
        self.ws: Optional[torch.Tensor] = None
        self.status: Optional[torch.Tensor] = None

    def _status(self, device) -> torch.Tensor:
        if self.status is None:
            self.status = torch.zeros(1, dtype=torch.int32, device=device)
        self.status.zero_()
        return self.status

    def _bufs(self, shard: Shard, importance, lse):
        bufs = self.b.PromptBuffers(shard.q, shard.k_layers, importance, lse)
        need = self.b.spf_score_workspace_bytes([bufs], self.scale)
        if self.ws is None or self.ws.numel() < need:
            self.ws = torch.empty(need, dtype=torch.uint8, device=shard.q.device)
        return bufs

    def shard_lse(self, shard):
        L, Hq, m, _ = shard.q.shape
        n = shard.hi - shard.lo
        lse = torch.empty(L * Hq * m, dtype=torch.float32, device=shard.q.device)
        scratch = torch.empty(n, dtype=torch.float32, device=shard.q.device)
        bufs = self._bufs(shard, scratch, lse)
        st = self._status(shard.q.device)
        self.b.spf_score_shard_lse_ex(bufs, self.ws, st, self.scale)
        if int(st.item()) != 0:                              # a row sum beyond fp32 or a wait that ran out: the general kernels
            self.b.spf_score_shard_lse(bufs, self.ws, self.scale)
        return lse.view(L, Hq, m)

    def shard_importance(self, shard, lse_all):
        n = shard.hi - shard.lo
        imp = torch.empty(n, dtype=torch.float32, device=shard.q.device)
        bufs = self._bufs(shard, imp, None)
        st = self._status(shard.q.device)
        self.b.spf_score_shard_apply_ex(bufs, lse_all.contiguous(), self.ws, st, self.scale)
        if int(st.item()) != 0:
            self.b.spf_score_shard_apply(bufs, lse_all.contiguous(), self.ws, self.scale)
        return imp

    def smooth(self, padded, pool_kernel):
        out = torch.empty_like(padded)
        self.b.spf_chunk_pool(padded, pool_kernel, 1, out)       # chunk 1: the smoothed value of every token
        return out

    def chunk_means(self, smoothed, chunk):
        n = smoothed.numel()
        out = torch.empty((n + chunk - 1) // chunk, dtype=torch.float32, device=smoothed.device)
        self.b.spf_chunk_pool(smoothed.contiguous(), 1, chunk, out)   # kernel 1: plain chunk means
        return out

    def select_topk(self, scores, k):
        kept = torch.empty(k, dtype=torch.int32, device=scores.device)
        self.b.spf_select_topk(scores.contiguous(), scores.numel(), k, kept)
        return kept.to(torch.int64)

    def compact(self, kept_local, chunk, shard):
        n, k = shard.hi - shard.lo, kept_local.numel()
        dev = shard.q.device
        ids = torch.empty(max(min(k * chunk, n), 1), dtype=torch.int32, device=dev)
        pos = torch.empty_like(ids)
        tok = torch.empty((max(k, 1), 2), dtype=torch.int32, device=dev)
        ch = torch.empty_like(tok)
        counts = torch.zeros(2, dtype=torch.int64, device=dev)
        if k > 0:
            self.b.spf_compact_spans(kept_local.to(torch.int32).contiguous(), k, chunk, n, shard.token_ids, shard.char_start,
                                     shard.char_end, ids, pos, tok, ch, counts)
        n_kept, n_spans = (int(x) for x in counts.cpu())
        return ids[:n_kept].long(), pos[:n_kept].long(), tok[:n_spans].long(), ch[:n_spans].long()


@dataclasses.dataclass
class ShardedSelection:
    """The whole prompt's selection, identical on every rank (host tensors)."""
    k: int
    kept: torch.Tensor         # int64 [k] chunk indices, ascending
    ids: torch.Tensor          # int64 [n_kept]
    pos: torch.Tensor          # int64 [n_kept] positions in the whole prompt
    tok_spans: torch.Tensor    # int64 [n_spans, 2]
    char_spans: torch.Tensor   # int64 [n_spans, 2]
    importance_local: torch.Tensor   # this rank's importance values (device of the shard)
    lse_all: torch.Tensor            # [L, Hq, m]


def _all_gather_padded(x: torch.Tensor, group) -> List[torch.Tensor]:
    """all_gather of 1-D tensors of different lengths (lengths first, then the data padded to the longest)."""
    world = dist.get_world_size(group)
    n = torch.tensor([x.numel()], dtype=torch.int64, device=x.device)
    sizes = [torch.zeros_like(n) for _ in range(world)]
    dist.all_gather(sizes, n, group=group)
    longest = max(int(s) for s in sizes)
    buf = torch.zeros(max(longest, 1), dtype=x.dtype, device=x.device)
    buf[:x.numel()] = x
    bufs = [torch.zeros_like(buf) for _ in range(world)]
    dist.all_gather(bufs, buf, group=group)
    return [b[:int(s)] for b, s in zip(bufs, sizes)]


def sharded_select(shard: Shard, n_tokens: int, keep_count: int, ops: ShardOps, chunk: int = 32, pool_kernel: int = 13,
                   group=None) -> ShardedSelection:
    """Scores and selects one prompt whose keys are spread over the ranks of `group` (ranges from shard_bounds).

    Every rank ends with the same selection.  `keep_count` is k, the number of chunks to keep (spf_keep_count).
    A rank whose range is empty (more ranks than chunks) takes part in the collectives with empty contributions.
    """
    rank, world = dist.get_rank(group), dist.get_world_size(group)
    dev = shard.q.device
    n_local = shard.hi - shard.lo
    half = pool_kernel // 2
    L, Hq, m, _ = shard.q.shape

    # 1. softmax denominators: log-sum-exp over the local keys, then log sum_r exp(lse_r) over the ranks
    lse_local = ops.shard_lse(shard).float() if n_local > 0 else torch.full((L, Hq, m), float("-inf"), device=dev)
    mx = lse_local.clone()
    dist.all_reduce(mx, op=dist.ReduceOp.MAX, group=group)
    total = torch.exp(lse_local - mx)
    dist.all_reduce(total, op=dist.ReduceOp.SUM, group=group)
    lse_all = mx + torch.log(total)

    # 2. importance of the local keys
    imp = ops.shard_importance(shard, lse_all).float() if n_local > 0 else torch.zeros(0, device=dev)

    # 3. smoothing needs pool_kernel / 2 values from each neighbour: gather every rank's first and last `half` values
    edge = torch.zeros(2 * half, dtype=torch.float32, device=dev)
    if half > 0 and n_local > 0:
        take = min(half, n_local)
        edge[:take] = imp[:take]                       # head, left-aligned
        edge[2 * half - take:] = imp[n_local - take:]  # tail, right-aligned
    edges = [torch.zeros_like(edge) for _ in range(world)]
    dist.all_gather(edges, edge, group=group)
    bounds = shard_bounds(n_tokens, world, chunk)
    scores_local = torch.zeros(0, dtype=torch.float32, device=dev)
    if n_local > 0:
        # the `half` importance values on either side of the local range, taken from as many neighbours as it needs
        # (a neighbour may hold fewer than `half` tokens); zeros beyond the ends of the prompt
        def neighbour_values(direction: int) -> torch.Tensor:
            vals: List[torch.Tensor] = []
            need, r = half, rank + direction
            while need > 0 and 0 <= r < world:
                n_r = bounds[r][1] - bounds[r][0]
                take = min(need, n_r, half)
                if take > 0:
                    e = edges[r]
                    part = e[2 * half - take:] if direction < 0 else e[:take]
                    vals.append(part)
                    need -= take
                if n_r > half:
                    break
                # a short neighbour (n_r <= half) contributed all it has; carry on to the next one
                r += direction
            if direction < 0:
                vals = vals[::-1]
            got = torch.cat(vals) if vals else torch.zeros(0, device=dev)
            pad = torch.zeros(half - got.numel(), device=dev)
            return torch.cat([pad, got]) if direction < 0 else torch.cat([got, pad])

        padded = torch.cat([neighbour_values(-1), imp, neighbour_values(+1)]).contiguous()
        smoothed = ops.smooth(padded, pool_kernel)[half:half + n_local]
        scores_local = ops.chunk_means(smoothed.contiguous(), chunk).float()

    # 4. every rank selects on all chunk scores
    gathered = _all_gather_padded(scores_local, group)
    scores = torch.cat(gathered)
    kept = ops.select_topk(scores, keep_count)
    chunk_lo = shard.lo // chunk
    n_chunks_local = scores_local.numel()
    mine = kept[(kept >= chunk_lo) & (kept < chunk_lo + n_chunks_local)] - chunk_lo

    # 5. local compaction, then stitch: positions and token spans become global, spans that meet at a rank boundary merge
    if n_local > 0 and mine.numel() > 0:
        ids, pos, tok, ch = ops.compact(mine, chunk, shard)
        pos, tok = pos + shard.lo, tok + shard.lo
    else:
        ids = pos = torch.zeros(0, dtype=torch.int64, device=dev)
        tok = ch = torch.zeros((0, 2), dtype=torch.int64, device=dev)
    all_ids = torch.cat(_all_gather_padded(ids, group)).cpu()
    all_pos = torch.cat(_all_gather_padded(pos, group)).cpu()
    all_tok = torch.cat(_all_gather_padded(tok.reshape(-1), group)).cpu().reshape(-1, 2)
    all_ch = torch.cat(_all_gather_padded(ch.reshape(-1), group)).cpu().reshape(-1, 2)
    merged_tok: List[List[int]] = []
    merged_ch: List[List[int]] = []
    for (a, b), (ca, cb) in zip(all_tok.tolist(), all_ch.tolist()):
        if merged_tok and merged_tok[-1][1] == a:      # the previous span ends where this one starts: one span
            merged_tok[-1][1] = b
            merged_ch[-1][1] = cb
        else:
            merged_tok.append([a, b])
            merged_ch.append([ca, cb])
    return ShardedSelection(keep_count, kept.cpu(), all_ids, all_pos,
                            torch.tensor(merged_tok, dtype=torch.int64).reshape(-1, 2),
                            torch.tensor(merged_ch, dtype=torch.int64).reshape(-1, 2), imp, lse_all)
