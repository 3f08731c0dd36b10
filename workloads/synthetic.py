"""Synthetic draft-model tensors shaped like the long-context workloads of the paper.

The paper evaluates on LongBench v1/v2, RULER and InfiniteBench Code.Debug with small
Llama- and Qwen3-family draft models (Section 4, Appendix A.2/A.3).  Neither the data nor
the weights are available offline, so these generators stand in for them: they emit the
two things the scoring path consumes -- post-RoPE lookahead queries ``Q[L,Hq,m,d]`` and the
prompt key cache ``K[L][Hkv,N,d]`` in bf16 -- plus token ids and per-token character
offsets, with the structure attention maps of such prompts have:

* an i.i.d. N(0,1) base,
* a rank-``r`` component shared by every layer and head (tokens that are "globally"
  salient for the lookahead queries),
* planted needle spans: runs of keys aligned with a per-(layer, kv-head) question
  direction that the queries also carry, *strong* (large logit boost) or *weak*
  (distractors), visible only to a random subset of (layer, kv-head) pairs
  ("retrieval heads"),
* optionally a per-layer query scale (sharper / flatter layers) and a recency component
  (keys near the end of the prompt aligned with a second query direction).

Everything is seeded.  Structural randomness (lengths, needle positions, retrieval
subsets, token ids, character lengths) comes from NumPy's PCG64 and is identical on every
machine; the bulk tensors come from ``torch.Generator`` on the requested device, so a
prompt generated on ``cuda`` differs bit-wise from one generated on ``cpu`` with the same
seed (the consumer copies the bytes it generated to whoever else needs them).

No arithmetic of the method lives here.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional, Sequence, Tuple

import numpy as np
import torch

GAMMA = 2.0           # weight of the shared low-rank component
BOOST_STRONG = 8.0    # logit boost (nats) of a strong needle key in a retrieval head
BOOST_WEAK = 2.0      # logit boost of a weak (distractor) needle key
BOOST_RECENCY = 4.0   # logit boost of the very last key in a recency head
RECENCY_TAU = 512.0   # decay length (tokens) of the recency component
RETRIEVAL_PROB = 0.25  # chance that a (layer, kv-head) pair sees a given needle
VOCAB = 32000
MAX_CHARS_PER_TOKEN = 8


@dataclasses.dataclass(frozen=True)
class WorkloadConfig:
    name: str
    n_layers: int
    n_q_heads: int
    n_kv_heads: int
    head_dim: int
    n_lookahead: int
    lengths: Tuple[int, ...]          # prompt lengths N, one per prompt
    chunk: int
    keep: Tuple[float, ...]           # keep ratios rho
    rank: int
    n_needles: int
    n_strong: int
    needle_len: Tuple[int, int]       # inclusive range of needle span lengths
    layer_scale: bool = False
    recency: bool = False
    seed: int = 0
    pool_kernel: int = 13

    @property
    def group(self) -> int:
        return self.n_q_heads // self.n_kv_heads

    def k_bytes(self) -> int:
        return sum(self.n_layers * self.n_kv_heads * n * self.head_dim * 2 for n in self.lengths)


def _ragged_lengths(seed: int, count: int, lo: int, hi: int) -> Tuple[int, ...]:
    rng = np.random.default_rng([seed, 0x5EED])
    return tuple(int(x) for x in rng.integers(lo, hi + 1, size=count))


CONFIGS = {
    # Tiny: the case the CPU oracle finishes in well under a second.
    "tiny": WorkloadConfig("tiny", 2, 4, 2, 64, 8, (2048,), 32, (0.25,), rank=8,
                           n_needles=4, n_strong=4, needle_len=(1, 1), seed=0),
    # Small-draft shape at 32k tokens.
    "small32k": WorkloadConfig("small32k", 16, 32, 8, 64, 8, (32768,), 32, (0.10,), rank=16,
                               n_needles=64, n_strong=16, needle_len=(16, 128), seed=1),
    # Wider heads, per-layer query scale, keep ratio swept.
    "wide64k": WorkloadConfig("wide64k", 28, 16, 8, 128, 8, (65536,), 64, (0.05, 0.10, 0.25, 0.50),
                              rank=16, n_needles=64, n_strong=16, needle_len=(16, 128),
                              layer_scale=True, seed=2),
    # Long context: the configuration the headline metric is quoted on.
    "long128k": WorkloadConfig("long128k", 16, 32, 8, 64, 16, (131072,), 32, (0.10,), rank=16,
                               n_needles=256, n_strong=64, needle_len=(16, 128), recency=True, seed=3),
    # The long-context geometry cut to 4 layers (K cache 512 MiB): sized for profiler captures.
    "long128k_l4": WorkloadConfig("long128k_l4", 4, 32, 8, 64, 16, (131072,), 32, (0.10,), rank=16,
                                  n_needles=256, n_strong=64, needle_len=(16, 128), recency=True, seed=3),
    # Ragged batch of 8 prompts.
    "ragged8": WorkloadConfig("ragged8", 28, 16, 8, 128, 8, _ragged_lengths(4, 8, 16384, 131072), 32,
                              (0.10,), rank=16, n_needles=64, n_strong=16, needle_len=(16, 128),
                              layer_scale=True, seed=4),
}


def small_config(name: str = "small", *, n_layers: int = 2, n_q_heads: int = 4, n_kv_heads: int = 2,
                 head_dim: int = 64, n_lookahead: int = 8, lengths: Sequence[int] = (1000,),
                 chunk: int = 32, keep: Sequence[float] = (0.25,), rank: int = 4, n_needles: int = 2,
                 n_strong: int = 1, needle_len: Tuple[int, int] = (4, 16), layer_scale: bool = False,
                 recency: bool = False, seed: int = 0, pool_kernel: int = 13) -> WorkloadConfig:
    """A free-form configuration for randomised small test shapes."""
    return WorkloadConfig(name, n_layers, n_q_heads, n_kv_heads, head_dim, n_lookahead, tuple(lengths),
                          chunk, tuple(keep), rank, n_needles, n_strong, needle_len, layer_scale,
                          recency, seed, pool_kernel)


@dataclasses.dataclass
class Prompt:
    cfg: WorkloadConfig
    index: int
    n_tokens: int
    q: torch.Tensor                    # bf16 [L, Hq, m, d]
    k: List[torch.Tensor]              # L tensors, bf16 [Hkv, N, d]
    token_ids: torch.Tensor            # int32 [N]
    char_start: torch.Tensor           # int32 [N]
    char_end: torch.Tensor             # int32 [N]
    needles: List[Tuple[int, int, bool]]  # (first token, length, strong?)

    def to(self, device) -> "Prompt":
        return dataclasses.replace(
            self, q=self.q.to(device), k=[t.to(device) for t in self.k],
            token_ids=self.token_ids.to(device), char_start=self.char_start.to(device),
            char_end=self.char_end.to(device))


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """The raw 16-bit patterns of a bf16 tensor, as a NumPy uint16 array (host copy)."""
    assert t.dtype == torch.bfloat16
    return t.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16)


def quantize_keys_e4m3(k: Sequence[torch.Tensor]):
    """An 8-bit copy of a bf16 key cache as a serving system would hold it: per (layer, kv-head) one fp32 scale
    (largest magnitude / 448, the format's largest number) and the keys divided by it, rounded to E4M3 by torch.
    Returns (L uint8 tensors [Hkv, N, d], fp32 scales [L, Hkv]).  Input preparation only: what the bytes MEAN is
    defined by the consumer (scale * E4M3 value)."""
    bytes_, scales = [], []
    for kl in k:
        amax = kl.float().abs().amax(dim=(1, 2)).clamp_min(1e-12)
        sc = (amax / 448.0).to(torch.float32)
        q8 = (kl.float() / sc[:, None, None]).to(torch.float8_e4m3fn)
        bytes_.append(q8.view(torch.uint8).contiguous())
        scales.append(sc)
    return bytes_, torch.stack(scales).contiguous()


def _place_needles(rng: np.random.Generator, n_tokens: int, cfg: WorkloadConfig):
    """Non-overlapping spans: one per equal segment of the prompt, uniform inside it."""
    count = cfg.n_needles
    if count == 0:
        return []
    seg = n_tokens // count
    lo, hi = cfg.needle_len
    hi = max(1, min(hi, seg - 1))
    lo = max(1, min(lo, hi))
    strong = np.zeros(count, dtype=bool)
    strong[rng.permutation(count)[: cfg.n_strong]] = True
    out = []
    for j in range(count):
        length = int(rng.integers(lo, hi + 1))
        if lo == hi == 1:
            # a single needle key: keep it away from chunk borders so that the smoothing
            # window stays inside one chunk
            base = j * seg + int(rng.integers(0, max(1, seg // cfg.chunk))) * cfg.chunk
            start = min(base + cfg.chunk // 2, n_tokens - 1)
        else:
            start = j * seg + int(rng.integers(0, seg - length + 1))
        out.append((start, length, bool(strong[j])))
    return out


def make_prompt(cfg: WorkloadConfig, index: int = 0, device: str = "cpu") -> Prompt:
    n = cfg.lengths[index]
    L, Hq, Hkv, d, m, r = cfg.n_layers, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.n_lookahead, cfg.rank
    G = cfg.group
    rng = np.random.default_rng([cfg.seed, index, 0xA11CE])
    gen = torch.Generator(device=device)
    gen.manual_seed(1_000_003 * cfg.seed + 7919 * index + 17)

    def randn(*shape):
        return torch.randn(*shape, generator=gen, device=device, dtype=torch.float32)

    needles = _place_needles(rng, n, cfg)
    # retrieval subsets: which (layer, kv-head) pairs see which needle
    sees = rng.random((len(needles), L, Hkv)) < RETRIEVAL_PROB
    for j in range(len(needles)):
        if not sees[j].any():
            sees[j, rng.integers(0, L), rng.integers(0, Hkv)] = True
    alpha = math.sqrt(BOOST_STRONG * math.sqrt(d))        # added to every query
    beta = {True: alpha, False: alpha * BOOST_WEAK / BOOST_STRONG}
    alpha_r = math.sqrt(BOOST_RECENCY * math.sqrt(d))
    layer_scales = rng.uniform(0.5, 2.0, size=L) if cfg.layer_scale else np.ones(L)
    recency_on = rng.random((L, Hkv)) < 0.5 if cfg.recency else np.zeros((L, Hkv), dtype=bool)

    tok_lat = randn(n, r) if r > 0 else None
    qry_lat = randn(m, r) if r > 0 else None
    if cfg.recency:
        pos = torch.arange(n, device=device, dtype=torch.float32)
        decay = torch.exp(-(float(n - 1) - pos) / RECENCY_TAU)

    q_layers, k_layers = [], []
    for l in range(L):
        kl = randn(Hkv, n, d)
        ql = randn(Hkv, G, m, d)
        if r > 0:
            basis = randn(Hkv, r, d) / math.sqrt(d)
            kl += GAMMA * torch.einsum("nr,hrd->hnd", tok_lat, basis)
            ql += GAMMA * torch.einsum("mr,hrd->hmd", qry_lat, basis)[:, None]
        if needles:
            u = torch.nn.functional.normalize(randn(Hkv, d), dim=-1)
            gain = np.zeros((Hkv, n), dtype=np.float32)
            for j, (s0, length, strong) in enumerate(needles):
                for h in np.nonzero(sees[j, l])[0]:
                    gain[h, s0:s0 + length] = beta[strong]
            kl += torch.from_numpy(gain).to(device)[:, :, None] * u[:, None, :]
            ql += alpha * u[:, None, None, :]
        if cfg.recency:
            v = torch.nn.functional.normalize(randn(Hkv, d), dim=-1)
            on = torch.from_numpy(recency_on[l].astype(np.float32)).to(device)
            kl += alpha_r * on[:, None, None] * decay[None, :, None] * v[:, None, :]
            ql += alpha_r * on[:, None, None, None] * v[:, None, None, :]
        ql *= float(layer_scales[l])
        q_layers.append(ql.reshape(Hq, m, d).to(torch.bfloat16))
        k_layers.append(kl.to(torch.bfloat16).contiguous())
        del kl, ql
    q = torch.stack(q_layers).contiguous()

    ids = rng.integers(0, VOCAB, size=n, dtype=np.int32)
    lens = rng.integers(1, MAX_CHARS_PER_TOKEN + 1, size=n, dtype=np.int64)
    ends = np.cumsum(lens)
    starts = ends - lens
    return Prompt(cfg, index, n, q, k_layers,
                  torch.from_numpy(ids).to(device),
                  torch.from_numpy(starts.astype(np.int32)).to(device),
                  torch.from_numpy(ends.astype(np.int32)).to(device),
                  needles)


def make_workload(cfg: WorkloadConfig, device: str = "cpu", prompts: Optional[Sequence[int]] = None):
    idx = range(len(cfg.lengths)) if prompts is None else prompts
    return [make_prompt(cfg, i, device) for i in idx]
