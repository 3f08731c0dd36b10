"""CPU oracle for speculative-prefill scoring, chunk selection and span compaction.

TEST INFRASTRUCTURE ONLY.  This is the plain, slow, fp64 statement of what the path
computes, written from the paper (Algorithm 1; Appendix A.1.1, A.1.2, A.3; Section 3.1-3.2).
It shares no code with the CUDA path and must never be called by it; only the tests, the
smoke check and the benchmark's CPU-baseline leg import it.

Every function is the definition written out.  NumPy matmul / exp / argsort serve as steps;
there is no blocking, fusion or reordering beyond what the definition states.

Notation (the paper's symbols in brackets): N prompt tokens [S], m lookahead queries [N],
L layers, Hq query heads [H], Hkv key/value heads, G = Hq/Hkv, d head dimension, c chunk
size, rho keep rate, C = ceil(N/c) chunks, k chunks kept, w pooling kernel (13).

Readings of points the paper leaves open (each is a switch or a documented choice):
  * softmax runs over the N prompt keys only, unmasked (every lookahead query sits after
    the whole prompt);
  * "attention scores" are post-softmax probabilities;
  * the max is joint over (layer, head), taken before the mean over lookahead queries;
  * pooling: stride 1, zero padding of w//2 on both sides, divisor always w;
  * a partial last chunk is averaged over the tokens it has;
  * k = clamp(ceil(rho*C), 1, C); equal scores -> the lower chunk index wins;
  * chunks j and j+1 both kept <=> same span; nothing else merges;
  * a span's characters run from the first token's start to the last token's end.
These readings are not pinned by printed values in the paper ("parity unpinned" for the
choice itself); the functions are pinned by the tests against closed forms, library
routines and brute force.
"""
from __future__ import annotations

import math
from typing import List, Optional, Sequence, Tuple

import numpy as np


# --------------------------------------------------------------------------------------
# inputs
# --------------------------------------------------------------------------------------
def bf16_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact value of bf16 bit patterns (uint16): bf16 is the top half of an IEEE fp32."""
    bits = np.ascontiguousarray(bits, dtype=np.uint16)
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def fp8_e4m3_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact value of 8-bit floating-point patterns (uint8) in the E4M3 format serving systems use for KV caches:
    1 sign bit, 4 exponent bits (bias 7), 3 mantissa bits; exponent field 0 holds the subnormals m/8 * 2^-6; there are
    no infinities, and exponent 15 with mantissa 7 is NaN (everything else with exponent 15 is an ordinary number,
    up to 448).  Written out from the format's definition, bit field by bit field."""
    bits = np.ascontiguousarray(bits, dtype=np.uint8).astype(np.int64)
    sign = np.where(bits & 0x80, -1.0, 1.0)
    e = (bits >> 3) & 0xF
    m = (bits & 0x7).astype(np.float64)
    normal = (1.0 + m / 8.0) * np.exp2((e - 7).astype(np.float64))
    subnormal = (m / 8.0) * 2.0 ** -6
    value = np.where(e == 0, subnormal, normal)
    value = np.where((e == 15) & (bits & 0x7 == 7), np.nan, value)
    return sign * value


# --------------------------------------------------------------------------------------
# Appendix A.1.1 -- attention-based token importance (Algorithm 1, AggregateMaxMean)
# --------------------------------------------------------------------------------------
def attention_logits(q_lh: np.ndarray, k_lh: np.ndarray, scale: float) -> np.ndarray:
    """z[i, s] = scale * sum_j q[i, j] * k[s, j] for one (layer, head): [m, d] x [N, d] -> [m, N]."""
    return scale * (q_lh @ k_lh.T)


def softmax_rows(z: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """Row softmax over the prompt keys and the row log-sum-exp: p = exp(z - lse)."""
    zmax = z.max(axis=1, keepdims=True)
    e = np.exp(z - zmax)
    tot = e.sum(axis=1, keepdims=True)
    return e / tot, (zmax + np.log(tot))[:, 0]


def token_importance(q_bits: np.ndarray, k_bits: Sequence[np.ndarray], scale: Optional[float] = None,
                     extra_lse: Optional[np.ndarray] = None) -> Tuple[np.ndarray, np.ndarray]:
    """Max-mean aggregation of lookahead attention (Appendix A.1.1).

    q_bits: uint16 [L, Hq, m, d] (bf16 patterns of the post-RoPE lookahead queries)
    k_bits: L arrays uint16 [Hkv, N, d] (bf16 patterns of the prompt key cache)
    Returns (I [N], lse [L, Hq, m]) in fp64 where
        p[l,h,i,:] = softmax_s(scale * Q[l,h,i] . K[l, h // G, s])
        A[i,s]     = max over all (l,h) of p[l,h,i,s]          (max over layer and head first)
        I[s]       = mean over i of A[i,s]                      (then mean over lookahead)
    extra_lse (optional, [L, Hq, m]): the natural log of what each row's softmax denominator holds besides the
    prompt keys (the lookahead step's own and earlier generated tokens -- a reading of a point the paper leaves
    open); then p = exp(z) / (sum_s exp(z) + exp(extra_lse)) and the returned lse is the log of that denominator.
    """
    L, Hq, m, d = q_bits.shape
    Hkv, N, d2 = k_bits[0].shape
    assert d2 == d and len(k_bits) == L and Hq % Hkv == 0
    G = Hq // Hkv
    if scale is None:
        scale = 1.0 / math.sqrt(d)
    A = np.zeros((m, N), dtype=np.float64)
    lse = np.zeros((L, Hq, m), dtype=np.float64)
    for l in range(L):
        for hk in range(Hkv):
            k_lh = bf16_to_f64(k_bits[l][hk])
            for g in range(G):
                h = hk * G + g
                p, lse[l, h] = softmax_rows(attention_logits(bf16_to_f64(q_bits[l, h]), k_lh, scale))
                if extra_lse is not None:
                    whole = np.logaddexp(lse[l, h], np.asarray(extra_lse, dtype=np.float64)[l, h])
                    p = p * np.exp(lse[l, h] - whole)[:, None]      # the prompt's share of the larger denominator
                    lse[l, h] = whole
                np.maximum(A, p, out=A)
    return A.mean(axis=0), lse


def token_importance_fp8(q_bits: np.ndarray, k_bytes: Sequence[np.ndarray], k_scale: np.ndarray,
                         scale: Optional[float] = None) -> Tuple[np.ndarray, np.ndarray]:
    """token_importance for a key cache stored in 8 bits (Section 3.1: the serving system's KV caches; a draft
    model served the same way keeps its keys quantised).  The cache format is an INPUT format: key (l, hk, s, j) has
    the value k_scale[l, hk] * E4M3(k_bytes[l][hk, s, j]), decoded exactly; everything after that is Appendix A.1.1
    unchanged.

    q_bits: uint16 [L, Hq, m, d] (bf16 patterns); k_bytes: L arrays uint8 [Hkv, N, d]; k_scale: fp32 [L, Hkv].
    Returns (I [N], lse [L, Hq, m]) in fp64.
    """
    L, Hq, m, d = q_bits.shape
    Hkv, N, d2 = k_bytes[0].shape
    assert d2 == d and len(k_bytes) == L and Hq % Hkv == 0
    k_scale = np.asarray(k_scale, dtype=np.float32).astype(np.float64).reshape(L, Hkv)
    G = Hq // Hkv
    if scale is None:
        scale = 1.0 / math.sqrt(d)
    A = np.zeros((m, N), dtype=np.float64)
    lse = np.zeros((L, Hq, m), dtype=np.float64)
    for l in range(L):
        for hk in range(Hkv):
            k_lh = k_scale[l, hk] * fp8_e4m3_to_f64(k_bytes[l][hk])
            for g in range(G):
                h = hk * G + g
                p, lse[l, h] = softmax_rows(attention_logits(bf16_to_f64(q_bits[l, h]), k_lh, scale))
                np.maximum(A, p, out=A)
    return A.mean(axis=0), lse


# --------------------------------------------------------------------------------------
# Appendix A.1.2 -- smoothing, chunking, top-K (Algorithm 1: AvgPool1D, PartitionIntoChunks,
# TopKChunks)
# --------------------------------------------------------------------------------------
def avg_pool(importance: np.ndarray, w: int = 13, count_include_pad: bool = True) -> np.ndarray:
    """Stride-1 average pooling with zero padding w//2, output length N (Appendix A.3: w = 13)."""
    assert w >= 1 and w % 2 == 1
    n = importance.shape[0]
    half = w // 2
    padded = np.zeros(n + 2 * half, dtype=np.float64)
    padded[half:half + n] = importance
    out = np.zeros(n, dtype=np.float64)
    for t in range(w):
        out += padded[t:t + n]
    if count_include_pad:
        return out / w
    ones = np.zeros(n + 2 * half)
    ones[half:half + n] = 1.0
    cnt = np.zeros(n)
    for t in range(w):
        cnt += ones[t:t + n]
    return out / cnt


def chunk_means(smoothed: np.ndarray, c: int) -> np.ndarray:
    """cs[j] = mean of the smoothed scores of tokens [j*c, min((j+1)*c, N))."""
    n = smoothed.shape[0]
    C = (n + c - 1) // c
    return np.array([smoothed[j * c:min((j + 1) * c, n)].mean() for j in range(C)], dtype=np.float64)


def keep_count(n_chunks: int, rho: float) -> int:
    """k = clamp(ceil(rho * C), 1, C): the number of chunks that a keep rate rho retains (Section 3.1)."""
    return max(1, min(n_chunks, int(math.ceil(rho * n_chunks - 1e-9))))


def select_topk(chunk_scores: np.ndarray, k: int) -> np.ndarray:
    """Indices of the k largest chunk scores (ties -> lower index), returned ascending."""
    order = np.argsort(-chunk_scores, kind="stable")      # stable: equal scores keep index order
    return np.sort(order[:k]).astype(np.int64)


# --------------------------------------------------------------------------------------
# Section 3.2 -- merge adjacent chunks, map draft-token ranges to text spans
# (Algorithm 1: MergeAdjacentChunks, MapDraftChunksToTextSpans)
# --------------------------------------------------------------------------------------
def select_topk_forced(chunk_scores: np.ndarray, k: int, force_first: bool = False, force_last: bool = False) -> np.ndarray:
    """TopKChunks with the first and / or last chunk kept whatever their scores (a reading of a point the paper
    leaves open): the forced chunks count towards k, the other k - forced are the best of the rest, ties to the
    lower index; ascending."""
    n = len(chunk_scores)
    forced = sorted({0} if force_first else set()) + ([n - 1] if force_last and not (force_first and n == 1) else [])
    if k < len(forced):
        raise ValueError("k is smaller than the number of forced chunks")
    rest = [j for j in range(n) if j not in forced]
    rest.sort(key=lambda j: (-float(chunk_scores[j]), j))        # stable: ties keep the lower index first
    return np.array(sorted(forced + rest[:k - len(forced)]), dtype=np.int64)


def merge_adjacent(kept: np.ndarray, c: int, n_tokens: int) -> np.ndarray:
    """Maximal runs of consecutive kept chunk indices -> token ranges [a, b), b clipped to N."""
    spans: List[Tuple[int, int]] = []
    for j in kept.tolist():
        a, b = j * c, min((j + 1) * c, n_tokens)
        if spans and spans[-1][1] == a:
            spans[-1] = (spans[-1][0], b)
        else:
            spans.append((a, b))
    return np.array(spans, dtype=np.int64).reshape(-1, 2)


def compact(kept: np.ndarray, c: int, n_tokens: int, token_ids: np.ndarray, char_start: np.ndarray,
            char_end: np.ndarray):
    """Kept token ids / positions in original order, merged token spans and their character spans."""
    tok_spans = merge_adjacent(kept, c, n_tokens)
    pos = np.concatenate([np.arange(a, b) for a, b in tok_spans]) if len(tok_spans) else np.zeros(0, np.int64)
    ids = token_ids[pos]
    char_spans = np.array([(char_start[a], char_end[b - 1]) for a, b in tok_spans], dtype=np.int64).reshape(-1, 2)
    return ids.astype(np.int64), pos.astype(np.int64), tok_spans, char_spans


# --------------------------------------------------------------------------------------
# whole path
# --------------------------------------------------------------------------------------
def compress(q_bits, k_bits, token_ids, char_start, char_end, *, chunk: int, keep: float,
             pool_kernel: int = 13, scale: Optional[float] = None):
    """Algorithm 1, from the aggregation of attention to the text spans, for one prompt."""
    importance, lse = token_importance(q_bits, k_bits, scale)
    n = importance.shape[0]
    cs = chunk_means(avg_pool(importance, pool_kernel), chunk)
    k = keep_count(cs.shape[0], keep)
    kept = select_topk(cs, k)
    ids, pos, tok_spans, char_spans = compact(kept, chunk, n, token_ids, char_start, char_end)
    return dict(importance=importance, lse=lse, chunk_scores=cs, k=k, kept=kept, ids=ids, pos=pos,
                tok_spans=tok_spans, char_spans=char_spans)


def keep_rate(target_tokens: int, budget_tokens: int) -> float:
    """Section 3.1: rho = compressed target length / original target length, at most 1 (0 for empty inputs)."""
    if target_tokens < 1 or budget_tokens < 1:
        return 0.0
    return min(1.0, budget_tokens / target_tokens)


def snap_budget(desired_tokens: int, block_tokens: int) -> int:
    """Section 3.1: compressed lengths are whole KV-cache blocks: the largest multiple of the block that is
    at most the desired length, and at least one block (0 for empty inputs)."""
    if desired_tokens < 1 or block_tokens < 1:
        return 0
    return max(1, desired_tokens // block_tokens) * block_tokens


def concat_with_delim(text: str, char_spans: Sequence[Sequence[int]], delim: str) -> str:
    """ConcatWithDelim of Algorithm 1 (Section 3.2, Appendix A.3): the spans' characters in order, the delimiter
    between consecutive spans only.  Python strings index by code point, which is how a tokenizer's offset mapping
    counts characters."""
    return delim.join(text[int(a):int(b)] for a, b in char_spans)
