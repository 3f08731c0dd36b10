// Chunk pooling, top-k chunk selection and span compaction (Appendix A.1.2, Section 3.2).
// These steps touch a few hundred KB at most; they are latency-bound and each is a single launch.
#include <algorithm>

#include "common.cuh"

namespace spf {
namespace {

// ------------------------------------------------------------------------------------------------
// spf_chunk_pool: one warp per chunk.  Each lane sums the w-wide windows of its tokens, the warp adds
// them up in a fixed order, so the result does not depend on scheduling.
// ------------------------------------------------------------------------------------------------
constexpr int kPoolWarps = 8;

__device__ __forceinline__ void chunk_pool_body(const float* __restrict__ importance, int64_t n_tokens, int half, float inv_w,
                                                int chunk, bool in_range_divisor, float* __restrict__ chunk_scores,
                                                int64_t n_chunks) {
  const int lane = threadIdx.x & 31;
  const int64_t j = (int64_t)blockIdx.x * kPoolWarps + (threadIdx.x >> 5);
  if (j >= n_chunks) return;
  const int64_t lo = j * chunk;
  const int64_t hi = min(lo + (int64_t)chunk, n_tokens);
  float sum = 0.f;
  for (int64_t s = lo + lane; s < hi; s += 32) {
    const int64_t a = max(s - half, (int64_t)0), b = min(s + half, n_tokens - 1);
    float win = 0.f;
    for (int64_t t = a; t <= b; ++t) win += __ldg(importance + t);
    // the window's divisor: always w (zeros beyond the ends), or the number of tokens it really covers
    sum += in_range_divisor ? win / (float)(b - a + 1) : win * inv_w;
  }
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, off);
  if (lane == 0) chunk_scores[j] = sum / (float)(hi - lo);
}

__global__ void __launch_bounds__(kPoolWarps * 32) chunk_pool_kernel(const float* __restrict__ importance, int64_t n_tokens,
                                                                      int half, float inv_w, int chunk, bool in_range_divisor,
                                                                      float* __restrict__ chunk_scores, int64_t n_chunks) {
  chunk_pool_body(importance, n_tokens, half, inv_w, chunk, in_range_divisor, chunk_scores, n_chunks);
}

// Batched calls: up to kBatchItems prompts per launch, their descriptors passed by value; blockIdx.y picks the prompt.
constexpr int kBatchItems = 32;
struct PoolBatch {
  spf_pool_item item[kBatchItems];
};
struct TopkBatch {
  spf_topk_item item[kBatchItems];
};
struct CompactBatch {
  spf_compact_item item[kBatchItems];
};

__global__ void __launch_bounds__(kPoolWarps * 32) chunk_pool_batch_kernel(const __grid_constant__ PoolBatch b, int half, float inv_w,
                                                                            int chunk) {
  const spf_pool_item& it = b.item[blockIdx.y];
  chunk_pool_body(it.importance, it.n_tokens, half, inv_w, chunk, false, it.chunk_scores, (it.n_tokens + chunk - 1) / chunk);
}

// ------------------------------------------------------------------------------------------------
// spf_select_topk: one CTA.  Scores map to unsigned keys whose integer order is the float order; a
// four-pass radix select (8 bits per pass, most significant first) finds the k-th largest key; then
// everything above it, plus the lowest-index entries equal to it, is written out in index order.
// ------------------------------------------------------------------------------------------------
constexpr int kTopkThreads = 1024;

__device__ __forceinline__ uint32_t order_key(float x) {
  x += 0.0f;  // -0 -> +0 so that the two zeros tie
  const uint32_t b = __float_as_uint(x);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}

// Key of chunk j: forced chunks (bit 0 of `force`: the first chunk, bit 1: the last) sort above every score.
__device__ __forceinline__ uint32_t chunk_key(const float* __restrict__ scores, int j, int n, int force) {
  if (((force & 1) && j == 0) || ((force & 2) && j == n - 1)) return 0xFFFFFFFFu;
  return order_key(scores[j]);
}

// Exclusive prefix count of `flag` over the CTA (thread order); *total gets the CTA-wide count.  The 32 warp totals
// are scanned by warp 0 with shuffles (slot 32 of warp_counts receives the CTA-wide total).
__device__ __forceinline__ int block_exclusive_count(bool flag, int* warp_counts, int* total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const unsigned ballot = __ballot_sync(0xffffffffu, flag);
  const int within = __popc(ballot & ((1u << lane) - 1u));
  __syncthreads();  // warp_counts may still be read from the previous use
  if (lane == 0) warp_counts[warp] = __popc(ballot);
  __syncthreads();
  if (warp == 0) {
    const int own = warp_counts[lane];
    int incl = own;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int v = __shfl_up_sync(0xffffffffu, incl, off);
      if (lane >= off) incl += v;
    }
    warp_counts[lane] = incl - own;                      // exclusive offset of warp `lane`
    if (lane == 31) warp_counts[32] = incl;
  }
  __syncthreads();
  *total = warp_counts[32];
  return warp_counts[warp] + within;
}

// One histogram increment per distinct bin of a warp instead of one per thread: scores share their top bits, so the
// first passes would otherwise send thousands of atomics to a handful of shared-memory words.
__device__ __forceinline__ void hist_add_aggregated(int* hist, bool take, uint32_t bin) {
  const unsigned peers = __match_any_sync(0xffffffffu, take ? bin : 0xffffffffu);
  if (take && (int)(__ffs(peers) - 1) == (int)(threadIdx.x & 31)) atomicAdd(&hist[bin], __popc(peers));
}

__device__ __forceinline__ void select_topk_body(const float* __restrict__ scores, int n, int k, int force,
                                                 int32_t* __restrict__ kept) {
  __shared__ int hist[256];
  __shared__ int warp_counts[kTopkThreads / 32 + 1];
  __shared__ uint32_t sh_prefix;
  __shared__ int sh_remaining;

  // up to kTopkCache keys per thread stay in registers for all passes (n <= 8192 chunks, i.e. prompts of up to 262 144
  // tokens at chunk 32); longer score arrays are re-read from global memory in every pass
  constexpr int kTopkCache = 8;
  const bool cached = n <= kTopkThreads * kTopkCache;
  uint32_t ck[kTopkCache];
  if (cached) {
#pragma unroll
    for (int i = 0; i < kTopkCache; ++i) {
      const int j = threadIdx.x + i * kTopkThreads;
      ck[i] = j < n ? chunk_key(scores, j, n, force) : 0u;
    }
  }
  uint32_t prefix = 0;     // the bits of the k-th largest key found so far
  uint32_t mask = 0;       // which bits of `prefix` are fixed
  int remaining = k;       // rank of the wanted key among the keys that match the prefix
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    for (int b = threadIdx.x; b < 256; b += kTopkThreads) hist[b] = 0;
    __syncthreads();
    if (cached) {
#pragma unroll
      for (int i = 0; i < kTopkCache; ++i) {
        const int j = threadIdx.x + i * kTopkThreads;
        if (i * kTopkThreads < n)                            // warp-uniform: whole warps take part or none
          hist_add_aggregated(hist, j < n && (ck[i] & mask) == prefix, (ck[i] >> shift) & 255u);
      }
    } else {
      for (int j0 = 0; j0 < n; j0 += kTopkThreads) {
        const int j = j0 + threadIdx.x;
        const uint32_t key = j < n ? chunk_key(scores, j, n, force) : 0u;
        hist_add_aggregated(hist, j < n && (key & mask) == prefix, (key >> shift) & 255u);
      }
    }
    __syncthreads();
    if (threadIdx.x < 32) {
      // warp 0 walks the 256 bins from the top: each lane owns 8 consecutive bins (lane 31 the highest)
      const int lane = threadIdx.x;
      int mine[8], own = 0;
#pragma unroll
      for (int e = 0; e < 8; ++e) {
        mine[e] = hist[lane * 8 + e];
        own += mine[e];
      }
      int above = own;                                   // inclusive suffix sum over lanes >= this one
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const int v = __shfl_down_sync(0xffffffffu, above, off);
        if (lane + off < 32) above += v;
      }
      above -= own;                                      // entries in bins owned by higher lanes
      const bool here = above < remaining && above + own >= remaining;   // the wanted rank falls into this lane's bins
      if (here) {
        int rem = remaining - above, b = 0;
        bool found = false;
#pragma unroll
        for (int e = 7; e >= 0; --e) {
          if (!found) {
            if (mine[e] >= rem || e == 0) {
              b = e;
              found = true;
            } else {
              rem -= mine[e];
            }
          }
        }
        sh_prefix = prefix | ((uint32_t)(lane * 8 + b) << shift);
        sh_remaining = rem;
      }
    }
    __syncthreads();
    prefix = sh_prefix;
    remaining = sh_remaining;
    mask |= 255u << shift;
    __syncthreads();
  }
  // `prefix` is now the k-th largest key; `remaining` of the entries equal to it are kept (lowest indices).
  int out_base = 0, eq_base = 0;
  for (int j0 = 0, it = 0; j0 < n; j0 += kTopkThreads, ++it) {
    const int j = j0 + threadIdx.x;
    uint32_t key = 0u;
    if (cached) {
#pragma unroll
      for (int i = 0; i < kTopkCache; ++i)
        if (i == it) key = ck[i];                            // constant indices keep the cache in registers
    } else if (j < n) {
      key = chunk_key(scores, j, n, force);
    }
    const bool gt = j < n && key > prefix;
    const bool eq = j < n && key == prefix;
    int eq_total, sel_total;
    const int eq_rank = eq_base + block_exclusive_count(eq, warp_counts, &eq_total);
    const bool sel = gt || (eq && eq_rank < remaining);
    const int pos = out_base + block_exclusive_count(sel, warp_counts, &sel_total);
    if (sel && pos < k) kept[pos] = j;
    out_base += sel_total;
    eq_base += eq_total;
  }
}

__global__ void __launch_bounds__(kTopkThreads) select_topk_kernel(const float* __restrict__ scores, int n, int k, int force,
                                                                    int32_t* __restrict__ kept) {
  select_topk_body(scores, n, k, force, kept);
}

__global__ void __launch_bounds__(kTopkThreads) select_topk_batch_kernel(const __grid_constant__ TopkBatch b) {
  const spf_topk_item& it = b.item[blockIdx.x];
  select_topk_body(it.chunk_scores, (int)it.n_chunks, (int)it.k, 0, it.kept_chunks);
}

// ------------------------------------------------------------------------------------------------
// spf_compact_spans.  Kept chunk r (ascending order) starts at output offset r * c because only the
// very last chunk of the prompt can be short and, if kept, it is the last one kept.  Block 0 finds
// the runs of consecutive chunks (a prefix count of run starts) and writes the spans and counts; the
// other blocks copy ids and positions, one warp per kept chunk.
// ------------------------------------------------------------------------------------------------
constexpr int kCompactThreads = 256;

__device__ __forceinline__ void compact_spans_body(
    const int32_t* __restrict__ kept, int k, int chunk, int64_t n_tokens, const int32_t* __restrict__ token_ids,
    const int32_t* __restrict__ char_start, const int32_t* __restrict__ char_end, int32_t* __restrict__ out_ids,
    int32_t* __restrict__ out_pos, int32_t* __restrict__ out_tok_spans, int32_t* __restrict__ out_char_spans,
    int64_t* __restrict__ out_counts) {
  const int64_t n_chunks = (n_tokens + chunk - 1) / chunk;
  if (blockIdx.x == 0) {
    __shared__ int warp_counts[kCompactThreads / 32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int span_base = 0;
    for (int r0 = 0; r0 < k; r0 += kCompactThreads) {
      const int r = r0 + threadIdx.x;
      int64_t j = -1;
      bool starts = false, ends = false;
      if (r < k) {
        j = kept[r];
        starts = r == 0 || kept[r - 1] + 1 != j;
        ends = r == k - 1 || kept[r + 1] != j + 1;
      }
      const unsigned ballot = __ballot_sync(0xffffffffu, starts);
      const int within = __popc(ballot & ((2u << lane) - 1u));  // inclusive
      __syncthreads();
      if (lane == 0) warp_counts[warp] = __popc(ballot);
      __syncthreads();
      int before = 0, all = 0;
      for (int w = 0; w < kCompactThreads / 32; ++w) {
        before += w < warp ? warp_counts[w] : 0;
        all += warp_counts[w];
      }
      const int span = span_base + before + within - 1;  // index of the run this chunk belongs to
      if (r < k && j >= 0 && j < n_chunks) {
        if (starts) {
          const int64_t a = j * chunk;
          out_tok_spans[2 * span] = (int32_t)a;
          out_char_spans[2 * span] = char_start[a];
        }
        if (ends) {
          const int64_t b = min((j + 1) * chunk, n_tokens);
          out_tok_spans[2 * span + 1] = (int32_t)b;
          out_char_spans[2 * span + 1] = char_end[b - 1];
        }
      }
      span_base += all;
    }
    if (threadIdx.x == 0) {
      const int64_t last = kept[k - 1];
      const int64_t last_size = min((last + 1) * chunk, n_tokens) - last * chunk;
      out_counts[0] = (int64_t)(k - 1) * chunk + last_size;
      out_counts[1] = span_base;
    }
    return;
  }
  const int warps = kCompactThreads / 32;
  const int lane = threadIdx.x & 31;
  const int64_t r = (int64_t)(blockIdx.x - 1) * warps + (threadIdx.x >> 5);
  if (r >= k) return;
  const int64_t j = kept[r];
  if (j < 0 || j >= n_chunks) return;
  const int64_t lo = j * chunk, hi = min(lo + chunk, n_tokens);
  for (int64_t s = lo + lane; s < hi; s += 32) {
    const int64_t o = r * chunk + (s - lo);
    out_ids[o] = token_ids[s];
    if (out_pos != nullptr) out_pos[o] = (int32_t)s;
  }
}

__global__ void __launch_bounds__(kCompactThreads) compact_spans_kernel(
    const int32_t* __restrict__ kept, int k, int chunk, int64_t n_tokens, const int32_t* __restrict__ token_ids,
    const int32_t* __restrict__ char_start, const int32_t* __restrict__ char_end, int32_t* __restrict__ out_ids,
    int32_t* __restrict__ out_pos, int32_t* __restrict__ out_tok_spans, int32_t* __restrict__ out_char_spans,
    int64_t* __restrict__ out_counts) {
  compact_spans_body(kept, k, chunk, n_tokens, token_ids, char_start, char_end, out_ids, out_pos, out_tok_spans, out_char_spans,
                     out_counts);
}

// ------------------------------------------------------------------------------------------------
// spf_select_compact: top-k and compaction of one prompt in ONE CTA (the two steps are latency-bound and the second
// only needs the first's k indices, so a second launch costs more than the work).  After the selection the same
// 1024 threads find the runs of consecutive kept chunks (a prefix count of run starts, as compact_spans_kernel's
// block 0 does) and copy ids and positions, one warp per kept chunk.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kTopkThreads) select_compact_kernel(
    const float* __restrict__ scores, int n, int k, int chunk, int64_t n_tokens, const int32_t* __restrict__ token_ids,
    const int32_t* __restrict__ char_start, const int32_t* __restrict__ char_end, int32_t* __restrict__ kept,
    int32_t* __restrict__ out_ids, int32_t* __restrict__ out_pos, int32_t* __restrict__ out_tok_spans,
    int32_t* __restrict__ out_char_spans, int64_t* __restrict__ out_counts) {
  select_topk_body(scores, n, k, 0, kept);
  __threadfence_block();
  __syncthreads();                                          // kept[0..k) is complete and visible to the whole CTA
  __shared__ int warp_counts[kTopkThreads / 32];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int32_t* kv = kept;                                 // written by other threads of this CTA a moment ago: read past L1
  int span_base = 0;
  for (int r0 = 0; r0 < k; r0 += kTopkThreads) {
    const int r = r0 + threadIdx.x;
    int64_t j = -1;
    bool starts = false, ends = false;
    if (r < k) {
      j = __ldcg(kv + r);
      starts = r == 0 || __ldcg(kv + r - 1) + 1 != j;
      ends = r == k - 1 || __ldcg(kv + r + 1) != j + 1;
    }
    const unsigned ballot = __ballot_sync(0xffffffffu, starts);
    const int within = __popc(ballot & ((2u << lane) - 1u));  // inclusive
    __syncthreads();
    if (lane == 0) warp_counts[warp] = __popc(ballot);
    __syncthreads();
    int before = 0, all = 0;
    for (int w = 0; w < kTopkThreads / 32; ++w) {
      before += w < warp ? warp_counts[w] : 0;
      all += warp_counts[w];
    }
    const int span = span_base + before + within - 1;      // index of the run this chunk belongs to
    if (r < k) {
      if (starts) {
        const int64_t a = j * chunk;
        out_tok_spans[2 * span] = (int32_t)a;
        out_char_spans[2 * span] = char_start[a];
      }
      if (ends) {
        const int64_t b = min((j + 1) * chunk, n_tokens);
        out_tok_spans[2 * span + 1] = (int32_t)b;
        out_char_spans[2 * span + 1] = char_end[b - 1];
      }
    }
    span_base += all;
  }
  const int64_t last = __ldcg(kv + k - 1);
  const int64_t n_kept = (int64_t)(k - 1) * chunk + (min((last + 1) * chunk, n_tokens) - last * chunk);
  if (threadIdx.x == 0) {
    out_counts[0] = n_kept;
    out_counts[1] = span_base;
  }
  // kept chunk r (ascending) starts at output offset r * chunk: only the prompt's last chunk can be short.  The
  // output is walked as one flat array so that every thread has several independent loads in flight
#pragma unroll 4
  for (int64_t o = threadIdx.x; o < n_kept; o += kTopkThreads) {
    const int64_t r = o / chunk;
    const int64_t t = (int64_t)__ldcg(kv + r) * chunk + (o - r * chunk);
    out_ids[o] = __ldg(token_ids + t);
    if (out_pos != nullptr) out_pos[o] = (int32_t)t;
  }
}

__global__ void __launch_bounds__(kCompactThreads) compact_spans_batch_kernel(const __grid_constant__ CompactBatch b, int chunk) {
  const spf_compact_item& it = b.item[blockIdx.y];
  if ((int64_t)blockIdx.x > 1 + (it.k + kCompactThreads / 32 - 1) / (kCompactThreads / 32)) return;
  compact_spans_body(it.kept_chunks, (int)it.k, chunk, it.n_tokens, it.token_ids, it.char_start, it.char_end, it.out_ids, it.out_pos,
                     it.out_tok_spans, it.out_char_spans, it.out_counts);
}

}  // namespace
}  // namespace spf

using namespace spf;

static int32_t chunk_pool_launch(const float* importance, int64_t n_tokens, int32_t pool_kernel, int32_t chunk,
                                 bool in_range_divisor, float* chunk_scores, void* cuda_stream) {
  clear_error();
  if (importance == nullptr || chunk_scores == nullptr) return fail(SPF_ERR_INVALID_ARG, "spf_chunk_pool: null pointer");
  if (n_tokens < 1) return fail(SPF_ERR_INVALID_ARG, "spf_chunk_pool: n_tokens must be >= 1 (got %lld)", (long long)n_tokens);
  if (pool_kernel < 1 || pool_kernel > 255 || pool_kernel % 2 == 0)
    return fail(SPF_ERR_INVALID_ARG, "spf_chunk_pool: pool_kernel must be odd and in [1, 255] (got %d)", pool_kernel);
  if (chunk < 1) return fail(SPF_ERR_INVALID_ARG, "spf_chunk_pool: chunk must be >= 1 (got %d)", chunk);
  const int64_t n_chunks = ceil_div(n_tokens, chunk);
  const int64_t blocks = ceil_div(n_chunks, kPoolWarps);
  if (blocks > 0x7fffffff) return fail(SPF_ERR_UNSUPPORTED, "spf_chunk_pool: too many chunks");
  chunk_pool_kernel<<<(unsigned)blocks, kPoolWarps * 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      importance, n_tokens, pool_kernel / 2, 1.0f / (float)pool_kernel, chunk, in_range_divisor, chunk_scores, n_chunks);
  SPF_CUDA_CHECK(cudaGetLastError());
  return SPF_OK;
}

extern "C" int32_t spf_chunk_pool(const float* importance, int64_t n_tokens, int32_t pool_kernel, int32_t chunk,
                                  float* chunk_scores, void* cuda_stream) {
  return chunk_pool_launch(importance, n_tokens, pool_kernel, chunk, false, chunk_scores, cuda_stream);
}

extern "C" int32_t spf_chunk_pool_edge(const float* importance, int64_t n_tokens, int32_t pool_kernel, int32_t chunk,
                                       int32_t edge_rule, float* chunk_scores, void* cuda_stream) {
  if (edge_rule != 0 && edge_rule != 1) {
    clear_error();
    return fail(SPF_ERR_INVALID_ARG, "spf_chunk_pool_edge: edge_rule must be 0 or 1 (got %d)", edge_rule);
  }
  return chunk_pool_launch(importance, n_tokens, pool_kernel, chunk, edge_rule == 1, chunk_scores, cuda_stream);
}

static int32_t select_topk_launch(const float* chunk_scores, int64_t n_chunks, int64_t k, int force, int32_t* kept_chunks,
                                  void* cuda_stream) {
  clear_error();
  if (chunk_scores == nullptr || kept_chunks == nullptr) return fail(SPF_ERR_INVALID_ARG, "spf_select_topk: null pointer");
  if (n_chunks < 1 || n_chunks > 0x7fffffff)
    return fail(SPF_ERR_INVALID_ARG, "spf_select_topk: n_chunks must be in [1, 2^31) (got %lld)", (long long)n_chunks);
  if (k < 1 || k > n_chunks)
    return fail(SPF_ERR_INVALID_ARG, "spf_select_topk: k must be in [1, n_chunks] (got k=%lld, n_chunks=%lld)", (long long)k,
                (long long)n_chunks);
  const int n_forced = (force & 1) + ((force & 2) && (n_chunks > 1 || !(force & 1)) ? 1 : 0);
  if (k < n_forced)
    return fail(SPF_ERR_INVALID_ARG, "spf_select_topk_forced: k = %lld is smaller than the %d forced chunks", (long long)k, n_forced);
  select_topk_kernel<<<1, kTopkThreads, 0, static_cast<cudaStream_t>(cuda_stream)>>>(chunk_scores, (int)n_chunks, (int)k, force,
                                                                                    kept_chunks);
  SPF_CUDA_CHECK(cudaGetLastError());
  return SPF_OK;
}

extern "C" int32_t spf_select_topk(const float* chunk_scores, int64_t n_chunks, int64_t k, int32_t* kept_chunks,
                                   void* cuda_stream) {
  return select_topk_launch(chunk_scores, n_chunks, k, 0, kept_chunks, cuda_stream);
}

extern "C" int32_t spf_select_topk_forced(const float* chunk_scores, int64_t n_chunks, int64_t k, int32_t force_first,
                                          int32_t force_last, int32_t* kept_chunks, void* cuda_stream) {
  return select_topk_launch(chunk_scores, n_chunks, k, (force_first ? 1 : 0) | (force_last ? 2 : 0), kept_chunks, cuda_stream);
}

extern "C" int32_t spf_compact_spans(const int32_t* kept_chunks, int64_t k, int32_t chunk, int64_t n_tokens,
                                     const int32_t* token_ids, const int32_t* char_start, const int32_t* char_end,
                                     int32_t* out_ids, int32_t* out_pos, int32_t* out_tok_spans, int32_t* out_char_spans,
                                     int64_t* out_counts, void* cuda_stream) {
  clear_error();
  if (kept_chunks == nullptr || token_ids == nullptr || char_start == nullptr || char_end == nullptr || out_ids == nullptr ||
      out_tok_spans == nullptr || out_char_spans == nullptr || out_counts == nullptr)
    return fail(SPF_ERR_INVALID_ARG, "spf_compact_spans: null pointer");
  if (chunk < 1) return fail(SPF_ERR_INVALID_ARG, "spf_compact_spans: chunk must be >= 1 (got %d)", chunk);
  if (n_tokens < 1 || n_tokens > 0x7fffffff)
    return fail(SPF_ERR_INVALID_ARG, "spf_compact_spans: n_tokens must be in [1, 2^31) (got %lld)", (long long)n_tokens);
  const int64_t n_chunks = ceil_div(n_tokens, chunk);
  if (k < 1 || k > n_chunks)
    return fail(SPF_ERR_INVALID_ARG, "spf_compact_spans: k must be in [1, n_chunks] (got k=%lld, n_chunks=%lld)", (long long)k,
                (long long)n_chunks);
  const int64_t blocks = 1 + ceil_div(k, kCompactThreads / 32);
  compact_spans_kernel<<<(unsigned)blocks, kCompactThreads, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      kept_chunks, (int)k, chunk, n_tokens, token_ids, char_start, char_end, out_ids, out_pos, out_tok_spans, out_char_spans,
      out_counts);
  SPF_CUDA_CHECK(cudaGetLastError());
  return SPF_OK;
}

// ------------------------------------------------------------------------------------------------ batched calls
extern "C" int32_t spf_chunk_pool_batch(const spf_pool_item* items, int32_t n_items, int32_t pool_kernel, int32_t chunk,
                                        void* cuda_stream) {
  clear_error();
  if (items == nullptr || n_items < 1) return fail(SPF_ERR_INVALID_ARG, "spf_chunk_pool_batch: null items or n_items < 1");
  if (pool_kernel < 1 || pool_kernel > 255 || pool_kernel % 2 == 0)
    return fail(SPF_ERR_INVALID_ARG, "spf_chunk_pool_batch: pool_kernel must be odd and in [1, 255] (got %d)", pool_kernel);
  if (chunk < 1) return fail(SPF_ERR_INVALID_ARG, "spf_chunk_pool_batch: chunk must be >= 1 (got %d)", chunk);
  for (int32_t i = 0; i < n_items; ++i) {
    if (items[i].importance == nullptr || items[i].chunk_scores == nullptr)
      return fail(SPF_ERR_INVALID_ARG, "spf_chunk_pool_batch: item %d: null pointer", i);
    if (items[i].n_tokens < 1) return fail(SPF_ERR_INVALID_ARG, "spf_chunk_pool_batch: item %d: n_tokens must be >= 1", i);
    if (ceil_div(ceil_div(items[i].n_tokens, chunk), kPoolWarps) > 0x7fffffff)
      return fail(SPF_ERR_UNSUPPORTED, "spf_chunk_pool_batch: item %d: too many chunks", i);
  }
  for (int32_t i0 = 0; i0 < n_items; i0 += kBatchItems) {
    const int cnt = std::min<int32_t>(kBatchItems, n_items - i0);
    PoolBatch b{};
    int64_t blocks = 1;
    for (int i = 0; i < cnt; ++i) {
      b.item[i] = items[i0 + i];
      blocks = std::max(blocks, ceil_div(ceil_div(items[i0 + i].n_tokens, chunk), kPoolWarps));
    }
    chunk_pool_batch_kernel<<<dim3((unsigned)blocks, (unsigned)cnt), kPoolWarps * 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        b, pool_kernel / 2, 1.0f / (float)pool_kernel, chunk);
    SPF_CUDA_CHECK(cudaGetLastError());
  }
  return SPF_OK;
}

extern "C" int32_t spf_select_topk_batch(const spf_topk_item* items, int32_t n_items, void* cuda_stream) {
  clear_error();
  if (items == nullptr || n_items < 1) return fail(SPF_ERR_INVALID_ARG, "spf_select_topk_batch: null items or n_items < 1");
  for (int32_t i = 0; i < n_items; ++i) {
    if (items[i].chunk_scores == nullptr || items[i].kept_chunks == nullptr)
      return fail(SPF_ERR_INVALID_ARG, "spf_select_topk_batch: item %d: null pointer", i);
    if (items[i].n_chunks < 1 || items[i].n_chunks > 0x7fffffff || items[i].k < 1 || items[i].k > items[i].n_chunks)
      return fail(SPF_ERR_INVALID_ARG, "spf_select_topk_batch: item %d: need 1 <= k <= n_chunks < 2^31 (k=%lld, n_chunks=%lld)", i,
                  (long long)items[i].k, (long long)items[i].n_chunks);
  }
  for (int32_t i0 = 0; i0 < n_items; i0 += kBatchItems) {
    const int cnt = std::min<int32_t>(kBatchItems, n_items - i0);
    TopkBatch b{};
    for (int i = 0; i < cnt; ++i) b.item[i] = items[i0 + i];
    select_topk_batch_kernel<<<cnt, kTopkThreads, 0, static_cast<cudaStream_t>(cuda_stream)>>>(b);
    SPF_CUDA_CHECK(cudaGetLastError());
  }
  return SPF_OK;
}

extern "C" int32_t spf_compact_spans_batch(const spf_compact_item* items, int32_t n_items, int32_t chunk, void* cuda_stream) {
  clear_error();
  if (items == nullptr || n_items < 1) return fail(SPF_ERR_INVALID_ARG, "spf_compact_spans_batch: null items or n_items < 1");
  if (chunk < 1) return fail(SPF_ERR_INVALID_ARG, "spf_compact_spans_batch: chunk must be >= 1 (got %d)", chunk);
  for (int32_t i = 0; i < n_items; ++i) {
    const spf_compact_item& it = items[i];
    if (it.kept_chunks == nullptr || it.token_ids == nullptr || it.char_start == nullptr || it.char_end == nullptr ||
        it.out_ids == nullptr || it.out_tok_spans == nullptr || it.out_char_spans == nullptr || it.out_counts == nullptr)
      return fail(SPF_ERR_INVALID_ARG, "spf_compact_spans_batch: item %d: null pointer", i);
    if (it.n_tokens < 1 || it.n_tokens > 0x7fffffff)
      return fail(SPF_ERR_INVALID_ARG, "spf_compact_spans_batch: item %d: n_tokens must be in [1, 2^31)", i);
    if (it.k < 1 || it.k > ceil_div(it.n_tokens, chunk))
      return fail(SPF_ERR_INVALID_ARG, "spf_compact_spans_batch: item %d: k must be in [1, n_chunks]", i);
  }
  for (int32_t i0 = 0; i0 < n_items; i0 += kBatchItems) {
    const int cnt = std::min<int32_t>(kBatchItems, n_items - i0);
    CompactBatch b{};
    int64_t blocks = 2;
    for (int i = 0; i < cnt; ++i) {
      b.item[i] = items[i0 + i];
      blocks = std::max(blocks, 1 + ceil_div(items[i0 + i].k, kCompactThreads / 32));
    }
    compact_spans_batch_kernel<<<dim3((unsigned)blocks, (unsigned)cnt), kCompactThreads, 0, static_cast<cudaStream_t>(cuda_stream)>>>(b, chunk);
    SPF_CUDA_CHECK(cudaGetLastError());
  }
  return SPF_OK;
}

extern "C" int32_t spf_select_compact(const float* chunk_scores, int64_t n_chunks, int64_t k, int32_t chunk, int64_t n_tokens,
                                      const int32_t* token_ids, const int32_t* char_start, const int32_t* char_end,
                                      int32_t* kept_chunks, int32_t* out_ids, int32_t* out_pos, int32_t* out_tok_spans,
                                      int32_t* out_char_spans, int64_t* out_counts, void* cuda_stream) {
  clear_error();
  if (chunk_scores == nullptr || kept_chunks == nullptr || token_ids == nullptr || char_start == nullptr || char_end == nullptr ||
      out_ids == nullptr || out_tok_spans == nullptr || out_char_spans == nullptr || out_counts == nullptr)
    return fail(SPF_ERR_INVALID_ARG, "spf_select_compact: null pointer");
  if (chunk < 1) return fail(SPF_ERR_INVALID_ARG, "spf_select_compact: chunk must be >= 1 (got %d)", chunk);
  if (n_tokens < 1 || n_tokens > 0x7fffffff)
    return fail(SPF_ERR_INVALID_ARG, "spf_select_compact: n_tokens must be in [1, 2^31) (got %lld)", (long long)n_tokens);
  if (n_chunks != ceil_div(n_tokens, chunk))
    return fail(SPF_ERR_INVALID_ARG, "spf_select_compact: n_chunks must be ceil(n_tokens / chunk) (got %lld for %lld tokens)",
                (long long)n_chunks, (long long)n_tokens);
  if (k < 1 || k > n_chunks)
    return fail(SPF_ERR_INVALID_ARG, "spf_select_compact: k must be in [1, n_chunks] (got k=%lld, n_chunks=%lld)", (long long)k,
                (long long)n_chunks);
  select_compact_kernel<<<1, kTopkThreads, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
      chunk_scores, (int)n_chunks, (int)k, chunk, n_tokens, token_ids, char_start, char_end, kept_chunks, out_ids, out_pos,
      out_tok_spans, out_char_spans, out_counts);
  SPF_CUDA_CHECK(cudaGetLastError());
  return SPF_OK;
}
