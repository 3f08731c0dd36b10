// Token-importance scoring, general path: two sweeps over the key cache with warp-level
// tensor-core tiles (mma.sync m16n8k16, bf16 in, fp32 out).
//
//   sweep 1 (score_lse_kernel)   row statistics of every softmax row (l, h, i): running max and
//                                sum of exp2 over the prompt keys, split over CTAs, then merged
//                                (merge_lse_kernel) into lse2[l,h,i] = log2 sum_s exp2(c * q.k).
//   sweep 2 (score_max_kernel)   for every key s and lookahead i, max over all (l, h) of
//                                c * q.k - lse2 (the log2 of the softmax probability; exp2 is
//                                monotone, so the max commutes with it), then one exp2 per (i, s)
//                                and the mean over i.
//
// Here c = softmax_scale * log2(e).  The attention tensor is never stored.  This path reads the
// key cache twice from HBM; it handles every supported shape and prompt length.
//
// Tile geometry.  One warp owns 32 consecutive keys of one (layer, kv-head) slab and all query rows
// of that kv-head's group: rows r = g * m_pad + i (g < G heads of the group, i < m lookahead
// queries, m_pad = m rounded up to 8, the whole padded to a multiple of 16 rows; padding rows are
// zero queries and are masked).  Query rows are the M dimension of the MMA, keys the N dimension,
// the head dimension the K dimension.
//
// Key fragments come straight from global memory: for a 32-wide block of the head dimension the
// thread with lane % 4 == q loads the 16 bytes at dims [8q, 8q+8) of key lane / 4.  Those 8
// values feed two MMAs; the packed query fragments (pack_q_kernel) use the same permutation of
// the head dimension, which is legal because a dot product does not care about the order of its
// terms.  Every 32-byte sector fetched is fully used and no shared memory is involved.
#include <algorithm>

#include "common.cuh"
#include "score.cuh"

namespace spf {
namespace {

constexpr int kWarpsPerCta = 4;
constexpr int kThreads = kWarpsPerCta * 32;
constexpr int kTileKeys = 32;

__device__ __forceinline__ uint4 load_key16(const __nv_bfloat16* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

// Eight E4M3 keys (8 bytes) -> eight bf16 values in the same order.  Exact: every E4M3 number, subnormals included,
// is an fp16 number (hardware conversion), and has at most four significant bits, so fp16 -> fp32 -> bf16 rounds nothing.
__device__ __forceinline__ uint32_t e4m3x2_to_bf16x2(uint16_t two) {
  uint32_t h2;
  asm("cvt.rn.f16x2.e4m3x2 %0, %1;" : "=r"(h2) : "h"(two));
  const __half2 h = *reinterpret_cast<const __half2*>(&h2);
  const float2 f = __half22float2(h);
  const __nv_bfloat162 b = __floats2bfloat162_rn(f.x, f.y);
  return *reinterpret_cast<const uint32_t*>(&b);
}

__device__ __forceinline__ uint4 load_key8_fp8(const uint8_t* p) {
  uint2 raw;
  asm volatile("ld.global.nc.L1::no_allocate.v2.u32 {%0,%1}, [%2];" : "=r"(raw.x), "=r"(raw.y) : "l"(p));
  uint4 v;
  v.x = e4m3x2_to_bf16x2((uint16_t)(raw.x & 0xffffu));
  v.y = e4m3x2_to_bf16x2((uint16_t)(raw.x >> 16));
  v.z = e4m3x2_to_bf16x2((uint16_t)(raw.y & 0xffffu));
  v.w = e4m3x2_to_bf16x2((uint16_t)(raw.y >> 16));
  return v;
}

__device__ __forceinline__ void mma_bf16(float (&d)[4], const uint4& a, uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a.x), "r"(a.y), "r"(a.z), "r"(a.w), "r"(b0), "r"(b1));
}

// The keys of one warp tile: [n-tile of 8 keys][32-wide block of the head dimension].
template <int D>
struct KeyTile {
  uint4 r[4][D / 32];
};

// Paged key cache (block_tokens > 0): the pointers of LayerPtrs are block pools, bf16 [blocks][Hkv][block_tokens][d];
// logical block b of the prompt is pool block table[b].  A 32-key tile never straddles a block (blocks are multiples
// of 128 tokens), so one table entry places a whole tile.
struct PagedView {
  const int32_t* table;
  int block_tokens;
  int64_t stride_block, n_pool_blocks;
};

// Element offset, from the (layer, kv-head) base pointer, of the row of key0 (the first key of a tile).
__device__ __forceinline__ int64_t tile_offset(int64_t key0, int64_t stride_tok, const PagedView& pv) {
  if (pv.block_tokens == 0) return key0 * stride_tok;
  int64_t block = __ldg(pv.table + key0 / pv.block_tokens);
  block = block < 0 ? 0 : (block >= pv.n_pool_blocks ? pv.n_pool_blocks - 1 : block);   // a bad entry must not fault
  return block * pv.stride_block + (key0 % pv.block_tokens) * stride_tok;
}

// FP8: the cache holds E4M3 bytes (strides then count bytes); the tile is widened to bf16 as it is loaded.
template <int D, bool FP8>
__device__ __forceinline__ void load_key_tile(KeyTile<D>& t, const __nv_bfloat16* slab, int64_t tile_off, int64_t key0,
                                              int64_t n_tokens, int64_t stride_tok, int lane) {
#pragma unroll
  for (int nt = 0; nt < 4; ++nt) {
    int64_t key = key0 + nt * 8 + (lane >> 2);
    key = key < n_tokens ? key : n_tokens - 1;  // ragged tail: read a valid row (of the same tile), mask later
    if constexpr (FP8) {
      const uint8_t* row = reinterpret_cast<const uint8_t*>(slab) + tile_off + (key - key0) * stride_tok + (lane & 3) * 8;
#pragma unroll
      for (int j = 0; j < D / 32; ++j) t.r[nt][j] = load_key8_fp8(row + j * 32);
    } else {
      const __nv_bfloat16* row = slab + tile_off + (key - key0) * stride_tok + (lane & 3) * 8;
#pragma unroll
      for (int j = 0; j < D / 32; ++j) t.r[nt][j] = load_key16(row + j * 32);
    }
  }
}

// Base of the (layer, kv-head) slab: strides count elements, i.e. bytes for an 8-bit cache.
template <bool FP8>
__device__ __forceinline__ const __nv_bfloat16* slab_base(const __nv_bfloat16* layer, int64_t head_offset) {
  if constexpr (FP8) return reinterpret_cast<const __nv_bfloat16*>(reinterpret_cast<const uint8_t*>(layer) + head_offset);
  return layer + head_offset;
}

inline PagedView paged_view(const ScoreProblem& p) {
  return PagedView{p.block_table, p.block_tokens, (int64_t)p.n_kv_heads * p.block_tokens * p.head_dim, p.n_pool_blocks};
}

// acc[mt][nt] = logits of rows 16*mt.. against keys 8*nt.. (fp32, unscaled).
template <int D, int MT>
__device__ __forceinline__ void tile_logits(float (&acc)[MT][4][4], const KeyTile<D>& kt, const uint4* __restrict__ qslab,
                                            int lane) {
#pragma unroll
  for (int mt = 0; mt < MT; ++mt)
#pragma unroll
    for (int nt = 0; nt < 4; ++nt)
#pragma unroll
      for (int e = 0; e < 4; ++e) acc[mt][nt][e] = 0.f;
#pragma unroll
  for (int kk = 0; kk < D / 16; ++kk) {
#pragma unroll
    for (int mt = 0; mt < MT; ++mt) {
      const uint4 a = __ldg(qslab + (mt * (D / 16) + kk) * 32 + lane);
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) {
        const uint4& kv = kt.r[nt][kk >> 1];
        if (kk & 1)
          mma_bf16(acc[mt][nt], a, kv.z, kv.w);
        else
          mma_bf16(acc[mt][nt], a, kv.x, kv.y);
      }
    }
  }
}

// Packs Q[l][hk*G+g][i][:] into MMA A-fragment order: one uint4 per (slab, m-tile, 16-wide k-step, lane).
__global__ void pack_q_kernel(const __nv_bfloat16* __restrict__ q, uint4* __restrict__ qf, int n_kv_heads, int group,
                              int n_lookahead, int m_pad, int head_dim, int n_mtiles) {
  const int slab = blockIdx.x;
  const int layer = slab / n_kv_heads, hk = slab % n_kv_heads;
  const int n_q_heads = n_kv_heads * group;
  const int ksteps = head_dim / 16;
  const int total = n_mtiles * ksteps * 32;
  const uint32_t* q32 = reinterpret_cast<const uint32_t*>(q);
  for (int idx = threadIdx.x; idx < total; idx += blockDim.x) {
    const int lane = idx & 31;
    const int kk = (idx >> 5) % ksteps;
    const int mt = (idx >> 5) / ksteps;
    const int dim = (kk >> 1) * 32 + (lane & 3) * 8 + (kk & 1) * 4;
    uint32_t v[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
      const int row = mt * 16 + (lane >> 2) + (e & 1) * 8;
      const int g = row / m_pad, i = row % m_pad;
      const int dd = dim + (e >> 1) * 2;
      v[e] = 0u;
      if (g < group && i < n_lookahead) {
        const int64_t off = (((int64_t)layer * n_q_heads + hk * group + g) * n_lookahead + i) * head_dim + dd;
        v[e] = q32[off >> 1];
      }
    }
    qf[(int64_t)slab * total + idx] = make_uint4(v[0], v[1], v[2], v[3]);
  }
}

// Sweep 1.  grid = (n_split, n_slabs); every warp strides over the slab's 32-key tiles.
template <int D, int MT, bool FP8>
__global__ void __launch_bounds__(kThreads) score_lse_kernel(LayerPtrs kp, const uint4* __restrict__ qf,
                                                              float2* __restrict__ partial, int64_t n_tokens,
                                                              int64_t stride_head, int64_t stride_tok, int n_kv_heads,
                                                              float c, const float* __restrict__ k_scale, PagedView pv) {
  const int slab = blockIdx.y;
  const int layer = slab / n_kv_heads, hk = slab % n_kv_heads;
  const __nv_bfloat16* kslab = slab_base<FP8>(kp.p[layer], hk * stride_head);
  if (FP8) c *= __ldg(k_scale + slab);                 // the slab's key scale multiplies every logit
  const uint4* qslab = qf + (int64_t)slab * (MT * (D / 16) * 32);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t n_tiles = (n_tokens + kTileKeys - 1) / kTileKeys;
  const int64_t stride = (int64_t)gridDim.x * kWarpsPerCta;

  float run_m[MT][2], run_l[MT][2];
#pragma unroll
  for (int mt = 0; mt < MT; ++mt)
#pragma unroll
    for (int b = 0; b < 2; ++b) run_m[mt][b] = -INFINITY, run_l[mt][b] = 0.f;

  int64_t tile = (int64_t)blockIdx.x * kWarpsPerCta + warp;
  KeyTile<D> cur;
  if (tile < n_tiles) load_key_tile<D, FP8>(cur, kslab, tile_offset(tile * kTileKeys, stride_tok, pv), tile * kTileKeys, n_tokens, stride_tok, lane);
  while (tile < n_tiles) {
    const int64_t next = tile + stride;
    KeyTile<D> nxt;
    if (next < n_tiles) load_key_tile<D, FP8>(nxt, kslab, tile_offset(next * kTileKeys, stride_tok, pv), next * kTileKeys, n_tokens, stride_tok, lane);

    float acc[MT][4][4];
    tile_logits<D, MT>(acc, cur, qslab, lane);

    const int64_t left = n_tokens - tile * kTileKeys;  // keys of this tile that exist
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int b = 0; b < 2; ++b) {
        float v[8];
        float mx = -INFINITY;
#pragma unroll
        for (int nt = 0; nt < 4; ++nt)
#pragma unroll
          for (int e = 0; e < 2; ++e) {
            const int key = nt * 8 + (lane & 3) * 2 + e;
            const float t = key < left ? acc[mt][nt][2 * b + e] * c : -INFINITY;
            v[nt * 2 + e] = t;
            mx = fmaxf(mx, t);
          }
        const float m_new = fmaxf(run_m[mt][b], mx);
        const float ref = m_new == -INFINITY ? 0.f : m_new;
        float s = 0.f;
#pragma unroll
        for (int x = 0; x < 8; ++x) s += fast_exp2(v[x] - ref);
        run_l[mt][b] = run_l[mt][b] * fast_exp2(run_m[mt][b] - ref) + s;
        run_m[mt][b] = m_new;
      }
    cur = nxt;
    tile = next;
  }

  // merge the four lanes of a quad (they hold different keys of the same rows), then the warps
  __shared__ float2 warp_stats[kWarpsPerCta][MT * 16];
#pragma unroll
  for (int mt = 0; mt < MT; ++mt)
#pragma unroll
    for (int b = 0; b < 2; ++b) {
      float m = run_m[mt][b], l = run_l[mt][b];
#pragma unroll
      for (int off = 1; off <= 2; off <<= 1) {
        const float m2 = __shfl_xor_sync(0xffffffffu, m, off);
        const float l2 = __shfl_xor_sync(0xffffffffu, l, off);
        const float mm = fmaxf(m, m2);
        const float ref = mm == -INFINITY ? 0.f : mm;
        l = l * fast_exp2(m - ref) + l2 * fast_exp2(m2 - ref);
        m = mm;
      }
      if ((lane & 3) == 0) warp_stats[warp][mt * 16 + (lane >> 2) + 8 * b] = make_float2(m, l);
    }
  __syncthreads();
  if (threadIdx.x < MT * 16) {
    float m = -INFINITY, l = 0.f;
#pragma unroll
    for (int w = 0; w < kWarpsPerCta; ++w) {
      const float2 s = warp_stats[w][threadIdx.x];
      const float mm = fmaxf(m, s.x);
      const float ref = mm == -INFINITY ? 0.f : mm;
      l = l * fast_exp2(m - ref) + s.y * fast_exp2(s.x - ref);
      m = mm;
    }
    partial[((int64_t)slab * gridDim.x + blockIdx.x) * (MT * 16) + threadIdx.x] = make_float2(m, l);
  }
}

// Merges the per-CTA partials of sweep 1: lse2[slab][row] = M + log2(Z); optional natural-log copy for the caller.
__global__ void merge_lse_kernel(const float2* __restrict__ partial, float* __restrict__ lse2, float* __restrict__ lse_out,
                                 const float* __restrict__ extra_lse, int n_split, int rows_pad, int n_kv_heads, int group, int n_lookahead, int m_pad) {
  const int slab = blockIdx.x;
  const int row = threadIdx.x;
  if (row >= rows_pad) return;
  float m = -INFINITY;
  for (int s = 0; s < n_split; ++s) m = fmaxf(m, partial[((int64_t)slab * n_split + s) * rows_pad + row].x);
  float z = 0.f;
  for (int s = 0; s < n_split; ++s) {
    const float2 p = partial[((int64_t)slab * n_split + s) * rows_pad + row];
    z += p.y * exp2f(p.x - m);
  }
  float v = m + log2f(z);
  const int g = row / m_pad, i = row % m_pad;
  const int layer = slab / n_kv_heads, hk = slab % n_kv_heads;
  const int64_t out_idx = (((int64_t)layer * n_kv_heads + hk) * group + g) * n_lookahead + i;
  const bool real = g < group && i < n_lookahead;
  if (extra_lse != nullptr && real) {
    // the denominator also holds exp(extra): log2-add, in the order that cannot overflow
    const float e = extra_lse[out_idx] * kLog2e;
    const float hi = fmaxf(v, e), lo = fminf(v, e);
    v = hi + log2f(1.f + exp2f(lo - hi));
  }
  lse2[(int64_t)slab * rows_pad + row] = v;
  if (lse_out != nullptr && real) lse_out[out_idx] = v * kLn2;
}

// Key-sharded scoring: the row log-sum-exps of the WHOLE prompt come from the caller (natural log, [L][Hq][m]); this
// lays them out as sweep 2 reads them (base 2, padded rows).
__global__ void load_lse_kernel(const float* __restrict__ lse_in, float* __restrict__ lse2, int rows_pad, int n_kv_heads,
                                int group, int n_lookahead, int m_pad) {
  const int slab = blockIdx.x;
  const int row = threadIdx.x;
  if (row >= rows_pad) return;
  const int g = row / m_pad, i = row % m_pad;
  const int layer = slab / n_kv_heads, hk = slab % n_kv_heads;
  float v = 0.f;
  if (g < group && i < n_lookahead) v = lse_in[(((int64_t)layer * n_kv_heads + hk) * group + g) * n_lookahead + i] * kLog2e;
  lse2[(int64_t)slab * rows_pad + row] = v;
}

// Sweep 2.  One warp owns 32 keys for all slabs.  NI = m_pad / 8 lookahead indices live in a thread.
template <int D, int MT, int NI, bool FP8>
__global__ void __launch_bounds__(kThreads) score_max_kernel(LayerPtrs kp, const uint4* __restrict__ qf,
                                                              const float* __restrict__ lse2, float* __restrict__ importance,
                                                              int64_t n_tokens, int64_t stride_head, int64_t stride_tok,
                                                              int n_layers, int n_kv_heads, int group, int n_lookahead,
                                                              float c, const float* __restrict__ k_scale, PagedView pv) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int64_t tile = (int64_t)blockIdx.x * kWarpsPerCta + warp;
  const int64_t n_tiles = (n_tokens + kTileKeys - 1) / kTileKeys;
  if (tile >= n_tiles) return;
  const int64_t key0 = tile * kTileKeys;
  const int n_slabs = n_layers * n_kv_heads;

  float amax[NI][8];
#pragma unroll
  for (int s = 0; s < NI; ++s)
#pragma unroll
    for (int x = 0; x < 8; ++x) amax[s][x] = -INFINITY;

  KeyTile<D> cur;
  const int64_t tile_off = tile_offset(key0, stride_tok, pv);   // the same for every layer and kv-head
  load_key_tile<D, FP8>(cur, kp.p[0], tile_off, key0, n_tokens, stride_tok, lane);
  for (int slab = 0; slab < n_slabs; ++slab) {
    KeyTile<D> nxt;
    if (slab + 1 < n_slabs) {
      const int l2 = (slab + 1) / n_kv_heads, h2 = (slab + 1) % n_kv_heads;
      load_key_tile<D, FP8>(nxt, slab_base<FP8>(kp.p[l2], h2 * stride_head), tile_off, key0, n_tokens, stride_tok, lane);
    }
    float acc[MT][4][4];
    tile_logits<D, MT>(acc, cur, qf + (int64_t)slab * (MT * (D / 16) * 32), lane);
    const float cs = FP8 ? c * __ldg(k_scale + slab) : c;
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
      for (int b = 0; b < 2; ++b) {
        const int g = (2 * mt + b) / NI;          // head of the group this row belongs to
        const int slot = (2 * mt + b) % NI;       // which of the thread's lookahead indices
        const int i = slot * 8 + (lane >> 2);
        const bool live = g < group && i < n_lookahead;
        const float lse = live ? __ldg(lse2 + (int64_t)slab * (MT * 16) + mt * 16 + (lane >> 2) + 8 * b) : INFINITY;
#pragma unroll
        for (int nt = 0; nt < 4; ++nt)
#pragma unroll
          for (int e = 0; e < 2; ++e)
            amax[slot][nt * 2 + e] = fmaxf(amax[slot][nt * 2 + e], fmaf(acc[mt][nt][2 * b + e], cs, -lse));
      }
    cur = nxt;
  }

  const float inv_m = 1.f / (float)n_lookahead;
#pragma unroll
  for (int x = 0; x < 8; ++x) {
    float s = 0.f;
#pragma unroll
    for (int slot = 0; slot < NI; ++slot) s += fast_exp2(amax[slot][x]);
    s += __shfl_xor_sync(0xffffffffu, s, 4);
    s += __shfl_xor_sync(0xffffffffu, s, 8);
    s += __shfl_xor_sync(0xffffffffu, s, 16);
    const int64_t key = key0 + (x >> 1) * 8 + (lane & 3) * 2 + (x & 1);
    if ((lane >> 2) == 0 && key < n_tokens) importance[key] = s * inv_m;
  }
}

template <int D, int MT>
void launch_lse(const ScoreProblem& p, const uint4* qf, float2* partial, int n_split, cudaStream_t stream) {
  dim3 grid(n_split, p.n_layers * p.n_kv_heads);
  if (p.k_scale != nullptr)
    score_lse_kernel<D, MT, true><<<grid, kThreads, 0, stream>>>(p.k, qf, partial, p.n_tokens, p.stride_head, p.stride_tok,
                                                                 p.n_kv_heads, p.c_log2, p.k_scale, paged_view(p));
  else
    score_lse_kernel<D, MT, false><<<grid, kThreads, 0, stream>>>(p.k, qf, partial, p.n_tokens, p.stride_head, p.stride_tok,
                                                                  p.n_kv_heads, p.c_log2, nullptr, paged_view(p));
}

template <int D, int MT, int NI>
void launch_max(const ScoreProblem& p, const uint4* qf, const float* lse2, cudaStream_t stream) {
  const int64_t n_tiles = ceil_div(p.n_tokens, kTileKeys);
  const unsigned grid = (unsigned)ceil_div(n_tiles, kWarpsPerCta);
  if (p.k_scale != nullptr)
    score_max_kernel<D, MT, NI, true><<<grid, kThreads, 0, stream>>>(p.k, qf, lse2, p.importance, p.n_tokens, p.stride_head,
                                                                       p.stride_tok, p.n_layers, p.n_kv_heads, p.group,
                                                                       p.n_lookahead, p.c_log2, p.k_scale, paged_view(p));
  else
    score_max_kernel<D, MT, NI, false><<<grid, kThreads, 0, stream>>>(p.k, qf, lse2, p.importance, p.n_tokens, p.stride_head,
                                                                        p.stride_tok, p.n_layers, p.n_kv_heads, p.group,
                                                                        p.n_lookahead, p.c_log2, nullptr, paged_view(p));
}

template <int D, int MT>
void launch_max_ni(const ScoreProblem& p, const uint4* qf, const float* lse2, cudaStream_t stream) {
  switch (p.m_pad / 8) {
    case 1: launch_max<D, MT, 1>(p, qf, lse2, stream); break;
    case 2: launch_max<D, MT, 2>(p, qf, lse2, stream); break;
    case 3: launch_max<D, MT, 3>(p, qf, lse2, stream); break;
    default: launch_max<D, MT, 4>(p, qf, lse2, stream); break;
  }
}

// phase 0: both sweeps; 1: sweep 1 and the merge only (row log-sum-exps of the keys given); 2: sweep 2 only, with the
// row log-sum-exps `lse_in` supplied by the caller
template <int D>
void launch_both(const ScoreProblem& p, const uint4* qf, float2* partial, float* lse2, int n_split, int phase, const float* lse_in,
                 cudaStream_t stream) {
  const int rows_pad = p.rows_pad;
  const int n_slabs = p.n_layers * p.n_kv_heads;
  auto merge = [&]() {
    merge_lse_kernel<<<n_slabs, 64, 0, stream>>>(partial, lse2, p.lse_out, p.extra_lse, n_split, rows_pad, p.n_kv_heads, p.group,
                                                 p.n_lookahead, p.m_pad);
  };
  if (phase == 2)
    load_lse_kernel<<<n_slabs, 64, 0, stream>>>(lse_in, lse2, rows_pad, p.n_kv_heads, p.group, p.n_lookahead, p.m_pad);
  const bool s1 = phase != 2, s2 = phase != 1;
  switch (rows_pad / 16) {
    case 1: if (s1) { launch_lse<D, 1>(p, qf, partial, n_split, stream); merge(); } if (s2) launch_max_ni<D, 1>(p, qf, lse2, stream); break;
    case 2: if (s1) { launch_lse<D, 2>(p, qf, partial, n_split, stream); merge(); } if (s2) launch_max_ni<D, 2>(p, qf, lse2, stream); break;
    case 3: if (s1) { launch_lse<D, 3>(p, qf, partial, n_split, stream); merge(); } if (s2) launch_max_ni<D, 3>(p, qf, lse2, stream); break;
    default: if (s1) { launch_lse<D, 4>(p, qf, partial, n_split, stream); merge(); } if (s2) launch_max_ni<D, 4>(p, qf, lse2, stream); break;
  }
}

struct MmaLayout {
  size_t qf_off, lse2_off, partial_off, total;
};

MmaLayout mma_layout(const ScoreProblem& p) {
  const size_t n_slabs = (size_t)p.n_layers * p.n_kv_heads;
  MmaLayout w;
  w.qf_off = 0;
  w.lse2_off = align_up(w.qf_off + n_slabs * p.rows_pad * p.head_dim * 2, 256);
  w.partial_off = align_up(w.lse2_off + n_slabs * p.rows_pad * sizeof(float), 256);
  w.total = align_up(w.partial_off + n_slabs * kMmaMaxSplit * p.rows_pad * sizeof(float2), 256);
  return w;
}

}  // namespace

size_t score_mma_workspace_bytes(const ScoreProblem& p) { return mma_layout(p).total; }

int32_t score_mma_launch_phase(const ScoreProblem& p, void* workspace, int sm_count, int phase, const float* lse_in,
                               cudaStream_t stream) {
  const MmaLayout w = mma_layout(p);
  char* base = static_cast<char*>(workspace);
  uint4* qf = reinterpret_cast<uint4*>(base + w.qf_off);
  float* lse2 = reinterpret_cast<float*>(base + w.lse2_off);
  float2* partial = reinterpret_cast<float2*>(base + w.partial_off);
  const int n_slabs = p.n_layers * p.n_kv_heads;

  // about four waves of four resident CTAs per SM, but never more splits than 128-key blocks
  int64_t n_split = ceil_div((int64_t)sm_count * 16, n_slabs);
  n_split = std::min<int64_t>(n_split, ceil_div(p.n_tokens, kTileKeys * kWarpsPerCta));
  n_split = std::max<int64_t>(1, std::min<int64_t>(n_split, kMmaMaxSplit));

  pack_q_kernel<<<n_slabs, 128, 0, stream>>>(p.q, qf, p.n_kv_heads, p.group, p.n_lookahead, p.m_pad, p.head_dim,
                                             p.rows_pad / 16);
  if (p.head_dim == 64)
    launch_both<64>(p, qf, partial, lse2, (int)n_split, phase, lse_in, stream);
  else
    launch_both<128>(p, qf, partial, lse2, (int)n_split, phase, lse_in, stream);
  SPF_CUDA_CHECK(cudaGetLastError());
  return SPF_OK;
}

int32_t score_mma_launch(const ScoreProblem& p, void* workspace, int sm_count, cudaStream_t stream) {
  return score_mma_launch_phase(p, workspace, sm_count, 0, nullptr, stream);
}

}  // namespace spf
