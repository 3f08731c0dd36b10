// Token-importance scoring, fused path: ONE persistent kernel that reads the key cache once from HBM.
//
// Why two visits per key tile.  The max over (layer, head) is taken over softmax PROBABILITIES, so a
// logit can only be compared across heads after its row's log-sum-exp is known, and that needs all N
// keys of the row.  Each (layer, kv-head) slab of keys is therefore visited twice:
//   visit 1 ("sum")  accumulates  sum_s exp2(c * q.k - ref)  per query row;
//   visit 2 ("max")  folds  max_{l,h} (q.k - lse/c)  into a running maximum per (lookahead i, key s).
// The two visits are software-pipelined `lag` slabs apart and travel TOGETHER through the pipeline: stage
// (t, j) holds tile j of slab t for visit 1 (streamed from HBM, kept in L2 with an evict-last hint) and
// tile j of slab t - lag for visit 2 (read again by the same CTA, so from L2, with an evict-first hint).
//
// Work split.  The grid is persistent (one CTA per SM).  CTA b owns key tiles b, b + grid, ... (128
// keys each) of EVERY slab, so its running maxima for those keys stay on its SM (in tensor memory, next to
// the accumulator stages) for the whole kernel and the importance of a key is written exactly once, at the end.
//
// One tile = one tcgen05 MMA group: A = 128 keys x d (shared memory, TMA, 128-byte swizzle),
// B = the slab's query rows x d (row j = i * G + g: lookahead i, head g of the GQA group), D = fp32
// [128 keys x NCOLS rows] in tensor memory.  Keys are TMEM lanes, so an epilogue thread owns one key
// and sees all query rows of it: the max over heads is in-thread.
//
// Warps.  0: TMA producer of the first-visit tiles.  1: MMA issuer.  2: log-sum-exp warp (turns a slab's complete
// row sums into the offsets of visit 2).  3: reference warp (hands the per-slab reference of visit 1 to the sum warps,
// two slabs ahead).  4..11: "sum" warps, the visit-1 half of every stage (exp2-bound).  12..19: "max" warps, the
// visit-2 half (ALU / shared-memory bound); they also add up the per-key sums of the sum warps, which reach them
// through a shared-memory buffer once per slab.  20: TMA producer of the second-visit tiles.  21: publisher (reports
// this CTA's finished share of a slab to the other CTAs).  The two epilogue groups run independently, so the exp2
// work and the max work overlap on every scheduler.  The per-slab loops of warps 2, 3 and 21 are chains of memory
// round trips; with short slabs (few tiles per CTA) such a chain, not the tiles, sets the pace as soon as it grows.
// Hence a warp for each, and hence the references are computed once for all CTAs (each CTA a share of the slabs, at
// the start) instead of by every CTA for every slab.
//
// 8-bit key caches (template parameter FP8): the key tiles are E4M3 bytes (rows of d bytes: 64-byte swizzle at d = 64,
// the 128-byte one at d = 128), the instruction kind is f8f6f4 with 32 bytes of the row per instruction, and the
// queries come as two E4M3 terms per element from split_q_kernel, accumulated into the same columns -- the same number
// of instructions per tile as for bf16.  The factor from accumulated dot product to base-2 logit then differs per slab
// (softmax scale x key scale / query scale), so the epilogue multiplies by a per-slab value where the bf16 kernel has
// a constant and keeps the running maxima in base-2 logits.  The bf16 instantiations compile to what they were.
//
// Reference.  Visit 1 subtracts one reference per slab inside the exp2 argument: the SMALLEST logit of the slab's
// rows against one fixed sample key, plus a margin of 60 (base-2 units).  Every row's largest logit is at least
// its own sample logit, hence at least reference - 60, and ex2.approx.ftz only flushes terms below reference - 126,
// i.e. terms more than 2^66 times smaller than the row's largest: no row can lose anything that matters, whatever
// the spread between the heads of a group.  What can still go wrong is overflow: a row sum reaches 2^128 when some
// logit lies about 188 - log2(keys at that level) base-2 units (157 at the very least, about 109 nats) above the
// slab's smallest sample logit.  That is detected (the sum is inf) and reported as SPF_ERR_RANGE; the caller can
// then use the general path.
//
// Cross-CTA step.  All CTAs use the same reference for a slab, so their partial sums can simply be added.
// To make the total independent of the order in which CTAs arrive, the fp32 partial sums are added
// EXACTLY: each is split over two 40-bit limbs of a 280-bit fixed-point accumulator per row (64-bit integer
// atomics, no carries needed), which covers every finite fp32 value.  A counter per slab tells the
// log-sum-exp warp of every CTA when all shares are in; it then converts the accumulator to lse itself.
// Results are bit-identical from run to run.  Because visit 1 never waits on another CTA and all CTAs are
// co-resident, the counters always fill.
//
// Every wait on a barrier, counter or flag in this file is bounded: on expiry the kernel records SPF_ERR_TIMEOUT,
// drains and returns normally.  The one wait that has no limit is the hardware's own: tcgen05.alloc blocks while
// another resident CTA on the SM holds tensor memory (this kernel asks for all of it), i.e. until that CTA exits.
#include <cuda.h>

#include <algorithm>
#include <mutex>

#include "common.cuh"
#include "score.cuh"

namespace spf {
namespace {

constexpr int kTileKeys = 128;
constexpr int kThreads = 704;          // warp 0 TMA (first visit), 1 MMA issue, 2 log-sum-exp, 3 references, 4..19 epilogue, 20 TMA (second visit), 21 publisher
constexpr int kProducer2Warp = 20;
#ifndef SPF_FUSED_LB
#define SPF_FUSED_LB kThreads
#endif
constexpr int kPublisherWarp = 21;
constexpr int kLimbs = 7;              // 40-bit limbs of the exact row-sum accumulators (covers every finite fp32)
constexpr int kLimbStride = 8;         // 64-bit words per row in the accumulator array
constexpr int kQStages = 2;
constexpr int kTmemStages = 4;         // upper bound; the launch picks 2..4 (FusedArgs::t_stages)
constexpr int kTmemColsAll = 512;      // the CTA takes all of its SM's tensor memory
constexpr int kRefSlots = 16;         // row references stay readable for this many slabs (must exceed the lag)
constexpr int kPubSlots = 16;        // slabs whose hand-over to the publisher may be pending at once
constexpr float kRefMargin = 60.f;     // base-2 units added to the sampled reference logit
constexpr unsigned long long kTimeoutNs = 2000000000ull;
// Key rows are d bf16 (128 or 256 bytes) or d E4M3 bytes (64 or 128).  A tile is stored as sub-tiles of 128 keys x one swizzle
// span: 128 bytes of the row (128-byte swizzle), or the whole row where it has only 64 bytes (64-byte swizzle).
__host__ __device__ constexpr int row_bytes(int d, bool fp8) { return fp8 ? d : 2 * d; }
__host__ __device__ constexpr int sub_row_bytes(int rowb) { return rowb > 128 ? 128 : rowb; }

struct FusedMaps {
  CUtensorMap q;                      // (d, g, i, slab) view of the query tensor; 8-bit keys: (d, row, slab * 2 + part) view of the split queries
  CUtensorMap k[kFusedMaxLayers];     // (d, key, kv-head) view of each layer's key cache
};

struct FusedArgs {
  const __nv_bfloat16* k_layers[kFusedMaxLayers];
  const __nv_bfloat16* q;
  int64_t n_tokens, stride_head, stride_tok;
  int n_layers, n_kv_heads, n_lookahead, n_tiles, tiles_per_cta_max, lag, k_stages, t_stages;
  int mode;               // 0: the whole computation; 1: first visit only (row log-sum-exps of these keys); 2: second visit only
  const float* lse_in;    // mode 2: row log-sum-exps supplied by the caller, natural log, [L][Hq][m]
  float c, inv_c;
  // 8-bit key caches: the queries reach the tensor cores as two E4M3 terms per element (see split_q_kernel), scaled per
  // slab; slab_scale[slab] turns an accumulated dot product into base-2 logits (softmax scale, key scale and query scale
  // in one factor) and key_scale[slab] is the key cache's own scale.  Null for bf16 caches.
  const float* slab_scale;
  const float* key_scale;
  unsigned long long* limbs;  // [slab][NCOLS][kLimbStride] exact fixed-point sums of exp2(c*q.k - ref) over all keys
  unsigned* counters;     // [slab] CTAs whose share of the slab's row sums is in the accumulators
  unsigned* refs;         // [slab] the slab's first-visit reference (float bits, lowest bit set; zero = not computed yet)
  float* lse_out;         // optional [L][Hq][m], natural log
  const float* extra_lse; // optional [L][Hq][m], natural log: what each row's denominator holds besides the prompt keys
  float* importance;      // [N]
  int32_t* dev_status;    // optional
  // paged key cache: block_tokens > 0, k_layers[l] is the pool of layer l, stride_block elements between pool blocks
  const int32_t* block_table;
  int block_tokens;
  int64_t stride_block, n_pool_blocks;
};

// ---------------------------------------------------------------------------------------------- PTX
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ unsigned long long global_timer() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}

struct Abort {
  volatile int* flag;      // shared: set once any wait of this CTA ran out
  int32_t* dev_status;     // global, may be null
  unsigned long long timeout_ns = kTimeoutNs;   // how long a single wait may last
};

__device__ __noinline__ void record_timeout(const Abort& ab) {
  *ab.flag = 1;
  if (ab.dev_status != nullptr) atomicCAS(ab.dev_status, 0, (int32_t)SPF_ERR_TIMEOUT);
}

// Waits for the phase with the given parity; false if the CTA is aborting or the wait ran out.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, const Abort& ab) {
  if (mbar_try_wait(bar, parity)) return true;
  unsigned long long t0 = 0;
  for (uint32_t it = 1;; ++it) {
    if (mbar_try_wait(bar, parity)) return true;
    if (it > 2u) __nanosleep(64);   // do not poll hot next to the warps that do the arithmetic
    if ((it & 63u) == 0u) {
      if (*ab.flag) return false;
      const unsigned long long now = global_timer();
      if (t0 == 0) t0 = now;
      if (now - t0 > ab.timeout_ns) {
        record_timeout(ab);
        return false;
      }
    }
  }
}

// Warp-collective form: every lane waits, and all lanes agree on the outcome (a timeout seen by one
// lane only must not split the warp in front of .aligned instructions).
// Waits for two barriers at once: both are polled before either answer is looked at, so that their latencies overlap.
__device__ __forceinline__ bool mbar_wait2(uint32_t bar_a, uint32_t parity_a, uint32_t bar_b, uint32_t parity_b, const Abort& ab) {
  bool a = mbar_try_wait(bar_a, parity_a);
  bool b = mbar_try_wait(bar_b, parity_b);
  if (a && b) return true;
  unsigned long long t0 = 0;
  for (uint32_t it = 1;; ++it) {
    if (!a) a = mbar_try_wait(bar_a, parity_a);
    if (!b) b = mbar_try_wait(bar_b, parity_b);
    if (a && b) return true;
    if (it > 2u) __nanosleep(64);
    if ((it & 63u) == 0u) {
      if (*ab.flag) return false;
      const unsigned long long now = global_timer();
      if (t0 == 0) t0 = now;
      if (now - t0 > ab.timeout_ns) {
        record_timeout(ab);
        return false;
      }
    }
  }
}
__device__ __forceinline__ bool mbar_wait2_warp(uint32_t bar_a, uint32_t parity_a, uint32_t bar_b, uint32_t parity_b, const Abort& ab) {
  return __all_sync(0xffffffffu, mbar_wait2(bar_a, parity_a, bar_b, parity_b, ab));
}
__device__ __forceinline__ bool mbar_wait_warp(uint32_t bar, uint32_t parity, const Abort& ab) {
  return __all_sync(0xffffffffu, mbar_wait(bar, parity, ab));
}

// Waits until *counter (global) has reached `target`, with acquire semantics.
__device__ __forceinline__ bool count_wait(const unsigned* counter, unsigned target, const Abort& ab) {
  unsigned long long t0 = 0;
  for (uint32_t it = 0;; ++it) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(counter) : "memory");
    if (v >= target) return true;
    if ((it & 15u) == 15u) {
      if (*ab.flag) return false;
      const unsigned long long now = global_timer();
      if (t0 == 0) t0 = now;
      if (now - t0 > ab.timeout_ns) {
        record_timeout(ab);
        return false;
      }
      __nanosleep(100);
    }
  }
}


// Waits until *flag (shared memory, written by another warp of the CTA) has reached `target`.
// Waits until a word that starts as zero has been set (by another CTA) and returns its value in `value`.
__device__ __forceinline__ bool word_wait(const unsigned* word, unsigned& value, const Abort& ab) {
  unsigned long long t0 = 0;
  for (uint32_t it = 0;; ++it) {
    unsigned v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(word) : "memory");
    if (v != 0u) {
      value = v;
      return true;
    }
    if ((it & 15u) == 15u) {
      if (*ab.flag) return false;
      const unsigned long long now = global_timer();
      if (t0 == 0) t0 = now;
      if (now - t0 > ab.timeout_ns) {
        record_timeout(ab);
        return false;
      }
      __nanosleep(100);
    }
  }
}

__device__ __forceinline__ bool flag_wait(const volatile int* flag, int target, const Abort& ab) {
  unsigned long long t0 = 0;
  for (uint32_t it = 0;; ++it) {
    if (*flag >= target) {
      __threadfence_block();
      return true;
    }
    if ((it & 15u) == 15u) {
      if (*ab.flag) return false;
      const unsigned long long now = global_timer();
      if (t0 == 0) t0 = now;
      if (now - t0 > ab.timeout_ns) {
        record_timeout(ab);
        return false;
      }
      __nanosleep(100);
    }
  }
}

__device__ __forceinline__ void tma_load_3d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, uint32_t bar,
                                            uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3, %4}], [%5], %6;"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(bar), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void tma_load_4d_hint(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3,
                                                 uint32_t bar, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3, %4, %5}], [%6], %7;"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar), "l"(policy)
      : "memory");
}
// L2 eviction priorities for the key tiles: the first visit's tile is read again `lag` slabs later (keep it), the
// second visit's tile is dead once it has been read (let it go first)
__device__ __forceinline__ uint64_t l2_policy_keep() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t l2_policy_drop() {
  uint64_t p;
  asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void tma_load_4d(uint32_t dst, const CUtensorMap* map, int c0, int c1, int c2, int c3,
                                            uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
      ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(c2), "r"(c3), "r"(bar)
      : "memory");
}

// True in exactly one lane of the (converged) warp, the same lane every time.
__device__ __forceinline__ bool elect_one() {
  uint32_t pred;
  asm volatile("{\n.reg .pred p;\nelect.sync _|p, 0xffffffff;\nselp.u32 %0, 1, 0, p;\n}" : "=r"(pred));
  return pred != 0;
}

__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tc_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// One tensor-core instruction: M = 128 keys x N query rows x 32 bytes of the head dimension (16 bf16, or 32 E4M3 with
// both operands in that format).
template <bool FP8>
__device__ __forceinline__ void tc_mma(uint32_t tmem_d, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
  if constexpr (FP8)
    asm volatile(
        "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p;\n}"
        ::"r"(tmem_d), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
  else
    asm volatile(
        "{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}"
        ::"r"(tmem_d), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}

// Shared-memory operand descriptor: K-major rows of SUBROW bytes (128 or 64) with the swizzle of that span, 8-row groups
// 8 * SUBROW bytes apart.
template <int SUBROW>
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr) {
  static_assert(SUBROW == 128 || SUBROW == 64, "swizzle span");
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);   // start address / 16
  d |= (uint64_t)1 << 16;                    // leading byte offset (not used by swizzled K-major operands)
  d |= (uint64_t)((8 * SUBROW) >> 4) << 32;  // stride byte offset: 8 rows
  d |= (uint64_t)1 << 46;                    // descriptor version of this architecture
  d |= (uint64_t)(SUBROW == 128 ? 2 : 4) << 61;   // 128-byte / 64-byte swizzle
  return d;
}

// One E4M3 byte as fp32 (exact).
__device__ __forceinline__ float e4m3_to_float(uint32_t byte) {
  uint32_t h2;
  asm("{\n.reg .b16 lo;\ncvt.u16.u32 lo, %1;\ncvt.rn.f16x2.e4m3x2 %0, lo;\n}" : "=r"(h2) : "r"(byte & 0xffu));
  return __half2float(__ushort_as_half((unsigned short)(h2 & 0xffffu)));
}
// fp32 to the nearest E4M3 byte (saturating).
__device__ __forceinline__ uint32_t float_to_e4m3(float x) {
  uint32_t out;
  asm("{\n.reg .b16 r;\ncvt.rn.satfinite.e4m3x2.f32 r, %1, %2;\ncvt.u32.u16 %0, r;\n}" : "=r"(out) : "f"(0.f), "f"(x));
  return out & 0xffu;
}

// Instruction descriptor: bf16 x bf16 (operand format 1) or E4M3 x E4M3 (format 0) -> fp32, both operands K-major,
// M = 128, N = n.
__host__ __device__ constexpr uint32_t instr_desc(int n, bool fp8) {
  return (1u << 4) | ((fp8 ? 0u : 1u) << 7) | ((fp8 ? 0u : 1u) << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kTileKeys >> 4) << 24);
}

// TMEM -> registers, in two parts: tmem_issue starts the (asynchronous) load of N consecutive columns of the warp's
// 32 lanes, tmem_wait completes every load the thread has started.  The registers are listed as in/out operands of the wait so that no use can move above it.
template <int N>
__device__ __forceinline__ void tmem_issue(uint32_t taddr, uint32_t (&r)[N]);
template <int N>
__device__ __forceinline__ void tmem_wait(uint32_t (&r)[N]);

template <>
__device__ __forceinline__ void tmem_issue<1>(uint32_t taddr, uint32_t (&r)[1]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x1.b32 {%0}, [%1];" : "=r"(r[0]) : "r"(taddr));
}
template <>
__device__ __forceinline__ void tmem_wait<1>(uint32_t (&r)[1]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;" : "+r"(r[0]) : : "memory");
}
template <>
__device__ __forceinline__ void tmem_issue<2>(uint32_t taddr, uint32_t (&r)[2]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x2.b32 {%0,%1}, [%2];" : "=r"(r[0]), "=r"(r[1]) : "r"(taddr));
}
template <>
__device__ __forceinline__ void tmem_wait<2>(uint32_t (&r)[2]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;" : "+r"(r[0]), "+r"(r[1]) : : "memory");
}
template <>
__device__ __forceinline__ void tmem_issue<4>(uint32_t taddr, uint32_t (&r)[4]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0,%1,%2,%3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3])
               : "r"(taddr));
}
template <>
__device__ __forceinline__ void tmem_wait<4>(uint32_t (&r)[4]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;" : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]) : : "memory");
}
// registers -> TMEM (the warp's 32 lanes, N consecutive columns); tmem_store_wait completes the thread's stores
template <int N>
__device__ __forceinline__ void tmem_store(uint32_t taddr, const uint32_t (&r)[N]);
template <>
__device__ __forceinline__ void tmem_store<1>(uint32_t taddr, const uint32_t (&r)[1]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x1.b32 [%0], {%1};" ::"r"(taddr), "r"(r[0]) : "memory");
}
template <>
__device__ __forceinline__ void tmem_store<2>(uint32_t taddr, const uint32_t (&r)[2]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x2.b32 [%0], {%1,%2};" ::"r"(taddr), "r"(r[0]), "r"(r[1]) : "memory");
}
template <>
__device__ __forceinline__ void tmem_store<4>(uint32_t taddr, const uint32_t (&r)[4]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x4.b32 [%0], {%1,%2,%3,%4};" ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3])
               : "memory");
}
template <>
__device__ __forceinline__ void tmem_store<8>(uint32_t taddr, const uint32_t (&r)[8]) {
  asm volatile("tcgen05.st.sync.aligned.32x32b.x8.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8};" ::"r"(taddr), "r"(r[0]), "r"(r[1]),
               "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7])
               : "memory");
}
__device__ __forceinline__ void tmem_store_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

template <>
__device__ __forceinline__ void tmem_issue<8>(uint32_t taddr, uint32_t (&r)[8]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x8.b32 {%0,%1,%2,%3,%4,%5,%6,%7}, [%8];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7])
               : "r"(taddr));
}
template <>
__device__ __forceinline__ void tmem_wait<8>(uint32_t (&r)[8]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7])
               :
               : "memory");
}
template <>
__device__ __forceinline__ void tmem_issue<16>(uint32_t taddr, uint32_t (&r)[16]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
}
template <>
__device__ __forceinline__ void tmem_wait<16>(uint32_t (&r)[16]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]), "+r"(r[8]),
                 "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15])
               :
               : "memory");
}
template <>
__device__ __forceinline__ void tmem_issue<32>(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,%17,%18,%19,%20,"
      "%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
}
template <>
__device__ __forceinline__ void tmem_wait<32>(uint32_t (&r)[32]) {
  asm volatile("tcgen05.wait::ld.sync.aligned;"
               : "+r"(r[0]), "+r"(r[1]), "+r"(r[2]), "+r"(r[3]), "+r"(r[4]), "+r"(r[5]), "+r"(r[6]), "+r"(r[7]), "+r"(r[8]),
                 "+r"(r[9]), "+r"(r[10]), "+r"(r[11]), "+r"(r[12]), "+r"(r[13]), "+r"(r[14]), "+r"(r[15]), "+r"(r[16]),
                 "+r"(r[17]), "+r"(r[18]), "+r"(r[19]), "+r"(r[20]), "+r"(r[21]), "+r"(r[22]), "+r"(r[23]), "+r"(r[24]),
                 "+r"(r[25]), "+r"(r[26]), "+r"(r[27]), "+r"(r[28]), "+r"(r[29]), "+r"(r[30]), "+r"(r[31])
               :
               : "memory");
}

// ---------------------------------------------------------------------------------------------- layout

struct SmemLayout {
  uint32_t k_off, q_off, xbuf_off, ref_off, rowoff_off, tileblk_off, bar_off, misc_off, total;
};

__host__ __device__ inline SmemLayout smem_layout(int d, bool fp8, int ncols, int group, int k_stages, int tiles_per_cta_max) {
  SmemLayout s;
  uint32_t o = 0;
  const uint32_t rowb = (uint32_t)row_bytes(d, fp8);
  s.k_off = o;        o += (uint32_t)k_stages * 2 * kTileKeys * rowb;                 // stages of two key tiles
  s.q_off = o;        o += (uint32_t)kQStages * 2 * (fp8 ? 2 : 1) * ncols * rowb;      // stages of two query tiles (two terms each for 8-bit keys)
  s.xbuf_off = o;     o += (uint32_t)ncols * (kTileKeys / 4) * 4;
  s.ref_off = o;      o += kRefSlots * 4;
  s.rowoff_off = o;   o += 4 * 64 * 4;
  s.tileblk_off = o;  o += ((uint32_t)tiles_per_cta_max * 4 + 15u) & ~15u;
  s.bar_off = o;      o += 64 * 8;
  s.misc_off = o;     o += 64;
  s.total = o;
  return s;
}

// mbarrier addresses inside the barrier block
struct Bars {
  uint32_t base;
  int k_stages;
  __device__ uint32_t k_full(int s) const { return base + 8u * s; }
  __device__ uint32_t k_empty(int s) const { return base + 8u * (k_stages + s); }
  __device__ uint32_t q_full(int s) const { return base + 8u * (2 * k_stages + s); }
  __device__ uint32_t q_empty(int s) const { return base + 8u * (2 * k_stages + kQStages + s); }
  __device__ uint32_t t_full(int s) const { return base + 8u * (2 * k_stages + 2 * kQStages + s); }
  __device__ uint32_t t_empty(int s) const { return base + 8u * (2 * k_stages + 2 * kQStages + kTmemStages + s); }
  __device__ uint32_t o_ready(int x) const { return base + 8u * (2 * k_stages + 2 * kQStages + 2 * kTmemStages + x); }
  __device__ uint32_t o_free(int x) const { return base + 8u * (2 * k_stages + 2 * kQStages + 2 * kTmemStages + 4 + x); }
  __device__ uint32_t epi_sync() const { return base + 8u * (2 * k_stages + 2 * kQStages + 2 * kTmemStages + 8); }
  __device__ uint32_t mma_done() const { return base + 8u * (2 * k_stages + 2 * kQStages + 2 * kTmemStages + 9); }
  __device__ uint32_t pub_ready(int b) const { return base + 8u * (2 * k_stages + 2 * kQStages + 2 * kTmemStages + 10 + b); }
  __device__ uint32_t x_ready() const { return base + 8u * (2 * k_stages + 2 * kQStages + 2 * kTmemStages + 10 + kPubSlots); }
  __device__ uint32_t x_free() const { return base + 8u * (2 * k_stages + 2 * kQStages + 2 * kTmemStages + 11 + kPubSlots); }
};
// 2 * 10 + 2 * 2 + 2 * 4 + 10 + 16 + 2 = 60 barriers at most (10 key stages, kTmemStages = 4); the block has room for 64.

struct Ring {
  int stage = 0;
  uint32_t phase = 0;
  int n;
  __device__ explicit Ring(int n_) : n(n_) {}
  __device__ void advance() {
    if (++stage == n) {
      stage = 0;
      phase ^= 1u;
    }
  }
};

// Barrier among the epilogue warps, with a bounded wait (an mbarrier with one arrival per warp).
struct EpiSync {
  uint32_t bar;
  uint32_t phase = 0;
  __device__ bool sync(int lane, const Abort& ab) {
    __syncwarp();
    if (lane == 0) mbar_arrive(bar);
    const bool ok = mbar_wait_warp(bar, phase, ab);
    phase ^= 1u;
    return ok;
  }
};

// ---------------------------------------------------------------------------------------------- kernel
template <int D, int NCOLS, int G, bool FP8>
__global__ void __launch_bounds__(SPF_FUSED_LB, 1) score_fused_kernel(const __grid_constant__ FusedMaps maps,
                                                                   const __grid_constant__ FusedArgs a) {
  constexpr int EW = 16;                        // epilogue warps: 8 for the first visit (sums), 8 for the second (maxima)
  constexpr int EWV = EW / 2;                   // per visit: two warps per TMEM lane quadrant, half of the columns each
  constexpr int CW = NCOLS / 2;                 // query rows (TMEM columns) per epilogue thread: 8, 16 or 32
  constexpr int CHK = CW < 16 ? CW : 16;        // columns per tensor-memory load
  constexpr int NCH = CW / CHK;                 // loads per tile and thread: 1 or 2
  constexpr int NI = NCOLS / G;          // lookahead slots per key in the running-max array
  constexpr int ROWB = row_bytes(D, FP8);                   // bytes per key row: 64, 128 or 256
  constexpr int SUBROW = sub_row_bytes(ROWB);               // the swizzle span: 128 bytes, or the whole 64-byte row
  constexpr int KSUB = ROWB / SUBROW;                       // sub-tiles per key tile
  constexpr int KSTEPS = SUBROW / 32;                       // tensor-core instructions per sub-tile (32 bytes of the row each)
  constexpr int XSUB = SUBROW / (FP8 ? 1 : 2);              // elements per sub-tile row: the TMA x coordinate of sub-tile h is h * XSUB
  constexpr int kSubTileBytes = kTileKeys * SUBROW;
  constexpr int kSlotBytes = KSUB * kSubTileBytes;          // one key tile
  constexpr int kStageBytes = 2 * kSlotBytes;               // slot 0: first-visit tile, slot 1: second-visit tile
  constexpr int QPARTS = FP8 ? 2 : 1;                       // 8-bit keys: the queries come as two E4M3 terms
  constexpr int kQSub = NCOLS * SUBROW;
  constexpr int kQSlotBytes = QPARTS * KSUB * kQSub;
  constexpr int kTmemCols = kTmemColsAll;
  constexpr int NIH = (NCOLS / 2) / G;   // lookahead slots per max-warp thread
  constexpr int AC = NIH < 8 ? NIH : 8;  // running maxima moved per tensor-memory load / store
  // tensor memory: t_stages stages of 2 x NCOLS accumulator columns, then the running maxima, [local tile][NI]
  // columns (lane = key), which therefore never leave the SM either
  const uint32_t amax_col0 = (uint32_t)(a.t_stages * 2 * NCOLS);
  static_assert(CHK % G == 0, "a thread must own whole GQA groups");

  extern __shared__ unsigned char smem_raw[];
  // 1024-byte alignment by offsetting the shared array itself, so that the compiler still knows these are
  // shared-memory addresses (a round trip through an integer would turn every access into a generic one)
  unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  const SmemLayout lay = smem_layout(D, FP8, NCOLS, G, a.k_stages, a.tiles_per_cta_max);
  unsigned char* k_tiles = smem + lay.k_off;
  unsigned char* q_tiles = smem + lay.q_off;
  float* xbuf = reinterpret_cast<float*>(smem + lay.xbuf_off);         // [NCOLS][32]: partial row sums of one slab, each over four keys
  float* ref_slots = reinterpret_cast<float*>(smem + lay.ref_off);   // [kRefSlots]: slab references, kept until the log-sum-exp warp has used them
  int* tile_block = reinterpret_cast<int*>(smem + lay.tileblk_off);   // paged key cache: pool block of each of the CTA's tiles
  float* rowoff = reinterpret_cast<float*>(smem + lay.rowoff_off);   // [4 slots][64]: what the epilogue subtracts per row
  volatile int* misc = reinterpret_cast<volatile int*>(smem + lay.misc_off);  // [0] abort, [1] tmem base, [3] references written
  volatile float* slab_c = reinterpret_cast<volatile float*>(smem + lay.misc_off + 32);   // [4]: 8-bit keys: slab_scale of the slab in slot x
  const Bars bars{smem_u32(smem + lay.bar_off), a.k_stages};
  const Abort ab{misc, a.dev_status};

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int cta = blockIdx.x, n_cta = gridDim.x;
  const int n_slabs = a.n_layers * a.n_kv_heads;
  const int my_tiles = (a.n_tiles - cta + n_cta - 1) / n_cta;      // tiles cta, cta + n_cta, ...
  const int rows_real = G * a.n_lookahead;                         // query rows that exist (<= NCOLS)

  // ------------------------------------------------------------------ set-up
  if (threadIdx.x == 0) {
    misc[0] = 0;
    misc[1] = 0;
    misc[3] = 0;
    for (int s = 0; s < a.k_stages; ++s) {
      mbar_init(bars.k_full(s), 2);            // one arrival per producer warp
      mbar_init(bars.k_empty(s), 1);
    }
    for (int s = 0; s < kQStages; ++s) {
      mbar_init(bars.q_full(s), 2);
      mbar_init(bars.q_empty(s), 1);
    }
    for (int s = 0; s < a.t_stages; ++s) {
      mbar_init(bars.t_full(s), 1);
      mbar_init(bars.t_empty(s), EW);
    }
    for (int x = 0; x < 4; ++x) {
      mbar_init(bars.o_ready(x), 1);
      mbar_init(bars.o_free(x), EWV);
    }
    mbar_init(bars.epi_sync(), EW);
    mbar_init(bars.mma_done(), 1);
    for (int b = 0; b < kPubSlots; ++b) mbar_init(bars.pub_ready(b), EWV);
    mbar_init(bars.x_ready(), EWV);
    mbar_init(bars.x_free(), EWV);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // paged key cache: a tile never straddles a block (blocks are multiples of 128 tokens), one lookup per tile for the whole kernel
  if (a.block_tokens > 0)
    for (int lt = threadIdx.x; lt < my_tiles; lt += kThreads)
      tile_block[lt] = a.block_table[(int64_t)(cta + lt * n_cta) * kTileKeys / a.block_tokens];
  // zero the query stages: rows the TMA box does not cover must read as zero
  for (uint32_t i = threadIdx.x * 16; i < (uint32_t)kQStages * 2 * kQSlotBytes; i += kThreads * 16)
    *reinterpret_cast<uint4*>(q_tiles + i) = make_uint4(0, 0, 0, 0);
  fence_async_smem();
  if (warp == 0) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32((const void*)&misc[1])),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = (uint32_t)misc[1];

  // ------------------------------------------------------------------ roles
  if (warp == 0 || warp == kProducer2Warp) {
    // ===== TMA producers.  Stage (t, j) of the key ring holds tile j of slab t (first visit, slot 0, streamed from HBM)
    // and the same tile of slab t - lag (second visit, slot 1, normally still in L2); per run t the query tiles of both
    // slabs go to one stage of the query ring.  One thread starts a copy only every few hundred cycles, whatever the
    // copy's size, and a single producer thread was what bounded the whole kernel; so each visit has a producer warp of
    // its own (warp 0: first visit, warp 20: second).  Both arrive on the stage's "full" barrier: with the byte count
    // of their copies, or plainly where their visit has no slab (the first and last `lag` runs) =====
    if (lane == 0) {
      const int v = warp == 0 ? 0 : 1;
      Ring kr(a.k_stages), qr(kQStages);
      const uint64_t policy = v == 0 ? l2_policy_keep() : l2_policy_drop();
      bool ok = true;
      for (int t = 0; ok && t < n_slabs + a.lag; ++t) {
        const bool valid = v == 0 ? (t < n_slabs && a.mode != 2) : (t >= a.lag && a.mode != 1);
        const int slab = v == 0 ? t : t - a.lag;
        if (!(ok = mbar_wait(bars.q_empty(qr.stage), qr.phase ^ 1u, ab))) break;
        if (valid) {
          if constexpr (FP8) {
            mbar_expect_tx(bars.q_full(qr.stage), (uint32_t)kQSlotBytes);
            for (int part = 0; part < QPARTS; ++part)
              for (int h = 0; h < KSUB; ++h)
                tma_load_3d(smem_u32(q_tiles + (qr.stage * 2 + v) * kQSlotBytes + (part * KSUB + h) * kQSub), &maps.q, h * XSUB, 0,
                            slab * QPARTS + part, bars.q_full(qr.stage), policy);
          } else {
            mbar_expect_tx(bars.q_full(qr.stage), (uint32_t)(KSUB * rows_real * 128));
            for (int h = 0; h < KSUB; ++h)
              tma_load_4d(smem_u32(q_tiles + (qr.stage * 2 + v) * kQSlotBytes + h * kQSub), &maps.q, h * 64, 0, 0, slab,
                          bars.q_full(qr.stage));
          }
        } else {
          mbar_arrive(bars.q_full(qr.stage));
        }
        qr.advance();
        const int layer = valid ? slab / a.n_kv_heads : 0, hk = valid ? slab % a.n_kv_heads : 0;
        for (int lt = 0; lt < my_tiles; ++lt) {
          const int key0 = (cta + lt * n_cta) * kTileKeys;
          if (!(ok = mbar_wait(bars.k_empty(kr.stage), kr.phase ^ 1u, ab))) break;
          if (valid) {
            mbar_expect_tx(bars.k_full(kr.stage), (uint32_t)kSlotBytes);
            for (int h = 0; h < KSUB; ++h) {
              const uint32_t dst = smem_u32(k_tiles + kr.stage * kStageBytes + v * kSlotBytes + h * kSubTileBytes);
              if (a.block_tokens > 0)
                tma_load_4d_hint(dst, &maps.k[layer], h * XSUB, key0 % a.block_tokens, hk, tile_block[lt], bars.k_full(kr.stage), policy);
              else
                tma_load_3d(dst, &maps.k[layer], h * XSUB, key0, hk, bars.k_full(kr.stage), policy);
            }
          } else {
            mbar_arrive(bars.k_full(kr.stage));
          }
          kr.advance();
        }
      }
    }
  } else if (warp == 1) {
    // ===== MMA issuer.  The whole warp walks the loop (addresses and descriptors stay warp-uniform); one elected
    // lane issues the tensor-core instructions =====
    {
      Ring kr(a.k_stages), qr(kQStages), tr(a.t_stages);
      constexpr uint32_t idesc = instr_desc(NCOLS, FP8);
      const uint64_t k_desc0 = smem_desc<SUBROW>(smem_u32(k_tiles));
      const uint64_t q_desc0 = smem_desc<SUBROW>(smem_u32(q_tiles));
      bool ok = true;
      for (int t = 0; ok && t < n_slabs + a.lag; ++t) {
        const bool v1 = t < n_slabs && a.mode != 2, v2 = t >= a.lag && a.mode != 1;
        if (!(ok = mbar_wait_warp(bars.q_full(qr.stage), qr.phase, ab))) break;
        const uint64_t bd0 = q_desc0 + (uint64_t)((qr.stage * 2 * kQSlotBytes) >> 4);
        for (int lt = 0; lt < my_tiles; ++lt) {
          if (!(ok = mbar_wait2_warp(bars.k_full(kr.stage), kr.phase, bars.t_empty(tr.stage), tr.phase ^ 1u, ab))) break;
          tc_fence_after();
          const uint32_t d_tmem = tmem_base + (uint32_t)(tr.stage * 2 * NCOLS);
          const uint64_t ad0 = k_desc0 + (uint64_t)((kr.stage * kStageBytes) >> 4);
          if (elect_one()) {
#pragma unroll
            for (int v = 0; v < 2; ++v) {
              if (v == 0 ? v1 : v2) {
                // 8-bit keys: the two query terms accumulate into the same columns
#pragma unroll
                for (int part = 0; part < QPARTS; ++part) {
#pragma unroll
                  for (int h = 0; h < KSUB; ++h) {
#pragma unroll
                    for (int ks = 0; ks < KSTEPS; ++ks)
                      tc_mma<FP8>(d_tmem + (uint32_t)(v * NCOLS), ad0 + (uint64_t)((v * kSlotBytes + h * kSubTileBytes) >> 4) + 2u * ks,
                                  bd0 + (uint64_t)((v * kQSlotBytes + (part * KSUB + h) * kQSub) >> 4) + 2u * ks, idesc,
                                  (uint32_t)((part | h | ks) != 0));
                  }
                }
              }
            }
            tc_commit(bars.k_empty(kr.stage));
            tc_commit(bars.t_full(tr.stage));
          }
          __syncwarp();
          kr.advance();
          tr.advance();
        }
        if (!ok) break;
        if (elect_one()) tc_commit(bars.q_empty(qr.stage));   // arrives once the MMAs of the run are done
        __syncwarp();
        qr.advance();
      }
      // leave only after everything issued has completed and signalled its barriers
      if (ok) {
        if (elect_one()) tc_commit(bars.mma_done());
        __syncwarp();
        mbar_wait_warp(bars.mma_done(), 0u, ab);
      }
    }
  } else if (warp == 2) {
    // ===== log-sum-exp warp: once every CTA has added its share of a slab's row sums, turns the exact totals into
    // the per-row offsets of the second visit; lane handles rows lane and lane + 32 =====
    bool ok = true;
    for (int slab = 0; ok && slab < n_slabs; ++slab) {
      const int x = 2 + (slab & 1);
      const int use = slab >> 1;                                // how often slot x was written before
      if (a.mode == 2) {
        // the row log-sum-exps come from the caller: no sums of our own to wait for
        float value[2] = {0.f, 0.f};
#pragma unroll
        for (int r = 0; r < 2; ++r) {
          const int row = lane + 32 * r;
          if (row < rows_real)
            value[r] = __ldg(a.lse_in + ((int64_t)slab * G + row % G) * a.n_lookahead + row / G) * kLog2e * (FP8 ? 1.f : a.inv_c);
        }
        if (use > 0) {
          if (!(ok = mbar_wait_warp(bars.o_free(x), (uint32_t)(use - 1) & 1u, ab))) break;
        }
#pragma unroll
        for (int r = 0; r < 2; ++r) {
          const int row = lane + 32 * r;
          if (row < NCOLS) rowoff[x * 64 + row] = value[r];
        }
        if constexpr (FP8) {
          if (lane == 0) slab_c[x] = __ldg(a.slab_scale + slab);
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(bars.o_ready(x));
        continue;
      }
      if (!(ok = __all_sync(0xffffffffu, count_wait(a.counters + slab, (unsigned)n_cta, ab)))) break;
      unsigned long long w[2][kLimbs];
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        const int row = min(lane + 32 * r, rows_real - 1);
        const unsigned long long* acc = a.limbs + ((int64_t)slab * NCOLS + row) * kLimbStride;
#pragma unroll
        for (int i = 0; i < kLimbs; ++i) w[r][i] = __ldcg(acc + i);
      }
      // the reference of this slab was written by the reference warp at least `lag` runs ago
      if (!(ok = __all_sync(0xffffffffu, flag_wait(&misc[3], slab + 1, ab)))) break;
      const float ref = ref_slots[slab % kRefSlots];
      float value[2] = {0.f, 0.f};
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        const int row = lane + 32 * r;
        if (row < rows_real) {
          double total = 0.0;                                  // sum of limb_i * 2^(40 i - 149), exact to 2^-53
#pragma unroll
          for (int i = kLimbs - 1; i >= 0; --i) total += __longlong_as_double((long long)(1023 + 40 * i - 149) << 52) * (double)w[r][i];
          // log2 of the total: its binary exponent plus the log2 of its mantissa in single precision
          const long long tb = __double_as_longlong(total);
          const int expo = (int)((tb >> 52) & 0x7ff) - 1023;
          const float mant = (float)__longlong_as_double((tb & 0x000fffffffffffffll) | 0x3ff0000000000000ll);
          float lse2 = ref + ((float)expo + log2f(mant));
          if (!(total > 0.0) || expo == 1024) lse2 = INFINITY;  // an empty or overflowed row sum
          const int64_t out_idx = ((int64_t)slab * G + row % G) * a.n_lookahead + row / G;
          if (a.extra_lse != nullptr) {
            // the denominator also holds exp(extra): log2-add, in the order that cannot overflow
            const float e = __ldg(a.extra_lse + out_idx) * kLog2e;
            const float hi = fmaxf(lse2, e), lo = fminf(lse2, e);
            lse2 = hi + log2f(1.f + exp2f(lo - hi));
          }
          if (!(lse2 > -INFINITY && lse2 < INFINITY) && a.dev_status != nullptr)
            atomicCAS(a.dev_status, 0, (int32_t)SPF_ERR_RANGE);
          value[r] = FP8 ? lse2 : lse2 * a.inv_c;               // lse in q.k units (8-bit keys: in base-2 logits, the scale differs per slab)
          if (cta == 0 && a.lse_out != nullptr) a.lse_out[out_idx] = lse2 * kLn2;
        }
      }
      if (a.mode == 1) continue;                                 // no second visit: nobody reads the offsets
      if (use > 0) {
        if (!(ok = mbar_wait_warp(bars.o_free(x), (uint32_t)(use - 1) & 1u, ab))) break;
      }
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        const int row = lane + 32 * r;
        if (row < NCOLS) rowoff[x * 64 + row] = value[r];
      }
      if constexpr (FP8) {
        if (lane == 0) slab_c[x] = __ldg(a.slab_scale + slab);
      }
      __syncwarp();
      if (lane == 0) mbar_arrive(bars.o_ready(x));
    }
  } else if (warp == 3) {
    // ===== reference warp.  The reference of a slab's first visit is the smallest logit of the slab's rows against one
    // fixed sample key, plus a margin.  It depends on the inputs only and is the same for every CTA, so the CTAs share
    // the work: CTA c computes the references of slabs c, c + n_cta, ... once, at the start, and stores them in global
    // memory (a zero word = not there yet, so a stored value has its lowest bit set: every reader sees the same
    // number, which is all that matters for a reference).  Afterwards the warp only feeds the epilogue: 32 slabs'
    // references are fetched at a time, one per lane, and written to the slot of slab - 2 as soon as that is free =====
    bool ok = true;
    const int64_t sample_key = a.n_tokens / 2;                  // the same key for every slab and CTA
    // where that key sits: its row inside its pool block when the cache is paged (a bad table entry is clamped: this is a
    // plain load, not a bounds-checked TMA copy)
    int64_t sample_block = 0, sample_row = sample_key;
    if (a.block_tokens > 0) {
      sample_block = min(max((int64_t)__ldg(a.block_table + sample_key / a.block_tokens), (int64_t)0), a.n_pool_blocks - 1);
      sample_row = sample_key % a.block_tokens;
    }
    constexpr int LPR = D / 8;                                  // lanes per row: 8 bf16 of it each
    constexpr int RPP = 32 / LPR;                               // rows per pass of the warp
    constexpr int PASSES = NCOLS / RPP;                         // 4..32
    constexpr int BATCH = PASSES < 8 ? PASSES : 8;              // loads in flight per lane
    for (int slab = cta; slab < n_slabs && a.mode != 2; slab += n_cta) {
      const int layer = slab / a.n_kv_heads, hk = slab % a.n_kv_heads;
      float kf[8];
      if constexpr (FP8) {
        // strides count bytes; a lane's 8 keys elements are 8 bytes
        const uint2 kv = __ldg(reinterpret_cast<const uint2*>(reinterpret_cast<const unsigned char*>(a.k_layers[layer]) +
                                                              hk * a.stride_head + sample_row * a.stride_tok) + lane % LPR);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          kf[e] = e4m3_to_float(kv.x >> (8 * e));
          kf[4 + e] = e4m3_to_float(kv.y >> (8 * e));
        }
      } else {
        const uint4 kv = __ldg(reinterpret_cast<const uint4*>(a.k_layers[layer] + sample_block * a.stride_block + hk * a.stride_head +
                                                              sample_row * a.stride_tok) + lane % LPR);
        const __nv_bfloat162* k2 = reinterpret_cast<const __nv_bfloat162*>(&kv);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float2 f = __bfloat1622float2(k2[e]);
          kf[2 * e] = f.x;
          kf[2 * e + 1] = f.y;
        }
      }
      // the smallest sample logit of the slab's rows (padding rows repeat a real one).  The smallest, so that no row's
      // sum can underflow (see the header).  A softmax scale is positive, so the smallest q.k is the smallest logit
      float ref = INFINITY;
#pragma unroll 1
      for (int p0 = 0; p0 < PASSES; p0 += BATCH) {
        uint4 qv[BATCH];
#pragma unroll
        for (int b = 0; b < BATCH; ++b) {
          const int row = min((p0 + b) * RPP + lane / LPR, rows_real - 1);
          qv[b] = __ldg(reinterpret_cast<const uint4*>(a.q + (((int64_t)slab * G + row % G) * a.n_lookahead + row / G) * D) + lane % LPR);
        }
#pragma unroll
        for (int b = 0; b < BATCH; ++b) {
          const __nv_bfloat162* q2 = reinterpret_cast<const __nv_bfloat162*>(&qv[b]);
          float dot = 0.f;
#pragma unroll
          for (int e = 0; e < 4; ++e) {
            const float2 qf = __bfloat1622float2(q2[e]);
            dot = fmaf(kf[2 * e], qf.x, fmaf(kf[2 * e + 1], qf.y, dot));
          }
#pragma unroll
          for (int off = LPR / 2; off >= 1; off >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, off);
          ref = fminf(ref, dot);
        }
      }
#pragma unroll
      for (int off = 16; off >= LPR; off >>= 1) ref = fminf(ref, __shfl_xor_sync(0xffffffffu, ref, off));
      ref = fmaf(ref, FP8 ? a.c * __ldg(a.key_scale + slab) : a.c, kRefMargin);   // base-2 units, plus the margin
      if (lane == 0) {
        const unsigned word = __float_as_uint(ref) | 1u;
        asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(a.refs + slab), "r"(word) : "memory");
      }
    }
    unsigned mine = 0u;                                          // lane's reference of slab (slab & ~31) + lane
    float mine_c = 0.f;                                          // 8-bit keys: and its slab_scale
    for (int slab = 0; ok && slab < n_slabs && a.mode != 2; ++slab) {
      if ((slab & 31) == 0) {
        mine = 1u;
        if constexpr (FP8) mine_c = slab + lane < n_slabs ? __ldg(a.slab_scale + slab + lane) : 0.f;
        const bool got = slab + lane >= n_slabs || word_wait(a.refs + slab + lane, mine, ab);
        if (!(ok = __all_sync(0xffffffffu, got))) break;
      }
      const float ref = __uint_as_float(__shfl_sync(0xffffffffu, mine, slab & 31));
      float ref_c = 0.f;
      if constexpr (FP8) ref_c = __shfl_sync(0xffffffffu, mine_c, slab & 31);
      const int x = slab & 1;
      const int use = slab >> 1;
      if (use > 0) {
        // free since the sum warps picked up the reference of slab - 2, i.e. since they began that slab
        if (!(ok = mbar_wait_warp(bars.o_free(x), (uint32_t)(use - 1) & 1u, ab))) break;
      }
      if (lane == 0) {
        rowoff[x * 64] = ref;
        if constexpr (FP8) slab_c[x] = ref_c;
        ref_slots[slab % kRefSlots] = ref;
        __threadfence_block();
        misc[3] = slab + 1;                                    // the log-sum-exp warp reads ref_slots after this
        mbar_arrive(bars.o_ready(x));
      }
      __syncwarp();
    }
  } else if (warp == kPublisherWarp) {
    // ===== publisher warp: once this CTA's shares of a slab have been added to the accumulators, orders those
    // additions before the arrival count and reports the CTA (keeps the fence and the atomic's round trip off the
    // epilogue warps) =====
    bool ok = true;
    for (int ps = 0; ok && ps < n_slabs && a.mode != 2; ++ps) {
      if (!(ok = mbar_wait_warp(bars.pub_ready(ps % kPubSlots), (uint32_t)(ps / kPubSlots) & 1u, ab))) break;
      if (lane == 0) {
        __threadfence();
        atomicAdd(a.counters + ps, 1u);
      }
      __syncwarp();
    }
  } else if (warp >= 4 && warp < 4 + EW) {
    // ===== epilogue.  Warps 4..11 ("sum" warps) take the first-visit tile of every stage, warps 12..19 ("max" warps)
    // the second-visit tile; warp % 4 picks the TMEM lane quadrant (32 keys), the next bit the half of the query
    // rows.  The two groups run on their own: the exp2-bound and the max-bound work overlap on each scheduler =====
    const int quad = warp & 3;
    const bool is_sum = warp < 4 + EWV;
    const int half = ((warp - 4) >> 2) & 1;
    const uint32_t lane_addr = (uint32_t)(quad * 32) << 16;
    const int n_full_tiles = (int)(a.n_tokens / kTileKeys);     // tiles below this index have 128 real keys
    Ring tr(a.t_stages);
    EpiSync es{bars.epi_sync()};
    bool ok = true;
    if (is_sum) {
      for (int t = 0; ok && t < n_slabs + a.lag; ++t) {
        if (t >= n_slabs || a.mode == 2) {
          // nothing to sum (any more): keep the stage hand-over going
          for (int lt = 0; lt < my_tiles; ++lt) {
            if (!(ok = mbar_wait_warp(bars.t_full(tr.stage), tr.phase, ab))) break;
            if (lane == 0) mbar_arrive(bars.t_empty(tr.stage));
            tr.advance();
          }
          continue;
        }
        const int slab = t, x1 = slab & 1;
        if (!(ok = mbar_wait_warp(bars.o_ready(x1), (uint32_t)(slab >> 1) & 1u, ab))) break;
        const float nref = -rowoff[x1 * 64];                    // one reference per slab
        const float c1 = FP8 ? slab_c[x1] : a.c;                // accumulated dot product -> base-2 logit
        __syncwarp();
        if (lane == 0) mbar_arrive(bars.o_free(x1));
        float sum[CW];
#pragma unroll
        for (int j = 0; j < CW; ++j) sum[j] = 0.f;
        for (int lt = 0; lt < my_tiles; ++lt) {
          const int tile = cta + lt * n_cta;
          const bool real = tile < n_full_tiles || (int64_t)tile * kTileKeys + quad * 32 + lane < a.n_tokens;
          if (!(ok = mbar_wait_warp(bars.t_full(tr.stage), tr.phase, ab))) break;
          tc_fence_after();
          const uint32_t taddr = tmem_base + lane_addr + (uint32_t)(tr.stage * 2 * NCOLS + half * CW);
          // chunk by chunk: load, wait, compute.  No load is kept in flight across the arithmetic: with one pending,
          // the warp's exp2 stream ran markedly slower (measured), and the other warps hide the latency anyway
#pragma unroll
          for (int c = 0; c < NCH; ++c) {
            uint32_t r[CHK];
            tmem_issue<CHK>(taddr + (uint32_t)(c * CHK), r);
            tmem_wait<CHK>(r);
            if (c + 1 == NCH) {
              // the stage can be overwritten: its last chunk is in registers
              tc_fence_before();
              __syncwarp();
              if (lane == 0) mbar_arrive(bars.t_empty(tr.stage));
              tr.advance();
            }
            // per-thread sums of exp2 over the thread's keys
            if (real) {
#pragma unroll
              for (int j = 0; j < CHK; ++j) sum[c * CHK + j] += fast_exp2(fmaf(__uint_as_float(r[j]), c1, nref));
            }
          }
        }
        if (!ok) break;
        // hand the per-key sums to the max warps through shared memory: they have the slack to add them up over
        // the 128 keys and into the row accumulators (in a fixed order, so the result stays deterministic)
        if (slab > 0) {
          if (!(ok = mbar_wait_warp(bars.x_free(), (uint32_t)(slab - 1) & 1u, ab))) break;
        }
        // two transposing butterfly steps first (sums over 4 keys, a quarter of the columns left per thread): the buffer
        // is a quarter of the size, which buys another stage of the key ring
        {
          int width = CW;
#pragma unroll
          for (int off = 16; off >= 8; off >>= 1) {
            width >>= 1;
            const bool upper = (lane & off) != 0;
#pragma unroll
            for (int j = 0; j < CW / 2; ++j) {
              if (j < width) {
                const float send = upper ? sum[j] : sum[j + width];
                const float keep = upper ? sum[j + width] : sum[j];
                sum[j] = keep + __shfl_xor_sync(0xffffffffu, send, off);
              }
            }
          }
        }
        {
          const int col0 = half * CW + ((lane & 16) ? CW / 2 : 0) + ((lane & 8) ? CW / 4 : 0);
          // the position within the row is permuted by the (lane & 24) bits so that the four column groups of a warp
          // do not collide on the same banks; the readers add up whole rows, so the order does not matter to them
          const int pos = ((quad ^ (lane >> 3)) & 3) * 8 + (lane & 7);
#pragma unroll
          for (int j = 0; j < CW / 4; ++j) xbuf[(col0 + j) * (kTileKeys / 4) + pos] = sum[j];
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(bars.x_ready());
      }
    } else {
      // adds up the per-key sums of slab `slab` (written by the sum warps) and adds each row's total, exactly, to the
      // row's fixed-point accumulator (value = mantissa * 2^(p - 149), p = biased exponent - 1)
      constexpr int XC = NCOLS / EWV;                          // rows per max warp: 2, 4 or 8
      const int xw = warp - 4 - EWV;                           // 0..7
      auto reduce_slab = [&](int slab) -> bool {
        if (!mbar_wait_warp(bars.x_ready(), (uint32_t)slab & 1u, ab)) return false;
        float tot = 0.f;
#pragma unroll
        for (int j = 0; j < XC; ++j) {
          float sacc = xbuf[(xw * XC + j) * (kTileKeys / 4) + lane];
#pragma unroll
          for (int off = 16; off >= 1; off >>= 1) sacc += __shfl_xor_sync(0xffffffffu, sacc, off);
          if (lane == j) tot = sacc;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(bars.x_free());
        if (lane < XC) {
          const uint32_t bits = __float_as_uint(tot);
          const uint32_t expo = bits >> 23;                  // sums are non-negative: no sign bit
          if (expo == 255u) {
            if (a.dev_status != nullptr) atomicCAS(a.dev_status, 0, (int32_t)SPF_ERR_RANGE);
          } else if (expo != 0u) {
            const unsigned long long mant = (unsigned long long)((bits & 0x7FFFFFu) | 0x800000u);
            const uint32_t pos = expo - 1u, limb = pos / 40u, off = pos % 40u;
            unsigned long long* acc = a.limbs + ((int64_t)slab * NCOLS + xw * XC + lane) * kLimbStride + limb;
            const unsigned long long lo = (mant << off) & ((1ull << 40) - 1ull), hi = mant >> (40u - off);
            atomicAdd(acc, lo);
            if (hi != 0ull) atomicAdd(acc + 1, hi);
          }
        }
        // hand over to the publisher warp, which makes the additions visible and counts this CTA in
        __syncwarp();
        if (lane == 0) mbar_arrive(bars.pub_ready(slab % kPubSlots));
        return true;
      };
      {
        uint32_t ninf[AC];
#pragma unroll
        for (int j = 0; j < AC; ++j) ninf[j] = 0xff800000u;      // -inf
        for (int lt = 0; lt < my_tiles; ++lt)
#pragma unroll
          for (int q = 0; q < NIH / AC; ++q)
            tmem_store<AC>(tmem_base + lane_addr + amax_col0 + (uint32_t)(lt * NI + half * NIH + q * AC), ninf);
        tmem_store_wait();
      }
      for (int t = 0; ok && t < n_slabs + a.lag; ++t) {
        if (t < a.lag || a.mode == 1) {
          for (int lt = 0; lt < my_tiles; ++lt) {
            if (!(ok = mbar_wait_warp(bars.t_full(tr.stage), tr.phase, ab))) break;
            if (lane == 0) mbar_arrive(bars.t_empty(tr.stage));
            tr.advance();
          }
          if (ok && t < n_slabs && a.mode != 2) ok = reduce_slab(t);
          continue;
        }
        const int slab = t - a.lag, x2 = 2 + (slab & 1);
        if (!(ok = mbar_wait_warp(bars.o_ready(x2), (uint32_t)(slab >> 1) & 1u, ab))) break;
        const float4* off2 = reinterpret_cast<const float4*>(rowoff + x2 * 64 + half * CW);
        [[maybe_unused]] const float c2 = FP8 ? slab_c[x2] : 0.f;
        for (int lt = 0; lt < my_tiles; ++lt) {
          if (!(ok = mbar_wait_warp(bars.t_full(tr.stage), tr.phase, ab))) break;
          tc_fence_after();
          const uint32_t taddr = tmem_base + lane_addr + (uint32_t)(tr.stage * 2 * NCOLS + NCOLS + half * CW);
          // this tile's running maxima come in with the first chunk (one wait covers both loads)
          const uint32_t am_addr = tmem_base + lane_addr + amax_col0 + (uint32_t)(lt * NI + half * NIH);
          uint32_t am[NIH / AC][AC];
#pragma unroll
          for (int q = 0; q < NIH / AC; ++q) tmem_issue<AC>(am_addr + (uint32_t)(q * AC), am[q]);
#pragma unroll
          for (int c = 0; c < NCH; ++c) {
            uint32_t r[CHK];
            tmem_issue<CHK>(taddr + (uint32_t)(c * CHK), r);
            tmem_wait<CHK>(r);
            if (c == 0) {
#pragma unroll
              for (int q = 0; q < NIH / AC; ++q) tmem_wait<AC>(am[q]);
            }
            if (c + 1 == NCH) {
              tc_fence_before();
              __syncwarp();
              if (lane == 0) mbar_arrive(bars.t_empty(tr.stage));
              tr.advance();
            }
            float o[CHK];
#pragma unroll
            for (int j = 0; j < CHK / 4; ++j) {
              const float4 v = off2[c * (CHK / 4) + j];
              o[4 * j] = v.x; o[4 * j + 1] = v.y; o[4 * j + 2] = v.z; o[4 * j + 3] = v.w;
            }
            // running max over (layer, head) of q.k - lse/c (slots past n_lookahead hold padding and are never read)
#pragma unroll
            for (int ii = 0; ii < CHK / G; ++ii) {
              // bf16 keys: q.k - lse/c, one scale for all slabs; 8-bit keys: base-2 logit - lse, the scale differs per slab
              float mx = FP8 ? fmaf(__uint_as_float(r[ii * G]), c2, -o[ii * G]) : __uint_as_float(r[ii * G]) - o[ii * G];
#pragma unroll
              for (int g = 1; g < G; ++g)
                mx = fmaxf(mx, FP8 ? fmaf(__uint_as_float(r[ii * G + g]), c2, -o[ii * G + g]) : __uint_as_float(r[ii * G + g]) - o[ii * G + g]);
              const int i = c * (CHK / G) + ii;
              am[i / AC][i % AC] = __float_as_uint(fmaxf(__uint_as_float(am[i / AC][i % AC]), mx));
            }
          }
#pragma unroll
          for (int q = 0; q < NIH / AC; ++q) tmem_store<AC>(am_addr + (uint32_t)(q * AC), am[q]);
          tmem_store_wait();
        }
        if (!ok) break;
        __syncwarp();
        if (lane == 0) mbar_arrive(bars.o_free(x2));
        if (t < n_slabs && a.mode != 2) ok = reduce_slab(t);
      }
    }
    // ---------------- importance: mean over lookahead of exp2(c * running max) ----------------
    tc_fence_before();
    if (ok) ok = es.sync(lane, ab);
    tc_fence_after();
    if (ok && misc[0] == 0 && a.mode != 1) {
      // the four warps of a TMEM lane quadrant share its tiles; a thread reads all lookahead slots of its key
      constexpr int FC = NI < 16 ? NI : 16;
      const float inv_m = 1.f / (float)a.n_lookahead;
      for (int lt = (warp - 4) >> 2; lt < my_tiles; lt += EW / 4) {
        const int64_t key = (int64_t)(cta + lt * n_cta) * kTileKeys + quad * 32 + lane;
        float sacc = 0.f;
#pragma unroll
        for (int q = 0; q < NI / FC; ++q) {
          uint32_t v[FC];
          tmem_issue<FC>(tmem_base + lane_addr + amax_col0 + (uint32_t)(lt * NI + q * FC), v);
          tmem_wait<FC>(v);
#pragma unroll
          for (int j = 0; j < FC; ++j)
            if (q * FC + j < a.n_lookahead) sacc += fast_exp2(FP8 ? __uint_as_float(v[j]) : __uint_as_float(v[j]) * a.c);
        }
        if (key < a.n_tokens) a.importance[key] = sacc * inv_m;
      }
    }
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (misc[0] != 0) {
    // a wait ran out somewhere: give copies and MMAs still in flight time to land before TMEM goes away
    const unsigned long long t0 = global_timer();
    while (global_timer() - t0 < 2000000ull) __nanosleep(1000);
  }
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

// ---------------------------------------------------------------------------------------------- 8-bit keys: query split
// The tensor cores multiply E4M3 keys only by operands of an 8-bit format, so a slab's bf16 queries are handed over as
// two E4M3 terms, q * S = hi + lo: hi = the nearest E4M3 of q * S, lo = the nearest E4M3 of the remainder.  S is a power
// of two per slab that puts the slab's largest |q| just below the format's maximum (448).  A bf16 has 8 significant
// bits and each term carries 4, so the pair is exact for every element within 2^9 of the slab's largest and off by at
// most 2^-17 of that largest value below (the remainder's last bits fall under the format's smallest step, 2^-9).  One
// block per slab writes [slab][term][NCOLS rows][d] bytes (row j = i * G + g, padding rows zero) and the slab's
// factor from accumulated dot product to base-2 logit: softmax scale * log2(e) * key scale / S.
__global__ void __launch_bounds__(256) split_q_kernel(const __nv_bfloat16* __restrict__ q, int G, int m, int d, int ncols,
                                                      const float* __restrict__ key_scale, float c, unsigned char* __restrict__ out,
                                                      float* __restrict__ slab_scale) {
  const int slab = blockIdx.x;
  const int rows = G * m, n = rows * d;
  __shared__ float red[8];
  __shared__ float s_scale;
  float mx = 0.f;
  for (int idx = threadIdx.x; idx < n; idx += blockDim.x) {
    const int j = idx / d, e = idx - j * d;
    mx = fmaxf(mx, fabsf(__bfloat162float(q[(((int64_t)slab * G + j % G) * m + j / G) * d + e])));
  }
  for (int off = 16; off >= 1; off >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, off));
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = mx;
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < 8; ++w) mx = fmaxf(mx, red[w]);
    // largest power of two S with mx * S <= 448 (mx = 0 or not finite: S = 1)
    float S = 1.f;
    if (mx > 0.f && mx < INFINITY) {
      int ex;
      const float fr = frexpf(448.f / mx, &ex);   // 448 / mx = fr * 2^ex, fr in [0.5, 1)
      (void)fr;
      S = ldexpf(1.f, max(-100, min(ex - 1, 100)));
    }
    s_scale = S;
    slab_scale[slab] = c * key_scale[slab] / S;
  }
  __syncthreads();
  const float S = s_scale;
  unsigned char* hi = out + (int64_t)slab * 2 * ncols * d;
  unsigned char* lo = hi + (int64_t)ncols * d;
  for (int idx = threadIdx.x; idx < ncols * d; idx += blockDim.x) {
    const int j = idx / d, e = idx - j * d;
    uint32_t h = 0u, l = 0u;
    if (j < rows) {
      const float v = __bfloat162float(q[(((int64_t)slab * G + j % G) * m + j / G) * d + e]) * S;
      h = float_to_e4m3(v);
      l = float_to_e4m3(v - e4m3_to_float(h));
    }
    hi[idx] = (unsigned char)h;
    lo[idx] = (unsigned char)l;
  }
}

// ---------------------------------------------------------------------------------------------- host
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static std::once_flag once;
  static EncodeTiledFn fn = nullptr;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult res;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &res) == cudaSuccess &&
        res == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  });
  return fn;
}

struct FusedPlan {
  bool ok = false;
  int ncols = 0, k_stages = 0, t_stages = 0, tiles_per_cta_max = 0, n_cta = 0, n_tiles = 0;
  SmemLayout lay{};
};

constexpr int kSmemBudget = 227 * 1024 - 1024;   // dynamic shared memory we may ask for, minus alignment slack

FusedPlan make_plan(const ScoreProblem& p, int sm_count) {
  FusedPlan pl;
  const int g = p.group;
  const bool fp8 = p.k_scale != nullptr;
  // 8-bit key caches: contiguous only, and the TMA wants 16-byte aligned layer pointers and strides (the general path
  // reads them 8 bytes at a time and takes what this refuses)
  if (fp8) {
    if (p.block_tokens > 0 || p.stride_tok % 16 != 0 || p.stride_head % 16 != 0) return pl;
    for (int l = 0; l < p.n_layers; ++l)
      if (reinterpret_cast<uintptr_t>(p.k.p[l]) % 16 != 0) return pl;
  }
  if (!(g == 1 || g == 2 || g == 4 || g == 8)) return pl;
  if (p.n_layers > kFusedMaxLayers) return pl;
  const int rows = g * p.n_lookahead;
  if (rows > 64) return pl;
  if (p.n_tokens > (int64_t)1 << 30) return pl;
  pl.ncols = rows <= 16 ? 16 : rows <= 32 ? 32 : 64;
  pl.n_tiles = (int)ceil_div(p.n_tokens, kTileKeys);
  pl.n_cta = std::min(std::min(sm_count, kFusedMaxCtas), pl.n_tiles);
  pl.tiles_per_cta_max = (int)ceil_div(pl.n_tiles, pl.n_cta);
  // tensor memory: as many accumulator stages (4 at most, 2 at least) as leave room for the running maxima
  const int amax_cols = pl.tiles_per_cta_max * (pl.ncols / g);
  for (int ts = kTmemStages; ts >= 2 && pl.t_stages == 0; --ts)
    if (ts * 2 * pl.ncols + amax_cols <= kTmemColsAll) pl.t_stages = ts;
  if (pl.t_stages == 0) return pl;
  for (int ks = 10; ks >= 2; --ks) {
    const SmemLayout lay = smem_layout(p.head_dim, fp8, pl.ncols, g, ks, pl.tiles_per_cta_max);
    if ((int)lay.total <= kSmemBudget) {
      pl.k_stages = ks;
      pl.lay = lay;
      pl.ok = true;
      break;
    }
  }
  return pl;
}

// How many slabs the second visit runs behind the first.  The cross-CTA hand-over of a slab's row sums takes
// about 5 us; with short slabs (few tiles per CTA) two slabs of lead do not cover it, so the lag grows until the
// slabs kept live for the second read (lag + 1 of them) would no longer sit comfortably in L2: 64 MB of them, i.e.
// three slabs of lead at 16 MB a slab (measured at 128k tokens, d = 64: lag 2..4 within 1 %, 5 and 6 cost 6 and 11 %;
// at 64k tokens, d = 128: lag 3 best, 2 and 4 cost 9 and 3 %, 5 costs 22 %).
int fused_lag(const ScoreProblem& p, int n_slabs) {
  const double slab_bytes = (double)p.n_tokens * row_bytes(p.head_dim, p.k_scale != nullptr);
  int lag = (int)(64.0 * 1024 * 1024 / slab_bytes) - 1;
  lag = std::max(2, std::min(lag, 8));
  return std::max(1, std::min(lag, n_slabs));
}

struct FusedWorkspace {
  size_t limbs_off, counters_off, refs_off, clear_bytes;   // [0, clear_bytes) is cleared before every launch
  size_t qsplit_off, slab_scale_off, total;               // 8-bit keys: the split queries and the per-slab factors
};

FusedWorkspace fused_workspace(const ScoreProblem& p) {
  const size_t n_slabs = (size_t)p.n_layers * p.n_kv_heads;
  FusedWorkspace w;
  w.limbs_off = 0;
  w.counters_off = align_up(n_slabs * 64 * kLimbStride * sizeof(unsigned long long), 256);
  w.refs_off = align_up(w.counters_off + n_slabs * sizeof(unsigned), 256);
  w.clear_bytes = align_up(w.refs_off + n_slabs * sizeof(unsigned), 256);
  w.qsplit_off = w.slab_scale_off = w.total = w.clear_bytes;
  if (p.k_scale != nullptr) {
    w.slab_scale_off = align_up(w.qsplit_off + n_slabs * 2 * 64 * (size_t)p.head_dim, 256);
    w.total = align_up(w.slab_scale_off + n_slabs * sizeof(float), 256);
  }
  return w;
}

// The kernel's cross-CTA hand-over needs every CTA of the grid on an SM at the same time.  The launch therefore asks the
// runtime for exactly that guarantee (a cooperative launch; no grid-wide barrier is used): a grid that cannot be
// co-resident -- fewer SMs available than the device reports, e.g. under MPS with a limited SM share -- is refused
// here instead of spinning into the bounded waits.  SMs that are merely busy with other kernels delay the launch;
// they do not break it.
template <int D, int NCOLS, int G, bool FP8>
int32_t launch_fused(const FusedMaps& maps, const FusedArgs& args, const FusedPlan& pl, cudaStream_t stream) {
  auto kern = score_fused_kernel<D, NCOLS, G, FP8>;
  const int smem_bytes = (int)pl.lay.total + 1024;
  SPF_CUDA_CHECK(cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes));
  int per_sm = 0;
  SPF_CUDA_CHECK(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, kern, kThreads, smem_bytes));
  if (per_sm < 1) return fail(SPF_ERR_UNSUPPORTED, "spf_score: the fused kernel does not fit an SM of this device");
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3((unsigned)pl.n_cta);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = (size_t)smem_bytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeCooperative;
  attr[0].val.cooperative = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  const cudaError_t err = cudaLaunchKernelEx(&cfg, kern, maps, args);
  if (err == cudaErrorCooperativeLaunchTooLarge) {
    (void)cudaGetLastError();
    return fail(SPF_ERR_UNSUPPORTED, "spf_score: the %d CTAs of the fused kernel cannot all be resident on this device; use the general path",
                pl.n_cta);
  }
  SPF_CUDA_CHECK(err);
  return SPF_OK;
}

template <int D, int NCOLS, bool FP8>
int32_t launch_fused_g(int g, const FusedMaps& maps, const FusedArgs& args, const FusedPlan& pl, cudaStream_t stream) {
  // a thread owns NCOLS / 2 query rows, which must hold whole GQA groups
  if constexpr (NCOLS >= 16) {
    switch (g) {
      case 1: return launch_fused<D, NCOLS, 1, FP8>(maps, args, pl, stream);
      case 2: return launch_fused<D, NCOLS, 2, FP8>(maps, args, pl, stream);
      case 4: return launch_fused<D, NCOLS, 4, FP8>(maps, args, pl, stream);
      default: return launch_fused<D, NCOLS, 8, FP8>(maps, args, pl, stream);
    }
  }
  return SPF_ERR_UNSUPPORTED;
}

template <int D, bool FP8>
int32_t launch_fused_n(int ncols, int g, const FusedMaps& maps, const FusedArgs& args, const FusedPlan& pl, cudaStream_t stream) {
  switch (ncols) {
    case 16: return launch_fused_g<D, 16, FP8>(g, maps, args, pl, stream);
    case 32: return launch_fused_g<D, 32, FP8>(g, maps, args, pl, stream);
    default: return launch_fused_g<D, 64, FP8>(g, maps, args, pl, stream);
  }
}

}  // namespace

// One CTA waits on an mbarrier that nothing ever arrives on, with the kernels' own bounded wait and a
// 20 ms limit: the wait must give up, record SPF_ERR_TIMEOUT and let the kernel return normally.
__global__ void bounded_wait_selftest_kernel(int32_t* dev_status) {
  __shared__ __align__(8) unsigned long long bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(smem_u32(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  const Abort ab{&abort_flag, dev_status, 20000000ull};
  mbar_wait_warp(smem_u32(&bar), 0u, ab);
  __syncthreads();
}

int32_t bounded_wait_selftest_launch(int32_t* dev_status, cudaStream_t stream) {
  bounded_wait_selftest_kernel<<<1, 64, 0, stream>>>(dev_status);
  SPF_CUDA_CHECK(cudaGetLastError());
  return SPF_OK;
}

bool score_fused_supported(const ScoreProblem& p, int sm_count) { return make_plan(p, sm_count).ok; }

size_t score_fused_workspace_bytes(const ScoreProblem& p) { return fused_workspace(p).total; }

int32_t score_fused_launch(const ScoreProblem& p, void* workspace, int sm_count, int32_t* dev_status, cudaStream_t stream, int mode,
                           const float* lse_in) {
  const FusedPlan pl = make_plan(p, sm_count);
  if (!pl.ok) return fail(SPF_ERR_UNSUPPORTED, "spf_score: shape not covered by the fused path");
  EncodeTiledFn encode = encode_fn();
  if (encode == nullptr) return fail(SPF_ERR_CUDA, "spf_score: cuTensorMapEncodeTiled is not available from the driver");
  const FusedWorkspace w = fused_workspace(p);
  char* base = static_cast<char*>(workspace);

  FusedMaps maps;
  const int d = p.head_dim, g = p.group, m = p.n_lookahead;
  const int n_slabs = p.n_layers * p.n_kv_heads;
  const bool fp8 = p.k_scale != nullptr;
  const int subrow = sub_row_bytes(row_bytes(d, fp8));
  const CUtensorMapSwizzle swizzle = subrow == 128 ? CU_TENSOR_MAP_SWIZZLE_128B : CU_TENSOR_MAP_SWIZZLE_64B;
  if (fp8) {
    // (d, row, slab * 2 + term) view of the split queries, which split_q_kernel writes below
    const cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)pl.ncols, (cuuint64_t)n_slabs * 2};
    const cuuint64_t strides[2] = {(cuuint64_t)d, (cuuint64_t)pl.ncols * d};
    const cuuint32_t box[3] = {(cuuint32_t)subrow, (cuuint32_t)pl.ncols, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    const CUresult r = encode(&maps.q, CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, base + w.qsplit_off, dims, strides, box, estr,
                              CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(SPF_ERR_CUDA, "spf_score_fp8: encoding the query tensor map failed (CUresult %d)", (int)r);
  } else {
    const cuuint64_t dims[4] = {(cuuint64_t)d, (cuuint64_t)g, (cuuint64_t)m, (cuuint64_t)n_slabs};
    const cuuint64_t strides[3] = {(cuuint64_t)m * d * 2, (cuuint64_t)d * 2, (cuuint64_t)g * m * d * 2};
    const cuuint32_t box[4] = {64, (cuuint32_t)g, (cuuint32_t)m, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    const CUresult r = encode(&maps.q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<__nv_bfloat16*>(p.q), dims, strides, box,
                              estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(SPF_ERR_CUDA, "spf_score: encoding the query tensor map failed (CUresult %d)", (int)r);
  }
  for (int l = 0; l < p.n_layers && p.block_tokens > 0; ++l) {
    // paged: (d, row in block, kv-head, pool block); a table entry outside the pool reads as zeros instead of faulting
    const cuuint64_t bt = (cuuint64_t)p.block_tokens;
    const cuuint64_t dims[4] = {(cuuint64_t)d, bt, (cuuint64_t)p.n_kv_heads, (cuuint64_t)p.n_pool_blocks};
    const cuuint64_t strides[3] = {(cuuint64_t)d * 2, bt * d * 2, (cuuint64_t)p.n_kv_heads * bt * d * 2};
    const cuuint32_t box[4] = {64, (cuuint32_t)kTileKeys, 1, 1};
    const cuuint32_t estr[4] = {1, 1, 1, 1};
    const CUresult r = encode(&maps.k[l], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<__nv_bfloat16*>(p.k.p[l]), dims, strides,
                              box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS)
      return fail(SPF_ERR_CUDA, "spf_score_paged: encoding the key tensor map of layer %d failed (CUresult %d)", l, (int)r);
  }
  for (int l = 0; l < p.n_layers && fp8; ++l) {
    // 8-bit keys: strides count bytes
    const cuuint64_t head_stride = p.n_kv_heads > 1 ? (cuuint64_t)p.stride_head : (cuuint64_t)p.stride_tok * p.n_tokens;
    const cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)p.n_tokens, (cuuint64_t)p.n_kv_heads};
    const cuuint64_t strides[2] = {(cuuint64_t)p.stride_tok, head_stride};
    const cuuint32_t box[3] = {(cuuint32_t)subrow, (cuuint32_t)kTileKeys, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    const CUresult r = encode(&maps.k[l], CU_TENSOR_MAP_DATA_TYPE_UINT8, 3, const_cast<__nv_bfloat16*>(p.k.p[l]), dims, strides, box, estr,
                              CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                              CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS)
      return fail(SPF_ERR_CUDA, "spf_score_fp8: encoding the key tensor map of layer %d failed (CUresult %d)", l, (int)r);
  }
  for (int l = 0; l < p.n_layers && p.block_tokens == 0 && !fp8; ++l) {
    const cuuint64_t head_stride = p.n_kv_heads > 1 ? (cuuint64_t)p.stride_head : (cuuint64_t)p.stride_tok * p.n_tokens;
    const cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)p.n_tokens, (cuuint64_t)p.n_kv_heads};
    const cuuint64_t strides[2] = {(cuuint64_t)p.stride_tok * 2, head_stride * 2};
    const cuuint32_t box[3] = {64, (cuuint32_t)kTileKeys, 1};
    const cuuint32_t estr[3] = {1, 1, 1};
    const CUresult r = encode(&maps.k[l], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<__nv_bfloat16*>(p.k.p[l]), dims, strides,
                              box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS)
      return fail(SPF_ERR_CUDA, "spf_score: encoding the key tensor map of layer %d failed (CUresult %d)", l, (int)r);
  }

  FusedArgs args{};
  for (int l = 0; l < p.n_layers; ++l) args.k_layers[l] = p.k.p[l];
  args.q = p.q;
  args.n_tokens = p.n_tokens;
  args.stride_head = p.stride_head;
  args.stride_tok = p.stride_tok;
  args.n_layers = p.n_layers;
  args.n_kv_heads = p.n_kv_heads;
  args.n_lookahead = m;
  args.n_tiles = pl.n_tiles;
  args.tiles_per_cta_max = pl.tiles_per_cta_max;
  args.lag = fused_lag(p, n_slabs);
  args.mode = mode;
  args.lse_in = lse_in;
  args.k_stages = pl.k_stages;
  args.t_stages = pl.t_stages;
  args.c = p.c_log2;
  args.inv_c = 1.0f / p.c_log2;
  args.limbs = reinterpret_cast<unsigned long long*>(base + w.limbs_off);
  args.counters = reinterpret_cast<unsigned*>(base + w.counters_off);
  args.refs = reinterpret_cast<unsigned*>(base + w.refs_off);
  args.slab_scale = fp8 ? reinterpret_cast<const float*>(base + w.slab_scale_off) : nullptr;
  args.key_scale = p.k_scale;
  args.lse_out = p.lse_out;
  args.extra_lse = p.extra_lse;
  args.importance = p.importance;
  args.dev_status = dev_status;
  args.block_table = p.block_table;
  args.block_tokens = p.block_tokens;
  args.stride_block = (int64_t)p.n_kv_heads * p.block_tokens * p.head_dim;
  args.n_pool_blocks = p.n_pool_blocks;

  SPF_CUDA_CHECK(cudaMemsetAsync(base, 0, w.clear_bytes, stream));
  if (fp8) {
    split_q_kernel<<<n_slabs, 256, 0, stream>>>(p.q, g, m, d, pl.ncols, p.k_scale, p.c_log2,
                                                reinterpret_cast<unsigned char*>(base + w.qsplit_off),
                                                reinterpret_cast<float*>(base + w.slab_scale_off));
    SPF_CUDA_CHECK(cudaGetLastError());
    if (d == 64) return launch_fused_n<64, true>(pl.ncols, g, maps, args, pl, stream);
    return launch_fused_n<128, true>(pl.ncols, g, maps, args, pl, stream);
  }
  if (d == 64) return launch_fused_n<64, false>(pl.ncols, g, maps, args, pl, stream);
  return launch_fused_n<128, false>(pl.ncols, g, maps, args, pl, stream);
}

}  // namespace spf
