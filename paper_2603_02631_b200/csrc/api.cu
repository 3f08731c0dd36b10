// Host side of the C ABI: argument validation, error text, dispatch of spf_score.
#include <atomic>
#include <cmath>
#include <cstring>
#include <mutex>

#include "common.cuh"
#include "score.cuh"

namespace spf {
namespace {

thread_local char g_error[512] = "";
std::atomic<int> g_score_path{0};  // 0 automatic, 1 general two-sweep path, 2 fused path

// Builds the per-prompt problem description; returns a status and leaves the reason in the error text.
int32_t make_problem(const spf_shape* shape, const spf_prompt& pr, int32_t index, ScoreProblem* out, int k_align = 16) {
  ScoreProblem p{};
  p.n_layers = shape->n_layers;
  p.n_q_heads = shape->n_q_heads;
  p.n_kv_heads = shape->n_kv_heads;
  p.head_dim = shape->head_dim;
  p.n_lookahead = shape->n_lookahead;
  if (p.n_layers < 1 || p.n_q_heads < 1 || p.n_kv_heads < 1 || p.n_lookahead < 1)
    return fail(SPF_ERR_INVALID_ARG, "spf_score: shape fields must be positive");
  if (p.n_layers > kMaxLayers) return fail(SPF_ERR_UNSUPPORTED, "spf_score: n_layers %d > %d", p.n_layers, kMaxLayers);
  if (p.head_dim != 64 && p.head_dim != 128)
    return fail(SPF_ERR_UNSUPPORTED, "spf_score: head_dim must be 64 or 128 (got %d)", p.head_dim);
  if (p.n_q_heads % p.n_kv_heads != 0)
    return fail(SPF_ERR_UNSUPPORTED, "spf_score: n_q_heads %d is not a multiple of n_kv_heads %d", p.n_q_heads, p.n_kv_heads);
  p.group = p.n_q_heads / p.n_kv_heads;
  if (p.n_lookahead > 32) return fail(SPF_ERR_UNSUPPORTED, "spf_score: n_lookahead %d > 32", p.n_lookahead);
  p.m_pad = (p.n_lookahead + 7) / 8 * 8;
  if (p.group * p.m_pad > 64)
    return fail(SPF_ERR_UNSUPPORTED, "spf_score: group %d x lookahead %d (padded to %d) exceeds 64 query rows per kv head",
                p.group, p.n_lookahead, p.m_pad);
  p.rows_pad = (p.group * p.m_pad + 15) / 16 * 16;
  const float scale = shape->softmax_scale > 0.f ? shape->softmax_scale : 1.0f / std::sqrt((float)p.head_dim);
  if (!std::isfinite(scale)) return fail(SPF_ERR_INVALID_ARG, "spf_score: softmax_scale is not finite");
  p.c_log2 = scale * kLog2e;

  if (pr.n_tokens < 1) return fail(SPF_ERR_INVALID_ARG, "spf_score: prompt %d: n_tokens must be >= 1", index);
  if (pr.n_tokens > 0x7fffffffLL) return fail(SPF_ERR_UNSUPPORTED, "spf_score: prompt %d: n_tokens >= 2^31", index);
  if (pr.k_layers == nullptr || pr.q == nullptr || pr.importance == nullptr)
    return fail(SPF_ERR_INVALID_ARG, "spf_score: prompt %d: null pointer", index);
  if (pr.k_stride_tok < p.head_dim || pr.k_stride_tok % 8 != 0)
    return fail(SPF_ERR_INVALID_ARG, "spf_score: prompt %d: k_stride_tok %lld must be >= head_dim and a multiple of 8", index,
                (long long)pr.k_stride_tok);
  if (pr.k_stride_head % 8 != 0 || (p.n_kv_heads > 1 && pr.k_stride_head < 1))
    return fail(SPF_ERR_INVALID_ARG, "spf_score: prompt %d: k_stride_head %lld must be positive and a multiple of 8", index,
                (long long)pr.k_stride_head);
  if (reinterpret_cast<uintptr_t>(pr.q) % 4 != 0)
    return fail(SPF_ERR_INVALID_ARG, "spf_score: prompt %d: q is not 4-byte aligned", index);
  for (int l = 0; l < p.n_layers; ++l) {
    const void* kp = pr.k_layers[l];
    if (kp == nullptr) return fail(SPF_ERR_INVALID_ARG, "spf_score: prompt %d: k_layers[%d] is null", index, l);
    if (reinterpret_cast<uintptr_t>(kp) % k_align != 0)
      return fail(SPF_ERR_INVALID_ARG, "spf_score: prompt %d: k_layers[%d] is not %d-byte aligned", index, l, k_align);
    p.k.p[l] = static_cast<const __nv_bfloat16*>(kp);
  }
  p.n_tokens = pr.n_tokens;
  p.stride_head = pr.k_stride_head;
  p.stride_tok = pr.k_stride_tok;
  p.q = static_cast<const __nv_bfloat16*>(pr.q);
  p.importance = pr.importance;
  p.lse_out = pr.lse;
  p.extra_lse = nullptr;
  p.k_scale = nullptr;
  p.block_table = nullptr;
  p.block_tokens = 0;
  p.n_pool_blocks = 0;
  *out = p;
  return SPF_OK;
}

int32_t device_sm_count(int* out) {
  int dev = 0;
  SPF_CUDA_CHECK(cudaGetDevice(&dev));
  static std::mutex mu;
  static int cached[64];
  std::lock_guard<std::mutex> lock(mu);
  if (dev < 0 || dev >= 64) return fail(SPF_ERR_CUDA, "device ordinal %d out of range", dev);
  if (cached[dev] == 0) SPF_CUDA_CHECK(cudaDeviceGetAttribute(&cached[dev], cudaDevAttrMultiProcessorCount, dev));
  *out = cached[dev];
  return SPF_OK;
}

}  // namespace

int32_t fail(int32_t code, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_error, sizeof(g_error), fmt, ap);
  va_end(ap);
  return code;
}

void clear_error() { g_error[0] = '\0'; }

}  // namespace spf

using namespace spf;

extern "C" size_t spf_score_workspace_bytes(const spf_shape* shape, const spf_prompt* prompts, int32_t n_prompts) {
  clear_error();
  if (shape == nullptr || prompts == nullptr || n_prompts < 1) {
    fail(SPF_ERR_INVALID_ARG, "spf_score_workspace_bytes: null argument or n_prompts < 1");
    return 0;
  }
  size_t need = 0;
  for (int32_t i = 0; i < n_prompts; ++i) {
    ScoreProblem p;
    if (make_problem(shape, prompts[i], i, &p) != SPF_OK) return 0;
    need = std::max(need, std::max(score_mma_workspace_bytes(p), score_fused_workspace_bytes(p)));
  }
  return need;
}

static int32_t score_impl(const spf_shape* shape, const spf_prompt* prompts, int32_t n_prompts, const float* const* extra_lse,
                          void* workspace, size_t workspace_bytes, int32_t* dev_status, void* cuda_stream, int path_override = -1) {
  clear_error();
  if (shape == nullptr || prompts == nullptr || n_prompts < 1)
    return fail(SPF_ERR_INVALID_ARG, "spf_score: null argument or n_prompts < 1");
  // validate everything before the first launch
  size_t need = 0;
  for (int32_t i = 0; i < n_prompts; ++i) {
    ScoreProblem p;
    const int32_t st = make_problem(shape, prompts[i], i, &p);
    if (st != SPF_OK) return st;
    need = std::max(need, std::max(score_mma_workspace_bytes(p), score_fused_workspace_bytes(p)));
  }
  if (workspace == nullptr || reinterpret_cast<uintptr_t>(workspace) % 256 != 0)
    return fail(SPF_ERR_WORKSPACE, "spf_score: workspace is null or not 256-byte aligned");
  if (workspace_bytes < need)
    return fail(SPF_ERR_WORKSPACE, "spf_score: workspace has %zu bytes, %zu needed", workspace_bytes, need);
  int sm_count = 0;
  {
    const int32_t st = device_sm_count(&sm_count);
    if (st != SPF_OK) return st;
  }
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  for (int32_t i = 0; i < n_prompts; ++i) {
    ScoreProblem p;
    make_problem(shape, prompts[i], i, &p);
    if (extra_lse != nullptr) p.extra_lse = extra_lse[i];
    const int path = path_override >= 0 ? path_override : g_score_path.load(std::memory_order_relaxed);
    const bool fused = path == 2 || (path == 0 && score_fused_supported(p, sm_count));
    const int32_t st = fused ? score_fused_launch(p, workspace, sm_count, dev_status, stream)
                             : score_mma_launch(p, workspace, sm_count, stream);
    if (st != SPF_OK) return st;
  }
  return SPF_OK;
}

namespace spf {
int32_t score_on_path(const spf_shape* shape, const spf_prompt* prompts, int32_t n_prompts, void* workspace, size_t workspace_bytes,
                      int32_t* dev_status, void* cuda_stream, int path) {
  return score_impl(shape, prompts, n_prompts, nullptr, workspace, workspace_bytes, dev_status, cuda_stream, path);
}
}  // namespace spf

extern "C" int32_t spf_score(const spf_shape* shape, const spf_prompt* prompts, int32_t n_prompts, void* workspace,
                             size_t workspace_bytes, int32_t* dev_status, void* cuda_stream) {
  return score_impl(shape, prompts, n_prompts, nullptr, workspace, workspace_bytes, dev_status, cuda_stream);
}

extern "C" int32_t spf_score_extra(const spf_shape* shape, const spf_prompt* prompts, int32_t n_prompts,
                                   const float* const* extra_lse, void* workspace, size_t workspace_bytes, int32_t* dev_status,
                                   void* cuda_stream) {
  return score_impl(shape, prompts, n_prompts, extra_lse, workspace, workspace_bytes, dev_status, cuda_stream);
}

// Paged key cache: the prompt is described as a contiguous one over its pool (same checks), then re-pointed at the blocks.
static int32_t make_paged_problem(const spf_shape* shape, const spf_paged_prompt& pp, int32_t index, ScoreProblem* out) {
  if (pp.block_tokens < 128 || pp.block_tokens % 128 != 0)
    return fail(SPF_ERR_INVALID_ARG, "spf_score_paged: prompt %d: block_tokens must be a positive multiple of 128 (got %d)", index,
                pp.block_tokens);
  if (pp.n_pool_blocks < 1 || pp.block_table == nullptr)
    return fail(SPF_ERR_INVALID_ARG, "spf_score_paged: prompt %d: empty pool or null block table", index);
  if (shape == nullptr) return fail(SPF_ERR_INVALID_ARG, "spf_score_paged: null shape");
  spf_prompt flat{};
  flat.n_tokens = pp.n_tokens;
  flat.k_layers = pp.k_pools;
  flat.k_stride_tok = shape->head_dim;
  flat.k_stride_head = (int64_t)pp.block_tokens * shape->head_dim;
  flat.q = pp.q;
  flat.importance = pp.importance;
  flat.lse = pp.lse;
  const int32_t st = make_problem(shape, flat, index, out);
  if (st != SPF_OK) return st;
  if (ceil_div(pp.n_tokens, pp.block_tokens) > 0x7fffffffLL) return fail(SPF_ERR_UNSUPPORTED, "spf_score_paged: too many blocks");
  out->block_table = pp.block_table;
  out->block_tokens = pp.block_tokens;
  out->n_pool_blocks = pp.n_pool_blocks;
  return SPF_OK;
}

extern "C" size_t spf_score_paged_workspace_bytes(const spf_shape* shape, const spf_paged_prompt* prompts, int32_t n_prompts) {
  clear_error();
  if (shape == nullptr || prompts == nullptr || n_prompts < 1) {
    fail(SPF_ERR_INVALID_ARG, "spf_score_paged_workspace_bytes: null argument or n_prompts < 1");
    return 0;
  }
  size_t need = 0;
  for (int32_t i = 0; i < n_prompts; ++i) {
    ScoreProblem p;
    if (make_paged_problem(shape, prompts[i], i, &p) != SPF_OK) return 0;
    need = std::max(need, std::max(score_mma_workspace_bytes(p), score_fused_workspace_bytes(p)));
  }
  return need;
}

extern "C" int32_t spf_score_paged(const spf_shape* shape, const spf_paged_prompt* prompts, int32_t n_prompts, void* workspace,
                                   size_t workspace_bytes, int32_t* dev_status, void* cuda_stream) {
  clear_error();
  if (shape == nullptr || prompts == nullptr || n_prompts < 1)
    return fail(SPF_ERR_INVALID_ARG, "spf_score_paged: null argument or n_prompts < 1");
  int sm_count = 0;
  {
    const int32_t st = device_sm_count(&sm_count);
    if (st != SPF_OK) return st;
  }
  size_t need = 0;
  for (int32_t i = 0; i < n_prompts; ++i) {
    ScoreProblem p;
    const int32_t st = make_paged_problem(shape, prompts[i], i, &p);
    if (st != SPF_OK) return st;
    need = std::max(need, std::max(score_mma_workspace_bytes(p), score_fused_workspace_bytes(p)));
  }
  if (workspace == nullptr || reinterpret_cast<uintptr_t>(workspace) % 256 != 0)
    return fail(SPF_ERR_WORKSPACE, "spf_score_paged: workspace is null or not 256-byte aligned");
  if (workspace_bytes < need)
    return fail(SPF_ERR_WORKSPACE, "spf_score_paged: workspace has %zu bytes, %zu needed", workspace_bytes, need);
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  for (int32_t i = 0; i < n_prompts; ++i) {
    ScoreProblem p;
    make_paged_problem(shape, prompts[i], i, &p);
    const int path = g_score_path.load(std::memory_order_relaxed);
    const bool fused = path == 2 || (path == 0 && score_fused_supported(p, sm_count));
    const int32_t st = fused ? score_fused_launch(p, workspace, sm_count, dev_status, stream)
                             : score_mma_launch(p, workspace, sm_count, stream);
    if (st != SPF_OK) return st;
  }
  return SPF_OK;
}

// 8-bit key cache: described as a bf16 prompt over the same pointers (the checks are the same: strides count elements,
// i.e. bytes here, rows must start 8-byte aligned), then marked with its scales.
static int32_t make_fp8_problem(const spf_shape* shape, const spf_fp8_prompt& fp, int32_t index, ScoreProblem* out) {
  if (fp.k_scale == nullptr) return fail(SPF_ERR_INVALID_ARG, "spf_score_fp8: prompt %d: k_scale is null", index);
  spf_prompt flat{};
  flat.n_tokens = fp.n_tokens;
  flat.k_layers = fp.k_layers;
  flat.k_stride_head = fp.k_stride_head;
  flat.k_stride_tok = fp.k_stride_tok;
  flat.q = fp.q;
  flat.importance = fp.importance;
  flat.lse = fp.lse;
  const int32_t st = make_problem(shape, flat, index, out, 8);      // rows of 8-bit keys are read 8 bytes at a time
  if (st != SPF_OK) return st;
  out->k_scale = fp.k_scale;
  return SPF_OK;
}

extern "C" size_t spf_score_fp8_workspace_bytes(const spf_shape* shape, const spf_fp8_prompt* prompts, int32_t n_prompts) {
  clear_error();
  if (shape == nullptr || prompts == nullptr || n_prompts < 1) {
    fail(SPF_ERR_INVALID_ARG, "spf_score_fp8_workspace_bytes: null argument or n_prompts < 1");
    return 0;
  }
  size_t need = 0;
  for (int32_t i = 0; i < n_prompts; ++i) {
    ScoreProblem p;
    if (make_fp8_problem(shape, prompts[i], i, &p) != SPF_OK) return 0;
    need = std::max(need, std::max(score_mma_workspace_bytes(p), score_fused_workspace_bytes(p)));
  }
  return need;
}

extern "C" int32_t spf_score_fp8(const spf_shape* shape, const spf_fp8_prompt* prompts, int32_t n_prompts, void* workspace,
                                 size_t workspace_bytes, int32_t* dev_status, void* cuda_stream) {
  clear_error();
  if (shape == nullptr || prompts == nullptr || n_prompts < 1)
    return fail(SPF_ERR_INVALID_ARG, "spf_score_fp8: null argument or n_prompts < 1");
  size_t need = 0;
  for (int32_t i = 0; i < n_prompts; ++i) {
    ScoreProblem p;
    const int32_t st = make_fp8_problem(shape, prompts[i], i, &p);
    if (st != SPF_OK) return st;
    need = std::max(need, std::max(score_mma_workspace_bytes(p), score_fused_workspace_bytes(p)));
  }
  if (workspace == nullptr || reinterpret_cast<uintptr_t>(workspace) % 256 != 0)
    return fail(SPF_ERR_WORKSPACE, "spf_score_fp8: workspace is null or not 256-byte aligned");
  if (workspace_bytes < need) return fail(SPF_ERR_WORKSPACE, "spf_score_fp8: workspace has %zu bytes, %zu needed", workspace_bytes, need);
  int sm_count = 0;
  {
    const int32_t st = device_sm_count(&sm_count);
    if (st != SPF_OK) return st;
  }
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  for (int32_t i = 0; i < n_prompts; ++i) {
    ScoreProblem p;
    make_fp8_problem(shape, prompts[i], i, &p);
    const int path = g_score_path.load(std::memory_order_relaxed);
    const bool fused = path == 2 || (path == 0 && score_fused_supported(p, sm_count));
    const int32_t st = fused ? score_fused_launch(p, workspace, sm_count, dev_status, stream) : score_mma_launch(p, workspace, sm_count, stream);
    if (st != SPF_OK) return st;
  }
  return SPF_OK;
}

// Key-sharded scoring: the two sweeps of the general path as separate calls.
static int32_t score_shard(const spf_shape* shape, const spf_prompt* prompt, int phase, const float* lse_in, void* workspace,
                           size_t workspace_bytes, void* cuda_stream, const char* who, bool allow_fused = false,
                           int32_t* dev_status = nullptr) {
  clear_error();
  if (shape == nullptr || prompt == nullptr) return fail(SPF_ERR_INVALID_ARG, "%s: null argument", who);
  spf_prompt pr = *prompt;
  float dummy = 0.f;
  if (phase == 1) {
    if (pr.lse == nullptr) return fail(SPF_ERR_INVALID_ARG, "%s: prompt->lse receives the result and must not be null", who);
    pr.importance = &dummy;   // not written by this phase; only passes the null check below
  } else if (lse_in == nullptr) {
    return fail(SPF_ERR_INVALID_ARG, "%s: lse is null", who);
  }
  ScoreProblem p;
  const int32_t st = make_problem(shape, pr, 0, &p);
  if (st != SPF_OK) return st;
  if (phase == 1) p.importance = nullptr;
  if (phase == 2) p.lse_out = nullptr;
  const size_t need = std::max(score_mma_workspace_bytes(p), score_fused_workspace_bytes(p));
  if (workspace == nullptr || reinterpret_cast<uintptr_t>(workspace) % 256 != 0)
    return fail(SPF_ERR_WORKSPACE, "%s: workspace is null or not 256-byte aligned", who);
  if (workspace_bytes < need) return fail(SPF_ERR_WORKSPACE, "%s: workspace has %zu bytes, %zu needed", who, workspace_bytes, need);
  int sm_count = 0;
  const int32_t sc = device_sm_count(&sm_count);
  if (sc != SPF_OK) return sc;
  const int path = g_score_path.load(std::memory_order_relaxed);
  if (allow_fused && (path == 2 || (path == 0 && score_fused_supported(p, sm_count))))
    return score_fused_launch(p, workspace, sm_count, dev_status, static_cast<cudaStream_t>(cuda_stream), phase, lse_in);
  return score_mma_launch_phase(p, workspace, sm_count, phase, lse_in, static_cast<cudaStream_t>(cuda_stream));
}

extern "C" int32_t spf_score_shard_lse(const spf_shape* shape, const spf_prompt* prompt, void* workspace, size_t workspace_bytes,
                                       void* cuda_stream) {
  return score_shard(shape, prompt, 1, nullptr, workspace, workspace_bytes, cuda_stream, "spf_score_shard_lse");
}

extern "C" int32_t spf_score_shard_apply(const spf_shape* shape, const spf_prompt* prompt, const float* lse, void* workspace,
                                         size_t workspace_bytes, void* cuda_stream) {
  return score_shard(shape, prompt, 2, lse, workspace, workspace_bytes, cuda_stream, "spf_score_shard_apply");
}

extern "C" int32_t spf_score_shard_lse_ex(const spf_shape* shape, const spf_prompt* prompt, void* workspace, size_t workspace_bytes,
                                          int32_t* dev_status, void* cuda_stream) {
  return score_shard(shape, prompt, 1, nullptr, workspace, workspace_bytes, cuda_stream, "spf_score_shard_lse_ex", true, dev_status);
}

extern "C" int32_t spf_score_shard_apply_ex(const spf_shape* shape, const spf_prompt* prompt, const float* lse, void* workspace,
                                            size_t workspace_bytes, int32_t* dev_status, void* cuda_stream) {
  return score_shard(shape, prompt, 2, lse, workspace, workspace_bytes, cuda_stream, "spf_score_shard_apply_ex", true, dev_status);
}

extern "C" int32_t spf_selftest_bounded_wait(int32_t* dev_status, void* cuda_stream) {
  clear_error();
  if (dev_status == nullptr) return fail(SPF_ERR_INVALID_ARG, "spf_selftest_bounded_wait: dev_status is null");
  return bounded_wait_selftest_launch(dev_status, static_cast<cudaStream_t>(cuda_stream));
}

extern "C" int32_t spf_set_score_path(int32_t path) {
  if (path < 0 || path > 2) return g_score_path.load(std::memory_order_relaxed);
  return g_score_path.exchange(path, std::memory_order_relaxed);
}

// ------------------------------------------------------------------------------------------------
// spf_score_static: scoring for callers that cannot allocate.  The scratch is this file-scope device
// array.  In host code its name is only a handle for the runtime, not a device address, so the
// address is looked up once per device with cudaGetSymbolAddress and that pointer goes to the kernels.
// ------------------------------------------------------------------------------------------------
static __device__ __align__(256) unsigned char g_static_scratch[SPF_STATIC_SCRATCH_BYTES];

namespace {

// Device address of g_static_scratch on the current device (looked up on the first call per device).
int32_t static_scratch_ptr(void** out) {
  int dev = 0;
  SPF_CUDA_CHECK(cudaGetDevice(&dev));
  static std::mutex mu;
  static void* cached[64];
  std::lock_guard<std::mutex> lock(mu);
  if (dev < 0 || dev >= 64) return fail(SPF_ERR_CUDA, "device ordinal %d out of range", dev);
  if (cached[dev] == nullptr) {
    void* ptr = nullptr;
    SPF_CUDA_CHECK(cudaGetSymbolAddress(&ptr, g_static_scratch));
    if (ptr == nullptr) return fail(SPF_ERR_CUDA, "spf_score_static: the scratch array has no device address");
    cached[dev] = ptr;
  }
  *out = cached[dev];
  return SPF_OK;
}

}  // namespace

extern "C" int32_t spf_score_static(const spf_shape* shape, const spf_prompt* prompts, int32_t n_prompts,
                                    void* cuda_stream) {
  clear_error();
  if (shape == nullptr || prompts == nullptr || n_prompts < 1)
    return fail(SPF_ERR_INVALID_ARG, "spf_score_static: null argument or n_prompts < 1");
  for (int32_t i = 0; i < n_prompts; ++i) {
    ScoreProblem p;
    const int32_t st = make_problem(shape, prompts[i], i, &p);
    if (st != SPF_OK) return st;
    const size_t need = score_mma_workspace_bytes(p);
    if (need > (size_t)SPF_STATIC_SCRATCH_BYTES)
      return fail(SPF_ERR_WORKSPACE,
                  "spf_score_static: prompt %d needs %zu bytes of scratch, the built-in array holds %zu; use spf_score "
                  "with a caller-provided workspace",
                  i, need, (size_t)SPF_STATIC_SCRATCH_BYTES);
  }
  int sm_count = 0;
  {
    const int32_t st = device_sm_count(&sm_count);
    if (st != SPF_OK) return st;
  }
  void* scratch = nullptr;
  {
    const int32_t st = static_scratch_ptr(&scratch);
    if (st != SPF_OK) return st;
  }
  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  for (int32_t i = 0; i < n_prompts; ++i) {
    ScoreProblem p;
    make_problem(shape, prompts[i], i, &p);
    // every kernel of this path writes the scratch words it later reads, so stale contents are harmless
    const int32_t st = score_mma_launch(p, scratch, sm_count, stream);
    if (st != SPF_OK) return st;
  }
  return SPF_OK;
}

extern "C" int64_t spf_keep_count(int64_t n_chunks, double keep_ratio) {
  if (n_chunks < 1) return 0;
  if (!(keep_ratio > 0.0)) return 1;
  const double want = std::ceil(keep_ratio * (double)n_chunks - 1e-9);
  if (want >= (double)n_chunks) return n_chunks;
  return want < 1.0 ? 1 : (int64_t)want;
}

extern "C" const char* spf_status_string(int32_t status) {
  switch (status) {
    case SPF_OK: return "ok";
    case SPF_ERR_INVALID_ARG: return "invalid argument";
    case SPF_ERR_UNSUPPORTED: return "unsupported shape";
    case SPF_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
    case SPF_ERR_CUDA: return "CUDA runtime error";
    case SPF_ERR_TIMEOUT: return "bounded device-side wait ran out";
    case SPF_ERR_RANGE: return "a softmax row overflowed fp32 in the fused path";
    default: return "unknown status";
  }
}

extern "C" const char* spf_last_error(void) { return g_error; }

extern "C" const char* spf_version(void) { return "0.1.0"; }
