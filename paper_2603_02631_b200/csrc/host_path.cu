// spf_compress_host: the four calls of the path chained for a prompt whose inputs and results are host buffers.
#include <algorithm>

#include "common.cuh"
#include "score.cuh"

namespace spf {
namespace {

struct Arena {
  size_t k, q, ids, cs, ce, importance, lse, scores, kept, out_ids, out_pos, tok, ch, counts, status, workspace, total;
};

size_t take(size_t* pos, size_t bytes) {
  const size_t at = *pos;
  *pos = align_up(at + bytes, 256);
  return at;
}

// Lays the arena out; returns false (with the reason recorded) when the arguments make no sense.
bool layout(const spf_shape* shape, int64_t n, const spf_select_params* prm, Arena* a, size_t* ws_bytes) {
  if (shape == nullptr || prm == nullptr || n < 1 || prm->chunk < 1) {
    fail(SPF_ERR_INVALID_ARG, "spf_compress_host: null argument, n_tokens < 1 or chunk < 1");
    return false;
  }
  if (shape->n_layers < 1 || shape->n_layers > kMaxLayers || shape->n_q_heads < 1 || shape->n_kv_heads < 1 || shape->head_dim < 1 ||
      shape->n_lookahead < 1) {
    fail(SPF_ERR_INVALID_ARG, "spf_compress_host: shape fields out of range");
    return false;
  }
  const size_t L = shape->n_layers, Hq = shape->n_q_heads, Hkv = shape->n_kv_heads, d = shape->head_dim, m = shape->n_lookahead;
  const int64_t n_chunks = ceil_div(n, prm->chunk);
  const int64_t k = spf_keep_count(n_chunks, prm->keep_ratio);
  const size_t kept_tokens = (size_t)std::min<int64_t>(k * prm->chunk, n);
  // the workspace need depends on the shape only through a prompt description: ask with placeholders for the pointers
  // (any 16-byte aligned non-null value passes the checks; nothing is dereferenced by the size query)
  const void* fake_layers[kMaxLayers];
  for (size_t l = 0; l < L; ++l) fake_layers[l] = reinterpret_cast<const void*>(uintptr_t{4096});
  spf_prompt pr{};
  pr.n_tokens = n;
  pr.k_layers = fake_layers;
  pr.k_stride_head = n * (int64_t)d;
  pr.k_stride_tok = (int64_t)d;
  pr.q = reinterpret_cast<const void*>(uintptr_t{4096});
  pr.importance = reinterpret_cast<float*>(uintptr_t{4096});
  *ws_bytes = spf_score_workspace_bytes(shape, &pr, 1);
  if (*ws_bytes == 0) return false;            // the reason is already recorded
  size_t pos = 0;
  a->k = take(&pos, L * Hkv * (size_t)n * d * 2);
  a->q = take(&pos, L * Hq * m * d * 2);
  a->ids = take(&pos, (size_t)n * 4);
  a->cs = take(&pos, (size_t)n * 4);
  a->ce = take(&pos, (size_t)n * 4);
  a->importance = take(&pos, (size_t)n * 4);
  a->lse = take(&pos, L * Hq * m * 4);
  a->scores = take(&pos, (size_t)n_chunks * 4);
  a->kept = take(&pos, (size_t)k * 4);
  a->out_ids = take(&pos, kept_tokens * 4);
  a->out_pos = take(&pos, kept_tokens * 4);
  a->tok = take(&pos, (size_t)k * 8);
  a->ch = take(&pos, (size_t)k * 8);
  a->counts = take(&pos, 16);
  a->status = take(&pos, 4);
  a->workspace = take(&pos, *ws_bytes);
  a->total = pos;
  return true;
}

}  // namespace
}  // namespace spf

using namespace spf;

extern "C" size_t spf_compress_host_arena_bytes(const spf_shape* shape, int64_t n_tokens, const spf_select_params* params) {
  clear_error();
  Arena a;
  size_t ws = 0;
  return layout(shape, n_tokens, params, &a, &ws) ? a.total : 0;
}

extern "C" int32_t spf_compress_host(const spf_shape* shape, int64_t n_tokens, const void* const* k_layers_host, const void* q_host,
                                     const int32_t* token_ids_host, const int32_t* char_start_host, const int32_t* char_end_host,
                                     const spf_select_params* params, void* arena, size_t arena_bytes, int32_t* out_ids_host,
                                     int32_t* out_pos_host, int32_t* out_tok_spans_host, int32_t* out_char_spans_host,
                                     int64_t* out_counts_host, void* cuda_stream) {
  clear_error();
  Arena a;
  size_t ws_bytes = 0;
  if (!layout(shape, n_tokens, params, &a, &ws_bytes)) return SPF_ERR_INVALID_ARG;
  if (k_layers_host == nullptr || q_host == nullptr || token_ids_host == nullptr || char_start_host == nullptr ||
      char_end_host == nullptr || out_ids_host == nullptr || out_tok_spans_host == nullptr || out_char_spans_host == nullptr ||
      out_counts_host == nullptr)
    return fail(SPF_ERR_INVALID_ARG, "spf_compress_host: null pointer");
  for (int l = 0; l < shape->n_layers; ++l)
    if (k_layers_host[l] == nullptr) return fail(SPF_ERR_INVALID_ARG, "spf_compress_host: k_layers_host[%d] is null", l);
  if (arena == nullptr || reinterpret_cast<uintptr_t>(arena) % 256 != 0)
    return fail(SPF_ERR_WORKSPACE, "spf_compress_host: arena is null or not 256-byte aligned");
  if (arena_bytes < a.total) return fail(SPF_ERR_WORKSPACE, "spf_compress_host: arena has %zu bytes, %zu needed", arena_bytes, a.total);

  cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
  char* base = static_cast<char*>(arena);
  const size_t L = shape->n_layers, Hq = shape->n_q_heads, Hkv = shape->n_kv_heads, d = shape->head_dim, m = shape->n_lookahead;
  const size_t layer_bytes = Hkv * (size_t)n_tokens * d * 2;
  const int64_t n_chunks = ceil_div(n_tokens, params->chunk);
  const int64_t k = spf_keep_count(n_chunks, params->keep_ratio);

  // inputs to the device (one copy per tensor, in order on the stream)
  const void* dev_layers[kMaxLayers];
  for (size_t l = 0; l < L; ++l) {
    SPF_CUDA_CHECK(cudaMemcpyAsync(base + a.k + l * layer_bytes, k_layers_host[l], layer_bytes, cudaMemcpyHostToDevice, stream));
    dev_layers[l] = base + a.k + l * layer_bytes;
  }
  SPF_CUDA_CHECK(cudaMemcpyAsync(base + a.q, q_host, L * Hq * m * d * 2, cudaMemcpyHostToDevice, stream));
  SPF_CUDA_CHECK(cudaMemcpyAsync(base + a.ids, token_ids_host, (size_t)n_tokens * 4, cudaMemcpyHostToDevice, stream));
  SPF_CUDA_CHECK(cudaMemcpyAsync(base + a.cs, char_start_host, (size_t)n_tokens * 4, cudaMemcpyHostToDevice, stream));
  SPF_CUDA_CHECK(cudaMemcpyAsync(base + a.ce, char_end_host, (size_t)n_tokens * 4, cudaMemcpyHostToDevice, stream));

  spf_prompt pr{};
  pr.n_tokens = n_tokens;
  pr.k_layers = dev_layers;
  pr.k_stride_head = n_tokens * (int64_t)d;
  pr.k_stride_tok = (int64_t)d;
  pr.q = base + a.q;
  pr.importance = reinterpret_cast<float*>(base + a.importance);
  pr.lse = reinterpret_cast<float*>(base + a.lse);
  int32_t* dev_status = reinterpret_cast<int32_t*>(base + a.status);
  int64_t counts[2] = {0, 0};
  int32_t device_status = 0;
  for (int attempt = 0; attempt < 2; ++attempt) {
    // attempt 0: the kernels spf_score would pick; attempt 1 (after a device-side range or timeout report): the general ones
    SPF_CUDA_CHECK(cudaMemsetAsync(dev_status, 0, 4, stream));
    int32_t st = attempt == 0 ? spf_score(shape, &pr, 1, base + a.workspace, ws_bytes, dev_status, stream)
                              : score_on_path(shape, &pr, 1, base + a.workspace, ws_bytes, dev_status, stream, 1);
    if (st != SPF_OK) return st;
    st = spf_chunk_pool(pr.importance, n_tokens, params->pool_kernel, params->chunk, reinterpret_cast<float*>(base + a.scores), stream);
    if (st != SPF_OK) return st;
    st = spf_select_topk(reinterpret_cast<const float*>(base + a.scores), n_chunks, k, reinterpret_cast<int32_t*>(base + a.kept), stream);
    if (st != SPF_OK) return st;
    st = spf_compact_spans(reinterpret_cast<const int32_t*>(base + a.kept), k, params->chunk, n_tokens,
                           reinterpret_cast<const int32_t*>(base + a.ids), reinterpret_cast<const int32_t*>(base + a.cs),
                           reinterpret_cast<const int32_t*>(base + a.ce), reinterpret_cast<int32_t*>(base + a.out_ids),
                           reinterpret_cast<int32_t*>(base + a.out_pos), reinterpret_cast<int32_t*>(base + a.tok),
                           reinterpret_cast<int32_t*>(base + a.ch), reinterpret_cast<int64_t*>(base + a.counts), stream);
    if (st != SPF_OK) return st;
    SPF_CUDA_CHECK(cudaMemcpyAsync(counts, base + a.counts, 16, cudaMemcpyDeviceToHost, stream));
    SPF_CUDA_CHECK(cudaMemcpyAsync(&device_status, dev_status, 4, cudaMemcpyDeviceToHost, stream));
    SPF_CUDA_CHECK(cudaStreamSynchronize(stream));
    if (device_status != SPF_ERR_RANGE && device_status != SPF_ERR_TIMEOUT) break;
  }
  if (device_status != 0) return fail(device_status, "spf_compress_host: device status %d (%s)", device_status, spf_status_string(device_status));
  const size_t n_kept = (size_t)counts[0], n_spans = (size_t)counts[1];
  SPF_CUDA_CHECK(cudaMemcpyAsync(out_ids_host, base + a.out_ids, n_kept * 4, cudaMemcpyDeviceToHost, stream));
  if (out_pos_host != nullptr)
    SPF_CUDA_CHECK(cudaMemcpyAsync(out_pos_host, base + a.out_pos, n_kept * 4, cudaMemcpyDeviceToHost, stream));
  SPF_CUDA_CHECK(cudaMemcpyAsync(out_tok_spans_host, base + a.tok, n_spans * 8, cudaMemcpyDeviceToHost, stream));
  SPF_CUDA_CHECK(cudaMemcpyAsync(out_char_spans_host, base + a.ch, n_spans * 8, cudaMemcpyDeviceToHost, stream));
  SPF_CUDA_CHECK(cudaStreamSynchronize(stream));
  out_counts_host[0] = counts[0];
  out_counts_host[1] = counts[1];
  return SPF_OK;
}
