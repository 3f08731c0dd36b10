// Internal description of one prompt's scoring problem and the entry points of the scoring paths.
#pragma once

#include "common.cuh"

namespace spf {

struct ScoreProblem {
  int n_layers, n_q_heads, n_kv_heads, group, head_dim, n_lookahead;
  int m_pad;     // n_lookahead rounded up to a multiple of 8
  int rows_pad;  // group * m_pad rounded up to a multiple of 16: query rows per kv-head tile
  float c_log2;  // softmax scale times log2(e): logits are handled in base-2 units
  int64_t n_tokens, stride_head, stride_tok;
  LayerPtrs k;
  const __nv_bfloat16* q;
  float* importance;
  float* lse_out;  // may be null
  // 8-bit key cache (k_scale != null): the layer pointers hold E4M3 bytes, strides count bytes, key (l, hk, s, j) has the
  // value k_scale[l * Hkv + hk] * E4M3(byte); only the general path reads this format
  const float* k_scale;
  const float* extra_lse;  // may be null: fp32 [L][Hq][m], natural log of what the row's denominator holds besides the prompt keys
  // paged key cache (block_tokens > 0): k.p[l] is layer l's block pool, bf16 [n_pool_blocks][Hkv][block_tokens][d];
  // logical block b of the prompt sits in pool block block_table[b] (device memory)
  const int32_t* block_table;
  int32_t block_tokens;
  int64_t n_pool_blocks;
};

constexpr int kMmaMaxSplit = 64;  // upper bound on the key splits of sweep 1 (sizes the partials buffer)

// General two-sweep path (warp-level mma.sync tiles, key cache read twice).
size_t score_mma_workspace_bytes(const ScoreProblem& p);
int32_t score_mma_launch(const ScoreProblem& p, void* workspace, int sm_count, cudaStream_t stream);
// phase 1: row log-sum-exps of the given keys only (to p.lse_out); phase 2: importance of the given keys from row
// log-sum-exps supplied by the caller (device, natural log, [L][Hq][m]); phase 0 is score_mma_launch
int32_t score_mma_launch_phase(const ScoreProblem& p, void* workspace, int sm_count, int phase, const float* lse_in,
                               cudaStream_t stream);

// Fused single-kernel path (tcgen05 + TMA, key cache read once from HBM).  Covers G in {1,2,4,8},
// G*m <= 64, up to kFusedMaxLayers layers and prompt lengths whose per-CTA state fits shared memory.
constexpr int kFusedMaxLayers = 64;
constexpr int kFusedMaxCtas = 256;  // upper bound on the persistent grid
bool score_fused_supported(const ScoreProblem& p, int sm_count);
size_t score_fused_workspace_bytes(const ScoreProblem& p);
// mode 0: the whole computation; 1: first visit only: row log-sum-exps over the given keys to p.lse_out (p.importance unused);
// 2: second visit only, with the rows' log-sum-exps `lse_in` (device, natural log, [L][Hq][m]) supplied by the caller
int32_t score_fused_launch(const ScoreProblem& p, void* workspace, int sm_count, int32_t* dev_status, cudaStream_t stream, int mode = 0,
                           const float* lse_in = nullptr);

// spf_score with the kernel path given for this call only (0 automatic, 1 general, 2 fused) instead of the process-wide setting.
int32_t score_on_path(const spf_shape* shape, const spf_prompt* prompts, int32_t n_prompts, void* workspace, size_t workspace_bytes,
                      int32_t* dev_status, void* cuda_stream, int path);

// Launches the one-CTA self-test of the kernels' bounded wait (see spf_selftest_bounded_wait).
int32_t bounded_wait_selftest_launch(int32_t* dev_status, cudaStream_t stream);

}  // namespace spf
