// Internal launch interface between api.cu and the kernel files.
#pragma once
#include <cuda_runtime.h>
#include <cstdint>

#include "ws_layout.cuh"

namespace dscale {

struct AllocArgs {
  void* ws;
  int n_bs;
  const int32_t* n_live;
  const float* scores;
  int scores_are_logits;
  const int32_t* draft_tokens;
  const int32_t* ctx_len;
  const int32_t* block_table;
  int max_pages;
  int num_pages;
  int n_kv_heads;
  int num_ctas;
  const int32_t* budget_rows;   // nullable device int32[1]: M_live; null = (W / 2) N (Eq. 3)
  int block_width;              // W: slots per request that exist (even, 2..16)
};
cudaError_t launch_alloc(const AllocArgs& a, cudaStream_t stream);

struct AcceptArgs {
  void* ws;
  int n_bs;
  const float* logits;
  int64_t ld;
  int vocab;
  int32_t* accept_len;
  int32_t* next_anchor;
  int32_t* out_tokens;
  int32_t* out_len;
  int32_t* ctx_len_inout;
  int n_kv_heads;
  int num_ctas;
};
cudaError_t launch_accept(const AcceptArgs& a, cudaStream_t stream);

struct AttnArgs {
  void* ws;
  int n_bs;
  const void* q;
  const void* k_cache;
  const void* v_cache;
  const int32_t* block_table;
  int max_pages;
  int num_pages;
  int n_q_heads;
  int n_kv_heads;
  float sm_scale;
  void* out;
  int num_ctas;
};
cudaError_t launch_attn_simt(const AttnArgs& a, cudaStream_t stream);
// returns cudaErrorNotSupported if the driver entry point for tensor maps is missing
cudaError_t launch_attn_tc(const AttnArgs& a, cudaStream_t stream);

struct SampleArgs {
  void* ws;
  int n_bs;
  const float* logits;
  int64_t ld;
  int vocab;
  float temperature;
  const float* u_accept;   // [8 n_bs] one uniform per packed row
  const float* u_draw;     // [n_bs]   one uniform per request
  int32_t* accept_len;
  int32_t* next_anchor;
  int32_t* out_tokens;
  int32_t* out_len;
  float* p_draft;          // nullable [8 n_bs]: P(candidate) per row
  int n_kv_heads;
  int num_ctas;
};
cudaError_t launch_accept_sampling(const SampleArgs& a, cudaStream_t stream);

// fused LM head + argmax + greedy acceptance (tensor cores)
cudaError_t launch_lm_head(void* ws, int n_bs, const void* hidden, const void* weight, int hidden_dim,
                           int vocab, int32_t* accept_len, int32_t* next_anchor, int32_t* out_tokens,
                           int32_t* out_len, int32_t* ctx_len_inout, float* row_max, int n_kv_heads,
                           int num_ctas, cudaStream_t stream);

// acceptance-predictor front end: drafter logits / hidden states -> predLogits
struct PredictArgs {
  void* ws;
  int n_bs;
  const int32_t* n_live;
  const float* draft_logits;   // [n_bs][15][ld]
  int64_t ld;
  int vocab;
  const void* draft_hidden;    // bf16 [n_bs][15][hidden_dim]
  int hidden_dim;
  const void* p_hidden;        // bf16 [64][hidden_dim]
  const void* p_logit;         // bf16 [32][vocab]
  const float* w1;             // [64][1735]
  const float* b1;             // [64]
  const float* w2;             // [15][64]
  const float* b2;             // [15]
  float* pred_logits;          // [n_bs][15]
  float* features_out;         // nullable [n_bs][1735]
  int n_kv_heads;
  int num_ctas;
};
cudaError_t launch_predictor(const PredictArgs& p, cudaStream_t stream);
cudaError_t predictor_prepare();

// comparison baseline: unpacked W = 16, one 128-row tile per (request, q-head)
cudaError_t launch_attn_padded(void* ws, int n_bs, const void* q_unpacked, const void* k_cache,
                               const void* v_cache, const int32_t* block_table, int max_pages,
                               int num_pages, const int32_t* ctx_len, int n_q_heads,
                               int n_kv_heads, float sm_scale, void* out_unpacked, int num_ctas,
                               cudaStream_t stream);

}  // namespace dscale
