// C ABI of the library: argument validation, the host-side workspace registry
// and dispatch to the kernel launchers.  No computation happens here.
#include <cuda_runtime.h>

#include <map>
#include <mutex>

#include "../../include/dscale.h"
#include "kernels.cuh"

namespace dscale {
cudaError_t attn_simt_prepare();
cudaError_t attn_tc_prepare();
}

namespace {

using namespace dscale;

struct WsInfo {
  size_t bytes;
  int n_bs, n_q_heads, n_kv_heads, num_ctas;
};
std::mutex g_mu;
std::map<const void*, WsInfo> g_ws;

bool lookup(const void* ws, int n_bs, WsInfo* out) {
  std::lock_guard<std::mutex> lk(g_mu);
  auto it = g_ws.find(ws);
  if (it == g_ws.end() || it->second.n_bs != n_bs) return false;
  *out = it->second;
  return true;
}

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

bool shape_ok(int n_bs, int n_q_heads, int n_kv_heads, int head_dim, int num_sms) {
  if (n_bs < 1 || n_bs > DSCALE_MAX_NBS) return false;
  if (head_dim != DSCALE_HEAD_DIM) return false;
  if (n_kv_heads < 1 || n_q_heads < n_kv_heads || n_q_heads % n_kv_heads) return false;
  const int G = n_q_heads / n_kv_heads;
  if (G > 8) return false;
  if (num_sms < 1 || num_sms > 4096) return false;
  return true;
}

}  // namespace

extern "C" {

size_t dscale_workspace_bytes(int n_bs, int n_q_heads, int n_kv_heads, int head_dim, int num_sms) {
  if (!shape_ok(n_bs, n_q_heads, n_kv_heads, head_dim, num_sms)) return 0;
  return ws_layout(n_bs, n_kv_heads, num_sms).total;
}

int dscale_workspace_init(void* ws, size_t bytes, int n_bs, int n_q_heads, int n_kv_heads,
                          int head_dim, int num_sms, void* stream) {
  if (!ws || !aligned(ws, 256)) return DSCALE_ERR_INVALID_ARG;
  if (!shape_ok(n_bs, n_q_heads, n_kv_heads, head_dim, num_sms)) return DSCALE_ERR_UNSUPPORTED;
  const WsLayout L = ws_layout(n_bs, n_kv_heads, num_sms);
  if (bytes < L.total) return DSCALE_ERR_WORKSPACE;
  // everything up to the split-KV partials starts at zero (status, tickets,
  // index sections, per-pair arrival counters); the partials need no init
  if (cudaMemsetAsync(ws, 0, L.part_o, (cudaStream_t)stream) != cudaSuccess) return DSCALE_ERR_CUDA;
  if (attn_simt_prepare() != cudaSuccess) return DSCALE_ERR_CUDA;
  if (attn_tc_prepare() != cudaSuccess) return DSCALE_ERR_CUDA;
  std::lock_guard<std::mutex> lk(g_mu);
  g_ws[ws] = WsInfo{bytes, n_bs, n_q_heads, n_kv_heads, num_sms};
  return DSCALE_OK;
}

int dscale_alloc_verify(void* ws, int n_bs, const int32_t* n_live, const float* scores,
                        int scores_are_logits, const int32_t* draft_tokens,
                        const int32_t* ctx_len, const int32_t* block_table, int max_pages,
                        int num_pages, void* stream) {
  if (!ws || !n_live || !scores || !draft_tokens || !ctx_len || !block_table)
    return DSCALE_ERR_INVALID_ARG;
  if (max_pages < 1 || num_pages < 1) return DSCALE_ERR_INVALID_ARG;
  if (!aligned(n_live, 4) || !aligned(scores, 4) || !aligned(draft_tokens, 4) ||
      !aligned(ctx_len, 4) || !aligned(block_table, 4))
    return DSCALE_ERR_INVALID_ARG;
  WsInfo info;
  if (!lookup(ws, n_bs, &info)) return DSCALE_ERR_WORKSPACE;
  AllocArgs a{ws, n_bs, n_live, scores, scores_are_logits ? 1 : 0, draft_tokens, ctx_len,
              block_table, max_pages, num_pages, info.n_kv_heads, info.num_ctas};
  return launch_alloc(a, (cudaStream_t)stream) == cudaSuccess ? DSCALE_OK : DSCALE_ERR_CUDA;
}

static int attn_common(void* ws, int n_bs, const void* q, const void* k_cache, const void* v_cache,
                       const int32_t* block_table, int max_pages, int num_pages, int n_q_heads,
                       int n_kv_heads, float sm_scale, void* out, AttnArgs* a) {
  if (!ws || !q || !k_cache || !v_cache || !block_table || !out) return DSCALE_ERR_INVALID_ARG;
  if (max_pages < 1 || num_pages < 1) return DSCALE_ERR_INVALID_ARG;
  if (!aligned(q, 16) || !aligned(out, 16) || !aligned(k_cache, 16) || !aligned(v_cache, 16) ||
      !aligned(block_table, 4))
    return DSCALE_ERR_INVALID_ARG;
  if (!(sm_scale > 0.0f)) return DSCALE_ERR_INVALID_ARG;
  WsInfo info;
  if (!lookup(ws, n_bs, &info)) return DSCALE_ERR_WORKSPACE;
  if (info.n_q_heads != n_q_heads || info.n_kv_heads != n_kv_heads) return DSCALE_ERR_WORKSPACE;
  *a = AttnArgs{ws, n_bs, q, k_cache, v_cache, block_table, max_pages, num_pages,
                n_q_heads, n_kv_heads, sm_scale, out, info.num_ctas};
  return DSCALE_OK;
}

int dscale_verify_attn(void* ws, int n_bs, const void* q, const void* k_cache,
                       const void* v_cache, const int32_t* block_table, int max_pages,
                       int num_pages, int n_q_heads, int n_kv_heads, float sm_scale, void* out,
                       void* stream) {
  AttnArgs a;
  int rc = attn_common(ws, n_bs, q, k_cache, v_cache, block_table, max_pages, num_pages,
                       n_q_heads, n_kv_heads, sm_scale, out, &a);
  if (rc != DSCALE_OK) return rc;
  if (n_q_heads / n_kv_heads != 4) return DSCALE_ERR_UNSUPPORTED;
  cudaError_t e = launch_attn_tc(a, (cudaStream_t)stream);
  if (e == cudaErrorNotSupported) return DSCALE_ERR_UNSUPPORTED;
  return e == cudaSuccess ? DSCALE_OK : DSCALE_ERR_CUDA;
}

int dscale_verify_attn_simt(void* ws, int n_bs, const void* q, const void* k_cache,
                            const void* v_cache, const int32_t* block_table, int max_pages,
                            int num_pages, int n_q_heads, int n_kv_heads, float sm_scale,
                            void* out, void* stream) {
  AttnArgs a;
  int rc = attn_common(ws, n_bs, q, k_cache, v_cache, block_table, max_pages, num_pages,
                       n_q_heads, n_kv_heads, sm_scale, out, &a);
  if (rc != DSCALE_OK) return rc;
  return launch_attn_simt(a, (cudaStream_t)stream) == cudaSuccess ? DSCALE_OK : DSCALE_ERR_CUDA;
}

int dscale_accept(void* ws, int n_bs, const float* logits, int64_t ld, int vocab,
                  int32_t* accept_len, int32_t* next_anchor, int32_t* out_tokens,
                  int32_t* out_len, int32_t* ctx_len_inout, void* stream) {
  if (!ws || !logits || !accept_len || !next_anchor || !out_tokens || !out_len)
    return DSCALE_ERR_INVALID_ARG;
  if (vocab < 1 || ld < vocab || (ld % 4) != 0 || !aligned(logits, 16))
    return DSCALE_ERR_INVALID_ARG;
  WsInfo info;
  if (!lookup(ws, n_bs, &info)) return DSCALE_ERR_WORKSPACE;
  AcceptArgs a{ws, n_bs, logits, ld, vocab, accept_len, next_anchor, out_tokens, out_len,
               ctx_len_inout, info.n_kv_heads, info.num_ctas};
  return launch_accept(a, (cudaStream_t)stream) == cudaSuccess ? DSCALE_OK : DSCALE_ERR_CUDA;
}

const int32_t* dscale_ws_field(const void* ws, int n_bs, int field) {
  if (!ws || n_bs < 1 || n_bs > DSCALE_MAX_NBS) return nullptr;
  const WsLayout L = ws_layout(n_bs, 1, 1);      // index sections depend on n_bs only
  size_t off;
  switch (field) {
    case DSCALE_WS_STATUS: off = L.hdr + H_STATUS * 4; break;
    case DSCALE_WS_N_LIVE: off = L.hdr + H_N_LIVE * 4; break;
    case DSCALE_WS_K: off = L.k; break;
    case DSCALE_WS_K0: off = L.k0; break;
    case DSCALE_WS_OFFSET: off = L.offset; break;
    case DSCALE_WS_Q_START: off = L.q_start; break;
    case DSCALE_WS_Q_END: off = L.q_end; break;
    case DSCALE_WS_TOKENS: off = L.tokens; break;
    case DSCALE_WS_POSITIONS: off = L.positions; break;
    case DSCALE_WS_KV_REFS: off = L.kv_refs; break;
    case DSCALE_WS_ROW_REQ: off = L.row_req; break;
    case DSCALE_WS_TOP1: off = L.top1; break;
    default: return nullptr;
  }
  return ws_ptr<int32_t>(ws, off);
}

int dscale_launches_per_call(int which) {
  switch (which) {
    case 0: return 1;   // dvl_alloc_kernel
    case 1: return 1;   // attn_tc_kernel (split-KV merge happens inside it)
    case 2: return 1;   // accept_kernel
    case 3: return 1;   // attn_simt_kernel
    default: return 0;
  }
}

}  // extern "C"
