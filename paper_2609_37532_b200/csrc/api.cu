// C ABI of the library: argument validation, the host-side workspace registry
// and dispatch to the kernel launchers.  No computation happens here.
#include <cuda_runtime.h>

#include <cstring>
#include <map>
#include <mutex>
#include <vector>

#include "../../include/dscale.h"
#include "kernels.cuh"

namespace dscale {
cudaError_t attn_simt_prepare();
cudaError_t attn_tc_prepare();
cudaError_t attn_padded_prepare();
cudaError_t lm_head_prepare();
void attn_tc_forget_maps();
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
  if (attn_padded_prepare() != cudaSuccess) return DSCALE_ERR_CUDA;
  if (lm_head_prepare() != cudaSuccess) return DSCALE_ERR_CUDA;
  if (predictor_prepare() != cudaSuccess) return DSCALE_ERR_CUDA;
  std::lock_guard<std::mutex> lk(g_mu);
  g_ws[ws] = WsInfo{bytes, n_bs, n_q_heads, n_kv_heads, num_sms};
  return DSCALE_OK;
}

namespace {
struct StepGraph {   // one instantiated graph of the host-driven step per workspace, keyed by every argument
  std::vector<uintptr_t> key;
  cudaGraphExec_t exec = nullptr;
};
std::map<const void*, StepGraph> g_step;
}  // namespace

int dscale_workspace_destroy(void* ws) {
  if (!ws) return DSCALE_ERR_INVALID_ARG;
  cudaGraphExec_t exec = nullptr;
  {
    std::lock_guard<std::mutex> lk(g_mu);
    auto it = g_ws.find(ws);
    if (it == g_ws.end()) return DSCALE_ERR_WORKSPACE;
    g_ws.erase(it);
    auto sg = g_step.find(ws);
    if (sg != g_step.end()) { exec = sg->second.exec; g_step.erase(sg); }
  }
  if (exec) cudaGraphExecDestroy(exec);
  // tensor-map descriptors are keyed on the q / K / V addresses, which the caller
  // is about to free or reuse along with the workspace: drop them all (they are
  // re-encoded on the next call that needs one)
  attn_tc_forget_maps();
  return DSCALE_OK;
}

static int alloc_common(void* ws, int n_bs, const int32_t* n_live, const float* scores,
                        int scores_are_logits, const int32_t* draft_tokens, const int32_t* ctx_len,
                        const int32_t* block_table, int max_pages, int num_pages,
                        const int32_t* budget_rows, int block_width, void* stream) {
  if (block_width < 2 || block_width > DSCALE_W || (block_width & 1)) return DSCALE_ERR_UNSUPPORTED;
  if (!ws || !n_live || !scores || !draft_tokens || !ctx_len || !block_table)
    return DSCALE_ERR_INVALID_ARG;
  if (max_pages < 1 || num_pages < 1) return DSCALE_ERR_INVALID_ARG;
  if (!aligned(n_live, 4) || !aligned(scores, 4) || !aligned(draft_tokens, 4) ||
      !aligned(ctx_len, 4) || !aligned(block_table, 4) || !aligned(budget_rows, 4))
    return DSCALE_ERR_INVALID_ARG;
  WsInfo info;
  if (!lookup(ws, n_bs, &info)) return DSCALE_ERR_WORKSPACE;
  AllocArgs a{ws, n_bs, n_live, scores, scores_are_logits ? 1 : 0, draft_tokens, ctx_len,
              block_table, max_pages, num_pages, info.n_kv_heads, info.num_ctas, budget_rows, block_width};
  return launch_alloc(a, (cudaStream_t)stream) == cudaSuccess ? DSCALE_OK : DSCALE_ERR_CUDA;
}

int dscale_alloc_verify(void* ws, int n_bs, const int32_t* n_live, const float* scores,
                        int scores_are_logits, const int32_t* draft_tokens,
                        const int32_t* ctx_len, const int32_t* block_table, int max_pages,
                        int num_pages, void* stream) {
  return alloc_common(ws, n_bs, n_live, scores, scores_are_logits, draft_tokens, ctx_len, block_table,
                      max_pages, num_pages, nullptr, DSCALE_W, stream);
}

int dscale_alloc_verify_ex(void* ws, int n_bs, const int32_t* n_live, const float* scores,
                           int scores_are_logits, const int32_t* draft_tokens,
                           const int32_t* ctx_len, const int32_t* block_table, int max_pages,
                           int num_pages, int block_width, const int32_t* budget_rows, void* stream) {
  return alloc_common(ws, n_bs, n_live, scores, scores_are_logits, draft_tokens, ctx_len, block_table,
                      max_pages, num_pages, budget_rows, block_width, stream);
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

int dscale_verify_attn_padded(void* ws, int n_bs, const void* q_unpacked, const void* k_cache,
                              const void* v_cache, const int32_t* block_table, int max_pages,
                              int num_pages, const int32_t* ctx_len, int n_q_heads,
                              int n_kv_heads, float sm_scale, void* out_unpacked, void* stream) {
  if (!ctx_len) return DSCALE_ERR_INVALID_ARG;
  AttnArgs a;
  int rc = attn_common(ws, n_bs, q_unpacked, k_cache, v_cache, block_table, max_pages, num_pages,
                       n_q_heads, n_kv_heads, sm_scale, out_unpacked, &a);
  if (rc != DSCALE_OK) return rc;
  cudaError_t e = launch_attn_padded(ws, n_bs, q_unpacked, k_cache, v_cache, block_table, max_pages,
                                     num_pages, ctx_len, n_q_heads, n_kv_heads, sm_scale,
                                     out_unpacked, a.num_ctas, (cudaStream_t)stream);
  if (e == cudaErrorNotSupported) return DSCALE_ERR_UNSUPPORTED;
  return e == cudaSuccess ? DSCALE_OK : DSCALE_ERR_CUDA;
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

namespace {
struct StagingLayout {
  size_t n_live, scores, draft, ctx_len, block_table, accept_len, next_anchor, out_tokens,
      out_len, total;
};
StagingLayout staging_layout(int n_bs, int max_pages) {
  StagingLayout S;
  size_t o = 0;
  S.n_live = o;      o = ws_align(o + 4);
  S.scores = o;      o = ws_align(o + size_t(n_bs) * 15 * 4);
  S.draft = o;       o = ws_align(o + size_t(n_bs) * 16 * 4);
  S.ctx_len = o;     o = ws_align(o + size_t(n_bs) * 4);
  S.block_table = o; o = ws_align(o + size_t(n_bs) * max_pages * 4);
  S.accept_len = o;  o = ws_align(o + size_t(n_bs) * 4);
  S.next_anchor = o; o = ws_align(o + size_t(n_bs) * 4);
  S.out_tokens = o;  o = ws_align(o + size_t(n_bs) * 16 * 4);
  S.out_len = o;     o = ws_align(o + size_t(n_bs) * 4);
  S.total = o;
  return S;
}

// Stage-in / stage-out for the host-buffer step.  Page-locked host memory is mapped into the
// device's address space, so one small kernel can fetch all five staged inputs of a step over
// the bus at once (65 KB at n_bs = 32), and another can write the four results back, instead
// of nine copy operations that run one after another with a fixed cost each (about 10 us per
// copy on this class of machine).  Memory that is not mapped (pageable buffers) takes the
// copy path.
constexpr int kStageRegions = 5;
struct StageCopy {
  const uint32_t* src[kStageRegions];
  uint32_t* dst[kStageRegions];
  int words[kStageRegions];
  int n;
};
__global__ void stage_copy_kernel(StageCopy c) {
  const int t = blockIdx.x * blockDim.x + threadIdx.x, nt = gridDim.x * blockDim.x;
  for (int r = 0; r < c.n; ++r)
    for (int i = t; i < c.words[r]; i += nt) c.dst[r][i] = c.src[r][i];
}
// the device's view of a page-locked host buffer, or nullptr if the device cannot address it
const void* mapped(const void* host) {
  cudaPointerAttributes at;
  if (cudaPointerGetAttributes(&at, host) != cudaSuccess) { cudaGetLastError(); return nullptr; }
  if (at.type != cudaMemoryTypeHost) return nullptr;
  return at.devicePointer;
}
bool launch_stage_copy(const StageCopy& c, cudaStream_t st) {
  int total = 0;
  for (int r = 0; r < c.n; ++r) total += c.words[r];
  const int blocks = total / (256 * 8) < 1 ? 1 : (total / (256 * 8) > 32 ? 32 : total / (256 * 8));
  stage_copy_kernel<<<blocks, 256, 0, st>>>(c);
  return cudaGetLastError() == cudaSuccess;
}
}  // namespace

size_t dscale_step_staging_bytes(int n_bs, int max_pages) {
  if (n_bs < 1 || n_bs > DSCALE_MAX_NBS || max_pages < 1) return 0;
  return staging_layout(n_bs, max_pages).total;
}

int dscale_verify_step_host(void* ws, int n_bs, const int32_t* h_n_live, const float* h_scores,
                            const int32_t* h_draft_tokens, const int32_t* h_ctx_len,
                            const int32_t* h_block_table, int max_pages, int num_pages,
                            void* staging, const dscale_layer* layers, int n_layers,
                            int n_q_heads, int n_kv_heads, float sm_scale, const float* logits,
                            int64_t ld, int vocab, int32_t* h_accept_len, int32_t* h_next_anchor,
                            int32_t* h_out_tokens, int32_t* h_out_len, void* stream) {
  if (!h_n_live || !h_scores || !h_draft_tokens || !h_ctx_len || !h_block_table || !staging ||
      !layers || !h_accept_len || !h_next_anchor || !h_out_tokens || !h_out_len)
    return DSCALE_ERR_INVALID_ARG;
  if (n_bs < 1 || n_bs > DSCALE_MAX_NBS || max_pages < 1 || n_layers < 0 || !aligned(staging, 256))
    return DSCALE_ERR_INVALID_ARG;
  const StagingLayout S = staging_layout(n_bs, max_pages);
  char* d = static_cast<char*>(staging);
  cudaStream_t st = (cudaStream_t)stream;
  auto h2d = [&](size_t off, const void* src, size_t bytes) {
    return cudaMemcpyAsync(d + off, src, bytes, cudaMemcpyHostToDevice, st) == cudaSuccess;
  };
  auto d2h = [&](void* dst, size_t off, size_t bytes) {
    return cudaMemcpyAsync(dst, d + off, bytes, cudaMemcpyDeviceToHost, st) == cudaSuccess;
  };
  {
    const void* hp[kStageRegions] = {h_n_live, h_scores, h_draft_tokens, h_ctx_len, h_block_table};
    const size_t off[kStageRegions] = {S.n_live, S.scores, S.draft, S.ctx_len, S.block_table};
    const int words[kStageRegions] = {1, n_bs * 15, n_bs * 16, n_bs, n_bs * max_pages};
    StageCopy c;
    c.n = kStageRegions;
    bool all_mapped = true;
    for (int r = 0; r < kStageRegions; ++r) {
      c.src[r] = static_cast<const uint32_t*>(mapped(hp[r]));
      c.dst[r] = reinterpret_cast<uint32_t*>(d + off[r]);
      c.words[r] = words[r];
      all_mapped = all_mapped && c.src[r] != nullptr;
    }
    if (all_mapped) {
      if (!launch_stage_copy(c, st)) return DSCALE_ERR_CUDA;
    } else {
      for (int r = 0; r < kStageRegions; ++r)
        if (!h2d(off[r], hp[r], size_t(words[r]) * 4)) return DSCALE_ERR_CUDA;
    }
  }
  const int32_t* d_bt = reinterpret_cast<const int32_t*>(d + S.block_table);
  int rc = dscale_alloc_verify(ws, n_bs, reinterpret_cast<const int32_t*>(d + S.n_live),
                               reinterpret_cast<const float*>(d + S.scores), 0,
                               reinterpret_cast<const int32_t*>(d + S.draft),
                               reinterpret_cast<const int32_t*>(d + S.ctx_len), d_bt, max_pages,
                               num_pages, stream);
  if (rc != DSCALE_OK) return rc;
  for (int l = 0; l < n_layers; ++l) {
    rc = dscale_verify_attn(ws, n_bs, layers[l].q, layers[l].k_cache, layers[l].v_cache, d_bt,
                            max_pages, num_pages, n_q_heads, n_kv_heads, sm_scale, layers[l].out,
                            stream);
    if (rc != DSCALE_OK) return rc;
  }
  rc = dscale_accept(ws, n_bs, logits, ld, vocab, reinterpret_cast<int32_t*>(d + S.accept_len),
                     reinterpret_cast<int32_t*>(d + S.next_anchor),
                     reinterpret_cast<int32_t*>(d + S.out_tokens),
                     reinterpret_cast<int32_t*>(d + S.out_len), nullptr, stream);
  if (rc != DSCALE_OK) return rc;
  {
    void* hp[4] = {h_accept_len, h_next_anchor, h_out_tokens, h_out_len};
    const size_t off[4] = {S.accept_len, S.next_anchor, S.out_tokens, S.out_len};
    const int words[4] = {n_bs, n_bs, n_bs * 16, n_bs};
    StageCopy c;
    c.n = 4;
    bool all_mapped = true;
    for (int r = 0; r < 4; ++r) {
      c.dst[r] = static_cast<uint32_t*>(const_cast<void*>(mapped(hp[r])));
      c.src[r] = reinterpret_cast<const uint32_t*>(d + off[r]);
      c.words[r] = words[r];
      all_mapped = all_mapped && c.dst[r] != nullptr;
    }
    if (all_mapped) {
      if (!launch_stage_copy(c, st)) return DSCALE_ERR_CUDA;
    } else {
      for (int r = 0; r < 4; ++r)
        if (!d2h(hp[r], off[r], size_t(words[r]) * 4)) return DSCALE_ERR_CUDA;
    }
  }
  return DSCALE_OK;
}

int dscale_verify_step_host_graph(void* ws, int n_bs, const int32_t* h_n_live, const float* h_scores,
                                  const int32_t* h_draft_tokens, const int32_t* h_ctx_len,
                                  const int32_t* h_block_table, int max_pages, int num_pages,
                                  void* staging, const dscale_layer* layers, int n_layers,
                                  int n_q_heads, int n_kv_heads, float sm_scale, const float* logits,
                                  int64_t ld, int vocab, int32_t* h_accept_len, int32_t* h_next_anchor,
                                  int32_t* h_out_tokens, int32_t* h_out_len, void* stream) {
  auto plain = [&]() {
    return dscale_verify_step_host(ws, n_bs, h_n_live, h_scores, h_draft_tokens, h_ctx_len, h_block_table,
                                   max_pages, num_pages, staging, layers, n_layers, n_q_heads, n_kv_heads,
                                   sm_scale, logits, ld, vocab, h_accept_len, h_next_anchor, h_out_tokens,
                                   h_out_len, stream);
  };
  if (!ws || !layers || n_layers < 0) return DSCALE_ERR_INVALID_ARG;
  cudaStream_t st = (cudaStream_t)stream;
  cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(st, &cs) != cudaSuccess) return DSCALE_ERR_CUDA;
  if (cs != cudaStreamCaptureStatusNone) return plain();        // the caller is capturing: just record
  if (st == nullptr || st == cudaStreamLegacy) return plain();  // the legacy default stream cannot capture

  auto up = [](const void* p) { return reinterpret_cast<uintptr_t>(p); };
  uint32_t scale_bits;
  memcpy(&scale_bits, &sm_scale, 4);
  std::vector<uintptr_t> key = {up(ws), (uintptr_t)n_bs, up(h_n_live), up(h_scores), up(h_draft_tokens),
                                up(h_ctx_len), up(h_block_table), (uintptr_t)max_pages, (uintptr_t)num_pages,
                                up(staging), (uintptr_t)n_layers, (uintptr_t)n_q_heads, (uintptr_t)n_kv_heads,
                                (uintptr_t)scale_bits, up(logits), (uintptr_t)ld, (uintptr_t)vocab,
                                up(h_accept_len), up(h_next_anchor), up(h_out_tokens), up(h_out_len)};
  for (int l = 0; l < n_layers; ++l) {
    key.push_back(up(layers[l].q)); key.push_back(up(layers[l].k_cache));
    key.push_back(up(layers[l].v_cache)); key.push_back(up(layers[l].out));
  }
  cudaGraphExec_t exec = nullptr;
  {
    std::lock_guard<std::mutex> lk(g_mu);
    if (g_ws.find(ws) == g_ws.end()) return DSCALE_ERR_WORKSPACE;
    auto it = g_step.find(ws);
    if (it != g_step.end() && it->second.exec && it->second.key == key) exec = it->second.exec;
  }
  if (!exec) {
    // capture outside the registry lock: the stage calls inside plain() take it themselves
    if (cudaStreamBeginCapture(st, cudaStreamCaptureModeThreadLocal) != cudaSuccess) return DSCALE_ERR_CUDA;
    const int rc = plain();
    cudaGraph_t graph = nullptr;
    const cudaError_t e = cudaStreamEndCapture(st, &graph);
    if (rc != DSCALE_OK || e != cudaSuccess || !graph) {
      if (graph) cudaGraphDestroy(graph);
      cudaGetLastError();
      return rc != DSCALE_OK ? rc : DSCALE_ERR_CUDA;
    }
    const cudaError_t ei = cudaGraphInstantiate(&exec, graph, 0);
    cudaGraphDestroy(graph);
    if (ei != cudaSuccess || !exec) return DSCALE_ERR_CUDA;
    cudaGraphExec_t old = nullptr;
    {
      std::lock_guard<std::mutex> lk(g_mu);
      StepGraph& sg = g_step[ws];
      old = sg.exec;
      sg.exec = exec;
      sg.key = key;
    }
    if (old) cudaGraphExecDestroy(old);
  }
  return cudaGraphLaunch(exec, st) == cudaSuccess ? DSCALE_OK : DSCALE_ERR_CUDA;
}

int dscale_lm_head_accept(void* ws, int n_bs, const void* hidden, const void* weight, int hidden_dim,
                          int vocab, int32_t* accept_len, int32_t* next_anchor, int32_t* out_tokens,
                          int32_t* out_len, int32_t* ctx_len_inout, float* row_max, void* stream) {
  if (!ws || !hidden || !weight || !accept_len || !next_anchor || !out_tokens || !out_len)
    return DSCALE_ERR_INVALID_ARG;
  if (!aligned(hidden, 16) || !aligned(weight, 16)) return DSCALE_ERR_INVALID_ARG;
  if (hidden_dim < 64 || hidden_dim % 64 != 0 || vocab < 16) return DSCALE_ERR_UNSUPPORTED;
  WsInfo info;
  if (!lookup(ws, n_bs, &info)) return DSCALE_ERR_WORKSPACE;
  cudaError_t e = launch_lm_head(ws, n_bs, hidden, weight, hidden_dim, vocab, accept_len, next_anchor,
                                 out_tokens, out_len, ctx_len_inout, row_max, info.n_kv_heads,
                                 info.num_ctas, (cudaStream_t)stream);
  if (e == cudaErrorNotSupported) return DSCALE_ERR_UNSUPPORTED;
  return e == cudaSuccess ? DSCALE_OK : DSCALE_ERR_CUDA;
}

int dscale_predict_scores(void* ws, int n_bs, const int32_t* n_live, const float* draft_logits, int64_t ld,
                          int vocab, const void* draft_hidden, int hidden_dim, const void* p_hidden,
                          const void* p_logit, const float* w1, const float* b1, const float* w2,
                          const float* b2, float* pred_logits, float* features_out, void* stream) {
  if (!ws || !n_live || !draft_logits || !draft_hidden || !p_hidden || !p_logit || !w1 || !b1 || !w2 || !b2 ||
      !pred_logits)
    return DSCALE_ERR_INVALID_ARG;
  if (!aligned(draft_logits, 16) || !aligned(draft_hidden, 16) || !aligned(p_hidden, 16) || !aligned(p_logit, 16))
    return DSCALE_ERR_INVALID_ARG;
  if (vocab < 16 || ld < vocab || ld % 4 != 0 || hidden_dim < 8 || hidden_dim % 8 != 0)
    return DSCALE_ERR_UNSUPPORTED;
  WsInfo info;
  if (!lookup(ws, n_bs, &info)) return DSCALE_ERR_WORKSPACE;
  PredictArgs p{ws, n_bs, n_live, draft_logits, ld, vocab, draft_hidden, hidden_dim, p_hidden, p_logit,
                w1, b1, w2, b2, pred_logits, features_out, info.n_kv_heads, info.num_ctas};
  return launch_predictor(p, (cudaStream_t)stream) == cudaSuccess ? DSCALE_OK : DSCALE_ERR_CUDA;
}

int dscale_accept_sampling(void* ws, int n_bs, const float* logits, int64_t ld, int vocab,
                           float temperature, const float* u_accept, const float* u_draw,
                           int32_t* accept_len, int32_t* next_anchor, int32_t* out_tokens,
                           int32_t* out_len, float* p_draft, void* stream) {
  if (!ws || !logits || !u_accept || !u_draw || !accept_len || !next_anchor || !out_tokens || !out_len)
    return DSCALE_ERR_INVALID_ARG;
  if (vocab < 1 || ld < vocab || (ld % 4) != 0 || !aligned(logits, 16) || !(temperature > 0.0f))
    return DSCALE_ERR_INVALID_ARG;
  if (vocab > DSCALE_SAMPLING_MAX_VOCAB) return DSCALE_ERR_TOO_LARGE;   // the draw kernel's group table
  WsInfo info;
  if (!lookup(ws, n_bs, &info)) return DSCALE_ERR_WORKSPACE;
  SampleArgs a{ws, n_bs, logits, ld, vocab, temperature, u_accept, u_draw, accept_len, next_anchor,
               out_tokens, out_len, p_draft, info.n_kv_heads, info.num_ctas};
  return launch_accept_sampling(a, (cudaStream_t)stream) == cudaSuccess ? DSCALE_OK : DSCALE_ERR_CUDA;
}

int dscale_select_bucket(const int32_t* buckets, int n_buckets, int n_live) {
  if (!buckets || n_buckets < 1 || n_live < 1) return DSCALE_ERR_INVALID_ARG;
  int best = 0;
  for (int b = 0; b < n_buckets; ++b) {
    if (buckets[b] < 1) return DSCALE_ERR_INVALID_ARG;
    if (buckets[b] >= n_live && (best == 0 || buckets[b] < best)) best = buckets[b];
  }
  return best ? best : DSCALE_ERR_TOO_LARGE;
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
    case 1: return 1;   // attn_tc_kernel (cut pairs are merged inside it)
    case 2: return 1;   // accept_kernel
    case 3: return 1;   // attn_simt_kernel
    case 4: return 1;   // attn_padded_kernel
    case 5: return 2;   // sample_stats_kernel + sample_draw_kernel
    case 6: return 1;   // lm_head_kernel
    case 7: return 2;   // pred_stream_kernel, pred_tail_kernel
    default: return 0;
  }
}

}  // extern "C"
