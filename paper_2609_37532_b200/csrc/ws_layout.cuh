// Fixed-address workspace layout (the paper's buffer_bs, Eq. 12).
//
// The caller allocates one block of device memory per captured capacity n_bs;
// every stage reads and writes its sections at offsets that depend only on
// (n_bs, n_kv_heads, num_ctas), so addresses and shapes never change between
// graph replays.  The int32 index sections come first and depend on n_bs
// alone, which is what dscale_ws_field relies on.
#pragma once
#include <cstddef>
#include <cstdint>

namespace dscale {

constexpr int kW = 16;            // verification slots per request (anchor + 15 candidates)
constexpr int kHalfW = 8;         // budget per live request (Eq. 3)
constexpr int kPage = 16;         // tokens per KV page
constexpr int kD = 128;           // head_dim
constexpr int kMaxNbs = 64;
constexpr int kTileTok = 128;     // keys per attention tile (8 pages)
constexpr int kAccMaxChunks = 16; // vocab chunks per row in the argmax
constexpr int kTcRows = 64;       // rows of the tensor-core query tile (GQA group 4 x 16 slots)
// Cost model of the attention schedule (slices are cut to equal cost, not to equal tile counts),
// fitted to per-CTA timestamps on the Qwen3-8B-shaped step: a key tile of a request with more than
// 8 window rows takes about 6 % longer (the second group of softmax warps works too), a new
// (request, kv-head) pair costs about 0.8 tile, and the last CTAs of a launch start 2-3 tiles late.
constexpr int kTileCostSmall = 64, kTileCostBig = 68, kRunCost = 50;
constexpr int kLateCtas = 8;
__device__ constexpr int kLateTiles[kLateCtas] = {2, 2, 2, 2, 2, 2, 2, 3};
// acceptance-predictor front end ("Acceptance predictor" paragraph)
constexpr int kPredPos = 15;          // new draft positions per request
constexpr int kPredConf = 18;         // confidence values per position
constexpr int kPredHid = 64;          // hidden-state projection width
constexpr int kPredLog = 32;          // logit projection width
constexpr int kPredCtx = 25;          // batch-context values
constexpr int kPredFeatures = kPredPos * (kPredConf + kPredHid + kPredLog) + kPredCtx;   // 1735
constexpr int kPredMlp = 64;          // hidden units of the predictor
constexpr int kPredMaxChunks = 32;    // vocabulary chunks per drafter-logit row
constexpr int kPredRec = 52;          // 16 top values, (max, sum, sum e z, sum z), 32 projections

// header words (int32)
enum HdrWord {
  H_STATUS = 0, H_N_LIVE = 1, H_M_LIVE = 2, H_TOTAL_TILES = 3, H_ACCEPT_TICKET = 4,
  H_MAGIC = 5, H_SAMPLE_TICKET = 6, H_LM_TICKET = 7, H_WORDS = 64
};

struct WsLayout {
  size_t hdr, k, k0, offset, q_start, q_end, tokens, positions, kv_refs, row_req, top1,
      kv_len, tile_prefix, qscores, amax_val, amax_idx, smp_m, smp_s, row_m, row_z, row_flag, req_row, req_rej, pair_cnt, pad_cnt, lm_val, lm_idx,
      part_o, part_ml, pred_part, pred_rowsum, pred_feat, slice_tab, total;
};

__host__ __device__ inline size_t ws_align(size_t x) { return (x + 255) & ~size_t(255); }

__host__ __device__ inline WsLayout ws_layout(int n_bs, int n_kv_heads, int num_ctas) {
  WsLayout L;
  size_t o = 0;
  const size_t m_bs = size_t(kHalfW) * n_bs;
  L.hdr = o;         o = ws_align(o + H_WORDS * 4);
  L.k = o;           o = ws_align(o + n_bs * 4);
  L.k0 = o;          o = ws_align(o + n_bs * 4);
  L.offset = o;      o = ws_align(o + (n_bs + 1) * 4);
  L.q_start = o;     o = ws_align(o + n_bs * 4);
  L.q_end = o;       o = ws_align(o + n_bs * 4);
  L.tokens = o;      o = ws_align(o + m_bs * 4);
  L.positions = o;   o = ws_align(o + m_bs * 4);
  L.kv_refs = o;     o = ws_align(o + m_bs * 4);
  L.row_req = o;     o = ws_align(o + m_bs * 4);
  L.top1 = o;        o = ws_align(o + m_bs * 4);
  L.kv_len = o;      o = ws_align(o + n_bs * 4);
  L.tile_prefix = o; o = ws_align(o + (n_bs + 1) * 4);
  L.qscores = o;     o = ws_align(o + size_t(n_bs) * kW * 4);
  L.amax_val = o;    o = ws_align(o + m_bs * kAccMaxChunks * 4);
  L.amax_idx = o;    o = ws_align(o + m_bs * kAccMaxChunks * 4);
  // sampling verifier: per (row, chunk) running (max, sum), per-row totals and
  // acceptance flags, per-request row that supplies the successor
  L.smp_m = o;       o = ws_align(o + m_bs * kAccMaxChunks * 4);
  L.smp_s = o;       o = ws_align(o + m_bs * kAccMaxChunks * 4);
  L.row_m = o;       o = ws_align(o + m_bs * 4);
  L.row_z = o;       o = ws_align(o + m_bs * 4);
  L.row_flag = o;    o = ws_align(o + m_bs * 4);
  L.req_row = o;     o = ws_align(o + n_bs * 4);
  L.req_rej = o;     o = ws_align(o + n_bs * 4);
  L.pair_cnt = o;    o = ws_align(o + size_t(n_bs) * n_kv_heads * 4);
  // arrival counters of the padded comparison kernel: one per (request, q-head), group <= 8
  L.pad_cnt = o;     o = ws_align(o + size_t(n_bs) * n_kv_heads * 8 * 4);
  // fused LM head: one (max logit, index) partial per (packed row, CTA)
  L.lm_val = o;      o = ws_align(o + m_bs * size_t(num_ctas) * 4);
  L.lm_idx = o;      o = ws_align(o + m_bs * size_t(num_ctas) * 4);
  // split-KV partials of the attention kernel: per CTA two slots (the segment
  // that starts its range and the one that ends it), each kTcRows rows of
  // (128 fp32 accumulators) plus (row max, row sum)
  L.part_o = o;      o = ws_align(o + size_t(num_ctas) * 2 * kTcRows * kD * 4);
  L.part_ml = o;     o = ws_align(o + size_t(num_ctas) * 2 * kTcRows * 2 * 4);
  // predictor front end: per (drafter-logit row, vocabulary chunk) a record of kPredRec
  // floats, per chunk the row sums of the fixed logit projection, per request the features
  L.pred_part = o;   o = ws_align(o + size_t(kPredPos) * n_bs * kPredMaxChunks * kPredRec * 4);
  {
    // partial row sums of the logit projection matrix: one vector of 32 per CTA of the stream grid
    const int row_groups = (kPredPos * n_bs + 31) / 32;
    const int slots = num_ctas > row_groups ? num_ctas : row_groups;
    L.pred_rowsum = o; o = ws_align(o + size_t(slots > kPredMaxChunks ? slots : kPredMaxChunks) * 32 * 4);
  }
  L.pred_feat = o;   o = ws_align(o + size_t(n_bs) * kPredFeatures * 4);
  // attention schedule: first linear key tile of every CTA's slice, [num_ctas + 1]
  L.slice_tab = o;   o = ws_align(o + (size_t(num_ctas) + 1) * 4);
  L.total = o;
  return L;
}

template <typename T>
__host__ __device__ inline T* ws_ptr(void* ws, size_t off) {
  return reinterpret_cast<T*>(reinterpret_cast<char*>(ws) + off);
}
template <typename T>
__host__ __device__ inline const T* ws_ptr(const void* ws, size_t off) {
  return reinterpret_cast<const T*>(reinterpret_cast<const char*>(ws) + off);
}

}  // namespace dscale
