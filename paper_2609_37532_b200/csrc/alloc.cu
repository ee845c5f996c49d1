// DVL allocation and flat-pack (Algorithm 1 from the scores down) in one
// thread block, with no host round trip and no inter-block synchronisation.
//
// Thread t = (request i = t / 16, slot j = t % 16), 1024 threads cover the
// maximum capacity of 64 requests.
//
//  1. one thread per request: running minimum (Eq. 6), sequential fp32 sum and
//     round-half-up seed (Eq. 7).  The additions use __fadd_rn so the compiler
//     can neither contract nor reorder them: k0 must be bit-identical to a
//     left-to-right IEEE binary32 evaluation.
//  2. budget adjustment (Eq. 9).  The paper's loop makes |delta| dependent
//     arg-max / arg-min rounds.  Because every request's scores are
//     non-increasing in j, that loop is a merge of sorted lists, and its result
//     is a rank selection: growing by delta takes the first delta elements of
//     {(i,j): k0_i <= j <= 15} ordered by (q descending, i ascending, j
//     ascending); shrinking by |delta| removes the first |delta| elements of
//     {(i,j): 1 <= j <= k0_i - 1} ordered by (q ascending, i ascending, j
//     descending).  Each candidate counts how many candidates precede it (a
//     suffix / prefix count per other request) and is taken iff that rank is
//     below |delta|: all 960 candidates in parallel, same tie-break as the loop.
//  3. offsets by a warp-shuffle prefix scan (Eq. 10), flat-pack of tokens,
//     positions and KV references with one thread per (request, slot) (Eq. 11),
//     sentinels (last two lines of Algorithm 1), and the per-request key-tile
//     prefix that the attention kernel's scheduler reads.
#include "kernels.cuh"

namespace dscale {

namespace {

__device__ __forceinline__ int warp_incl_scan(int v, int lane) {
#pragma unroll
  for (int d = 1; d < 32; d <<= 1) {
    int u = __shfl_up_sync(0xffffffffu, v, d);
    if (lane >= d) v += u;
  }
  return v;
}

__global__ void __launch_bounds__(1024, 1) dvl_alloc_kernel(AllocArgs a, WsLayout L) {
  __shared__ float sQ[kMaxNbs][kW];
  __shared__ int sK0[kMaxNbs];
  __shared__ int sAdj[kMaxNbs];
  __shared__ int sK[kMaxNbs];
  __shared__ int sOff[kMaxNbs + 1];
  __shared__ int sCtx[kMaxNbs];
  __shared__ int sTilePre[kMaxNbs + 1];
  __shared__ int sStatus;
  __shared__ int sWarpTot[4];

  const int t = threadIdx.x;
  const int i = t >> 4, j = t & 15;
  const int n_bs = a.n_bs;
  const int Wd = a.block_width;                       // slots per request that exist (<= kW)
  int* hdr = ws_ptr<int>(a.ws, L.hdr);

  if (t == 0) sStatus = 0;
  if (t < kMaxNbs) { sAdj[t] = 0; sK0[t] = 0; sCtx[t] = 0; }
  __syncthreads();

  int N = *a.n_live;
  if (N < 1 || N > n_bs) {
    if (t == 0) atomicOr(&sStatus, 4 /*BAD_LEN*/);
    N = N < 1 ? 1 : n_bs;
  }

  // ---- 1. prefix scores and seed, one thread per live request -------------
  if (j == 0 && i < N) {
    int st = 0;
    float q = 1.0f, lhat = 0.0f;
    sQ[i][0] = 1.0f;
    for (int jj = Wd; jj < kW; ++jj) sQ[i][jj] = 0.0f;    // slots a narrower block does not have
    for (int jj = 1; jj < Wd; ++jj) {
      float s = a.scores[i * (kW - 1) + jj - 1];
      if (a.scores_are_logits) s = (float)(1.0 / (1.0 + exp(-(double)s)));
      if (!(s >= 0.0f)) { s = 0.0f; st |= 1; }      // NaN or negative
      if (s > 1.0f) { s = 1.0f; st |= 1; }
      q = s < q ? s : q;                            // Eq. 6
      sQ[i][jj] = q;
      lhat = __fadd_rn(lhat, q);                    // Eq. 7, left to right
    }
    int r = (int)floorf(__fadd_rn(lhat, 0.5f));
    sK0[i] = min(Wd, max(1, r));
    int c = a.ctx_len[i];
    const int c_max = a.max_pages * kPage - kW;
    if (c < 0 || c > c_max) { st |= 4; c = c < 0 ? 0 : c_max; }
    sCtx[i] = c;
    if (st) atomicOr(&sStatus, st);
  }
  __syncthreads();

  // ---- 2. budget adjustment as a rank selection ----------------------------
  int sum0 = 0;
  for (int r = 0; r < N; ++r) sum0 += sK0[r];
  // verification budget M_live: 8 N (Eq. 3) unless the caller gives one; any value in
  // [N, 16 N] that fits the packed capacity 8 N_bs is served, others are clamped and flagged
  int m_budget = (Wd / 2) * N;
  if (a.budget_rows) {
    const int want = *a.budget_rows;
    const int hi = min(Wd * N, kHalfW * n_bs);
    m_budget = want < N ? N : (want > hi ? hi : want);
    if (m_budget != want && t == 0) atomicOr(&sStatus, 4 /*BAD_LEN*/);
  }
  const int delta = m_budget - sum0;
  if (i < N && delta != 0) {
    const int k0i = sK0[i];
    const float v = sQ[i][j];
    if (delta > 0 && j >= k0i && j < Wd) {
      int rank = j - k0i;
      for (int r = 0; r < N && rank < delta; ++r) {
        if (r == i) continue;
        const int k0r = sK0[r];
        int c = 0;
        if (r < i) { for (int jj = k0r; jj < Wd && sQ[r][jj] >= v; ++jj) ++c; }
        else       { for (int jj = k0r; jj < Wd && sQ[r][jj] >  v; ++jj) ++c; }
        rank += c;
      }
      if (rank < delta) atomicAdd(&sAdj[i], 1);
    } else if (delta < 0 && j >= 1 && j <= k0i - 1) {
      int rank = k0i - 1 - j;
      for (int r = 0; r < N && rank < -delta; ++r) {
        if (r == i) continue;
        const int k0r = sK0[r];
        int c = 0;
        if (r < i) { for (int jj = k0r - 1; jj >= 1 && sQ[r][jj] <= v; --jj) ++c; }
        else       { for (int jj = k0r - 1; jj >= 1 && sQ[r][jj] <  v; --jj) ++c; }
        rank += c;
      }
      if (rank < -delta) atomicAdd(&sAdj[i], -1);
    }
  }
  __syncthreads();

  // ---- 3. offsets and key-tile prefix: two-warp shuffle scan ---------------
  if (t < kMaxNbs) {
    const int lane = t & 31, w = t >> 5;
    const int kk = (t < N) ? sK0[t] + sAdj[t] : 0;
    sK[t] = kk;
    const int tiles = (t < N) ? (sCtx[t] + kk + kTileTok - 1) / kTileTok : 0;
    int sk = warp_incl_scan(kk, lane);
    int stl = warp_incl_scan(tiles, lane);
    if (lane == 31) { sWarpTot[w] = sk; sWarpTot[2 + w] = stl; }
    __syncwarp();
    // second warp adds the first warp's totals (visible after the block sync below)
    sOff[t + 1] = sk;
    sTilePre[t + 1] = stl;
  }
  __syncthreads();
  if (t >= 32 && t < kMaxNbs) { sOff[t + 1] += sWarpTot[0]; sTilePre[t + 1] += sWarpTot[2]; }
  if (t == 0) { sOff[0] = 0; sTilePre[0] = 0; }
  __syncthreads();

  const int m_live = m_budget;
  const int m_bs = kHalfW * n_bs;
  int* wk = ws_ptr<int>(a.ws, L.k);
  int* wk0 = ws_ptr<int>(a.ws, L.k0);
  int* woff = ws_ptr<int>(a.ws, L.offset);
  int* wqs = ws_ptr<int>(a.ws, L.q_start);
  int* wqe = ws_ptr<int>(a.ws, L.q_end);
  int* wtok = ws_ptr<int>(a.ws, L.tokens);
  int* wpos = ws_ptr<int>(a.ws, L.positions);
  int* wref = ws_ptr<int>(a.ws, L.kv_refs);
  int* wreq = ws_ptr<int>(a.ws, L.row_req);
  int* wkvl = ws_ptr<int>(a.ws, L.kv_len);
  int* wtp = ws_ptr<int>(a.ws, L.tile_prefix);
  float* wq = ws_ptr<float>(a.ws, L.qscores);

  // per-request fields; sentinels: k = 0, offset_{i+1} = M_live
  if (t < n_bs) {
    const bool live = t < N;
    const int off = live ? sOff[t] : m_live;
    wk[t] = sK[t];
    wk0[t] = live ? sK0[t] : 0;
    woff[t + 1] = live ? sOff[t + 1] : m_live;
    wqs[t] = off;
    wqe[t] = off + sK[t];
    wkvl[t] = live ? sCtx[t] + sK[t] : 0;
    wtp[t + 1] = sTilePre[min(t + 1, kMaxNbs)];
    if (t == 0) { woff[0] = 0; wtp[0] = 0; }
  }
  if (i < n_bs) wq[i * kW + j] = (i < N) ? sQ[i][j] : 0.0f;

  // flat-pack (Eq. 11): one thread per (request, slot)
  if (i < N && j < sK[i]) {
    const int s = sOff[i] + j;
    const int pos = sCtx[i] + j;
    int page = a.block_table[(size_t)i * a.max_pages + pos / kPage];
    if (page < 0 || page >= a.num_pages) { atomicOr(&sStatus, 2); page = 0; }
    wtok[s] = a.draft_tokens[i * kW + j];
    wpos[s] = pos;
    wref[s] = page * kPage + pos % kPage;
    wreq[s] = i;
  }
  // tail placeholders: (token 0, position 0, first KV ref of the first request)
  if (t >= m_live && t < m_bs) {
    const int pos = sCtx[0];
    int page = a.block_table[pos / kPage];
    if (page < 0 || page >= a.num_pages) page = 0;
    wtok[t] = 0;
    wpos[t] = 0;
    wref[t] = page * kPage + pos % kPage;
    wreq[t] = -1;
  }
  // ---- attention schedule: slice c of the persistent grid starts at linear key tile
  // slice_tab[c] (request-major, then kv-head, then tile).  Slices have equal COST under a
  // measured model of the attention kernel: a tile of a request with more than 8 window rows
  // costs 6 % more (both groups of softmax warps work), and every (request, kv-head) pair a
  // CTA starts costs about 0.8 tile (epilogue of the previous pair, first scores of the next).
  // The last CTAs of a launch start late (they land on the SMs that finished the previous
  // launch last) and get two to three tiles less.  Small tile counts (under 8 per CTA) are
  // cut by count, and with fewer tiles than CTAs the first T CTAs get one tile each.
  for (int cta = t; cta <= a.num_ctas; cta += blockDim.x) {
    const int n_kv = a.n_kv_heads;
    const long long T = (long long)sTilePre[kMaxNbs] * n_kv;
    const long long C = T < a.num_ctas ? T : a.num_ctas;
    long long tile = T;
    if (cta < C) {
      const bool by_count = T < 8 * C;
      const int run_cost = by_count ? 0 : kRunCost;
      auto tile_cost = [&](int r) { return by_count ? 1 : (sK[r] > 8 ? kTileCostBig : kTileCostSmall); };
      long long W = 0;
      for (int r = 0; r < N; ++r)
        W += ((long long)(sTilePre[r + 1] - sTilePre[r]) * tile_cost(r) + run_cost) * n_kv;
      // late starters: the last kLateCtas CTAs give up kLateTiles[.] tiles each
      const bool skew = !by_count && C >= 4 * kLateCtas && T / C >= 24;
      long long pen_total = 0, pen_before = 0;
      if (skew) {
        for (int j = 0; j < kLateCtas; ++j) {
          const long long pen = (long long)kLateTiles[j] * kTileCostSmall;
          pen_total += pen;
          if (C - kLateCtas + j < cta) pen_before += pen;
        }
      }
      const long long Wv = W + pen_total;                    // equal shares of a slightly longer list ...
      const long long x = (long long)cta * Wv / C - pen_before;   // ... of which the late starters give some back
      long long acc = 0;
      for (int r = 0; r < N; ++r) {
        const int n_r = sTilePre[r + 1] - sTilePre[r];
        const long long pair_cost = (long long)n_r * tile_cost(r) + run_cost;
        const long long rc = pair_cost * n_kv;
        if (x < acc + rc) {
          const long long g = (x - acc) / pair_cost, within = (x - acc) % pair_cost;
          long long in_pair = within > run_cost ? (within - run_cost) / tile_cost(r) : 0;
          if (in_pair >= n_r) in_pair = n_r - 1;
          tile = (long long)sTilePre[r] * n_kv + g * n_r + in_pair;
          break;
        }
        acc += rc;
      }
    }
    ws_ptr<int>(a.ws, L.slice_tab)[cta] = (int)tile;
  }
  __syncthreads();
  if (t == 0) {
    hdr[H_N_LIVE] = N;
    hdr[H_M_LIVE] = m_live;
    hdr[H_TOTAL_TILES] = sTilePre[kMaxNbs];
    if (sStatus) atomicOr(&hdr[H_STATUS], sStatus);
  }
}

}  // namespace

cudaError_t launch_alloc(const AllocArgs& a, cudaStream_t stream) {
  WsLayout L = ws_layout(a.n_bs, a.n_kv_heads, a.num_ctas);
  dvl_alloc_kernel<<<1, 1024, 0, stream>>>(a, L);
  return cudaGetLastError();
}

}  // namespace dscale
