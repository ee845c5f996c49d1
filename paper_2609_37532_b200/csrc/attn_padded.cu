// Comparison baseline: unpacked W = 16 verify attention with the prefill-shaped
// 128-row tile (Section 2.1 of the paper: one computation block handles one
// request's query tile for ONE head; a verification request supplies 16 rows,
// the other 112 rows of the tile are masked but still occupy it).
//
// What this kernel deliberately keeps from that design, so that the comparison
// with dscale_verify_attn is about the method and not about kernel quality:
//   * every live request verifies all 16 slots (no DVL lengths, 16 N rows);
//   * the tile belongs to one (request, q-head): K/V are streamed once per
//     q-head, i.e. 4 times per kv-head for a GQA group of 4;
//   * the MMAs run on the full M = 128 tile and the softmax warps process all
//     128 rows, live or not.
// Everything else is the same machinery as the packed kernel (TMA page boxes,
// tcgen05 MMAs with TMEM accumulators, a persistent grid over an even split of
// the key tiles, in-kernel merge of cut pairs), in its simplest form.
#include "kernels.cuh"
#include "tc_ptx.cuh"
#include "tile_schedule.cuh"

#include <map>
#include <mutex>

namespace dscale {

namespace {

constexpr int kThreads = 192;               // 4 softmax warps, producer, MMA issuer
constexpr int kSoftmaxThreads = 128;
constexpr int kStages = 3;
constexpr int kRows = 128;                  // tile rows (16 live)
constexpr int kSlotBytes = kTileTok * kD * 2;
constexpr int kHalfSlot = kSlotBytes / 2;
constexpr int kQBytes = kRows * kD * 2;     // 32 KB (two 64-column halves of 128 rows)
constexpr int kPBytes = kRows * kTileTok * 2;
constexpr int kPageBoxBytes = kPage * 64 * 2;

constexpr int kOffQ = 0;
constexpr int kOffP = kOffQ + 2 * kQBytes;
constexpr int kOffKV = kOffP + 2 * kPBytes;
constexpr int kOffBar = kOffKV + kStages * kSlotBytes;
constexpr int kOffMisc = kOffBar + 8 * 24;
constexpr int kOffTile = kOffMisc + 32;
constexpr int kSmemUse = kOffTile + (kMaxNbs + 1) * 4 + 12;
constexpr int kSmemBytes = kSmemUse + 1024;
static_assert(kSmemBytes <= 232448, "exceeds the 227 KB shared memory of an sm_100 CTA");

enum Bar { B_KV_FULL = 0, B_KV_EMPTY = kStages, B_Q_FULL = 2 * kStages, B_Q_EMPTY = B_Q_FULL + 2,
           B_S_FULL = B_Q_EMPTY + 2, B_P_FULL = B_S_FULL + 2, B_O_FULL = B_P_FULL + 2,
           B_GROUP = B_O_FULL + 2 };

// bf16 x bf16 -> fp32, M = 128, N = 128
constexpr uint32_t kIdescBase = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) |
                                ((128u >> 4) << 24);
constexpr uint32_t kIdescS = kIdescBase;
constexpr uint32_t kIdescPV = kIdescBase | (1u << 16);

struct PaddedArgs {
  void* ws;
  int n_bs;
  const int32_t* ctx_len;
  const int32_t* block_table;
  int max_pages, num_pages;
  int n_q_heads, n_kv_heads;
  float sm_scale;
  void* out;                       // bf16 [n_bs][16][n_q_heads][128]
};

__global__ void __launch_bounds__(kThreads, 1)
attn_padded_kernel(PaddedArgs a, WsLayout L, const __grid_constant__ CUtensorMap tm_q,
                   const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v) {
  extern __shared__ unsigned char smem_dyn[];
  const uint32_t raw = smem_u32(smem_dyn);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* sm = smem_dyn + (base - raw);
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(sm + kOffMisc);
  volatile int* s_abort = reinterpret_cast<volatile int*>(sm + kOffMisc + 4);
  int* s_ticket = reinterpret_cast<int*>(sm + kOffMisc + 8);
  volatile int* s_dummy = reinterpret_cast<volatile int*>(sm + kOffMisc + 16);
  int* s_tile = reinterpret_cast<int*>(sm + kOffTile);
  auto bar = [&](int b) { return base + kOffBar + 8u * b; };

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int c = blockIdx.x;
  int* hdr = ws_ptr<int>(a.ws, L.hdr);
  const int n_bs = a.n_bs, Hq = a.n_q_heads, G = a.n_q_heads / a.n_kv_heads;
  const int N = min(max(hdr[H_N_LIVE], 1), n_bs);

  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(bar(B_KV_FULL + s), 1); mbar_init(bar(B_KV_EMPTY + s), 1); }
    for (int b = 0; b < 2; ++b) {
      mbar_init(bar(B_Q_FULL + b), 1); mbar_init(bar(B_Q_EMPTY + b), 1);
      mbar_init(bar(B_S_FULL + b), 1); mbar_init(bar(B_P_FULL + b), kSoftmaxThreads);
      mbar_init(bar(B_O_FULL + b), 1);
    }
    mbar_init(bar(B_GROUP), kSoftmaxThreads);
    *s_abort = 0;
    *s_dummy = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // per-request key-tile counts for W = 16 slots each (prefix-summed below)
  if (tid < n_bs) {
    const int ctx = min(max(a.ctx_len[tid], 0), a.max_pages * kPage - kW);
    s_tile[tid + 1] = tid < N ? (ctx + kW + kTileTok - 1) / kTileTok : 0;
  }
  __syncthreads();
  if (tid == 0) {
    s_tile[0] = 0;
    for (int i = 0; i < n_bs; ++i) s_tile[i + 1] += s_tile[i];
  }
  // rows 16..127 of both Q buffers stay zero for the whole kernel (TMA only
  // writes the 16 live rows): masked rows then carry finite scores
  for (int x = tid; x < 2 * kQBytes / 16; x += kThreads)
    st_shared_v4(base + kOffQ + x * 16, 0, 0, 0, 0);
  if (warp == 5) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;"
                 ::"r"(smem_u32(s_tmem)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  fence_async_smem();
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *s_tmem;

  const long long T = (long long)s_tile[n_bs] * Hq;
  const int C = (int)min((long long)gridDim.x, T);
  const long long sl_begin = c < C ? slice_begin(c, T, C) : 0;
  const long long sl_end = c < C ? slice_begin(c + 1, T, C) : 0;
  __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(a.out);
  auto ctx_of = [&](int i) { return min(max(a.ctx_len[i], 0), a.max_pages * kPage - kW); };

  if (warp == 4) {
    // ===================================================== TMA producer warp
    Scheduler sch; sch.init(s_tile, n_bs, Hq, sl_begin, sl_end);
    Segment sg;
    unsigned u = 0;
    int seg = 0;
    bool ok = true;
    const int pg_l = lane >> 1, half = lane & 1;
    while (ok && sch.next(sg)) {
      const int qb = seg & 1;
      ok = mbar_wait(bar(B_Q_EMPTY + qb), ((seg >> 1) & 1) ^ 1, s_abort);
      if (!ok) break;
      if (lane == 0) {
        mbar_expect_tx(bar(B_Q_FULL + qb), 2 * kW * 128);
        tma_load_5d(base + kOffQ + qb * kQBytes, &tm_q, bar(B_Q_FULL + qb), 0, 0, sg.g, 0, sg.i);
        tma_load_5d(base + kOffQ + qb * kQBytes + kQBytes / 2, &tm_q, bar(B_Q_FULL + qb), 0, 1,
                    sg.g, 0, sg.i);
      }
      const int len = ctx_of(sg.i) + kW;
      const int kvh = sg.g / G;
      const int* bt = a.block_table + (size_t)sg.i * a.max_pages;
      auto fetch_page = [&](int t) -> int {
        const int p = t * (kTileTok / kPage) + pg_l;
        int id = 0;
        if (lane < 16 && p * kPage < len) {
          id = bt[p];
          if (id < 0 || id >= a.num_pages) { atomicOr(&hdr[H_STATUS], 2); id = 0; }
        }
        return id;
      };
      int page_next = fetch_page(sg.t0);
      for (int t = sg.t0; t < sg.t1 && ok; ++t) {
        const int page = page_next;
        if (t + 1 < sg.t1) page_next = fetch_page(t + 1);
        const int valid_tok = min(kTileTok, len - t * kTileTok);
        const int n_pages = (valid_tok + kPage - 1) / kPage;
#pragma unroll
        for (int which = 0; which < 2; ++which, ++u) {
          const int slot = u % kStages;
          ok = mbar_wait(bar(B_KV_EMPTY + slot), ((u / kStages) & 1) ^ 1, s_abort);
          if (!ok) break;
          if (lane == 0) mbar_expect_tx(bar(B_KV_FULL + slot), n_pages * 2 * kPageBoxBytes);
          __syncwarp();
          if (lane < 16 && pg_l < n_pages) {
            tma_load_5d(base + kOffKV + slot * kSlotBytes + half * kHalfSlot + pg_l * kPageBoxBytes,
                        which == 0 ? &tm_k : &tm_v, bar(B_KV_FULL + slot), 0, half, 0, kvh, page);
          }
        }
      }
      ++seg;
    }
    if (!ok) {
      for (unsigned v = (u > kStages ? u - kStages : 0); v < u; ++v)
        mbar_wait(bar(B_KV_FULL + v % kStages), (v / kStages) & 1, s_dummy);
    }
  } else if (warp == 5) {
    // ============================================================ MMA issuer
    if (lane == 0) {
      Scheduler sch; sch.init(s_tile, n_bs, Hq, sl_begin, sl_end);
      Segment sg;
      unsigned it = 0;
      int seg = 0;
      bool ok = true;
      bool first_of_run[2] = {true, true};
      auto issue_pv = [&](unsigned pt) -> bool {
        const int b = pt & 1;
        const unsigned uv = 2 * pt + 1;
        const int slot = uv % kStages;
        if (!mbar_wait(bar(B_P_FULL + b), (pt >> 1) & 1, s_abort)) return false;
        if (!mbar_wait(bar(B_KV_FULL + slot), (uv / kStages) & 1, s_abort)) return false;
        tc_fence_after();
        const uint32_t p_base = base + kOffP + b * kPBytes;
        const uint32_t v_base = base + kOffKV + slot * kSlotBytes;
#pragma unroll
        for (int kk = 0; kk < kTileTok / 16; ++kk) {
          const uint64_t ad = smem_desc(p_base + (kk >> 2) * (kRows * 128) + (kk & 3) * 32, 16, 1024);
          const uint64_t bd = smem_desc(v_base + kk * (16 * 128), kHalfSlot, 1024);
          umma(tmem + 256, ad, bd, kIdescPV, (kk > 0) || !first_of_run[b]);
        }
        umma_commit(bar(B_O_FULL + b));
        umma_commit(bar(B_KV_EMPTY + slot));
        return true;
      };
      while (ok && sch.next(sg)) {
        const int qb = seg & 1;
        ok = mbar_wait(bar(B_Q_FULL + qb), (seg >> 1) & 1, s_abort);
        for (int t = sg.t0; t < sg.t1 && ok; ++t, ++it) {
          const int b = it & 1;
          first_of_run[b] = (t == sg.t0);
          const unsigned uk = 2 * it;
          const int slot = uk % kStages;
          ok = mbar_wait(bar(B_KV_FULL + slot), (uk / kStages) & 1, s_abort);
          if (!ok) break;
          tc_fence_after();
          const uint32_t q_base = base + kOffQ + qb * kQBytes;
          const uint32_t k_base = base + kOffKV + slot * kSlotBytes;
#pragma unroll
          for (int kk = 0; kk < kD / 16; ++kk) {
            const uint64_t ad = smem_desc(q_base + (kk >> 2) * (kRows * 128) + (kk & 3) * 32, 16, 1024);
            const uint64_t bd = smem_desc(k_base + (kk >> 2) * kHalfSlot + (kk & 3) * 32, 16, 1024);
            umma(tmem + b * 128, ad, bd, kIdescS, kk > 0);
          }
          umma_commit(bar(B_S_FULL + b));
          umma_commit(bar(B_KV_EMPTY + slot));
          if (t + 1 == sg.t1) umma_commit(bar(B_Q_EMPTY + qb));
          if (it >= 1) ok = issue_pv(it - 1);
        }
        ++seg;
      }
      if (ok && it >= 1) ok = issue_pv(it - 1);
    }
    __syncwarp();
  } else {
    // ====================================================== softmax warps 0-3
    // capacity rows of requests beyond N are written as zero
    {
      const long long n16 = (long long)(n_bs - N) * kW * Hq * (kD * 2 / 16);
      uint4* dst = reinterpret_cast<uint4*>(out + (size_t)N * kW * Hq * kD);
      for (long long x = (long long)c * kSoftmaxThreads + tid; x < n16;
           x += (long long)gridDim.x * kSoftmaxThreads)
        dst[x] = make_uint4(0, 0, 0, 0);
    }
    const int row = warp * 32 + lane;                 // tile row = TMEM lane; slot j = row for row < 16
    const bool live = row < kW;
    const uint32_t t_lane = tmem + ((uint32_t)(warp * 32) << 16);
    const uint32_t o_addr = t_lane + 256;
    const float scale_log2 = a.sm_scale * 1.4426950408889634f;
    // partial slots: [cta][2][16 rows][128] fp32 and (max, sum), carved from the
    // packed kernel's partial area (disjoint use: the two kernels never overlap)
    float* part_o = ws_ptr<float>(a.ws, L.part_o);
    float* part_ml = ws_ptr<float>(a.ws, L.part_ml);
    int* pair_cnt = ws_ptr<int>(a.ws, L.pad_cnt);

    Scheduler sch; sch.init(s_tile, n_bs, Hq, sl_begin, sl_end);
    Segment sg;
    unsigned it = 0;
    bool ok = true;
    int pend_i[2], pend_h[2], pend_n[2], n_pend = 0;
    auto wait_pv = [&](unsigned pt) -> bool {
      return mbar_wait(bar(B_O_FULL + (pt & 1)), (pt >> 1) & 1, s_abort);
    };

    while (ok && sch.next(sg)) {
      const int ctx = ctx_of(sg.i);
      const int len = ctx + kW;
      const int pos = live ? ctx + row : (1 << 30);        // masked rows: treated as seeing everything
      float m_ref = -INFINITY, l_run = 0.0f;
      for (int t = sg.t0; t < sg.t1 && ok; ++t, ++it) {
        const int b = it & 1;
        ok = mbar_wait(bar(B_S_FULL + b), (it >> 1) & 1, s_abort);
        if (!ok) break;
        tc_fence_after();
        float s[kTileTok];
        tmem_ld128(t_lane + b * 128, s);
        // keys at or beyond the request's key count are invisible to every row
        const int vis = min(min(kTileTok, len - t * kTileTok), max(0, pos + 1 - t * kTileTok));
        float m8[8];
#pragma unroll
        for (int x = 0; x < 8; ++x) m8[x] = -INFINITY;
        if (vis >= kTileTok) {
#pragma unroll
          for (int x = 0; x < kTileTok; ++x) m8[x & 7] = fmaxf(m8[x & 7], s[x]);
        } else {
#pragma unroll
          for (int x = 0; x < kTileTok; ++x) m8[x & 7] = (x < vis) ? fmaxf(m8[x & 7], s[x]) : m8[x & 7];
        }
        float mx = fmaxf(fmaxf(fmaxf(m8[0], m8[1]), fmaxf(m8[2], m8[3])),
                         fmaxf(fmaxf(m8[4], m8[5]), fmaxf(m8[6], m8[7]))) * scale_log2;
        float factor = 1.0f;
        bool need = false;
        if (t == sg.t0) {
          m_ref = mx;
        } else if (mx > m_ref + 8.0f) {
          factor = ex2(m_ref - mx);
          m_ref = mx;
          l_run *= factor;
          need = true;
        }
        if (__any_sync(0xffffffffu, need)) {
          ok = wait_pv(it - 1);
          if (!ok) break;
          tc_fence_after();
#pragma unroll
          for (int ch = 0; ch < 4; ++ch) {
            float o[32];
            tmem_ld32(o_addr + ch * 32, o);
#pragma unroll
            for (int x = 0; x < 32; ++x) o[x] *= factor;
            tmem_st32(o_addr + ch * 32, o);
          }
          tmem_st_wait();
        }
        const float m_safe = (m_ref == -INFINITY) ? 0.0f : m_ref;
        if (it >= 2) { ok = wait_pv(it - 2); if (!ok) break; }
        const uint32_t p_row = base + kOffP + b * kPBytes + row * 128;
        float ps[8];
#pragma unroll
        for (int x = 0; x < 8; ++x) ps[x] = 0.0f;
#pragma unroll
        for (int chunk = 0; chunk < kTileTok / 8; ++chunk) {
          float p[8];
#pragma unroll
          for (int x = 0; x < 8; ++x) {
            const float e = ex2(fmaf(s[chunk * 8 + x], scale_log2, -m_safe));
            p[x] = (chunk * 8 + x < vis) ? e : 0.0f;
            ps[x] += p[x];
          }
          const uint32_t addr = p_row + (chunk >> 3) * (kRows * 128) + (((chunk & 7) ^ (row & 7)) << 4);
          st_shared_v4(addr, pack_bf16(p[0], p[1]), pack_bf16(p[2], p[3]), pack_bf16(p[4], p[5]),
                       pack_bf16(p[6], p[7]));
        }
        l_run += ((ps[0] + ps[1]) + (ps[2] + ps[3])) + ((ps[4] + ps[5]) + (ps[6] + ps[7]));
        // last tile of the pair: V rows at or beyond the key count must be finite
        if (t + 1 == sg.n_tiles && len - t * kTileTok < kTileTok) {
          const unsigned uv = 2 * it + 1;
          const int slot = uv % kStages;
          ok = mbar_wait(bar(B_KV_FULL + slot), (uv / kStages) & 1, s_abort);
          if (!ok) break;
          const int first = len - t * kTileTok;
          const int n_chunks = (kTileTok - first) * 16;
          const uint32_t v_base = base + kOffKV + slot * kSlotBytes;
          for (int x = tid; x < n_chunks; x += kSoftmaxThreads) {
            const int r = first + (x >> 4), hc = x & 15;
            st_shared_v4(v_base + (hc >> 3) * kHalfSlot + r * 128 + ((hc & 7) << 4), 0, 0, 0, 0);
          }
        }
        tc_fence_before();
        fence_async_smem();
        mbar_arrive(bar(B_P_FULL + b));
      }
      if (!ok) break;
      ok = wait_pv(it - 1);
      if (!ok) break;
      tc_fence_after();
      float acc[kD];
      tmem_ld128(o_addr, acc);
      tc_fence_before();
      const bool whole = (sg.t0 == 0 && sg.t1 == sg.n_tiles);
      if (whole) {
        if (live) {
          const float inv = 1.0f / l_run;
          uint4* dst = reinterpret_cast<uint4*>(out + (((size_t)sg.i * kW + row) * Hq + sg.g) * kD);
#pragma unroll
          for (int d = 0; d < kD; d += 8)
            dst[d >> 3] = make_uint4(pack_bf16(acc[d] * inv, acc[d + 1] * inv),
                                     pack_bf16(acc[d + 2] * inv, acc[d + 3] * inv),
                                     pack_bf16(acc[d + 4] * inv, acc[d + 5] * inv),
                                     pack_bf16(acc[d + 6] * inv, acc[d + 7] * inv));
        }
      } else {
        const int slot_id = c * 2 + (sg.first_of_cta ? 0 : 1);
        if (live) {
          float4* po = reinterpret_cast<float4*>(part_o + ((size_t)slot_id * kW + row) * kD);
#pragma unroll
          for (int d = 0; d < kD; d += 4) po[d >> 2] = make_float4(acc[d], acc[d + 1], acc[d + 2], acc[d + 3]);
          *reinterpret_cast<float2*>(&part_ml[((size_t)slot_id * kW + row) * 2]) = make_float2(m_ref, l_run);
        }
        pend_i[n_pend] = sg.i; pend_h[n_pend] = sg.g; pend_n[n_pend] = sg.n_tiles;
        ++n_pend;
      }
    }
    // ---- publish the partial runs, merge the pairs this CTA is last to reach
    if (ok && n_pend > 0) {
      unsigned group_phase = 0;
      auto group_sync = [&]() -> bool {
        mbar_arrive(bar(B_GROUP));
        const bool r = mbar_wait(bar(B_GROUP), group_phase & 1, s_abort);
        ++group_phase;
        return r;
      };
      __threadfence();
      ok = group_sync();
      if (ok && lane == 0 && warp < n_pend) {
        const int x = warp;
        const long long p0 = ((long long)s_tile[pend_i[x]] * Hq) + (long long)pend_h[x] * pend_n[x];
        const int n_contrib = cta_of(p0 + pend_n[x] - 1, T, C) - cta_of(p0, T, C) + 1;
        int* cnt = &pair_cnt[pend_i[x] * Hq + pend_h[x]];
        const int old = atomicAdd(cnt, 1);
        s_ticket[x] = (old == n_contrib - 1);
        if (old == n_contrib - 1) *cnt = 0;
      }
      if (ok) ok = group_sync();
      for (int x = 0; ok && x < n_pend; ++x) {
        if (!s_ticket[x]) continue;
        __threadfence();
        const int pi = pend_i[x], ph = pend_h[x];
        const long long p0 = ((long long)s_tile[pi] * Hq) + (long long)ph * pend_n[x];
        const int c_lo = cta_of(p0, T, C), c_hi = cta_of(p0 + pend_n[x] - 1, T, C);
        // thread t: slot row t / 8, columns 16 (t % 8) .. + 15
        const int r = tid >> 3, col = (tid & 7) * 16;
        float av[16];
        float m_run = -INFINITY, l_tot = 0.0f;
#pragma unroll
        for (int d = 0; d < 16; ++d) av[d] = 0.0f;
        for (int cc = c_lo; cc <= c_hi; ++cc) {
          const int sid = cc * 2 + (slice_begin(cc, T, C) >= p0 ? 0 : 1);
          const float2 ml = __ldcg(reinterpret_cast<const float2*>(&part_ml[((size_t)sid * kW + r) * 2]));
          const float4* po = reinterpret_cast<const float4*>(part_o + ((size_t)sid * kW + r) * kD + col);
          const float4 v0 = __ldcg(po), v1 = __ldcg(po + 1), v2 = __ldcg(po + 2), v3 = __ldcg(po + 3);
          const float m_tot = fmaxf(m_run, ml.x);
          const float m_s = (m_tot == -INFINITY) ? 0.0f : m_tot;
          const float w0 = ex2(m_run - m_s), w1 = ex2(ml.x - m_s);
          const float vv[16] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w,
                                v2.x, v2.y, v2.z, v2.w, v3.x, v3.y, v3.z, v3.w};
#pragma unroll
          for (int d = 0; d < 16; ++d) av[d] = av[d] * w0 + vv[d] * w1;
          l_tot = l_tot * w0 + ml.y * w1;
          m_run = m_tot;
        }
        const float inv = 1.0f / l_tot;
        uint4* dst = reinterpret_cast<uint4*>(out + (((size_t)pi * kW + r) * Hq + ph) * kD + col);
        dst[0] = make_uint4(pack_bf16(av[0] * inv, av[1] * inv), pack_bf16(av[2] * inv, av[3] * inv),
                            pack_bf16(av[4] * inv, av[5] * inv), pack_bf16(av[6] * inv, av[7] * inv));
        dst[1] = make_uint4(pack_bf16(av[8] * inv, av[9] * inv), pack_bf16(av[10] * inv, av[11] * inv),
                            pack_bf16(av[12] * inv, av[13] * inv), pack_bf16(av[14] * inv, av[15] * inv));
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (tid == 0 && *s_abort) atomicOr(&hdr[H_STATUS], 8 /*TIMEOUT*/);
  if (warp == 5) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
  }
}

// ------------------------------------------------------------ host: tensor maps
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn get_encode() {
  static EncodeTiledFn fn = nullptr;
  static bool tried = false;
  if (!tried) {
    tried = true;
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

bool encode(CUtensorMap* out, const void* ptr, int rank, const cuuint64_t* dims,
            const cuuint64_t* strides, const cuuint32_t* box) {
  EncodeTiledFn enc = get_encode();
  if (!enc) return false;
  cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  return enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, rank, const_cast<void*>(ptr), dims, strides, box,
             estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
             CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

cudaError_t attn_padded_prepare() {
  return cudaFuncSetAttribute(attn_padded_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              kSmemBytes);
}

cudaError_t launch_attn_padded(void* ws, int n_bs, const void* q_unpacked, const void* k_cache,
                               const void* v_cache, const int32_t* block_table, int max_pages,
                               int num_pages, const int32_t* ctx_len, int n_q_heads,
                               int n_kv_heads, float sm_scale, void* out_unpacked, int num_ctas,
                               cudaStream_t stream) {
  WsLayout L = ws_layout(n_bs, n_kv_heads, num_ctas);
  CUtensorMap tq, tk, tv;
  {
    // q: [n_bs][16][n_q][128] viewed as (d_lo 64, d_hi 2, head, slot 16, request)
    cuuint64_t dims[5] = {64, 2, (cuuint64_t)n_q_heads, (cuuint64_t)kW, (cuuint64_t)n_bs};
    cuuint64_t strides[4] = {128, (cuuint64_t)kD * 2, (cuuint64_t)n_q_heads * kD * 2,
                             (cuuint64_t)kW * n_q_heads * kD * 2};
    cuuint32_t box[5] = {64, 1, 1, (cuuint32_t)kW, 1};
    if (!encode(&tq, q_unpacked, 5, dims, strides, box)) return cudaErrorNotSupported;
  }
  for (int which = 0; which < 2; ++which) {
    cuuint64_t dims[5] = {64, 2, (cuuint64_t)kPage, (cuuint64_t)n_kv_heads, (cuuint64_t)num_pages};
    cuuint64_t strides[4] = {128, 256, (cuuint64_t)kPage * kD * 2, (cuuint64_t)n_kv_heads * kPage * kD * 2};
    cuuint32_t box[5] = {64, 1, (cuuint32_t)kPage, 1, 1};
    if (!encode(which ? &tv : &tk, which ? v_cache : k_cache, 5, dims, strides, box))
      return cudaErrorNotSupported;
  }
  PaddedArgs a{ws, n_bs, ctx_len, block_table, max_pages, num_pages, n_q_heads, n_kv_heads, sm_scale,
               out_unpacked};
  attn_padded_kernel<<<num_ctas, kThreads, kSmemBytes, stream>>>(a, L, tq, tk, tv);
  return cudaGetLastError();
}

}  // namespace dscale
