// Fused LM head + target-token argmax + greedy acceptance for the packed rows.
//
// top1[s] = argmax_v sum_h hidden[s][h] * weight[v][h]  for the 8N live packed
// rows, without ever writing the 8N x V logits (at N = 32 that is 155 MB of fp32
// written and read back, next to 1.24 GB of bf16 weights that have to be read
// anyway).  A dense contraction: this one belongs on the tensor cores.
//
// Up to 128 packed rows: each CTA of a persistent grid owns a contiguous range of
// vocabulary columns, cut into equal tiles of n_tile <= 256 columns (a multiple
// of 16, chosen on the host so that all CTAs get the same number of equal tiles),
// and accumulates a tile in TMEM, so every weight element is read from HBM
// exactly once; the hidden rows are re-read from L2.
//   warp 4   TMA producer: per 64-wide k step the hidden box [128 rows][64] and
//            the weight box [n_tile rows][64], 128-byte swizzle, ring of
//            shared-memory stages with mbarrier expect-tx; one lane per box.
//   warp 5   one thread issues tcgen05.mma (M128, N = n_tile, K16 x 4 per step).
//   warps 0-3  epilogue: thread = packed row; tcgen05.ld 32 columns at a time,
//            running (max, first index); after the CTA's last tile one partial
//            per (row, CTA) goes to the workspace.
// More than 128 rows: pairs of CTAs (cta_group::2, further down), which halve the
// hidden-state traffic per weight byte.  (The one-CTA kernel is written for up to
// four row tiles; only the one-tile form is built and used.)
// The last CTA to finish (ticket, nobody waits) merges the partials in vocabulary
// order -- so equal maxima resolve to the lowest index -- and runs the acceptance
// loop of the "Prefix verifier" paragraph.
#include <climits>
#include <mutex>

#include "kernels.cuh"
#include "tc_ptx.cuh"

namespace dscale {

#ifdef DSCALE_WAIT_TEST
__device__ int g_lm_drop_cta = -1, g_lm_drop_step = -1;
#endif

namespace {

constexpr int kThreads = 192;
constexpr int kEpiThreads = 128;
constexpr int kKStep = 64;                       // bf16 elements per k step = one 128-byte swizzle row
constexpr int kATile = 128 * kKStep * 2;         // 16 KB: 128 rows x 64 columns

struct LmShape {
  int m_tiles;        // row tiles of 128 packed rows
  int n_tile;         // vocabulary columns per tile (multiple of 16, <= 256)
  int tiles_per_cta;
  int cols_per_cta;   // n_tile * tiles_per_cta
  int stages;
  int stage_bytes;
  int b_bytes;        // bytes of one weight box, rounded up to 1024
  int a_rows;         // rows of one hidden box
  int smem_bytes;
};

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float* v) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];\n\t"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
#pragma unroll
  for (int x = 0; x < 16; ++x) v[x] = __uint_as_float(r[x]);
}

struct LmArgs {
  void* ws;
  int n_bs;
  int hidden_dim;
  int vocab;
  int32_t* accept_len;
  int32_t* next_anchor;
  int32_t* out_tokens;
  int32_t* out_len;
  int32_t* ctx_len_inout;
  float* row_max;          // nullable [8 n_bs]: the winning logit of every live row
};

// Running (max, first index) over the n fp32 accumulator columns at TMEM address
// `taddr` of this thread's lane; column x is vocabulary entry col0 + x.  The
// loads are warp-collective, so dead rows load too and only skip the compare.
__device__ __forceinline__ void scan_acc(uint32_t taddr, int n, int col0, int vocab, bool live,
                                         float& best, int& best_i) {
  for (int ch = 0; ch + 32 <= n; ch += 32) {
    float v[32];
    tmem_ld32(taddr + ch, v);
    if (live) {
#pragma unroll
      for (int x = 0; x < 32; ++x) {
        const int col = col0 + ch + x;
        if (col < vocab && v[x] > best) { best = v[x]; best_i = col; }
      }
    }
  }
  if (n & 16) {
    const int ch = n & ~31;
    float v[16];
    tmem_ld16(taddr + ch, v);
    if (live) {
#pragma unroll
      for (int x = 0; x < 16; ++x) {
        const int col = col0 + ch + x;
        if (col < vocab && v[x] > best) { best = v[x]; best_i = col; }
      }
    }
  }
}

// After a CTA's last tile: one (max, index) partial per (row, part) goes to the
// workspace; the last CTA to finish (ticket, nobody waits) merges the parts in
// vocabulary order -- so equal maxima resolve to the lowest index -- and runs the
// acceptance loop of the "Prefix verifier" paragraph.  Called by the 128 epilogue
// threads of a CTA; `rows[m]` is the packed row this thread holds in best[m].
__device__ __forceinline__ void lm_finish(const LmArgs& a, const WsLayout& L, int* hdr, int m_live,
                                          const float* best, const int* best_i, const int* rows, int n_m,
                                          int part, int n_parts, int n_ctas, bool ok, uint32_t bar_group,
                                          volatile int* s_abort, int* s_last, int tid, int* scratch) {
  float* pv = ws_ptr<float>(a.ws, L.lm_val);
  int* pi = ws_ptr<int>(a.ws, L.lm_idx);
#pragma unroll
  for (int m = 0; m < 4; ++m) {
    if (m < n_m && rows[m] < m_live) {
      pv[(size_t)rows[m] * n_parts + part] = best[m];
      pi[(size_t)rows[m] * n_parts + part] = best_i[m];
    }
  }
  __threadfence();
  unsigned group_phase = 0;
  auto group_sync = [&]() -> bool {                   // bounded barrier of the 128 epilogue threads
    mbar_arrive(bar_group);
    const bool r = mbar_wait(bar_group, group_phase & 1, s_abort);
    ++group_phase;
    return r;
  };
  ok = ok && group_sync();
  if (ok && tid == 0) *s_last = (atomicAdd(&hdr[H_LM_TICKET], 1) == n_ctas - 1);
  ok = ok && group_sync();
  if (!(ok && *s_last)) return;
  __threadfence();
  if (tid == 0) hdr[H_LM_TICKET] = 0;                 // ready for the next launch
  int* top1 = ws_ptr<int>(a.ws, L.top1);
  const int m_bs = kHalfW * a.n_bs;
  const int* wtok = ws_ptr<int>(a.ws, L.tokens);
  int* s_top1 = scratch;                              // the operand ring is idle by now
  int* s_tok = scratch + m_bs;
  for (int r = tid; r < m_bs; r += kEpiThreads) {
    int bi = 0;
    if (r < m_live) {
      float bv = -INFINITY;
      bi = INT_MAX;
      for (int cc = 0; cc < n_parts; ++cc) {
        const float v = __ldcg(&pv[(size_t)r * n_parts + cc]);
        const int i2 = __ldcg(&pi[(size_t)r * n_parts + cc]);
        if (v > bv || (v == bv && i2 < bi)) { bv = v; bi = i2; }
      }
      if (bi == INT_MAX) bi = 0;
      if (a.row_max) a.row_max[r] = bv;
    }
    top1[r] = bi;
    s_top1[r] = bi;
    s_tok[r] = wtok[r];
  }
  ok = group_sync();
  const int N = hdr[H_N_LIVE];
  const int* wk = ws_ptr<int>(a.ws, L.k);
  const int* woff = ws_ptr<int>(a.ws, L.offset);
  if (ok && tid < a.n_bs) {
    const int i = tid;
    int32_t* ot = a.out_tokens + i * kW;
    if (i < N) {
      // a chain of dependent reads: on the shared-memory copies, not on global memory
      const int ki = wk[i], oi = woff[i];
      int acc = 0;
      while (acc < ki - 1 && s_top1[oi + acc] == s_tok[oi + acc + 1]) ++acc;
      const int nxt = s_top1[oi + acc];
      for (int j = 0; j < kW; ++j) ot[j] = j < acc ? s_tok[oi + 1 + j] : (j == acc ? nxt : -1);
      a.accept_len[i] = acc;
      a.next_anchor[i] = nxt;
      a.out_len[i] = acc + 1;
      if (a.ctx_len_inout) a.ctx_len_inout[i] += acc + 1;
    } else {
      for (int j = 0; j < kW; ++j) ot[j] = -1;
      a.accept_len[i] = 0;
      a.next_anchor[i] = -1;
      a.out_len[i] = 0;
    }
  }
}

// Everything the two single-thread issue loops touch per k step is kept in
// registers and advanced incrementally (ring slot, phase, descriptor words): a
// lone thread retires a dependent instruction every few cycles, so an integer
// division or a descriptor rebuilt from scratch in those loops costs more than
// the MMAs they issue.
template <int M_TILES>
__global__ void __launch_bounds__(kThreads, 1)
lm_head_kernel(LmArgs a, WsLayout L, LmShape sh, const __grid_constant__ CUtensorMap tm_a,
               const __grid_constant__ CUtensorMap tm_b) {
  extern __shared__ unsigned char smem_dyn[];
  const uint32_t raw = smem_u32(smem_dyn);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* sm = smem_dyn + (base - raw);
  const int off_bar = sh.stages * sh.stage_bytes;
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(sm + off_bar + 256);
  volatile int* s_abort = reinterpret_cast<volatile int*>(sm + off_bar + 260);
  int* s_last = reinterpret_cast<int*>(sm + off_bar + 264);
  const uint32_t bar0 = base + off_bar;
  auto bar = [&](int b) { return bar0 + 8u * b; };
  const int B_FULL = 0, B_EMPTY = sh.stages, B_ACC_FULL = 2 * sh.stages, B_ACC_EMPTY = B_ACC_FULL + 1,
            B_GROUP = B_ACC_FULL + 2, B_DRAIN = B_ACC_FULL + 3;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int c = blockIdx.x, C = gridDim.x;
  int* hdr = ws_ptr<int>(a.ws, L.hdr);
  const int m_live = hdr[H_M_LIVE];

  if (tid == 0) {
    for (int s = 0; s < sh.stages; ++s) { mbar_init(bar(B_FULL + s), 1); mbar_init(bar(B_EMPTY + s), 1); }
    mbar_init(bar(B_ACC_FULL), 1);
    mbar_init(bar(B_ACC_EMPTY), kEpiThreads);
    mbar_init(bar(B_GROUP), kEpiThreads);
    mbar_init(bar(B_DRAIN), 1);
    s_abort[0] = 0; s_abort[2] = 0; s_abort[3] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 5) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;"
                 ::"r"(smem_u32(s_tmem)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (warp == 4 && lane == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_a) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_b) : "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *s_tmem;

  const int col_begin = c * sh.cols_per_cta;
  int my_tiles = 0;
  for (int t = 0; t < sh.tiles_per_cta; ++t) my_tiles += (col_begin + t * sh.n_tile < a.vocab);
  const int k_steps = a.hidden_dim / kKStep;

  if (warp == 4) {
    // ===================================================== TMA producer
    // lane m < M_TILES copies hidden box m, lane M_TILES the weight box: the
    // copies of a k step are issued by one warp instruction
    const bool is_a = lane < M_TILES, is_b = lane == M_TILES;
    const CUtensorMap* map = is_a ? &tm_a : &tm_b;
    const uint32_t dst_off = (is_a ? lane : M_TILES) * kATile;
    const uint32_t tx_bytes = M_TILES * (uint32_t)sh.a_rows * kKStep * 2 + (uint32_t)sh.n_tile * kKStep * 2;
    int slot = 0, issued = 0;
    uint32_t empty_parity = 1, st = base;
    bool ok = true;
    for (int t = 0; t < my_tiles && ok; ++t) {
      const int c1 = is_a ? lane * 128 : col_begin + t * sh.n_tile;
      for (int kb = 0; kb < k_steps; ++kb) {
        ok = mbar_wait(bar(B_EMPTY + slot), empty_parity, s_abort);
        if (!ok) break;
        if (lane == 0) mbar_expect_tx(bar(B_FULL + slot), tx_bytes);
        __syncwarp();
#ifdef DSCALE_WAIT_TEST
        // wait-limit test build only: the weight box of one k step of one CTA is left out (the
        // barrier stays armed), so that every wait behind it runs into its limit
        const bool drop = is_b && c == g_lm_drop_cta && issued == g_lm_drop_step;
#else
        constexpr bool drop = false;
#endif
        if ((is_a || is_b) && !drop) tma_load_2d(st + dst_off, map, bar(B_FULL + slot), kb * kKStep, c1);
        ++issued;
        st += sh.stage_bytes;
        if (++slot == sh.stages) { slot = 0; empty_parity ^= 1; st = base; }
      }
    }
    if (!ok) {
      // a wait ran out: before shared memory is given back, wait (bounded, on a flag of its own) for
      // the copies of the last ring's worth of k steps, each on the phase it was armed for
      for (int back = 1; back <= sh.stages && back <= issued; ++back) {
        const int it = issued - back;
        mbar_wait(bar(B_FULL + it % sh.stages), (uint32_t)(it / sh.stages) & 1u, s_abort + 2);
      }
    }
    __syncwarp();
  } else if (warp == 5) {
    // ===================================================== MMA issuer
    if (lane == 0) {
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(sh.n_tile >> 3) << 17) |
                             ((128u >> 4) << 24);
      const uint64_t desc_hi = smem_desc(0, 16, 1024);          // everything but the start address
      const uint32_t stage_step = (uint32_t)sh.stage_bytes >> 4;
      int slot = 0;
      uint32_t full_parity = 0, st_lo = base >> 4;
      bool ok = true;
      for (int t = 0; t < my_tiles && ok; ++t) {
        ok = mbar_wait(bar(B_ACC_EMPTY), (t & 1) ^ 1, s_abort);        // accumulators drained
        if (!ok) break;
        tc_fence_after();
        for (int kb = 0; kb < k_steps; ++kb) {
          ok = mbar_wait(bar(B_FULL + slot), full_parity, s_abort);
          if (!ok) break;
          tc_fence_after();
          const uint32_t b_lo = st_lo + M_TILES * (kATile >> 4);
#pragma unroll
          for (int ks = 0; ks < kKStep / 16; ++ks) {
#pragma unroll
            for (int m = 0; m < M_TILES; ++m)
              umma(tmem + m * sh.n_tile, desc_hi | (uint64_t)(st_lo + m * (kATile >> 4) + ks * 2),
                   desc_hi | (uint64_t)(b_lo + ks * 2), idesc, (kb | ks) != 0);
          }
          umma_commit(bar(B_EMPTY + slot));
          st_lo += stage_step;
          if (++slot == sh.stages) { slot = 0; full_parity ^= 1; st_lo = base >> 4; }
        }
        if (ok) umma_commit(bar(B_ACC_FULL));
      }
      if (!ok) {
        // a wait ran out: the products issued so far must have finished before tensor memory is released
        umma_commit(bar(B_DRAIN));
        mbar_wait(bar(B_DRAIN), 0, s_abort + 3);
      }
    }
    __syncwarp();
  } else {
    // ===================================================== epilogue warps 0-3
    const uint32_t t_lane = tmem + ((uint32_t)(warp * 32) << 16);
    float best[4];
    int best_i[4];
    int rows[4];
#pragma unroll
    for (int m = 0; m < 4; ++m) { best[m] = -INFINITY; best_i[m] = INT_MAX; rows[m] = m * 128 + tid; }
    bool ok = true;
    for (int t = 0; t < my_tiles && ok; ++t) {
      ok = mbar_wait(bar(B_ACC_FULL), t & 1, s_abort);
      if (!ok) break;
      tc_fence_after();
      const int col0 = col_begin + t * sh.n_tile;
#pragma unroll
      for (int m = 0; m < M_TILES; ++m)
        scan_acc(t_lane + m * sh.n_tile, sh.n_tile, col0, a.vocab, rows[m] < m_live, best[m], best_i[m]);
      tc_fence_before();
      mbar_arrive(bar(B_ACC_EMPTY));
    }
    lm_finish(a, L, hdr, m_live, best, best_i, rows, M_TILES, c, C, C, ok, bar(B_GROUP), s_abort, s_last, tid,
              reinterpret_cast<int*>(sm));
  }

  tc_fence_before();
  __syncthreads();
  if (tid == 0 && *s_abort) atomicOr(&hdr[H_STATUS], 8 /*TIMEOUT*/);
  if (warp == 5) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
  }
}

// ---------------------------------------------------------------------------
// CTA-pair variant for more than 128 packed rows (cta_group::2).
//
// With one CTA per tile the 256 x 4096 hidden block is re-read from L2 for every
// 208 vocabulary columns and takes more than half of the shared-memory ring, so
// the weight bytes in flight per SM -- what bounds a stream at HBM latency --
// are few.  A pair of CTAs on neighbouring SMs issues M = 256 MMAs instead: each
// CTA stages only ITS 128 hidden rows and HALF of every weight tile, the tensor
// cores read the other half from the partner's shared memory, and each CTA
// accumulates its 128 rows x N columns in its own TMEM.  Per pass a pair covers
// 256 rows x 2N columns (rows <= 256) or 512 rows x N columns.
//   both CTAs   warp 4: TMA producer into the own ring; the transaction bytes of
//               both CTAs complete on the LEADER's full barrier.
//               warps 0-3: epilogue over the own 128 rows per row block.
//   leader      warp 5: issues the MMAs; tcgen05.commit arrives on the empty /
//               accumulator-full barriers of both CTAs.
// Every wait is bounded; the two CTAs meet at a cluster barrier before the
// tensor memory is released.
struct PairShape {
  int m_pairs;        // row blocks of 256 packed rows (1 or 2)
  int n_acc;          // accumulators per row block (2 or 1): m_pairs * n_acc = 2
  int n;              // N of one MMA (multiple of 16, <= 256); each CTA stages n / 2 weight rows
  int passes;
  int cols_per_pair;  // n * n_acc * passes
  int stages;
  int stage_bytes;
  int b_bytes;        // one staged half weight tile
  int smem_bytes;
};

__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA load into the own shared memory whose bytes complete on a barrier that may
// live in the partner CTA (cluster address)
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* map, uint32_t bar_cluster,
                                                 int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar_cluster), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void umma_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void umma_commit_pair(uint32_t bar_cluster) {
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];"
               ::"r"(bar_cluster) : "memory");
}

template <int M_PAIRS>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads, 1)
lm_head_pair_kernel(LmArgs a, WsLayout L, PairShape sh, const __grid_constant__ CUtensorMap tm_a,
                    const __grid_constant__ CUtensorMap tm_b) {
  constexpr int N_ACC = 2 / M_PAIRS;
  extern __shared__ unsigned char smem_dyn[];
  const uint32_t raw = smem_u32(smem_dyn);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* sm = smem_dyn + (base - raw);
  const int off_bar = sh.stages * sh.stage_bytes;
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(sm + off_bar + 256);
  volatile int* s_abort = reinterpret_cast<volatile int*>(sm + off_bar + 260);
  int* s_last = reinterpret_cast<int*>(sm + off_bar + 264);
  const uint32_t bar0 = base + off_bar;
  auto bar = [&](int b) { return bar0 + 8u * b; };
  const int B_FULL = 0, B_EMPTY = sh.stages, B_ACC_FULL = 2 * sh.stages, B_ACC_EMPTY = B_ACC_FULL + 1,
            B_GROUP = B_ACC_FULL + 2, B_DRAIN = B_ACC_FULL + 3;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const uint32_t rank = cluster_rank();              // 0 = leader (issues the MMAs)
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  int* hdr = ws_ptr<int>(a.ws, L.hdr);
  const int m_live = hdr[H_M_LIVE];

  if (tid == 0) {
    for (int s = 0; s < sh.stages; ++s) { mbar_init(bar(B_FULL + s), 1); mbar_init(bar(B_EMPTY + s), 1); }
    mbar_init(bar(B_ACC_FULL), 1);
    mbar_init(bar(B_ACC_EMPTY), 2 * kEpiThreads);    // the epilogue threads of both CTAs
    mbar_init(bar(B_GROUP), kEpiThreads);
    mbar_init(bar(B_DRAIN), 1);
    s_abort[0] = 0; s_abort[2] = 0; s_abort[3] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 5) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], 512;"
                 ::"r"(smem_u32(s_tmem)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  if (warp == 4 && lane == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_a) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_b) : "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                                 // the partner's barriers exist before anything signals them
  tc_fence_after();
  const uint32_t tmem = *s_tmem;

  const int col_begin = pair * sh.cols_per_pair;
  const int pass_cols = sh.n * N_ACC;
  int my_passes = 0;
  for (int t = 0; t < sh.passes; ++t) my_passes += (col_begin + t * pass_cols < a.vocab);
  const int k_steps = a.hidden_dim / kKStep;
  const int half = sh.n >> 1;

  if (warp == 4) {
    // ===================================================== TMA producer (both CTAs)
    // lane p < M_PAIRS copies this CTA's 128 hidden rows of row block p, lane
    // M_PAIRS + j its half of the weight tile of accumulator j
    const bool is_a = lane < M_PAIRS, is_b = lane >= M_PAIRS && lane < M_PAIRS + N_ACC;
    const int j = lane - M_PAIRS;
    const CUtensorMap* map = is_a ? &tm_a : &tm_b;
    const uint32_t dst_off = is_a ? lane * kATile : M_PAIRS * kATile + j * sh.b_bytes;
    const uint32_t payload = (uint32_t)M_PAIRS * kATile + (uint32_t)N_ACC * half * kKStep * 2;
    const uint32_t full0 = map_to_cta(bar(B_FULL), 0);           // the leader's full barriers
    int slot = 0, issued = 0;
    uint32_t empty_parity = 1, st = base;
    bool ok = true;
    for (int t = 0; t < my_passes && ok; ++t) {
      const int c1 = is_a ? lane * 256 + (int)rank * 128 : col_begin + t * pass_cols + j * sh.n + (int)rank * half;
      for (int kb = 0; kb < k_steps; ++kb) {
        ok = mbar_wait(bar(B_EMPTY + slot), empty_parity, s_abort);
        if (!ok) break;
        if (lane == 0 && rank == 0) mbar_expect_tx(bar(B_FULL + slot), 2 * payload);
        __syncwarp();
        if (is_a || is_b) tma_load_2d_pair(st + dst_off, map, full0 + 8u * slot, kb * kKStep, c1);
        ++issued;
        st += sh.stage_bytes;
        if (++slot == sh.stages) { slot = 0; empty_parity ^= 1; st = base; }
      }
    }
    if (!ok && rank == 0) {
      // a wait ran out: the full barriers live in this CTA and count the bytes of both CTAs, so the
      // leader waits (bounded, on a flag of its own) for the last ring's worth of k steps it armed;
      // the peer stays in the cluster barrier at the end until the leader is through
      for (int back = 1; back <= sh.stages && back <= issued; ++back) {
        const int it = issued - back;
        mbar_wait(bar(B_FULL + it % sh.stages), (uint32_t)(it / sh.stages) & 1u, s_abort + 2);
      }
    }
    __syncwarp();
  } else if (warp == 5) {
    // ===================================================== MMA issuer (leader only)
    if (lane == 0 && rank == 0) {
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(sh.n >> 3) << 17) |
                             ((256u >> 4) << 24);
      const uint64_t desc_hi = smem_desc(0, 16, 1024);
      const uint32_t stage_step = (uint32_t)sh.stage_bytes >> 4, b_step = (uint32_t)sh.b_bytes >> 4;
      const uint32_t peer_bar0 = map_to_cta(bar0, 1);
      int slot = 0;
      uint32_t full_parity = 0, st_lo = base >> 4;
      bool ok = true;
      for (int t = 0; t < my_passes && ok; ++t) {
        ok = mbar_wait(bar(B_ACC_EMPTY), (t & 1) ^ 1, s_abort);        // both CTAs drained their accumulators
        if (!ok) break;
        tc_fence_after();
        for (int kb = 0; kb < k_steps; ++kb) {
          ok = mbar_wait(bar(B_FULL + slot), full_parity, s_abort);
          if (!ok) break;
          tc_fence_after();
          const uint32_t b_lo = st_lo + M_PAIRS * (kATile >> 4);
#pragma unroll
          for (int ks = 0; ks < kKStep / 16; ++ks) {
#pragma unroll
            for (int p = 0; p < M_PAIRS; ++p) {
#pragma unroll
              for (int j = 0; j < N_ACC; ++j)
                umma_pair(tmem + (p * N_ACC + j) * sh.n, desc_hi | (uint64_t)(st_lo + p * (kATile >> 4) + ks * 2),
                          desc_hi | (uint64_t)(b_lo + j * b_step + ks * 2), idesc, (kb | ks) != 0);
            }
          }
          umma_commit_pair(bar(B_EMPTY + slot));
          umma_commit_pair(peer_bar0 + 8u * (B_EMPTY + slot));
          st_lo += stage_step;
          if (++slot == sh.stages) { slot = 0; full_parity ^= 1; st_lo = base >> 4; }
        }
        if (ok) {
          umma_commit_pair(bar(B_ACC_FULL));
          umma_commit_pair(peer_bar0 + 8u * B_ACC_FULL);
        }
      }
      if (!ok) {
        // a wait ran out: the products issued so far (they write both CTAs' tensor memory) must have
        // finished before either CTA releases it; both stay in the cluster barrier until then
        umma_commit_pair(bar(B_DRAIN));
        mbar_wait(bar(B_DRAIN), 0, s_abort + 3);
      }
    }
    __syncwarp();
  } else {
    // ===================================================== epilogue warps 0-3 (both CTAs)
    const uint32_t t_lane = tmem + ((uint32_t)(warp * 32) << 16);
    const uint32_t acc_empty = map_to_cta(bar(B_ACC_EMPTY), 0);
    float best[4];
    int best_i[4];
    int rows[4];
#pragma unroll
    for (int m = 0; m < 4; ++m) { best[m] = -INFINITY; best_i[m] = INT_MAX; rows[m] = m * 256 + (int)rank * 128 + tid; }
    bool ok = true;
    for (int t = 0; t < my_passes && ok; ++t) {
      ok = mbar_wait(bar(B_ACC_FULL), t & 1, s_abort);
      if (!ok) break;
      tc_fence_after();
      const int col0 = col_begin + t * pass_cols;
#pragma unroll
      for (int p = 0; p < M_PAIRS; ++p) {
#pragma unroll
        for (int j = 0; j < N_ACC; ++j)
          scan_acc(t_lane + (p * N_ACC + j) * sh.n, sh.n, col0 + j * sh.n, a.vocab, rows[p] < m_live, best[p],
                   best_i[p]);
      }
      tc_fence_before();
      mbar_arrive_cluster(acc_empty);
    }
    lm_finish(a, L, hdr, m_live, best, best_i, rows, M_PAIRS, pair, n_pairs, (int)gridDim.x, ok,
              bar(B_GROUP), s_abort, s_last, tid, reinterpret_cast<int*>(sm));
  }

  tc_fence_before();
  __syncthreads();
  if (tid == 0 && *s_abort) atomicOr(&hdr[H_STATUS], 8 /*TIMEOUT*/);
  cluster_sync_all();                                 // nobody leaves while the partner may still touch this CTA
  if (warp == 5) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
  }
}

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
bool encode_2d(CUtensorMap* out, const void* ptr, int inner, int rows, int box_rows,
               CUtensorMapL2promotion promo) {
  EncodeTiledFn enc = get_encode();
  if (!enc) return false;
  cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)inner * 2};
  cuuint32_t box[2] = {(cuuint32_t)kKStep, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, promo,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

LmShape plan(int n_bs, int vocab, int num_ctas) {
  LmShape s;
  const int rows = kHalfW * n_bs;
  s.m_tiles = (rows + 127) / 128;
  s.a_rows = rows < 128 ? rows : 128;
  int cols = (vocab + num_ctas - 1) / num_ctas;
  cols = (cols + 15) & ~15;
  int n_max = (512 / s.m_tiles) & ~15;
  if (n_max > 256) n_max = 256;
  s.tiles_per_cta = (cols + n_max - 1) / n_max;
  s.n_tile = (((cols + s.tiles_per_cta - 1) / s.tiles_per_cta) + 15) & ~15;
  if (s.n_tile > ((vocab + 15) & ~15)) s.n_tile = (vocab + 15) & ~15;
  s.cols_per_cta = s.n_tile * s.tiles_per_cta;
  s.b_bytes = (s.n_tile * kKStep * 2 + 1023) & ~1023;
  s.stage_bytes = s.m_tiles * kATile + s.b_bytes;
  s.stages = (200 * 1024) / s.stage_bytes;
  if (s.stages > 8) s.stages = 8;
  s.smem_bytes = s.stages * s.stage_bytes + 512 + 1024;
  return s;
}

PairShape plan_pair(int n_bs, int vocab, int pairs) {
  PairShape s;
  const int rows = kHalfW * n_bs;
  s.m_pairs = (rows + 255) / 256;
  s.n_acc = 2 / s.m_pairs;
  int cols = (vocab + pairs - 1) / pairs;
  const int per_pass_max = 256 * s.n_acc;
  s.passes = (cols + per_pass_max - 1) / per_pass_max;
  const int per_acc = (cols + s.passes * s.n_acc - 1) / (s.passes * s.n_acc);
  s.n = (per_acc + 15) & ~15;
  if (s.n < 32) s.n = 32;
  s.cols_per_pair = s.n * s.n_acc * s.passes;
  s.b_bytes = (s.n / 2) * kKStep * 2;                 // n / 2 rows of 128 bytes: a multiple of 1024
  s.stage_bytes = s.m_pairs * kATile + s.n_acc * s.b_bytes;
  s.stages = (222 * 1024) / s.stage_bytes;
  if (s.stages > 4) s.stages = 4;                     // measured: a fifth stage does not pay
  s.smem_bytes = s.stages * s.stage_bytes + 512 + 1024;
  return s;
}

// CTA pairs that can be resident at once with the ring at its largest (one CTA
// per SM either way); a grid beyond it would run a second, nearly empty wave.
int resident_pairs(int num_ctas) {
  // The answer depends on the device (SM count, shared memory), not on the grid asked
  // about, so it is kept per device; a failed query is not kept.
  static std::mutex mu;
  static int cached[64];
  static bool have[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 0;
  std::lock_guard<std::mutex> lk(mu);
  if (!have[dev]) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2);
    cfg.blockDim = dim3(kThreads);
    cfg.dynamicSmemBytes = 224 * 1024;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeClusterDimension;
    at[0].val.clusterDim.x = 2; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
    cfg.attrs = at; cfg.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, lm_head_pair_kernel<1>, &cfg) != cudaSuccess) { cudaGetLastError(); return 0; }
    cached[dev] = n;
    have[dev] = true;
  }
  const int want = num_ctas / 2;
  return cached[dev] < want ? cached[dev] : want;
}

}  // namespace

cudaError_t lm_head_prepare() {
  const void* fns[] = {(const void*)lm_head_kernel<1>,
                       (const void*)lm_head_pair_kernel<1>, (const void*)lm_head_pair_kernel<2>};
  for (const void* f : fns) {
    cudaError_t e = cudaFuncSetAttribute(f, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (e != cudaSuccess) return e;
  }
  return cudaSuccess;
}

cudaError_t launch_lm_head(void* ws, int n_bs, const void* hidden, const void* weight, int hidden_dim,
                           int vocab, int32_t* accept_len, int32_t* next_anchor, int32_t* out_tokens,
                           int32_t* out_len, int32_t* ctx_len_inout, float* row_max, int n_kv_heads,
                           int num_ctas, cudaStream_t stream) {
  WsLayout L = ws_layout(n_bs, n_kv_heads, num_ctas);
  LmArgs a{ws, n_bs, hidden_dim, vocab, accept_len, next_anchor, out_tokens, out_len, ctx_len_inout, row_max};
  CUtensorMap ta, tb;
  const int pairs = kHalfW * n_bs > 128 ? resident_pairs(num_ctas) : 0;
  if (pairs >= 1) {
    // more than one row tile: CTA pairs
    PairShape ps = plan_pair(n_bs, vocab, pairs);
    if (ps.stages < 2) return cudaErrorNotSupported;
    const int b_box = ps.n / 2 < vocab ? ps.n / 2 : vocab;
    if (!encode_2d(&ta, hidden, hidden_dim, kHalfW * n_bs, 128, CU_TENSOR_MAP_L2_PROMOTION_L2_128B) ||
        !encode_2d(&tb, weight, hidden_dim, vocab, b_box, CU_TENSOR_MAP_L2_PROMOTION_L2_256B))
      return cudaErrorNotSupported;
    if (ps.m_pairs == 1) lm_head_pair_kernel<1><<<pairs * 2, kThreads, ps.smem_bytes, stream>>>(a, L, ps, ta, tb);
    else lm_head_pair_kernel<2><<<pairs * 2, kThreads, ps.smem_bytes, stream>>>(a, L, ps, ta, tb);
    return cudaGetLastError();
  }
  LmShape sh = plan(n_bs, vocab, num_ctas);
  if (sh.stages < 2 || sh.n_tile < 16) return cudaErrorNotSupported;
  if (!encode_2d(&ta, hidden, hidden_dim, kHalfW * n_bs, sh.a_rows, CU_TENSOR_MAP_L2_PROMOTION_L2_128B) ||
      !encode_2d(&tb, weight, hidden_dim, vocab, sh.n_tile < vocab ? sh.n_tile : vocab,
                 CU_TENSOR_MAP_L2_PROMOTION_L2_256B))
    return cudaErrorNotSupported;
  if (sh.m_tiles != 1) return cudaErrorNotSupported;    // more than 128 rows need a resident CTA pair
  lm_head_kernel<1><<<num_ctas, kThreads, sh.smem_bytes, stream>>>(a, L, sh, ta, tb);
  return cudaGetLastError();
}

#ifdef DSCALE_WAIT_TEST
// Wait-limit test build only: leave out the weight copy of k step `step` (counted from the CTA's
// first) of CTA `cta` of the one-CTA-per-tile LM-head kernel in every following launch; (-1, -1)
// switches it off.  HOST call.
extern "C" int dscale_test_drop_lm_copy(int cta, int step) {
  if (cudaMemcpyToSymbol(g_lm_drop_cta, &cta, sizeof(int)) != cudaSuccess) return -3;
  if (cudaMemcpyToSymbol(g_lm_drop_step, &step, sizeof(int)) != cudaSuccess) return -3;
  return 0;
}
#endif

}  // namespace dscale
