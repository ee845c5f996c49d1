// Packed ragged verify attention on the sm_100a tensor cores.
//
// Shape of the work.  Per live request i and kv-head g the query tile is the
// GQA group's 4 q-heads x the k_i <= 16 live window rows = at most 64 rows:
// exactly one M = 64 tcgen05 tile (row m = 16 h_local + j), instead of the
// 128-row prefill tile that would leave 112 masked rows per request and head
// (Eq. 2).  Keys and values are streamed once per kv-head in tiles of 128
// tokens (8 pages).  The kernel is HBM-bound; the tensor cores only have to
// keep up with the K/V stream.
//
// Schedule.  The key tiles of all (request, kv-head) pairs form one linear
// list (the per-request tile prefix comes from the allocation kernel); CTA c
// of a persistent grid of one CTA per SM takes the contiguous slice
// [c T / C, (c+1) T / C).  A slice cuts at most its first and its last pair;
// those produce an un-normalised partial (O, m, l).  Partials are published with
// a fence and a ticket on a per-pair counter, and the last CTA to reach a pair
// merges it and writes its rows -- nobody waits for another CTA.  The partial of
// a slice's first run is published in the background by a helper warp; the CTA
// that ends its slice inside a pair normally finds the other partials already
// published, has them copied into shared memory behind its last tiles and
// finishes the pair without a global round trip.  Pairs inside a slice are
// written directly.
// The grid and every address are independent of the lengths, so a captured
// launch replays at any mix of lengths.
//
// Pipeline inside a CTA (32 (10 + kProducers) threads):
//   warps 8..  producers (kProducers warps, each copying its share of every tile's pages):
//              per tile, 16 TMA box copies of K (a 64-column half of one
//              16-token page each, 2 KB) and 8 of V (a whole page-head, 4 KB), 128-byte
//              swizzle, into a 5-deep ring of 32 KB slots; page ids are fetched two
//              tiles ahead.  Both the copy engine and the single MMA-issuing thread pay
//              about 100 SM cycles per instruction whatever its size, and once the SM
//              clock drops under the power cap either count can bound the stream:
//              24 copies and 16 products per tile keep both below the memory time
//              (32 + 16 made the copies the bound, 16 + 24 the products).
//   next warp  issues tcgen05.mma (one lane; the warp's loop is warp-uniform): S = Q K^T (M64 N128 K128, bf16 in,
//              fp32 in TMEM) for tile t, then O_t = P_{t-1} V_{t-1}; completion
//              is signalled with tcgen05.commit on mbarriers.
//   warps 0-7  softmax.  Tile rows are head-major (m = 16 h_local + j), so q-head
//              h_local sits in TMEM lanes 32 h_local .. 32 h_local + 15, which
//              warps h_local and h_local + 4 may read.  Warp h_local takes window
//              rows j = 0..7, warp h_local + 4 rows j = 8..15: a thread owns one
//              row together with the three other threads of its quad
//              (tcgen05.ld.16x256b), and a request with k_i <= 8 leaves the
//              second group of warps idle.  They keep the running max / sum and
//              write P as bf16 into swizzled shared memory for the second MMA.  O stays in
//              TMEM for a whole run of tiles (the second MMA accumulates onto
//              it); it is only rescaled in place when a row maximum outgrows its
//              reference by 2^8, and read back once per run for the epilogue.
//   last warp  publisher: fence + ticket for the first run's partial.
// S is triple-buffered in TMEM (3 x 128 columns) next to O (128 columns), P and
// Q are double-buffered in shared memory; the MMA thread issues whichever of the
// two products is ready, scores up to two tiles ahead of the softmax.
//
// Every wait is bounded: when a wait runs out the CTA sets the TIMEOUT status
// bit, stops issuing work, drains its outstanding copies and releases TMEM.
#include <cuda.h>
#include <cuda_bf16.h>

#include <map>
#include <mutex>

#include "kernels.cuh"
#include "tc_ptx.cuh"
#include "tile_schedule.cuh"

namespace dscale {

#ifdef DSCALE_WAIT_TEST
__device__ int g_drop_cta = -1, g_drop_tile = -1;
#endif

namespace {

#ifndef DSCALE_PRODUCERS
#define DSCALE_PRODUCERS 2
#endif
constexpr int kProducers = DSCALE_PRODUCERS;            // copy-issuing warps (a power of two, at most 8)
constexpr int kPagesPerProducer = (kTileTok / kPage) / kProducers;
constexpr int kSoftmaxThreads = 256;
constexpr int kWarpProducer = 8, kWarpMma = 8 + kProducers, kWarpPublisher = 9 + kProducers;
constexpr int kThreads = 32 * (10 + kProducers);
constexpr int kStages = 5;
constexpr int kSlotBytes = kTileTok * kD * 2;           // 32 KB: one K or V tile
constexpr int kHalfSlot = kSlotBytes / 2;               // K tile: one 64-column half [128 tok][128 B]
constexpr int kPageBytes = kPage * kD * 2;              // V tile: 4 KB per page-head = one TMA box
constexpr int kPageHalf = kPageBytes / 2;               // a page's 64-column half [16 tok][128 B]
constexpr int kQBytes = kTcRows * kD * 2;               // 16 KB
constexpr int kPBytes = kTcRows * kTileTok * 2;         // 16 KB

// shared memory map (offsets from a 1024-byte aligned base)
constexpr int kOffQ = 0;                                 // 2 x 16 KB
constexpr int kOffP = kOffQ + 2 * kQBytes;               // 2 x 16 KB
constexpr int kOffKV = kOffP + 2 * kPBytes;              // 5 x 32 KB
constexpr int kOffBar = kOffKV + kStages * kSlotBytes;   // mbarriers
constexpr int kNumBars = 2 * kStages + 2 + 2 + 3 + 2 + 2 + 6;
constexpr int kOffMisc = kOffBar + 8 * 32;               // tmem base, abort flag, tickets
constexpr int kOffTile = kOffMisc + 64;                  // tile prefix, kMaxNbs + 1 ints
constexpr int kOffSlice = kOffTile + (kMaxNbs + 1) * 4 + 12;   // slice starts, up to kMaxCtas + 1 ints
constexpr int kMaxCtas = 255;
constexpr int kSmemUse = kOffSlice + (kMaxCtas + 1) * 4;
constexpr int kSmemBytes = kSmemUse + 1024;              // slack for base alignment
static_assert(kNumBars <= 32, "barrier area");
static_assert(kSmemBytes <= 232448, "exceeds the 227 KB shared memory of an sm_100 CTA");

enum Bar { B_KV_FULL = 0, B_KV_EMPTY = kStages, B_Q_FULL = 2 * kStages, B_Q_EMPTY = B_Q_FULL + 2,
           B_S_FULL = B_Q_EMPTY + 2, B_P_FULL = B_S_FULL + 3, B_O_FULL = B_P_FULL + 2,
           B_GROUP = B_O_FULL + 2,   // the 128 softmax threads among themselves
           B_PART = B_GROUP + 1,     // softmax -> publisher: the first run's partial is stored
           B_PUB = B_PART + 1,       // publisher -> softmax: that partial is published
           B_PARTNER = B_PUB + 1,    // producer -> softmax: partner partials landed (or not)
           B_MERGE = B_PARTNER + 1,  // bulk copies of the end-phase merge
           B_DRAIN = B_MERGE + 1 };  // products still in flight when a wait ran out

// instruction descriptor: bf16 x bf16 -> fp32, M = 64, N = 128; B is K-major
// for S = Q K^T and MN-major (tokens are the K dimension) for O = P V
constexpr uint32_t idesc(uint32_t n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | ((n >> 3) << 17) | ((64u >> 4) << 24);
}
constexpr uint32_t kIdescS = idesc(128);
constexpr uint32_t kIdescPV = idesc(128) | (1u << 16);


// How a run's result reaches the output.
//   WHOLE    the run is its whole pair: rows are written directly.
//   PUBLISH  first run of a slice, more runs follow: the partial is stored and a
//            publisher warp publishes it in the background.
//   TAIL     last run of a slice, the pair starts in this slice: the producer
//            checks whether all other contributors are published and, if so,
//            copies their partials into shared memory (fast path).
//   FINAL    last run, any other shape: stored and published after the main loop.
enum RunKind { RUN_WHOLE = 0, RUN_PUBLISH = 1, RUN_TAIL = 2, RUN_FINAL = 3 };
__device__ __forceinline__ int run_kind(const Segment& s, bool more) {
  if (s.t0 == 0 && s.t1 == s.n_tiles) return RUN_WHOLE;
  if (more) return RUN_PUBLISH;                 // only a slice's first run can be partial and not last
  return (s.t0 == 0) ? RUN_TAIL : RUN_FINAL;
}
constexpr int kMaxFastPartners = 3;

// --------------------------------------------------------------------- kernel
__global__ void __launch_bounds__(kThreads, 1)
attn_tc_kernel(AttnArgs a, WsLayout L, const __grid_constant__ CUtensorMap tm_q,
               const __grid_constant__ CUtensorMap tm_k, const __grid_constant__ CUtensorMap tm_v) {
  extern __shared__ unsigned char smem_dyn[];
  const uint32_t raw = smem_u32(smem_dyn);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* sm = smem_dyn + (base - raw);
  volatile int* s_abort = reinterpret_cast<volatile int*>(sm + kOffMisc + 4);
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(sm + kOffMisc);
  int* s_ticket = reinterpret_cast<int*>(sm + kOffMisc + 8);          // two ints
  volatile int* s_fast = reinterpret_cast<volatile int*>(sm + kOffMisc + 20);      // partner partials in smem
  volatile int* s_head_last = reinterpret_cast<volatile int*>(sm + kOffMisc + 24); // publisher took the last ticket
  volatile int* s_dummy = reinterpret_cast<volatile int*>(sm + kOffMisc + 16);
  volatile int* s_lock = reinterpret_cast<volatile int*>(sm + kOffMisc + 32);     // one per q-head: O rescale turn
  int* s_tile = reinterpret_cast<int*>(sm + kOffTile);
  int* s_slice = reinterpret_cast<int*>(sm + kOffSlice);
  auto bar = [&](int b) { return base + kOffBar + 8u * b; };

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int c = blockIdx.x;
  int* hdr = ws_ptr<int>(a.ws, L.hdr);
  const int n_bs = a.n_bs, n_kv = a.n_kv_heads, Hq = a.n_q_heads;

  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) { mbar_init(bar(B_KV_FULL + s), kProducers); mbar_init(bar(B_KV_EMPTY + s), 1); }
    for (int b = 0; b < 2; ++b) {
      mbar_init(bar(B_Q_FULL + b), 1); mbar_init(bar(B_Q_EMPTY + b), 1);
      mbar_init(bar(B_P_FULL + b), kSoftmaxThreads);
      mbar_init(bar(B_O_FULL + b), 1);
    }
    for (int b = 0; b < 3; ++b) mbar_init(bar(B_S_FULL + b), 1);
    mbar_init(bar(B_GROUP), kSoftmaxThreads);
    mbar_init(bar(B_PART), kSoftmaxThreads);
    mbar_init(bar(B_PUB), 1);
    mbar_init(bar(B_PARTNER), 1);
    mbar_init(bar(B_MERGE), 1);
    mbar_init(bar(B_DRAIN), 1);
    *s_abort = 0;
    *s_dummy = 0;
    for (int x = 0; x < 4; ++x) s_lock[x] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == kWarpMma) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;"
                 ::"r"(smem_u32(s_tmem)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (warp == kWarpProducer && lane == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_q) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_k) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_v) : "memory");
  }
  // Programmatic dependent launch.  This kernel may become resident while the
  // preceding kernel of the stream is still finishing on other SMs.  Until
  // griddepcontrol.wait it only touches data that the immediately preceding
  // kernel cannot be writing: the allocation's metadata in the workspace (the
  // allocation kernel never lets its dependents start early), the block table,
  // and K/V pages that lie wholly below the committed context (the cache is
  // append-only).  Q, the window's K/V pages and every write (outputs, split-KV
  // scratch) come after the wait.  The next kernel may start its own preamble
  // as soon as SMs free up.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  for (int x = tid; x <= n_bs; x += kThreads) s_tile[x] = ws_ptr<int>(a.ws, L.tile_prefix)[x];
  for (int x = tid; x <= (int)gridDim.x; x += kThreads) s_slice[x] = ws_ptr<int>(a.ws, L.slice_tab)[x];
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *s_tmem;
  const bool is_producer = warp >= kWarpProducer && warp < kWarpProducer + kProducers;
  if (!is_producer) asm volatile("griddepcontrol.wait;" ::: "memory");   // the producers wait later

  const long long T = (long long)s_tile[n_bs] * n_kv;
  // with fewer tiles than CTAs only the first T CTAs get a (one-tile) slice, so
  // that every CTA in [0, C) has work and the per-pair contributor count is exact
  const int C = (int)min((long long)gridDim.x, T);
  long long sl_begin = c < C ? s_slice[c] : 0;
  long long sl_end = c < C ? s_slice[c + 1] : 0;
  // a slice table that does not belong to this tile prefix (allocation not run on this
  // workspace, or run for another grid) must not be followed
  if (sl_begin < 0 || sl_begin > sl_end || sl_end > T || (c + 1 == C && sl_end != T)) {
    if (tid == 0) atomicOr(&hdr[H_STATUS], 4 /*BAD_LEN*/);
    sl_begin = sl_end = 0;
  }
  auto cta_of = [&](long long Lt) { return cta_of_tab(s_slice, C, Lt); };
  const int* kv_len = ws_ptr<int>(a.ws, L.kv_len);

  if (is_producer) {
    // ===================================================== TMA producer warps
    // The copy engine takes about 50 cycles to accept an instruction from a single warp and
    // then about one cycle per 43 bytes; instructions from several warps overlap the first
    // part.  One warp alone cannot feed more than about 6 TB/s over the chip even from L2,
    // so the boxes of a tile are spread over kProducers warps: warp pw copies pages
    // pw * kPagesPerProducer .. of every K and V tile.  Only the first of them moves Q and
    // the partner partials of the slice's last pair.
    const int pw = warp - kWarpProducer;
    Scheduler sch; sch.init(s_tile, n_bs, n_kv, sl_begin, sl_end);
    Segment sg;
    unsigned u = 0;            // ring sequence number: K of tile it -> 2 it, V -> 2 it + 1
    int seg = 0;
    bool ok = true;
    bool waited = false;       // griddepcontrol.wait done
    // V: lane l < kPagesPerProducer copies one of this warp's pages as one 4 KB box.  K: lanes l
    // and l + kPagesPerProducer copy the two 64-column halves of that page as 2 KB boxes.
    const int pg_l = pw * kPagesPerProducer + (lane & (kPagesPerProducer - 1));
    const int k_half = (lane / kPagesPerProducer) & 1;
    // K/V are read exactly once per launch: mark them evict-first in L2
    const uint64_t kv_policy = make_policy_evict_first();
    while (ok && sch.next(sg)) {
      const int qb = seg & 1;
      const int len = kv_len[sg.i];
      const int* bt = a.block_table + (size_t)sg.i * a.max_pages;
      // Page ids are loaded two tiles ahead and only looked at when their tile is issued: the
      // load's round trip (several hundred cycles while every SM streams) then lies off this
      // warp's path, which the copy instructions themselves already fill.
      auto load_page = [&](int t) -> int {
        const int p = t * (kTileTok / kPage) + pg_l;
        return (lane < 2 * kPagesPerProducer && t < sg.t1 && p * kPage < len) ? __ldg(bt + p) : 0;
      };
      auto checked = [&](int id) -> int {
        if (id < 0 || id >= a.num_pages) { atomicOr(&hdr[H_STATUS], 2); id = 0; }
        return id;
      };
      auto fetch_page = [&](int t) -> int { return checked(load_page(t)); };
      auto issue_tile = [&](int t, int page) -> bool {       // K then V of key tile t into the ring
        const int valid_tok = min(kTileTok, len - t * kTileTok);
        const int n_pages = (valid_tok + kPage - 1) / kPage;
#pragma unroll
        for (int which = 0; which < 2; ++which, ++u) {
          const int slot = u % kStages;
          if (!mbar_wait(bar(B_KV_EMPTY + slot), ((u / kStages) & 1) ^ 1, s_abort)) return false;
          const int mine = min(kPagesPerProducer, max(0, n_pages - pw * kPagesPerProducer));   // pages of this warp
          if (lane == 0) mbar_expect_tx(bar(B_KV_FULL + slot), mine * kPageBytes);
          __syncwarp();
#ifdef DSCALE_WAIT_TEST
          // wait-limit test build only: the copies of one K tile of one CTA are left out (the
          // barrier stays armed), so that every wait behind it runs into its limit
          if (which == 0 && c == g_drop_cta && (int)(u / 2) == g_drop_tile) continue;
#endif
          if (which == 0) {
            if (lane < 2 * kPagesPerProducer && pg_l < n_pages)
              tma_load_5d_hint(base + kOffKV + slot * kSlotBytes + k_half * kHalfSlot + pg_l * kPageHalf,
                               &tm_k, bar(B_KV_FULL + slot), 0, k_half, 0, sg.g, page, kv_policy);
          } else if (lane < kPagesPerProducer && pg_l < n_pages) {
            tma_load_5d_hint(base + kOffKV + slot * kSlotBytes + pg_l * kPageBytes,
                             &tm_v, bar(B_KV_FULL + slot), 0, 0, 0, sg.g, page, kv_policy);
          }
        }
        return true;
      };
      const int row0 = ws_ptr<int>(a.ws, L.offset)[sg.i];      // metadata: safe before the wait
      int t_first = sg.t0;
      if (!waited) {
        // before the grid dependency is resolved: up to two key tiles that lie wholly
        // below the committed context of the first run's request
        const int ctx0 = len - ws_ptr<int>(a.ws, L.k)[sg.i];
        while (ok && t_first < sg.t1 && t_first < sg.t0 + 2 && (t_first + 1) * kTileTok <= ctx0) {
          ok = issue_tile(t_first, fetch_page(t_first));
          ++t_first;
        }
        asm volatile("griddepcontrol.wait;" ::: "memory");
        waited = true;
        if (!ok) break;
      }
      if (pw == 0) ok = mbar_wait(bar(B_Q_EMPTY + qb), ((seg >> 1) & 1) ^ 1, s_abort);
      if (!ok) break;
      if (pw == 0 && lane == 0) {
        mbar_expect_tx(bar(B_Q_FULL + qb), kQBytes);
        tma_load_4d(base + kOffQ + qb * kQBytes, &tm_q, bar(B_Q_FULL + qb), 0, 0, row0, sg.g * 4);
        tma_load_4d(base + kOffQ + qb * kQBytes + kQBytes / 2, &tm_q, bar(B_Q_FULL + qb), 0, 1,
                    row0, sg.g * 4);
      }
      int page_1 = load_page(t_first), page_2 = load_page(t_first + 1);
      for (int t = t_first; t < sg.t1 && ok; ++t) {
        const int page = checked(page_1);
        page_1 = page_2;
        page_2 = load_page(t + 2);
        ok = issue_tile(t, page);
      }
      if (ok && pw == 0 && run_kind(sg, sch.more()) == RUN_TAIL) {
        // The slice ends inside this pair.  If every other contributor has already
        // published its partial (the usual case: they computed theirs at the start
        // of their slices), fetch those partials into ring slots behind the last
        // tiles, so that the softmax warps can finish the pair without a single
        // global round trip.
        const long long p0 = ((long long)s_tile[sg.i] * n_kv) + (long long)sg.g * sg.n_tiles;
        const int c_hi = cta_of(p0 + sg.n_tiles - 1);
        const int others = c_hi - c;                       // this CTA holds the pair's first tiles
        int fast = 0;
        if (others <= kMaxFastPartners) {
          const int seen = ld_acquire_gpu(&ws_ptr<int>(a.ws, L.pair_cnt)[sg.i * n_kv + sg.g]);
          if (seen == others) fast = others;
        }
        if (fast) {
          fence_async_all();
          const float* part_o = ws_ptr<float>(a.ws, L.part_o);
          const float* part_ml = ws_ptr<float>(a.ws, L.part_ml);
          float* s_ml = reinterpret_cast<float*>(sm + kOffQ + ((seg + 1) & 1) * kQBytes);  // unused Q buffer
          for (int x = 0; x < fast && ok; ++x, ++u) {
            const int sid = (c + 1 + x) * 2;               // their run starts their slice: slot 0
            const int slot = u % kStages;
            ok = mbar_wait(bar(B_KV_EMPTY + slot), ((u / kStages) & 1) ^ 1, s_abort);
            if (!ok) break;
            if (lane == 0) {
              mbar_expect_tx_only(bar(B_PARTNER), kTcRows * kD * 4);
              bulk_load(base + kOffKV + slot * kSlotBytes, part_o + (size_t)sid * kTcRows * kD,
                        kTcRows * kD * 4, bar(B_PARTNER));
            }
            reinterpret_cast<float4*>(s_ml + x * kTcRows * 2)[lane] =
                __ldcg(reinterpret_cast<const float4*>(part_ml + (size_t)sid * kTcRows * 2) + lane);
          }
        }
        __syncwarp();
        if (lane == 0) { *s_fast = ok ? fast : 0; mbar_arrive(bar(B_PARTNER)); }
      }
      ++seg;
    }
    if (!waited) asm volatile("griddepcontrol.wait;" ::: "memory");
    // on an aborted run, let the copies already issued land before the CTA's
    // shared memory is released (bounded, like every other wait)
    if (!ok) {
      for (unsigned v = (u > kStages ? u - kStages : 0); v < u; ++v)
        mbar_wait(bar(B_KV_FULL + v % kStages), (v / kStages) & 1, s_dummy);
    }
  } else if (warp == kWarpMma) {
    // ============================================================ MMA issuer
    // Event-driven issue.  S = Q K^T of tile x goes into TMEM buffer x % 3 as soon
    // as its K slot has landed and that buffer's previous tile (x - 3) has been
    // read by the softmax warps; O += P V of tile y as soon as P_y and V_y are
    // there.  Scores may run up to two tiles ahead of the softmax, which frees K
    // slots early and keeps more page copies in flight.
    // The whole warp runs the loop, so that cursors, barrier tests and descriptors are
    // warp-uniform values; only the tcgen05 instructions themselves are issued by one
    // lane.  Ring slots, phases and descriptors advance incrementally (no division, no
    // descriptor rebuilt per instruction).
    {
      const bool leader = lane == 0;
      auto ready = [&](uint32_t b_addr, uint32_t parity) {
        return __all_sync(0xffffffffu, mbar_test(b_addr, parity));
      };
      Scheduler sch; sch.init(s_tile, n_bs, n_kv, sl_begin, sl_end);
      Segment sg;
      const unsigned total = (unsigned)(sl_end - sl_begin);
      unsigned next_s = 0, next_pv = 0;
      int seg = -1, t = 0, t_end = 0;            // S cursor: current run and tile inside it
      bool q_ready = false;
      unsigned run_start_mask = 0;               // bit (x % 4): tile x starts a run
      // ring cursors: K of tile x is ring item 2 x, V is item 2 x + 1; item u sits in slot
      // u % kStages in phase (u / kStages) & 1
      int k_slot = 0, k_phase = 0, v_slot = 1 % kStages, v_phase = (1 / kStages) & 1;
      int s_buf = 0;                             // score buffer next_s % 3
      // descriptors of the operands at their base addresses; a k step adds a constant
      const uint64_t q_desc0 = smem_desc(base + kOffQ, 16, 1024);
      const uint64_t p_desc0 = smem_desc(base + kOffP, 16, 1024);
      const uint64_t k_desc0 = smem_desc(base + kOffKV, 16, 1024);
      const uint64_t v_desc0 = smem_desc(base + kOffKV, kPageHalf, 1024);
      bool ok = true;
      long long t_idle = clock64();
      while (ok && next_pv < total) {
        bool progressed = false;
        // ---- O += P V for the oldest tile whose P is ready
        if (next_pv < next_s) {
          const unsigned pt = next_pv;
          const int b = pt & 1;
          if (ready(bar(B_P_FULL + b), (pt >> 1) & 1) && ready(bar(B_KV_FULL + v_slot), v_phase)) {
            tc_fence_after();
            // A = P [64 rows][128 tok] K-major: 64-token blocks of 8 KB, 32 B per 16 tokens.
            // B = V, MN-major (d contiguous): k step kk = page kk = [2 halves][16 tok][128 B];
            // 2 KB between the two 64-column halves, 1 KB between its two 8-token groups.
            const uint64_t ad = p_desc0 + (uint64_t)(b * (kPBytes >> 4));
            const uint64_t bd = v_desc0 + (uint64_t)(v_slot * (kSlotBytes >> 4));
            const uint32_t fresh = (run_start_mask >> (pt & 3)) & 1;
            if (leader) {
              umma(tmem + 384, ad, bd, kIdescPV, fresh ^ 1u);
#pragma unroll
              for (int kk = 1; kk < kTileTok / 16; ++kk)
                umma_acc(tmem + 384, ad + (uint64_t)((kk >> 2) * ((kTcRows * 128) >> 4) + (kk & 3) * 2),
                         bd + (uint64_t)(kk * (kPageBytes >> 4)), kIdescPV);
              umma_commit(bar(B_O_FULL + b));
              umma_commit(bar(B_KV_EMPTY + v_slot));
            }
            __syncwarp();
            v_slot += 2; if (v_slot >= kStages) { v_slot -= kStages; v_phase ^= 1; }
            ++next_pv;
            progressed = true;
          }
        }
        // ---- S = Q K^T for the next tile, at most two tiles ahead of the P V cursor
        if (next_s < total && next_s <= next_pv + 2) {
          if (t == t_end) {                         // next run
            sch.next(sg);
            ++seg; t = sg.t0; t_end = sg.t1; q_ready = false;
          }
          const int qb = seg & 1;
          if (!q_ready) q_ready = ready(bar(B_Q_FULL + qb), (seg >> 1) & 1);
          if (q_ready && ready(bar(B_KV_FULL + k_slot), k_phase)) {
            tc_fence_after();
            // A = Q [64 rows][128 d], B = K [2 halves][128 tok][128 B], both K-major:
            // 64-column blocks, 32 bytes per k step inside a block, 8-row groups 1 KB apart
            const uint64_t ad = q_desc0 + (uint64_t)(qb * (kQBytes >> 4));
            const uint64_t bd = k_desc0 + (uint64_t)(k_slot * (kSlotBytes >> 4));
            const uint32_t d_s = tmem + s_buf * 128;
            if (leader) {
              umma_new(d_s, ad, bd, kIdescS);
#pragma unroll
              for (int kk = 1; kk < kD / 16; ++kk)
                umma_acc(d_s, ad + (uint64_t)((kk >> 2) * ((kTcRows * 128) >> 4) + (kk & 3) * 2),
                         bd + (uint64_t)((kk >> 2) * (kHalfSlot >> 4) + (kk & 3) * 2), kIdescS);
              umma_commit(bar(B_S_FULL + s_buf));
              umma_commit(bar(B_KV_EMPTY + k_slot));
              if (t + 1 == t_end) umma_commit(bar(B_Q_EMPTY + qb));
            }
            __syncwarp();
            run_start_mask = (run_start_mask & ~(1u << (next_s & 3))) | ((t == sg.t0 ? 1u : 0u) << (next_s & 3));
            k_slot += 2; if (k_slot >= kStages) { k_slot -= kStages; k_phase ^= 1; }
            if (++s_buf == 3) s_buf = 0;
            ++t;
            ++next_s;
            progressed = true;
          }
        }
        if (progressed) {
          t_idle = clock64();
        } else {
          if (*s_abort) ok = false;
          else if (clock64() - t_idle > kWaitCycles) { *s_abort = 1; ok = false; }
        }
      }
      if (!ok) {
        // A wait ran out somewhere in this CTA.  Products issued so far may still be running:
        // tensor memory must not be released under them, so wait (bounded) for their completion.
        if (leader) umma_commit(bar(B_DRAIN));
        __syncwarp();
        mbar_wait(bar(B_DRAIN), 0, s_dummy);
      }
    }
    __syncwarp();
  } else if (warp == kWarpPublisher) {
    // ========================================================= publisher warp
    // Publishes the partial of the slice's first run in the background: waits
    // until the softmax threads have stored it, fences, and takes a ticket on the
    // pair's counter.  The fence and the atomic are global round trips of a few
    // microseconds while the SM streams; here they delay nobody.
    Scheduler sch; sch.init(s_tile, n_bs, n_kv, sl_begin, sl_end);
    Segment sg;
    if (sch.next(sg) && run_kind(sg, sch.more()) == RUN_PUBLISH) {
      if (mbar_wait(bar(B_PART), 0, s_abort)) {
        __threadfence();
        if (lane == 0) {
          const long long p0 = ((long long)s_tile[sg.i] * n_kv) + (long long)sg.g * sg.n_tiles;
          const int n_contrib = cta_of(p0 + sg.n_tiles - 1) - cta_of(p0) + 1;
          int* cnt = &ws_ptr<int>(a.ws, L.pair_cnt)[sg.i * n_kv + sg.g];
          const int old = atomicAdd(cnt, 1);
          *s_head_last = (old == n_contrib - 1);          // then this CTA merges it after its loop
          if (old == n_contrib - 1) *cnt = 0;             // ready for the next launch
          mbar_arrive(bar(B_PUB));
        }
      }
    }
    __syncwarp();
  } else {
    // ====================================================== softmax warps 0-7
    // rows of capacity beyond M_live are written as zero, spread over the grid
    {
      const int m_live = hdr[H_M_LIVE];
      const long long n16 = (long long)(kHalfW * n_bs - m_live) * Hq * (kD * 2 / 16);
      uint4* dst = reinterpret_cast<uint4*>(reinterpret_cast<__nv_bfloat16*>(a.out) +
                                            (size_t)m_live * Hq * kD);
      for (long long x = (long long)c * kSoftmaxThreads + tid; x < n16;
           x += (long long)gridDim.x * kSoftmaxThreads)
        dst[x] = make_uint4(0, 0, 0, 0);
    }
    // Warp w reads the TMEM lanes of q-head wq = w % 4 (tile rows 16 wq .. 16 wq + 15) and
    // works on window rows j = 8 (w / 4) + 0..7 of it.  tcgen05.ld.16x256b hands thread t,
    // for each 8-column group n, the column pair 8 n + 2 (t % 4) + {0, 1} of row t / 4 and
    // of row t / 4 + 8; the thread keeps the pair of its own row.  A row is shared by the
    // 4 threads of a quad.
    const int quad = lane & 3;
    const int wq = warp & 3, half = warp >> 2;
    const int j_row = 8 * half + (lane >> 2);          // window slot of this thread's row
    const int m_row = 16 * wq + j_row;                 // its tile row
    const uint32_t t_lane = tmem + ((uint32_t)(wq * 32) << 16);
    const uint32_t o_addr = t_lane + 384;
    const float scale_log2 = a.sm_scale * 1.4426950408889634f;
    float* part_o = ws_ptr<float>(a.ws, L.part_o);
    float* part_ml = ws_ptr<float>(a.ws, L.part_ml);
    __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(a.out);
    int* pair_cnt = ws_ptr<int>(a.ws, L.pair_cnt);

    Scheduler sch; sch.init(s_tile, n_bs, n_kv, sl_begin, sl_end);
    Segment sg;
    unsigned it = 0;
    bool ok = true;
    int head_i = -1, head_g = 0, head_n = 0;   // first run, published in the background
    int fin_i = -1, fin_g = 0, fin_n = 0;      // last run, published after the loop
    int seg = 0;
    auto wait_pv = [&](unsigned pt) -> bool {        // P.V of tile pt has completed
      return mbar_wait(bar(B_O_FULL + (pt & 1)), (pt >> 1) & 1, s_abort);
    };
    auto quad_max = [](float v) {
      v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 1));
      return fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 2));
    };
    auto quad_sum = [](float v) {
      v += __shfl_xor_sync(0xffffffffu, v, 1);
      return v + __shfl_xor_sync(0xffffffffu, v, 2);
    };
    // this thread's 32 values (16 column pairs) of a 16-lane x 128-column TMEM block
    auto load_own = [&](uint32_t taddr, float* v) {
      float r[64];
      tmem_ld_16x128(taddr, r);
#pragma unroll
      for (int n = 0; n < 16; ++n) {
        v[2 * n] = half ? r[4 * n + 2] : r[4 * n];
        v[2 * n + 1] = half ? r[4 * n + 3] : r[4 * n + 1];
      }
    };
    // fold a partial (O row in shared memory at o_row, its (max, sum) = ml) into this
    // thread's share of its row
    auto fold_row = [&](float* acc, float& m_run, float& l_run, uint32_t o_row, float2 ml) {
      const float m_tot = fmaxf(m_run, ml.x);
      const float m_s = (m_tot == -INFINITY) ? 0.0f : m_tot;
      const float w_me = ex2(m_run - m_s), w_o = ex2(ml.x - m_s);
#pragma unroll
      for (int n = 0; n < 16; ++n) {
        const float2 v = ld_shared_v2f(o_row + (8 * n + 2 * quad) * 4);
        acc[2 * n] = acc[2 * n] * w_me + v.x * w_o;
        acc[2 * n + 1] = acc[2 * n + 1] * w_me + v.y * w_o;
      }
      l_run = l_run * w_me + ml.y * w_o;
      m_run = m_tot;
    };
    // normalise and write this thread's share of its row: 16 column pairs
    auto write_row = [&](const float* acc, float l, int oi, int g) {
      const float inv = 1.0f / l;
      __nv_bfloat16* dst = out + ((size_t)(oi + j_row) * Hq + g * 4 + wq) * kD + 2 * quad;
#pragma unroll
      for (int n = 0; n < 16; ++n)
        *reinterpret_cast<uint32_t*>(dst + 8 * n) = pack_bf16(acc[2 * n] * inv, acc[2 * n + 1] * inv);
    };

    while (ok && sch.next(sg)) {
      const int ki = ws_ptr<int>(a.ws, L.k)[sg.i];
      const int oi = ws_ptr<int>(a.ws, L.offset)[sg.i];
      const int len = kv_len[sg.i];
      const bool live = j_row < ki;
      const bool warp_live = 8 * half < ki;            // warp-uniform: some row of this warp is live
      const int pos = live ? ws_ptr<int>(a.ws, L.positions)[oi + j_row] : -1;
      // O accumulates in TMEM relative to a reference maximum m_ref that is only
      // raised (and O rescaled) when the row maximum outgrows it by 2^8.  l_part
      // is this thread's share of the row sum (summed over the quad at the end).
      float m_ref = -INFINITY, l_part = 0.0f;

      for (int t = sg.t0; t < sg.t1 && ok; ++t, ++it) {
        const int b = it & 1;
        const int b3 = it % 3;                   // the three score buffers in TMEM
        ok = mbar_wait(bar(B_S_FULL + b3), (it / 3) & 1, s_abort);
        if (!ok) break;
        tc_fence_after();
        // A warp without live rows only keeps in step: its arrival on the P barrier of tile
        // `it` must not land in the phase of tile it - 2, which ends with that tile's P.V.
        if (!warp_live && it >= 2) { ok = wait_pv(it - 2); if (!ok) break; }
        if (warp_live) {
          float s[32];
          load_own(t_lane + b3 * 128, s);
          const int vis = min(kTileTok, max(0, pos + 1 - t * kTileTok));     // visible columns of the row
          float m4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
          if (vis >= kTileTok) {
#pragma unroll
            for (int n = 0; n < 16; ++n) {
              m4[(2 * n) & 3] = fmaxf(m4[(2 * n) & 3], s[2 * n]);
              m4[(2 * n + 1) & 3] = fmaxf(m4[(2 * n + 1) & 3], s[2 * n + 1]);
            }
          } else if (vis > 0) {                        // (a row that is not live has vis = 0)
#pragma unroll
            for (int n = 0; n < 16; ++n) {
              const int col = 8 * n + 2 * quad;
              if (col < vis) m4[(2 * n) & 3] = fmaxf(m4[(2 * n) & 3], s[2 * n]);
              if (col + 1 < vis) m4[(2 * n + 1) & 3] = fmaxf(m4[(2 * n + 1) & 3], s[2 * n + 1]);
            }
          }
          const float mx = quad_max(fmaxf(fmaxf(m4[0], m4[1]), fmaxf(m4[2], m4[3]))) * scale_log2;
          bool need = false;
          float factor = 1.0f;
          if (t == sg.t0) {
            m_ref = mx;                                // the run's first P.V starts a fresh O
          } else if (live && mx > m_ref + 8.0f) {
            factor = ex2(m_ref - mx);
            m_ref = mx;
            l_part *= factor;
            need = true;
          }
          if (__any_sync(0xffffffffu, need)) {
            // Rescale this warp's O rows in TMEM before the next P.V accumulates.  The
            // 16-lane load / store also carries the sibling warp's 8 rows (written back
            // unchanged), so the two warps of a q-head take turns.
            ok = wait_pv(it - 1);
            if (!ok) break;
            if (lane == 0) {
              const long long t0 = clock64();
              while (atomicCAS(const_cast<int*>(&s_lock[wq]), 0, 1) != 0) {
                if (*s_abort || clock64() - t0 > kWaitCycles) { *s_abort = 1; break; }
              }
            }
            __syncwarp();
            if (*s_abort) { ok = false; break; }
            tc_fence_after();
            float o[64];
            tmem_ld_16x128(o_addr, o);
#pragma unroll
            for (int n = 0; n < 16; ++n) {
              if (half) { o[4 * n + 2] *= factor; o[4 * n + 3] *= factor; }
              else { o[4 * n] *= factor; o[4 * n + 1] *= factor; }
            }
            tmem_st_16x128(o_addr, o);
            tmem_st_wait();
            tc_fence_before();
            __syncwarp();
            if (lane == 0) { __threadfence_block(); atomicExch(const_cast<int*>(&s_lock[wq]), 0); }
          }
          // P[b] was last read by the P.V of tile it - 2
          if (it >= 2) { ok = wait_pv(it - 2); if (!ok) break; }
          const float m_safe = (m_ref == -INFINITY) ? 0.0f : m_ref;
          const uint32_t p_row = base + kOffP + b * kPBytes + quad * 4 + m_row * 128;
          const int sw = m_row & 7;
          float ps0 = 0.0f, ps1 = 0.0f;
          if (vis >= kTileTok) {
            // every column visible (all tiles but a pair's last one or two)
#pragma unroll
            for (int n = 0; n < 16; ++n) {
              const float p0 = ex2(fmaf(s[2 * n], scale_log2, -m_safe));
              const float p1 = ex2(fmaf(s[2 * n + 1], scale_log2, -m_safe));
              ps0 += p0; ps1 += p1;
              st_shared_b32(p_row + (n >> 3) * (kTcRows * 128) + (((n & 7) ^ sw) << 4), pack_bf16(p0, p1));
            }
          } else if (live) {
#pragma unroll
            for (int n = 0; n < 16; ++n) {
              const int col = 8 * n + 2 * quad;
              float p0 = ex2(fmaf(s[2 * n], scale_log2, -m_safe));
              float p1 = ex2(fmaf(s[2 * n + 1], scale_log2, -m_safe));
              p0 = (col < vis) ? p0 : 0.0f;
              p1 = (col + 1 < vis) ? p1 : 0.0f;
              ps0 += p0; ps1 += p1;
              st_shared_b32(p_row + (n >> 3) * (kTcRows * 128) + (((n & 7) ^ sw) << 4), pack_bf16(p0, p1));
            }
          }
          l_part += ps0 + ps1;
        }
        // last tile of the pair: V rows at or beyond the request's key count
        // must be finite (0 x NaN would poison the row): zero them once the
        // copy has landed
        if (t + 1 == sg.n_tiles && len - t * kTileTok < kTileTok) {
          const unsigned uv = 2 * it + 1;
          const int slot = uv % kStages;
          ok = mbar_wait(bar(B_KV_FULL + slot), (uv / kStages) & 1, s_abort);
          if (!ok) break;
          const int first = len - t * kTileTok;                    // first invalid token row
          const int n_chunks = (kTileTok - first) * 16;            // 16-byte chunks, both halves
          const uint32_t v_base = base + kOffKV + slot * kSlotBytes;
          for (int x = tid; x < n_chunks; x += kSoftmaxThreads) {
            const int r = first + (x >> 4), hc = x & 15;
            st_shared_v4(v_base + (r >> 4) * kPageBytes + (hc >> 3) * kPageHalf + (r & 15) * 128 + ((hc & 7) << 4), 0, 0, 0, 0);
          }
        }
        tc_fence_before();
        fence_async_smem();
        mbar_arrive(bar(B_P_FULL + b));
      }
      if (!ok) break;
      ok = wait_pv(it - 1);                            // the run's last P.V
      if (!ok) break;
      tc_fence_after();
      float acc[32];
      load_own(o_addr, acc);
      tc_fence_before();
      float l_run = quad_sum(l_part);

      const int kind = run_kind(sg, sch.more());
      bool write_rows = (kind == RUN_WHOLE);
      bool store_partial = (kind == RUN_PUBLISH || kind == RUN_FINAL);
      if (kind == RUN_TAIL) {
        ok = mbar_wait(bar(B_PARTNER), 0, s_abort);
        if (!ok) break;
        const int fast = *s_fast;
        if (fast > 0) {
          // all other contributors' partials sit in ring slots 2 it, 2 it + 1, ...:
          // fold them into this thread's row and finish the pair here
          const uint32_t ml_base = base + kOffQ + ((seg + 1) & 1) * kQBytes;
          for (int x = 0; x < fast; ++x) {
            const uint32_t o_slot = base + kOffKV + ((2 * it + x) % kStages) * kSlotBytes;
            if (live)
              fold_row(acc, m_ref, l_run, o_slot + m_row * (kD * 4),
                       ld_shared_v2f(ml_base + (x * kTcRows + m_row) * 8));
          }
          if (tid == 0) pair_cnt[sg.i * n_kv + sg.g] = 0;      // ready for the next launch
          write_rows = true;
        } else {
          store_partial = true;                                // ordinary path after the loop
        }
      }
      if (write_rows && live) write_row(acc, l_run, oi, sg.g);
      if (store_partial) {
        // A run that covers only part of its pair: store the un-normalised partial.
        // Nothing in the main loop waits on global memory (a round trip costs
        // microseconds while every SM is streaming).
        const int slot_id = c * 2 + (sg.first_of_cta ? 0 : 1);
        if (live) {
          float* po = part_o + ((size_t)slot_id * kTcRows + m_row) * kD + 2 * quad;
#pragma unroll
          for (int n = 0; n < 16; ++n)
            *reinterpret_cast<float2*>(po + 8 * n) = make_float2(acc[2 * n], acc[2 * n + 1]);
          if (quad == 0)
            *reinterpret_cast<float2*>(&part_ml[((size_t)slot_id * kTcRows + m_row) * 2]) =
                make_float2(m_ref, l_run);
        }
        if (kind == RUN_PUBLISH) {
          mbar_arrive(bar(B_PART));                            // the publisher warp takes over
          head_i = sg.i; head_g = sg.g; head_n = sg.n_tiles;
        } else {
          fin_i = sg.i; fin_g = sg.g; fin_n = sg.n_tiles;      // published below, after the loop
        }
      }
      ++seg;
    }
    // ---- end phase: publish what is left, merge the pairs this CTA is last to reach
    if (ok && (fin_i >= 0 || head_i >= 0)) {
      unsigned group_phase = 0, merge_phase = 0;
      auto group_sync = [&]() -> bool {                 // bounded barrier of the softmax threads
        mbar_arrive(bar(B_GROUP));
        const bool r = mbar_wait(bar(B_GROUP), group_phase & 1, s_abort);
        ++group_phase;
        return r;
      };
      int merge_i[2], merge_g[2], merge_n[2], n_merge = 0;
      if (fin_i >= 0) {
        __threadfence();
        ok = group_sync();
        if (ok && tid == 0) {
          const long long p0 = ((long long)s_tile[fin_i] * n_kv) + (long long)fin_g * fin_n;
          const int n_contrib = cta_of(p0 + fin_n - 1) - cta_of(p0) + 1;
          int* cnt = &pair_cnt[fin_i * n_kv + fin_g];
          const int old = atomicAdd(cnt, 1);
          s_ticket[0] = (old == n_contrib - 1);
          if (old == n_contrib - 1) *cnt = 0;           // ready for the next launch
        }
        if (ok) ok = group_sync();
        if (ok && s_ticket[0]) { merge_i[n_merge] = fin_i; merge_g[n_merge] = fin_g; merge_n[n_merge] = fin_n; ++n_merge; }
      }
      if (ok && head_i >= 0) {
        ok = mbar_wait(bar(B_PUB), 0, s_abort);
        if (ok && *s_head_last) { merge_i[n_merge] = head_i; merge_g[n_merge] = head_g; merge_n[n_merge] = head_n; ++n_merge; }
      }
      // Merge: all contributors' partials are bulk-copied into the (now idle) K/V
      // ring, up to kStages at a time, and every thread folds its share of its row.
      for (int x = 0; ok && x < n_merge; ++x) {
        __threadfence();
        const int pi = merge_i[x], pg = merge_g[x];
        const int ki = ws_ptr<int>(a.ws, L.k)[pi];
        const int oi = ws_ptr<int>(a.ws, L.offset)[pi];
        const bool live = j_row < ki;
        const long long p0 = ((long long)s_tile[pi] * n_kv) + (long long)pg * merge_n[x];
        const int c_lo = cta_of(p0), c_hi = cta_of(p0 + merge_n[x] - 1);
        float acc[32];
        float m_run = -INFINITY, l_run = 0.0f;
#pragma unroll
        for (int d = 0; d < 32; ++d) acc[d] = 0.0f;
        for (int cb = c_lo; cb <= c_hi && ok; cb += kStages) {
          const int nb = min(kStages, c_hi - cb + 1);
          ok = group_sync();                            // everybody is done with the ring slots
          if (!ok) break;
          if (tid == 0) {
            fence_async_all();
            mbar_expect_tx(bar(B_MERGE), nb * kTcRows * kD * 4);
            for (int y = 0; y < nb; ++y) {
              const int cc = cb + y;
              const int sid = cc * 2 + (s_slice[cc] >= p0 ? 0 : 1);
              bulk_load(base + kOffKV + y * kSlotBytes, part_o + (size_t)sid * kTcRows * kD,
                        kTcRows * kD * 4, bar(B_MERGE));
            }
          }
          float2 ml[kStages];
#pragma unroll
          for (int y = 0; y < kStages; ++y) {
            const int cc = min(cb + y, c_hi);
            const int sid = cc * 2 + (s_slice[cc] >= p0 ? 0 : 1);
            ml[y] = live ? __ldcg(reinterpret_cast<const float2*>(&part_ml[((size_t)sid * kTcRows + m_row) * 2]))
                         : make_float2(-INFINITY, 0.0f);
          }
          ok = mbar_wait(bar(B_MERGE), merge_phase & 1, s_abort);
          ++merge_phase;
          if (!ok) break;
#pragma unroll
          for (int y = 0; y < kStages; ++y) {
            if (y < nb && live)
              fold_row(acc, m_run, l_run, base + kOffKV + y * kSlotBytes + m_row * (kD * 4), ml[y]);
          }
        }
        if (ok && live) write_row(acc, l_run, oi, pg);
      }
    }
  }

  // ------------------------------------------------------------------ teardown
  tc_fence_before();
  __syncthreads();
  if (tid == 0 && *s_abort) atomicOr(&hdr[H_STATUS], 8 /*TIMEOUT*/);
  if (warp == kWarpMma) {
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

struct MapKey {
  const void* ptr; int a, b;
  bool operator<(const MapKey& o) const {
    return ptr != o.ptr ? ptr < o.ptr : (a != o.a ? a < o.a : b < o.b);
  }
};
std::mutex g_map_mu;
std::map<MapKey, CUtensorMap> g_kv_maps, g_q_maps;

// K or V of one layer: [num_pages][n_kv][16 tok][128 d].
// whole_page = false (K): viewed as (d_lo 64, d_hi 2, tok 16, head, page), one box = one
// 64-column half of a page-head, 2 KB, [16 tok][128 B]; the score product wants all 128
// keys of a tile 128 bytes apart within a half.
// whole_page = true (V): viewed as (d_lo 64, tok 16, d_hi 2, head, page), one box = one
// whole page-head, 4 KB, landing as [2 column halves][16 tok][128 B]; the second product
// takes one page per k step, so half the copy instructions do.
bool kv_map(const void* ptr, int n_kv, int num_pages, bool whole_page, CUtensorMap* out) {
  std::lock_guard<std::mutex> lk(g_map_mu);
  MapKey key{ptr, n_kv, whole_page ? -num_pages : num_pages};
  auto it = g_kv_maps.find(key);
  if (it != g_kv_maps.end()) { *out = it->second; return true; }
  EncodeTiledFn enc = get_encode();
  if (!enc) return false;
  cuuint64_t dims[5] = {64, 2, (cuuint64_t)kPage, (cuuint64_t)n_kv, (cuuint64_t)num_pages};
  cuuint64_t strides[4] = {128, 256, (cuuint64_t)kPage * kD * 2, (cuuint64_t)n_kv * kPage * kD * 2};
  cuuint32_t box[5] = {64, 1, (cuuint32_t)kPage, 1, 1};
  if (whole_page) {
    dims[1] = kPage; dims[2] = 2;
    strides[0] = 256; strides[1] = 128;
    box[1] = kPage; box[2] = 2;
  }
  cuuint32_t estr[5] = {1, 1, 1, 1, 1};
  CUresult r = enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 5, const_cast<void*>(ptr), dims, strides,
                   box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return false;
  if (g_kv_maps.size() > 4096) g_kv_maps.clear();
  g_kv_maps[key] = *out;
  return true;
}

// q: [rows][n_q][128] viewed as (d_lo 64, d_hi 2, row, head); box = 16 rows x 4 heads, which
// lands in shared memory head-major: tile row m = 16 h_local + j
bool q_map(const void* ptr, int n_q, int rows, CUtensorMap* out) {
  std::lock_guard<std::mutex> lk(g_map_mu);
  MapKey key{ptr, n_q, rows};
  auto it = g_q_maps.find(key);
  if (it != g_q_maps.end()) { *out = it->second; return true; }
  EncodeTiledFn enc = get_encode();
  if (!enc) return false;
  cuuint64_t dims[4] = {64, 2, (cuuint64_t)rows, (cuuint64_t)n_q};
  cuuint64_t strides[3] = {128, (cuuint64_t)n_q * kD * 2, (cuuint64_t)kD * 2};
  cuuint32_t box[4] = {64, 1, 16, 4};
  cuuint32_t estr[4] = {1, 1, 1, 1};
  CUresult r = enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(ptr), dims, strides,
                   box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                   CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) return false;
  if (g_q_maps.size() > 4096) g_q_maps.clear();
  g_q_maps[key] = *out;
  return true;
}

}  // namespace

void attn_tc_forget_maps() {
  std::lock_guard<std::mutex> lk(g_map_mu);
  g_kv_maps.clear();
  g_q_maps.clear();
}

cudaError_t attn_tc_prepare() {
  return cudaFuncSetAttribute(attn_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              kSmemBytes);
}

cudaError_t launch_attn_tc(const AttnArgs& a, cudaStream_t stream) {
  if (a.num_ctas > kMaxCtas) return cudaErrorNotSupported;      // the slice table is staged in shared memory
  WsLayout L = ws_layout(a.n_bs, a.n_kv_heads, a.num_ctas);
  CUtensorMap tq, tk, tv;
  if (!q_map(a.q, a.n_q_heads, kHalfW * a.n_bs, &tq) ||
      !kv_map(a.k_cache, a.n_kv_heads, a.num_pages, false, &tk) ||
      !kv_map(a.v_cache, a.n_kv_heads, a.num_pages, true, &tv))
    return cudaErrorNotSupported;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(a.num_ctas);
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = kSmemBytes;
  cfg.stream = stream;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, attn_tc_kernel, a, L, tq, tk, tv);
}

}  // namespace dscale

#ifdef DSCALE_WAIT_TEST
// Wait-limit test build only: leave out the K copies of key tile `tile` (counted inside the
// slice) of CTA `cta` in every following launch; (-1, -1) switches it off.  HOST call.
extern "C" int dscale_test_drop_copy(int cta, int tile) {
  if (cudaMemcpyToSymbol(dscale::g_drop_cta, &cta, sizeof(int)) != cudaSuccess) return -3;
  if (cudaMemcpyToSymbol(dscale::g_drop_tile, &tile, sizeof(int)) != cudaSuccess) return -3;
  return 0;
}
#endif
