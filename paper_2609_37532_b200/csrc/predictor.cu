// Acceptance-predictor front end: drafter logits and hidden states -> 1735
// features -> 1735-64-15 perceptron -> predLogits ("Acceptance predictor"
// paragraph, Eq. 4 and Eq. 5).  Two launches (the tail is scheduled while the stream runs):
//
//  pred_stream_kernel    the only pass over the drafter logits (15 N rows x V fp32,
//                        292 MB at N = 32: an HBM stream).  A CTA of 16 compute warps
//                        and a copy warp owns 32 rows x one vocabulary chunk; the copy
//                        warp fills a shared-memory ring with TMA boxes, warp w streams
//                        rows w and w + 16 with 128-bit shared loads and keeps, per row,
//                        the running (sum e^{z-top}, sum e^{z-top} z, sum z) and the 16
//                        largest values (sorted in lanes 0-15; a new value enters only
//                        if it beats the 16th, found by a warp vote, so the steady state
//                        costs one compare per four elements; `top`, the reference of
//                        the exponentials, is the head of that list).  The fixed 32 x V
//                        logit projection is a dense contraction with K = V: next to
//                        every 128-column sub-tile of logits the ring holds the matching
//                        32 x 128 tile of the projection matrix, and the 16 warps each
//                        issue one k = 8 step of m16n8k8 tf32 MMAs over it (operands
//                        z - pivot, rounded to tf32).  Warp-level MMAs on purpose: 4.7
//                        GFLOP ride along with a 292 MB stream, there is no tensor-core
//                        time to win.  One record per (row, chunk) goes to the workspace.
//                        The CTAs of the grid behind the (row group, chunk) CTAs compute
//                        the 64 x H hidden-state projection of all rows (bf16 MMAs) on
//                        the SMs the stream leaves free.
//  pred_tail_kernel      per request: merges the chunk records into the 18
//                        confidence values and the centred logit projection per
//                        position, appends the hidden projection and the batch
//                        context, then relu(W1 f + b1), W2 h + b2.
#include <cfloat>
#include <climits>
#include <cuda_bf16.h>

#include "kernels.cuh"
#include "tc_ptx.cuh"

namespace dscale {

#ifdef DSCALE_WAIT_TEST
__device__ int g_pred_drop_cta = -1, g_pred_drop_sub = -1;
#endif

namespace {

constexpr int kWarps = 16;                      // warps per CTA = k steps of 8 per sub-tile
constexpr int kRowsPerCta = 2 * kWarps;         // each warp streams two rows
constexpr int kStreamThreads = (kWarps + 1) * 32;   // + one copy warp
constexpr int kSub = 128;                       // columns per sub-tile: one float4 per lane
constexpr int kStride = kSub + 4;               // shared-memory row stride in floats (conflict-free fragments)

struct StreamArgs {
  const float* logits;      // [15 n_bs][ld]
  int64_t ld;
  int vocab;
  const int32_t* n_live;
  int n_bs;
  const __nv_bfloat16* p_logit;   // [32][vocab]
  float* part;              // [15 n_bs][chunks][kPredRec]
  float* rowsum;            // [row groups][chunks][32]: partial row sums of the projection matrix
  int chunks;
  int chunk_len;            // multiple of kSub
  int stream_ctas;          // chunks x row groups; the CTAs behind them serve the hidden projection
  int* status;              // workspace status word
  const __nv_bfloat16* hidden;     // [n_bs][15][hidden_dim]
  int hidden_dim;
  const __nv_bfloat16* p_hidden;   // [64][hidden_dim]
  float* feat;                     // [n_bs][1735]
};
constexpr int kHidThreads = 256;                // threads of one hidden-projection job
constexpr int kHidJobs = kWarps * 32 / kHidThreads;   // jobs side by side in a CTA that serves them
constexpr int kHidSlices = 4;                   // 16 of the 64 outputs per job

__device__ __forceinline__ void mma_tf32(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ float4 ldg_stream4(const float* p) {
  float4 r;
  asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
               : "=f"(r.x), "=f"(r.y), "=f"(r.z), "=f"(r.w)
               : "l"(p));
  return r;
}

// Sorted (descending) list of the 16 largest values seen, one per lane 0..15.
// `v` is warp-uniform.  Lanes >= 16 carry don't-care values.
__device__ __forceinline__ void top16_insert(float& tv, float v, int lane) {
  const float up = __shfl_up_sync(0xffffffffu, tv, 1);
  if (v > tv) tv = (lane > 0 && v > up) ? up : v;
}
// offer one value per lane; only values above the current 16th enter
__device__ __forceinline__ void top16_offer(float& tv, float& tau, float z, int lane) {
  unsigned mask = __ballot_sync(0xffffffffu, z > tau);
  while (mask) {
    const int src = __ffs(mask) - 1;
    mask &= mask - 1;
    top16_insert(tv, __shfl_sync(0xffffffffu, z, src), lane);
    tau = __shfl_sync(0xffffffffu, tv, 15);
  }
}

// Shared-memory ring: per stage the 32 rows' sub-tile of raw fp32 logits (16 KB) and
// the 32 x 128 bf16 tile of the projection matrix (8 KB), filled by a copy warp with
// six TMA boxes per stage; the 16 compute warps only wait for "full" and signal
// "empty", so a warp that is busy inserting into its top-16 list holds nobody up
// until the ring runs dry.  (Tried on the way: every warp copying its own rows and
// waiting for the slowest warp once per stage; one bulk copy per row, which is
// bound by the copy engine's per-instruction cost; per-thread cp.async issued by a
// single warp, which is bound by that warp's instruction issue.)  The layout
// inside a stage is the 128-byte XOR swizzle, so that the MMA fragment loads are
// free of bank conflicts.  One CTA per SM, one wave.
constexpr int kStages = 8;
constexpr int kZStage = kRowsPerCta * kSub * 4;           // 16 KB: 4 column groups x 32 rows x 128 bytes
constexpr int kPStage = kPredLog * kSub * 2;              // 8 KB: 2 column groups x 32 outputs x 128 bytes
constexpr int kOffP = kStages * kZStage;
constexpr int kOffPivot = kOffP + kStages * kPStage;
constexpr int kOffBar = kOffPivot + kRowsPerCta * 4;
constexpr int kOffAbort = kOffBar + 2 * kStages * 8;       // full[kStages], empty[kStages]
constexpr int kStreamSmem = kOffAbort + 16 + 1024;        // + slack to align the ring to 1024 bytes

// byte offset of logit (row r, column c) inside a stage's swizzled logit tile
__device__ __forceinline__ uint32_t z_off(int r, int c) {
  return (uint32_t)((c >> 5) * (kRowsPerCta * 128) + r * 128 + ((((c & 31) >> 2) ^ (r & 7)) << 4) + ((c & 3) << 2));
}
// byte offset of projection weight (output j, column c) inside a stage's swizzled tile
__device__ __forceinline__ uint32_t p_off(int j, int c) {
  return (uint32_t)((c >> 6) * 4096 + j * 128 + ((((c & 63) >> 3) ^ (j & 7)) << 4) + ((c & 7) << 1));
}
__device__ __forceinline__ void tma_box_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1)
      : "memory");
}
// 16-byte asynchronous copy global -> shared; bytes beyond `valid` are written as zeros
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, int valid) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(valid) : "memory");
}
// arrive on the barrier once all earlier cp.async of this thread have landed
__device__ __forceinline__ void cp_async_arrive(uint32_t bar) {
  asm volatile("cp.async.mbarrier.arrive.noinc.shared::cta.b64 [%0];" ::"r"(bar) : "memory");
}

// Running statistics of one logit row in one lane.  `top` is the largest value of the row seen
// so far by the whole warp (the head of the sorted list, the same in all lanes): it is the
// reference of the exponentials, so the steady state needs no rescaling and the lanes' sums
// are merged by plain addition.  A value above the reference is above the 16th as well, so
// the reference only moves inside the (rare) list-update path.
struct RowStat {
  float s, t, zsum;          // sum e, sum e z, sum z with e = exp(z - top)
  float nref;                // -top log2(e); 0 while nothing finite has been seen
  float top;
  float tv, tau;             // sorted top-16 (lane = rank) and the current 16th value
};
constexpr float kLog2e = 1.4426950408889634f;
__device__ __forceinline__ void row_init(RowStat& r) {
  r.s = r.t = r.zsum = r.nref = 0.f;
  r.top = -INFINITY; r.tv = -INFINITY; r.tau = -INFINITY;
}
// The rare part of a list update: some lane holds a second value above the 16th.  The first
// component equal to the lane's maximum is the one already offered; the others are offered
// component by component against the 16th as it stands, which is fetched once per component.
// Kept out of line: it runs a few times per row and chunk, and inlined (twice, unrolled four times)
// it made the hot loop larger and the whole kernel 1 us slower.  Returns (list entry
// of this lane, new 16th).
__device__ __noinline__ float2 offer_rest(float tv, float tau, float4 z, float zl, int lane) {
  const bool mx = z.x == zl, my = !mx && z.y == zl, mz = !mx && !my && z.z == zl;
  const float rest[4] = {mx ? -INFINITY : z.x, my ? -INFINITY : z.y, mz ? -INFINITY : z.z,
                         (mx || my || mz) ? z.w : -INFINITY};
#pragma unroll 1
  for (int x = 0; x < 4; ++x) {
    const float rv = x == 0 ? rest[0] : (x == 1 ? rest[1] : (x == 2 ? rest[2] : rest[3]));
    unsigned m = __ballot_sync(0xffffffffu, rv > tau);
    if (m) {
      while (m) {
        const int src = __ffs(m) - 1;
        m &= m - 1;
        top16_insert(tv, __shfl_sync(0xffffffffu, rv, src), lane);
      }
      tau = __shfl_sync(0xffffffffu, tv, 15);
    }
  }
  return make_float2(tv, tau);
}

// The list-update path of one row: called by the whole warp with the ballot of the lanes whose
// maximum beats the 16th.  What a warp pays here is latency, a chain of warp collectives, so the
// chain is kept short: the candidates are inserted one after another without looking at the new
// 16th in between (a value that is too small changes no lane), whether some lane holds a SECOND
// value above the 16th is decided up front against the old threshold (rare; then the other three
// values of every lane are offered as well), the new 16th is fetched once at the end, and the
// row maximum follows from the candidates themselves.
__device__ __forceinline__ void row_event(RowStat& r, float4 z, float zl, unsigned cand, int lane) {
  const float m01 = fmaxf(z.x, z.y), n01 = fminf(z.x, z.y), m23 = fmaxf(z.z, z.w), n23 = fminf(z.z, z.w);
  const float second = fmaxf(fminf(m01, m23), m01 >= m23 ? n01 : n23);   // second largest of the four
  const bool more = __any_sync(0xffffffffu, second > r.tau);
  float vmax = -INFINITY;                                   // warp-uniform: the largest candidate
  while (cand) {
    const int src = __ffs(cand) - 1;
    cand &= cand - 1;
    const float v = __shfl_sync(0xffffffffu, zl, src);
    top16_insert(r.tv, v, lane);
    vmax = fmaxf(vmax, v);
  }
  r.tau = __shfl_sync(0xffffffffu, r.tv, 15);
  if (more) {
    const float2 lt = offer_rest(r.tv, r.tau, z, zl, lane);
    r.tv = lt.x; r.tau = lt.y;
  }
  if (vmax > r.top) {                                       // a new maximum: move the reference
    const float f = r.top == -INFINITY ? 0.f : ex2((r.top - vmax) * kLog2e);
    r.s *= f; r.t *= f;
    r.top = vmax;
    r.nref = -(vmax * kLog2e);
  }
}

// one row, the careful path for the end of the vocabulary: values at or beyond col_hi do not count
__device__ __forceinline__ void row_update(RowStat& r, float4 z, int c, int col_hi, int lane) {
  if (c >= col_hi) z.x = -INFINITY;
  if (c + 1 >= col_hi) z.y = -INFINITY;
  if (c + 2 >= col_hi) z.z = -INFINITY;
  if (c + 3 >= col_hi) z.w = -INFINITY;
  const float zl = fmaxf(fmaxf(z.x, z.y), fmaxf(z.z, z.w));
  const unsigned cand = __ballot_sync(0xffffffffu, zl > r.tau);
  if (cand) row_event(r, z, zl, cand, lane);
  const float zz[4] = {z.x, z.y, z.z, z.w};
#pragma unroll
  for (int x = 0; x < 4; ++x) {
    if (zz[x] != -INFINITY) {
      const float e = ex2(fmaf(zz[x], kLog2e, r.nref));
      r.s += e; r.t = fmaf(e, zz[x], r.t); r.zsum += zz[x];
    }
  }
}

// two rows at once, written so that the two rows' chains are independent instructions of one
// basic block
__device__ __forceinline__ void row_update2(RowStat& a, RowStat& b, float4 za, float4 zb, int c, int col_hi,
                                            int lane) {
  if (c - 4 * lane + kSub > col_hi) {                       // ragged end (warp-uniform test): the careful path
    row_update(a, za, c, col_hi, lane);
    row_update(b, zb, c, col_hi, lane);
    return;
  }
  const float la = fmaxf(fmaxf(za.x, za.y), fmaxf(za.z, za.w));
  const float lb = fmaxf(fmaxf(zb.x, zb.y), fmaxf(zb.z, zb.w));
  if (__any_sync(0xffffffffu, la > a.tau || lb > b.tau)) {  // rare once the lists have warmed up
    const unsigned ca = __ballot_sync(0xffffffffu, la > a.tau), cb = __ballot_sync(0xffffffffu, lb > b.tau);
    if (ca) row_event(a, za, la, ca, lane);
    if (cb) row_event(b, zb, lb, cb, lane);
  }
  const float na = a.nref, nb = b.nref;
  const float xa[4] = {za.x, za.y, za.z, za.w}, xb[4] = {zb.x, zb.y, zb.z, zb.w};
#pragma unroll
  for (int x = 0; x < 4; ++x) {
    const float ea = ex2(fmaf(xa[x], kLog2e, na)), eb = ex2(fmaf(xb[x], kLog2e, nb));
    a.s += ea; b.s += eb;
    a.t = fmaf(ea, xa[x], a.t); b.t = fmaf(eb, xb[x], b.t);
    a.zsum += xa[x]; b.zsum += xb[x];
  }
}

__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// ---------------------------------------------------------------------------
// Hidden-state projection: [15 N rows x H] . [H x 64], a small dense contraction
// (0.25 GFLOP at N = 32, H = 4096) on warp-level bf16 MMAs.  It does not depend on the
// logit stream: the CTAs of the stream grid that are left over once every (row group,
// chunk) has its CTA serve it, two jobs of 256 threads side by side, while the stream runs
// on the other SMs.  (As a kernel of its own ahead of the stream it held the stream's CTAs
// off its SMs for the 10 us it ran: the two did not share an SM.)  A job owns 16 rows x 16
// outputs; its 8 warps split H in blocks of 32 and are summed through shared memory.  The
// k slots of the MMA are a permutation of the 32 columns of a block (the same one for both
// operands), so every fragment is one 16-byte load.
__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ void job_barrier(int job) {
  asm volatile("bar.sync %0, %1;" ::"r"(job + 1), "r"(kHidThreads) : "memory");
}
__device__ void hidden_jobs(const StreamArgs& a, int live_rows, int first_item, int item_stride, int job,
                            int tid /* within the job */, float* red /* [8][256] */) {
  constexpr int kOut = kPredHid / kHidSlices;               // 16 outputs = 2 n-tiles
  const int warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int H = a.hidden_dim;
  const int row_tiles = (live_rows + 15) / 16;
  for (int item = first_item; item < row_tiles * kHidSlices; item += item_stride) {
    const int row0 = (item / kHidSlices) * 16, j0 = (item % kHidSlices) * kOut;
    const int r_lo = min(row0 + g, live_rows - 1), r_hi = min(row0 + g + 8, live_rows - 1);
    const __nv_bfloat16* h_lo = a.hidden + (size_t)r_lo * H;
    const __nv_bfloat16* h_hi = a.hidden + (size_t)r_hi * H;
    const __nv_bfloat16* p0 = a.p_hidden + (size_t)(j0 + g) * H;
    const __nv_bfloat16* p1 = a.p_hidden + (size_t)(j0 + 8 + g) * H;
    float d[2][4];
#pragma unroll
    for (int x = 0; x < 2; ++x) d[x][0] = d[x][1] = d[x][2] = d[x][3] = 0.f;
    const uint4 zero4 = make_uint4(0, 0, 0, 0);
    constexpr int kStep = 32 * (kHidThreads / 32);          // columns per round of the 8 warps
#pragma unroll 4
    for (int kb = warp * 32; kb < H; kb += kStep) {
      const int c = kb + 8 * t;                            // hidden_dim % 8 == 0: a chunk is in or out
      const bool in = c < H;
      const uint4 alo = in ? __ldg(reinterpret_cast<const uint4*>(h_lo + c)) : zero4;
      const uint4 ahi = in ? __ldg(reinterpret_cast<const uint4*>(h_hi + c)) : zero4;
      const uint4 b0 = in ? __ldg(reinterpret_cast<const uint4*>(p0 + c)) : zero4;
      const uint4 b1 = in ? __ldg(reinterpret_cast<const uint4*>(p1 + c)) : zero4;
      mma_bf16(d[0], alo.x, ahi.x, alo.y, ahi.y, b0.x, b0.y);
      mma_bf16(d[0], alo.z, ahi.z, alo.w, ahi.w, b0.z, b0.w);
      mma_bf16(d[1], alo.x, ahi.x, alo.y, ahi.y, b1.x, b1.y);
      mma_bf16(d[1], alo.z, ahi.z, alo.w, ahi.w, b1.z, b1.w);
    }
    float* rw = red + warp * (16 * kOut);
#pragma unroll
    for (int nt = 0; nt < 2; ++nt) {
      rw[g * kOut + 8 * nt + 2 * t] = d[nt][0];
      rw[g * kOut + 8 * nt + 2 * t + 1] = d[nt][1];
      rw[(g + 8) * kOut + 8 * nt + 2 * t] = d[nt][2];
      rw[(g + 8) * kOut + 8 * nt + 2 * t + 1] = d[nt][3];
    }
    job_barrier(job);
    {
      const int x = tid;                                    // 16 rows x 16 outputs = 256 = kHidThreads
      float acc = 0.f;
#pragma unroll
      for (int w = 0; w < kHidThreads / 32; ++w) acc += red[w * (16 * kOut) + x];
      const int row = row0 + (x >> 4), j = j0 + (x & 15);
      if (row < live_rows) {
        const int i = row / kPredPos, p = row - i * kPredPos;
        a.feat[(size_t)i * kPredFeatures + kPredPos * kPredConf + p * kPredHid + j] = acc;
      }
    }
    job_barrier(job);                                       // the buffer is free for the next item
  }
}

__global__ void __launch_bounds__(kStreamThreads, 1)
pred_stream_kernel(StreamArgs a, const __grid_constant__ CUtensorMap tm_z, const __grid_constant__ CUtensorMap tm_p) {
  extern __shared__ unsigned char smem_raw[];
  const uint32_t raw = smem_u32(smem_raw);
  const uint32_t sbase = (raw + 1023u) & ~1023u;
  unsigned char* smem = smem_raw + (sbase - raw);
  float* pivots = reinterpret_cast<float*>(smem + kOffPivot);
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + kOffAbort);
  auto psm = [&](int st, int j, int c) -> unsigned short* {
    return reinterpret_cast<unsigned short*>(smem + kOffP + st * kPStage + p_off(j, c));
  };
  auto full = [&](int st) { return sbase + kOffBar + 8u * st; };
  auto empty = [&](int st) { return sbase + kOffBar + 8u * (kStages + st); };

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  // the tail kernel behind this one may be scheduled now: it touches nothing this grid writes
  // before its own wait on this grid's completion
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  int n = *a.n_live;
  n = n < 0 ? 0 : (n > a.n_bs ? a.n_bs : n);
  const int live_rows = kPredPos * n;
  if ((int)blockIdx.x >= a.stream_ctas) {
    // ===================================================== hidden-state projection
    if (warp < kHidJobs * (kHidThreads / 32) && live_rows > 0) {
      const int job = tid / kHidThreads;
      hidden_jobs(a, live_rows, ((int)blockIdx.x - a.stream_ctas) * kHidJobs + job,
                  ((int)gridDim.x - a.stream_ctas) * kHidJobs, job, tid - job * kHidThreads,
                  reinterpret_cast<float*>(smem) + job * (kHidThreads / 32) * 256);
    }
    return;
  }
  const int row_group = (int)blockIdx.x / a.chunks;
  const int row0 = row_group * kRowsPerCta;
  if (row0 >= live_rows) return;
  const int chunk = (int)blockIdx.x % a.chunks;
  const int col_lo = chunk * a.chunk_len;
  const int col_hi = min(a.vocab, col_lo + a.chunk_len);
  if (col_lo >= col_hi) return;
  const int n_sub = (col_hi - col_lo + kSub - 1) / kSub;

  // warp w owns rows w and w + 16 of the CTA's 32 (one in each 16-row MMA tile)
  const int my_row[2] = {row0 + warp, row0 + warp + kWarps};
  const bool live[2] = {warp < kWarps && my_row[0] < live_rows, warp < kWarps && my_row[1] < live_rows};
  const bool p_vec = (a.vocab & 7) == 0;               // projection rows 16-byte aligned
  // The centring term of the logit projection needs the row sums of the projection matrix.  Its
  // tiles pass through the shared memory of every row group's CTAs; the live row groups take
  // turns by sub-tile, so each CTA sums a share of its chunk and none is slower than the others.
  const int live_groups = (live_rows + kRowsPerCta - 1) / kRowsPerCta;
  const int pj = tid >> 4, pq = tid & 15;               // projection tile piece: (output, 8 columns)

  if (tid == 0) {
    // full: the copy warp's expect-tx arrival (plus one arrival when that warp stores the
    // projection tile by hand); empty: every compute warp has finished with the stage
    for (int st = 0; st < kStages; ++st) {
      mbar_init(full(st), p_vec ? 1 : 2);
      mbar_init(empty(st), kWarps);
    }
    s_abort[0] = 0; s_abort[1] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp < kWarps && lane < 2) pivots[warp + kWarps * lane] = live[lane] ? a.logits[(size_t)my_row[lane] * a.ld] : 0.f;
  __syncthreads();

  if (warp == kWarps) {
    // ===================================================== copy warp
    // Per 24 KB stage six TMA boxes, one lane each: four of 32 columns x 32 rows of
    // logits, two of 64 columns x 32 outputs of the projection matrix (128-byte
    // swizzle; columns beyond the vocabulary and rows beyond the tensor arrive as
    // zeros).  With an odd vocabulary the projection rows are not 16-byte aligned and
    // are stored by hand (slow, but such vocabularies are not the case to tune for).
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_z) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_p) : "memory");
    }
    int st = 0;
    uint32_t parity = 1;                                    // a fresh barrier passes a wait on parity 1
    bool ok = true;
    for (int v = 0; v < n_sub && ok; ++v) {
      ok = mbar_wait(empty(st), parity, s_abort);
      if (!ok) break;
      const int c = col_lo + v * kSub;
      if (lane == 0) mbar_expect_tx(full(st), kZStage + (p_vec ? kPStage : 0));
      __syncwarp();
#ifdef DSCALE_WAIT_TEST
      // wait-limit test build only: the logit boxes of one sub-tile of one CTA are left out (the
      // barrier stays armed), so that every wait behind it runs into its limit
      const bool drop = (int)blockIdx.x == g_pred_drop_cta && v == g_pred_drop_sub;
#else
      constexpr bool drop = false;
#endif
      if (lane < 4 && !drop) tma_box_2d(sbase + st * kZStage + lane * (kRowsPerCta * 128), &tm_z, full(st), c + 32 * lane, row0);
      else if (lane >= 4 && lane < 6 && p_vec)
        tma_box_2d(sbase + kOffP + st * kPStage + (lane - 4) * 4096, &tm_p, full(st), c + 64 * (lane - 4), 0);
      if (!p_vec) {
        for (int e = lane; e < kPredLog * kSub; e += 32) {
          const int j = e >> 7, cc = e & 127;
          *psm(st, j, cc) = c + cc < col_hi ? __bfloat16_as_ushort(a.p_logit[(size_t)j * a.vocab + c + cc])
                                            : (unsigned short)0;
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(full(st));
      }
      if (++st == kStages) { st = 0; parity ^= 1; }
    }
    // every stage issued has been, or will be, waited for by the compute warps; on an
    // aborted run wait (bounded) for the copies in flight before the CTA may exit
    if (!ok) {
      for (int x = 0; x < kStages; ++x) { mbar_wait(full(x), 0, s_abort + 1); mbar_wait(full(x), 1, s_abort + 1); }
    }
  }

  RowStat rs[2];
  row_init(rs[0]); row_init(rs[1]);
  float p_rowsum = 0.f;
  float d[2][4][4];
#pragma unroll
  for (int h = 0; h < 2; ++h)
#pragma unroll
    for (int x = 0; x < 4; ++x) d[h][x][0] = d[h][x][1] = d[h][x][2] = d[h][x][3] = 0.f;
  const int g = lane >> 2, t = lane & 3;

  // Per-thread constants of the loop.  The k slots (t, t + 4) of this warp's MMA step
  // stand for columns 8 warp + 2t and + 2t + 1 (the same permutation for both
  // operands), so a fragment is one 8-byte logit load per row and one 4-byte load of
  // a bf16 pair per output tile.  Columns beyond the vocabulary need no mask here:
  // both tiles are zero there.
  float piv[4];
  uint32_t zo[4];
#pragma unroll
  for (int x = 0; x < 4; ++x) {                             // rows g, g + 8, g + 16, g + 24
    piv[x] = pivots[g + 8 * x];
    zo[x] = z_off(g + 8 * x, 8 * (warp & 15) + 2 * t);
  }
  const uint32_t po = kOffP + p_off(g, 8 * (warp & 15) + 2 * t);    // + 1024 per output tile
  const uint32_t so0 = z_off(warp & 15, 4 * lane), so1 = z_off((warp & 15) + kWarps, 4 * lane);
  const uint32_t ro = kOffP + p_off(pj & 31, 8 * pq);               // row sums: eight weights of output pj
  int rs_turn = row_group;                                          // sub-tiles until this CTA's turn

  int st = 0;
  uint32_t parity = 0;
  bool ok = true;
  for (int u = 0; u < n_sub && warp < kWarps; ++u) {
    ok = mbar_wait(full(st), parity, s_abort);
    if (!ok) break;
    const unsigned char* zst = smem + st * kZStage;
    const unsigned char* pst = smem + st * kPStage;
    // ---- row statistics on the exact fp32 values
    const int c = col_lo + u * kSub + 4 * lane;
    // both rows unconditionally (a dead row holds whatever the copy brought: its results are
    // never written), so that the two dependency chains interleave
    row_update2(rs[0], rs[1], *reinterpret_cast<const float4*>(zst + so0),
                *reinterpret_cast<const float4*>(zst + so1), c, col_hi, lane);
    // ---- this warp's k step of the logit projection, both 16-row tiles
    {
      uint32_t bw[4];
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) bw[nt] = *reinterpret_cast<const uint32_t*>(pst + po + 1024 * nt);
#pragma unroll
      for (int h = 0; h < 2; ++h) {
        const float2 zlo = *reinterpret_cast<const float2*>(zst + zo[2 * h]);
        const float2 zhi = *reinterpret_cast<const float2*>(zst + zo[2 * h + 1]);
        uint32_t af[4];
        // z - pivot, rounded to tf32 the way cvt.rna does (add half a tf32 ulp to the bit pattern;
        // the tensor core ignores the low 13 bits), on the integer pipe instead of the conversion unit
        af[0] = __float_as_uint(zlo.x - piv[2 * h]) + 0x1000u;
        af[1] = __float_as_uint(zhi.x - piv[2 * h + 1]) + 0x1000u;
        af[2] = __float_as_uint(zlo.y - piv[2 * h]) + 0x1000u;
        af[3] = __float_as_uint(zhi.y - piv[2 * h + 1]) + 0x1000u;
#pragma unroll
        for (int nt = 0; nt < 4; ++nt) mma_tf32(d[h][nt], af, bw[nt] << 16, bw[nt] & 0xffff0000u);
      }
    }
    // ---- row sums of the projection matrix (this row group's turn)
    if (rs_turn == 0) {
      rs_turn = live_groups;
      const uint4 w = *reinterpret_cast<const uint4*>(pst + ro);
      const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
#pragma unroll
      for (int x = 0; x < 4; ++x)
        p_rowsum += __uint_as_float(ww[x] << 16) + __uint_as_float(ww[x] & 0xffff0000u);
    }
    --rs_turn;
    __syncwarp();
    if (lane == 0) mbar_arrive(empty(st));                  // this warp is done with the stage
    if (++st == kStages) { st = 0; parity ^= 1; }
  }
  __syncthreads();
  if (*s_abort) {
    // Some wait ran out (the copy warp has already waited for its copies): flag the
    // status word and leave.
    if (tid == 0) atomicOr(a.status, 8 /*TIMEOUT*/);
    return;
  }

  // ---- row statistics: merge the 32 lanes (one reference per row: plain sums), write the records
#pragma unroll
  for (int x = 0; x < 2; ++x) {
    float s_sum = rs[x].s, t_sum = rs[x].t, z_sum = rs[x].zsum;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      s_sum += __shfl_xor_sync(0xffffffffu, s_sum, o);
      t_sum += __shfl_xor_sync(0xffffffffu, t_sum, o);
      z_sum += __shfl_xor_sync(0xffffffffu, z_sum, o);
    }
    if (live[x]) {
      float* rec = a.part + ((size_t)my_row[x] * a.chunks + chunk) * kPredRec;
      if (lane < 16) rec[lane] = rs[x].tv;
      if (lane == 0) { rec[16] = rs[x].top; rec[17] = s_sum; rec[18] = t_sum; rec[19] = z_sum; }
    }
  }
  // ---- projection: sum the 16 warps' k slices through shared memory (the ring is idle now)
  float* red = reinterpret_cast<float*>(smem);
  constexpr int kTile = kRowsPerCta * kPredLog;             // 1024 projections per CTA
  static_assert(kStages * kZStage >= kWarps * kTile * 4, "reduction buffer");
  if (warp < kWarps) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
#pragma unroll
      for (int nt = 0; nt < 4; ++nt) {
        float* q = red + warp * kTile + (16 * h + g) * kPredLog + 8 * nt + 2 * t;
        q[0] = d[h][nt][0]; q[1] = d[h][nt][1];
        q[8 * kPredLog] = d[h][nt][2]; q[8 * kPredLog + 1] = d[h][nt][3];
      }
    }
  }
  __syncthreads();
  for (int e = tid; e < kTile; e += kStreamThreads) {
    float acc = 0.f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) acc += red[w * kTile + e];
    const int r = e >> 5, j = e & 31;
    if (row0 + r < live_rows)
      a.part[((size_t)(row0 + r) * a.chunks + chunk) * kPredRec + 20 + j] = acc;
  }
  if (warp < kWarps) {
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) p_rowsum += __shfl_xor_sync(0xffffffffu, p_rowsum, o);
    if (pq == 0) a.rowsum[((size_t)row_group * a.chunks + chunk) * kPredLog + pj] = p_rowsum;
  }
}

// ---------------------------------------------------------------------------
struct FeatArgs {
  const float* logits;
  int64_t ld;
  int vocab;
  const int32_t* n_live;
  int n_bs;
  const __nv_bfloat16* hidden;     // [n_bs][15][hidden_dim]
  int hidden_dim;
  const __nv_bfloat16* p_hidden;   // [64][hidden_dim]
  const float* part;
  const float* rowsum;
  int chunks;
  float* feat;                     // [n_bs][1735]
};

// ---------------------------------------------------------------------------
struct MlpArgs {
  const int32_t* n_live;
  int n_bs;
  const float* feat;
  const float* w1;   // [64][1735]
  const float* b1;
  const float* w2;   // [15][64]
  const float* b2;
  float* pred_logits;   // [n_bs][15]
  float* features_out;  // nullable [n_bs][1735]
  int* status;          // workspace status word
};

// ---------------------------------------------------------------------------
// Per request, behind the stream: merge the chunk records into the 18 confidence values and the
// centred logit projection of each position, append the hidden-state projection and the batch
// context, then relu(W1 f + b1) and W2 h + b2.  A request is served by a cluster of four CTAs:
// each merges a quarter of the positions and stores its features into the shared memory of all
// four, and each computes 16 of the 64 hidden units from its own quarter of W1 (111 KB, fetched
// into shared memory by one bulk copy), so that no single SM has to pull all of W1 through its
// L2 port; the hidden units meet in the first CTA, which applies W2.  The launch uses
// programmatic stream serialisation: everything that depends only on the call's inputs (the W1
// copy, the pivots, the biases) happens before the grid dependency is waited for, while the
// logit stream is still running.
constexpr int kTailCtas = 4;                                // CTAs (one cluster) per request
constexpr int kTailThreads = 512;                           // 16 warps: a hidden unit each
constexpr int kTailUnits = kPredMlp / kTailCtas;            // hidden units per CTA
constexpr int kTailW1 = kTailUnits * kPredFeatures;         // floats of W1 per CTA (111,040 bytes)
constexpr int kTailMergeWarps = (kPredPos + kTailCtas - 1) / kTailCtas;   // positions per CTA
constexpr int kTailSf = (kPredFeatures + 3) / 4 * 4;
constexpr int kTailCand = 16 * kPredMaxChunks;              // candidate values of one position
constexpr int kTailRest = kTailThreads / 32 - kTailMergeWarps;    // warps that do not merge a position
constexpr int kTailSmem = (kTailW1 + kTailSf + kPredMlp + kTailRest * kPredLog + kTailMergeWarps * kTailCand) * 4 + 32;
static_assert(kTailUnits * 32 == kTailThreads, "one warp per hidden unit");
static_assert((kTailW1 * 4) % 16 == 0, "bulk copy size");

// order-preserving key of a float for integer warp reductions; a NaN gets the lowest key
__device__ __forceinline__ unsigned f2key(float v) {
  const unsigned u = __float_as_uint(v);
  return v == v ? (u ^ ((u >> 31) ? 0xffffffffu : 0x80000000u)) : 0u;
}
__device__ __forceinline__ float key2f(unsigned k) {
  return __uint_as_float(k ^ ((k >> 31) ? 0x80000000u : 0xffffffffu));
}
__device__ __forceinline__ uint32_t tail_cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// store into the same shared-memory variable of another CTA of the cluster
__device__ __forceinline__ void st_cluster(const float* local, uint32_t rank, float v) {
  uint32_t addr;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(addr) : "r"(smem_u32(local)), "r"(rank));
  asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}
__device__ __forceinline__ void tail_cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;\n\tbarrier.cluster.wait.acquire.aligned;" ::: "memory");
}

__global__ void __cluster_dims__(kTailCtas, 1, 1) __launch_bounds__(kTailThreads, 1)
pred_tail_kernel(FeatArgs a, MlpArgs m) {
  extern __shared__ __align__(16) unsigned char tail_smem[];
  float* w1s = reinterpret_cast<float*>(tail_smem);         // this CTA's 16 rows of W1
  float* sf = w1s + kTailW1;                                // the request's feature vector
  float* sh = sf + kTailSf;                                 // hidden units (complete in CTA 0)
  float* rsp = sh + kPredMlp;                               // partial row sums of the projection matrix, one array per non-merging warp
  float* cs = rsp + kTailRest * kPredLog;                   // candidate staging, one array per merging warp
  const uint32_t bar = smem_u32(cs + kTailMergeWarps * kTailCand);
  volatile int* s_abort = reinterpret_cast<volatile int*>(cs + kTailMergeWarps * kTailCand + 2);
  const uint32_t rank = tail_cluster_rank();
  const int i = blockIdx.x / kTailCtas;
  int n = *a.n_live;
  n = n < 0 ? 0 : (n > a.n_bs ? a.n_bs : n);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const bool live = i < n;                                  // the same for the four CTAs of a cluster
  const bool bulk = (reinterpret_cast<uintptr_t>(m.w1) & 15) == 0;
  const int unit = kTailUnits * (int)rank + warp;           // this warp's hidden unit
  // ---- before the grid dependency: inputs of the call only
  if (tid == 0) {
    mbar_init(bar, 1);
    s_abort[0] = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    if (live && bulk) {
      mbar_expect_tx(bar, kTailW1 * 4);
      bulk_load(smem_u32(w1s), m.w1 + (size_t)rank * kTailW1, kTailW1 * 4, bar);
    }
  }
  const int p = (int)rank + kTailCtas * warp;               // the position a merging warp serves
  const bool merges = warp < kTailMergeWarps && p < kPredPos;
  float pivot = 0.f, b1v = 0.f;
  if (live) {
    if (merges) pivot = a.logits[(size_t)(i * kPredPos + p) * a.ld];
    b1v = m.b1[unit];
  }
  __syncthreads();                                          // the barrier is initialised for every waiter
  pdl_wait();
  if (!live) {                                              // dead request: zeros (the whole cluster leaves)
    if (rank == 0) {
      if (tid < kPredPos) m.pred_logits[i * kPredPos + tid] = 0.f;
      if (m.features_out)
        for (int x = tid; x < kPredFeatures; x += kTailThreads) m.features_out[(size_t)i * kPredFeatures + x] = 0.f;
    }
    return;
  }
  float centre = 0.f, craw = 0.f;                           // mean(z) - pivot and P (z - pivot) of a merging warp's position
  if (merges) {
    // ---- confidence values and centred logit projection of position p
    const int row = i * kPredPos + p;
    const float* rec0 = a.part + (size_t)row * a.chunks * kPredRec;
    float* cw = cs + warp * kTailCand;
    // all loads of this position first (independent), then the merges
    for (int e = lane; e < 16 * a.chunks; e += 32) cw[e] = rec0[(size_t)(e >> 4) * kPredRec + (e & 15)];
    float proj = 0.f;
#pragma unroll 8
    for (int c = 0; c < a.chunks; ++c) proj += rec0[(size_t)c * kPredRec + 20 + lane];
    float mx = -INFINITY, s_sum = 0.f, t_sum = 0.f, z_sum = 0.f;   // the chunks' (max, sum, sum e z, sum z): lane = chunk
    if (lane < a.chunks) {
      const float* r = rec0 + (size_t)lane * kPredRec;
      mx = r[16]; s_sum = r[17]; t_sum = r[18]; z_sum = r[19];
    }
    __syncwarp();
    // The 16 largest of all chunks' candidates, in order.  Every chunk's list is sorted, so
    // this is a merge: lane c holds the head of chunk c, the warp maximum (an integer
    // reduction on order-preserving keys) is the next value, the first lane holding it advances.
    float tv = -INFINITY;                                   // lane j < 16: the (j + 1)-th largest
    int ptr = 0;
    unsigned head = lane < a.chunks ? f2key(cw[16 * lane]) : 0u;
#pragma unroll 1
    for (int j = 0; j < 16; ++j) {
      const unsigned gm = __reduce_max_sync(0xffffffffu, head);
      const unsigned who = __ballot_sync(0xffffffffu, head == gm);
      if (lane == __ffs(who) - 1) {
        ++ptr;
        head = (lane < a.chunks && ptr < 16) ? f2key(cw[16 * lane + ptr]) : 0u;
      }
      if (lane == j) tv = gm != 0u ? key2f(gm) : -INFINITY;
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float m2 = __shfl_xor_sync(0xffffffffu, mx, o);
      const float s2 = __shfl_xor_sync(0xffffffffu, s_sum, o);
      const float t2 = __shfl_xor_sync(0xffffffffu, t_sum, o);
      z_sum += __shfl_xor_sync(0xffffffffu, z_sum, o);
      const float mm = fmaxf(mx, m2);
      const float r1 = mx == -INFINITY ? 0.f : expf(mx - mm), r2 = m2 == -INFINITY ? 0.f : expf(m2 - mm);
      s_sum = s_sum * r1 + s2 * r2;
      t_sum = t_sum * r1 + t2 * r2;
      mx = mm;
    }
    const float lse = mx + logf(s_sum);
    const float top = __shfl_sync(0xffffffffu, tv, 0);
    float conf = 0.f;
    if (lane == 0) conf = top;
    else if (lane < 16) conf = top - tv;
    else if (lane == 16) conf = top - lse;
    else if (lane == 17) conf = lse - t_sum / s_sum;
    // logit projection of z - mean(z): the stream accumulated P (z - pivot)
    const float mean = z_sum / (float)a.vocab;
    centre = mean - pivot;
    craw = proj;
#pragma unroll
    for (uint32_t dst = 0; dst < kTailCtas; ++dst)
      if (lane < kPredConf) st_cluster(sf + p * kPredConf + lane, dst, conf);
  } else if (warp >= kTailMergeWarps) {
    // ---- the other warps: the row sums of the projection matrix (the stream's CTAs left one
    // partial vector per live row group and chunk; lane = output, a fixed order of summation),
    // the hidden-state projection of this request and the batch context
    const int slots = (kPredPos * n + kRowsPerCta - 1) / kRowsPerCta * a.chunks;
    float rs = 0.f;
#pragma unroll 4
    for (int x = warp - kTailMergeWarps; x < slots; x += kTailRest) rs += a.rowsum[(size_t)x * kPredLog + lane];
    rsp[(warp - kTailMergeWarps) * kPredLog + lane] = rs;
    constexpr int kRest = kTailRest * 32;
    const float* hsrc = a.feat + (size_t)i * kPredFeatures + kPredPos * kPredConf;
    for (int x = tid - kTailMergeWarps * 32; x < kPredPos * kPredHid; x += kRest) sf[kPredPos * kPredConf + x] = hsrc[x];
    if (warp == kTailMergeWarps && lane < kPredCtx)
      sf[kPredFeatures - kPredCtx + lane] = lane == 0 ? (float)n : (lane == 3 ? 1.f : 0.f);
  }
  __syncthreads();
  if (merges) {
    float rs = 0.f;
#pragma unroll
    for (int x = 0; x < kTailRest; ++x) rs += rsp[x * kPredLog + lane];
    const float cproj = craw - centre * rs;
#pragma unroll
    for (uint32_t dst = 0; dst < kTailCtas; ++dst)
      st_cluster(sf + kPredPos * (kPredConf + kPredHid) + p * kPredLog + lane, dst, cproj);
  }
  tail_cluster_sync();                                      // the feature vector is complete in all four CTAs
  if (rank == 0 && m.features_out)
    for (int x = tid; x < kPredFeatures; x += kTailThreads) m.features_out[(size_t)i * kPredFeatures + x] = sf[x];
  {
    // ---- warp w: hidden unit 16 rank + w from this CTA's rows of W1
    bool have = bulk && mbar_wait(bar, 0, s_abort);
    const float* wrow = have ? w1s + warp * kPredFeatures : m.w1 + (size_t)unit * kPredFeatures;
    float acc = 0.f;
#pragma unroll 8
    for (int x = lane; x < kPredFeatures; x += 32) acc = fmaf(wrow[x], sf[x], acc);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) st_cluster(sh + unit, 0, fmaxf(acc + b1v, 0.f));
    if (bulk && !have) {
      // the copy did not land within the limit: flag it, and do not leave while it may still be writing
      if (lane == 0) atomicOr(m.status, 8 /*TIMEOUT*/);
      volatile int again = 0;
      mbar_wait(bar, 0, &again);
    }
  }
  tail_cluster_sync();                                      // all 64 hidden units are in CTA 0
  if (rank == 0 && warp < kPredPos) {
    const float* w = m.w2 + warp * kPredMlp;
    float acc = w[lane] * sh[lane] + w[lane + 32] * sh[lane + 32];
#pragma unroll
    for (int x = 16; x > 0; x >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, x);
    if (lane == 0) m.pred_logits[i * kPredPos + warp] = acc + m.b2[warp];
  }
}

}  // namespace

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                  const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                  const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn pred_encode_fn() {
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
// row-major [rows][inner] matrix with a row pitch, box [box_rows][box_inner], 128-byte swizzle
static bool pred_encode(CUtensorMap* out, CUtensorMapDataType dt, const void* ptr, uint64_t inner, uint64_t rows,
                        uint64_t pitch_bytes, uint32_t box_inner, uint32_t box_rows) {
  EncodeTiledFn enc = pred_encode_fn();
  if (!enc) return false;
  cuuint64_t dims[2] = {inner, rows};
  cuuint64_t strides[1] = {pitch_bytes};
  cuuint32_t box[2] = {box_inner, box_rows};
  cuuint32_t es[2] = {1, 1};
  return enc(out, dt, 2, const_cast<void*>(ptr), dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
             CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

cudaError_t predictor_prepare() {
  cudaError_t e = cudaFuncSetAttribute(pred_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kStreamSmem);
  if (e != cudaSuccess) return e;
  return cudaFuncSetAttribute(pred_tail_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kTailSmem);
}

int predictor_chunks(int n_bs, int vocab, int num_ctas, int* chunk_len_out) {
  const int row_groups = (kPredPos * n_bs + kRowsPerCta - 1) / kRowsPerCta;
  // one CTA per SM, a single wave; about one SM in sixteen is left to the hidden-state projection
  const int spare = num_ctas / 16 > 1 ? num_ctas / 16 : 1;
  int chunks = (num_ctas - spare) / row_groups;
  chunks = chunks < 1 ? 1 : (chunks > kPredMaxChunks ? kPredMaxChunks : chunks);
  int chunk_len = (vocab + chunks - 1) / chunks;
  chunk_len = (chunk_len + kSub - 1) / kSub * kSub;
  chunks = (vocab + chunk_len - 1) / chunk_len;
  if (chunk_len_out) *chunk_len_out = chunk_len;
  return chunks;
}

cudaError_t launch_predictor(const PredictArgs& p, cudaStream_t stream) {
  WsLayout L = ws_layout(p.n_bs, p.n_kv_heads, p.num_ctas);
  int chunk_len = 0;
  const int chunks = predictor_chunks(p.n_bs, p.vocab, p.num_ctas, &chunk_len);
  float* part = ws_ptr<float>(p.ws, L.pred_part);
  float* rowsum = ws_ptr<float>(p.ws, L.pred_rowsum);
  float* feat = ws_ptr<float>(p.ws, L.pred_feat);
  const int row_groups = (kPredPos * p.n_bs + kRowsPerCta - 1) / kRowsPerCta;

  const int stream_ctas = chunks * row_groups;
  // the hidden-state projection: the SMs the stream leaves free, but no more CTAs than jobs
  const int hid_items = (kPredPos * p.n_bs + 15) / 16 * kHidSlices;
  int hid_ctas = p.num_ctas - stream_ctas;
  hid_ctas = hid_ctas < 1 ? 1 : hid_ctas;
  hid_ctas = hid_ctas > (hid_items + kHidJobs - 1) / kHidJobs ? (hid_items + kHidJobs - 1) / kHidJobs : hid_ctas;
  StreamArgs sa{p.draft_logits, p.ld, p.vocab, p.n_live, p.n_bs,
                reinterpret_cast<const __nv_bfloat16*>(p.p_logit), part, rowsum, chunks, chunk_len,
                stream_ctas, ws_ptr<int>(p.ws, L.hdr) + H_STATUS,
                reinterpret_cast<const __nv_bfloat16*>(p.draft_hidden), p.hidden_dim,
                reinterpret_cast<const __nv_bfloat16*>(p.p_hidden), feat};
  CUtensorMap tz, tp;
  if (!pred_encode(&tz, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, p.draft_logits, (uint64_t)p.vocab,
                   (uint64_t)kPredPos * p.n_bs, (uint64_t)p.ld * 4, 32, kRowsPerCta))
    return cudaErrorNotSupported;
  if ((p.vocab & 7) == 0) {
    if (!pred_encode(&tp, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, p.p_logit, (uint64_t)p.vocab, kPredLog,
                     (uint64_t)p.vocab * 2, 64, kPredLog))
      return cudaErrorNotSupported;
  } else {
    tp = tz;                                            // never used: odd vocabularies stage the matrix by hand
  }
  FeatArgs fa{p.draft_logits, p.ld, p.vocab, p.n_live, p.n_bs,
              reinterpret_cast<const __nv_bfloat16*>(p.draft_hidden), p.hidden_dim,
              reinterpret_cast<const __nv_bfloat16*>(p.p_hidden), part, rowsum, chunks, feat};
  // Two launches.  The stream grid carries the hidden-state projection on the CTAs behind its
  // (row group, chunk) CTAs; the tail kernel (feature merge + perceptron) is launched with
  // programmatic stream serialisation and does everything that depends only on the call's
  // inputs while the stream is still running.
  pred_stream_kernel<<<dim3(stream_ctas + hid_ctas), kStreamThreads, kStreamSmem, stream>>>(sa, tz, tp);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  MlpArgs ma{p.n_live, p.n_bs, feat, p.w1, p.b1, p.w2, p.b2, p.pred_logits, p.features_out,
             ws_ptr<int>(p.ws, L.hdr) + H_STATUS};
  {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(kTailCtas * p.n_bs);
    cfg.blockDim = dim3(kTailThreads);
    cfg.dynamicSmemBytes = kTailSmem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    e = cudaLaunchKernelEx(&cfg, pred_tail_kernel, fa, ma);
  }
  return e;
}

#ifdef DSCALE_WAIT_TEST
// Wait-limit test build only: leave out the logit copies of sub-tile `sub` of CTA `cta` of the
// predictor's stream kernel in every following launch; (-1, -1) switches it off.  HOST call.
extern "C" int dscale_test_drop_pred_copy(int cta, int sub) {
  if (cudaMemcpyToSymbol(g_pred_drop_cta, &cta, sizeof(int)) != cudaSuccess) return -3;
  if (cudaMemcpyToSymbol(g_pred_drop_sub, &sub, sizeof(int)) != cudaSuccess) return -3;
  return 0;
}
#endif

}  // namespace dscale
