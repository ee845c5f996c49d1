// Prefix verification under a sampling target policy (temperature > 0).
//
// P = softmax(logits / T) at every packed row.  The candidate of slot j + 1 is
// accepted with probability P(x) (uniform u_accept of row j); at the first
// rejection the successor is drawn from P with x removed and renormalised, and
// if all selected candidates pass it is drawn from the unmodified P of the last
// selected row ("Prefix verifier" paragraph).  The random numbers are inputs.
//
// Two launches, both pure streams over the logits:
//   1. sample_stats_kernel, grid (vocab chunks, packed rows): running (max, sum)
//      of 2^(l * log2e / T) per chunk; the last block to finish (ticket) combines
//      the chunks per row, evaluates P(x) and the acceptance test of every row,
//      and scans each request for its first rejection.
//   2. sample_draw_kernel, one block per request: inverse-CDF draw on the row that
//      supplies the successor -- per-warp totals over 32 contiguous ranges, the
//      warp holding the target, then 32-wide shuffle scans inside its range.
#include <climits>

#include "kernels.cuh"

namespace dscale {

namespace {

constexpr int kStatThreads = 256;
constexpr int kDrawThreads = 1024;

struct MS { float m, s; };   // running maximum (log2 domain) and sum of 2^(z - m)

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ void ms_add(MS& a, float z) {
  if (z > a.m) { a.s = a.s * ex2f(a.m - z) + 1.0f; a.m = z; }
  else a.s += ex2f(z - a.m);
}
__device__ __forceinline__ MS ms_merge(MS a, MS b) {
  const float m = fmaxf(a.m, b.m);
  if (m == -INFINITY) return MS{-INFINITY, 0.0f};
  return MS{m, a.s * ex2f(a.m - m) + b.s * ex2f(b.m - m)};
}

__global__ void __launch_bounds__(kStatThreads)
sample_stats_kernel(SampleArgs a, WsLayout L, int chunks, int chunk_len) {
  int* hdr = ws_ptr<int>(a.ws, L.hdr);
  const int m_live = hdr[H_M_LIVE];
  const int s = blockIdx.y;
  if (s >= m_live) return;
  const int c = blockIdx.x, tid = threadIdx.x;
  float* pm = ws_ptr<float>(a.ws, L.smp_m);
  float* ps = ws_ptr<float>(a.ws, L.smp_s);
  const float scale = 1.4426950408889634f / a.temperature;

  const float* row = a.logits + (size_t)s * a.ld;
  const int lo = c * chunk_len;
  const int hi = min(a.vocab, lo + chunk_len);
  MS acc{-INFINITY, 0.0f};
  if (lo < hi) {
    const int n4 = (hi - lo) >> 2;
    const float4* p4 = reinterpret_cast<const float4*>(row + lo);
    // batches of 8 x 128-bit loads per thread: all loads of a batch are in flight
    // together, then one maximum and one branch-free sum per batch
    for (int x0 = tid; x0 < n4; x0 += 8 * kStatThreads) {
      float4 v[8];
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        const int x = x0 + j * kStatThreads;
        v[j] = x < n4 ? __ldg(p4 + x) : make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
      }
      float m = -INFINITY;
#pragma unroll
      for (int j = 0; j < 8; ++j) m = fmaxf(m, fmaxf(fmaxf(v[j].x, v[j].y), fmaxf(v[j].z, v[j].w)));
      m *= scale;
      float s0 = 0.0f, s1 = 0.0f, s2 = 0.0f, s3 = 0.0f;
#pragma unroll
      for (int j = 0; j < 8; ++j) {
        s0 += ex2f(fmaf(v[j].x, scale, -m)); s1 += ex2f(fmaf(v[j].y, scale, -m));
        s2 += ex2f(fmaf(v[j].z, scale, -m)); s3 += ex2f(fmaf(v[j].w, scale, -m));
      }
      acc = ms_merge(acc, MS{m, (s0 + s1) + (s2 + s3)});
    }
    for (int e = lo + 4 * n4 + tid; e < hi; e += kStatThreads) ms_add(acc, row[e] * scale);
  }
#pragma unroll
  for (int d = 16; d > 0; d >>= 1)
    acc = ms_merge(acc, MS{__shfl_xor_sync(0xffffffffu, acc.m, d), __shfl_xor_sync(0xffffffffu, acc.s, d)});
  __shared__ float sm_m[kStatThreads / 32], sm_s[kStatThreads / 32];
  __shared__ int s_last;
  if ((tid & 31) == 0) { sm_m[tid >> 5] = acc.m; sm_s[tid >> 5] = acc.s; }
  __syncthreads();
  if (tid == 0) {
    for (int w = 1; w < kStatThreads / 32; ++w) acc = ms_merge(acc, MS{sm_m[w], sm_s[w]});
    pm[(size_t)s * kAccMaxChunks + c] = acc.m;
    ps[(size_t)s * kAccMaxChunks + c] = acc.s;
    __threadfence();
    s_last = (atomicAdd(&hdr[H_SAMPLE_TICKET], 1) == chunks * m_live - 1);
  }
  __syncthreads();
  if (!s_last) return;

  // ---- last block: per-row totals, acceptance tests, first rejection per request
  __threadfence();
  if (tid == 0) hdr[H_SAMPLE_TICKET] = 0;
  float* row_m = ws_ptr<float>(a.ws, L.row_m);
  float* row_z = ws_ptr<float>(a.ws, L.row_z);
  int* row_flag = ws_ptr<int>(a.ws, L.row_flag);
  const int* wk = ws_ptr<int>(a.ws, L.k);
  const int* woff = ws_ptr<int>(a.ws, L.offset);
  const int* wtok = ws_ptr<int>(a.ws, L.tokens);
  const int* wreq = ws_ptr<int>(a.ws, L.row_req);
  for (int r = tid; r < m_live; r += kStatThreads) {
    MS t{-INFINITY, 0.0f};
    for (int cc = 0; cc < chunks; ++cc)
      t = ms_merge(t, MS{__ldcg(&pm[(size_t)r * kAccMaxChunks + cc]), __ldcg(&ps[(size_t)r * kAccMaxChunks + cc])});
    row_m[r] = t.m;
    row_z[r] = t.s;
    const int i = wreq[r];
    const int j = r - woff[i];
    float p = 0.0f;
    if (j < wk[i] - 1) {                                   // the row has a candidate to judge
      const int x = wtok[r + 1];
      p = exp2f(a.logits[(size_t)r * a.ld + x] * scale - t.m) / t.s;
    }
    row_flag[r] = a.u_accept[r] < p;
    if (a.p_draft) a.p_draft[r] = p;
  }
  __syncthreads();
  const int N = hdr[H_N_LIVE];
  if (tid < a.n_bs) {
    const int i = tid;
    int* req_row = ws_ptr<int>(a.ws, L.req_row);
    int* req_rej = ws_ptr<int>(a.ws, L.req_rej);
    if (i < N) {
      const int ki = wk[i], oi = woff[i];
      int acc_n = 0;
      while (acc_n < ki - 1 && row_flag[oi + acc_n]) ++acc_n;
      req_row[i] = oi + acc_n;
      req_rej[i] = acc_n < ki - 1 ? wtok[oi + acc_n + 1] : -1;
      a.accept_len[i] = acc_n;
    } else {
      req_row[i] = -1;
      req_rej[i] = -1;
      a.accept_len[i] = 0;
    }
  }
}

__global__ void __launch_bounds__(kDrawThreads) sample_draw_kernel(SampleArgs a, WsLayout L) {
  const int i = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int* hdr = ws_ptr<int>(a.ws, L.hdr);
  const int N = hdr[H_N_LIVE];
  int32_t* ot = a.out_tokens + i * kW;
  if (i >= N) {
    if (tid < kW) ot[tid] = -1;
    if (tid == 0) { a.next_anchor[i] = -1; a.out_len[i] = 0; }
    return;
  }
  const int r = ws_ptr<int>(a.ws, L.req_row)[i];
  const int xrej = ws_ptr<int>(a.ws, L.req_rej)[i];
  const float M = ws_ptr<float>(a.ws, L.row_m)[r];
  const float scale = 1.4426950408889634f / a.temperature;
  const float* row = a.logits + (size_t)r * a.ld;
  const int V = a.vocab;
  const int R = (((V + 31) / 32) + 127) & ~127;             // elements per warp range, multiple of 128
  const int lo = warp * R, hi = min(V, lo + R);
  auto weight = [&](int v) { return v == xrej ? 0.0f : ex2f(row[v] * scale - M); };

  // range totals: 128-bit loads (rows are 16-byte aligned, R is a multiple of 4)
  float part = 0.0f;
  {
    const int n4 = hi > lo ? (hi - lo) >> 2 : 0;
    const float4* p4 = reinterpret_cast<const float4*>(row + lo);
    float p0 = 0.0f, p1 = 0.0f, p2 = 0.0f, p3 = 0.0f;
    for (int x = lane; x < n4; x += 32) {
      const float4 q = __ldg(p4 + x);
      const int v = lo + 4 * x;
      p0 += v == xrej ? 0.0f : ex2f(q.x * scale - M);
      p1 += v + 1 == xrej ? 0.0f : ex2f(q.y * scale - M);
      p2 += v + 2 == xrej ? 0.0f : ex2f(q.z * scale - M);
      p3 += v + 3 == xrej ? 0.0f : ex2f(q.w * scale - M);
    }
    part = (p0 + p1) + (p2 + p3);
    for (int v = lo + 4 * n4 + lane; v < hi; v += 32) part += weight(v);
  }
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) part += __shfl_xor_sync(0xffffffffu, part, d);
  __shared__ float s_wt[32];
  __shared__ int s_pick;
  if (lane == 0) s_wt[warp] = part;
  if (tid == 0) s_pick = -1;
  __syncthreads();
  // every thread scans the 32 warp totals in order (same arithmetic everywhere)
  float total = 0.0f;
  for (int w = 0; w < 32; ++w) total += s_wt[w];
  const float target = a.u_draw[i] * total;
  int w_star = -1;
  float before = 0.0f;
  {
    float run = 0.0f;
    for (int w = 0; w < 32; ++w) {
      if (w_star < 0 && s_wt[w] > 0.0f && run + s_wt[w] > target) { w_star = w; before = run; }
      run += s_wt[w];
    }
    if (w_star < 0)                                          // rounding at the very end: last non-empty range
      for (int w = 31; w >= 0; --w) if (s_wt[w] > 0.0f) { w_star = w; before = total - s_wt[w]; break; }
  }
  // The target lies in warp range w_star.  All warps now work on that range: totals of
  // its 32-element groups, then one warp locates the group, then the element.
  __shared__ float s_gt[1024];
  const int lo_s = w_star * R, hi_s = min(V, lo_s + R);
  const int n_groups = (hi_s - lo_s + 31) / 32;              // <= 1024 for vocab <= 2^20
  for (int g = warp; g < n_groups; g += 32) {
    const int v = lo_s + 32 * g + lane;
    float wv = v < hi_s ? weight(v) : 0.0f;
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) wv += __shfl_xor_sync(0xffffffffu, wv, d);
    if (lane == 0) s_gt[g] = wv;
  }
  __syncthreads();
  if (warp == 0) {
    float rem = target - before;
    int group = -1, last_group = -1;
    for (int g0 = 0; g0 < n_groups && group < 0; g0 += 32) {
      const float gv = g0 + lane < n_groups ? s_gt[g0 + lane] : 0.0f;
      float cum = gv;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const float u = __shfl_up_sync(0xffffffffu, cum, d);
        if (lane >= d) cum += u;
      }
      const unsigned hit = __ballot_sync(0xffffffffu, gv > 0.0f && cum > rem);
      const unsigned pos = __ballot_sync(0xffffffffu, gv > 0.0f);
      if (pos) last_group = g0 + 31 - __clz(pos);
      if (hit) {
        group = g0 + __ffs(hit) - 1;
        rem -= __shfl_sync(0xffffffffu, cum - gv, __ffs(hit) - 1);   // weight before that group
      } else {
        rem -= __shfl_sync(0xffffffffu, cum, 31);
      }
    }
    if (group < 0) { group = last_group; rem = INFINITY; }     // rounding: last group with weight
    // the element inside the group
    int pick = -1;
    if (group >= 0) {
      const int v = lo_s + 32 * group + lane;
      const float wv = v < hi_s ? weight(v) : 0.0f;
      float cum = wv;
#pragma unroll
      for (int d = 1; d < 32; d <<= 1) {
        const float u = __shfl_up_sync(0xffffffffu, cum, d);
        if (lane >= d) cum += u;
      }
      const unsigned hit = __ballot_sync(0xffffffffu, wv > 0.0f && cum > rem);
      const unsigned pos = __ballot_sync(0xffffffffu, wv > 0.0f);
      if (hit) pick = lo_s + 32 * group + __ffs(hit) - 1;
      else if (pos) pick = lo_s + 32 * group + 31 - __clz(pos);  // rounding: last token with weight
    }
    if (lane == 0) s_pick = pick;
  }
  __syncthreads();
  const int nxt = s_pick < 0 ? 0 : s_pick;
  const int acc_n = a.accept_len[i];
  const int oi = ws_ptr<int>(a.ws, L.offset)[i];
  const int* wtok = ws_ptr<int>(a.ws, L.tokens);
  if (tid < kW) ot[tid] = tid < acc_n ? wtok[oi + 1 + tid] : (tid == acc_n ? nxt : -1);
  if (tid == 0) { a.next_anchor[i] = nxt; a.out_len[i] = acc_n + 1; }
}

}  // namespace

cudaError_t launch_accept_sampling(const SampleArgs& a, cudaStream_t stream) {
  WsLayout L = ws_layout(a.n_bs, a.n_kv_heads, a.num_ctas);
  int chunks = a.vocab / 16384;
  chunks = chunks < 1 ? 1 : (chunks > kAccMaxChunks ? kAccMaxChunks : chunks);
  int chunk_len = ((a.vocab + chunks - 1) / chunks + 3) & ~3;
  sample_stats_kernel<<<dim3(chunks, kHalfW * a.n_bs), kStatThreads, 0, stream>>>(a, L, chunks, chunk_len);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  sample_draw_kernel<<<a.n_bs, kDrawThreads, 0, stream>>>(a, L);
  return cudaGetLastError();
}

}  // namespace dscale
