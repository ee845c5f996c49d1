// Greedy prefix verification: vocabulary argmax per packed row, then the
// accepted-prefix scan per request, in one launch.
//
// The argmax is a pure HBM stream (8N rows x vocab fp32 read once).  The live logits are
// taken as one ragged sequence of 16-byte vectors (row-major, ceil(vocab / 4) per row) and cut
// into one equal span per warp of a grid of two 512-thread CTAs per SM: every warp streams
// its span with 128-bit read-only loads that bypass L1, eight in flight per lane (128 KB in
// flight per SM), keeps a per-thread running (max, first index), and at the end of a row
// segment reduces it with warp shuffles and folds it into the row's 64-bit key in the
// workspace with one atomicMax: key = (order-preserving bits of the value, ~index), so that the
// largest key is the largest value and, among equal values, the lowest index.  A NaN or
// -inf is never offered, an untouched key (0) means token 0.  No partial arrays, no block
// barrier in the stream.  The last CTA to finish (a ticket in the workspace header, no
// waiting) turns the keys into target tokens, clears them for the next launch, and
// runs the sequential acceptance loop of the "Prefix verifier" paragraph with
// one thread per request (on shared-memory copies of the row results and the
// packed tokens), writing the outputs of Algorithm 2, lines 21-26.
// M_live is read on the device, so the same captured launch serves every N <= n_bs.
#include <cfloat>
#include <climits>

#include "kernels.cuh"

namespace dscale {

namespace {

constexpr int kAccThreads = 512;

struct Best {
  float v;
  int i;
};

__device__ __forceinline__ void take(Best& b, float v, int i) {
  // strict '>' with indices visited in increasing order keeps the first maximum;
  // a NaN compares false and is never taken
  if (v > b.v) { b.v = v; b.i = i; }
}
__device__ __forceinline__ Best merge(Best a, Best b) {
  if (b.v > a.v || (b.v == a.v && b.i < a.i)) return b;
  return a;
}

__device__ __forceinline__ float4 ldg_stream(const float4* p) {
  float4 r;
  asm volatile("ld.global.nc.L1::no_allocate.v4.f32 {%0,%1,%2,%3}, [%4];"
               : "=f"(r.x), "=f"(r.y), "=f"(r.z), "=f"(r.w)
               : "l"(p));
  return r;
}

__device__ __forceinline__ unsigned long long key_of(float v, int i) {
  unsigned u = v == 0.0f ? 0u : __float_as_uint(v);    // -0 and +0 are one value
  u ^= (u >> 31) ? 0xffffffffu : 0x80000000u;          // unsigned order = float order
  return ((unsigned long long)u << 32) | (unsigned)(~i);
}

__global__ void __launch_bounds__(kAccThreads, 2) accept_kernel(AcceptArgs a, WsLayout L) {
  int* hdr = ws_ptr<int>(a.ws, L.hdr);
  const int m_live = hdr[H_M_LIVE];
  const int tid = threadIdx.x, lane = tid & 31;
  unsigned long long* row_key = ws_ptr<unsigned long long>(a.ws, L.amax_val);   // [8 n_bs], 0 = untouched
  __shared__ int sLast;
  // The acceptance loop at the end is a chain of dependent reads: it runs on shared-memory copies
  // of the per-row results and of the packed tokens, lengths and offsets.  The copies of the
  // allocation's outputs are fetched now, by every CTA (2 KB, from L2), so that the one CTA that
  // ends up last does not start a round of loads when everybody else has already left.
  __shared__ int s_top1[kHalfW * kMaxNbs];
  __shared__ int s_tok[kHalfW * kMaxNbs];
  __shared__ int s_k[kMaxNbs], s_off[kMaxNbs];
  {
    const int* wtok = ws_ptr<int>(a.ws, L.tokens);
    const int* wk = ws_ptr<int>(a.ws, L.k);
    const int* woff = ws_ptr<int>(a.ws, L.offset);
    for (int r = tid; r < kHalfW * a.n_bs; r += kAccThreads) s_tok[r] = wtok[r];
    for (int r = tid; r < a.n_bs; r += kAccThreads) { s_k[r] = wk[r]; s_off[r] = woff[r]; }
  }

  // this warp's span of the ragged vector sequence
  const long long nv = (a.vocab + 3) >> 2;                      // vectors per row
  const long long total = nv * m_live;
  const long long n_warps = (long long)gridDim.x * (kAccThreads / 32);
  const long long w = (long long)blockIdx.x * (kAccThreads / 32) + (tid >> 5);
  long long pos = total * w / n_warps;
  const long long end = total * (w + 1) / n_warps;
  while (pos < end) {
    const int s = (int)(pos / nv);
    const int v0 = (int)(pos - (long long)s * nv);
    const int v1 = (int)min(nv, v0 + (end - pos));                // segment [v0, v1) of row s
    const float4* p4 = reinterpret_cast<const float4*>(a.logits + (size_t)s * a.ld);
    const bool ragged = (a.vocab & 3) && v1 == nv;                // the row's last vector is partly padding
    const int v1_full = ragged ? v1 - 1 : v1;
    Best b{-INFINITY, INT_MAX};
    int x = v0 + lane;
    for (; x + 7 * 32 < v1_full; x += 8 * 32) {                   // eight 128-bit loads in flight
      float4 v[8];
#pragma unroll
      for (int q = 0; q < 8; ++q) v[q] = ldg_stream(p4 + x + q * 32);
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        const int e = 4 * (x + q * 32);
        take(b, v[q].x, e); take(b, v[q].y, e + 1); take(b, v[q].z, e + 2); take(b, v[q].w, e + 3);
      }
    }
    for (; x < v1_full; x += 32) {
      const float4 v = ldg_stream(p4 + x);
      const int e = 4 * x;
      take(b, v.x, e); take(b, v.y, e + 1); take(b, v.z, e + 2); take(b, v.w, e + 3);
    }
    if (ragged && lane == 0) {
      const float* row = a.logits + (size_t)s * a.ld;
      for (int e = 4 * v1_full; e < a.vocab; ++e) take(b, row[e], e);
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
      Best o{__shfl_xor_sync(0xffffffffu, b.v, d), __shfl_xor_sync(0xffffffffu, b.i, d)};
      b = merge(b, o);
    }
    if (lane == 0 && b.i != INT_MAX) atomicMax(&row_key[s], key_of(b.v, b.i));
    pos += v1 - v0;
  }
  __threadfence();
  __syncthreads();
  if (tid == 0) sLast = (atomicAdd(&hdr[H_ACCEPT_TICKET], 1) == (int)gridDim.x - 1);
  __syncthreads();
  if (!sLast) return;

  // ---- last block: keys -> target tokens, then the acceptance loop ----------
  __threadfence();
  if (tid == 0) hdr[H_ACCEPT_TICKET] = 0;           // ready for the next replay
  const int n_bs = a.n_bs;
  const int m_bs = kHalfW * n_bs;
  int* top1 = ws_ptr<int>(a.ws, L.top1);
  for (int r = tid; r < m_bs; r += kAccThreads) {
    int best = 0;
    if (r < m_live) {
      const unsigned long long key = __ldcg(&row_key[r]);
      if (key != 0ull) best = (int)~(unsigned)(key & 0xffffffffull);   // untouched: no entry beat -inf
      row_key[r] = 0ull;                            // ready for the next replay
    }
    top1[r] = best;
    s_top1[r] = best;
  }
  __syncthreads();
  const int N = hdr[H_N_LIVE];
  for (int i = tid; i < n_bs; i += kAccThreads) {
    int* ot = a.out_tokens + i * kW;
    if (i < N) {
      const int ki = s_k[i], oi = s_off[i];
      int acc = 0;
      while (acc < ki - 1 && s_top1[oi + acc] == s_tok[oi + acc + 1]) ++acc;
      const int nxt = s_top1[oi + acc];
      for (int jj = 0; jj < kW; ++jj)
        ot[jj] = jj < acc ? s_tok[oi + 1 + jj] : (jj == acc ? nxt : -1);
      a.accept_len[i] = acc;
      a.next_anchor[i] = nxt;
      a.out_len[i] = acc + 1;
      if (a.ctx_len_inout) a.ctx_len_inout[i] += acc + 1;
    } else {
      for (int jj = 0; jj < kW; ++jj) ot[jj] = -1;
      a.accept_len[i] = 0;
      a.next_anchor[i] = -1;
      a.out_len[i] = 0;
    }
  }
}

}  // namespace

cudaError_t launch_accept(const AcceptArgs& a, cudaStream_t stream) {
  WsLayout L = ws_layout(a.n_bs, a.n_kv_heads, a.num_ctas);
  // two CTAs per SM; small problems get fewer, so that a warp's span is at least 4 KB
  const long long vecs = (long long)((a.vocab + 3) >> 2) * kHalfW * a.n_bs;
  long long ctas = vecs / (256 * (kAccThreads / 32));
  ctas = ctas < 1 ? 1 : (ctas > 2LL * a.num_ctas ? 2LL * a.num_ctas : ctas);
  accept_kernel<<<dim3((unsigned)ctas), kAccThreads, 0, stream>>>(a, L);
  return cudaGetLastError();
}

}  // namespace dscale
