// Greedy prefix verification: vocabulary argmax per packed row, then the
// accepted-prefix scan per request, in one launch.
//
// The argmax is a pure HBM stream (8N rows x vocab fp32 read once).  The grid
// is (vocab chunks, 8 n_bs rows); a block streams its chunk with 128-bit
// read-only loads that bypass L1, up to eight loads in flight per thread, keeps a
// per-thread running (max, first index), reduces it with warp shuffles and
// writes one partial to the workspace.  The last block to finish (a ticket in
// the workspace header, no waiting) merges the partials in chunk order and
// runs the sequential acceptance loop of the "Prefix verifier" paragraph with
// one thread per request (on shared-memory copies of the row results and the
// packed tokens), writing the outputs of Algorithm 2, lines 21-26.  (One warp
// per (row, chunk) without any block barrier was tried and is slower: 49 vs 39 us.)
// Rows at or beyond M_live = 8N (read on the device) exit immediately, so the
// same captured launch serves every N <= n_bs.
#include <cfloat>
#include <climits>

#include "kernels.cuh"

namespace dscale {

namespace {

constexpr int kAccThreads = 256;

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

__global__ void __launch_bounds__(kAccThreads) accept_kernel(AcceptArgs a, WsLayout L, int chunks,
                                                             int chunk_len) {
  int* hdr = ws_ptr<int>(a.ws, L.hdr);
  const int m_live = hdr[H_M_LIVE];
  const int s = blockIdx.y;
  if (s >= m_live) return;
  const int c = blockIdx.x;
  const int tid = threadIdx.x;
  float* pval = ws_ptr<float>(a.ws, L.amax_val);
  int* pidx = ws_ptr<int>(a.ws, L.amax_idx);

  const float* row = a.logits + (size_t)s * a.ld;
  const int lo = c * chunk_len;
  const int hi = min(a.vocab, lo + chunk_len);
  Best b{-INFINITY, INT_MAX};
  if (lo < hi) {
    const int n4 = (hi - lo) >> 2;                  // chunk_len % 4 == 0, row 16-byte aligned
    const float4* p4 = reinterpret_cast<const float4*>(row + lo);
    int x = tid;
    for (; x + 7 * kAccThreads < n4; x += 8 * kAccThreads) {      // eight 128-bit loads in flight
      float4 v[8];
#pragma unroll
      for (int q = 0; q < 8; ++q) v[q] = ldg_stream(p4 + x + q * kAccThreads);
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        const int e = lo + 4 * (x + q * kAccThreads);
        take(b, v[q].x, e); take(b, v[q].y, e + 1); take(b, v[q].z, e + 2); take(b, v[q].w, e + 3);
      }
    }
    for (; x + 3 * kAccThreads < n4; x += 4 * kAccThreads) {
      float4 v0 = ldg_stream(p4 + x);
      float4 v1 = ldg_stream(p4 + x + kAccThreads);
      float4 v2 = ldg_stream(p4 + x + 2 * kAccThreads);
      float4 v3 = ldg_stream(p4 + x + 3 * kAccThreads);
      int e = lo + 4 * x;
      take(b, v0.x, e); take(b, v0.y, e + 1); take(b, v0.z, e + 2); take(b, v0.w, e + 3);
      e += 4 * kAccThreads;
      take(b, v1.x, e); take(b, v1.y, e + 1); take(b, v1.z, e + 2); take(b, v1.w, e + 3);
      e += 4 * kAccThreads;
      take(b, v2.x, e); take(b, v2.y, e + 1); take(b, v2.z, e + 2); take(b, v2.w, e + 3);
      e += 4 * kAccThreads;
      take(b, v3.x, e); take(b, v3.y, e + 1); take(b, v3.z, e + 2); take(b, v3.w, e + 3);
    }
    for (; x < n4; x += kAccThreads) {
      float4 v0 = ldg_stream(p4 + x);
      const int e = lo + 4 * x;
      take(b, v0.x, e); take(b, v0.y, e + 1); take(b, v0.z, e + 2); take(b, v0.w, e + 3);
    }
    for (int e = lo + 4 * n4 + tid; e < hi; e += kAccThreads) take(b, row[e], e);
  }
  // warp-shuffle reduction, then across the 8 warps
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) {
    Best o{__shfl_xor_sync(0xffffffffu, b.v, d), __shfl_xor_sync(0xffffffffu, b.i, d)};
    b = merge(b, o);
  }
  __shared__ float sv[kAccThreads / 32];
  __shared__ int si[kAccThreads / 32];
  __shared__ int sLast;
  if ((tid & 31) == 0) { sv[tid >> 5] = b.v; si[tid >> 5] = b.i; }
  __syncthreads();
  if (tid == 0) {
    for (int w = 1; w < kAccThreads / 32; ++w) b = merge(b, Best{sv[w], si[w]});
    pval[(size_t)s * kAccMaxChunks + c] = b.v;
    pidx[(size_t)s * kAccMaxChunks + c] = b.i;
    __threadfence();
    const int ticket = atomicAdd(&hdr[H_ACCEPT_TICKET], 1);
    sLast = (ticket == chunks * m_live - 1);
  }
  __syncthreads();
  if (!sLast) return;

  // ---- last block: merge partials, then the acceptance loop ----------------
  __threadfence();
  if (tid == 0) hdr[H_ACCEPT_TICKET] = 0;           // ready for the next replay
  const int n_bs = a.n_bs;
  const int m_bs = kHalfW * n_bs;
  // The acceptance loop is a chain of dependent reads: run it on shared-memory copies
  // of the per-row results and the packed tokens, not on global memory.
  __shared__ int s_top1[kHalfW * kMaxNbs];
  __shared__ int s_tok[kHalfW * kMaxNbs];
  int* top1 = ws_ptr<int>(a.ws, L.top1);
  const int* wtok = ws_ptr<int>(a.ws, L.tokens);
  for (int r = tid; r < m_bs; r += kAccThreads) {
    int best = 0;
    if (r < m_live) {
      Best bb{-INFINITY, INT_MAX};
      for (int cc = 0; cc < chunks; ++cc) {
        Best o{__ldcg(&pval[(size_t)r * kAccMaxChunks + cc]),
               __ldcg(&pidx[(size_t)r * kAccMaxChunks + cc])};
        bb = merge(bb, o);
      }
      best = bb.i == INT_MAX ? 0 : bb.i;            // row without any finite / -inf-beating entry
    }
    top1[r] = best;
    s_top1[r] = best;
    s_tok[r] = wtok[r];
  }
  __syncthreads();
  const int N = hdr[H_N_LIVE];
  const int* wk = ws_ptr<int>(a.ws, L.k);
  const int* woff = ws_ptr<int>(a.ws, L.offset);
  for (int i = tid; i < n_bs; i += kAccThreads) {
    int* ot = a.out_tokens + i * kW;
    if (i < N) {
      const int ki = wk[i], oi = woff[i];
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
  int chunks = a.vocab / 16384;
  chunks = chunks < 1 ? 1 : (chunks > kAccMaxChunks ? kAccMaxChunks : chunks);
  int chunk_len = (a.vocab + chunks - 1) / chunks;
  chunk_len = (chunk_len + 3) & ~3;
  dim3 grid(chunks, kHalfW * a.n_bs);
  accept_kernel<<<grid, kAccThreads, 0, stream>>>(a, L, chunks, chunk_len);
  return cudaGetLastError();
}

}  // namespace dscale
