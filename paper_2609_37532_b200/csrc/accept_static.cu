// dscale_accept_static: greedy prefix verification with no workspace and no
// allocation of any kind.
//
// Some callers cannot hand this library a workspace or let it allocate one: a
// serving loop in which cudaMalloc would stall every stream of the device, or a
// plug-in that is given raw input / output pointers by its host runtime and no
// allocator.  For them the scratch the row argmax needs (per-chunk partial
// maxima, the per-row result and the arrival ticket) lives in a file-scope
// __device__ array below, of fixed size, held by every GPU that loads the
// library until the process exits.  The caller passes only inputs and outputs.
//
// Consequences of sharing one array:
//   * calls that overlap on the GPU (different streams, or different host
//     threads) race on it -- serialise them;
//   * the array keeps what the previous call left in it; the ticket word that
//     must start at zero is cleared on the stream at the start of every call;
//   * the first call on each device looks up the array's device address
//     (cudaGetSymbolAddress) -- make that first call outside any stream capture.
#include <cuda_runtime.h>

#include <cfloat>
#include <climits>
#include <mutex>

#include "../../include/dscale.h"

namespace {

constexpr int kW = 16, kHalfW = 8;
constexpr int kMaxRows = kHalfW * DSCALE_MAX_NBS;       // 512 packed rows
constexpr int kMaxChunks = 16;
constexpr int kThreads = 256;
constexpr int kMaxDevices = 64;

// scratch layout (bytes): [0,256) ticket | partial values | partial indices | top1
constexpr size_t kOffVal = 256;
constexpr size_t kOffIdx = kOffVal + size_t(kMaxRows) * kMaxChunks * 4;
constexpr size_t kOffTop1 = kOffIdx + size_t(kMaxRows) * kMaxChunks * 4;
constexpr size_t kScratchBytes = kOffTop1 + size_t(kMaxRows) * 4;   // 67,840 bytes

static __device__ __align__(256) unsigned char g_accept_scratch[kScratchBytes];

// In host code the name g_accept_scratch is only a handle; the device address
// of the array is looked up once per device and cached here.
std::mutex g_mu;
void* g_scratch_ptr[kMaxDevices] = {};

cudaError_t scratch_address(void** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lk(g_mu);
  if (!g_scratch_ptr[dev]) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_accept_scratch);     // with `dev` current
    if (e != cudaSuccess) return e;
    g_scratch_ptr[dev] = p;
  }
  *out = g_scratch_ptr[dev];
  return cudaSuccess;
}

struct Best { float v; int i; };
__device__ __forceinline__ void take(Best& b, float v, int i) { if (v > b.v) { b.v = v; b.i = i; } }
__device__ __forceinline__ Best merge(Best a, Best b) {
  return (b.v > a.v || (b.v == a.v && b.i < a.i)) ? b : a;
}

struct Args {
  unsigned char* scratch;
  int n_bs;
  const int32_t* n_live;
  const int32_t* k;
  const int32_t* offset;
  const int32_t* tokens;
  const float* logits;
  int64_t ld;
  int vocab;
  int32_t* accept_len;
  int32_t* next_anchor;
  int32_t* out_tokens;
  int32_t* out_len;
  int chunks, chunk_len;
};

__global__ void __launch_bounds__(kThreads) accept_static_kernel(Args a) {
  int* ticket = reinterpret_cast<int*>(a.scratch);
  float* pval = reinterpret_cast<float*>(a.scratch + kOffVal);
  int* pidx = reinterpret_cast<int*>(a.scratch + kOffIdx);
  int* top1 = reinterpret_cast<int*>(a.scratch + kOffTop1);
  int N = *a.n_live;
  N = N < 1 ? 1 : (N > a.n_bs ? a.n_bs : N);
  // live packed rows = the end boundary of the last live request (Eq. 10): the
  // lengths may come from an allocation under any budget, not only 8 N.  Clamped
  // to the rows the launch and the scratch were sized for.
  const int cap = kHalfW * a.n_bs;
  int m_live = a.offset[N];
  m_live = m_live < 1 ? 1 : (m_live > cap ? cap : m_live);
  const int s = blockIdx.y;
  if (s >= m_live) return;
  const int c = blockIdx.x, tid = threadIdx.x;

  const float* row = a.logits + (size_t)s * a.ld;
  const int lo = c * a.chunk_len;
  const int hi = min(a.vocab, lo + a.chunk_len);
  Best b{-INFINITY, INT_MAX};
  if (lo < hi) {
    const int n4 = (hi - lo) >> 2;
    const float4* p4 = reinterpret_cast<const float4*>(row + lo);
    for (int x = tid; x < n4; x += kThreads) {
      const float4 v = __ldg(p4 + x);
      const int e = lo + 4 * x;
      take(b, v.x, e); take(b, v.y, e + 1); take(b, v.z, e + 2); take(b, v.w, e + 3);
    }
    for (int e = lo + 4 * n4 + tid; e < hi; e += kThreads) take(b, row[e], e);
  }
#pragma unroll
  for (int d = 16; d > 0; d >>= 1) {
    Best o{__shfl_xor_sync(0xffffffffu, b.v, d), __shfl_xor_sync(0xffffffffu, b.i, d)};
    b = merge(b, o);
  }
  __shared__ float sv[kThreads / 32];
  __shared__ int si[kThreads / 32];
  __shared__ int s_last;
  if ((tid & 31) == 0) { sv[tid >> 5] = b.v; si[tid >> 5] = b.i; }
  __syncthreads();
  if (tid == 0) {
    for (int w = 1; w < kThreads / 32; ++w) b = merge(b, Best{sv[w], si[w]});
    pval[(size_t)s * kMaxChunks + c] = b.v;
    pidx[(size_t)s * kMaxChunks + c] = b.i;
    __threadfence();
    s_last = (atomicAdd(ticket, 1) == a.chunks * m_live - 1);
  }
  __syncthreads();
  if (!s_last) return;

  __threadfence();
  if (tid == 0) *ticket = 0;
  for (int r = tid; r < m_live; r += kThreads) {
    Best bb{-INFINITY, INT_MAX};
    for (int cc = 0; cc < a.chunks; ++cc)
      bb = merge(bb, Best{__ldcg(&pval[(size_t)r * kMaxChunks + cc]), __ldcg(&pidx[(size_t)r * kMaxChunks + cc])});
    top1[r] = bb.i == INT_MAX ? 0 : bb.i;
  }
  __syncthreads();
  if (tid < a.n_bs) {
    const int i = tid;
    int32_t* ot = a.out_tokens + i * kW;
    // a request whose rows do not lie inside [0, m_live) (lengths and offsets are
    // the caller's) gets the sentinel outputs instead of an out-of-range read
    const int ki = i < N ? a.k[i] : 0, oi = i < N ? a.offset[i] : 0;
    if (i < N && ki >= 1 && ki <= kW && oi >= 0 && oi + ki <= m_live) {
      int acc = 0;
      while (acc < ki - 1 && top1[oi + acc] == a.tokens[oi + acc + 1]) ++acc;
      const int nxt = top1[oi + acc];
      for (int j = 0; j < kW; ++j) ot[j] = j < acc ? a.tokens[oi + 1 + j] : (j == acc ? nxt : -1);
      a.accept_len[i] = acc;
      a.next_anchor[i] = nxt;
      a.out_len[i] = acc + 1;
    } else {
      for (int j = 0; j < kW; ++j) ot[j] = -1;
      a.accept_len[i] = 0;
      a.next_anchor[i] = -1;
      a.out_len[i] = 0;
    }
  }
}

inline bool aligned(const void* p, size_t n) { return (reinterpret_cast<uintptr_t>(p) % n) == 0; }

}  // namespace

extern "C" int dscale_accept_static(int n_bs, const int32_t* n_live, const int32_t* k,
                                    const int32_t* offset, const int32_t* tokens,
                                    const float* logits, int64_t ld, int vocab,
                                    int32_t* accept_len, int32_t* next_anchor,
                                    int32_t* out_tokens, int32_t* out_len, void* stream) {
  if (!n_live || !k || !offset || !tokens || !logits || !accept_len || !next_anchor ||
      !out_tokens || !out_len)
    return DSCALE_ERR_INVALID_ARG;
  if (n_bs < 1 || vocab < 1 || ld < vocab || (ld % 4) != 0 || !aligned(logits, 16))
    return DSCALE_ERR_INVALID_ARG;
  if (n_bs > DSCALE_ACCEPT_STATIC_MAX_NBS) return DSCALE_ERR_TOO_LARGE;   // scratch is sized for 64 requests
  void* scratch = nullptr;
  if (scratch_address(&scratch) != cudaSuccess) return DSCALE_ERR_CUDA;
  cudaStream_t st = (cudaStream_t)stream;
  // the ticket must start at zero whatever an earlier (possibly failed) call left
  if (cudaMemsetAsync(scratch, 0, 256, st) != cudaSuccess) return DSCALE_ERR_CUDA;
  int chunks = vocab / 16384;
  chunks = chunks < 1 ? 1 : (chunks > kMaxChunks ? kMaxChunks : chunks);
  int chunk_len = ((vocab + chunks - 1) / chunks + 3) & ~3;
  Args a{static_cast<unsigned char*>(scratch), n_bs, n_live, k, offset, tokens, logits, ld, vocab,
         accept_len, next_anchor, out_tokens, out_len, chunks, chunk_len};
  accept_static_kernel<<<dim3(chunks, kHalfW * n_bs), kThreads, 0, st>>>(a);
  return cudaGetLastError() == cudaSuccess ? DSCALE_OK : DSCALE_ERR_CUDA;
}
