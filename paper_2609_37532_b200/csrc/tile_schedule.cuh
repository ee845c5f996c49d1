// Stream-K style schedule over key tiles, shared by the tensor-core attention
// kernels: all key tiles of all (request, head) pairs form one linear list and
// CTA c of a persistent grid owns the slice [c T / C, (c + 1) T / C).
#pragma once
#include <cstdint>

namespace dscale {
namespace {

// One maximal run of tiles of a single (request, kv-head) pair inside a CTA's slice.
struct Segment {
  int i, g;          // request, kv-head
  int t0, t1;        // tile range of the pair covered here
  int n_tiles;       // tiles of the whole pair
  bool first_of_cta; // the run starts at the slice start
};

struct Scheduler {
  const int* tile_pre;   // shared copy, [n_bs + 1]
  int n_bs, n_kv;
  long long pos, end, begin;
  int i;                 // search hint

  __device__ void init(const int* tp, int n_bs_, int n_kv_, long long b, long long e) {
    tile_pre = tp; n_bs = n_bs_; n_kv = n_kv_; begin = pos = b; end = e; i = 0;
  }
  __device__ bool next(Segment& s) {
    if (pos >= end) return false;
    while (i < n_bs && (long long)tile_pre[i + 1] * n_kv <= pos) ++i;
    const int n_i = tile_pre[i + 1] - tile_pre[i];
    const long long rem = pos - (long long)tile_pre[i] * n_kv;
    s.i = i;
    s.g = (int)(rem / n_i);
    s.t0 = (int)(rem % n_i);
    const long long room = end - pos;
    s.t1 = (int)((long long)(n_i - s.t0) <= room ? n_i : s.t0 + room);
    s.n_tiles = n_i;
    s.first_of_cta = (pos == begin);
    pos += s.t1 - s.t0;
    return true;
  }
  __device__ bool more() const { return pos < end; }   // runs left after the one just returned
};

__device__ __forceinline__ long long slice_begin(int c, long long T, int C) { return (long long)c * T / C; }
// the CTA whose slice holds linear tile index L
__device__ __forceinline__ int cta_of(long long L, long long T, int C) {
  return (int)(((L + 1) * C + T - 1) / T) - 1;
}


}  // namespace
}  // namespace dscale
