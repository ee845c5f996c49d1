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

// Slices are equal, except that the last two CTAs get fewer tiles.  Blocks are handed to
// SMs in index order as the SMs fall free, so with programmatic dependent launch the
// last block of a launch lands on the SM that finished the previous launch last: it
// starts its preamble when the others have long finished theirs (measured: first MMA
// 4-5 us later for the last block, 1.5 us for the one before), and with an equal share
// it would again finish last, launch after launch.  Three tiles and one tile less
// (about 4.8 and 1.6 us of streaming) let them finish with the rest.
__device__ __forceinline__ void slice_skew(long long T, int C, int& d1, int& d2) {
  const bool on = C >= 8 && T / C >= 24;
  d1 = on ? 3 : 0;
  d2 = on ? 1 : 0;
}
__device__ __forceinline__ long long slice_begin(int c, long long T, int C) {
  int d1, d2;
  slice_skew(T, C, d1, d2);
  const long long Tv = T + d1 + d2;                   // equal shares of a slightly longer list ...
  if (c >= C) return T;
  if (c == C - 1) return (long long)(C - 1) * Tv / C - d2;   // ... and the last two give some back
  return (long long)c * Tv / C;
}
// the CTA whose slice holds linear tile index L
__device__ __forceinline__ int cta_of(long long L, long long T, int C) {
  int d1, d2;
  slice_skew(T, C, d1, d2);
  if (d1) {
    if (L >= slice_begin(C - 1, T, C)) return C - 1;
    if (L >= slice_begin(C - 2, T, C)) return C - 2;
  }
  const long long Tv = T + d1 + d2;
  return (int)(((L + 1) * C + Tv - 1) / Tv) - 1;
}

// The packed kernel reads its slice starts from a table the allocation kernel writes
// (equal-cost slices): tab[c] = first linear tile of CTA c, tab[C] = T, non-decreasing.
// The CTA whose slice holds linear tile L: the last c with tab[c] <= L.
__device__ __forceinline__ int cta_of_tab(const int* tab, int C, long long L) {
  int lo = 0, hi = C;                      // invariant: tab[lo] <= L < tab[hi]
  while (hi - lo > 1) {
    const int mid = (lo + hi) >> 1;
    if (tab[mid] <= L) lo = mid; else hi = mid;
  }
  return lo;
}

}  // namespace
}  // namespace dscale
