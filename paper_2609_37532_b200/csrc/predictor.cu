// Acceptance-predictor front end: drafter logits and hidden states -> 1735
// features -> 1735-64-15 perceptron -> predLogits ("Acceptance predictor"
// paragraph, Eq. 4 and Eq. 5).  Three launches:
//
//  pred_stream_kernel    the only pass over the drafter logits (15 N rows x V fp32,
//                        292 MB at N = 32: an HBM stream).  A CTA of 16 warps owns
//                        16 rows x one vocabulary chunk; warp w streams row w with
//                        coalesced 128-bit loads and keeps, per row, the running
//                        (max, sum e^{z-max}, sum e^{z-max} z, sum z) and the 16
//                        largest values (sorted in lanes 0-15; a new value enters
//                        only if it beats the 16th, found by a warp ballot, so the
//                        steady state costs one compare per element).  The fixed
//                        32 x V logit projection is a dense contraction with K = V:
//                        every 128-column sub-tile is also stored to shared memory
//                        (minus a per-row pivot, rounded to tf32) next to the
//                        matching 32 x 128 tile of the projection matrix, and the
//                        16 warps each issue one k = 8 step of m16n8k8 tf32 MMAs
//                        over it.  Warp-level MMAs on purpose: 4.7 GFLOP ride
//                        along with a 292 MB stream, there is no tensor-core
//                        time to win, and the rows are already in registers.
//                        One record per (row, chunk) goes to the workspace.
//  pred_features_kernel  per request: merges the chunk records into the 18
//                        confidence values and the centred logit projection per
//                        position, computes the 64 x H hidden-state projection,
//                        appends the batch context.
//  pred_mlp_kernel       per request: relu(W1 f + b1), W2 h + b2.
#include <cfloat>
#include <climits>
#include <cuda_bf16.h>

#include "kernels.cuh"

namespace dscale {

namespace {

constexpr int kRowsPerCta = 16;                 // = warps per CTA = k steps per sub-tile
constexpr int kStreamThreads = kRowsPerCta * 32;
constexpr int kSub = 128;                       // columns per sub-tile: one float4 per lane
constexpr int kStride = kSub + 4;               // shared-memory row stride in floats (conflict-free fragments)
constexpr int kStreamSmem = 2 * (kRowsPerCta + kPredLog) * kStride * 4;   // 50,688 bytes

struct StreamArgs {
  const float* logits;      // [15 n_bs][ld]
  int64_t ld;
  int vocab;
  const int32_t* n_live;
  int n_bs;
  const __nv_bfloat16* p_logit;   // [32][vocab]
  float* part;              // [15 n_bs][chunks][kPredRec]
  float* rowsum;            // [chunks][32]
  int chunks;
  int chunk_len;            // multiple of kSub
};

__device__ __forceinline__ float to_tf32(float x) {
  uint32_t r;
  asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x));
  return __uint_as_float(r);
}
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

__global__ void __launch_bounds__(kStreamThreads, 2) pred_stream_kernel(StreamArgs a) {
  extern __shared__ __align__(16) float stream_smem[];
  float (*zs)[kRowsPerCta][kStride] = reinterpret_cast<float (*)[kRowsPerCta][kStride]>(stream_smem);
  float (*ps)[kPredLog][kStride] =
      reinterpret_cast<float (*)[kPredLog][kStride]>(stream_smem + 2 * kRowsPerCta * kStride);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  int n = *a.n_live;
  n = n < 0 ? 0 : (n > a.n_bs ? a.n_bs : n);
  const int live_rows = kPredPos * n;
  const int row0 = blockIdx.y * kRowsPerCta;
  if (row0 >= live_rows) return;
  const int chunk = blockIdx.x;
  const int col_lo = chunk * a.chunk_len;
  const int col_hi = min(a.vocab, col_lo + a.chunk_len);
  if (col_lo >= col_hi) return;
  const int n_sub = (col_hi - col_lo + kSub - 1) / kSub;

  const bool live = row0 + warp < live_rows;
  const int row = live ? row0 + warp : row0;          // dead rows re-read a live one; results dropped
  const float* zrow = a.logits + (size_t)row * a.ld;
  const float pivot = zrow[0];

  // projection-matrix staging: thread -> (output j, 8 columns)
  const int pj = tid >> 4, pq = tid & 15;
  const __nv_bfloat16* prow = a.p_logit + (size_t)pj * a.vocab;
  const bool p_vec = (a.vocab & 7) == 0;               // 16-byte loads stay aligned
  float p_rowsum = 0.f;

  auto load_z = [&](int s) -> float4 {
    const int c = col_lo + s * kSub + 4 * lane;
    float4 z = make_float4(-INFINITY, -INFINITY, -INFINITY, -INFINITY);
    if (c < col_hi) {
      z = ldg_stream4(zrow + c);                        // rows are padded to ld % 4 == 0
      if (c + 1 >= col_hi) z.y = -INFINITY;
      if (c + 2 >= col_hi) z.z = -INFINITY;
      if (c + 3 >= col_hi) z.w = -INFINITY;
    }
    return z;
  };
  auto load_p = [&](int s, float (&pv)[8]) {
    const int c = col_lo + s * kSub + 8 * pq;
    if (p_vec && c + 8 <= col_hi) {
      const uint4 u = __ldg(reinterpret_cast<const uint4*>(prow + c));
      const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
      for (int x = 0; x < 4; ++x) {
        pv[2 * x] = __uint_as_float(w[x] << 16);
        pv[2 * x + 1] = __uint_as_float(w[x] & 0xffff0000u);
      }
    } else {
#pragma unroll
      for (int x = 0; x < 8; ++x) pv[x] = c + x < col_hi ? __bfloat162float(prow[c + x]) : 0.f;
    }
  };

  float m = -INFINITY, s_sum = 0.f, t_sum = 0.f, z_sum = 0.f;
  float tv = -INFINITY, tau = -INFINITY;
  float d[4][4];
#pragma unroll
  for (int x = 0; x < 4; ++x) d[x][0] = d[x][1] = d[x][2] = d[x][3] = 0.f;
  const int g = lane >> 2, t = lane & 3;

  float4 z_next = load_z(0);
  float p_next[8];
  load_p(0, p_next);
  for (int s = 0; s < n_sub; ++s) {
    const int b = s & 1;
    const float4 z = z_next;
    // stage this sub-tile: logits minus pivot as tf32 (0 beyond the chunk), projection tile as fp32
    {
      float4 c4;
      c4.x = z.x == -INFINITY ? 0.f : to_tf32(z.x - pivot);
      c4.y = z.y == -INFINITY ? 0.f : to_tf32(z.y - pivot);
      c4.z = z.z == -INFINITY ? 0.f : to_tf32(z.z - pivot);
      c4.w = z.w == -INFINITY ? 0.f : to_tf32(z.w - pivot);
      *reinterpret_cast<float4*>(&zs[b][warp][4 * lane]) = c4;
      *reinterpret_cast<float4*>(&ps[b][pj][8 * pq]) = make_float4(p_next[0], p_next[1], p_next[2], p_next[3]);
      *reinterpret_cast<float4*>(&ps[b][pj][8 * pq + 4]) = make_float4(p_next[4], p_next[5], p_next[6], p_next[7]);
#pragma unroll
      for (int x = 0; x < 8; ++x) p_rowsum += p_next[x];
    }
    if (s + 1 < n_sub) { z_next = load_z(s + 1); load_p(s + 1, p_next); }
    __syncthreads();

    // ---- row statistics on the exact fp32 values
    {
      const float zl = fmaxf(fmaxf(z.x, z.y), fmaxf(z.z, z.w));
      if (zl > m) {
        const float r = __expf(m - zl);                 // m = -inf gives 0
        s_sum *= r; t_sum *= r; m = zl;
      }
      const float zz[4] = {z.x, z.y, z.z, z.w};
#pragma unroll
      for (int x = 0; x < 4; ++x) {
        if (zz[x] != -INFINITY) {
          const float e = __expf(zz[x] - m);
          s_sum += e; t_sum = fmaf(e, zz[x], t_sum); z_sum += zz[x];
        }
      }
      top16_offer(tv, tau, z.x, lane);
      top16_offer(tv, tau, z.y, lane);
      top16_offer(tv, tau, z.z, lane);
      top16_offer(tv, tau, z.w, lane);
    }
    // ---- this warp's k step of the logit projection: columns 8 warp .. 8 warp + 7
    {
      const int k0 = 8 * warp;
      uint32_t af[4];
      af[0] = __float_as_uint(zs[b][g][k0 + t]);
      af[1] = __float_as_uint(zs[b][g + 8][k0 + t]);
      af[2] = __float_as_uint(zs[b][g][k0 + t + 4]);
      af[3] = __float_as_uint(zs[b][g + 8][k0 + t + 4]);
#pragma unroll
      for (int nt = 0; nt < 4; ++nt)
        mma_tf32(d[nt], af, __float_as_uint(ps[b][8 * nt + g][k0 + t]),
                 __float_as_uint(ps[b][8 * nt + g][k0 + t + 4]));
    }
  }

  // ---- row statistics: merge the 32 lanes
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float m2 = __shfl_xor_sync(0xffffffffu, m, o);
    const float s2 = __shfl_xor_sync(0xffffffffu, s_sum, o);
    const float t2 = __shfl_xor_sync(0xffffffffu, t_sum, o);
    z_sum += __shfl_xor_sync(0xffffffffu, z_sum, o);
    const float mm = fmaxf(m, m2);
    const float r1 = m == -INFINITY ? 0.f : __expf(m - mm), r2 = m2 == -INFINITY ? 0.f : __expf(m2 - mm);
    s_sum = s_sum * r1 + s2 * r2;
    t_sum = t_sum * r1 + t2 * r2;
    m = mm;
  }
  float* rec = a.part + ((size_t)(row0 + warp) * a.chunks + chunk) * kPredRec;
  if (live) {
    if (lane < 16) rec[lane] = tv;
    if (lane == 0) { rec[16] = m; rec[17] = s_sum; rec[18] = t_sum; rec[19] = z_sum; }
  }
  // ---- projection: sum the 16 warps' k slices through shared memory
  __syncthreads();
  float* red = &ps[0][0][0];                            // 16 x 512 floats fit the two projection buffers
  static_assert(2 * kPredLog * kStride >= kRowsPerCta * 512, "reduction buffer");
#pragma unroll
  for (int nt = 0; nt < 4; ++nt) {
    red[warp * 512 + g * 32 + 8 * nt + 2 * t] = d[nt][0];
    red[warp * 512 + g * 32 + 8 * nt + 2 * t + 1] = d[nt][1];
    red[warp * 512 + (g + 8) * 32 + 8 * nt + 2 * t] = d[nt][2];
    red[warp * 512 + (g + 8) * 32 + 8 * nt + 2 * t + 1] = d[nt][3];
  }
  __syncthreads();
  {
    float acc = 0.f;
#pragma unroll
    for (int w = 0; w < kRowsPerCta; ++w) acc += red[w * 512 + tid];
    const int r = tid >> 5, j = tid & 31;
    if (row0 + r < live_rows)
      a.part[((size_t)(row0 + r) * a.chunks + chunk) * kPredRec + 20 + j] = acc;
  }
  // ---- row sums of the projection matrix over this chunk (first row group only)
  if (blockIdx.y == 0) {
#pragma unroll
    for (int o = 8; o > 0; o >>= 1) p_rowsum += __shfl_xor_sync(0xffffffffu, p_rowsum, o);
    if (pq == 0) a.rowsum[chunk * kPredLog + pj] = p_rowsum;
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

constexpr int kFeatThreads = 256;
constexpr int kHidPerBlock = 16;   // hidden-projection outputs per block: grid.y = 1 + 64 / 16

__global__ void __launch_bounds__(kFeatThreads) pred_features_kernel(FeatArgs a) {
  const int i = blockIdx.x;
  int n = *a.n_live;
  n = n < 0 ? 0 : (n > a.n_bs ? a.n_bs : n);
  if (i >= n) return;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  float* f = a.feat + (size_t)i * kPredFeatures;

  if (blockIdx.y == 0) {
    // ---- confidence values and centred logit projection, one warp per position
    for (int p = warp; p < kPredPos; p += kFeatThreads / 32) {
      const int row = i * kPredPos + p;
      const float* rec0 = a.part + (size_t)row * a.chunks * kPredRec;
      float tv = -INFINITY, tau = -INFINITY;
      for (int c = 0; c < a.chunks; ++c) {
        const float cand = lane < 16 ? rec0[(size_t)c * kPredRec + lane] : -INFINITY;
        top16_offer(tv, tau, cand, lane);
      }
      // merge the chunks' (max, sum, sum e z, sum z): lane = chunk
      float m = -INFINITY, s_sum = 0.f, t_sum = 0.f, z_sum = 0.f;
      if (lane < a.chunks) {
        const float* r = rec0 + (size_t)lane * kPredRec;
        m = r[16]; s_sum = r[17]; t_sum = r[18]; z_sum = r[19];
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float m2 = __shfl_xor_sync(0xffffffffu, m, o);
        const float s2 = __shfl_xor_sync(0xffffffffu, s_sum, o);
        const float t2 = __shfl_xor_sync(0xffffffffu, t_sum, o);
        z_sum += __shfl_xor_sync(0xffffffffu, z_sum, o);
        const float mm = fmaxf(m, m2);
        const float r1 = m == -INFINITY ? 0.f : expf(m - mm), r2 = m2 == -INFINITY ? 0.f : expf(m2 - mm);
        s_sum = s_sum * r1 + s2 * r2;
        t_sum = t_sum * r1 + t2 * r2;
        m = mm;
      }
      const float lse = m + logf(s_sum);
      const float top = __shfl_sync(0xffffffffu, tv, 0);
      float* fc = f + p * kPredConf;
      if (lane == 0) fc[0] = top;
      else if (lane < 16) fc[lane] = top - tv;
      else if (lane == 16) fc[16] = top - lse;
      else if (lane == 17) fc[17] = lse - t_sum / s_sum;
      // logit projection of z - mean(z): the kernel accumulated P (z - pivot)
      const float pivot = a.logits[(size_t)row * a.ld];
      const float mean = z_sum / (float)a.vocab;
      float proj = 0.f, rs = 0.f;
      for (int c = 0; c < a.chunks; ++c) {
        proj += rec0[(size_t)c * kPredRec + 20 + lane];
        rs += a.rowsum[c * kPredLog + lane];
      }
      f[kPredPos * (kPredConf + kPredHid) + p * kPredLog + lane] = proj - (mean - pivot) * rs;
    }
    if (warp == 0 && lane < kPredCtx)
      f[kPredFeatures - kPredCtx + lane] = lane == 0 ? (float)n : (lane == 3 ? 1.f : 0.f);
  } else {
    // ---- hidden-state projection: kHidPerBlock outputs x 15 positions, two outputs per warp
    const int H = a.hidden_dim;
    const __nv_bfloat16* hbase = a.hidden + (size_t)i * kPredPos * H;
    for (int jj = warp; jj < kHidPerBlock; jj += kFeatThreads / 32) {
      const int j = (blockIdx.y - 1) * kHidPerBlock + jj;
      const __nv_bfloat16* prow = a.p_hidden + (size_t)j * H;
      float acc[kPredPos];
#pragma unroll
      for (int p = 0; p < kPredPos; ++p) acc[p] = 0.f;
      for (int c = 8 * lane; c < H; c += 256) {         // hidden_dim % 8 == 0
        const uint4 pu = __ldg(reinterpret_cast<const uint4*>(prow + c));
        const uint32_t pw[4] = {pu.x, pu.y, pu.z, pu.w};
        float pf[8];
#pragma unroll
        for (int x = 0; x < 4; ++x) {
          pf[2 * x] = __uint_as_float(pw[x] << 16);
          pf[2 * x + 1] = __uint_as_float(pw[x] & 0xffff0000u);
        }
#pragma unroll
        for (int p = 0; p < kPredPos; ++p) {
          const uint4 hu = __ldg(reinterpret_cast<const uint4*>(hbase + (size_t)p * H + c));
          const uint32_t hw[4] = {hu.x, hu.y, hu.z, hu.w};
#pragma unroll
          for (int x = 0; x < 4; ++x) {
            acc[p] = fmaf(pf[2 * x], __uint_as_float(hw[x] << 16), acc[p]);
            acc[p] = fmaf(pf[2 * x + 1], __uint_as_float(hw[x] & 0xffff0000u), acc[p]);
          }
        }
      }
#pragma unroll
      for (int p = 0; p < kPredPos; ++p) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc[p] += __shfl_xor_sync(0xffffffffu, acc[p], o);
      }
      if (lane == 0) {
#pragma unroll
        for (int p = 0; p < kPredPos; ++p) f[kPredPos * kPredConf + p * kPredHid + j] = acc[p];
      }
    }
  }
}

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
};

__global__ void __launch_bounds__(256) pred_mlp_kernel(MlpArgs a) {
  __shared__ float sf[kPredFeatures];
  __shared__ float sh[kPredMlp];
  const int i = blockIdx.x;
  int n = *a.n_live;
  n = n < 0 ? 0 : (n > a.n_bs ? a.n_bs : n);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  if (i >= n) {                                           // dead request: zeros
    if (tid < kPredPos) a.pred_logits[i * kPredPos + tid] = 0.f;
    if (a.features_out)
      for (int x = tid; x < kPredFeatures; x += 256) a.features_out[(size_t)i * kPredFeatures + x] = 0.f;
    return;
  }
  for (int x = tid; x < kPredFeatures; x += 256) {
    const float v = a.feat[(size_t)i * kPredFeatures + x];
    sf[x] = v;
    if (a.features_out) a.features_out[(size_t)i * kPredFeatures + x] = v;
  }
  __syncthreads();
  for (int j = warp; j < kPredMlp; j += 8) {
    const float* w = a.w1 + (size_t)j * kPredFeatures;
    float acc = 0.f;
    for (int x = lane; x < kPredFeatures; x += 32) acc = fmaf(w[x], sf[x], acc);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
    if (lane == 0) sh[j] = fmaxf(acc + a.b1[j], 0.f);
  }
  __syncthreads();
  for (int o = warp; o < kPredPos; o += 8) {
    const float* w = a.w2 + o * kPredMlp;
    float acc = w[lane] * sh[lane] + w[lane + 32] * sh[lane + 32];
#pragma unroll
    for (int x = 16; x > 0; x >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, x);
    if (lane == 0) a.pred_logits[i * kPredPos + o] = acc + a.b2[o];
  }
}

}  // namespace

cudaError_t predictor_prepare() {
  return cudaFuncSetAttribute(pred_stream_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kStreamSmem);
}

int predictor_chunks(int n_bs, int vocab, int num_ctas, int* chunk_len_out) {
  const int row_groups = (kPredPos * n_bs + kRowsPerCta - 1) / kRowsPerCta;
  int chunks = (3 * num_ctas + row_groups - 1) / row_groups;      // about three CTAs per SM
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

  StreamArgs sa{p.draft_logits, p.ld, p.vocab, p.n_live, p.n_bs,
                reinterpret_cast<const __nv_bfloat16*>(p.p_logit), part, rowsum, chunks, chunk_len};
  pred_stream_kernel<<<dim3(chunks, row_groups), kStreamThreads, kStreamSmem, stream>>>(sa);
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  FeatArgs fa{p.draft_logits, p.ld, p.vocab, p.n_live, p.n_bs,
              reinterpret_cast<const __nv_bfloat16*>(p.draft_hidden), p.hidden_dim,
              reinterpret_cast<const __nv_bfloat16*>(p.p_hidden), part, rowsum, chunks, feat};
  pred_features_kernel<<<dim3(p.n_bs, 1 + kPredHid / kHidPerBlock), kFeatThreads, 0, stream>>>(fa);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  MlpArgs ma{p.n_live, p.n_bs, feat, p.w1, p.b1, p.w2, p.b2, p.pred_logits, p.features_out};
  pred_mlp_kernel<<<p.n_bs, 256, 0, stream>>>(ma);
  return cudaGetLastError();
}

}  // namespace dscale
