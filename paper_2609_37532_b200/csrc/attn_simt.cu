// Packed ragged verify attention on plain CUDA cores.
//
// One thread block per (kv-head g, request i) handles the G * k_i live query
// rows of that GQA group (G q-heads x k_i window rows), so each K/V page is
// read once per kv-head.  Keys are streamed in tiles of 32 tokens through
// shared memory; inside a tile lane l of a warp owns token l for the q.K dot
// product and owns output columns 4l..4l+3 for the P.V update, with the usual
// running (max, sum) softmax state per row.  Row validity follows Eq. 15: only
// rows j < k_i exist, row j sees logical keys 0 .. positions[offset_i + j].
// Keys at or beyond ctx_i + k_i are never loaded (they may hold anything).
//
// This kernel is the slow, simple GPU statement of the operation: it covers any
// GQA group size and is the on-device cross-check of the tensor-core kernel.
#include <cuda_bf16.h>

#include "kernels.cuh"

namespace dscale {

namespace {

constexpr int kSimtThreads = 256;
constexpr int kSimtWarps = kSimtThreads / 32;
constexpr int kSimtTile = 32;            // tokens per tile
constexpr int kKPad = kD + 2;            // bf16 elements per K row in smem (bank-conflict free)
constexpr int kMaxRowsPerWarp = 16;      // G <= 8: 128 rows / 8 warps

__global__ void __launch_bounds__(kSimtThreads) attn_simt_kernel(AttnArgs a, WsLayout L, int G) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  __nv_bfloat16* sKt = reinterpret_cast<__nv_bfloat16*>(smem_raw);            // [32][130]
  __nv_bfloat16* sVt = sKt + kSimtTile * kKPad;                               // [32][128]
  __nv_bfloat16* sQ = sVt + kSimtTile * kD;                                   // [G*16][128]

  const int g = blockIdx.x, i = blockIdx.y;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int* hdr = ws_ptr<int>(a.ws, L.hdr);
  const int N = hdr[H_N_LIVE];
  const int Hq = a.n_q_heads;
  __nv_bfloat16* out = reinterpret_cast<__nv_bfloat16*>(a.out);

  if (i >= N) {
    // capacity rows beyond M_live: 8 rows per unused request slot, written as zero
    const int row0 = kHalfW * i;
    for (int e = tid; e < kHalfW * G * kD; e += kSimtThreads) {
      const int r = e / (G * kD), rem = e % (G * kD);
      out[((size_t)(row0 + r) * Hq + g * G) * kD + rem] = __float2bfloat16(0.0f);
    }
    return;
  }

  const int ki = ws_ptr<int>(a.ws, L.k)[i];
  const int oi = ws_ptr<int>(a.ws, L.offset)[i];
  const int kv_len = ws_ptr<int>(a.ws, L.kv_len)[i];
  const int* positions = ws_ptr<int>(a.ws, L.positions);
  const int R = G * ki;                                      // live rows: r = hq * ki + j
  const __nv_bfloat16* q = reinterpret_cast<const __nv_bfloat16*>(a.q);
  const __nv_bfloat16* kc = reinterpret_cast<const __nv_bfloat16*>(a.k_cache);
  const __nv_bfloat16* vc = reinterpret_cast<const __nv_bfloat16*>(a.v_cache);
  int* status = const_cast<int*>(&hdr[H_STATUS]);

  for (int e = tid; e < R * kD; e += kSimtThreads) {
    const int r = e / kD, d = e % kD;
    const int hq = r / ki, j = r % ki;
    sQ[r * kD + d] = q[((size_t)(oi + j) * Hq + g * G + hq) * kD + d];
  }

  float m_run[kMaxRowsPerWarp], l_run[kMaxRowsPerWarp], o_acc[kMaxRowsPerWarp][4];
  int pos_r[kMaxRowsPerWarp];
#pragma unroll
  for (int x = 0; x < kMaxRowsPerWarp; ++x) {
    m_run[x] = -INFINITY; l_run[x] = 0.0f;
    o_acc[x][0] = o_acc[x][1] = o_acc[x][2] = o_acc[x][3] = 0.0f;
    const int r = warp + x * kSimtWarps;
    pos_r[x] = r < R ? positions[oi + r % ki] : -1;
  }

  const float scale_log2 = a.sm_scale * 1.4426950408889634f;
  for (int t0 = 0; t0 < kv_len; t0 += kSimtTile) {
    __syncthreads();
    // cooperative load of the K and V tile; tokens >= kv_len are zero-filled
    for (int e = tid; e < kSimtTile * (kD / 8); e += kSimtThreads) {
      const int tl = e / (kD / 8), c8 = e % (kD / 8);
      const int tok = t0 + tl;
      uint4 kv4 = make_uint4(0, 0, 0, 0), vv4 = make_uint4(0, 0, 0, 0);
      if (tok < kv_len) {
        int page = a.block_table[(size_t)i * a.max_pages + tok / kPage];
        if (page < 0 || page >= a.num_pages) { atomicOr(status, 2); page = 0; }
        const size_t base = (((size_t)page * a.n_kv_heads + g) * kPage + tok % kPage) * kD + c8 * 8;
        kv4 = *reinterpret_cast<const uint4*>(kc + base);
        vv4 = *reinterpret_cast<const uint4*>(vc + base);
      }
      // K rows are padded to 130 elements: 4-byte stores
      uint32_t* kd = reinterpret_cast<uint32_t*>(sKt + tl * kKPad + c8 * 8);
      kd[0] = kv4.x; kd[1] = kv4.y; kd[2] = kv4.z; kd[3] = kv4.w;
      *reinterpret_cast<uint4*>(sVt + tl * kD + c8 * 8) = vv4;
    }
    __syncthreads();
#pragma unroll
    for (int x = 0; x < kMaxRowsPerWarp; ++x) {
      const int r = warp + x * kSimtWarps;
      if (r >= R) break;
      // s = q_r . k_lane
      const __nv_bfloat162* qr = reinterpret_cast<const __nv_bfloat162*>(sQ + r * kD);
      const __nv_bfloat162* kr = reinterpret_cast<const __nv_bfloat162*>(sKt + lane * kKPad);
      float s = 0.0f;
#pragma unroll 16
      for (int d2 = 0; d2 < kD / 2; ++d2) {
        const float2 qf = __bfloat1622float2(qr[d2]);
        const float2 kf = __bfloat1622float2(kr[d2]);
        s = fmaf(qf.x, kf.x, s);
        s = fmaf(qf.y, kf.y, s);
      }
      const bool visible = (t0 + lane) <= pos_r[x];
      s = visible ? s * scale_log2 : -INFINITY;
      float tmax = s;
#pragma unroll
      for (int d = 16; d > 0; d >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, d));
      const float m_new = fmaxf(m_run[x], tmax);
      if (m_new == -INFINITY) continue;                        // nothing visible yet
      const float alpha = exp2f(m_run[x] - m_new);             // exp2(-inf) = 0 on the first tile
      const float p = visible ? exp2f(s - m_new) : 0.0f;
      float psum = p;
#pragma unroll
      for (int d = 16; d > 0; d >>= 1) psum += __shfl_xor_sync(0xffffffffu, psum, d);
      l_run[x] = l_run[x] * alpha + psum;
      m_run[x] = m_new;
      float o0 = o_acc[x][0] * alpha, o1 = o_acc[x][1] * alpha, o2 = o_acc[x][2] * alpha,
            o3 = o_acc[x][3] * alpha;
#pragma unroll 8
      for (int tl = 0; tl < kSimtTile; ++tl) {
        const float pt = __shfl_sync(0xffffffffu, p, tl);
        const uint2 v2 = *reinterpret_cast<const uint2*>(sVt + tl * kD + lane * 4);
        const float2 va = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&v2.x));
        const float2 vb = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162*>(&v2.y));
        o0 = fmaf(pt, va.x, o0); o1 = fmaf(pt, va.y, o1);
        o2 = fmaf(pt, vb.x, o2); o3 = fmaf(pt, vb.y, o3);
      }
      o_acc[x][0] = o0; o_acc[x][1] = o1; o_acc[x][2] = o2; o_acc[x][3] = o3;
    }
  }

#pragma unroll
  for (int x = 0; x < kMaxRowsPerWarp; ++x) {
    const int r = warp + x * kSimtWarps;
    if (r >= R) break;
    const int hq = r / ki, j = r % ki;
    const float inv = 1.0f / l_run[x];
    __nv_bfloat162 a01 = __floats2bfloat162_rn(o_acc[x][0] * inv, o_acc[x][1] * inv);
    __nv_bfloat162 a23 = __floats2bfloat162_rn(o_acc[x][2] * inv, o_acc[x][3] * inv);
    uint2 pk;
    pk.x = *reinterpret_cast<uint32_t*>(&a01);
    pk.y = *reinterpret_cast<uint32_t*>(&a23);
    *reinterpret_cast<uint2*>(out + ((size_t)(oi + j) * Hq + g * G + hq) * kD + lane * 4) = pk;
  }
}

}  // namespace

// Opt in to the shared-memory size of the largest group (called once per
// device from dscale_workspace_init, outside any stream capture).
cudaError_t attn_simt_prepare() {
  return cudaFuncSetAttribute(attn_simt_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                              64 * 1024);
}

cudaError_t launch_attn_simt(const AttnArgs& a, cudaStream_t stream) {
  WsLayout L = ws_layout(a.n_bs, a.n_kv_heads, a.num_ctas);
  const int G = a.n_q_heads / a.n_kv_heads;
  const size_t smem = size_t(kSimtTile) * kKPad * 2 + size_t(kSimtTile) * kD * 2 +
                      size_t(G) * kW * kD * 2;
  dim3 grid(a.n_kv_heads, a.n_bs);
  attn_simt_kernel<<<grid, kSimtThreads, smem, stream>>>(a, L, G);
  return cudaGetLastError();
}

}  // namespace dscale
