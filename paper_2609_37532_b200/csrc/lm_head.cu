// Fused LM head + target-token argmax + greedy acceptance for the packed rows.
//
// top1[s] = argmax_v sum_h hidden[s][h] * weight[v][h]  for the 8N live packed
// rows, without ever writing the 8N x V logits (at N = 32 that is 155 MB of fp32
// written and read back, next to 1.24 GB of bf16 weights that have to be read
// anyway).  A dense contraction: this one belongs on the tensor cores.
//
// Each CTA of a persistent grid owns a contiguous range of vocabulary columns,
// cut into equal tiles of n_tile <= 256 columns (a multiple of 16, chosen on the
// host so that all CTAs get the same number of equal tiles).  For a tile it
// accumulates all <= 4 row tiles of 128 packed rows at once in TMEM
// (m_tiles x n_tile fp32 columns), so every weight element is read from HBM
// exactly once; the hidden rows (2 MB) are re-read from L2.
//   warp 4   TMA producer: per 64-wide k step the hidden boxes [128 rows][64]
//            and the weight box [n_tile rows][64], 128-byte swizzle, ring of
//            shared-memory stages with mbarrier expect-tx.
//   warp 5   one thread issues tcgen05.mma (M128, N = n_tile, K16 x 4 per step).
//   warps 0-3  epilogue: thread = packed row; tcgen05.ld 32 columns at a time,
//            running (max, first index); after the CTA's last tile one partial
//            per (row, CTA) goes to the workspace.
// The last CTA to finish (ticket, nobody waits) merges the partials in vocabulary
// order -- so equal maxima resolve to the lowest index -- and runs the acceptance
// loop of the "Prefix verifier" paragraph.
#include <climits>

#include "kernels.cuh"
#include "tc_ptx.cuh"

namespace dscale {

namespace {

constexpr int kThreads = 192;
constexpr int kEpiThreads = 128;
constexpr int kKStep = 64;                       // bf16 elements per k step = one 128-byte swizzle row
constexpr int kATile = 128 * kKStep * 2;         // 16 KB: 128 rows x 64 columns

struct LmShape {
  int m_tiles;        // row tiles of 128 packed rows
  int n_tile;         // vocabulary columns per tile (multiple of 16, <= 256)
  int tiles_per_cta;
  int cols_per_cta;   // n_tile * tiles_per_cta
  int stages;
  int stage_bytes;
  int b_bytes;        // bytes of one weight box, rounded up to 1024
  int a_rows;         // rows of one hidden box
  int smem_bytes;
};

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes "
      "[%0], [%1, {%3, %4}], [%2];"
      ::"r"(dst), "l"(map), "r"(bar), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float* v) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];\n\t"
      "tcgen05.wait::ld.sync.aligned;"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
#pragma unroll
  for (int x = 0; x < 16; ++x) v[x] = __uint_as_float(r[x]);
}

struct LmArgs {
  void* ws;
  int n_bs;
  int hidden_dim;
  int vocab;
  int32_t* accept_len;
  int32_t* next_anchor;
  int32_t* out_tokens;
  int32_t* out_len;
  int32_t* ctx_len_inout;
  float* row_max;          // nullable [8 n_bs]: the winning logit of every live row
};

__global__ void __launch_bounds__(kThreads, 1)
lm_head_kernel(LmArgs a, WsLayout L, LmShape sh, const __grid_constant__ CUtensorMap tm_a,
               const __grid_constant__ CUtensorMap tm_b) {
  extern __shared__ unsigned char smem_dyn[];
  const uint32_t raw = smem_u32(smem_dyn);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* sm = smem_dyn + (base - raw);
  const int off_bar = sh.stages * sh.stage_bytes;
  uint32_t* s_tmem = reinterpret_cast<uint32_t*>(sm + off_bar + 256);
  volatile int* s_abort = reinterpret_cast<volatile int*>(sm + off_bar + 260);
  int* s_last = reinterpret_cast<int*>(sm + off_bar + 264);
  auto bar = [&](int b) { return base + off_bar + 8u * b; };
  const int B_FULL = 0, B_EMPTY = sh.stages, B_ACC_FULL = 2 * sh.stages, B_ACC_EMPTY = B_ACC_FULL + 1,
            B_GROUP = B_ACC_FULL + 2;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int c = blockIdx.x, C = gridDim.x;
  int* hdr = ws_ptr<int>(a.ws, L.hdr);
  const int m_live = hdr[H_M_LIVE];

  if (tid == 0) {
    for (int s = 0; s < sh.stages; ++s) { mbar_init(bar(B_FULL + s), 1); mbar_init(bar(B_EMPTY + s), 1); }
    mbar_init(bar(B_ACC_FULL), 1);
    mbar_init(bar(B_ACC_EMPTY), kEpiThreads);
    mbar_init(bar(B_GROUP), kEpiThreads);
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 5) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;"
                 ::"r"(smem_u32(s_tmem)) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  if (warp == 4 && lane == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_a) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tm_b) : "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *s_tmem;

  const int col_begin = c * sh.cols_per_cta;
  int my_tiles = 0;
  for (int t = 0; t < sh.tiles_per_cta; ++t) my_tiles += (col_begin + t * sh.n_tile < a.vocab);
  const int k_steps = a.hidden_dim / kKStep;
  const uint32_t a_box_bytes = (uint32_t)sh.a_rows * kKStep * 2;
  const uint32_t b_box_bytes = (uint32_t)sh.n_tile * kKStep * 2;

  if (warp == 4) {
    // ===================================================== TMA producer
    if (lane == 0) {
      unsigned u = 0;
      bool ok = true;
      for (int t = 0; t < my_tiles && ok; ++t) {
        const int col0 = col_begin + t * sh.n_tile;
        for (int kb = 0; kb < k_steps && ok; ++kb, ++u) {
          const int slot = u % sh.stages;
          ok = mbar_wait(bar(B_EMPTY + slot), ((u / sh.stages) & 1) ^ 1, s_abort);
          if (!ok) break;
          mbar_expect_tx(bar(B_FULL + slot), sh.m_tiles * a_box_bytes + b_box_bytes);
          const uint32_t st = base + slot * sh.stage_bytes;
          for (int m = 0; m < sh.m_tiles; ++m)
            tma_load_2d(st + m * kATile, &tm_a, bar(B_FULL + slot), kb * kKStep, m * 128);
          tma_load_2d(st + sh.m_tiles * kATile, &tm_b, bar(B_FULL + slot), kb * kKStep, col0);
        }
      }
    }
    __syncwarp();
  } else if (warp == 5) {
    // ===================================================== MMA issuer
    if (lane == 0) {
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(sh.n_tile >> 3) << 17) |
                             ((128u >> 4) << 24);
      unsigned u = 0;
      bool ok = true;
      for (int t = 0; t < my_tiles && ok; ++t) {
        ok = mbar_wait(bar(B_ACC_EMPTY), (t & 1) ^ 1, s_abort);      // accumulators drained
        if (!ok) break;
        tc_fence_after();
        for (int kb = 0; kb < k_steps && ok; ++kb, ++u) {
          const int slot = u % sh.stages;
          ok = mbar_wait(bar(B_FULL + slot), (u / sh.stages) & 1, s_abort);
          if (!ok) break;
          tc_fence_after();
          const uint32_t st = base + slot * sh.stage_bytes;
          const uint32_t b_base = st + sh.m_tiles * kATile;
#pragma unroll
          for (int ks = 0; ks < kKStep / 16; ++ks) {
            const uint64_t bd = smem_desc(b_base + ks * 32, 16, 1024);
            for (int m = 0; m < sh.m_tiles; ++m) {
              const uint64_t ad = smem_desc(st + m * kATile + ks * 32, 16, 1024);
              umma(tmem + m * sh.n_tile, ad, bd, idesc, (kb | ks) != 0);
            }
          }
          umma_commit(bar(B_EMPTY + slot));
        }
        if (ok) umma_commit(bar(B_ACC_FULL));
      }
    }
    __syncwarp();
  } else {
    // ===================================================== epilogue warps 0-3
    const uint32_t t_lane = tmem + ((uint32_t)(warp * 32) << 16);
    float best[4];
    int best_i[4];
#pragma unroll
    for (int m = 0; m < 4; ++m) { best[m] = -INFINITY; best_i[m] = INT_MAX; }
    bool ok = true;
    for (int t = 0; t < my_tiles && ok; ++t) {
      ok = mbar_wait(bar(B_ACC_FULL), t & 1, s_abort);
      if (!ok) break;
      tc_fence_after();
      const int col0 = col_begin + t * sh.n_tile;
#pragma unroll
      for (int m = 0; m < 4; ++m) {
        if (m < sh.m_tiles) {
          const bool live = m * 128 + tid < m_live;           // warp-uniform only per row; loads are collective
          for (int ch = 0; ch + 32 <= sh.n_tile; ch += 32) {
            float v[32];
            tmem_ld32(t_lane + m * sh.n_tile + ch, v);
            if (live) {
#pragma unroll
              for (int x = 0; x < 32; ++x) {
                const int col = col0 + ch + x;
                if (col < a.vocab && v[x] > best[m]) { best[m] = v[x]; best_i[m] = col; }
              }
            }
          }
          if (sh.n_tile & 16) {
            const int ch = sh.n_tile & ~31;
            float v[16];
            tmem_ld16(t_lane + m * sh.n_tile + ch, v);
            if (live) {
#pragma unroll
              for (int x = 0; x < 16; ++x) {
                const int col = col0 + ch + x;
                if (col < a.vocab && v[x] > best[m]) { best[m] = v[x]; best_i[m] = col; }
              }
            }
          }
        }
      }
      tc_fence_before();
      mbar_arrive(bar(B_ACC_EMPTY));
    }
    // one partial per (row, CTA); CTAs without columns write the neutral element
    float* pv = ws_ptr<float>(a.ws, L.lm_val);
    int* pi = ws_ptr<int>(a.ws, L.lm_idx);
#pragma unroll
    for (int m = 0; m < 4; ++m) {
      const int row = m * 128 + tid;
      if (m < sh.m_tiles && row < m_live) {
        pv[(size_t)row * C + c] = best[m];
        pi[(size_t)row * C + c] = best_i[m];
      }
    }
    __threadfence();
    unsigned group_phase = 0;
    auto group_sync = [&]() -> bool {                 // bounded barrier of the 128 epilogue threads
      mbar_arrive(bar(B_GROUP));
      const bool r = mbar_wait(bar(B_GROUP), group_phase & 1, s_abort);
      ++group_phase;
      return r;
    };
    ok = ok && group_sync();
    if (ok && tid == 0) *s_last = (atomicAdd(&hdr[H_LM_TICKET], 1) == C - 1);
    ok = ok && group_sync();
    if (ok && *s_last) {
      // ---- last CTA: merge in vocabulary order, then the acceptance loop
      __threadfence();
      if (tid == 0) hdr[H_LM_TICKET] = 0;
      int* top1 = ws_ptr<int>(a.ws, L.top1);
      const int m_bs = kHalfW * a.n_bs;
      for (int r = tid; r < m_bs; r += kEpiThreads) {
        int bi = 0;
        if (r < m_live) {
          float bv = -INFINITY;
          bi = INT_MAX;
          for (int cc = 0; cc < C; ++cc) {
            const float v = __ldcg(&pv[(size_t)r * C + cc]);
            const int i2 = __ldcg(&pi[(size_t)r * C + cc]);
            if (v > bv || (v == bv && i2 < bi)) { bv = v; bi = i2; }
          }
          if (bi == INT_MAX) bi = 0;
          if (a.row_max) a.row_max[r] = bv;
        }
        top1[r] = bi;
      }
      ok = group_sync();
      const int N = hdr[H_N_LIVE];
      const int* wk = ws_ptr<int>(a.ws, L.k);
      const int* woff = ws_ptr<int>(a.ws, L.offset);
      const int* wtok = ws_ptr<int>(a.ws, L.tokens);
      if (ok && tid < a.n_bs) {
        const int i = tid;
        int32_t* ot = a.out_tokens + i * kW;
        if (i < N) {
          const int ki = wk[i], oi = woff[i];
          int acc = 0;
          while (acc < ki - 1 && top1[oi + acc] == wtok[oi + acc + 1]) ++acc;
          const int nxt = top1[oi + acc];
          for (int j = 0; j < kW; ++j) ot[j] = j < acc ? wtok[oi + 1 + j] : (j == acc ? nxt : -1);
          a.accept_len[i] = acc;
          a.next_anchor[i] = nxt;
          a.out_len[i] = acc + 1;
          if (a.ctx_len_inout) a.ctx_len_inout[i] += acc + 1;
        } else {
          for (int j = 0; j < kW; ++j) ot[j] = -1;
          a.accept_len[i] = 0;
          a.next_anchor[i] = -1;
          a.out_len[i] = 0;
        }
      }
    }
  }

  tc_fence_before();
  __syncthreads();
  if (tid == 0 && *s_abort) atomicOr(&hdr[H_STATUS], 8 /*TIMEOUT*/);
  if (warp == 5) {
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
  }
}

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
bool encode_2d(CUtensorMap* out, const void* ptr, int inner, int rows, int box_rows,
               CUtensorMapL2promotion promo) {
  EncodeTiledFn enc = get_encode();
  if (!enc) return false;
  cuuint64_t dims[2] = {(cuuint64_t)inner, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)inner * 2};
  cuuint32_t box[2] = {(cuuint32_t)kKStep, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1, 1};
  return enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, promo,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

LmShape plan(int n_bs, int vocab, int num_ctas) {
  LmShape s;
  const int rows = kHalfW * n_bs;
  s.m_tiles = (rows + 127) / 128;
  s.a_rows = rows < 128 ? rows : 128;
  int cols = (vocab + num_ctas - 1) / num_ctas;
  cols = (cols + 15) & ~15;
  int n_max = (512 / s.m_tiles) & ~15;
  if (n_max > 256) n_max = 256;
  s.tiles_per_cta = (cols + n_max - 1) / n_max;
  s.n_tile = (((cols + s.tiles_per_cta - 1) / s.tiles_per_cta) + 15) & ~15;
  if (s.n_tile > ((vocab + 15) & ~15)) s.n_tile = (vocab + 15) & ~15;
  s.cols_per_cta = s.n_tile * s.tiles_per_cta;
  s.b_bytes = (s.n_tile * kKStep * 2 + 1023) & ~1023;
  s.stage_bytes = s.m_tiles * kATile + s.b_bytes;
  s.stages = (200 * 1024) / s.stage_bytes;
  if (s.stages > 8) s.stages = 8;
  s.smem_bytes = s.stages * s.stage_bytes + 512 + 1024;
  return s;
}

}  // namespace

cudaError_t lm_head_prepare() {
  return cudaFuncSetAttribute(lm_head_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
}

cudaError_t launch_lm_head(void* ws, int n_bs, const void* hidden, const void* weight, int hidden_dim,
                           int vocab, int32_t* accept_len, int32_t* next_anchor, int32_t* out_tokens,
                           int32_t* out_len, int32_t* ctx_len_inout, float* row_max, int n_kv_heads,
                           int num_ctas, cudaStream_t stream) {
  WsLayout L = ws_layout(n_bs, n_kv_heads, num_ctas);
  LmShape sh = plan(n_bs, vocab, num_ctas);
  if (sh.stages < 2 || sh.n_tile < 16) return cudaErrorNotSupported;
  CUtensorMap ta, tb;
  if (!encode_2d(&ta, hidden, hidden_dim, kHalfW * n_bs, sh.a_rows, CU_TENSOR_MAP_L2_PROMOTION_L2_128B) ||
      !encode_2d(&tb, weight, hidden_dim, vocab, sh.n_tile < vocab ? sh.n_tile : vocab,
                 CU_TENSOR_MAP_L2_PROMOTION_L2_128B))
    return cudaErrorNotSupported;
  LmArgs a{ws, n_bs, hidden_dim, vocab, accept_len, next_anchor, out_tokens, out_len, ctx_len_inout, row_max};
  lm_head_kernel<<<num_ctas, kThreads, sh.smem_bytes, stream>>>(a, L, sh, ta, tb);
  return cudaGetLastError();
}

}  // namespace dscale
