/*
 * dscale.h -- C ABI of the DScale verify-side hot path for NVIDIA B200 (sm_100a).
 *
 * One decode step of block-diffusion speculative decoding verifies, for each
 * of N live requests, a window of W = 16 slots (slot 0 = the known anchor,
 * slots 1..15 = draft candidates).  This library implements the three
 * verify-side stages of that step:
 *
 *   dscale_alloc_verify   DVL allocation and flat-pack   (Algorithm 1, Eq. 6-11)
 *   dscale_verify_attn    packed ragged verify attention (Section 3.2, Eq. 2, Eq. 15)
 *   dscale_accept         greedy prefix verification     ("Prefix verifier", Algorithm 2)
 *
 * General rules
 * -------------
 *  - Unless a parameter is marked HOST, every pointer is a DEVICE pointer that
 *    the caller owns.  No call allocates or frees DEVICE memory, and none
 *    synchronises.  Host-side state the library does keep: one registry entry
 *    per initialised workspace, tensor-map descriptors keyed on the q / K / V
 *    addresses it has seen (a few hundred bytes each), and, for
 *    dscale_verify_step_host_graph only, one instantiated CUDA graph per
 *    workspace (driver memory).  dscale_workspace_destroy drops all of it.
 *  - Every call only enqueues kernels on `stream` (a cudaStream_t passed as
 *    void*).  All shapes are fixed by the arguments, every data-dependent
 *    quantity (N, lengths, offsets, context lengths) is read on the device,
 *    and all intermediate state lives at fixed addresses inside the caller's
 *    workspace (Eq. 12): a CUDA graph captured once over these calls can be
 *    replayed with new inputs written to the same addresses.
 *  - Return value: DSCALE_OK, or a negative DSCALE_ERR_* code, in which case
 *    nothing was enqueued.  Faults that only the device can see (a page id out
 *    of range, a NaN score, a bounded wait that ran out) are reported through
 *    the sticky status word in the workspace (dscale_ws_field(.., DSCALE_WS_STATUS));
 *    the kernels stay in bounds in that case and finish.
 *  - Fixed by this build: W = 16, head_dim = 128, KV page = 16 tokens,
 *    budget = 8 slots per live request, n_bs <= DSCALE_MAX_NBS.
 *
 * Layouts
 * -------
 *  KV cache (one layer):  bf16 [num_pages][n_kv_heads][16][128]; logical token t
 *      of request i lives in page block_table[i][t / 16], slot t % 16.
 *  Packed rows:           row s = offset_i + j holds slot j of request i
 *      (Eq. 11); M_bs = 8 * n_bs rows are always present, M_live = 8 * N are live.
 *  q / out:               bf16 [M_bs][n_q_heads][128]; q-head h uses kv-head
 *      h / (n_q_heads / n_kv_heads).
 *  logits:                fp32 [M_bs][ld], ld >= vocab, ld % 4 == 0.
 */
#ifndef DSCALE_H_
#define DSCALE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define DSCALE_W 16
#define DSCALE_HEAD_DIM 128
#define DSCALE_PAGE 16
#define DSCALE_MAX_NBS 64

enum {
  DSCALE_OK = 0,
  DSCALE_ERR_INVALID_ARG = -1,   /* null / misaligned pointer, size out of range  */
  DSCALE_ERR_UNSUPPORTED = -2,   /* shape this build has no kernel for            */
  DSCALE_ERR_CUDA = -3,          /* a CUDA runtime / driver call failed           */
  DSCALE_ERR_WORKSPACE = -4,     /* workspace too small or not initialised        */
  DSCALE_ERR_TOO_LARGE = -5      /* size beyond a fixed built-in capacity         */
};

/* bits of the device status word (0 = OK; bits are OR-ed, sticky until
 * dscale_workspace_init is called again) */
enum {
  DSCALE_STATUS_OK = 0,
  DSCALE_STATUS_BAD_SCORE = 1,   /* score NaN or outside [0,1] (clamped)          */
  DSCALE_STATUS_BAD_PAGE = 2,    /* page id outside [0, num_pages) (page 0 used)  */
  DSCALE_STATUS_BAD_LEN = 4,     /* N or a context length out of range (clamped)  */
  DSCALE_STATUS_TIMEOUT = 8      /* a bounded device-side wait ran out            */
};

/* fields readable through dscale_ws_field */
enum {
  DSCALE_WS_STATUS = 0,     /* int32 [1]                                              */
  DSCALE_WS_K = 1,          /* int32 [n_bs]      verify lengths k_i (0 for sentinels) */
  DSCALE_WS_OFFSET = 2,     /* int32 [n_bs + 1]  Eq. 10, sentinels = M_live           */
  DSCALE_WS_Q_START = 3,    /* int32 [n_bs]      offset_i            (Alg. 2 l.14-16) */
  DSCALE_WS_Q_END = 4,      /* int32 [n_bs]      offset_i + k_i                       */
  DSCALE_WS_TOKENS = 5,     /* int32 [8 n_bs]    packed token ids                     */
  DSCALE_WS_POSITIONS = 6,  /* int32 [8 n_bs]    packed positions ctx_i + j           */
  DSCALE_WS_KV_REFS = 7,    /* int32 [8 n_bs]    packed cache slots page*16 + t%16    */
  DSCALE_WS_ROW_REQ = 8,    /* int32 [8 n_bs]    request of each packed row, -1 tail  */
  DSCALE_WS_TOP1 = 9,       /* int32 [8 n_bs]    target argmax per packed row         */
  DSCALE_WS_K0 = 10,        /* int32 [n_bs]      seed lengths of Eq. 7                */
  DSCALE_WS_N_LIVE = 11     /* int32 [1]         N as seen by the last allocation     */
};

/*
 * Size in bytes of the workspace for capacity n_bs (the paper's N_bs) and the
 * given head geometry.  num_sms = number of SMs of the device the calls will
 * run on (it fixes the persistent attention grid and its split-KV scratch).
 * Returns 0 for unsupported arguments.  HOST call, no CUDA activity.
 */
size_t dscale_workspace_bytes(int n_bs, int n_q_heads, int n_kv_heads, int head_dim, int num_sms);

/*
 * Prepare a workspace: zeroes the status word, the counters and the index
 * sections (the Alloc(N_bs, 8 N_bs) of Algorithm 2, line 4).  ws must be
 * 256-byte aligned device memory of at least dscale_workspace_bytes(...).
 * Call once, before capturing or running the other calls.
 */
int dscale_workspace_init(void* ws, size_t bytes, int n_bs, int n_q_heads, int n_kv_heads,
                          int head_dim, int num_sms, void* stream);

/*
 * Forget a workspace: removes its registry entry, destroys the step graph that
 * dscale_verify_step_host_graph cached for it, and drops the cached tensor-map
 * descriptors (they are keyed on buffer addresses that the caller is about to
 * free or reuse).  HOST call; call it before freeing the workspace memory, with
 * no work on the workspace in flight.  The device memory itself stays the
 * caller's.  Returns DSCALE_ERR_WORKSPACE for a pointer that is not registered.
 */
int dscale_workspace_destroy(void* ws);

/*
 * DVL allocation and flat-pack (Algorithm 1 from its second line; Eq. 6, 7, 9, 10, 11).
 *
 *   n_live        [1]  N, 1 <= N <= n_bs, read on the device
 *   scores        fp32 [n_bs][15]; slot j = 1..15.  scores_are_logits = 0: the
 *                 values are per-position acceptance probabilities in [0,1];
 *                 = 1: predictor logits, the sigmoid of Algorithm 1 is applied.
 *                 A running minimum (Eq. 6) is always applied.
 *   draft_tokens  int32 [n_bs][16]; slot 0 = anchor
 *   ctx_len       int32 [n_bs]; tokens of request i already in the cache, the
 *                 anchor excluded.  The K/V of slot j is expected at logical
 *                 position ctx_len[i] + j.
 *   block_table   int32 [n_bs][max_pages]
 *
 * Writes into the workspace: Q, k0, k, offset, q_start, q_end, packed tokens,
 * positions (ctx_i + j), kv_refs (page * 16 + slot), row_req, the sentinels of
 * Algorithm 1's last two lines, and the tile schedule the attention kernel
 * reads.  sum_i k_i = 8 N exactly, 1 <= k_i <= 16, ties in the grow / shrink
 * choice go to the lowest request index.  One kernel, one thread block.
 */
int dscale_alloc_verify(void* ws, int n_bs, const int32_t* n_live, const float* scores,
                        int scores_are_logits, const int32_t* draft_tokens,
                        const int32_t* ctx_len, const int32_t* block_table, int max_pages,
                        int num_pages, void* stream);

/*
 * The same allocation for another block width and / or another verification
 * budget.  block_width = W is the number of slots a request's block has (even,
 * 2..16; the paper's drafters have 16 and it leaves other widths open): only the
 * first W - 1 scores and W draft tokens of each row are read (the array shapes
 * stay [n_bs][15] and [n_bs][16]), seeds are clipped to [1, W], no request grows
 * beyond W.  budget_rows is a nullable device int32[1] read by the kernel:
 * sum_i k_i = budget_rows; null means W N / 2 (Eq. 3; Eq. 9 holds for any
 * total).  Served range: N <= budget_rows <= min(W N, 8 n_bs) (every request
 * keeps its anchor, none exceeds its block, the packed arrays keep their 8 n_bs
 * rows); a value outside is clamped into the range and DSCALE_STATUS_BAD_LEN is
 * set.  Everything downstream reads M_live from the workspace and needs no
 * change.  DSCALE_ERR_UNSUPPORTED for an odd or out-of-range block_width.
 */
int dscale_alloc_verify_ex(void* ws, int n_bs, const int32_t* n_live, const float* scores,
                           int scores_are_logits, const int32_t* draft_tokens,
                           const int32_t* ctx_len, const int32_t* block_table, int max_pages,
                           int num_pages, int block_width, const int32_t* budget_rows, void* stream);

/*
 * Packed ragged verify attention for one layer (Section 3.2; Eq. 15 and the
 * sentence after it).  For live request i, row j < k_i, q-head h:
 *     out[offset_i + j][h] = softmax(q[offset_i + j][h] . K^T * sm_scale) V
 * over the logical keys 0 .. positions[offset_i + j] of request i (its whole
 * committed context and the window slots up to j), kv-head h / group.  Rows
 * at or beyond M_live are written as zero.  Lengths, offsets and positions are
 * the ones dscale_alloc_verify left in the workspace.
 *
 * The query tile is sized to the live rows: one 64-row tensor-core tile holds
 * the 4 q-heads of a GQA group times the <= 16 window rows, so each K/V page is
 * read from HBM once per kv-head.  Requires n_q_heads / n_kv_heads == 4;
 * returns DSCALE_ERR_UNSUPPORTED otherwise (use dscale_verify_attn_simt).
 *
 *   q, out        bf16 [8 n_bs][n_q_heads][128], 16-byte aligned
 *   k_cache, v_cache  bf16 [num_pages][n_kv_heads][16][128], 16-byte aligned
 */
int dscale_verify_attn(void* ws, int n_bs, const void* q, const void* k_cache,
                       const void* v_cache, const int32_t* block_table, int max_pages,
                       int num_pages, int n_q_heads, int n_kv_heads, float sm_scale, void* out,
                       void* stream);

/*
 * Same operation and arguments on plain CUDA cores (no tensor cores, any GQA
 * group size that divides n_q_heads).  Slow; kept as the in-library
 * cross-check of the tensor-core kernel and for shapes it does not cover.
 */
int dscale_verify_attn_simt(void* ws, int n_bs, const void* q, const void* k_cache,
                            const void* v_cache, const int32_t* block_table, int max_pages,
                            int num_pages, int n_q_heads, int n_kv_heads, float sm_scale,
                            void* out, void* stream);

/*
 * Comparison baseline, not part of the method: verify attention the way the
 * paper describes the native path (Section 2.1) -- every live request verifies
 * all W = 16 slots, and each (request, q-head) owns one 128-row tile of which
 * 16 rows are live (Eq. 2: 112 masked rows, 87.5 %).  K/V are streamed once per
 * q-head.  Same kernel machinery as dscale_verify_attn otherwise.
 *
 *   q_unpacked, out_unpacked   bf16 [n_bs][16][n_q_heads][128]; row j of request i
 *                 sees the logical keys 0 .. ctx_len[i] + j; requests >= N are
 *                 written as zero
 *   ctx_len       int32 [n_bs], as given to dscale_alloc_verify (N is taken from
 *                 the workspace, so an allocation must have run)
 */
int dscale_verify_attn_padded(void* ws, int n_bs, const void* q_unpacked, const void* k_cache,
                              const void* v_cache, const int32_t* block_table, int max_pages,
                              int num_pages, const int32_t* ctx_len, int n_q_heads,
                              int n_kv_heads, float sm_scale, void* out_unpacked, void* stream);

/*
 * Greedy prefix verification and output building ("Prefix verifier" paragraph;
 * Algorithm 2, lines 21-26).  top1[s] = first index of the maximum of
 * logits[s][0..vocab) for s < M_live (a NaN never counts as a maximum).
 * Request i accepts candidates while top1[offset_i + a] == tokens[offset_i + a + 1],
 * a < k_i - 1; the successor is top1[offset_i + a_i].
 *
 *   accept_len   int32 [n_bs]      a_i (0 for sentinels)
 *   next_anchor  int32 [n_bs]      successor token (-1 for sentinels)
 *   out_tokens   int32 [n_bs][16]  accepted candidates, then the successor, then -1
 *   out_len      int32 [n_bs]      a_i + 1 (0 for sentinels)
 *   ctx_len_inout  nullable; if given, ctx_len[i] += a_i + 1 for live i (the
 *                 boundary write-back; not idempotent across replays)
 */
int dscale_accept(void* ws, int n_bs, const float* logits, int64_t ld, int vocab,
                  int32_t* accept_len, int32_t* next_anchor, int32_t* out_tokens,
                  int32_t* out_len, int32_t* ctx_len_inout, void* stream);

/*
 * One whole verify step driven from HOST buffers: what Algorithm 2 does between
 * "stage inputs" and "read outputs" (lines 10-21).  The staged inputs
 * (N, scores, draft tokens, context lengths, block table) are copied from host
 * memory into `staging`, the three stages are enqueued (allocation, attention
 * for each of n_layers layers, acceptance), and the outputs are copied back to
 * host memory, all asynchronously on `stream`; the results are valid after the
 * caller synchronises the stream.  Host buffers should be page-locked: the
 * staged inputs are then fetched, and the results written back, by one small
 * kernel each over the buffers' device mapping (2 launches more per step);
 * pageable buffers are served by ordinary copies, which are then not asynchronous.
 *
 *   h_*          HOST pointers, same shapes as in the per-stage calls
 *   staging      DEVICE scratch of at least dscale_step_staging_bytes(n_bs, max_pages)
 *                bytes, 256-byte aligned, owned by the caller, reused every step
 *   layers       HOST array of n_layers entries of DEVICE pointers (q, k_cache,
 *                v_cache, out of each layer; layouts as in dscale_verify_attn)
 *   logits       DEVICE fp32 [8 n_bs][ld] (produced on the device by the LM head)
 */
typedef struct dscale_layer {
  const void* q;
  const void* k_cache;
  const void* v_cache;
  void* out;
} dscale_layer;

size_t dscale_step_staging_bytes(int n_bs, int max_pages);

int dscale_verify_step_host(void* ws, int n_bs, const int32_t* h_n_live, const float* h_scores,
                            const int32_t* h_draft_tokens, const int32_t* h_ctx_len,
                            const int32_t* h_block_table, int max_pages, int num_pages,
                            void* staging, const dscale_layer* layers, int n_layers,
                            int n_q_heads, int n_kv_heads, float sm_scale, const float* logits,
                            int64_t ld, int vocab, int32_t* h_accept_len, int32_t* h_next_anchor,
                            int32_t* h_out_tokens, int32_t* h_out_len, void* stream);

/*
 * The same step as ONE replayed CUDA graph, which is what Algorithm 2 does: stage
 * the inputs at fixed addresses, replay, read the outputs (lines 10-21).  Same
 * arguments and results as dscale_verify_step_host.  The first call with a given
 * set of arguments captures the copies and launches into a graph and instantiates
 * it (this allocates driver memory and takes about a millisecond); later calls
 * with the same pointers and sizes only launch that graph.  One graph is kept per
 * workspace; other arguments replace it.  The host buffers must stay where they
 * are between calls (their addresses are part of the graph) and must be
 * page-locked.  If `stream` is already being captured, or is the legacy default
 * stream, the call degrades to dscale_verify_step_host.
 */
int dscale_verify_step_host_graph(void* ws, int n_bs, const int32_t* h_n_live, const float* h_scores,
                                  const int32_t* h_draft_tokens, const int32_t* h_ctx_len,
                                  const int32_t* h_block_table, int max_pages, int num_pages,
                                  void* staging, const dscale_layer* layers, int n_layers,
                                  int n_q_heads, int n_kv_heads, float sm_scale, const float* logits,
                                  int64_t ld, int vocab, int32_t* h_accept_len, int32_t* h_next_anchor,
                                  int32_t* h_out_tokens, int32_t* h_out_len, void* stream);

/*
 * Fused LM head + greedy prefix verification: dscale_accept without the logits.
 * The target token of packed row s is argmax_v sum_h hidden[s][h] * weight[v][h]
 * (the LM head applied to the M = 8N packed rows DVL leaves: Section 2.2 and the
 * last sentence of Section 3.2), computed
 * on the tensor cores tile by tile with a running (max, first index) per row, so
 * the 8N x V logits are never written; then the same acceptance loop and outputs
 * as dscale_accept (Algorithm 2, lines 21-26).
 *
 *   hidden   bf16 [8 n_bs][hidden_dim], packed rows, hidden_dim % 64 == 0
 *   weight   bf16 [vocab][hidden_dim] (one row per vocabulary entry), vocab >= 16
 *   row_max  nullable fp32 [8 n_bs]: receives the winning logit of every live row
 * Products are accumulated in fp32; two logits closer than fp32 rounding of the
 * dot product may resolve differently from an exact evaluation.
 * All pointers are device pointers owned by the caller; hidden and weight must be
 * 16-byte aligned.  dscale_alloc_verify must have run on ws for this step.  Outputs
 * as for dscale_accept.  One launch on `stream`, no allocation, no synchronisation;
 * the first call on a device queries the occupancy of the CTA-pair kernel and
 * should come before any stream capture.  Returns DSCALE_ERR_UNSUPPORTED for
 * hidden_dim % 64 != 0 or vocab < 16 (and for more than 128 packed rows on a device
 * that cannot keep a cluster of two CTAs resident), DSCALE_ERR_WORKSPACE for an unknown ws,
 * DSCALE_ERR_INVALID_ARG for null or misaligned pointers.
 */
int dscale_lm_head_accept(void* ws, int n_bs, const void* hidden, const void* weight, int hidden_dim,
                          int vocab, int32_t* accept_len, int32_t* next_anchor, int32_t* out_tokens,
                          int32_t* out_len, int32_t* ctx_len_inout, float* row_max, void* stream);

/*
 * Acceptance-predictor front end ("Acceptance predictor" paragraph, Eq. 4 and
 * Eq. 5): the step before dscale_alloc_verify.  For every live request and each
 * of its 15 new draft positions p:
 *   confidence (18): top drafter logit; its gaps to the logits of ranks 2..16;
 *                    log-probability of the top token; entropy of softmax(z)
 *   hidden projection (64):  p_hidden  . draft_hidden[i][p]
 *   logit projection (32):   p_logit . (z - mean(z)),  z = draft_logits[i][p]
 * features_i = [confidence (270, position-major) | hidden projections (960) |
 * logit projections (480) | batch context (25: entry 0 = N, entry 3 = 1)]: 1735
 * values; pred_logits[i] = w2 relu(w1 features_i + b1) + b2.  The result is what
 * dscale_alloc_verify takes as `scores` with scores_are_logits = 1.
 *
 *   n_live        device int32[1]
 *   draft_logits  fp32 [n_bs][15][ld], ld >= vocab, ld % 4 == 0, finite values
 *   draft_hidden  bf16 [n_bs][15][hidden_dim], hidden_dim % 8 == 0
 *   p_hidden      bf16 [64][hidden_dim]      p_logit  bf16 [32][vocab]
 *   w1 fp32 [64][1735], b1 fp32 [64], w2 fp32 [15][64], b2 fp32 [15]
 *   pred_logits   fp32 [n_bs][15] out; rows of requests >= N are set to 0
 *   features_out  nullable fp32 [n_bs][1735] out (rows >= N set to 0)
 * fp32 arithmetic; the logit projection rounds (z - z[0]) to tf32 for the tensor
 * cores (the centring is applied afterwards, exactly).  All pointers are device
 * pointers owned by the caller, 16-byte aligned.  Four launches on `stream`, no
 * allocation, no synchronisation; scratch lives in ws.  vocab >= 16.
 * Errors: DSCALE_ERR_INVALID_ARG (null / misaligned), DSCALE_ERR_UNSUPPORTED
 * (shape rules above), DSCALE_ERR_WORKSPACE (unknown ws).
 */
int dscale_predict_scores(void* ws, int n_bs, const int32_t* n_live, const float* draft_logits, int64_t ld,
                          int vocab, const void* draft_hidden, int hidden_dim, const void* p_hidden,
                          const void* p_logit, const float* w1, const float* b1, const float* w2,
                          const float* b2, float* pred_logits, float* features_out, void* stream);

/*
 * Prefix verification under a sampling target policy ("Prefix verifier"
 * paragraph, temperature > 0).  P = softmax(logits / temperature) at each packed
 * row.  The candidate x in slot j + 1 is accepted iff u_accept[offset_i + j] < P(x);
 * at the first rejection the successor is drawn from P with x removed and the
 * rest renormalised, and if all k_i - 1 selected candidates pass it is drawn
 * from the unmodified P of the last selected row.  The draw is the first index
 * whose cumulative weight exceeds u_draw[i] times the total (inverse CDF in
 * index order).  Random numbers are inputs, so the lengths do not depend on them
 * and a replayed graph only needs fresh uniforms at the same addresses.
 *
 *   u_accept  fp32 [8 n_bs], one uniform in [0,1) per packed row
 *   u_draw    fp32 [n_bs],   one uniform in [0,1) per request
 *   p_draft   nullable fp32 [8 n_bs]: receives P(candidate) of every row that has one
 *   outputs   as in dscale_accept
 * Logits must be finite.  Probabilities are evaluated in fp32; a draw whose
 * target falls within rounding of a boundary of the cumulative sum may return
 * the neighbouring token.  vocab <= DSCALE_SAMPLING_MAX_VOCAB (the draw kernel
 * keeps one partial sum per 1024 tokens in a fixed table), otherwise
 * DSCALE_ERR_TOO_LARGE and nothing is enqueued.
 */
#define DSCALE_SAMPLING_MAX_VOCAB (1 << 20)
int dscale_accept_sampling(void* ws, int n_bs, const float* logits, int64_t ld, int vocab,
                           float temperature, const float* u_accept, const float* u_draw,
                           int32_t* accept_len, int32_t* next_anchor, int32_t* out_tokens,
                           int32_t* out_len, float* p_draft, void* stream);

/*
 * Greedy prefix verification for callers that can neither allocate nor keep a
 * workspace.  (The paper has no counterpart to this call: it exists for
 * deployment reasons only.)  Typical users: a serving loop in which a cudaMalloc
 * would stall every stream of the device, or a plug-in that only receives input
 * and output pointers from its host runtime.  Same result as dscale_accept, but
 * the lengths, offsets and packed tokens are passed in explicitly and the
 * scratch of the row argmax lives in a fixed __device__ array inside the
 * library (about 66 KB per GPU, held until the process exits).  The call
 * allocates nothing and frees nothing.
 *
 *   n_live [1], k [n_bs], offset [n_bs + 1], tokens [8 n_bs]   int32, device:
 *         as produced by dscale_alloc_verify (workspace fields N_LIVE, K,
 *         OFFSET, TOKENS) or by the caller, under any budget and block width
 *         that dscale_alloc_verify_ex serves: the number of live packed rows is
 *         read on the device as offset[N] (clamped to 8 n_bs)
 *   logits, ld, vocab and the four outputs: as in dscale_accept
 * A live request whose rows do not lie inside the live packed rows (k outside
 * 1..16, a negative offset, offset + k beyond offset[N]) gets the outputs of a
 * sentinel (length 0, next anchor -1); there is no status word in this call.
 *
 * Limits and rules: n_bs <= DSCALE_ACCEPT_STATIC_MAX_NBS, otherwise
 * DSCALE_ERR_TOO_LARGE is returned and nothing is enqueued.  All calls on a GPU
 * share the one scratch array, so two calls that may run at the same time on
 * that GPU (different streams or threads) race: serialise them.  The first call
 * on each device looks up the array's address; make that call before any stream
 * capture begins.
 */
#define DSCALE_ACCEPT_STATIC_MAX_NBS 64
int dscale_accept_static(int n_bs, const int32_t* n_live, const int32_t* k, const int32_t* offset,
                         const int32_t* tokens, const float* logits, int64_t ld, int vocab,
                         int32_t* accept_len, int32_t* next_anchor, int32_t* out_tokens,
                         int32_t* out_len, void* stream);

/*
 * Bucket selection for a pool of captured capacities (Eq. 13):
 * N_bs = min{ b in buckets : b >= n_live }.  HOST call.  Returns the chosen
 * capacity, or DSCALE_ERR_TOO_LARGE if no bucket is large enough,
 * DSCALE_ERR_INVALID_ARG for an empty / non-positive bucket set or n_live < 1.
 * Each bucket has its own workspace and captured graph (Algorithm 2, lines 3-8);
 * requests beyond n_live inside the chosen bucket are sentinels (Eq. 14).
 */
int dscale_select_bucket(const int32_t* buckets, int n_buckets, int n_live);

/*
 * Device address of a workspace field (see DSCALE_WS_*), for tests and for
 * callers that feed packed fields to other kernels.  HOST call; returns NULL
 * for a bad field id.  The address depends only on (ws, n_bs).
 */
const int32_t* dscale_ws_field(const void* ws, int n_bs, int field);

/* Number of kernels the three stage calls enqueue (for launch accounting):
 * which = 0 alloc, 1 attention, 2 accept, 3 attention (simt), 4 attention (padded),
 * 5 accept (sampling), 6 fused LM head + accept, 7 predictor front end. */
int dscale_launches_per_call(int which);

#ifdef __cplusplus
}
#endif
#endif  /* DSCALE_H_ */
