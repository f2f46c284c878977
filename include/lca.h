/* Latent-Condensed Attention (LCA) for NVIDIA B200 (sm_100a) -- C ABI.
 *
 * The library computes the prefill / decode hot path of LCA: condensation of the distant
 * history in MLA's latent space (query-aware weighted pooling of C^KV, arg-max anchor selection
 * of K^R) followed by attention of the absorbed-form queries [q_latent | q_rope] over the
 * condensed representatives plus the uncondensed local window, and the same dual path for
 * grouped-query attention (pool V, select K).  Section / equation numbers below refer to the
 * paper "Latent-Condensed Transformer for Efficient Long Context Modeling".
 *
 * Conventions that hold for every entry point
 *   - All tensor pointers are DEVICE pointers owned by the caller, 16-byte aligned, dense
 *     row-major with the shapes stated; element type bf16 unless stated.  `lca_params*` is a
 *     HOST pointer.  `stream` is a cudaStream_t passed as void* (NULL = the legacy default stream).
 *   - Calls are asynchronous on `stream`; nothing is allocated, freed or kept between calls
 *     unless an entry point says otherwise; the workspace `ws` may be reused by the next call
 *     on the same stream.
 *   - Return value: LCA_OK (0) or a negative lca_status.  Arguments are validated on the host
 *     first; an invalid call launches nothing and writes nothing.
 *   - Token positions are 0-based in the ABI (the paper's formulas are 1-based).
 *
 * Partition of a length-L sequence (Sec. 4.2): m = floor((L-w)/g) groups of g tokens,
 * G_j = {j*g .. (j+1)*g-1}; the last k = L - m*g = w + (L-w) mod g tokens form the local window.
 * When L < w+g there is no group: m = 0, k = L and every entry point degenerates to plain
 * causal attention (Sec. 4.3).  `lca_partition` returns (m, k).
 *
 * Condensed-cache layout (Sec. 4.3 "Decoding and Online Cache Update"), per sequence:
 *   rows 0..m-1   representatives in group order: cache_sem[j] = c_rep_j (Eq. 7, rounded to
 *                 nearest-even bf16), cache_pos[j] = k^R of the anchor token I_j (Eq. 8, bit copy)
 *   rows m..m+k-1 the last k tokens in token order (bit copies)
 * GQA (Sec. 5.4): the same per KV head with cache_sem = pooled V, cache_pos = selected K.
 */
#ifndef LCA_H_
#define LCA_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum lca_status {
  LCA_OK = 0,
  LCA_ERR_INVALID_ARG = -1,        /* NULL where a pointer is required, non-positive size, ...   */
  LCA_ERR_UNSUPPORTED_SHAPE = -2,  /* a head dimension / group size no kernel is built for       */
  LCA_ERR_MISALIGNED = -3,         /* a tensor pointer that is not 16-byte aligned               */
  LCA_ERR_WORKSPACE_TOO_SMALL = -4,
  LCA_ERR_CUDA = -5,               /* a CUDA runtime call or a launch failed                     */
  LCA_ERR_DEVICE_TIMEOUT = -6,     /* a bounded device-side wait expired (reported by lca_last_device_status) */
  LCA_ERR_STATIC_SCRATCH_EXCEEDED = -7  /* lca_condense_static_scratch: the problem needs more than LCA_STATIC_SCRATCH_BYTES */
} lca_status;

enum { LCA_VARIANT_MLA = 0, LCA_VARIANT_GQA = 1 };
/* How a group is reduced to one vector (Table 5 ablates these for c_rep and for k^R_rep):
 *   MAXPOOL  element-wise maximum over the g tokens      MEANPOOL  plain mean
 *   WEIGHTED sum_i alpha_i x_i with the Eq. 6 weights    MAXSEL    the vector of the arg-max token (Eq. 8)
 * DEFAULT is the method itself: WEIGHTED for the semantic part (Eq. 7), MAXSEL for the positional part. */
enum { LCA_REDUCE_DEFAULT = 0, LCA_REDUCE_MAXPOOL = 1, LCA_REDUCE_MEANPOOL = 2, LCA_REDUCE_WEIGHTED = 3, LCA_REDUCE_MAXSEL = 4 };
enum { LCA_WS_CONDENSE = 0, LCA_WS_PREFILL = 1, LCA_WS_DECODE = 2, LCA_WS_UPDATE = 3,
       LCA_WS_CONDENSE_VARLEN = 4, LCA_WS_PREFILL_VARLEN = 5 };

/* Problem statement = the REQUIRE line of Alg. 1 (L, C^KV, K^R, Q, w, g) plus the head layout.
 *   MLA: n_kv_heads = 1, d_sem = d_c (512), d_pos = d_R (64); logits use [sem | pos], values = sem.
 *   GQA: d_sem = d_pos = head_dim (128); logits use pos (= K) only, values = sem (= V);
 *        n_q_heads must be a multiple of n_kv_heads.
 *   n_summary_q: number of trailing queries averaged into the summary query (Alg. 1, first step;
 *                Table 8 varies it); 0 means g; clamped to L.
 *   softmax_scale: 1/sqrt(d_h), used for the importance scores (Sec. 4.2) and the attention (Eq. 10).
 *   rep_logit_bias: added to the logit of every representative; 0 = Alg. 1 as printed,
 *                log(g) = the group-size-weighted form analysed in the proof of Theorem 1.
 *   sem_reducer / pos_reducer: 0 = the method (Eq. 7 / Eq. 8); other values reproduce the operators
 *                ablated in Table 5 (lca_condense only; lca_decode_update always uses the method's). */
typedef struct lca_params {
  int32_t variant;
  int32_t batch;
  int32_t seq_len;
  int32_t n_q_heads;
  int32_t n_kv_heads;
  int32_t d_sem;
  int32_t d_pos;
  int32_t group_size;
  int32_t window;
  int32_t n_summary_q;
  float softmax_scale;
  float rep_logit_bias;
  int32_t sem_reducer;   /* LCA_REDUCE_*: how lca_condense forms cache_sem[j] (c_rep; GQA: v_rep) */
  int32_t pos_reducer;   /* LCA_REDUCE_*: how it forms cache_pos[j] (k^R_rep; GQA: k_rep).  anchor_idx is always the arg-max token */
} lca_params;

/* (m, k) of Sec. 4.2 for one sequence of p->seq_len tokens.  Host only, no device work. */
int lca_partition(const lca_params* p, int32_t* m, int32_t* k);

/* Bytes of device workspace `which` (LCA_WS_*) needs for these parameters (0 is possible).
 * Returns 0 for invalid parameters as well; the entry point then reports the error. */
size_t lca_workspace_bytes(const lca_params* p, int32_t which);

/* Condensation: Alg. 1 up to the local window (summary query, Eq. 6 group softmax, Eq. 7 pooling, Eq. 8
 * anchors, Eq. 9 local window) for `batch` sequences.
 *   q_tail_sem [B, n, H, d_sem], q_tail_pos [B, n, H, d_pos]: the LAST n = n_summary_q query
 *       positions of each sequence (MLA: q_latent and q_rope; GQA: q_tail_sem = NULL and
 *       q_tail_pos = Q).  q_tail_batch_stride = rows (positions) between consecutive sequences
 *       in these arrays (n for a packed tail, L when pointing into a full [B,L,H,d] tensor).
 *       Ignored (may be NULL) when qbar_opt is given.
 *   qbar_opt   [B, n_kv_heads, dk] fp32, dk = d_sem+d_pos (MLA) or d_pos (GQA), or NULL: a
 *       caller-supplied summary query (e.g. the streaming update of Sec. 4.3).
 *   kv_sem [B, L, n_kv_heads, d_sem], kv_pos [B, L, n_kv_heads, d_pos]: C^KV, K^R (GQA: V, K).
 *   cache_sem [B, m+k, n_kv_heads, d_sem], cache_pos [B, m+k, n_kv_heads, d_pos]: out, layout above.
 *   anchor_idx [B, m, n_kv_heads] int32 out: absolute token index of I_j (lowest index on ties).
 *   scores_opt [B, n_kv_heads, m*g] fp64 out or NULL: the importance scores s_i the kernel used.
 *   ws / ws_bytes: >= lca_workspace_bytes(p, LCA_WS_CONDENSE).
 * The summary query and the importance scores are evaluated in fp64, so the arg-max anchors
 * follow the exact scores (lowest index on exact ties); the group softmax (Eq. 6) and the
 * pooling (Eq. 7) are fp32, and c_rep is rounded once, to bf16 (nearest even). */
int lca_condense(const lca_params* p, const void* q_tail_sem, const void* q_tail_pos,
                 int64_t q_tail_batch_stride, const float* qbar_opt, const void* kv_sem,
                 const void* kv_pos, void* cache_sem, void* cache_pos, int32_t* anchor_idx,
                 double* scores_opt, void* ws, size_t ws_bytes, void* stream);

/* The same condensation for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this entry point exists only for the way the library is called.)
 *
 * Who needs it: code that runs where cudaMalloc is off limits -- a plug-in inside a serving
 * process whose memory is handed out once at start-up by its own pool, a real-time loop that
 * may not take the allocator's lock, a host thread that is not allowed to synchronise the
 * device (cudaMalloc and cudaFree may do that).  lca_condense needs a few hundred KB of scratch
 * for the summary query; here that scratch is a fixed array of LCA_STATIC_SCRATCH_BYTES that is
 * part of the library image on every GPU that loads it, from load until the process exits.
 *
 * Arguments, results and arithmetic are those of lca_condense without `ws` / `ws_bytes`; the
 * output is bit-identical.  The call allocates nothing and frees nothing.
 *   - Limit: lca_workspace_bytes(p, LCA_WS_CONDENSE) must not exceed LCA_STATIC_SCRATCH_BYTES
 *     (1 MiB: one MLA sequence with up to 128 heads and 64 summary positions uses 0.6 MB; a
 *     batch of 64 such sequences does not fit).  Larger problems return
 *     LCA_ERR_STATIC_SCRATCH_EXCEEDED and launch nothing: use lca_condense with your own buffer.
 *   - The first call on each device looks up the array's device address (the device that is
 *     current at the call).  Make that first call outside any stream capture; later calls on the
 *     same device do no set-up work.
 *   - All calls on one device share the one array, and it keeps whatever the previous call left
 *     there.  Nothing in it has to start at zero: every element a call reads was written earlier
 *     in that same call.  Two calls that may overlap on the GPU (different streams, no
 *     dependency between them) race on the array and give wrong results; order them. */
#define LCA_STATIC_SCRATCH_BYTES (1u << 20)
int lca_condense_static_scratch(const lca_params* p, const void* q_tail_sem, const void* q_tail_pos,
                                int64_t q_tail_batch_stride, const float* qbar_opt,
                                const void* kv_sem, const void* kv_pos, void* cache_sem,
                                void* cache_pos, int32_t* anchor_idx, double* scores_opt,
                                void* stream);

/* Prefill attention, Eq. 10 evaluated at every prefix length (causal): the query at position t
 * attends to the representatives of the m_t = floor((t+1-w)/g) groups that lie wholly outside its
 * window (0 if t+1 < w+g; read from rows 0..m_t-1 of the cache) and to the tokens m_t*g..t
 * (read from kv_sem / kv_pos).  window >= seq_len gives dense causal attention (Eq. 5).
 *   q_sem [B, L, H, d_sem] (MLA; NULL for GQA), q_pos [B, L, H, d_pos]
 *   kv_sem, kv_pos, cache_sem, cache_pos: as for lca_condense (the cache may be NULL when m = 0)
 *   out [B, L, H, d_sem] bf16: softmax-weighted sum of the sem vectors (latent space for MLA)
 *   lse_opt [B, L, H] fp32 or NULL: natural-log sum-exp of the logits of each row
 * fp32 softmax and accumulation, bf16 tensor-core products.  `out` may be aligned to 16 bytes only;
 * where it is aligned to 32 bytes the tensor-core kernels store 32 bytes per instruction. */
int lca_prefill_attention(const lca_params* p, const void* q_sem, const void* q_pos,
                          const void* kv_sem, const void* kv_pos, const void* cache_sem,
                          const void* cache_pos, void* out, float* lse_opt, void* ws,
                          size_t ws_bytes, void* stream);

/* Batches of sequences of different lengths (Alg. 1 takes one L per sequence: a batch is `batch` independent runs,
 * each with its own L_b, m_b = floor((L_b - w)/g) and k_b).  The sequences are packed one after the other, without
 * padding, in every tensor:
 *   q_sem / q_pos  [T, H, d]          T = sum of L_b           kv_sem / kv_pos [T, n_kv_heads, d]
 *   cache_sem / cache_pos [R, n_kv_heads, d]   R = sum of (m_b + k_b), each sequence in the layout stated at the top
 *   anchor_idx [M, n_kv_heads]        M = sum of m_b (token indices count from the start of their own sequence)
 *   out [T, H, d_sem], lse_opt [T, H]
 * seq_lens [batch] is a HOST array of positive lengths; p->seq_len is ignored, except that lca_workspace_bytes(p,
 * LCA_WS_CONDENSE_VARLEN / LCA_WS_PREFILL_VARLEN) sizes the workspace for sequences of at most p->seq_len tokens.
 * lca_varlen_layout fills the prefix sums (batch + 1 entries each, any of them may be NULL): first token row, first
 * cache row and first anchor_idx row of every sequence, totals in the last entry.  Host only.
 * lca_condense_varlen takes the WHOLE packed query tensors and averages the last min(n_summary_q, L_b) positions of
 * each sequence (or uses qbar_opt [batch, n_kv_heads, dk]); it does not return the scores.  Results are those of one
 * call per sequence, bit for bit.  The calls copy a few small tables to the device from pageable host memory, which
 * orders the host behind earlier work of `stream`. */
int lca_varlen_layout(const lca_params* p, const int32_t* seq_lens, int64_t* token_offsets,
                      int64_t* cache_row_offsets, int64_t* group_offsets);
int lca_condense_varlen(const lca_params* p, const int32_t* seq_lens, const void* q_sem, const void* q_pos,
                        const float* qbar_opt, const void* kv_sem, const void* kv_pos, void* cache_sem,
                        void* cache_pos, int32_t* anchor_idx, void* ws, size_t ws_bytes, void* stream);
int lca_prefill_attention_varlen(const lca_params* p, const int32_t* seq_lens, const void* q_sem,
                                 const void* q_pos, const void* kv_sem, const void* kv_pos,
                                 const void* cache_sem, const void* cache_pos, void* out, float* lse_opt,
                                 void* ws, size_t ws_bytes, void* stream);

/* Decode attention (Sec. 4.3): one new query per sequence attends to every valid row of that
 * sequence's condensed cache (the caller has appended the new token's own row).
 *   q_sem [B, H, d_sem] (NULL for GQA), q_pos [B, H, d_pos]
 *   cache_sem [B, cache_row_capacity, n_kv_heads, d_sem], cache_pos likewise with d_pos
 *   cache_rows [B] int32 (device): valid rows of each sequence, clamped to [0, cache_row_capacity]
 *       (the tensor-core kernels fetch whole tiles of 128 rows: rows between cache_rows[b] and the
 *       end of the buffers take no part in the result but must hold finite numbers, e.g. zeros)
 *   n_rep: leading rows that are representatives (they receive rep_logit_bias)
 *   out [B, H, d_sem] bf16, lse_opt [B, H] fp32 or NULL
 * p->seq_len, group_size and window are not used here. */
int lca_decode_attention(const lca_params* p, const void* q_sem, const void* q_pos,
                         const void* cache_sem, const void* cache_pos, const int32_t* cache_rows,
                         int32_t cache_row_capacity, int32_t n_rep, void* out, float* lse_opt,
                         void* ws, size_t ws_bytes, void* stream);

/* Online cache update while decoding (Sec. 4.3 "Decoding and Online Cache Update").  The caller
 * appends the row of every newly generated token after the valid rows of its sequence and counts
 * it in cache_rows[b].  This call then looks at every sequence: when its uncondensed tokens
 * (cache_rows[b] - n_rep[b]) have reached window + group_size, the EARLIEST group_size of them are
 * condensed into one representative with the summary query of the last queries (importance
 * scores as in Sec. 4.2, Eq. 6 softmax, Eq. 7 pooling, Eq. 8 anchor), the representative is
 * written to row n_rep[b], the remaining tokens move up by group_size - 1 rows, n_rep[b] grows by
 * one and cache_rows[b] shrinks by group_size - 1: the cache stays at m + w .. m + w + g - 1 rows
 * in the layout [representatives ; tokens in order].  Sequences below the threshold are untouched.
 *   q_tail_sem / q_tail_pos / q_tail_batch_stride / qbar_opt: the last n_summary_q (0 = g) queries
 *       of each sequence or a ready summary query, exactly as for lca_condense
 *   cache_sem [B, cache_row_capacity, n_kv_heads, d_sem], cache_pos likewise: in / out
 *   n_rep [B], cache_rows [B] int32 (device): in / out
 *   anchor_out [B, n_kv_heads] int32 (device): offset 0..g-1 of the anchor token inside the
 *       condensed group, or -1 where nothing was condensed
 *   ws / ws_bytes: >= lca_workspace_bytes(p, LCA_WS_UPDATE); p->seq_len is not used. */
int lca_decode_update(const lca_params* p, const void* q_tail_sem, const void* q_tail_pos,
                      int64_t q_tail_batch_stride, const float* qbar_opt, void* cache_sem,
                      void* cache_pos, int32_t cache_row_capacity, int32_t* n_rep,
                      int32_t* cache_rows, int32_t* anchor_out, void* ws, size_t ws_bytes,
                      void* stream);

/* ---- Ring layout of the decode cache -------------------------------------------------------
 * Sec. 4.3 fixes what the cache holds while decoding (the m representatives and the most recent
 * tokens) and how a group is condensed, not where the rows live.  In the packed layout above the
 * representatives are followed by the tokens in order, so every update moves the whole window up
 * by group_size - 1 rows.  In the ring layout nothing moves:
 *   rows [0, R), R = window + group_size: the uncondensed tokens; token number n of the sequence
 *                (0-based, counted from the start of the sequence) is at row n % R
 *   rows [R, R + n_rep[b]): the representatives in group order
 * State per sequence: n_rep[b] and n_tok[b] (tokens of the sequence so far); the uncondensed tokens
 * are n_rep[b]*group_size .. n_tok[b]-1, at most R of them (and, once a sequence has representatives,
 * at least `window` of them: the state lca_ring_from_packed and every update leave; with fewer, ring rows
 * of condensed tokens would be attended to).  The caller writes the row of a new
 * token at row n_tok[b] % R and then counts it in n_tok[b].  window must be a multiple of group_size
 * (groups leave the ring whole), ring_row_capacity >= R + the representatives the sequence will have;
 * buffers are [B, ring_row_capacity, n_kv_heads, d_sem | d_pos].  Rows that hold nothing yet must hold
 * finite numbers (e.g. zeros), as for lca_decode_attention.
 *
 * lca_ring_from_packed: the step from a packed cache (lca_condense output, or a packed decode cache)
 * to the ring layout: representatives to rows R.., token i of the packed tail to row
 * (n_rep[b]*group_size + i) % R, n_tok_out[b] = n_rep[b]*group_size + packed_rows[b] - n_rep[b].
 *   packed_rows [B], n_rep [B] int32 (device); packed_sem / packed_pos [B, packed_row_capacity, ...].
 *   A sequence with more than R packed tokens, or more representatives than fit behind the ring, is
 *   truncated to what fits (the caller sizes the buffers; nothing is written out of bounds). */
int lca_ring_from_packed(const lca_params* p, const void* packed_sem, const void* packed_pos,
                         const int32_t* packed_rows, const int32_t* n_rep, int32_t packed_row_capacity,
                         void* ring_sem, void* ring_pos, int32_t ring_row_capacity, int32_t* n_tok_out,
                         void* stream);

/* lca_decode_attention over the ring layout: the query attends to the n_rep[b] representatives (each
 * with rep_logit_bias) and to the uncondensed tokens n_rep[b]*g .. n_tok[b]-1 (the caller has written
 * and counted the new token's own row).  Ring rows that still hold tokens of an already condensed
 * group are left out.  Same arithmetic, outputs and workspace (LCA_WS_DECODE) as lca_decode_attention;
 * n_rep, n_tok [B] int32 (device). */
int lca_decode_attention_ring(const lca_params* p, const void* q_sem, const void* q_pos,
                              const void* ring_sem, const void* ring_pos, const int32_t* n_rep,
                              const int32_t* n_tok, int32_t ring_row_capacity, void* out, float* lse_opt,
                              void* ws, size_t ws_bytes, void* stream);

/* lca_decode_update over the ring layout: a sequence with window + group_size uncondensed tokens has
 * its earliest group (ring rows (n_rep[b]*g) % R .. +g-1) condensed exactly as in lca_decode_update;
 * the representative is written to row R + n_rep[b] and n_rep[b] grows by one.  No other row and no
 * other counter changes (n_tok is read only).  A sequence whose representative region is full
 * (R + n_rep[b] == ring_row_capacity) is left alone, anchor_out = -1.
 * Summary-query arguments, anchor_out and workspace (LCA_WS_UPDATE) as for lca_decode_update. */
int lca_decode_update_ring(const lca_params* p, const void* q_tail_sem, const void* q_tail_pos,
                           int64_t q_tail_batch_stride, const float* qbar_opt, void* ring_sem,
                           void* ring_pos, int32_t ring_row_capacity, int32_t* n_rep, const int32_t* n_tok,
                           int32_t* anchor_out, void* ws, size_t ws_bytes, void* stream);

/* The update on the ring layout with a running summary query, called once per decode step after the
 * step's token has been written and counted (Sec. 4.3: an update scores with the mean of the last g queries):
 *   1. qsum[b, hk, :] += sum over the query heads of KV head hk of this step's [q_sem | q_pos] (fp64;
 *      MLA: dk = d_sem + d_pos, GQA: dk = d_pos), qcount[b] += 1;
 *   2. every sequence that is due (window + group_size uncondensed tokens) is condensed exactly as by
 *      lca_decode_update_ring with the summary query qsum / (qcount * heads per KV head), i.e. the mean of
 *      the queries of all steps since its previous update (the last group_size queries when this is
 *      called at every step), and its qsum and qcount are cleared.
 * No query tail is re-read: a step costs the bytes of that step's queries.
 *   q_sem [B, H, d_sem] (NULL for GQA), q_pos [B, H, d_pos]: this step's queries
 *   qsum [B, n_kv_heads, dk] fp64, qcount [B] int32 (device, in / out): zero them when a sequence
 *        starts; to include queries of the prefill, call this with them before decoding starts (a
 *        sequence that is not due only accumulates)
 *   the other arguments as for lca_decode_update_ring; p->n_summary_q must be 0 or group_size. */
int lca_decode_step_update_ring(const lca_params* p, const void* q_sem, const void* q_pos, double* qsum,
                                int32_t* qcount, void* ring_sem, void* ring_pos, int32_t ring_row_capacity,
                                int32_t* n_rep, const int32_t* n_tok, int32_t* anchor_out, void* ws,
                                size_t ws_bytes, void* stream);

/* Value up-projection of the latent attention output (Alg. 1: v = c W^UV; Sec. 4.3: in the absorbed
 * form the attention result lives in the latent space and W^UV is applied to it once per query and
 * head):   out_v[t, h, :] = attn_latent[t, h, :] . W^UV[h]
 *   attn_latent [n_tokens, n_heads, d_latent] bf16: `out` of lca_prefill_attention / lca_decode_attention
 *                                                   (n_tokens = batch * seq_len, or batch for decode)
 *   w_uv        [n_heads, d_latent, d_v] bf16 (d_v contiguous)
 *   out_v       [n_tokens, n_heads, d_v] bf16 (products in bf16 on the tensor cores, fp32 sums, one rounding)
 * Built for d_latent = 512, d_v = 128 (DeepSeek-V2 / V3); other sizes return LCA_ERR_UNSUPPORTED_SHAPE.
 * Needs no workspace.  n_tokens = 0 is a no-op. */
int lca_latent_to_value(const void* attn_latent, const void* w_uv, void* out_v, int64_t n_tokens,
                        int32_t n_heads, int32_t d_latent, int32_t d_v, void* stream);

/* Which attention implementation lca_prefill_attention / lca_decode_attention use:
 *   0 = automatic (tensor-core kernels where the shape is supported, else the scalar kernel),
 *   1 = force the scalar (CUDA-core) kernel, 2 = force the tensor-core kernel (unsupported
 *   shapes then return LCA_ERR_UNSUPPORTED_SHAPE).  Process-wide; returns the previous value. */
int lca_set_attention_impl(int impl);

/* Number of kernels the library has launched since it was loaded (all entry points). */
int64_t lca_launch_count(void);

/* Status word written by bounded device-side waits of the most recent tensor-core launch on the
 * current device: 0 = none expired.  Synchronises `stream`.  Returns LCA_OK or
 * LCA_ERR_DEVICE_TIMEOUT / LCA_ERR_CUDA. */
int lca_last_device_status(void* stream);

/* Self-test of the time-out mechanism (the paper has no counterpart).  Every device-side wait of
 * the tensor-core kernels gives up after a fixed number of SM cycles, records a code in the status
 * word that lca_last_device_status reads, and the kernel returns in an orderly way.  This call
 * launches a one-thread kernel that waits, with the same routine and a limit of `limit_cycles`
 * (1 .. 1e8), on a barrier nobody ever arrives on: afterwards lca_last_device_status returns
 * LCA_ERR_DEVICE_TIMEOUT once, and the next ordinary call works as usual.  Nothing faults, traps or
 * waits longer than the limit. */
int lca_selftest_bounded_wait(int64_t limit_cycles, void* stream);

const char* lca_status_string(int status);
int lca_version(void);

#ifdef __cplusplus
}
#endif
#endif /* LCA_H_ */
