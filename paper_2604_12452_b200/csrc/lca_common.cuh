// Shared declarations of the LCA CUDA library (device helpers, launch bookkeeping).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/lca.h"

namespace lca {

typedef __nv_bfloat16 bf16;
typedef __nv_bfloat162 bf162;

// Launch bookkeeping (lca_launch_count).
void note_launch(int n = 1);

// Partition of Sec. 4.2 on the host.
inline void partition(int64_t L, int64_t w, int64_t g, int64_t* m, int64_t* k) {
  if (L < w + g) { *m = 0; *k = L; return; }
  *m = (L - w) / g;
  *k = L - (*m) * g;
}

// Representatives visible to the query at 0-based position p (prefix length p+1).
__host__ __device__ inline int reps_visible(int p, int w, int g) {
  int t = p + 1;
  return (t < w + g) ? 0 : (t - w) / g;
}

// Ragged batches (sequences of different lengths packed one after the other).  Device arrays of B + 1 prefix sums:
// first token row, first cache row and first group of every sequence.  tok_off == nullptr means a uniform batch
// (every sequence p->seq_len long), where the same quantities follow from the batch index by multiplication.
struct SeqTab {
  const int32_t* tok_off;
  const int32_t* cache_off;
  const int32_t* grp_off;
  int B;
};
// Largest b in [0, B) with off[b] <= x (off is non-decreasing, off[0] = 0 <= x < off[B]).
__device__ inline int seq_of(const int32_t* off, int B, long long x) {
  int lo = 0, hi = B - 1;
  while (lo < hi) {
    const int mid = (lo + hi + 1) >> 1;
    if ((long long)off[mid] <= x) lo = mid; else hi = mid - 1;
  }
  return lo;
}

// Bytes of the device copy of the three prefix arrays (at the start of the workspace of a ragged call).
inline size_t seq_table_bytes(int B) { return ((size_t)3 * (B + 1) * sizeof(int32_t) + 15) / 16 * 16; }

// Rows of a sequence's decode cache that take part in the attention (Sec. 4.3), for both cache layouts:
//   packed  [representatives ; tokens in order]: rows [0, cache_rows[b]); the first n_rep_bias of them are representatives;
//   ring    the uncondensed tokens in a ring of R = window + group_size rows (token number n of the sequence at row
//           n % R), the representatives in group order from row R on.  With n_rep representatives and n_tok tokens so
//           far the uncondensed tokens are n_rep*g .. n_tok-1 (at most R of them); the ring rows between the newest
//           token and the oldest uncondensed one hold condensed tokens that have not been overwritten yet.  Because
//           groups leave the ring whole and R is a multiple of g, those rows are one run that does not wrap.
struct DecodeLayout {
  const int32_t* cache_rows;                               // packed layout
  const int32_t* ring_n_rep; const int32_t* ring_n_tok;    // ring layout (ring_n_tok != nullptr)
  int cap, n_rep_bias, R, g;
};
// Row x takes part iff x < rows_end and not inv_lo <= x < inv_hi; it gets the representatives' bias iff bias_lo <= x < bias_hi.
struct DecodeSpan { int rows_end, inv_lo, inv_hi, bias_lo, bias_hi; };
__device__ __forceinline__ DecodeSpan decode_span(const DecodeLayout& d, int b) {
  DecodeSpan s;
  if (!d.ring_n_tok) {
    s.rows_end = min(max(d.cache_rows[b], 0), d.cap);
    s.inv_lo = s.inv_hi = s.rows_end;
    s.bias_lo = 0; s.bias_hi = min(d.n_rep_bias, s.rows_end);
    return s;
  }
  const int n_rep = min(max(d.ring_n_rep[b], 0), max(d.cap - d.R, 0));
  const long long first = (long long)n_rep * d.g;          // oldest uncondensed token
  const int c = (int)min(max((long long)d.ring_n_tok[b] - first, 0ll), (long long)d.R);
  if (n_rep == 0) {                                        // the ring has not wrapped: tokens 0 .. c-1 at rows 0 .. c-1
    s.rows_end = min(c, d.cap);
    s.inv_lo = s.inv_hi = s.rows_end;
    s.bias_lo = s.bias_hi = 0;
    return s;
  }
  s.rows_end = d.R + n_rep;
  s.bias_lo = d.R; s.bias_hi = s.rows_end;
  const int h = (int)(first % d.R);                        // row of the oldest uncondensed token
  if (c == d.R) { s.inv_lo = s.inv_hi = 0; }
  else {
    s.inv_lo = (h + c) % d.R;                              // row the next token will take
    s.inv_hi = h == 0 ? d.R : h;
    if (s.inv_lo > s.inv_hi) s.inv_hi = d.R;               // fewer than `window` tokens behind representatives: not a state the update produces
  }
  return s;
}

__device__ inline double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ inline float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// ---- host-side launchers implemented in the .cu files ---------------------------------------
struct CondenseLaunch {
  const lca_params* p;
  const void* q_tail_sem; const void* q_tail_pos; int64_t q_tail_batch_stride;
  const float* qbar_opt;
  const void* kv_sem; const void* kv_pos;
  void* cache_sem; void* cache_pos; int32_t* anchor_idx; double* scores_opt;
  void* ws; size_t ws_bytes; cudaStream_t stream;
  // ragged batch: host prefix sums (B + 1 entries each) and their device copies; all null for a uniform batch
  const int32_t* h_tok_off; const int32_t* h_cache_off; const int32_t* h_grp_off;
  SeqTab tab;
};
size_t condense_workspace_bytes(const lca_params* p);
int condense_launch(const CondenseLaunch& a);
size_t condense_smem_bytes(const lca_params* p);
size_t update_workspace_bytes(const lca_params* p);
size_t update_smem_bytes(const lca_params* p);
// n_tok == nullptr: packed layout (n_rows in / out); otherwise ring layout (n_rows unused, n_tok read only)
int update_launch(const lca_params* p, const void* q_tail_sem, const void* q_tail_pos, int64_t q_tail_batch_stride,
                  const float* qbar_opt, void* cache_sem, void* cache_pos, int cap, int32_t* n_rep, int32_t* n_rows,
                  const int32_t* n_tok, int32_t* anchor_out, void* ws, cudaStream_t stream);
int update_step_launch(const lca_params* p, const void* q_sem, const void* q_pos, double* qsum, int32_t* qcount,
                       void* ring_sem, void* ring_pos, int cap, int32_t* n_rep, const int32_t* n_tok,
                       int32_t* anchor_out, void* ws, cudaStream_t stream);
int ring_from_packed_launch(const lca_params* p, const void* packed_sem, const void* packed_pos, const int32_t* packed_rows,
                            const int32_t* n_rep, int packed_cap, void* ring_sem, void* ring_pos, int ring_cap,
                            int32_t* n_tok_out, cudaStream_t stream);
int condense_take_status();   // nonzero once if a bounded wait of the condense kernel expired
int condense_static_scratch_address(void** out);   // device address of the library's fixed scratch array

// One description of an attention problem for every implementation.  Each query row (b, t, h)
// attends to   A) rows [0, n_a) of a "cache" source   and   B) rows [b_first, b_last] of a
// "token" source, where for prefill n_a = reps_visible(t), B = [n_a*g, t], and for decode
// A = the rows of the sequence's cache that decode_span() names, B empty.  The first min(n_a, bias_rows)
// A rows receive rep_logit_bias (prefill: all of them; decode: the rows decode_span() names).
struct AttnProblem {
  int variant;                 // LCA_VARIANT_*
  int batch, q_len, n_q_heads, n_kv_heads, d_sem, d_pos;
  int decode;                  // 0 prefill, 1 decode
  int seq_len, group_size, window;       // prefill only
  const int32_t* cache_rows;   // decode only (device)
  int cache_row_capacity;      // rows per sequence in the cache arrays
  int n_rep_bias;              // decode: rows that get the bias
  // decode over the ring layout (see DecodeLayout): per-sequence counters (device); null = packed layout.
  // group_size and window then give the ring size.
  const int32_t* ring_n_rep; const int32_t* ring_n_tok;
  float softmax_scale, rep_logit_bias;
  const void* q_sem; const void* q_pos;  // [B, q_len, H, d]
  const void* kv_sem; const void* kv_pos;        // [B, seq_len, Hkv, d]  (prefill)
  const void* cache_sem; const void* cache_pos;  // [B, cap, Hkv, d]
  void* out; float* lse;                  // [B, q_len, H, d_sem], [B, q_len, H]
  void* ws; size_t ws_bytes;
  cudaStream_t stream;
  // ragged prefill batch: host prefix sums (B + 1 entries) and their device copies; null for a uniform batch.
  // q_len / seq_len then hold the longest sequence, cache_row_capacity is unused.
  const int32_t* h_tok_off; const int32_t* h_cache_off;
  SeqTab tab;
};
int attn_simt_launch(const AttnProblem& a);     // scalar kernel, every supported head shape
bool attn_tc_supported(const AttnProblem& a);   // tensor-core (tcgen05) kernels
size_t attn_tc_workspace_bytes(const AttnProblem& a);
int attn_tc_launch(const AttnProblem& a);
int attn_tc_device_status(cudaStream_t stream);
size_t attn_tc2_ragged_workspace_bytes(int batch, int longest, int n_q_heads);
size_t attn_tc2_decode_workspace_bytes(int batch, int n_q_heads);     // MLA shape, CTA-pair kernel
int bounded_wait_selftest_launch(long long limit_cycles, cudaStream_t stream);
int latent_to_value_launch(const void* latent, const void* w_uv, void* out, long long n_tokens, int n_heads,
                           int d_latent, int d_v, cudaStream_t stream);
int latent_to_value_take_status();

}  // namespace lca
