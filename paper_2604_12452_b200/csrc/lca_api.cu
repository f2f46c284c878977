// C-ABI entry points of the LCA library: host-side validation and dispatch to the kernels.
#include <atomic>
#include <vector>

#include "lca_common.cuh"

namespace lca {
static std::atomic<long long> g_launches{0};
static std::atomic<int> g_attn_impl{0};
void note_launch(int n) { g_launches.fetch_add(n); }

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

static int check_params(const lca_params* p, bool need_partition) {
  if (!p) return LCA_ERR_INVALID_ARG;
  if (p->variant != LCA_VARIANT_MLA && p->variant != LCA_VARIANT_GQA) return LCA_ERR_INVALID_ARG;
  if (p->batch <= 0 || p->n_q_heads <= 0 || p->n_kv_heads <= 0 || p->d_sem <= 0 || p->d_pos <= 0)
    return LCA_ERR_INVALID_ARG;
  if (p->n_q_heads % p->n_kv_heads != 0) return LCA_ERR_INVALID_ARG;
  if (p->variant == LCA_VARIANT_MLA && p->n_kv_heads != 1) return LCA_ERR_INVALID_ARG;
  if (!(p->softmax_scale > 0.f) || !(p->rep_logit_bias == p->rep_logit_bias)) return LCA_ERR_INVALID_ARG;
  if (p->sem_reducer < 0 || p->sem_reducer > 4 || p->pos_reducer < 0 || p->pos_reducer > 4) return LCA_ERR_INVALID_ARG;
  if (need_partition) {
    if (p->seq_len <= 0 || p->group_size <= 0 || p->window < 0 || p->n_summary_q < 0)
      return LCA_ERR_INVALID_ARG;
  }
  // feature dimensions must be whole 16-byte rows for the vectorised paths
  if (p->d_sem % 8 != 0 || p->d_pos % 8 != 0) return LCA_ERR_UNSUPPORTED_SHAPE;
  return LCA_OK;
}

static bool simt_shape_ok(const lca_params* p) {
  if (p->variant == LCA_VARIANT_MLA) return (p->d_sem == 512 || p->d_sem == 128) && p->d_pos == 64;
  return (p->d_sem == 128 && p->d_pos == 128) || (p->d_sem == 64 && p->d_pos == 64);
}

// Prefix sums of a ragged batch on the host: tokens, cache rows (m_b + k_b) and groups (m_b) before sequence b.
struct HostSeqTable {
  std::vector<int32_t> tok, cache, grp;
  int longest = 0;
};
static int build_seq_table(const lca_params* p, const int32_t* seq_lens, HostSeqTable* t) {
  const int B = p->batch;
  t->tok.assign(B + 1, 0); t->cache.assign(B + 1, 0); t->grp.assign(B + 1, 0);
  long long tok = 0, cache = 0, grp = 0;
  for (int b = 0; b < B; ++b) {
    if (seq_lens[b] <= 0) return LCA_ERR_INVALID_ARG;
    int64_t m, k;
    partition(seq_lens[b], p->window, p->group_size, &m, &k);
    tok += seq_lens[b]; cache += m + k; grp += m;
    if (tok > 0x7fffff00ll) return LCA_ERR_UNSUPPORTED_SHAPE;     // row coordinates are 32-bit
    t->tok[b + 1] = (int32_t)tok; t->cache[b + 1] = (int32_t)cache; t->grp[b + 1] = (int32_t)grp;
    if (seq_lens[b] > t->longest) t->longest = seq_lens[b];
  }
  return LCA_OK;
}
// Copies the three arrays to the start of `ws` (stream-ordered) and returns the device view.
static int upload_seq_table(const HostSeqTable& t, int B, void* ws, cudaStream_t stream, SeqTab* tab) {
  int32_t* d = static_cast<int32_t*>(ws);
  const size_t n = (size_t)(B + 1) * sizeof(int32_t);
  if (cudaMemcpyAsync(d, t.tok.data(), n, cudaMemcpyHostToDevice, stream) != cudaSuccess ||
      cudaMemcpyAsync(d + (B + 1), t.cache.data(), n, cudaMemcpyHostToDevice, stream) != cudaSuccess ||
      cudaMemcpyAsync(d + 2 * (B + 1), t.grp.data(), n, cudaMemcpyHostToDevice, stream) != cudaSuccess)
    return LCA_ERR_CUDA;
  tab->tok_off = d; tab->cache_off = d + (B + 1); tab->grp_off = d + 2 * (B + 1); tab->B = B;
  return LCA_OK;
}

static int run_attention(const AttnProblem& a) {
  const int impl = g_attn_impl.load();
  if (impl != 1 && attn_tc_supported(a)) {
    if (a.ws_bytes < attn_tc_workspace_bytes(a)) return LCA_ERR_WORKSPACE_TOO_SMALL;
    if (attn_tc_workspace_bytes(a) > 0 && (!a.ws || !aligned16(a.ws))) return LCA_ERR_INVALID_ARG;
    return attn_tc_launch(a);
  }
  if (impl == 2) return LCA_ERR_UNSUPPORTED_SHAPE;
  return attn_simt_launch(a);
}
}  // namespace lca

using namespace lca;

extern "C" {

int lca_version(void) { return 100; }

const char* lca_status_string(int s) {
  switch (s) {
    case LCA_OK: return "ok";
    case LCA_ERR_INVALID_ARG: return "invalid argument";
    case LCA_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
    case LCA_ERR_MISALIGNED: return "pointer not 16-byte aligned";
    case LCA_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case LCA_ERR_CUDA: return "CUDA error";
    case LCA_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
    case LCA_ERR_STATIC_SCRATCH_EXCEEDED: return "problem needs more scratch than the fixed LCA_STATIC_SCRATCH_BYTES array; use lca_condense with a caller buffer";
    default: return "unknown status";
  }
}

int64_t lca_launch_count(void) { return (int64_t)g_launches.load(); }

int lca_set_attention_impl(int impl) {
  if (impl < 0 || impl > 2) return g_attn_impl.load();
  return g_attn_impl.exchange(impl);
}

int lca_partition(const lca_params* p, int32_t* m, int32_t* k) {
  int st = check_params(p, true);
  if (st != LCA_OK) return st;
  if (!m || !k) return LCA_ERR_INVALID_ARG;
  int64_t mm, kk;
  partition(p->seq_len, p->window, p->group_size, &mm, &kk);
  *m = (int32_t)mm; *k = (int32_t)kk;
  return LCA_OK;
}

size_t lca_workspace_bytes(const lca_params* p, int32_t which) {
  if (check_params(p, which != LCA_WS_DECODE && which != LCA_WS_UPDATE) != LCA_OK) return 0;
  if (which == LCA_WS_CONDENSE) return condense_workspace_bytes(p);
  if (which == LCA_WS_CONDENSE_VARLEN) return seq_table_bytes(p->batch) + condense_workspace_bytes(p);
  if (which == LCA_WS_PREFILL_VARLEN) return attn_tc2_ragged_workspace_bytes(p->batch, p->seq_len, p->n_q_heads);
  if (which == LCA_WS_UPDATE) return update_workspace_bytes(p);
  if (which == LCA_WS_PREFILL || which == LCA_WS_DECODE) {
    AttnProblem a = {};
    a.variant = p->variant; a.batch = p->batch; a.q_len = which == LCA_WS_DECODE ? 1 : p->seq_len;
    a.n_q_heads = p->n_q_heads; a.n_kv_heads = p->n_kv_heads; a.d_sem = p->d_sem; a.d_pos = p->d_pos;
    a.decode = which == LCA_WS_DECODE; a.seq_len = p->seq_len; a.group_size = p->group_size; a.window = p->window;
    return attn_tc_supported(a) ? attn_tc_workspace_bytes(a) : 0;
  }
  return 0;
}

int lca_condense(const lca_params* p, const void* q_tail_sem, const void* q_tail_pos,
                 int64_t q_tail_batch_stride, const float* qbar_opt, const void* kv_sem,
                 const void* kv_pos, void* cache_sem, void* cache_pos, int32_t* anchor_idx,
                 double* scores_opt, void* ws, size_t ws_bytes, void* stream) {
  int st = check_params(p, true);
  if (st != LCA_OK) return st;
  int64_t m, k;
  partition(p->seq_len, p->window, p->group_size, &m, &k);
  if (!kv_sem || !kv_pos || !cache_sem || !cache_pos) return LCA_ERR_INVALID_ARG;
  if (m > 0) {
    if (!anchor_idx) return LCA_ERR_INVALID_ARG;
    if (!qbar_opt) {
      if (!q_tail_pos || (p->variant == LCA_VARIANT_MLA && !q_tail_sem)) return LCA_ERR_INVALID_ARG;
      int n = p->n_summary_q > 0 ? p->n_summary_q : p->group_size;
      if (n > p->seq_len) n = p->seq_len;
      if (q_tail_batch_stride < n) return LCA_ERR_INVALID_ARG;
      if (!aligned16(q_tail_pos) || (q_tail_sem && !aligned16(q_tail_sem))) return LCA_ERR_MISALIGNED;
    }
    if (!ws || !aligned16(ws)) return LCA_ERR_INVALID_ARG;
    if (ws_bytes < condense_workspace_bytes(p)) return LCA_ERR_WORKSPACE_TOO_SMALL;
    if (condense_smem_bytes(p) > 227u * 1024u) return LCA_ERR_UNSUPPORTED_SHAPE;
  }
  if (!aligned16(kv_sem) || !aligned16(kv_pos) || !aligned16(cache_sem) || !aligned16(cache_pos))
    return LCA_ERR_MISALIGNED;
  CondenseLaunch c = {p, q_tail_sem, q_tail_pos, q_tail_batch_stride, qbar_opt, kv_sem, kv_pos,
                      cache_sem, cache_pos, anchor_idx, scores_opt, ws, ws_bytes, (cudaStream_t)stream};
  return condense_launch(c);
}

int lca_varlen_layout(const lca_params* p, const int32_t* seq_lens, int64_t* token_offsets,
                      int64_t* cache_row_offsets, int64_t* group_offsets) {
  int st = check_params(p, false);
  if (st != LCA_OK) return st;
  if (p->group_size <= 0 || p->window < 0 || !seq_lens) return LCA_ERR_INVALID_ARG;
  HostSeqTable t;
  st = build_seq_table(p, seq_lens, &t);
  if (st != LCA_OK) return st;
  for (int b = 0; b <= p->batch; ++b) {
    if (token_offsets) token_offsets[b] = t.tok[b];
    if (cache_row_offsets) cache_row_offsets[b] = t.cache[b];
    if (group_offsets) group_offsets[b] = t.grp[b];
  }
  return LCA_OK;
}

int lca_condense_varlen(const lca_params* p, const int32_t* seq_lens, const void* q_sem, const void* q_pos,
                        const float* qbar_opt, const void* kv_sem, const void* kv_pos, void* cache_sem,
                        void* cache_pos, int32_t* anchor_idx, void* ws, size_t ws_bytes, void* stream) {
  int st = check_params(p, false);
  if (st != LCA_OK) return st;
  if (p->group_size <= 0 || p->window < 0 || p->n_summary_q < 0 || !seq_lens) return LCA_ERR_INVALID_ARG;
  if (!kv_sem || !kv_pos || !cache_sem || !cache_pos) return LCA_ERR_INVALID_ARG;
  HostSeqTable t;
  st = build_seq_table(p, seq_lens, &t);
  if (st != LCA_OK) return st;
  lca_params q = *p;
  q.seq_len = t.longest;                                   // sizes the summary-query scratch
  if (t.grp[p->batch] > 0) {
    if (!anchor_idx) return LCA_ERR_INVALID_ARG;
    if (!qbar_opt) {
      if (!q_pos || (p->variant == LCA_VARIANT_MLA && !q_sem)) return LCA_ERR_INVALID_ARG;
      if (!aligned16(q_pos) || (q_sem && !aligned16(q_sem))) return LCA_ERR_MISALIGNED;
    }
    if (condense_smem_bytes(&q) > 227u * 1024u) return LCA_ERR_UNSUPPORTED_SHAPE;
  }
  if (!ws || !aligned16(ws)) return LCA_ERR_INVALID_ARG;
  if (ws_bytes < seq_table_bytes(p->batch) + condense_workspace_bytes(&q)) return LCA_ERR_WORKSPACE_TOO_SMALL;
  if (!aligned16(kv_sem) || !aligned16(kv_pos) || !aligned16(cache_sem) || !aligned16(cache_pos))
    return LCA_ERR_MISALIGNED;
  CondenseLaunch c = {&q, q_sem, q_pos, 0, qbar_opt, kv_sem, kv_pos, cache_sem, cache_pos, anchor_idx, nullptr,
                      static_cast<char*>(ws) + seq_table_bytes(p->batch), ws_bytes - seq_table_bytes(p->batch),
                      (cudaStream_t)stream};
  c.h_tok_off = t.tok.data(); c.h_cache_off = t.cache.data(); c.h_grp_off = t.grp.data();
  st = upload_seq_table(t, p->batch, ws, (cudaStream_t)stream, &c.tab);
  if (st != LCA_OK) return st;
  return condense_launch(c);
}

int lca_prefill_attention_varlen(const lca_params* p, const int32_t* seq_lens, const void* q_sem,
                                 const void* q_pos, const void* kv_sem, const void* kv_pos,
                                 const void* cache_sem, const void* cache_pos, void* out, float* lse_opt,
                                 void* ws, size_t ws_bytes, void* stream) {
  int st = check_params(p, false);
  if (st != LCA_OK) return st;
  if (p->group_size <= 0 || p->window < 0 || !seq_lens) return LCA_ERR_INVALID_ARG;
  if (!q_pos || !kv_sem || !kv_pos || !out) return LCA_ERR_INVALID_ARG;
  if (p->variant == LCA_VARIANT_MLA && !q_sem) return LCA_ERR_INVALID_ARG;
  HostSeqTable t;
  st = build_seq_table(p, seq_lens, &t);
  if (st != LCA_OK) return st;
  if (t.grp[p->batch] > 0 && (!cache_sem || !cache_pos)) return LCA_ERR_INVALID_ARG;
  if (!aligned16(q_pos) || !aligned16(kv_sem) || !aligned16(kv_pos) || !aligned16(out) ||
      (q_sem && !aligned16(q_sem)) || (cache_sem && !aligned16(cache_sem)) || (cache_pos && !aligned16(cache_pos)))
    return LCA_ERR_MISALIGNED;
  if (!simt_shape_ok(p)) return LCA_ERR_UNSUPPORTED_SHAPE;
  if (!ws || !aligned16(ws)) return LCA_ERR_INVALID_ARG;
  if (ws_bytes < attn_tc2_ragged_workspace_bytes(p->batch, t.longest, p->n_q_heads)) return LCA_ERR_WORKSPACE_TOO_SMALL;
  AttnProblem a = {};
  a.variant = p->variant; a.batch = p->batch; a.q_len = t.longest; a.n_q_heads = p->n_q_heads;
  a.n_kv_heads = p->n_kv_heads; a.d_sem = p->d_sem; a.d_pos = p->d_pos; a.decode = 0;
  a.seq_len = t.longest; a.group_size = p->group_size; a.window = p->window;
  a.cache_rows = nullptr; a.cache_row_capacity = 0; a.n_rep_bias = 0;
  a.softmax_scale = p->softmax_scale; a.rep_logit_bias = p->rep_logit_bias;
  a.q_sem = q_sem; a.q_pos = q_pos; a.kv_sem = kv_sem; a.kv_pos = kv_pos;
  a.cache_sem = cache_sem; a.cache_pos = cache_pos; a.out = out; a.lse = lse_opt;
  a.ws = ws; a.ws_bytes = ws_bytes; a.stream = (cudaStream_t)stream;
  a.h_tok_off = t.tok.data(); a.h_cache_off = t.cache.data();
  st = upload_seq_table(t, p->batch, ws, (cudaStream_t)stream, &a.tab);
  if (st != LCA_OK) return st;
  return run_attention(a);
}

int lca_condense_static_scratch(const lca_params* p, const void* q_tail_sem, const void* q_tail_pos,
                                int64_t q_tail_batch_stride, const float* qbar_opt,
                                const void* kv_sem, const void* kv_pos, void* cache_sem,
                                void* cache_pos, int32_t* anchor_idx, double* scores_opt,
                                void* stream) {
  int st = check_params(p, true);
  if (st != LCA_OK) return st;
  if (condense_workspace_bytes(p) > (size_t)LCA_STATIC_SCRATCH_BYTES) return LCA_ERR_STATIC_SCRATCH_EXCEEDED;
  void* scratch = nullptr;
  st = condense_static_scratch_address(&scratch);     // first call on a device: one address look-up
  if (st != LCA_OK) return st;
  return lca_condense(p, q_tail_sem, q_tail_pos, q_tail_batch_stride, qbar_opt, kv_sem, kv_pos,
                      cache_sem, cache_pos, anchor_idx, scores_opt, scratch, LCA_STATIC_SCRATCH_BYTES, stream);
}

int lca_prefill_attention(const lca_params* p, const void* q_sem, const void* q_pos,
                          const void* kv_sem, const void* kv_pos, const void* cache_sem,
                          const void* cache_pos, void* out, float* lse_opt, void* ws,
                          size_t ws_bytes, void* stream) {
  int st = check_params(p, true);
  if (st != LCA_OK) return st;
  int64_t m, k;
  partition(p->seq_len, p->window, p->group_size, &m, &k);
  if (!q_pos || !kv_sem || !kv_pos || !out) return LCA_ERR_INVALID_ARG;
  if (p->variant == LCA_VARIANT_MLA && !q_sem) return LCA_ERR_INVALID_ARG;
  if (m > 0 && (!cache_sem || !cache_pos)) return LCA_ERR_INVALID_ARG;
  if (!aligned16(q_pos) || !aligned16(kv_sem) || !aligned16(kv_pos) || !aligned16(out) ||
      (q_sem && !aligned16(q_sem)) || (cache_sem && !aligned16(cache_sem)) ||
      (cache_pos && !aligned16(cache_pos)))
    return LCA_ERR_MISALIGNED;
  if (!simt_shape_ok(p)) return LCA_ERR_UNSUPPORTED_SHAPE;
  AttnProblem a = {};
  a.variant = p->variant; a.batch = p->batch; a.q_len = p->seq_len; a.n_q_heads = p->n_q_heads;
  a.n_kv_heads = p->n_kv_heads; a.d_sem = p->d_sem; a.d_pos = p->d_pos; a.decode = 0;
  a.seq_len = p->seq_len; a.group_size = p->group_size; a.window = p->window;
  a.cache_rows = nullptr; a.cache_row_capacity = (int)(m + k); a.n_rep_bias = 0;
  a.softmax_scale = p->softmax_scale; a.rep_logit_bias = p->rep_logit_bias;
  a.q_sem = q_sem; a.q_pos = q_pos; a.kv_sem = kv_sem; a.kv_pos = kv_pos;
  a.cache_sem = cache_sem; a.cache_pos = cache_pos; a.out = out; a.lse = lse_opt;
  a.ws = ws; a.ws_bytes = ws_bytes; a.stream = (cudaStream_t)stream;
  return run_attention(a);
}

int lca_decode_attention(const lca_params* p, const void* q_sem, const void* q_pos,
                         const void* cache_sem, const void* cache_pos, const int32_t* cache_rows,
                         int32_t cache_row_capacity, int32_t n_rep, void* out, float* lse_opt,
                         void* ws, size_t ws_bytes, void* stream) {
  int st = check_params(p, false);
  if (st != LCA_OK) return st;
  if (!q_pos || !cache_sem || !cache_pos || !cache_rows || !out) return LCA_ERR_INVALID_ARG;
  if (p->variant == LCA_VARIANT_MLA && !q_sem) return LCA_ERR_INVALID_ARG;
  if (cache_row_capacity <= 0 || n_rep < 0) return LCA_ERR_INVALID_ARG;
  if (!aligned16(q_pos) || !aligned16(cache_sem) || !aligned16(cache_pos) || !aligned16(out) ||
      (q_sem && !aligned16(q_sem)))
    return LCA_ERR_MISALIGNED;
  if (!simt_shape_ok(p)) return LCA_ERR_UNSUPPORTED_SHAPE;
  AttnProblem a = {};
  a.variant = p->variant; a.batch = p->batch; a.q_len = 1; a.n_q_heads = p->n_q_heads;
  a.n_kv_heads = p->n_kv_heads; a.d_sem = p->d_sem; a.d_pos = p->d_pos; a.decode = 1;
  a.seq_len = 0; a.group_size = 1; a.window = 0;
  a.cache_rows = cache_rows; a.cache_row_capacity = cache_row_capacity; a.n_rep_bias = n_rep;
  a.softmax_scale = p->softmax_scale; a.rep_logit_bias = p->rep_logit_bias;
  a.q_sem = q_sem; a.q_pos = q_pos; a.kv_sem = nullptr; a.kv_pos = nullptr;
  a.cache_sem = cache_sem; a.cache_pos = cache_pos; a.out = out; a.lse = lse_opt;
  a.ws = ws; a.ws_bytes = ws_bytes; a.stream = (cudaStream_t)stream;
  return run_attention(a);
}

int lca_decode_update(const lca_params* p, const void* q_tail_sem, const void* q_tail_pos,
                      int64_t q_tail_batch_stride, const float* qbar_opt, void* cache_sem,
                      void* cache_pos, int32_t cache_row_capacity, int32_t* n_rep,
                      int32_t* cache_rows, int32_t* anchor_out, void* ws, size_t ws_bytes,
                      void* stream) {
  int st = check_params(p, false);
  if (st != LCA_OK) return st;
  if (p->group_size <= 0 || p->window < 0 || p->n_summary_q < 0) return LCA_ERR_INVALID_ARG;
  if (!cache_sem || !cache_pos || !n_rep || !cache_rows || !anchor_out || cache_row_capacity <= 0)
    return LCA_ERR_INVALID_ARG;
  if (!qbar_opt) {
    if (!q_tail_pos || (p->variant == LCA_VARIANT_MLA && !q_tail_sem)) return LCA_ERR_INVALID_ARG;
    const int n = p->n_summary_q > 0 ? p->n_summary_q : p->group_size;
    if (q_tail_batch_stride < n) return LCA_ERR_INVALID_ARG;
    if (!aligned16(q_tail_pos) || (q_tail_sem && !aligned16(q_tail_sem))) return LCA_ERR_MISALIGNED;
  }
  if (!aligned16(cache_sem) || !aligned16(cache_pos)) return LCA_ERR_MISALIGNED;
  if (!ws || !aligned16(ws)) return LCA_ERR_INVALID_ARG;
  if (ws_bytes < update_workspace_bytes(p)) return LCA_ERR_WORKSPACE_TOO_SMALL;
  if (update_smem_bytes(p) > 227u * 1024u) return LCA_ERR_UNSUPPORTED_SHAPE;
  return update_launch(p, q_tail_sem, q_tail_pos, q_tail_batch_stride, qbar_opt, cache_sem, cache_pos,
                       cache_row_capacity, n_rep, cache_rows, nullptr, anchor_out, ws, (cudaStream_t)stream);
}

// The ring layout needs whole groups to leave the ring: window a multiple of group_size.
static int check_ring(const lca_params* p, int32_t ring_row_capacity) {
  if (p->group_size <= 0 || p->window < 0 || p->window % p->group_size != 0) return LCA_ERR_INVALID_ARG;
  if ((int64_t)p->window + p->group_size > (int64_t)ring_row_capacity) return LCA_ERR_INVALID_ARG;
  return LCA_OK;
}

int lca_ring_from_packed(const lca_params* p, const void* packed_sem, const void* packed_pos,
                         const int32_t* packed_rows, const int32_t* n_rep, int32_t packed_row_capacity,
                         void* ring_sem, void* ring_pos, int32_t ring_row_capacity, int32_t* n_tok_out,
                         void* stream) {
  int st = check_params(p, false);
  if (st != LCA_OK) return st;
  if (!packed_sem || !packed_pos || !packed_rows || !n_rep || !ring_sem || !ring_pos || !n_tok_out ||
      packed_row_capacity <= 0)
    return LCA_ERR_INVALID_ARG;
  st = check_ring(p, ring_row_capacity);
  if (st != LCA_OK) return st;
  if (!aligned16(packed_sem) || !aligned16(packed_pos) || !aligned16(ring_sem) || !aligned16(ring_pos))
    return LCA_ERR_MISALIGNED;
  if (((size_t)p->n_kv_heads * p->d_sem * 2) % 16 || ((size_t)p->n_kv_heads * p->d_pos * 2) % 16) return LCA_ERR_UNSUPPORTED_SHAPE;
  return ring_from_packed_launch(p, packed_sem, packed_pos, packed_rows, n_rep, packed_row_capacity, ring_sem, ring_pos,
                                 ring_row_capacity, n_tok_out, (cudaStream_t)stream);
}

int lca_decode_attention_ring(const lca_params* p, const void* q_sem, const void* q_pos,
                              const void* ring_sem, const void* ring_pos, const int32_t* n_rep,
                              const int32_t* n_tok, int32_t ring_row_capacity, void* out, float* lse_opt,
                              void* ws, size_t ws_bytes, void* stream) {
  int st = check_params(p, false);
  if (st != LCA_OK) return st;
  if (!q_pos || !ring_sem || !ring_pos || !n_rep || !n_tok || !out) return LCA_ERR_INVALID_ARG;
  if (p->variant == LCA_VARIANT_MLA && !q_sem) return LCA_ERR_INVALID_ARG;
  st = check_ring(p, ring_row_capacity);
  if (st != LCA_OK) return st;
  if (!aligned16(q_pos) || !aligned16(ring_sem) || !aligned16(ring_pos) || !aligned16(out) || (q_sem && !aligned16(q_sem)))
    return LCA_ERR_MISALIGNED;
  if (!simt_shape_ok(p)) return LCA_ERR_UNSUPPORTED_SHAPE;
  AttnProblem a = {};
  a.variant = p->variant; a.batch = p->batch; a.q_len = 1; a.n_q_heads = p->n_q_heads;
  a.n_kv_heads = p->n_kv_heads; a.d_sem = p->d_sem; a.d_pos = p->d_pos; a.decode = 1;
  a.seq_len = 0; a.group_size = p->group_size; a.window = p->window;
  a.cache_rows = nullptr; a.cache_row_capacity = ring_row_capacity; a.n_rep_bias = 0;
  a.ring_n_rep = n_rep; a.ring_n_tok = n_tok;
  a.softmax_scale = p->softmax_scale; a.rep_logit_bias = p->rep_logit_bias;
  a.q_sem = q_sem; a.q_pos = q_pos; a.kv_sem = nullptr; a.kv_pos = nullptr;
  a.cache_sem = ring_sem; a.cache_pos = ring_pos; a.out = out; a.lse = lse_opt;
  a.ws = ws; a.ws_bytes = ws_bytes; a.stream = (cudaStream_t)stream;
  return run_attention(a);
}

int lca_decode_update_ring(const lca_params* p, const void* q_tail_sem, const void* q_tail_pos,
                           int64_t q_tail_batch_stride, const float* qbar_opt, void* ring_sem,
                           void* ring_pos, int32_t ring_row_capacity, int32_t* n_rep, const int32_t* n_tok,
                           int32_t* anchor_out, void* ws, size_t ws_bytes, void* stream) {
  int st = check_params(p, false);
  if (st != LCA_OK) return st;
  if (p->n_summary_q < 0) return LCA_ERR_INVALID_ARG;
  if (!ring_sem || !ring_pos || !n_rep || !n_tok || !anchor_out) return LCA_ERR_INVALID_ARG;
  st = check_ring(p, ring_row_capacity);
  if (st != LCA_OK) return st;
  if (!qbar_opt) {
    if (!q_tail_pos || (p->variant == LCA_VARIANT_MLA && !q_tail_sem)) return LCA_ERR_INVALID_ARG;
    const int n = p->n_summary_q > 0 ? p->n_summary_q : p->group_size;
    if (q_tail_batch_stride < n) return LCA_ERR_INVALID_ARG;
    if (!aligned16(q_tail_pos) || (q_tail_sem && !aligned16(q_tail_sem))) return LCA_ERR_MISALIGNED;
  }
  if (!aligned16(ring_sem) || !aligned16(ring_pos)) return LCA_ERR_MISALIGNED;
  if (!ws || !aligned16(ws)) return LCA_ERR_INVALID_ARG;
  if (ws_bytes < update_workspace_bytes(p)) return LCA_ERR_WORKSPACE_TOO_SMALL;
  if (update_smem_bytes(p) > 227u * 1024u) return LCA_ERR_UNSUPPORTED_SHAPE;
  return update_launch(p, q_tail_sem, q_tail_pos, q_tail_batch_stride, qbar_opt, ring_sem, ring_pos,
                       ring_row_capacity, n_rep, nullptr, n_tok, anchor_out, ws, (cudaStream_t)stream);
}

int lca_decode_step_update_ring(const lca_params* p, const void* q_sem, const void* q_pos, double* qsum,
                                int32_t* qcount, void* ring_sem, void* ring_pos, int32_t ring_row_capacity,
                                int32_t* n_rep, const int32_t* n_tok, int32_t* anchor_out, void* ws,
                                size_t ws_bytes, void* stream) {
  int st = check_params(p, false);
  if (st != LCA_OK) return st;
  if (!q_pos || !qsum || !qcount || !ring_sem || !ring_pos || !n_rep || !n_tok || !anchor_out) return LCA_ERR_INVALID_ARG;
  if (p->variant == LCA_VARIANT_MLA && !q_sem) return LCA_ERR_INVALID_ARG;
  if (p->n_summary_q != 0 && p->n_summary_q != p->group_size) return LCA_ERR_INVALID_ARG;   // the sum runs from update to update
  st = check_ring(p, ring_row_capacity);
  if (st != LCA_OK) return st;
  if (!aligned16(q_pos) || (q_sem && !aligned16(q_sem)) || !aligned16(ring_sem) || !aligned16(ring_pos) || !aligned16(qsum))
    return LCA_ERR_MISALIGNED;
  if (!ws || !aligned16(ws)) return LCA_ERR_INVALID_ARG;
  if (ws_bytes < update_workspace_bytes(p)) return LCA_ERR_WORKSPACE_TOO_SMALL;
  if (update_smem_bytes(p) > 227u * 1024u) return LCA_ERR_UNSUPPORTED_SHAPE;
  return update_step_launch(p, q_sem, q_pos, qsum, qcount, ring_sem, ring_pos, ring_row_capacity, n_rep, n_tok,
                            anchor_out, ws, (cudaStream_t)stream);
}

int lca_latent_to_value(const void* attn_latent, const void* w_uv, void* out_v, int64_t n_tokens,
                        int32_t n_heads, int32_t d_latent, int32_t d_v, void* stream) {
  if (n_tokens < 0 || n_heads <= 0 || d_latent <= 0 || d_v <= 0) return LCA_ERR_INVALID_ARG;
  if (n_tokens == 0) return LCA_OK;
  if (!attn_latent || !w_uv || !out_v) return LCA_ERR_INVALID_ARG;
  if (!aligned16(attn_latent) || !aligned16(w_uv) || !aligned16(out_v)) return LCA_ERR_MISALIGNED;
  return latent_to_value_launch(attn_latent, w_uv, out_v, n_tokens, n_heads, d_latent, d_v, (cudaStream_t)stream);
}

int lca_selftest_bounded_wait(int64_t limit_cycles, void* stream) {
  if (limit_cycles < 1 || limit_cycles > 100000000ll) return LCA_ERR_INVALID_ARG;     // at most ~50 ms
  return bounded_wait_selftest_launch((long long)limit_cycles, (cudaStream_t)stream);
}

int lca_last_device_status(void* stream) {
  const int st = attn_tc_device_status((cudaStream_t)stream);      // synchronises the stream
  const int cst = condense_take_status(), ust = latent_to_value_take_status();
  if (cst < 0 || ust < 0) return LCA_ERR_CUDA;
  if (cst > 0 || ust > 0) return LCA_ERR_DEVICE_TIMEOUT;
  return st;
}

}  // extern "C"
