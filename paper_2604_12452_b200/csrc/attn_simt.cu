// Scalar (CUDA-core) attention over the condensed context: Eq. 10 at every prefix length, and the
// decode step of Sec. 4.3.  One warp per query row (b, t, h); lanes split the feature dimension,
// keys are visited one by one with an online softmax in fp32.  This kernel exists for head
// shapes the tensor-core kernels do not cover and as an independent device-side cross-check;
// it makes no attempt to reach the tensor-core roofline.
#include "lca_common.cuh"

namespace lca {

struct SimtArgs {
  const bf16* q_sem; const bf16* q_pos;
  const bf16* kv_sem; const bf16* kv_pos;
  const bf16* cache_sem; const bf16* cache_pos;
  bf16* out; float* lse;
  int B, q_len, Hq, Hkv, decode, L, g, w, cap;
  float scale, bias;
  SeqTab tab;              // ragged prefill batch (tok_off != nullptr): q_len, L and cap are unused
  DecodeLayout dl;         // decode: which cache rows take part
  long long n_rows;        // query rows of the launch (tokens x heads)
};

template <int D_SEM, int D_POS, bool SEM_IN_LOGIT>
__global__ void __launch_bounds__(128)
attn_simt_kernel(SimtArgs a) {
  constexpr int PS = D_SEM / 64;   // bf16 pairs per lane, sem part
  constexpr int PP = D_POS / 64;   // pos part
  const int lane = threadIdx.x & 31;
  const long long row = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= a.n_rows) return;
  const int h = (int)(row % a.Hq);
  int t = (int)((row / a.Hq) % a.q_len);
  int b = (int)(row / ((long long)a.Hq * a.q_len));
  size_t kbase = (size_t)b * a.L, cbase = (size_t)b * a.cap;       // first token row / cache row of the sequence
  if (a.tab.tok_off) {
    const long long tok = row / a.Hq;
    b = seq_of(a.tab.tok_off, a.tab.B, tok);
    t = (int)(tok - a.tab.tok_off[b]);
    kbase = (size_t)a.tab.tok_off[b]; cbase = (size_t)a.tab.cache_off[b];
  }
  const int hk = h / (a.Hq / a.Hkv);

  float qs[2 * PS > 0 ? 2 * PS : 1], qp[2 * PP > 0 ? 2 * PP : 1];
  if (SEM_IN_LOGIT) {
    const bf162* src = reinterpret_cast<const bf162*>(a.q_sem + (size_t)row * D_SEM);
#pragma unroll
    for (int i = 0; i < PS; ++i) {
      float2 f = __bfloat1622float2(src[lane + 32 * i]);
      qs[2 * i] = f.x * a.scale; qs[2 * i + 1] = f.y * a.scale;
    }
  }
  {
    const bf162* src = reinterpret_cast<const bf162*>(a.q_pos + (size_t)row * D_POS);
#pragma unroll
    for (int i = 0; i < PP; ++i) {
      float2 f = __bfloat1622float2(src[lane + 32 * i]);
      qp[2 * i] = f.x * a.scale; qp[2 * i + 1] = f.y * a.scale;
    }
  }

  int n_a, b_first, b_last;
  DecodeSpan sp;
  if (a.decode) {
    sp = decode_span(a.dl, b);
    n_a = sp.rows_end;
    b_first = 0; b_last = -1;
  } else {
    n_a = reps_visible(t, a.w, a.g);
    b_first = n_a * a.g; b_last = t;
    sp.rows_end = n_a; sp.inv_lo = sp.inv_hi = 0; sp.bias_lo = 0; sp.bias_hi = n_a;
  }

  float acc[2 * PS];
#pragma unroll
  for (int i = 0; i < 2 * PS; ++i) acc[i] = 0.f;
  float mx = -INFINITY, l = 0.f;

  const int n_total = n_a + (b_last - b_first + 1);
  int n_seen = 0;
  for (int x = 0; x < n_total; ++x) {
    const bf16 *ks, *kp;
    float add = 0.f;
    if (x < n_a) {
      if (x >= sp.inv_lo && x < sp.inv_hi) continue;       // ring layout: a condensed token that is still in its row
      size_t r = (cbase + x) * a.Hkv + hk;
      ks = a.cache_sem + r * D_SEM; kp = a.cache_pos + r * D_POS;
      if (x >= sp.bias_lo && x < sp.bias_hi) add = a.bias;
    } else {
      size_t r = (kbase + (b_first + x - n_a)) * a.Hkv + hk;
      ks = a.kv_sem + r * D_SEM; kp = a.kv_pos + r * D_POS;
    }
    ++n_seen;
    float2 v[PS];
#pragma unroll
    for (int i = 0; i < PS; ++i) v[i] = __bfloat1622float2(reinterpret_cast<const bf162*>(ks)[lane + 32 * i]);
    float s = 0.f;
    if (SEM_IN_LOGIT) {
#pragma unroll
      for (int i = 0; i < PS; ++i) s += qs[2 * i] * v[i].x + qs[2 * i + 1] * v[i].y;
    }
#pragma unroll
    for (int i = 0; i < PP; ++i) {
      float2 f = __bfloat1622float2(reinterpret_cast<const bf162*>(kp)[lane + 32 * i]);
      s += qp[2 * i] * f.x + qp[2 * i + 1] * f.y;
    }
    s = warp_sum(s) + add;
    const float mn = fmaxf(mx, s);
    const float corr = __expf(mx - mn);
    const float pw = __expf(s - mn);
    l = l * corr + pw;
#pragma unroll
    for (int i = 0; i < PS; ++i) {
      acc[2 * i] = acc[2 * i] * corr + pw * v[i].x;
      acc[2 * i + 1] = acc[2 * i + 1] * corr + pw * v[i].y;
    }
    mx = mn;
  }
  const float inv = n_seen > 0 ? 1.f / l : 0.f;
  bf162* dst = reinterpret_cast<bf162*>(a.out + (size_t)row * D_SEM);
#pragma unroll
  for (int i = 0; i < PS; ++i)
    dst[lane + 32 * i] = __floats2bfloat162_rn(acc[2 * i] * inv, acc[2 * i + 1] * inv);
  if (a.lse && lane == 0) a.lse[row] = n_seen > 0 ? mx + logf(l) : -INFINITY;
}

int attn_simt_launch(const AttnProblem& p) {
  SimtArgs a;
  a.q_sem = (const bf16*)p.q_sem; a.q_pos = (const bf16*)p.q_pos;
  a.kv_sem = (const bf16*)p.kv_sem; a.kv_pos = (const bf16*)p.kv_pos;
  a.cache_sem = (const bf16*)p.cache_sem; a.cache_pos = (const bf16*)p.cache_pos;
  a.out = (bf16*)p.out; a.lse = p.lse;
  a.B = p.batch; a.q_len = p.q_len; a.Hq = p.n_q_heads; a.Hkv = p.n_kv_heads; a.decode = p.decode;
  a.L = p.seq_len; a.g = p.group_size; a.w = p.window; a.cap = p.cache_row_capacity;
  a.scale = p.softmax_scale; a.bias = p.rep_logit_bias;
  a.dl = DecodeLayout{p.cache_rows, p.ring_n_rep, p.ring_n_tok, p.cache_row_capacity, p.n_rep_bias, p.window + p.group_size, p.group_size};
  const long long rows = p.h_tok_off ? (long long)p.h_tok_off[p.batch] * p.n_q_heads : (long long)p.batch * p.q_len * p.n_q_heads;
  a.tab = p.h_tok_off ? p.tab : SeqTab{};
  a.n_rows = rows;
  if (rows == 0) return LCA_OK;
  const unsigned blocks = (unsigned)((rows + 3) / 4);
  if (p.variant == LCA_VARIANT_MLA && p.d_sem == 512 && p.d_pos == 64)
    attn_simt_kernel<512, 64, true><<<blocks, 128, 0, p.stream>>>(a);
  else if (p.variant == LCA_VARIANT_MLA && p.d_sem == 128 && p.d_pos == 64)
    attn_simt_kernel<128, 64, true><<<blocks, 128, 0, p.stream>>>(a);
  else if (p.variant == LCA_VARIANT_GQA && p.d_sem == 128 && p.d_pos == 128)
    attn_simt_kernel<128, 128, false><<<blocks, 128, 0, p.stream>>>(a);
  else if (p.variant == LCA_VARIANT_GQA && p.d_sem == 64 && p.d_pos == 64)
    attn_simt_kernel<64, 64, false><<<blocks, 128, 0, p.stream>>>(a);
  else
    return LCA_ERR_UNSUPPORTED_SHAPE;
  note_launch();
  return cudaGetLastError() == cudaSuccess ? LCA_OK : LCA_ERR_CUDA;
}

}  // namespace lca
