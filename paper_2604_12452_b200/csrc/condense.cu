// Condensation kernels: summary query (Alg. 1 line 1), group scores + softmax (Sec. 4.2, Eq. 6),
// weighted pooling (Eq. 7), anchor selection (Eq. 8) and the local-window copy (Eq. 9).
//
// The work is HBM-bound (about 2 flop per byte): every history token is read from global memory
// exactly once into shared memory (one CTA per group), scored against the summary query,
// soft-maxed within the group, pooled, and the representative plus the anchor's positional row
// are written straight into the condensed cache.  All arithmetic is fp64: it costs a few percent
// of the fp64 pipe at HBM speed and makes the arg-max and the bf16 rounding of c_rep follow the
// exact scores rather than an fp32 accumulation order.
#include <mutex>

#include "lca_common.cuh"

namespace lca {

static const int QBAR_ROWS_PER_CHUNK = 64;
static const int QBAR_THREADS = 128;
static const int CONDENSE_THREADS = 256;

// ---------------------------------------------------------------------------- summary query
// Partial sums of the query tail.  Rows of one KV head = (position, query head in its group).
// grid (nchunks, Hkv, B); each thread owns column pairs tid, tid+T, ...
__global__ void qbar_partial_kernel(const bf16* __restrict__ q_sem, const bf16* __restrict__ q_pos,
                                    int64_t batch_stride_rows, int n_pos, int Hq, int Hkv, int d_sem,
                                    int d_pos, int sem_in_logit, double* __restrict__ partial) {
  const int chunk = blockIdx.x, hk = blockIdx.y, b = blockIdx.z;
  const int rep = Hq / Hkv;
  const int n_rows = n_pos * rep;
  const int r0 = chunk * QBAR_ROWS_PER_CHUNK;
  const int r1 = min(n_rows, r0 + QBAR_ROWS_PER_CHUNK);
  const int dk = (sem_in_logit ? d_sem : 0) + d_pos;
  const int sem_pairs = sem_in_logit ? d_sem / 2 : 0;
  double* dst = partial + (((size_t)b * Hkv + hk) * gridDim.x + chunk) * dk;
  for (int pr = threadIdx.x; pr < dk / 2; pr += blockDim.x) {
    double a0 = 0.0, a1 = 0.0;
    for (int r = r0; r < r1; ++r) {
      const int pos = r / rep, head = hk * rep + r % rep;
      const size_t row = ((size_t)b * batch_stride_rows + pos) * Hq + head;
      const bf16* src = (pr < sem_pairs) ? q_sem + row * d_sem + 2 * pr
                                         : q_pos + row * d_pos + 2 * (pr - sem_pairs);
      const bf162 v = *reinterpret_cast<const bf162*>(src);
      a0 += (double)__low2float(v);
      a1 += (double)__high2float(v);
    }
    dst[2 * pr] = a0;
    dst[2 * pr + 1] = a1;
  }
}

// Sum the chunk partials in chunk order and divide by the number of averaged rows.
// grid (Hkv, B)
__global__ void qbar_final_kernel(const double* __restrict__ partial, int nchunks, int dk,
                                  double count, double* __restrict__ qbar) {
  const size_t stream_id = (size_t)blockIdx.y * gridDim.x + blockIdx.x;
  const double* src = partial + stream_id * nchunks * dk;
  for (int c = threadIdx.x; c < dk; c += blockDim.x) {
    double s = 0.0;
    for (int ch = 0; ch < nchunks; ++ch) s += src[(size_t)ch * dk + c];
    qbar[stream_id * dk + c] = s / count;
  }
}

__global__ void qbar_widen_kernel(const float* __restrict__ src, double* __restrict__ dst, int n) {
  int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) dst[i] = (double)src[i];
}

// --------------------------------------------------------------------------------- condense
struct CondenseArgs {
  const bf16* kv_sem; const bf16* kv_pos; const double* qbar;
  bf16* cache_sem; bf16* cache_pos; int32_t* anchor; double* scores;
  int L, Hkv, d_sem, d_pos, g, m, cache_rows, sem_in_logit;
  double scale;
};

__device__ inline void cp_async16(void* smem_dst, const void* gmem_src) {
  unsigned s = (unsigned)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(s), "l"(gmem_src) : "memory");
}
__device__ inline void cp_async_wait_all() {
  asm volatile("cp.async.commit_group;\ncp.async.wait_group 0;\n" ::: "memory");
}

// grid (m, Hkv, B), CONDENSE_THREADS threads, dynamic smem = tile + q_bar + scores + alpha.
__global__ void __launch_bounds__(CONDENSE_THREADS)
condense_kernel(CondenseArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int j = blockIdx.x, hk = blockIdx.y, b = blockIdx.z;
  const int g = a.g, d_sem = a.d_sem, d_pos = a.d_pos;
  const int dk = (a.sem_in_logit ? d_sem : 0) + d_pos;
  bf16* t_sem = reinterpret_cast<bf16*>(smem_raw);                 // [g][d_sem]
  bf16* t_pos = t_sem + (size_t)g * d_sem;                         // [g][d_pos]
  double* s_q = reinterpret_cast<double*>(t_pos + (size_t)g * d_pos);   // [dk]
  double* s_s = s_q + dk;                                          // [g] scores
  double* s_a = s_s + g;                                           // [g] alpha
  __shared__ int s_anchor;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
  const size_t tok0 = (size_t)b * a.L + (size_t)j * g;             // first token of G_j
  const size_t row_stride_sem = (size_t)a.Hkv * d_sem, row_stride_pos = (size_t)a.Hkv * d_pos;

  // 1. the g tokens of the group: global -> shared, 16 B per copy, each byte read once
  {
    const int cps = d_sem / 8, cpp = d_pos / 8;                    // 16-byte chunks per row
    const bf16* gs = a.kv_sem + tok0 * row_stride_sem + (size_t)hk * d_sem;
    const bf16* gp = a.kv_pos + tok0 * row_stride_pos + (size_t)hk * d_pos;
    for (int x = tid; x < g * cps; x += blockDim.x) {
      int i = x / cps, c = x % cps;
      cp_async16(t_sem + (size_t)i * d_sem + c * 8, gs + (size_t)i * row_stride_sem + c * 8);
    }
    for (int x = tid; x < g * cpp; x += blockDim.x) {
      int i = x / cpp, c = x % cpp;
      cp_async16(t_pos + (size_t)i * d_pos + c * 8, gp + (size_t)i * row_stride_pos + c * 8);
    }
    const double* qb = a.qbar + ((size_t)b * a.Hkv + hk) * dk;
    for (int c = tid; c < dk; c += blockDim.x) s_q[c] = qb[c];
    cp_async_wait_all();
  }
  __syncthreads();

  // 2. importance scores s_i = scale * q_bar . k_i   (one warp per token, fp64)
  const int sem_off = a.sem_in_logit ? d_sem : 0;
  for (int i = warp; i < g; i += nwarps) {
    double acc = 0.0;
    if (a.sem_in_logit) {
      const bf162* row = reinterpret_cast<const bf162*>(t_sem + (size_t)i * d_sem);
      for (int pr = lane; pr < d_sem / 2; pr += 32) {
        bf162 v = row[pr];
        acc = fma(s_q[2 * pr], (double)__low2float(v), acc);
        acc = fma(s_q[2 * pr + 1], (double)__high2float(v), acc);
      }
    }
    {
      const bf162* row = reinterpret_cast<const bf162*>(t_pos + (size_t)i * d_pos);
      for (int pr = lane; pr < d_pos / 2; pr += 32) {
        bf162 v = row[pr];
        acc = fma(s_q[sem_off + 2 * pr], (double)__low2float(v), acc);
        acc = fma(s_q[sem_off + 2 * pr + 1], (double)__high2float(v), acc);
      }
    }
    acc = warp_sum(acc);
    if (lane == 0) s_s[i] = acc * a.scale;
  }
  __syncthreads();

  // 3. group softmax (Eq. 6) and arg-max (Eq. 8; lowest index on ties), warp 0
  if (warp == 0) {
    double best = -INFINITY;
    int besti = 0x7fffffff;
    for (int i = lane; i < g; i += 32) {
      double s = s_s[i];
      if (s > best) { best = s; besti = i; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      double ob = __shfl_xor_sync(0xffffffffu, best, o);
      int oi = __shfl_xor_sync(0xffffffffu, besti, o);
      if (ob > best || (ob == best && oi < besti)) { best = ob; besti = oi; }
    }
    double z = 0.0;
    for (int i = lane; i < g; i += 32) {
      double e = exp(s_s[i] - best);
      s_a[i] = e;
      z += e;
    }
    z = warp_sum(z);
    for (int i = lane; i < g; i += 32) s_a[i] = s_a[i] / z;
    if (lane == 0) s_anchor = besti;
  }
  __syncthreads();

  // 4. weighted pooling c_rep = sum_i alpha_i c_i (Eq. 7), one column pair per thread
  const size_t out_row = (size_t)b * a.cache_rows + j;
  {
    bf16* dst = a.cache_sem + (out_row * a.Hkv + hk) * d_sem;
    for (int pr = tid; pr < d_sem / 2; pr += blockDim.x) {
      double a0 = 0.0, a1 = 0.0;
      for (int i = 0; i < g; ++i) {
        bf162 v = *reinterpret_cast<const bf162*>(t_sem + (size_t)i * d_sem + 2 * pr);
        double al = s_a[i];
        a0 = fma(al, (double)__low2float(v), a0);
        a1 = fma(al, (double)__high2float(v), a1);
      }
      bf162 o;
      o.x = double_to_bf16_rn(a0);
      o.y = double_to_bf16_rn(a1);
      *reinterpret_cast<bf162*>(dst + 2 * pr) = o;
    }
  }
  // 5. positional anchor: bit copy of the arg-max token's positional row
  {
    const int ia = s_anchor;
    const uint4* src = reinterpret_cast<const uint4*>(t_pos + (size_t)ia * d_pos);
    uint4* dst = reinterpret_cast<uint4*>(a.cache_pos + (out_row * a.Hkv + hk) * d_pos);
    for (int c = tid; c < d_pos / 8; c += blockDim.x) dst[c] = src[c];
    if (tid == 0) a.anchor[((size_t)b * a.m + j) * a.Hkv + hk] = j * g + ia;
  }
  if (a.scores) {
    double* sc = a.scores + (((size_t)b * a.Hkv + hk) * a.m + j) * g;
    for (int i = tid; i < g; i += blockDim.x) sc[i] = s_s[i];
  }
}

// ------------------------------------------------------------------------------ local window
// Copies, for every sequence, one contiguous block of `bytes16` 16-byte words.
__global__ void copy_blocks_kernel(const uint4* __restrict__ src, uint4* __restrict__ dst,
                                   size_t src_batch_stride16, size_t dst_batch_stride16,
                                   size_t src_off16, size_t dst_off16, size_t n16) {
  const uint4* s = src + (size_t)blockIdx.y * src_batch_stride16 + src_off16;
  uint4* d = dst + (size_t)blockIdx.y * dst_batch_stride16 + dst_off16;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n16;
       i += (size_t)gridDim.x * blockDim.x)
    d[i] = s[i];
}

// ------------------------------------------------------------------------------------- host
static int n_summary(const lca_params* p) {
  int n = p->n_summary_q > 0 ? p->n_summary_q : p->group_size;
  return n > p->seq_len ? p->seq_len : n;
}
static int key_dim(const lca_params* p) {
  return (p->variant == LCA_VARIANT_MLA ? p->d_sem : 0) + p->d_pos;
}
static int qbar_chunks(const lca_params* p) {
  int rows = n_summary(p) * (p->n_q_heads / p->n_kv_heads);
  return (rows + QBAR_ROWS_PER_CHUNK - 1) / QBAR_ROWS_PER_CHUNK;
}

size_t condense_workspace_bytes(const lca_params* p) {
  size_t streams = (size_t)p->batch * p->n_kv_heads;
  size_t dk = (size_t)key_dim(p);
  return (streams * dk + streams * dk * (size_t)qbar_chunks(p)) * sizeof(double);
}

size_t condense_smem_bytes(const lca_params* p) {
  size_t g = (size_t)p->group_size;
  return g * (size_t)(p->d_sem + p->d_pos) * sizeof(bf16) + ((size_t)key_dim(p) + 2 * g) * sizeof(double);
}

int condense_launch(const CondenseLaunch& c) {
  const lca_params* p = c.p;
  int64_t m, k;
  partition(p->seq_len, p->window, p->group_size, &m, &k);
  const int dk = key_dim(p);
  const int sem_in_logit = p->variant == LCA_VARIANT_MLA;
  const int B = p->batch, Hkv = p->n_kv_heads;
  double* qbar = reinterpret_cast<double*>(c.ws);
  double* partial = qbar + (size_t)B * Hkv * dk;

  if (m > 0) {
    if (c.qbar_opt) {
      int n = B * Hkv * dk;
      qbar_widen_kernel<<<(n + 255) / 256, 256, 0, c.stream>>>(c.qbar_opt, qbar, n);
      note_launch();
    } else {
      const int nch = qbar_chunks(p);
      dim3 grid(nch, Hkv, B);
      qbar_partial_kernel<<<grid, QBAR_THREADS, 0, c.stream>>>(
          (const bf16*)c.q_tail_sem, (const bf16*)c.q_tail_pos, c.q_tail_batch_stride, n_summary(p),
          p->n_q_heads, Hkv, p->d_sem, p->d_pos, sem_in_logit, partial);
      double count = (double)n_summary(p) * (double)(p->n_q_heads / Hkv);
      qbar_final_kernel<<<dim3(Hkv, B), QBAR_THREADS, 0, c.stream>>>(partial, nch, dk, count, qbar);
      note_launch(2);
    }
    CondenseArgs a;
    a.kv_sem = (const bf16*)c.kv_sem; a.kv_pos = (const bf16*)c.kv_pos; a.qbar = qbar;
    a.cache_sem = (bf16*)c.cache_sem; a.cache_pos = (bf16*)c.cache_pos;
    a.anchor = c.anchor_idx; a.scores = c.scores_opt;
    a.L = p->seq_len; a.Hkv = Hkv; a.d_sem = p->d_sem; a.d_pos = p->d_pos; a.g = p->group_size;
    a.m = (int)m; a.cache_rows = (int)(m + k); a.sem_in_logit = sem_in_logit;
    a.scale = (double)p->softmax_scale;
    size_t smem = condense_smem_bytes(p);
    if (cudaFuncSetAttribute(condense_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
      return LCA_ERR_CUDA;
    condense_kernel<<<dim3((unsigned)m, Hkv, B), CONDENSE_THREADS, smem, c.stream>>>(a);
    note_launch();
  }
  if (k > 0) {
    // rows L-k..L-1 of each sequence -> cache rows m..m+k-1 (one contiguous block per sequence)
    const size_t row_sem = (size_t)Hkv * p->d_sem * sizeof(bf16) / 16;
    const size_t row_pos = (size_t)Hkv * p->d_pos * sizeof(bf16) / 16;
    const unsigned blocks = 148 * 4;
    copy_blocks_kernel<<<dim3(blocks, B), 256, 0, c.stream>>>(
        (const uint4*)c.kv_sem, (uint4*)c.cache_sem, (size_t)p->seq_len * row_sem, (size_t)(m + k) * row_sem,
        (size_t)(p->seq_len - k) * row_sem, (size_t)m * row_sem, (size_t)k * row_sem);
    copy_blocks_kernel<<<dim3(blocks, B), 256, 0, c.stream>>>(
        (const uint4*)c.kv_pos, (uint4*)c.cache_pos, (size_t)p->seq_len * row_pos, (size_t)(m + k) * row_pos,
        (size_t)(p->seq_len - k) * row_pos, (size_t)m * row_pos, (size_t)k * row_pos);
    note_launch(2);
  }
  return cudaGetLastError() == cudaSuccess ? LCA_OK : LCA_ERR_CUDA;
}

// ------------------------------------------------------------------ fixed scratch (no allocation)
// Scratch of lca_condense_static_scratch: part of the library image on every device.  In host
// code the name below is only a handle; the device address comes from cudaGetSymbolAddress, asked
// once per device with that device current, and that address is what the kernels receive.
static __device__ __align__(256) unsigned char g_condense_static_scratch[LCA_STATIC_SCRATCH_BYTES];

int condense_static_scratch_address(void** out) {
  static std::mutex mu;
  static void* addr[64] = {};
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return LCA_ERR_CUDA;
  std::lock_guard<std::mutex> lock(mu);
  if (!addr[dev]) {
    void* p = nullptr;
    if (cudaGetSymbolAddress(&p, g_condense_static_scratch) != cudaSuccess || !p) return LCA_ERR_CUDA;
    addr[dev] = p;
  }
  *out = addr[dev];
  return LCA_OK;
}

}  // namespace lca
