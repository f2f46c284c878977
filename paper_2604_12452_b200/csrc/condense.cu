// Condensation kernels: summary query (Alg. 1, first step), group scores + softmax (Sec. 4.2, Eq. 6),
// weighted pooling (Eq. 7), anchor selection (Eq. 8) and the local-window copy (Eq. 9).
//
// The work is HBM-bound (about 2 flop per byte): every history token is read from global memory
// exactly once into shared memory, scored against the summary query, soft-maxed within its
// group, pooled, and the representative plus the anchor's positional row are written straight
// into the condensed cache.  The summary query and the scores are fp64, so the arg-max follows
// the exact scores rather than an fp32 accumulation order; the softmax weights and the pooling
// are fp32 (the fp64 pipe could not keep up with HBM for both), c_rep is rounded once to bf16.
#include <mutex>

#include <cuda.h>

#include "lca_common.cuh"

namespace lca {

static const int QBAR_ROWS_PER_CHUNK = 64;
static const int CONDENSE_THREADS = 512;

// ---------------------------------------------------------------------------- summary query
// Row lanes of qbar_partial_kernel for a key of `pieces` 16-byte pieces: about 288 threads per CTA.  With the 72 pieces
// of the MLA key that is four lanes, so that a chunk of 64 rows is two full rounds of eight rows per lane.
static int qbar_row_lanes(int pieces) {
  int lanes = 288 / pieces;
  return lanes < 1 ? 1 : lanes > 16 ? 16 : lanes;
}
// Partial sums of the query tail.  Rows of one KV head = (position, query head in its group);
// a chunk is QBAR_ROWS_PER_CHUNK rows and has its own partial sum; a CTA takes `chunks_per_cta` consecutive chunks one
// after the other (the sums do not depend on that number).  grid (CTAs, Hkv, B).  A thread owns one 16-byte piece
// (8 columns) of the key dimension and every row_lanes-th row of the chunk, so that consecutive
// threads read a whole query row and each thread has many independent loads in flight; the
// row lanes are then added up through shared memory in a fixed order.
// Ragged batch (tab.tok_off != nullptr): q_sem / q_pos are the whole packed query arrays and the tail of
// sequence b is its last min(n_pos, L_b) positions.
__global__ void qbar_partial_kernel(const bf16* __restrict__ q_sem, const bf16* __restrict__ q_pos,
                                    int64_t batch_stride_rows, int n_pos, int Hq, int Hkv, int d_sem,
                                    int d_pos, int sem_in_logit, int row_lanes, double* __restrict__ partial, SeqTab tab,
                                    int nchunks, int chunks_per_cta) {
  extern __shared__ double s_part_all[];                 // [2][row_lanes][dk]: chunks alternate, one barrier per chunk
  const int hk = blockIdx.y, b = blockIdx.z;
  const int rep = Hq / Hkv;
  long long first_pos = (long long)b * batch_stride_rows;     // row (position) of the first averaged query
  if (tab.tok_off) {
    const int len = tab.tok_off[b + 1] - tab.tok_off[b];
    n_pos = min(n_pos, len);
    first_pos = (long long)tab.tok_off[b] + len - n_pos;
  }
  const int n_rows = n_pos * rep;
  const int dk = (sem_in_logit ? d_sem : 0) + d_pos;
  const int pieces = dk / 8, sem_pieces = sem_in_logit ? d_sem / 8 : 0;
  const int pc = threadIdx.x % pieces, rl = threadIdx.x / pieces;
  for (int chunk = blockIdx.x * chunks_per_cta; chunk < min(nchunks, (int)(blockIdx.x + 1) * chunks_per_cta); ++chunk) {
  double* s_part = s_part_all + (size_t)(chunk & 1) * row_lanes * dk;
  const int r0 = chunk * QBAR_ROWS_PER_CHUNK;
  const int r1 = min(n_rows, r0 + QBAR_ROWS_PER_CHUNK);
  double acc[8];
#pragma unroll
  for (int i = 0; i < 8; ++i) acc[i] = 0.0;
  if (rl < row_lanes) {
    // Several rows per step: all loads of a step are issued before the first one is used (the kernel is bound by memory
    // latency otherwise); rows behind the end of the chunk contribute exact zeros, the order of the sums is fixed.
    // The piece of this thread lies in one of the two arrays, whose rows are d elements apart.
    const bool in_sem = pc < sem_pieces;
    const bf16* arr = in_sem ? q_sem + 8 * pc : q_pos + 8 * (pc - sem_pieces);
    const size_t d = in_sem ? d_sem : d_pos;
    auto add_row = [&](const uint4& x) {
      const unsigned w[4] = {x.x, x.y, x.z, x.w};
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        acc[2 * i] += (double)__uint_as_float(w[i] << 16);
        acc[2 * i + 1] += (double)__uint_as_float(w[i] & 0xffff0000u);
      }
    };
    int r = r0 + rl;
    if (Hkv == 1) {
      // one KV head: the rows of the tail are consecutive rows of the query arrays, so the loads of a thread are a fixed
      // stride apart (no per-row index arithmetic, no guards).  Eight rows per step: with sixteen the registers allow
      // only two CTAs per SM and the kernel was slower.
      const size_t step = (size_t)row_lanes * d / 8;
      for (; r + 7 * row_lanes < r1; r += 8 * row_lanes) {
        const uint4* src = reinterpret_cast<const uint4*>(arr + ((size_t)first_pos * Hq + r) * d);
        uint4 v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) v[u] = src[u * step];
#pragma unroll
        for (int u = 0; u < 8; ++u) add_row(v[u]);
      }
    }
    for (; r < r1; r += 8 * row_lanes) {
      uint4 v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int rr = r + u * row_lanes;
        v[u] = make_uint4(0u, 0u, 0u, 0u);
        if (rr < r1) {
          const size_t row = Hkv == 1 ? (size_t)first_pos * Hq + rr
                                      : ((size_t)first_pos + rr / rep) * Hq + hk * rep + rr % rep;
          v[u] = *reinterpret_cast<const uint4*>(arr + row * d);
        }
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) add_row(v[u]);
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) s_part[(size_t)rl * dk + 8 * pc + i] = acc[i];
  }
  __syncthreads();
  double* dst = partial + (((size_t)b * Hkv + hk) * nchunks + chunk) * dk;
  for (int c = threadIdx.x; c < dk; c += blockDim.x) {
    double sum = 0.0;
    for (int l = 0; l < row_lanes; ++l) sum += s_part[(size_t)l * dk + c];
    dst[c] = sum;
  }
  // no second barrier: the next chunk writes the other half of s_part_all, and the chunk after it passes the next
  // chunk's barrier before it writes this half again
  }
}

// Sum the chunk partials in chunk order and divide by the number of averaged rows.
// grid (Hkv, B)
__global__ void qbar_final_kernel(const double* __restrict__ partial, int nchunks, int dk,
                                  double count, double* __restrict__ qbar, SeqTab tab, int n_pos, int rep) {
  const size_t stream_id = (size_t)blockIdx.y * gridDim.x + blockIdx.x;
  if (tab.tok_off) {
    const int b = blockIdx.y;
    count = (double)min(n_pos, tab.tok_off[b + 1] - tab.tok_off[b]) * (double)rep;
  }
  const double* src = partial + stream_id * nchunks * dk;
  for (int c = threadIdx.x; c < dk; c += blockDim.x) {
    double s = 0.0;
#pragma unroll 16
    for (int ch = 0; ch < nchunks; ++ch) s += __ldg(src + (size_t)ch * dk + c);     // loads run ahead of the adds
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
  int sem_reducer, pos_reducer;   // LCA_REDUCE_* with DEFAULT already resolved
  long long n_groups;          // B * Hkv * m   (ragged batch: Hkv * sum of m_b)
  double scale;
  SeqTab tab;                  // ragged batch: L, m and cache_rows above are unused
};

// Where group `grp` of the launch lives: the KV head varies fastest, grp = (b * m + j) * Hkv + hk (ragged batch: the groups
// of sequence b start at grp_off[b] * Hkv), so that the CTAs of a persistent launch, which work on consecutive groups at any
// one time, read all heads of the same token rows together (a token row holds the Hkv heads side by side; one head at a
// time would touch an eighth of every DRAM page with Hkv = 8) and grp % Hkv is the head.
struct GroupLoc { int b, hk, j; long long tok0, out_row, grp_row; };     // first token row, cache row, row of anchor_idx
__device__ inline GroupLoc locate_group(const CondenseArgs& a, long long grp) {
  GroupLoc l;
  if (a.tab.tok_off) {
    int lo = 0, hi = a.tab.B - 1;
    while (lo < hi) {
      const int mid = (lo + hi + 1) >> 1;
      if ((long long)a.tab.grp_off[mid] * a.Hkv <= grp) lo = mid; else hi = mid - 1;
    }
    l.b = lo;
    const int m_b = a.tab.grp_off[lo + 1] - a.tab.grp_off[lo];
    const long long local = grp - (long long)a.tab.grp_off[lo] * a.Hkv;
    l.hk = (int)(local % a.Hkv); l.j = (int)(local / a.Hkv);
    (void)m_b;
    l.tok0 = (long long)a.tab.tok_off[lo] + (long long)l.j * a.g;
    l.out_row = (long long)a.tab.cache_off[lo] + l.j;
    l.grp_row = (long long)a.tab.grp_off[lo] + l.j;
  } else {
    l.hk = (int)(grp % a.Hkv);
    const long long bj = grp / a.Hkv;
    l.j = (int)(bj % a.m); l.b = (int)(bj / a.m);
    l.tok0 = (long long)l.b * a.L + (long long)l.j * a.g;
    l.out_row = (long long)l.b * a.cache_rows + l.j;
    l.grp_row = (long long)l.b * a.m + l.j;
  }
  return l;
}

__device__ inline void cp_async16(void* smem_dst, const void* gmem_src) {
  unsigned s = (unsigned)__cvta_generic_to_shared(smem_dst);
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(s), "l"(gmem_src) : "memory");
}

// Persistent CTAs (as many per SM as shared memory allows, at most two by registers); group index = (b * Hkv + hk) * m + j.  Two shared-memory stages:
// while a group is scored and pooled, the next one streams in with 16-byte cp.async copies, so
// every history byte is read from HBM once and the loads never wait for the arithmetic.
// A stage holds the g tokens [g][d_sem] and [g][d_pos] in bf16 and the summary query in fp64.
// Scores stay in fp64 (the arg-max must follow the exact scores); the group softmax and the
// pooling run in fp32, c_rep is rounded once to bf16.
__global__ void __launch_bounds__(CONDENSE_THREADS, 2)
condense_kernel(CondenseArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int g = a.g, d_sem = a.d_sem, d_pos = a.d_pos;
  const int dk = (a.sem_in_logit ? d_sem : 0) + d_pos;
  const size_t stage_bytes = (size_t)g * (d_sem + d_pos) * sizeof(bf16) + (size_t)dk * sizeof(double);
  double* s_s = reinterpret_cast<double*>(smem_raw + 2 * stage_bytes);      // [g] scores
  float* s_a = reinterpret_cast<float*>(s_s + g);                           // [g] alpha
  __shared__ int s_anchor;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
  const size_t row_stride_sem = (size_t)a.Hkv * d_sem, row_stride_pos = (size_t)a.Hkv * d_pos;
  const int cps = d_sem / 8, cpp = d_pos / 8, cpq = dk / 2;                 // 16-byte pieces per row / of q_bar

  auto stage_ptr = [&](int st) { return smem_raw + (size_t)st * stage_bytes; };
  auto prefetch = [&](long long grp, int st) {
    const GroupLoc loc = locate_group(a, grp);
    const int hk = loc.hk;
    const long long bh = (long long)loc.b * a.Hkv + hk;
    bf16* t_sem = reinterpret_cast<bf16*>(stage_ptr(st));
    bf16* t_pos = t_sem + (size_t)g * d_sem;
    double* s_q = reinterpret_cast<double*>(t_pos + (size_t)g * d_pos);
    const size_t tok0 = (size_t)loc.tok0;
    const bf16* gs = a.kv_sem + tok0 * row_stride_sem + (size_t)hk * d_sem;
    const bf16* gp = a.kv_pos + tok0 * row_stride_pos + (size_t)hk * d_pos;
    for (int x = tid; x < g * cps; x += blockDim.x) {
      const int i = x / cps, c = x % cps;
      cp_async16(t_sem + (size_t)i * d_sem + c * 8, gs + (size_t)i * row_stride_sem + c * 8);
    }
    for (int x = tid; x < g * cpp; x += blockDim.x) {
      const int i = x / cpp, c = x % cpp;
      cp_async16(t_pos + (size_t)i * d_pos + c * 8, gp + (size_t)i * row_stride_pos + c * 8);
    }
    const double* qb = a.qbar + (size_t)bh * dk;
    for (int x = tid; x < cpq; x += blockDim.x) cp_async16(s_q + 2 * x, qb + 2 * x);
  };

  long long grp = blockIdx.x;
  if (grp < a.n_groups) prefetch(grp, 0);
  asm volatile("cp.async.commit_group;\n" ::: "memory");
  for (int it = 0; grp < a.n_groups; ++it, grp += gridDim.x) {
    const int st = it & 1;
    const long long next = grp + gridDim.x;
    if (next < a.n_groups) prefetch(next, st ^ 1);
    asm volatile("cp.async.commit_group;\ncp.async.wait_group 1;\n" ::: "memory");
    __syncthreads();

    const GroupLoc loc = locate_group(a, grp);
    const int j = loc.j, hk = loc.hk;
    const bf16* t_sem = reinterpret_cast<const bf16*>(stage_ptr(st));
    const bf16* t_pos = t_sem + (size_t)g * d_sem;
    const double* s_q = reinterpret_cast<const double*>(t_pos + (size_t)g * d_pos);

    // 1. importance scores s_i = scale * q_bar . k_i   (one warp per token, fp64)
    const int sem_off = a.sem_in_logit ? d_sem : 0;
    for (int i = warp; i < g; i += nwarps) {
      double acc0 = 0.0, acc1 = 0.0;
      if (a.sem_in_logit) {
        const bf162* row = reinterpret_cast<const bf162*>(t_sem + (size_t)i * d_sem);
        for (int pr = lane; pr < d_sem / 2; pr += 32) {
          const bf162 v = row[pr];
          acc0 = fma(s_q[2 * pr], (double)__low2float(v), acc0);
          acc1 = fma(s_q[2 * pr + 1], (double)__high2float(v), acc1);
        }
      }
      {
        const bf162* row = reinterpret_cast<const bf162*>(t_pos + (size_t)i * d_pos);
        for (int pr = lane; pr < d_pos / 2; pr += 32) {
          const bf162 v = row[pr];
          acc0 = fma(s_q[sem_off + 2 * pr], (double)__low2float(v), acc0);
          acc1 = fma(s_q[sem_off + 2 * pr + 1], (double)__high2float(v), acc1);
        }
      }
      const double acc = warp_sum(acc0 + acc1);
      if (lane == 0) s_s[i] = acc * a.scale;
    }
    __syncthreads();

    // 2. arg-max on the fp64 scores (Eq. 8; lowest index on ties) and group softmax (Eq. 6), warp 0
    if (warp == 0) {
      double best = -INFINITY;
      int besti = 0x7fffffff;
      for (int i = lane; i < g; i += 32) {
        const double s = s_s[i];
        if (s > best) { best = s; besti = i; }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const double ob = __shfl_xor_sync(0xffffffffu, best, o);
        const int oi = __shfl_xor_sync(0xffffffffu, besti, o);
        if (ob > best || (ob == best && oi < besti)) { best = ob; besti = oi; }
      }
      float z = 0.f;
      for (int i = lane; i < g; i += 32) {
        const float e = expf((float)(s_s[i] - best));
        s_a[i] = e;
        z += e;
      }
      z = warp_sum(z);
      const float inv = 1.f / z;
      for (int i = lane; i < g; i += 32) s_a[i] *= inv;
      if (lane == 0) s_anchor = besti;
    }
    __syncthreads();

    // 3. the representative: semantic part (Eq. 7 by default) and positional part (Eq. 8 by
    //    default), each reduced over the g tokens by the chosen operator, one column pair per thread
    const size_t out_row = (size_t)loc.out_row;
    const int ia = s_anchor;
    auto reduce = [&](const bf16* tile, int d, int mode, bf16* dst, int tid0) {
      for (int pr = tid0; pr < d / 2; pr += blockDim.x) {
        if (mode == LCA_REDUCE_MAXSEL) {
          *reinterpret_cast<bf162*>(dst + 2 * pr) = *reinterpret_cast<const bf162*>(tile + (size_t)ia * d + 2 * pr);
          continue;
        }
        float a0 = mode == LCA_REDUCE_MAXPOOL ? -INFINITY : 0.f, a1 = a0;
#pragma unroll 8
        for (int i = 0; i < g; ++i) {
          const float2 v = __bfloat1622float2(*reinterpret_cast<const bf162*>(tile + (size_t)i * d + 2 * pr));
          if (mode == LCA_REDUCE_MAXPOOL) { a0 = fmaxf(a0, v.x); a1 = fmaxf(a1, v.y); }
          else if (mode == LCA_REDUCE_MEANPOOL) { a0 += v.x; a1 += v.y; }
          else { const float al = s_a[i]; a0 = fmaf(al, v.x, a0); a1 = fmaf(al, v.y, a1); }
        }
        if (mode == LCA_REDUCE_MEANPOOL) { a0 /= (float)g; a1 /= (float)g; }
        *reinterpret_cast<bf162*>(dst + 2 * pr) = __floats2bfloat162_rn(a0, a1);
      }
    };
    reduce(t_sem, d_sem, a.sem_reducer, a.cache_sem + (out_row * a.Hkv + hk) * d_sem, tid);
    reduce(t_pos, d_pos, a.pos_reducer, a.cache_pos + (out_row * a.Hkv + hk) * d_pos, blockDim.x - 1 - tid);
    {
      const int rt = blockDim.x - 1 - tid;
      if (rt == 0) a.anchor[(size_t)loc.grp_row * a.Hkv + hk] = j * g + ia;
      if (a.scores) {
        double* sc = a.scores + (((size_t)loc.b * a.Hkv + hk) * a.m + j) * g;
        for (int i = rt; i < g; i += blockDim.x) sc[i] = s_s[i];
      }
    }
    __syncthreads();        // the stage and the score arrays are free for the next round
  }
  asm volatile("cp.async.wait_group 0;\n" ::: "memory");
}

// ----------------------------------------------------- condense, MLA shape with g = 64 (the fast path)
// Same results as condense_kernel for d_sem = 512, d_pos = 64, g = 64 and one KV stream, laid out for the
// instruction budget HBM speed leaves (about 3000 issue cycles per group and SM, for 73 KB of input).  The
// CTA is split into roles that work on different groups at the same time and meet only through mbarriers:
//   * one producer thread fetches a group (64 KB + 8 KB of contiguous memory) with two bulk copies
//     (cp.async.bulk) into one of three stages;
//   * sixteen score warps: warp w takes tokens w, w+16, w+32, w+48; lane l holds the 18 components of q_bar
//     it needs in registers (columns 8l..8l+7 and 256+8l..256+8l+7 of the latent part, 2l, 2l+1 of the rope
//     part) as fp32, reads its share of a token with two 16-byte and one 4-byte load, and forms the product
//     sum in fp32 together with max_c |k_ic|; one transposed shuffle reduction per four tokens;
//   * one arbiter warp takes the group's arg-max and softmax from those 64 sums.  An fp32 sum of this kernel
//     passes through at most 15 roundings (9 multiply-adds per chain, the chain pair, 5 shuffle levels) and
//     q_bar is rounded once to fp32, so |s32_i - s_i| <= 16 u (1 + 16 u) sum_c |q_c| |k_ic| <= 16 u (1 + 16 u)
//     |q_bar|_1 max_c |k_ic| with u = 2^-24.  Where the two largest sums of a group are further apart than
//     MARGIN_FACTOR |q_bar|_1 max_ic |k_ic| (twice that bound with a quarter of slack and the rounding of |q_bar|_1
//     and of the difference), the fp32 arg-max is the arg-max of the exact scores.  Every other group (about one
//     in a thousand; exact ties included) is scored again by the arbiter warp in fp64, and so is every group when
//     the caller asked for the scores: anchors always follow the fp64 scores, lowest index on ties;
//   * four pool warps, one group behind: four output columns per thread, fp32 pairs, alpha read four tokens at
//     a time; they also copy the anchor's rope row and write the anchor index.
namespace fast {
constexpr int G = 64, DS = 512, DP = 64, DK = DS + DP, STAGES = 3;
constexpr int SCORE_WARPS = 16, POOL_WARPS = 4;
constexpr int WARP_ARBITER = SCORE_WARPS, WARP_POOL0 = SCORE_WARPS + 1, WARP_PRODUCER = WARP_POOL0 + POOL_WARPS;
constexpr int THREADS = 32 * (WARP_PRODUCER + 1);
constexpr int SEM_BYTES = G * DS * 2, POS_BYTES = G * DP * 2, STAGE_BYTES = SEM_BYTES + POS_BYTES;
constexpr int OFF_A = STAGES * STAGE_BYTES;                 // float[2][G] alpha
constexpr int OFF_S32 = OFF_A + 2 * G * 4;                  // float[2][G] fp32 sums q_bar . k_i (before the scale)
constexpr int OFF_NRM = OFF_S32 + 2 * G * 4;                // float[2][G] max_c |k_ic|
constexpr int OFF_BAR = OFF_NRM + 2 * G * 4;                // mbarriers: full[3] free[3] scored[2] ready[2] afree[2], then flags
constexpr int SMEM_BYTES = OFF_BAR + 128;
constexpr float MARGIN_FACTOR = 48.0f * 5.9604644775390625e-08f;
static_assert(SMEM_BYTES <= 232448, "shared memory budget of one SM");
static_assert(G / SCORE_WARPS == 4, "four tokens per score warp");
constexpr long long WAIT_CYCLES = 2000000000ll;
}  // namespace fast

static __device__ int g_condense_status = 0;

__device__ __forceinline__ bool cond_wait(unsigned bar, unsigned parity, volatile int* abort_flag) {
  unsigned done = 0;
  long long t0 = 0;
  while (true) {
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    if (done) return true;
    if (t0 == 0) t0 = clock64();
    if (*abort_flag || clock64() - t0 > fast::WAIT_CYCLES) { *abort_flag = 1; return false; }
    __nanosleep(40);                                      // leave the issue slots to the working warps
  }
}
__device__ __forceinline__ void cond_arrive(unsigned bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ float f32_max3_abs(float acc, float a, float b) {     // max(acc, |a|, |b|)
  return fmaxf(fmaxf(acc, fabsf(a)), fabsf(b));
}
__device__ __forceinline__ unsigned long long f32x2(float lo, float hi) {
  unsigned long long r;
  asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
  return r;
}
__device__ __forceinline__ unsigned long long fma_f32x2(unsigned long long a, unsigned long long b, unsigned long long c) {
  unsigned long long r;
  asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
  return r;
}

// The exact scores of one group by one warp (the arbiter), q_bar in fp64 from global memory: token by token,
// lane l takes the same 18 columns as in the fp32 pass; every lane ends up with the scores of tokens l and l + 32.
__device__ __noinline__ void score_group_fp64(const unsigned char* t_sem, const unsigned char* t_pos, const double* qbar,
                                              int lane, double scale, double& s_lo, double& s_hi) {
  using namespace fast;
  double q[18];
#pragma unroll
  for (int i = 0; i < 8; ++i) { q[i] = qbar[8 * lane + i]; q[8 + i] = qbar[256 + 8 * lane + i]; }
  q[16] = qbar[DS + 2 * lane]; q[17] = qbar[DS + 2 * lane + 1];
  s_lo = 0.0; s_hi = 0.0;
#pragma unroll 1
  for (int i = 0; i < G; ++i) {
    const uint4 v0 = *reinterpret_cast<const uint4*>(t_sem + (size_t)i * (DS * 2) + 16 * lane);
    const uint4 v1 = *reinterpret_cast<const uint4*>(t_sem + (size_t)i * (DS * 2) + 512 + 16 * lane);
    const unsigned vp = *reinterpret_cast<const unsigned*>(t_pos + (size_t)i * (DP * 2) + 4 * lane);
    const unsigned w[9] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w, vp};
    double acc0 = 0.0, acc1 = 0.0;
#pragma unroll
    for (int k = 0; k < 9; ++k) {
      acc0 = fma(q[2 * k], (double)__uint_as_float(w[k] << 16), acc0);
      acc1 = fma(q[2 * k + 1], (double)__uint_as_float(w[k] & 0xffff0000u), acc1);
    }
    const double c = warp_sum(acc0 + acc1) * scale;       // the same value in every lane (xor butterfly)
    if ((i & 31) == lane) { if (i < 32) s_lo = c; else s_hi = c; }
  }
}

__global__ void __launch_bounds__(fast::THREADS, 1)
condense_mla64_kernel(CondenseArgs a) {
  using namespace fast;
  extern __shared__ __align__(128) unsigned char smem[];
  float* s_a = reinterpret_cast<float*>(smem + OFF_A);
  float* s_s32 = reinterpret_cast<float*>(smem + OFF_S32);
  float* s_nrm = reinterpret_cast<float*>(smem + OFF_NRM);
  const unsigned bar0 = (unsigned)__cvta_generic_to_shared(smem + OFF_BAR);
  auto BAR_FULL = [&](int st) { return bar0 + 8 * st; };
  auto BAR_FREE = [&](int st) { return bar0 + 24 + 8 * st; };
  auto BAR_SCORED = [&](int p) { return bar0 + 48 + 8 * p; };     // sums of parity p written by the score warps
  auto BAR_READY = [&](int p) { return bar0 + 64 + 8 * p; };      // alpha / anchor of parity p written
  auto BAR_AFREE = [&](int p) { return bar0 + 80 + 8 * p; };      // ... and consumed
  volatile int* s_anchor = reinterpret_cast<volatile int*>(smem + OFF_BAR + 96);   // [2]
  volatile int* s_abort = reinterpret_cast<volatile int*>(smem + OFF_BAR + 104);
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  if (tid == 0) {
    for (int st = 0; st < STAGES; ++st) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(BAR_FULL(st)) : "memory");
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(BAR_FREE(st)), "r"(POOL_WARPS) : "memory");
    }
    for (int p = 0; p < 2; ++p) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(BAR_SCORED(p)), "r"(SCORE_WARPS) : "memory");
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(BAR_READY(p)) : "memory");
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(BAR_AFREE(p)), "r"(POOL_WARPS) : "memory");
    }
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  const long long first = blockIdx.x, stride = gridDim.x;
  const long long n_mine = first < a.n_groups ? (a.n_groups - first + stride - 1) / stride : 0;

  if (warp == WARP_PRODUCER) {
    // ===================================================== producer
    if (lane == 0) {
      for (long long it = 0; it < n_mine; ++it) {
        const int st = (int)(it % STAGES);
        if (it >= STAGES && !cond_wait(BAR_FREE(st), (unsigned)((it / STAGES - 1) & 1), s_abort)) break;
        const long long grp = first + it * stride;
        const size_t tok0 = (size_t)locate_group(a, grp).tok0;
        const unsigned dst = (unsigned)__cvta_generic_to_shared(smem + (size_t)st * STAGE_BYTES);
        const unsigned bar = BAR_FULL(st);
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(STAGE_BYTES) : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(dst), "l"(a.kv_sem + tok0 * DS), "r"(SEM_BYTES), "r"(bar) : "memory");
        asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                     ::"r"(dst + SEM_BYTES), "l"(a.kv_pos + tok0 * DP), "r"(POS_BYTES), "r"(bar) : "memory");
      }
    }
  } else if (warp < SCORE_WARPS) {
    // ===================================================== fp32 product sums and max |k| of four tokens per warp
    unsigned long long q2[9];                             // q_bar components of this lane, in pairs (two FMAs per instruction)
    long long cur_b = -1;
    for (long long it = 0; it < n_mine; ++it) {
      const int st = (int)(it % STAGES), p = (int)(it & 1);
      const long long grp = first + it * stride;
      const long long b = a.tab.tok_off ? seq_of(a.tab.grp_off, a.tab.B, grp) : grp / a.m;
      if (b != cur_b) {                                   // rare: the next sequence's summary query
        cur_b = b;
        const double* qb = a.qbar + (size_t)b * DK;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          q2[i] = f32x2((float)qb[8 * lane + 2 * i], (float)qb[8 * lane + 2 * i + 1]);
          q2[4 + i] = f32x2((float)qb[256 + 8 * lane + 2 * i], (float)qb[256 + 8 * lane + 2 * i + 1]);
        }
        q2[8] = f32x2((float)qb[DS + 2 * lane], (float)qb[DS + 2 * lane + 1]);
      }
      if (!cond_wait(BAR_FULL(st), (unsigned)((it / STAGES) & 1), s_abort)) break;
      if (it >= 2 && !cond_wait(BAR_AFREE(p), (unsigned)(((it >> 1) - 1) & 1), s_abort)) break;
      const unsigned char* t_sem = smem + (size_t)st * STAGE_BYTES;
      const unsigned char* t_pos = t_sem + SEM_BYTES;
      float v[8];                                         // sums of the four tokens, then their max |k|
#pragma unroll
      for (int tt = 0; tt < 4; ++tt) {
        const int i = warp + SCORE_WARPS * tt;
        const uint4 v0 = *reinterpret_cast<const uint4*>(t_sem + (size_t)i * (DS * 2) + 16 * lane);
        const uint4 v1 = *reinterpret_cast<const uint4*>(t_sem + (size_t)i * (DS * 2) + 512 + 16 * lane);
        const unsigned vp = *reinterpret_cast<const unsigned*>(t_pos + (size_t)i * (DP * 2) + 4 * lane);
        const unsigned w[9] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w, vp};
        unsigned long long acc = f32x2(0.f, 0.f);        // even / odd components: the same two fp32 chains as scalar FMAs
        float kmax = 0.f;
#pragma unroll
        for (int k = 0; k < 9; ++k) {
          const float lo = __uint_as_float(w[k] << 16), hi = __uint_as_float(w[k] & 0xffff0000u);
          acc = fma_f32x2(q2[k], f32x2(lo, hi), acc);
          kmax = f32_max3_abs(kmax, lo, hi);
        }
        float acc0, acc1;
        asm("mov.b64 {%0, %1}, %2;" : "=f"(acc0), "=f"(acc1) : "l"(acc));
        v[tt] = acc0 + acc1;
        v[4 + tt] = kmax;
      }
      // transposed reduction over the warp: lanes with bit 4 clear add up the sums, the others take the maxima;
      // bits 3 and 2 select the token; lanes 0, 4, ..., 28 end up with one result each
      const bool up16 = (lane & 16) != 0, up8 = (lane & 8) != 0, up4 = (lane & 4) != 0;
      auto comb = [&](float x, float y) { return up16 ? fmaxf(x, y) : x + y; };
      float r[4], t2[2];
#pragma unroll
      for (int i = 0; i < 4; ++i) r[i] = comb(up16 ? v[4 + i] : v[i], __shfl_xor_sync(0xffffffffu, up16 ? v[i] : v[4 + i], 16));
#pragma unroll
      for (int i = 0; i < 2; ++i) t2[i] = comb(up8 ? r[2 + i] : r[i], __shfl_xor_sync(0xffffffffu, up8 ? r[i] : r[2 + i], 8));
      float c = comb(up4 ? t2[1] : t2[0], __shfl_xor_sync(0xffffffffu, up4 ? t2[0] : t2[1], 4));
      c = comb(c, __shfl_xor_sync(0xffffffffu, c, 2));
      c = comb(c, __shfl_xor_sync(0xffffffffu, c, 1));
      if ((lane & 3) == 0) (up16 ? s_nrm : s_s32)[p * G + warp + SCORE_WARPS * ((lane >> 2) & 3)] = c;
      __syncwarp();
      if (lane == 0) cond_arrive(BAR_SCORED(p));
    }
  } else if (warp == WARP_ARBITER) {
    // ===================================================== arg-max (fp32 where provably exact, else fp64) and softmax
    const bool exact_all = a.scores != nullptr;
    const float scale32 = (float)a.scale;
    long long cur_b = -1;
    float q_l1 = 0.f;                                     // |q_bar|_1 of the current sequence (fp32 values, fp32 sum)
    for (long long it = 0; it < n_mine; ++it) {
      const int st = (int)(it % STAGES), p = (int)(it & 1);
      const long long grp = first + it * stride;
      const long long b = a.tab.tok_off ? seq_of(a.tab.grp_off, a.tab.B, grp) : grp / a.m;
      const double* qb = a.qbar + (size_t)b * DK;
      if (b != cur_b) {
        cur_b = b;
        float t = 0.f;
        for (int x = lane; x < DK; x += 32) t += fabsf((float)qb[x]);
        q_l1 = warp_sum(t);
      }
      if (!cond_wait(BAR_SCORED(p), (unsigned)((it >> 1) & 1), s_abort)) break;
      const float sa = s_s32[p * G + lane], sb = s_s32[p * G + lane + 32];
      float m1, m2;
      int i1;
      if (sb > sa) { m1 = sb; i1 = lane + 32; m2 = sa; } else { m1 = sa; i1 = lane; m2 = sb; }
      float km = fmaxf(s_nrm[p * G + lane], s_nrm[p * G + lane + 32]);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float om1 = __shfl_xor_sync(0xffffffffu, m1, o), om2 = __shfl_xor_sync(0xffffffffu, m2, o);
        const int oi = __shfl_xor_sync(0xffffffffu, i1, o);
        km = fmaxf(km, __shfl_xor_sync(0xffffffffu, km, o));
        m2 = fmaxf(fminf(m1, om1), fmaxf(m2, om2));       // a repeated maximum counts twice
        if (om1 > m1 || (om1 == m1 && oi < i1)) { m1 = om1; i1 = oi; }
      }
      const bool exact = exact_all || !(m1 - m2 > MARGIN_FACTOR * q_l1 * km);   // also taken when a value is not finite
      float ea, eb;
      int besti;
      if (exact) {
        if (!cond_wait(BAR_FULL(st), (unsigned)((it / STAGES) & 1), s_abort)) break;    // complete; makes the tile visible here
        const unsigned char* t_sem = smem + (size_t)st * STAGE_BYTES;
        double da, db;
        score_group_fp64(t_sem, t_sem + SEM_BYTES, qb, lane, a.scale, da, db);
        double best = da; besti = lane;
        if (db > best) { best = db; besti = lane + 32; }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          const double ob = __shfl_xor_sync(0xffffffffu, best, o);
          const int oi = __shfl_xor_sync(0xffffffffu, besti, o);
          if (ob > best || (ob == best && oi < besti)) { best = ob; besti = oi; }
        }
        ea = expf((float)(da - best)); eb = expf((float)(db - best));
        if (a.scores) {
          double* sc = a.scores + (size_t)grp * G;            // one KV stream: group grp of the launch is row grp
          sc[lane] = da; sc[lane + 32] = db;
        }
      } else {
        besti = i1;
        ea = expf((sa - m1) * scale32); eb = expf((sb - m1) * scale32);
      }
      const float inv = 1.f / warp_sum(ea + eb);
      s_a[p * G + lane] = ea * inv; s_a[p * G + lane + 32] = eb * inv;
      if (lane == 0) s_anchor[p] = besti;
      __syncwarp();
      if (lane == 0) cond_arrive(BAR_READY(p));
    }
  } else {
    // ===================================================== pooling and outputs, one group behind
    const int pt = tid - 32 * WARP_POOL0;                 // 0..127: output columns 4 pt .. 4 pt + 3
    for (long long it = 0; it < n_mine; ++it) {
      const int st = (int)(it % STAGES), p = (int)(it & 1);
      const long long grp = first + it * stride;
      const GroupLoc loc = locate_group(a, grp);
      const int j = loc.j;
      if (!cond_wait(BAR_READY(p), (unsigned)((it >> 1) & 1), s_abort)) break;
      if (!cond_wait(BAR_FULL(st), (unsigned)((it / STAGES) & 1), s_abort)) break;     // complete long ago
      const unsigned char* t_sem = smem + (size_t)st * STAGE_BYTES;
      const unsigned char* t_pos = t_sem + SEM_BYTES;
      const size_t out_row = (size_t)loc.out_row;
      unsigned long long acc01 = f32x2(0.f, 0.f), acc23 = f32x2(0.f, 0.f);
      const uint2* col = reinterpret_cast<const uint2*>(t_sem) + pt;
      const float* al_base = s_a + p * G;
#pragma unroll 4                                           // sixteen tokens' loads in flight: the one pooling warp of a scheduler waits for shared memory otherwise
      for (int i = 0; i < G; i += 4) {
        const float4 al = *reinterpret_cast<const float4*>(al_base + i);
        const float alv[4] = {al.x, al.y, al.z, al.w};
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const uint2 w = col[(i + u) * (DS / 4)];
          const unsigned long long al2 = f32x2(alv[u], alv[u]);
          acc01 = fma_f32x2(al2, f32x2(__uint_as_float(w.x << 16), __uint_as_float(w.x & 0xffff0000u)), acc01);
          acc23 = fma_f32x2(al2, f32x2(__uint_as_float(w.y << 16), __uint_as_float(w.y & 0xffff0000u)), acc23);
        }
      }
      {
        float a0, a1, a2, a3;
        asm("mov.b64 {%0, %1}, %2;" : "=f"(a0), "=f"(a1) : "l"(acc01));
        asm("mov.b64 {%0, %1}, %2;" : "=f"(a2), "=f"(a3) : "l"(acc23));
        const bf162 lo = __floats2bfloat162_rn(a0, a1), hi = __floats2bfloat162_rn(a2, a3);
        uint2 o;
        o.x = *reinterpret_cast<const unsigned*>(&lo); o.y = *reinterpret_cast<const unsigned*>(&hi);
        *reinterpret_cast<uint2*>(a.cache_sem + out_row * DS + 4 * pt) = o;
      }
      const int ia = s_anchor[p];
      if (pt < DP / 8)
        reinterpret_cast<uint4*>(a.cache_pos + out_row * DP)[pt] = reinterpret_cast<const uint4*>(t_pos + (size_t)ia * (DP * 2))[pt];
      if (pt == 32) a.anchor[grp] = j * G + ia;
      __syncwarp();
      if (lane == 0) { cond_arrive(BAR_AFREE(p)); cond_arrive(BAR_FREE(st)); }
    }
  }
  __syncthreads();
  if (tid == 0 && *s_abort) atomicCAS(&g_condense_status, 0, 1);
}

// ----------------------------------------------------- condense, GQA shape (head dimension 128) with g = 64
// The role-split structure of condense_mla64_kernel for keys / values of 128 columns that are interleaved by KV head
// in memory ([L, Hkv, 128]): a group of one KV head is 64 rows of 256 bytes, 256 Hkv bytes apart, fetched as two
// tiled TMA boxes (keys 16 KB, values 16 KB) into one of six stages.  Four score warps (16 tokens each: eight tokens per
// pass, a token's 128 columns over four lanes), the arbiter warp (arg-max: fp32 where the margin proves it, fp64
// otherwise; softmax), one pool warp (four value columns per lane; anchor key row, index), one producer thread.
// An fp32 sum passes through at most 19 roundings here (16 multiply-adds per chain, the chain pair, 2 shuffle levels).
namespace gfast {
constexpr int G = 64, D = 128, STAGES = 6;
constexpr int SCORE_WARPS = 4;
constexpr int WARP_ARBITER = SCORE_WARPS, WARP_POOL = SCORE_WARPS + 1, WARP_PRODUCER = SCORE_WARPS + 2;
constexpr int THREADS = 32 * (WARP_PRODUCER + 1);
constexpr int TILE_BYTES = G * D * 2, STAGE_BYTES = 2 * TILE_BYTES;         // keys, then values
constexpr int OFF_A = STAGES * STAGE_BYTES;                 // float[2][G] alpha
constexpr int OFF_S32 = OFF_A + 2 * G * 4, OFF_NRM = OFF_S32 + 2 * G * 4, OFF_BAR = OFF_NRM + 2 * G * 4;
constexpr int SMEM_BYTES = OFF_BAR + 192;
constexpr float MARGIN_FACTOR = 60.0f * 5.9604644775390625e-08f;
static_assert(SMEM_BYTES <= 232448, "shared memory budget of one SM");
}  // namespace gfast

struct GqaCondenseMaps { CUtensorMap k, v; };

__global__ void __launch_bounds__(gfast::THREADS, 1)
condense_gqa64_kernel(CondenseArgs a, const __grid_constant__ GqaCondenseMaps maps) {
  using namespace gfast;
  extern __shared__ __align__(128) unsigned char smem[];
  float* s_a = reinterpret_cast<float*>(smem + OFF_A);
  float* s_s32 = reinterpret_cast<float*>(smem + OFF_S32);
  float* s_nrm = reinterpret_cast<float*>(smem + OFF_NRM);
  const unsigned bar0 = (unsigned)__cvta_generic_to_shared(smem + OFF_BAR);
  auto BAR_FULL = [&](int st) { return bar0 + 8 * st; };
  auto BAR_FREE = [&](int st) { return bar0 + 8 * (STAGES + st); };
  auto BAR_SCORED = [&](int p) { return bar0 + 8 * (2 * STAGES + p); };
  auto BAR_READY = [&](int p) { return bar0 + 8 * (2 * STAGES + 2 + p); };
  auto BAR_AFREE = [&](int p) { return bar0 + 8 * (2 * STAGES + 4 + p); };
  volatile int* s_anchor = reinterpret_cast<volatile int*>(smem + OFF_BAR + 8 * (2 * STAGES + 6));   // [2]
  volatile int* s_abort = s_anchor + 2;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  if (tid == 0) {
    for (int st = 0; st < STAGES; ++st) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(BAR_FULL(st)) : "memory");
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(BAR_FREE(st)) : "memory");
    }
    for (int p = 0; p < 2; ++p) {
      asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(BAR_SCORED(p)), "r"(SCORE_WARPS) : "memory");
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(BAR_READY(p)) : "memory");
      asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(BAR_AFREE(p)) : "memory");
    }
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();

  const long long first = blockIdx.x, stride = gridDim.x;
  const long long n_mine = first < a.n_groups ? (a.n_groups - first + stride - 1) / stride : 0;

  if (warp == WARP_PRODUCER) {
    if (lane == 0) {
      for (long long it = 0; it < n_mine; ++it) {
        const int st = (int)(it % STAGES);
        if (it >= STAGES && !cond_wait(BAR_FREE(st), (unsigned)((it / STAGES - 1) & 1), s_abort)) break;
        const GroupLoc loc = locate_group(a, first + it * stride);
        const unsigned dst = (unsigned)__cvta_generic_to_shared(smem + (size_t)st * STAGE_BYTES);
        const unsigned bar = BAR_FULL(st);
        asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(STAGE_BYTES) : "memory");
        asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
                     ::"r"(dst), "l"(&maps.k), "r"(0), "r"(loc.hk), "r"((int)loc.tok0), "r"(bar) : "memory");
        asm volatile("cp.async.bulk.tensor.3d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
                     ::"r"(dst + TILE_BYTES), "l"(&maps.v), "r"(0), "r"(loc.hk), "r"((int)loc.tok0), "r"(bar) : "memory");
      }
    }
  } else if (warp < SCORE_WARPS) {
    // ===================================================== fp32 product sums and max |k| of sixteen tokens per warp
    const int tsub = lane >> 2, slice = lane & 3;           // token inside a pass of eight, 32-column slice
    float q[32];
    long long cur_stream = -1;
    for (long long it = 0; it < n_mine; ++it) {
      const int st = (int)(it % STAGES), p = (int)(it & 1);
      const GroupLoc loc = locate_group(a, first + it * stride);
      const long long stream = (long long)loc.b * a.Hkv + loc.hk;
      if (stream != cur_stream) {                           // the next KV stream's summary query
        cur_stream = stream;
        const double* qb = a.qbar + (size_t)stream * D + 32 * slice;
#pragma unroll
        for (int i = 0; i < 32; ++i) q[i] = (float)qb[i];
      }
      if (!cond_wait(BAR_FULL(st), (unsigned)((it / STAGES) & 1), s_abort)) break;
      if (it >= 2 && !cond_wait(BAR_AFREE(p), (unsigned)(((it >> 1) - 1) & 1), s_abort)) break;
      const unsigned char* t_k = smem + (size_t)st * STAGE_BYTES;
#pragma unroll
      for (int pass = 0; pass < 2; ++pass) {
        const int i = 16 * warp + 8 * pass + tsub;          // token of this lane
        const uint4* src = reinterpret_cast<const uint4*>(t_k + (size_t)i * (D * 2) + 64 * slice);
        float acc0 = 0.f, acc1 = 0.f, kmax = 0.f;
#pragma unroll
        for (int x = 0; x < 4; ++x) {
          const uint4 v = src[x];
          const unsigned w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const float lo = __uint_as_float(w[k] << 16), hi = __uint_as_float(w[k] & 0xffff0000u);
            acc0 = fmaf(q[8 * x + 2 * k], lo, acc0);
            acc1 = fmaf(q[8 * x + 2 * k + 1], hi, acc1);
            kmax = f32_max3_abs(kmax, lo, hi);
          }
        }
        float sum = acc0 + acc1;
        sum += __shfl_xor_sync(0xffffffffu, sum, 1); kmax = fmaxf(kmax, __shfl_xor_sync(0xffffffffu, kmax, 1));
        sum += __shfl_xor_sync(0xffffffffu, sum, 2); kmax = fmaxf(kmax, __shfl_xor_sync(0xffffffffu, kmax, 2));
        if (slice == 0) { s_s32[p * G + i] = sum; s_nrm[p * G + i] = kmax; }
      }
      __syncwarp();
      if (lane == 0) cond_arrive(BAR_SCORED(p));
    }
  } else if (warp == WARP_ARBITER) {
    // ===================================================== arg-max (fp32 where provably exact, else fp64) and softmax
    const bool exact_all = a.scores != nullptr;
    const float scale32 = (float)a.scale;
    long long cur_stream = -1;
    float q_l1 = 0.f;
    for (long long it = 0; it < n_mine; ++it) {
      const int st = (int)(it % STAGES), p = (int)(it & 1);
      const GroupLoc loc = locate_group(a, first + it * stride);
      const long long stream = (long long)loc.b * a.Hkv + loc.hk;
      const double* qb = a.qbar + (size_t)stream * D;
      if (stream != cur_stream) {
        cur_stream = stream;
        float t = 0.f;
        for (int x = lane; x < D; x += 32) t += fabsf((float)qb[x]);
        q_l1 = warp_sum(t);
      }
      if (!cond_wait(BAR_SCORED(p), (unsigned)((it >> 1) & 1), s_abort)) break;
      const float sa = s_s32[p * G + lane], sb = s_s32[p * G + lane + 32];
      float m1, m2;
      int i1;
      if (sb > sa) { m1 = sb; i1 = lane + 32; m2 = sa; } else { m1 = sa; i1 = lane; m2 = sb; }
      float km = fmaxf(s_nrm[p * G + lane], s_nrm[p * G + lane + 32]);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float om1 = __shfl_xor_sync(0xffffffffu, m1, o), om2 = __shfl_xor_sync(0xffffffffu, m2, o);
        const int oi = __shfl_xor_sync(0xffffffffu, i1, o);
        km = fmaxf(km, __shfl_xor_sync(0xffffffffu, km, o));
        m2 = fmaxf(fminf(m1, om1), fmaxf(m2, om2));
        if (om1 > m1 || (om1 == m1 && oi < i1)) { m1 = om1; i1 = oi; }
      }
      const bool exact = exact_all || !(m1 - m2 > MARGIN_FACTOR * q_l1 * km);
      float ea, eb;
      int besti;
      if (exact) {
        if (!cond_wait(BAR_FULL(st), (unsigned)((it / STAGES) & 1), s_abort)) break;
        const unsigned char* t_k = smem + (size_t)st * STAGE_BYTES;
        // fp64 scores token by token: lane l takes columns 4 l .. 4 l + 3; lanes l and l + 32 keep the results
        double qd[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) qd[i] = qb[4 * lane + i];
        double da = 0.0, db = 0.0;
#pragma unroll 1
        for (int i = 0; i < G; ++i) {
          const uint2 v = *reinterpret_cast<const uint2*>(t_k + (size_t)i * (D * 2) + 8 * lane);
          double acc = qd[0] * (double)__uint_as_float(v.x << 16);
          acc = fma(qd[1], (double)__uint_as_float(v.x & 0xffff0000u), acc);
          acc = fma(qd[2], (double)__uint_as_float(v.y << 16), acc);
          acc = fma(qd[3], (double)__uint_as_float(v.y & 0xffff0000u), acc);
          const double c = warp_sum(acc) * a.scale;
          if ((i & 31) == lane) { if (i < 32) da = c; else db = c; }
        }
        double best = da; besti = lane;
        if (db > best) { best = db; besti = lane + 32; }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          const double ob = __shfl_xor_sync(0xffffffffu, best, o);
          const int oi = __shfl_xor_sync(0xffffffffu, besti, o);
          if (ob > best || (ob == best && oi < besti)) { best = ob; besti = oi; }
        }
        ea = expf((float)(da - best)); eb = expf((float)(db - best));
        if (a.scores) {
          double* sc = a.scores + (((size_t)loc.b * a.Hkv + loc.hk) * a.m + loc.j) * G;
          sc[lane] = da; sc[lane + 32] = db;
        }
      } else {
        besti = i1;
        ea = expf((sa - m1) * scale32); eb = expf((sb - m1) * scale32);
      }
      const float inv = 1.f / warp_sum(ea + eb);
      s_a[p * G + lane] = ea * inv; s_a[p * G + lane + 32] = eb * inv;
      if (lane == 0) s_anchor[p] = besti;
      __syncwarp();
      if (lane == 0) cond_arrive(BAR_READY(p));
    }
  } else if (warp == WARP_POOL) {
    // ===================================================== pooling of the values and outputs, one group behind
    for (long long it = 0; it < n_mine; ++it) {
      const int st = (int)(it % STAGES), p = (int)(it & 1);
      const GroupLoc loc = locate_group(a, first + it * stride);
      if (!cond_wait(BAR_READY(p), (unsigned)((it >> 1) & 1), s_abort)) break;
      if (!cond_wait(BAR_FULL(st), (unsigned)((it / STAGES) & 1), s_abort)) break;     // complete long ago
      const unsigned char* t_k = smem + (size_t)st * STAGE_BYTES;
      const uint2* col = reinterpret_cast<const uint2*>(t_k + TILE_BYTES) + lane;      // value columns 4 lane .. 4 lane + 3
      const float* al_base = s_a + p * G;
      unsigned long long acc01 = f32x2(0.f, 0.f), acc23 = f32x2(0.f, 0.f);
#pragma unroll 4
      for (int i = 0; i < G; i += 4) {
        const float4 al = *reinterpret_cast<const float4*>(al_base + i);
        const float alv[4] = {al.x, al.y, al.z, al.w};
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const uint2 w = col[(i + u) * (D / 4)];
          const unsigned long long al2 = f32x2(alv[u], alv[u]);
          acc01 = fma_f32x2(al2, f32x2(__uint_as_float(w.x << 16), __uint_as_float(w.x & 0xffff0000u)), acc01);
          acc23 = fma_f32x2(al2, f32x2(__uint_as_float(w.y << 16), __uint_as_float(w.y & 0xffff0000u)), acc23);
        }
      }
      const size_t orow = (size_t)loc.out_row * a.Hkv + loc.hk;
      {
        float a0, a1, a2, a3;
        asm("mov.b64 {%0, %1}, %2;" : "=f"(a0), "=f"(a1) : "l"(acc01));
        asm("mov.b64 {%0, %1}, %2;" : "=f"(a2), "=f"(a3) : "l"(acc23));
        const bf162 lo = __floats2bfloat162_rn(a0, a1), hi = __floats2bfloat162_rn(a2, a3);
        uint2 o;
        o.x = *reinterpret_cast<const unsigned*>(&lo); o.y = *reinterpret_cast<const unsigned*>(&hi);
        *reinterpret_cast<uint2*>(a.cache_sem + orow * D + 4 * lane) = o;
      }
      const int ia = s_anchor[p];
      reinterpret_cast<uint2*>(a.cache_pos + orow * D)[lane] = reinterpret_cast<const uint2*>(t_k + (size_t)ia * (D * 2))[lane];
      if (lane == 0) a.anchor[(size_t)loc.grp_row * a.Hkv + loc.hk] = loc.j * G + ia;
      __syncwarp();
      if (lane == 0) { cond_arrive(BAR_AFREE(p)); cond_arrive(BAR_FREE(st)); }
    }
  }
  __syncthreads();
  if (tid == 0 && *s_abort) atomicCAS(&g_condense_status, 0, 1);
}

bool make_tensor_map_rows(CUtensorMap* map, const void* ptr, int d, int heads, long long rows, int box_rows);

int condense_take_status() {
  int st = 0;
  if (cudaMemcpyFromSymbol(&st, g_condense_status, sizeof(int)) != cudaSuccess) return -1;
  if (st != 0) { int zero = 0; cudaMemcpyToSymbol(g_condense_status, &zero, sizeof(int)); }
  return st;
}

// ------------------------------------------------------------------------------ local window
// Copies, for every sequence, one contiguous block of `bytes16` 16-byte words.
// Two block copies per sequence in one launch (blockIdx.z: the semantic and the positional part).
struct CopySeg { const uint4* src; uint4* dst; size_t src_batch_stride16, dst_batch_stride16, src_off16, dst_off16, n16, row16; };
// Ragged batch: the segment of sequence blockIdx.y (its last k tokens -> cache rows m .. m + k - 1) follows from the table.
__global__ void copy_blocks_kernel(const CopySeg a, const CopySeg b, SeqTab tab, int g) {
  const CopySeg& c = blockIdx.z == 0 ? a : b;
  size_t src_off = (size_t)blockIdx.y * c.src_batch_stride16 + c.src_off16;
  size_t dst_off = (size_t)blockIdx.y * c.dst_batch_stride16 + c.dst_off16;
  size_t n16 = c.n16;
  if (tab.tok_off) {
    const int s = blockIdx.y;
    const int len = tab.tok_off[s + 1] - tab.tok_off[s], m = tab.grp_off[s + 1] - tab.grp_off[s], k = len - m * g;
    src_off = (size_t)(tab.tok_off[s] + len - k) * c.row16;
    dst_off = (size_t)(tab.cache_off[s] + m) * c.row16;
    n16 = (size_t)k * c.row16;
  }
  const uint4* sp = c.src + src_off;
  uint4* dp = c.dst + dst_off;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n16; i += (size_t)gridDim.x * blockDim.x)
    dp[i] = sp[i];
}

// ------------------------------------------------------------------------------------- host
static int n_summary(const lca_params* p) {
  int n = p->n_summary_q > 0 ? p->n_summary_q : p->group_size;
  return n > p->seq_len ? p->seq_len : n;
}
static int key_dim(const lca_params* p) {
  return (p->variant == LCA_VARIANT_MLA ? p->d_sem : 0) + p->d_pos;
}
// Chunks per CTA of a summary-query launch: one keeps the GPU busy when there are few rows; with many sequences four
// amortise the start-up of a CTA (a CTA of one 64-row chunk reads 74 KB and is gone).
static int qbar_chunks_per_cta(long long total_rows) {
  return total_rows >= 256ll * 1024 ? 4 : 1;
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

static bool condense_fast_shape(const lca_params* p) {
  const bool method = (p->sem_reducer == LCA_REDUCE_DEFAULT || p->sem_reducer == LCA_REDUCE_WEIGHTED) &&
                      (p->pos_reducer == LCA_REDUCE_DEFAULT || p->pos_reducer == LCA_REDUCE_MAXSEL);
  return method && p->variant == LCA_VARIANT_MLA && p->d_sem == 512 && p->d_pos == 64 && p->group_size == 64 && p->n_kv_heads == 1;
}

static bool condense_gqa_fast_shape(const lca_params* p) {
  const bool method = (p->sem_reducer == LCA_REDUCE_DEFAULT || p->sem_reducer == LCA_REDUCE_WEIGHTED) &&
                      (p->pos_reducer == LCA_REDUCE_DEFAULT || p->pos_reducer == LCA_REDUCE_MAXSEL);
  return method && p->variant == LCA_VARIANT_GQA && p->d_sem == 128 && p->d_pos == 128 && p->group_size == 64;
}

size_t condense_smem_bytes(const lca_params* p) {
  if (condense_fast_shape(p)) return fast::SMEM_BYTES;
  if (condense_gqa_fast_shape(p)) return gfast::SMEM_BYTES;
  const size_t g = (size_t)p->group_size;
  const size_t stage = g * (size_t)(p->d_sem + p->d_pos) * sizeof(bf16) + (size_t)key_dim(p) * sizeof(double);
  return 2 * stage + g * (sizeof(double) + sizeof(float));
}

int condense_launch(const CondenseLaunch& c) {
  const lca_params* p = c.p;
  const bool ragged = c.h_tok_off != nullptr;
  int64_t m, k;
  partition(p->seq_len, p->window, p->group_size, &m, &k);       // uniform batch; a ragged one takes them from the table
  const int dk = key_dim(p);
  const int sem_in_logit = p->variant == LCA_VARIANT_MLA;
  const int B = p->batch, Hkv = p->n_kv_heads;
  const long long total_groups = ragged ? (long long)c.h_grp_off[B] : (long long)B * m;      // per KV stream
  double* qbar = reinterpret_cast<double*>(c.ws);
  double* partial = qbar + (size_t)B * Hkv * dk;

  if (total_groups > 0) {
    if (c.qbar_opt) {
      int n = B * Hkv * dk;
      qbar_widen_kernel<<<(n + 255) / 256, 256, 0, c.stream>>>(c.qbar_opt, qbar, n);
      note_launch();
    } else {
      const int n_req = ragged ? (p->n_summary_q > 0 ? p->n_summary_q : p->group_size) : n_summary(p);
      const int rows_q = n_req * (p->n_q_heads / Hkv);
      const int cpc = qbar_chunks_per_cta((long long)rows_q * Hkv * B);
      const int nch = (rows_q + QBAR_ROWS_PER_CHUNK - 1) / QBAR_ROWS_PER_CHUNK;
      dim3 grid((nch + cpc - 1) / cpc, Hkv, B);
      const int pieces = dk / 8;
      const int row_lanes = qbar_row_lanes(pieces);
      const int threads = ((pieces * row_lanes + 31) / 32) * 32;
      const int n = n_req;
      qbar_partial_kernel<<<grid, threads, (size_t)2 * row_lanes * dk * sizeof(double), c.stream>>>(
          (const bf16*)c.q_tail_sem, (const bf16*)c.q_tail_pos, c.q_tail_batch_stride, n,
          p->n_q_heads, Hkv, p->d_sem, p->d_pos, sem_in_logit, row_lanes, partial, c.tab, nch, cpc);
      double count = (double)n * (double)(p->n_q_heads / Hkv);
      qbar_final_kernel<<<dim3(Hkv, B), dk < 1024 ? ((dk + 31) / 32) * 32 : 1024, 0, c.stream>>>(partial, nch, dk, count, qbar, c.tab, n,
                                                                                              p->n_q_heads / Hkv);
      note_launch(2);
    }
    CondenseArgs a;
    a.kv_sem = (const bf16*)c.kv_sem; a.kv_pos = (const bf16*)c.kv_pos; a.qbar = qbar;
    a.cache_sem = (bf16*)c.cache_sem; a.cache_pos = (bf16*)c.cache_pos;
    a.anchor = c.anchor_idx; a.scores = c.scores_opt;
    a.L = p->seq_len; a.Hkv = Hkv; a.d_sem = p->d_sem; a.d_pos = p->d_pos; a.g = p->group_size;
    a.m = (int)m; a.cache_rows = (int)(m + k); a.sem_in_logit = sem_in_logit;
    a.scale = (double)p->softmax_scale;
    a.n_groups = total_groups * Hkv;
    a.tab = c.tab;
    a.sem_reducer = p->sem_reducer == LCA_REDUCE_DEFAULT ? LCA_REDUCE_WEIGHTED : p->sem_reducer;
    a.pos_reducer = p->pos_reducer == LCA_REDUCE_DEFAULT ? LCA_REDUCE_MAXSEL : p->pos_reducer;
    int dev = 0, sms = 148;
    if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    const long long ctas = a.n_groups < sms ? a.n_groups : sms;
    if (condense_fast_shape(p)) {
      if (cudaFuncSetAttribute(condense_mla64_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, fast::SMEM_BYTES) != cudaSuccess)
        return LCA_ERR_CUDA;
      condense_mla64_kernel<<<dim3((unsigned)ctas), fast::THREADS, fast::SMEM_BYTES, c.stream>>>(a);
    } else if (condense_gqa_fast_shape(p)) {
      GqaCondenseMaps maps;
      const long long rows = ragged ? (long long)c.h_tok_off[B] : (long long)B * p->seq_len;
      if (!make_tensor_map_rows(&maps.k, c.kv_pos, 128, Hkv, rows, gfast::G) ||
          !make_tensor_map_rows(&maps.v, c.kv_sem, 128, Hkv, rows, gfast::G))
        return LCA_ERR_CUDA;
      if (cudaFuncSetAttribute(condense_gqa64_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, gfast::SMEM_BYTES) != cudaSuccess)
        return LCA_ERR_CUDA;
      // a grid that is a multiple of the KV heads: every CTA then stays with one head (its summary query stays in registers)
      const long long ctas_h = ctas >= Hkv ? ctas / Hkv * Hkv : ctas;
      condense_gqa64_kernel<<<dim3((unsigned)ctas_h), gfast::THREADS, gfast::SMEM_BYTES, c.stream>>>(a, maps);
    } else {
      size_t smem = condense_smem_bytes(p);
      if (cudaFuncSetAttribute(condense_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
        return LCA_ERR_CUDA;
      // as many resident CTAs per SM as shared memory and registers allow: a group is little work between
      // block-wide barriers, so several CTAs per SM overlap each other's phases
      int per_sm = 1;
      if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, condense_kernel, CONDENSE_THREADS, smem) != cudaSuccess || per_sm < 1) {
        cudaGetLastError();
        per_sm = 1;
      }
      const long long resident = (long long)sms * per_sm;
      condense_kernel<<<dim3((unsigned)(a.n_groups < resident ? a.n_groups : resident)), CONDENSE_THREADS, smem, c.stream>>>(a);
    }
    note_launch();
  }
  if (ragged || k > 0) {
    // the last k tokens of each sequence -> cache rows m..m+k-1 (one contiguous block per sequence)
    const size_t row_sem = (size_t)Hkv * p->d_sem * sizeof(bf16) / 16;
    const size_t row_pos = (size_t)Hkv * p->d_pos * sizeof(bf16) / 16;
    const unsigned blocks = B >= 148 ? 8 : 148 * 2;
    const CopySeg sem = {(const uint4*)c.kv_sem, (uint4*)c.cache_sem, (size_t)p->seq_len * row_sem, (size_t)(m + k) * row_sem,
                         (size_t)(p->seq_len - k) * row_sem, (size_t)m * row_sem, (size_t)k * row_sem, row_sem};
    const CopySeg pos = {(const uint4*)c.kv_pos, (uint4*)c.cache_pos, (size_t)p->seq_len * row_pos, (size_t)(m + k) * row_pos,
                         (size_t)(p->seq_len - k) * row_pos, (size_t)m * row_pos, (size_t)k * row_pos, row_pos};
    copy_blocks_kernel<<<dim3(blocks, B, 2), 256, 0, c.stream>>>(sem, pos, c.tab, p->group_size);
    note_launch();
  }
  return cudaGetLastError() == cudaSuccess ? LCA_OK : LCA_ERR_CUDA;
}

// ------------------------------------------------------------------ online cache update (decode)
// Sec. 4.3 "Decoding and Online Cache Update": when the buffer of uncondensed tokens of a sequence
// has grown to window + g rows, its earliest g tokens become one representative (Eq. 6-8 with the
// summary query of the last g queries), stored right after the existing representatives, and the
// remaining tokens move up by g - 1 rows, so the cache keeps the layout [representatives ; tokens].
// Ring layout (n_tok != nullptr): the uncondensed tokens live in a ring of R = w + g rows (token n at row n % R), the
// representatives from row R on; the new representative goes to row R + n_rep and nothing else moves.
struct UpdateArgs {
  bf16* cache_sem; bf16* cache_pos; const double* qbar;
  int32_t* n_rep; int32_t* n_rows; const int32_t* n_tok; int32_t* anchor_out;
  int cap, Hkv, d_sem, d_pos, g, w, sem_in_logit;
  double scale;
  int32_t* qcount;             // streaming summary query: positions summed so far per sequence (null otherwise)
};
// Does sequence b condense a group now, and where: first row of the group, row of the new representative.
__device__ __forceinline__ bool update_due(const UpdateArgs& a, int b, int& group_row, int& rep_row) {
  const int nr = a.n_rep[b];
  if (a.n_tok) {
    const int R = a.w + a.g;
    const long long first = (long long)nr * a.g;
    if (nr < 0 || (long long)a.n_tok[b] - first < R || R + nr >= a.cap) return false;
    group_row = (int)(first % R); rep_row = R + nr;
    return true;
  }
  if (a.n_rows[b] - nr < a.w + a.g || nr + a.g > a.cap) return false;
  group_row = nr; rep_row = nr;
  return true;
}

// grid (Hkv, B), 256 threads: condense rows n_rep .. n_rep + g - 1 of one KV stream.  Same
// arithmetic as the condense kernels: fp64 scores, arg-max on them, fp32 softmax and pooling.
__device__ __forceinline__ void update_condense_body(const UpdateArgs& a, unsigned char* smem_raw) {
  const int hk = blockIdx.x, b = blockIdx.y;
  const int g = a.g, d_sem = a.d_sem, d_pos = a.d_pos;
  int group_row, rep_row;
  if (!update_due(a, b, group_row, rep_row)) {           // nothing to condense yet
    if (threadIdx.x == 0) a.anchor_out[b * a.Hkv + hk] = -1;
    return;
  }
  const int dk = (a.sem_in_logit ? d_sem : 0) + d_pos;
  bf16* t_sem = reinterpret_cast<bf16*>(smem_raw);
  bf16* t_pos = t_sem + (size_t)g * d_sem;
  double* s_q = reinterpret_cast<double*>(t_pos + (size_t)g * d_pos);
  double* s_s = s_q + dk;
  float* s_a = reinterpret_cast<float*>(s_s + g);
  __shared__ int s_anchor;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarps = blockDim.x >> 5;
  const size_t row0 = (size_t)b * a.cap + group_row, rowr = (size_t)b * a.cap + rep_row;
  const size_t rs_sem = (size_t)a.Hkv * d_sem, rs_pos = (size_t)a.Hkv * d_pos;
  const bf16* gs = a.cache_sem + row0 * rs_sem + (size_t)hk * d_sem;
  const bf16* gp = a.cache_pos + row0 * rs_pos + (size_t)hk * d_pos;
  bf16* out_sem = a.cache_sem + rowr * rs_sem + (size_t)hk * d_sem;     // packed layout: the group's first row
  bf16* out_pos = a.cache_pos + rowr * rs_pos + (size_t)hk * d_pos;
  const int cps = d_sem / 8, cpp = d_pos / 8;
  for (int x = tid; x < g * cps; x += blockDim.x) {
    const int i = x / cps, c = x % cps;
    reinterpret_cast<uint4*>(t_sem + (size_t)i * d_sem)[c] = reinterpret_cast<const uint4*>(gs + (size_t)i * rs_sem)[c];
  }
  for (int x = tid; x < g * cpp; x += blockDim.x) {
    const int i = x / cpp, c = x % cpp;
    reinterpret_cast<uint4*>(t_pos + (size_t)i * d_pos)[c] = reinterpret_cast<const uint4*>(gp + (size_t)i * rs_pos)[c];
  }
  const double* qb = a.qbar + ((size_t)b * a.Hkv + hk) * dk;
  for (int c = tid; c < dk; c += blockDim.x) s_q[c] = qb[c];
  __syncthreads();
  const int sem_off = a.sem_in_logit ? d_sem : 0;
  for (int i = warp; i < g; i += nwarps) {
    double acc = 0.0;
    if (a.sem_in_logit)
      for (int c = lane; c < d_sem; c += 32) acc = fma(s_q[c], (double)__bfloat162float(t_sem[(size_t)i * d_sem + c]), acc);
    for (int c = lane; c < d_pos; c += 32) acc = fma(s_q[sem_off + c], (double)__bfloat162float(t_pos[(size_t)i * d_pos + c]), acc);
    acc = warp_sum(acc);
    if (lane == 0) s_s[i] = acc * a.scale;
  }
  __syncthreads();
  if (warp == 0) {
    double best = -INFINITY;
    int besti = 0x7fffffff;
    for (int i = lane; i < g; i += 32) { const double v = s_s[i]; if (v > best) { best = v; besti = i; } }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const double ob = __shfl_xor_sync(0xffffffffu, best, o);
      const int oi = __shfl_xor_sync(0xffffffffu, besti, o);
      if (ob > best || (ob == best && oi < besti)) { best = ob; besti = oi; }
    }
    float z = 0.f;
    for (int i = lane; i < g; i += 32) { const float e = expf((float)(s_s[i] - best)); s_a[i] = e; z += e; }
    z = warp_sum(z);
    const float inv = 1.f / z;
    for (int i = lane; i < g; i += 32) s_a[i] *= inv;
    if (lane == 0) s_anchor = besti;
  }
  __syncthreads();
  for (int c = tid; c < d_sem; c += blockDim.x) {
    float acc = 0.f;
    for (int i = 0; i < g; ++i) acc = fmaf(s_a[i], __bfloat162float(t_sem[(size_t)i * d_sem + c]), acc);
    out_sem[c] = __float2bfloat16_rn(acc);               // the new representative
  }
  const int ia = s_anchor;
  for (int c = tid; c < d_pos; c += blockDim.x) out_pos[c] = t_pos[(size_t)ia * d_pos + c];
  if (tid == 0) a.anchor_out[b * a.Hkv + hk] = ia;
}
__global__ void __launch_bounds__(256) update_condense_kernel(UpdateArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  update_condense_body(a, smem_raw);
}

// grid (B), 1024 threads: move rows [n_rep + g, n_rows) up to [n_rep + 1, ...) and update the
// counters.  Source and destination overlap (destination below source), so the rows are moved in
// ascending chunks that are loaded completely before any of their bytes is stored.
__global__ void __launch_bounds__(1024) update_shift_kernel(UpdateArgs a) {
  const int b = blockIdx.x;
  int group_row, rep_row;
  if (!update_due(a, b, group_row, rep_row)) return;
  const int nr = a.n_rep[b];
  if (a.n_tok) {                                           // ring layout: only the counters change
    if (threadIdx.x == 0) {
      a.n_rep[b] = nr + 1;
      if (a.qcount) a.qcount[b] = 0;                       // its running query sum has been used and cleared
    }
    return;
  }
  const int rows = a.n_rows[b];
  const int n_move = rows - (nr + a.g);
  for (int pass = 0; pass < 2; ++pass) {
    const size_t row16 = (size_t)a.Hkv * (pass ? a.d_pos : a.d_sem) * sizeof(bf16) / 16;
    uint4* base = reinterpret_cast<uint4*>(pass ? a.cache_pos : a.cache_sem) + (size_t)b * a.cap * row16;
    const uint4* src = base + (size_t)(nr + a.g) * row16;
    uint4* dst = base + (size_t)(nr + 1) * row16;
    const size_t n16 = (size_t)n_move * row16;
    if (a.g > 1)
      for (size_t c0 = 0; c0 < n16; c0 += 4 * 1024) {
        uint4 v[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) { const size_t i = c0 + u * 1024 + threadIdx.x; if (i < n16) v[u] = src[i]; }
        __syncthreads();
#pragma unroll
        for (int u = 0; u < 4; ++u) { const size_t i = c0 + u * 1024 + threadIdx.x; if (i < n16) dst[i] = v[u]; }
        __syncthreads();
      }
  }
  if (threadIdx.x == 0) { a.n_rep[b] = nr + 1; a.n_rows[b] = rows - (a.g - 1); }
}

size_t update_workspace_bytes(const lca_params* p) {
  const int n = p->n_summary_q > 0 ? p->n_summary_q : p->group_size;
  const int rows = n * (p->n_q_heads / p->n_kv_heads);
  const size_t chunks = (size_t)(rows + QBAR_ROWS_PER_CHUNK - 1) / QBAR_ROWS_PER_CHUNK;
  return (size_t)p->batch * p->n_kv_heads * key_dim(p) * (1 + chunks) * sizeof(double);
}

size_t update_smem_bytes(const lca_params* p) {
  const size_t g = (size_t)p->group_size;
  return g * (size_t)(p->d_sem + p->d_pos) * sizeof(bf16) + (size_t)key_dim(p) * sizeof(double) + g * (sizeof(double) + sizeof(float));
}

int update_launch(const lca_params* p, const void* q_tail_sem, const void* q_tail_pos, int64_t q_tail_batch_stride,
                  const float* qbar_opt, void* cache_sem, void* cache_pos, int cap, int32_t* n_rep, int32_t* n_rows,
                  const int32_t* n_tok, int32_t* anchor_out, void* ws, cudaStream_t stream) {
  const int dk = key_dim(p), B = p->batch, Hkv = p->n_kv_heads;
  const int sem_in_logit = p->variant == LCA_VARIANT_MLA;
  double* qbar = reinterpret_cast<double*>(ws);
  double* partial = qbar + (size_t)B * Hkv * dk;
  if (qbar_opt) {
    const int n = B * Hkv * dk;
    qbar_widen_kernel<<<(n + 255) / 256, 256, 0, stream>>>(qbar_opt, qbar, n);
    note_launch();
  } else {
    const int n = p->n_summary_q > 0 ? p->n_summary_q : p->group_size;
    const int rows = n * (p->n_q_heads / Hkv);
    const int cpc = qbar_chunks_per_cta((long long)rows * Hkv * B);
    const int nch = (rows + QBAR_ROWS_PER_CHUNK - 1) / QBAR_ROWS_PER_CHUNK;
    const int pieces = dk / 8;
    const int row_lanes = qbar_row_lanes(pieces);
    const int threads = ((pieces * row_lanes + 31) / 32) * 32;
    qbar_partial_kernel<<<dim3((nch + cpc - 1) / cpc, Hkv, B), threads, (size_t)2 * row_lanes * dk * sizeof(double), stream>>>(
        (const bf16*)q_tail_sem, (const bf16*)q_tail_pos, q_tail_batch_stride, n, p->n_q_heads, Hkv, p->d_sem, p->d_pos,
        sem_in_logit, row_lanes, partial, SeqTab{}, nch, cpc);
    qbar_final_kernel<<<dim3(Hkv, B), dk < 1024 ? ((dk + 31) / 32) * 32 : 1024, 0, stream>>>(
        partial, nch, dk, (double)n * (double)(p->n_q_heads / Hkv), qbar, SeqTab{}, n, p->n_q_heads / Hkv);
    note_launch(2);
  }
  UpdateArgs a;
  a.cache_sem = (bf16*)cache_sem; a.cache_pos = (bf16*)cache_pos; a.qbar = qbar;
  a.n_rep = n_rep; a.n_rows = n_rows; a.n_tok = n_tok; a.anchor_out = anchor_out; a.qcount = nullptr;
  a.cap = cap; a.Hkv = Hkv; a.d_sem = p->d_sem; a.d_pos = p->d_pos; a.g = p->group_size; a.w = p->window;
  a.sem_in_logit = sem_in_logit; a.scale = (double)p->softmax_scale;
  const size_t smem = update_smem_bytes(p);
  if (cudaFuncSetAttribute(update_condense_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return LCA_ERR_CUDA;
  update_condense_kernel<<<dim3(Hkv, B), 256, smem, stream>>>(a);
  update_shift_kernel<<<dim3(B), n_tok ? 32 : 1024, 0, stream>>>(a);
  note_launch(2);
  return cudaGetLastError() == cudaSuccess ? LCA_OK : LCA_ERR_CUDA;
}

// Streaming summary query (ring layout, one call per decode step), fused with the condensation of the sequences that
// are due.  grid (Hkv, B), 256 threads.  First qsum[b, hk, :] += sum over the query heads of KV head hk of this step's
// [q_sem | q_pos] (fp64: sums of bf16 values are exact as long as their exponents span less than 2^30): a thread owns one
// 16-byte piece of the key dimension and every eighth head, eight loads in flight, the eight head lanes are added through
// shared memory in a fixed order.  A sequence that is not due keeps the sum and counts the position.  A sequence that is
// due takes the mean over everything summed since its previous update as its summary query, clears the sum and runs the
// condensation of its earliest group in the same CTA; its counters are advanced by that CTA when there is one KV head
// (the CTA is then the only one that reads them), by update_shift_kernel afterwards otherwise.
static const int QSUM_HEAD_LANES = 8;
static const int RING_STEP_THREADS = 576;
__global__ void __launch_bounds__(RING_STEP_THREADS) ring_step_kernel(const bf16* __restrict__ q_sem, const bf16* __restrict__ q_pos, int Hq,
                                                        double* __restrict__ qsum, double* __restrict__ qbar, UpdateArgs a) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  const int hk = blockIdx.x, b = blockIdx.y;
  const int rep = Hq / a.Hkv;
  const int sem_cols = a.sem_in_logit ? a.d_sem : 0, dk = sem_cols + a.d_pos;
  const int pieces = dk / 8, sem_pieces = sem_cols / 8;
  int group_row, rep_row;
  const bool due = update_due(a, b, group_row, rep_row);
  const int n = a.qcount[b] + 1;                           // only used when due, and then no CTA of this launch writes qcount[b]
  double* s_part = reinterpret_cast<double*>(smem_raw);    // [QSUM_HEAD_LANES][dk]
  for (int x = threadIdx.x; x < pieces * QSUM_HEAD_LANES; x += blockDim.x) {
    const int pc = x % pieces, hl = x / pieces;
    double acc[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = 0.0;
    for (int h = hl; h < rep; h += 8 * QSUM_HEAD_LANES) {
      uint4 v[8];
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const int hh = h + u * QSUM_HEAD_LANES;
        v[u] = make_uint4(0u, 0u, 0u, 0u);
        if (hh < rep) {
          const size_t row = (size_t)b * Hq + (size_t)hk * rep + hh;
          const bf16* src = pc < sem_pieces ? q_sem + row * a.d_sem + 8 * pc : q_pos + row * a.d_pos + 8 * (pc - sem_pieces);
          v[u] = *reinterpret_cast<const uint4*>(src);
        }
      }
#pragma unroll
      for (int u = 0; u < 8; ++u) {
        const unsigned w[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          acc[2 * i] += (double)__uint_as_float(w[i] << 16);
          acc[2 * i + 1] += (double)__uint_as_float(w[i] & 0xffff0000u);
        }
      }
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) s_part[(size_t)hl * dk + 8 * pc + i] = acc[i];
  }
  __syncthreads();
  double* acc_g = qsum + ((size_t)b * a.Hkv + hk) * dk;
  double* out = qbar + ((size_t)b * a.Hkv + hk) * dk;
  for (int c = threadIdx.x; c < dk; c += blockDim.x) {
    double sum = acc_g[c];
    for (int l = 0; l < QSUM_HEAD_LANES; ++l) sum += s_part[(size_t)l * dk + c];
    if (due) { out[c] = sum / ((double)n * (double)rep); acc_g[c] = 0.0; }
    else acc_g[c] = sum;
  }
  if (!due) {
    if (hk == 0 && threadIdx.x == 0) a.qcount[b] = n;
    if (threadIdx.x == 0) a.anchor_out[b * a.Hkv + hk] = -1;
    return;
  }
  __syncthreads();                                         // the summary query written above is read back by the whole CTA
  update_condense_body(a, smem_raw);
  if (a.Hkv == 1 && threadIdx.x == 0) { a.n_rep[b] += 1; a.qcount[b] = 0; }
}

int update_step_launch(const lca_params* p, const void* q_sem, const void* q_pos, double* qsum, int32_t* qcount,
                       void* ring_sem, void* ring_pos, int cap, int32_t* n_rep, const int32_t* n_tok,
                       int32_t* anchor_out, void* ws, cudaStream_t stream) {
  const int B = p->batch, Hkv = p->n_kv_heads;
  UpdateArgs a;
  a.cache_sem = (bf16*)ring_sem; a.cache_pos = (bf16*)ring_pos; a.qbar = reinterpret_cast<double*>(ws);
  a.n_rep = n_rep; a.n_rows = nullptr; a.n_tok = n_tok; a.anchor_out = anchor_out;
  a.cap = cap; a.Hkv = Hkv; a.d_sem = p->d_sem; a.d_pos = p->d_pos; a.g = p->group_size; a.w = p->window;
  a.sem_in_logit = p->variant == LCA_VARIANT_MLA; a.scale = (double)p->softmax_scale;
  a.qcount = qcount;
  size_t smem = update_smem_bytes(p);
  const size_t part = (size_t)QSUM_HEAD_LANES * key_dim(p) * sizeof(double);
  if (smem < part) smem = part;
  if (cudaFuncSetAttribute(ring_step_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return LCA_ERR_CUDA;
  ring_step_kernel<<<dim3(Hkv, B), RING_STEP_THREADS, smem, stream>>>((const bf16*)q_sem, (const bf16*)q_pos, p->n_q_heads, qsum,
                                                                      reinterpret_cast<double*>(ws), a);
  note_launch();
  if (Hkv > 1) {
    update_shift_kernel<<<dim3(B), 32, 0, stream>>>(a);
    note_launch();
  }
  return cudaGetLastError() == cudaSuccess ? LCA_OK : LCA_ERR_CUDA;
}

// Packed cache [representatives ; tokens in order] -> ring layout (see UpdateArgs): the step between the prefill
// condensation and decoding on the ring.  grid (chunks, B, 2): z = 0 the semantic part, 1 the positional part.
struct RingCopyArgs {
  const uint4* src[2]; uint4* dst[2]; size_t row16[2];      // 16-byte pieces per row
  const int32_t* packed_rows; const int32_t* n_rep; int32_t* n_tok_out;
  int packed_cap, ring_cap, R, g;
};
__global__ void __launch_bounds__(256) ring_from_packed_kernel(RingCopyArgs a) {
  const int b = blockIdx.y, z = blockIdx.z;
  const int rows = min(max(a.packed_rows[b], 0), a.packed_cap);
  const int nr = min(max(a.n_rep[b], 0), rows);
  const int n_tok_rows = min(rows - nr, a.R);               // tokens beyond the ring's size cannot be placed
  const int n_rep_rows = min(nr, max(a.ring_cap - a.R, 0));
  const long long first = (long long)nr * a.g;
  const size_t row16 = a.row16[z];
  const uint4* src = a.src[z] + (size_t)b * a.packed_cap * row16;
  uint4* dst = a.dst[z] + (size_t)b * a.ring_cap * row16;
  const size_t n16 = (size_t)(n_rep_rows + n_tok_rows) * row16;
  for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < n16; i += (size_t)gridDim.x * blockDim.x) {
    const int r = (int)(i / row16);
    const size_t piece = i % row16;
    int srow, drow;
    if (r < n_rep_rows) { srow = r; drow = a.R + r; }
    else { const int t = r - n_rep_rows; srow = nr + t; drow = (int)((first + t) % a.R); }
    dst[(size_t)drow * row16 + piece] = src[(size_t)srow * row16 + piece];
  }
  if (z == 0 && blockIdx.x == 0 && threadIdx.x == 0) a.n_tok_out[b] = (int32_t)(first + (rows - nr));
}

int ring_from_packed_launch(const lca_params* p, const void* packed_sem, const void* packed_pos, const int32_t* packed_rows,
                            const int32_t* n_rep, int packed_cap, void* ring_sem, void* ring_pos, int ring_cap,
                            int32_t* n_tok_out, cudaStream_t stream) {
  RingCopyArgs a;
  a.src[0] = (const uint4*)packed_sem; a.src[1] = (const uint4*)packed_pos;
  a.dst[0] = (uint4*)ring_sem; a.dst[1] = (uint4*)ring_pos;
  a.row16[0] = (size_t)p->n_kv_heads * p->d_sem * sizeof(bf16) / 16;
  a.row16[1] = (size_t)p->n_kv_heads * p->d_pos * sizeof(bf16) / 16;
  a.packed_rows = packed_rows; a.n_rep = n_rep; a.n_tok_out = n_tok_out;
  a.packed_cap = packed_cap; a.ring_cap = ring_cap; a.R = p->window + p->group_size; a.g = p->group_size;
  const unsigned chunks = p->batch >= 148 ? 4 : (unsigned)((148 * 4 + p->batch - 1) / p->batch);
  ring_from_packed_kernel<<<dim3(chunks, p->batch, 2), 256, 0, stream>>>(a);
  note_launch();
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
