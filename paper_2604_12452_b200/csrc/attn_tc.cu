// Tensor-core attention over the condensed context for grouped-query heads of dimension 128, one 128-row query tile
// per CTA: TMA-staged 128-byte-swizzled tiles, tcgen05.mma with accumulators in tensor memory, online softmax in
// fp32.  The library uses this kernel for GQA DECODE (Sec. 4.3, 5.4: one query token per sequence, so a CTA's tile
// holds the query heads of one KV head); GQA prefill runs on attn_gqa2_kernel (two query tiles per CTA), the MLA shape
// on attn_tc2_kernel (CTA pairs).  The tile walk below still covers the prefill case (representatives, then local
// tokens) because it is the same code; this file also holds the tensor-map helpers and the dispatch of all three.
//
// One CTA owns a tile of 128 query rows = TB consecutive tokens x HB heads that share one
// key/value stream.  It walks the rows of the condensed cache (prefill: the representatives any of
// its tokens may see, then the local tokens) in tiles of BN keys:
//     S  = Q K^T        (tcgen05.mma, A = Q and B = K tile from shared memory, D in TMEM)
//     P  = exp2(S*c - m) with per-row masks only on boundary tiles (two softmax threads per row,
//          S read from TMEM, P written back to TMEM as packed bf16)
//     O += P V          (tcgen05.mma, A = P from TMEM, B = V tile from shared memory)
// Roles: warp 0 issues TMA loads, warp 1 owns TMEM and issues every MMA, warps 2..9 do the
// softmax, the (rare) rescale of O when the running maximum grows by more than 2^8, and the
// epilogue.  Every wait is bounded; on expiry the CTA records a code in a global status word,
// drains and returns.
#include <cstring>

#include "lca_common.cuh"
#include "tc_common.cuh"

namespace lca {
using namespace tc;

static __device__ int g_tc_status = 0;

static constexpr int ROWS = 128;          // query rows per CTA (TMEM lanes)
static constexpr int BN = 128;            // keys per tile
static constexpr int CHUNK_BYTES_Q = ROWS * 128;   // one 64-column chunk of the query tile
static constexpr int CHUNK_BYTES_KV = BN * 128;    // one 64-column chunk of a key/value tile
static constexpr float RESCALE_THRESHOLD = 8.0f;   // log2 units

struct TcParams {
  CUtensorMap q_sem, q_pos, kv_sem, kv_pos, cache_sem, cache_pos;   // 3-D {d, heads, rows}
  bf16* out; float* lse;
  DecodeLayout dl;                // decode: which rows of a sequence's cache take part (packed or ring layout)
  int B, q_len, Hq, Hkv, L, g, w, cap, decode;
  int HB, TB, n_tok_tiles, d_out;
  int out_wide;                   // out is 32-byte aligned: 256-bit stores
  float scale_log2, bias_log2;
};

// Shared-memory plan of the 1-CTA kernel.  NK_SEM / NK_POS: 64-column key chunks taken from the
// sem / pos tensors; NV: value chunks (taken from the sem tensor).  When V_IN_K the value chunks
// are the first NV key chunks of the same tile (MLA: values are the latents), else they are
// loaded separately (GQA).
template <int NK_SEM, int NK_POS, int NV, bool V_IN_K, int STAGES>
struct Plan1 {
  static constexpr int NK = NK_SEM + NK_POS;
  static constexpr int Q_BYTES = NK * CHUNK_BYTES_Q;
  static constexpr int K_STAGE = NK * CHUNK_BYTES_KV;
  static constexpr int V_STAGE = V_IN_K ? 0 : NV * CHUNK_BYTES_KV;
  static constexpr int OFF_Q = 0;
  static constexpr int OFF_K = OFF_Q + Q_BYTES;
  static constexpr int OFF_V = OFF_K + STAGES * K_STAGE;
  static constexpr int OFF_BAR = OFF_V + STAGES * V_STAGE;
  static constexpr int NBAR = 1 + 4 * STAGES + 2 + 2 + 1;
  static constexpr int OFF_MISC = OFF_BAR + NBAR * 8;
  static constexpr int OFF_RED = OFF_MISC + 16;          // float [3][2][128]: row maxima (two tiles in flight) and row sums
  static constexpr int BYTES = OFF_RED + 6 * 128 * 4 + 1024;     // + slack to align the base to 1024 B
  // tensor memory columns
  static constexpr int TM_S0 = 0, TM_S1 = BN, TM_O = 2 * BN;
  static constexpr int TM_COLS = 512;
  static_assert(2 * BN + NV * 64 <= 512, "TMEM budget");
};

constexpr int POLY_OF_4 = 1;   // exponentials out of every four that go to the FMA pipe (interior tiles)

template <int NK_SEM, int NK_POS, int NV, bool V_IN_K, int STAGES>
__global__ void __launch_bounds__(320, 1)
attn_tc1_kernel(const __grid_constant__ TcParams p) {
  using P = Plan1<NK_SEM, NK_POS, NV, V_IN_K, STAGES>;
  constexpr int NK = P::NK;
  extern __shared__ unsigned char smem_dyn[];
  const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  unsigned char* base_ptr = smem_dyn + (base - smem_u32(smem_dyn));
  const uint32_t sQ = base + P::OFF_Q, sK = base + P::OFF_K, sV = base + P::OFF_V;
  const uint32_t bars = base + P::OFF_BAR;
  auto BAR_Q = [&]() { return bars; };
  auto BAR_KFULL = [&](int s) { return bars + 8 * (1 + s); };
  auto BAR_KEMPTY = [&](int s) { return bars + 8 * (1 + STAGES + s); };
  auto BAR_VFULL = [&](int s) { return bars + 8 * (1 + 2 * STAGES + s); };
  auto BAR_VEMPTY = [&](int s) { return bars + 8 * (1 + 3 * STAGES + s); };
  auto BAR_SFULL = [&](int i) { return bars + 8 * (1 + 4 * STAGES + i); };
  auto BAR_PFULL = [&](int i) { return bars + 8 * (3 + 4 * STAGES + i); };
  const uint32_t BAR_ODONE = bars + 8 * (5 + 4 * STAGES);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + P::OFF_MISC);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + P::OFF_MISC + 4);

  // the warp index through a shuffle: provably warp-uniform, so the role branches below are uniform branches
  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;

  // ---- which rows, which key tiles
  const int tile = p.n_tok_tiles - 1 - (int)blockIdx.x;      // heaviest (latest) query tiles first
  const int hb = blockIdx.y, b = blockIdx.z;
  const int t0 = tile * p.TB;
  const int t1 = min(t0 + p.TB, p.q_len) - 1;
  const int head0 = hb * p.HB;
  const int hk = (p.Hkv == 1) ? 0 : hb;
  int nA, nB, first_lo, n_a_lo, n_a_hi;
  if (p.decode) {
    n_a_hi = n_a_lo = decode_span(p.dl, b).rows_end;
    first_lo = 0; nB = 0;
  } else {
    n_a_lo = reps_visible(t0, p.w, p.g);
    n_a_hi = reps_visible(t1, p.w, p.g);
    first_lo = n_a_lo * p.g;
    nB = (t1 - first_lo + BN) / BN;
  }
  nA = (n_a_hi + BN - 1) / BN;
  const int n_tiles = nA + nB;

  if (threadIdx.x == 0) {
    mbar_init(BAR_Q(), 1);
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(BAR_KFULL(s), 1); mbar_init(BAR_KEMPTY(s), 1);
      mbar_init(BAR_VFULL(s), 1); mbar_init(BAR_VEMPTY(s), 1);
    }
    for (int i = 0; i < 2; ++i) { mbar_init(BAR_SFULL(i), 1); mbar_init(BAR_PFULL(i), 256); }
    mbar_init(BAR_ODONE, 1);
    *abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 1) {                    // TMEM: allocated and freed by the same warp
    tmem_alloc(smem_u32((const void*)tmem_slot), P::TM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  auto fail = [&](int code) {
    atomicCAS(&g_tc_status, 0, code);
    *abort_flag = 1;
  };

  if (warp == 0) {
    // =============================================================== TMA producer
    if (lane == 0 && n_tiles > 0) {
      prefetch_tmap(&p.q_pos); prefetch_tmap(&p.kv_pos); prefetch_tmap(&p.kv_sem);
      mbar_expect_tx(BAR_Q(), P::Q_BYTES);
      const int qrow = b * p.q_len + t0;
      for (int c = 0; c < NK_SEM; ++c) tma_load_3d(sQ + c * CHUNK_BYTES_Q, &p.q_sem, c * 64, head0, qrow, BAR_Q());
      for (int c = 0; c < NK_POS; ++c) tma_load_3d(sQ + (NK_SEM + c) * CHUNK_BYTES_Q, &p.q_pos, c * 64, head0, qrow, BAR_Q());
      for (int j = 0; j < n_tiles; ++j) {
        const int s = j % STAGES, round = j / STAGES;
        const bool isA = j < nA;
        const int row = isA ? b * p.cap + j * BN : b * p.L + first_lo + (j - nA) * BN;
        const CUtensorMap* msem = isA ? &p.cache_sem : &p.kv_sem;
        const CUtensorMap* mpos = isA ? &p.cache_pos : &p.kv_pos;
        if (!mbar_wait(BAR_KEMPTY(s), (round & 1) ^ 1, abort_flag)) { fail(ERR_WAIT_KV_EMPTY); break; }
        mbar_expect_tx(BAR_KFULL(s), P::K_STAGE);
        for (int c = 0; c < NK_SEM; ++c) tma_load_3d(sK + s * P::K_STAGE + c * CHUNK_BYTES_KV, msem, c * 64, hk, row, BAR_KFULL(s));
        for (int c = 0; c < NK_POS; ++c) tma_load_3d(sK + s * P::K_STAGE + (NK_SEM + c) * CHUNK_BYTES_KV, mpos, c * 64, hk, row, BAR_KFULL(s));
        if (!V_IN_K) {
          if (!mbar_wait(BAR_VEMPTY(s), (round & 1) ^ 1, abort_flag)) { fail(ERR_WAIT_KV_EMPTY); break; }
          mbar_expect_tx(BAR_VFULL(s), P::V_STAGE);
          for (int c = 0; c < NV; ++c) tma_load_3d(sV + s * P::V_STAGE + c * CHUNK_BYTES_KV, msem, c * 64, hk, row, BAR_VFULL(s));
        }
      }
    }
  } else if (warp == 1) {
    // =============================================================== MMA issuer
    // The whole warp walks the loop converged (every lane polls the barriers); one elected lane issues.
    constexpr uint32_t IDESC_S = umma_idesc_bf16(ROWS, BN, false, false);
    constexpr uint32_t IDESC_PV = umma_idesc_bf16(ROWS, NV * 64, false, true);
    const uint32_t leader = elect_one();
    bool ok = n_tiles > 0;
    if (ok) {
      ok = mbar_wait(BAR_Q(), 0, abort_flag);
      if (!ok && leader) fail(ERR_WAIT_Q);
    }
    const uint64_t qd0 = umma_desc_sw128(sQ, 16, 1024);
    auto issue_pv = [&](int j) -> bool {      // O += P_j V_j
      const int s = j % STAGES, round = j / STAGES;
      bool good = mbar_wait(BAR_PFULL(j & 1), (j >> 1) & 1, abort_flag);
      if (good && !V_IN_K) good = mbar_wait(BAR_VFULL(s), round & 1, abort_flag);
      if (!good) { if (leader) fail(ERR_WAIT_P_FULL); return false; }
      const uint32_t vbase = V_IN_K ? sK + s * P::K_STAGE : sV + s * P::V_STAGE;
      // Rows of the cache beyond the valid count (decode, last tile) may hold anything; their
      // probabilities are exactly 0, so zero the value rows to keep 0 * garbage out of O.
      if (p.decode && (j + 1) * BN > n_a_hi) {
        const int first_bad = n_a_hi - j * BN;
        for (int idx = lane; idx < (BN - first_bad) * 8 * NV; idx += 32) {
          const int c = idx / ((BN - first_bad) * 8), rem = idx % ((BN - first_bad) * 8);
          const int r = first_bad + rem / 8, q = rem % 8;
          const uint32_t a = vbase + c * CHUNK_BYTES_KV + r * 128 + q * 16;
          asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(a), "r"(0) : "memory");
        }
        fence_proxy_async_smem();
        __syncwarp();
      }
      tc_fence_after();
      const uint32_t ptm = tmem + ((j & 1) ? P::TM_S1 : P::TM_S0);
      const uint64_t vd0 = umma_desc_sw128(vbase, CHUNK_BYTES_KV, 1024);
#pragma unroll
      for (int k = 0; k < BN / 16; ++k)
        umma_ts_elected(leader, tmem + P::TM_O, ptm + k * 8, desc_add(vd0, (k * 2048) >> 4), IDESC_PV, (j > 0 || k > 0) ? 1u : 0u);
      umma_commit_elected(leader, V_IN_K ? BAR_KEMPTY(s) : BAR_VEMPTY(s));
      umma_commit_elected(leader, BAR_ODONE);
      return true;
    };
    for (int j = 0; ok && j < n_tiles; ++j) {
      const int s = j % STAGES, round = j / STAGES;
      ok = mbar_wait(BAR_KFULL(s), round & 1, abort_flag);
      if (!ok) { if (leader) fail(ERR_WAIT_KV_FULL); break; }
      tc_fence_after();
      const uint32_t stm = tmem + ((j & 1) ? P::TM_S1 : P::TM_S0);
      // descriptors are built once; per instruction only the start address moves
      const uint64_t kd0 = umma_desc_sw128(sK + s * P::K_STAGE, 16, 1024);
#pragma unroll
      for (int c = 0; c < NK; ++c) {
#pragma unroll
        for (int k = 0; k < 4; ++k)
          umma_ss_elected(leader, stm, desc_add(qd0, (c * CHUNK_BYTES_Q + k * 32) >> 4),
                          desc_add(kd0, (c * CHUNK_BYTES_KV + k * 32) >> 4), IDESC_S, (c > 0 || k > 0) ? 1u : 0u);
      }
      umma_commit_elected(leader, BAR_SFULL(j & 1));
      if (!V_IN_K) umma_commit_elected(leader, BAR_KEMPTY(s));
      if (j >= 1) ok = issue_pv(j - 1);
    }
    if (ok && n_tiles > 0) issue_pv(n_tiles - 1);
  } else {
    // =============================================================== softmax / epilogue (256 threads)
    // Two threads per query row: warps 2-5 take keys 0..63 of a tile, warps 6-9 keys 64..127 (a
    // warp may only touch the 32 TMEM lanes of its quarter, warp & 3).  One thread per row was
    // twice as slow as the tensor core at this head size.  The halves combine their row maxima
    // through shared memory; that barrier also orders every read of S before any write of P,
    // which reuses the S columns.
    const int quarter = warp & 3, half = warp >= 6 ? 1 : 0;
    const int r = quarter * 32 + lane;            // query row of this thread
    const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
    const int tl = r / p.HB, hl = r % p.HB;
    const int t_row = t0 + tl;
    const bool row_valid = t_row < p.q_len;
    int n_a_row, first_row;
    // rows [inv_lo, inv_hi) of the cache part do not take part (ring layout); rows [bias_lo, bias_hi) are representatives
    DecodeSpan sp = {};
    if (p.decode) { sp = decode_span(p.dl, b); n_a_row = n_a_hi; first_row = 0; }
    else { n_a_row = reps_visible(min(t_row, p.q_len - 1), p.w, p.g); sp.bias_hi = n_a_row; first_row = n_a_row * p.g; }
    volatile float* red = reinterpret_cast<volatile float*>(base_ptr + P::OFF_RED);          // [3][2][128]
    volatile int* fail_word = reinterpret_cast<volatile int*>(base_ptr + P::OFF_MISC + 8);   // [2]
    if (half == 0 && r < 2) fail_word[r] = 0;
    asm volatile("bar.sync 1, 256;" ::: "memory");
    // All 256 threads execute exactly one named barrier per tile, whatever happens: a thread whose
    // wait expired marks the tile's fail word before the barrier and everybody leaves after it.
    float m_ref = -INFINITY, l_sum = 0.f;
    bool ok = true;
    for (int j = 0; j < n_tiles; ++j) {
      if (ok) {
        ok = mbar_wait(BAR_SFULL(j & 1), (j >> 1) & 1, abort_flag);
        if (!ok && lane == 0) fail(ERR_WAIT_S_FULL);
      }
      ok = __all_sync(0xffffffffu, ok);
      const uint32_t stm = tmem + lane_base + ((j & 1) ? P::TM_S1 : P::TM_S0);
      uint32_t sr[2][32];
      float tmax = -INFINITY;
      bool plain = false;
      const bool isA = j < nA;
      const int key0 = (isA ? j * BN : first_lo + (j - nA) * BN) + 64 * half;   // first key of this thread's columns
      if (ok) {
        tc_fence_after();
        tmem_ld32(stm + 64 * half, sr[0]);
        tmem_ld32(stm + 64 * half + 32, sr[1]);
        tmem_wait_ld();
        const int tile_key0 = key0 - 64 * half;
        bool need_mask;
        int lo, hi;                                  // visible columns of this thread: lo <= c <= hi
        if (isA) { lo = 0; hi = n_a_row - key0 - 1; need_mask = tile_key0 + BN > n_a_lo; }
        else { lo = first_row - key0; hi = t_row - key0; need_mask = (tile_key0 < n_a_hi * p.g) || (tile_key0 + BN - 1 > t0); }
        bool tile_bias = false;
        if (isA) {
          need_mask = need_mask || (tile_key0 < sp.inv_hi && tile_key0 + BN > sp.inv_lo);
          tile_bias = p.bias_log2 != 0.f && tile_key0 < sp.bias_hi && tile_key0 + BN > sp.bias_lo;
        }
        plain = !need_mask && !tile_bias;
        if (plain) {
          // interior tile: the raw products stay in sr, the (positive) scale is applied to the maximum
          // here and folded into the exponent's multiply-add below
          float t0m = -INFINITY, t1m = -INFINITY, t2m = -INFINITY, t3m = -INFINITY;    // four short chains
#pragma unroll
          for (int i = 0; i < 32; i += 2) {
            t0m = fmaxf(t0m, __uint_as_float(sr[0][i])); t1m = fmaxf(t1m, __uint_as_float(sr[0][i + 1]));
            t2m = fmaxf(t2m, __uint_as_float(sr[1][i])); t3m = fmaxf(t3m, __uint_as_float(sr[1][i + 1]));
          }
          tmax = fmaxf(fmaxf(t0m, t1m), fmaxf(t2m, t3m)) * p.scale_log2;
        } else {
          // boundary tile: scale, bias and mask with selects only (per-element branches cost ~25 cycles
          // each here), four short maximum chains
          const float bias = tile_bias ? p.bias_log2 : 0.f;
          const int lo_m = need_mask ? lo : -(1 << 30), hi_m = need_mask ? hi : (1 << 30);
          // columns [blo, blo + bspan) receive the bias, columns [ilo, ilo + ispan) are left out (both empty outside the cache part)
          const int blo = sp.bias_lo - key0, ilo = sp.inv_lo - key0;
          const unsigned bspan = isA ? (unsigned)(sp.bias_hi - sp.bias_lo) : 0u, ispan = isA ? (unsigned)(sp.inv_hi - sp.inv_lo) : 0u;
          float tm[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
          for (int q = 0; q < 2; ++q) {
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              const int c = q * 32 + i;
              float s = fmaf(__uint_as_float(sr[q][i]), p.scale_log2, (unsigned)(c - blo) < bspan ? bias : 0.f);
              s = ((c >= lo_m) & (c <= hi_m) & !((unsigned)(c - ilo) < ispan)) ? s : -INFINITY;
              sr[q][i] = __float_as_uint(s);
              tm[i & 3] = fmaxf(tm[i & 3], s);
            }
          }
          tmax = fmaxf(fmaxf(tm[0], tm[1]), fmaxf(tm[2], tm[3]));
        }
      } else {
        fail_word[j & 1] = 1;
      }
      red[((j & 1) * 2 + half) * 128 + r] = tmax;
      asm volatile("bar.sync 1, 256;" ::: "memory");
      if (fail_word[j & 1]) { ok = false; continue; }          // uniform over the 256 threads
      tmax = fmaxf(tmax, red[((j & 1) * 2 + (half ^ 1)) * 128 + r]);
      // running maximum: rescale O only when it grows by more than the threshold
      bool need = false;
      float factor = 1.f;
      if (j == 0) m_ref = tmax;
      else if (tmax > m_ref + RESCALE_THRESHOLD) { need = true; factor = exp2f(m_ref - tmax); }
      if (__any_sync(0xffffffffu, need)) {
        ok = mbar_wait(BAR_ODONE, (j - 1) & 1, abort_flag);       // P_{j-1} V_{j-1} has landed in O
        if (!ok && lane == 0) fail(ERR_WAIT_O_DONE);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) continue;                                        // reported at the next tile's barrier
        tc_fence_after();
#pragma unroll
        for (int q = NV * half; q < NV * half + NV; ++q) {         // this half's share of the O columns
          uint32_t o[32];
          tmem_ld32(tmem + lane_base + P::TM_O + q * 32, o);
          tmem_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * factor);
          tmem_st32(tmem + lane_base + P::TM_O + q * 32, o);
        }
        if (need) { l_sum *= factor; m_ref = tmax; }
      }
      const float m_use = (m_ref == -INFINITY) ? 0.f : m_ref;
      float rs0 = 0.f, rs1 = 0.f;
      uint32_t pk[32];
      const float e_mul = plain ? p.scale_log2 : 1.f;       // sr holds raw products (plain) or scaled logits
      if (plain) {
        // Interior tile: every logit is finite.  POLY_OF_4 of every four exponentials are evaluated on the
        // FMA pipe, the others on the special-function unit, so that the two pipes share the 16384 per tile.
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const float a0 = fmaf(__uint_as_float(sr[i >> 4][(2 * i) & 31]), e_mul, -m_use);
          const float a1 = fmaf(__uint_as_float(sr[i >> 4][(2 * i + 1) & 31]), e_mul, -m_use);
          const float p0 = ((2 * i) & 3) < POLY_OF_4 ? exp2_fma(a0) : exp2f(a0);
          const float p1 = ((2 * i + 1) & 3) < POLY_OF_4 ? exp2_fma(a1) : exp2f(a1);
          rs0 += p0; rs1 += p1;
          pk[i] = pack_bf16x2(p0, p1);
        }
      } else {
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          const float p0 = exp2f(fmaf(__uint_as_float(sr[i >> 4][(2 * i) & 31]), e_mul, -m_use));
          const float p1 = exp2f(fmaf(__uint_as_float(sr[i >> 4][(2 * i + 1) & 31]), e_mul, -m_use));
          rs0 += p0; rs1 += p1;
          pk[i] = pack_bf16x2(p0, p1);
        }
      }
      l_sum += rs0 + rs1;
      if (j >= 1 && ok) {
        // keep in step with the P V barrier (a parity wait only tells phases apart while the waiter is at most one
        // phase behind): P V of tile j - 1 was issued before this tile's softmax began and is normally complete
        ok = mbar_wait(BAR_ODONE, (j - 1) & 1, abort_flag);
        if (!ok && lane == 0) fail(ERR_WAIT_O_DONE);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) continue;                                        // reported at the next tile's barrier
      }
      tmem_st32(stm + 32 * half, pk);     // P columns 32*half .. 32*half+31 = keys 64*half .. 64*half+63
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(BAR_PFULL(j & 1));
    }
    // ---- epilogue: O / l -> bf16 -> global
    if (ok && n_tiles > 0) {
      ok = mbar_wait(BAR_ODONE, (n_tiles - 1) & 1, abort_flag);
      if (!ok && lane == 0) fail(ERR_WAIT_O_DONE);
    }
    ok = __all_sync(0xffffffffu, ok);
    if (!ok) fail_word[0] = fail_word[1] = 1;
    red[(4 + half) * 128 + r] = l_sum;
    asm volatile("bar.sync 1, 256;" ::: "memory");
    if (!fail_word[0]) {
      const float l_tot = l_sum + red[(4 + (half ^ 1)) * 128 + r];
      tc_fence_after();
      const float inv = (n_tiles > 0 && l_tot > 0.f) ? 1.f / l_tot : 0.f;
      const size_t orow = ((size_t)b * p.q_len + t_row) * p.Hq + head0 + hl;
      bf16* dst = p.out + orow * p.d_out;
#pragma unroll
      for (int q = NV * half; q < NV * half + NV; ++q) {
        uint32_t o[32];
        if (n_tiles > 0) { tmem_ld32(tmem + lane_base + P::TM_O + q * 32, o); tmem_wait_ld(); }
        else {
#pragma unroll
          for (int i = 0; i < 32; ++i) o[i] = 0;
        }
        if (row_valid && hl < p.HB && head0 + hl < p.Hq) {
          // 32 bytes per store: every lane writes whole sectors of its own row
#pragma unroll
          for (int v = 0; v < 2; ++v) {
            uint32_t w[8];
#pragma unroll
            for (int e = 0; e < 8; ++e)
              w[e] = pack_bf16x2(__uint_as_float(o[16 * v + 2 * e]) * inv, __uint_as_float(o[16 * v + 2 * e + 1]) * inv);
            st_global_32B(dst + q * 32 + 16 * v, w, p.out_wide != 0);
          }
        }
      }
      if (p.lse && row_valid && half == 0)
        p.lse[orow] = (n_tiles > 0 && l_tot > 0.f) ? (m_ref + log2f(l_tot)) * 0.6931471805599453f : -INFINITY;
    }
    tc_fence_before();
  }
  // ---- teardown: let straggling bulk copies land if the CTA gave up, then free TMEM
  if (*abort_flag && warp == 0 && lane == 0) {
    const long long t0c = clock64();
    while (clock64() - t0c < 2000000ll) { __nanosleep(1000); }
  }
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, P::TM_COLS);
  }
}

// ----------------------------------------------------------------------------------- host
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* ptr = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ptr, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(ptr);
  }
  return fn;
}

// bf16 tensor [rows, heads, d] (d contiguous) viewed as 3-D {d, heads, rows}; box {64, box_heads, box_rows}
bool make_tensor_map_3d(CUtensorMap* map, const void* ptr, int d, int heads, long long rows, int box_heads, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  if (!ptr) { memset(map, 0, sizeof(*map)); return true; }
  cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)heads, (cuuint64_t)rows};
  cuuint64_t strides[2] = {(cuuint64_t)d * 2, (cuuint64_t)d * 2 * heads};
  cuuint32_t box[3] = {64, (cuuint32_t)box_heads, (cuuint32_t)box_rows};
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// The same tensor with unswizzled boxes of whole rows: box {d, 1, box_rows} lands as a plain [box_rows][d] array
// (the condensation kernels read their tiles with ordinary shared-memory loads).
bool make_tensor_map_rows(CUtensorMap* map, const void* ptr, int d, int heads, long long rows, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn || !ptr) return false;
  cuuint64_t dims[3] = {(cuuint64_t)d, (cuuint64_t)heads, (cuuint64_t)rows};
  cuuint64_t strides[2] = {(cuuint64_t)d * 2, (cuuint64_t)d * 2 * heads};
  cuuint32_t box[3] = {(cuuint32_t)d, 1, (cuuint32_t)box_rows};
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// A [rows][64 * chunks] bf16 matrix seen as (64 columns, rows, 64-column chunks): one box then brings
// several column chunks of the same rows, each landing as its own 128-byte-swizzled [rows][64] block
// (chunk after chunk), in a single request instead of one request per chunk.
bool make_tensor_map_chunks(CUtensorMap* map, const void* ptr, int chunks, long long rows, int box_rows, int box_chunks) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  if (!ptr) { memset(map, 0, sizeof(*map)); return true; }
  cuuint64_t dims[3] = {64, (cuuint64_t)rows, (cuuint64_t)chunks};
  cuuint64_t strides[2] = {(cuuint64_t)chunks * 128, 128};
  cuuint32_t box[3] = {64, (cuuint32_t)box_rows, (cuuint32_t)box_chunks};
  cuuint32_t estr[3] = {1, 1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(ptr), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

static bool gqa128_shape(const AttnProblem& a) {
  if (a.variant != LCA_VARIANT_GQA || a.d_sem != 128 || a.d_pos != 128) return false;
  const int rep = a.n_q_heads / a.n_kv_heads;
  return rep >= 1 && rep <= 128 && 128 % rep == 0;
}

bool attn_tc2_supported(const AttnProblem& a);
int attn_tc2_launch(const AttnProblem& a);
int attn_tc2_take_status();
bool attn_gqa2_supported(const AttnProblem& a);      // prefill of the same shape, two query tiles per CTA
int attn_gqa2_launch(const AttnProblem& a);
int attn_gqa2_take_status();

bool attn_tc_supported(const AttnProblem& a) { return gqa128_shape(a) || attn_tc2_supported(a); }
size_t attn_tc_workspace_bytes(const AttnProblem& a) {
  return (a.decode && attn_tc2_supported(a)) ? attn_tc2_decode_workspace_bytes(a.batch, a.n_q_heads) : 0;
}

int attn_tc_launch(const AttnProblem& a) {
  if (attn_tc2_supported(a)) return attn_tc2_launch(a);
  if (attn_gqa2_supported(a)) return attn_gqa2_launch(a);
  if (!gqa128_shape(a)) return LCA_ERR_UNSUPPORTED_SHAPE;
  TcParams p;
  memset(&p, 0, sizeof(p));
  const int rep = a.n_q_heads / a.n_kv_heads;
  p.HB = rep; p.TB = ROWS / rep;
  p.B = a.batch; p.q_len = a.q_len; p.Hq = a.n_q_heads; p.Hkv = a.n_kv_heads; p.L = a.seq_len;
  p.g = a.group_size; p.w = a.window; p.cap = a.cache_row_capacity;
  p.dl = DecodeLayout{a.cache_rows, a.ring_n_rep, a.ring_n_tok, a.cache_row_capacity, a.n_rep_bias, a.window + a.group_size, a.group_size};
  p.decode = a.decode; p.n_tok_tiles = (a.q_len + p.TB - 1) / p.TB; p.d_out = a.d_sem;
  p.scale_log2 = a.softmax_scale * 1.4426950408889634f;
  p.bias_log2 = a.rep_logit_bias * 1.4426950408889634f;
  p.out = (bf16*)a.out; p.lse = a.lse;
  p.out_wide = (reinterpret_cast<uintptr_t>(a.out) & 31u) == 0;
  const long long qrows = (long long)a.batch * a.q_len;
  bool ok = make_tensor_map_3d(&p.q_sem, nullptr, 0, 0, 0, 0, 0);
  ok = ok && make_tensor_map_3d(&p.q_pos, a.q_pos, a.d_pos, a.n_q_heads, qrows, p.HB, p.TB);
  ok = ok && make_tensor_map_3d(&p.kv_sem, a.kv_sem, a.d_sem, a.n_kv_heads, (long long)a.batch * a.seq_len, 1, BN);
  ok = ok && make_tensor_map_3d(&p.kv_pos, a.kv_pos, a.d_pos, a.n_kv_heads, (long long)a.batch * a.seq_len, 1, BN);
  ok = ok && make_tensor_map_3d(&p.cache_sem, a.cache_sem, a.d_sem, a.n_kv_heads, (long long)a.batch * a.cache_row_capacity, 1, BN);
  ok = ok && make_tensor_map_3d(&p.cache_pos, a.cache_pos, a.d_pos, a.n_kv_heads, (long long)a.batch * a.cache_row_capacity, 1, BN);
  if (!ok) return LCA_ERR_CUDA;
  using PL = Plan1<0, 2, 2, false, 2>;
  auto kern = attn_tc1_kernel<0, 2, 2, false, 2>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, PL::BYTES) != cudaSuccess)
    return LCA_ERR_CUDA;
  dim3 grid(p.n_tok_tiles, a.n_kv_heads, a.batch);
  kern<<<grid, 320, PL::BYTES, a.stream>>>(p);
  note_launch();
  return cudaGetLastError() == cudaSuccess ? LCA_OK : LCA_ERR_CUDA;
}

// Self-test of the bounded wait: one thread waits on a barrier that nobody arrives on, with a short limit,
// and reports the expiry exactly as the attention kernels do (status word, then an orderly return).
__global__ void bounded_wait_selftest_kernel(long long limit_cycles) {
  __shared__ __align__(8) unsigned long long bar_mem;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    mbar_init(smem_u32(&bar_mem), 1);
    fence_mbar_init();
    if (!mbar_wait_limit(smem_u32(&bar_mem), 0, &abort_flag, limit_cycles)) atomicCAS(&g_tc_status, 0, ERR_WAIT_PEER);
  }
}

int bounded_wait_selftest_launch(long long limit_cycles, cudaStream_t stream) {
  bounded_wait_selftest_kernel<<<1, 32, 0, stream>>>(limit_cycles);
  note_launch();
  return cudaGetLastError() == cudaSuccess ? LCA_OK : LCA_ERR_CUDA;
}

int attn_tc_device_status(cudaStream_t stream) {
  if (cudaStreamSynchronize(stream) != cudaSuccess) return LCA_ERR_CUDA;
  int st = 0;
  if (cudaMemcpyFromSymbol(&st, g_tc_status, sizeof(int)) != cudaSuccess) return LCA_ERR_CUDA;
  int st2 = attn_tc2_take_status();
  const int st3 = attn_gqa2_take_status();
  if (st2 < 0 || st3 < 0) return LCA_ERR_CUDA;
  if (st3 != 0) st2 = st3;
  if (st == 0 && st2 != 0) return LCA_ERR_DEVICE_TIMEOUT;
  if (st != 0) {
    int zero = 0;
    cudaMemcpyToSymbol(g_tc_status, &zero, sizeof(int));
    return LCA_ERR_DEVICE_TIMEOUT;
  }
  return LCA_OK;
}

}  // namespace lca
