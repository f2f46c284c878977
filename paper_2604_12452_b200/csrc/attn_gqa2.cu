// Prefill attention for the grouped-query shape (head dimension 128; Sec. 5.4) with two query tiles in
// flight per CTA.
//
// With d = 128 the tensor work of a key tile (S = Q K^T and O += P V) is about as long as the exponentials
// of its softmax take on the special-function unit, so a kernel in which all softmax threads work on the
// same tile leaves the tensor pipe idle for half of the time.  Here a CTA owns 256 query rows = two
// sub-tiles of 128 rows (TB consecutive tokens x the HB query heads of one KV head, and the next TB
// tokens); both read the same key / value stages.  Tensor memory holds exactly two independent sets: per
// sub-tile two S buffers of 64 columns (key tiles of 64) and O in 128 columns; the probabilities of a tile
// overwrite the first half of their S buffer and feed P V from tensor memory.  Each sub-tile has its own
// group of 128 softmax threads (one thread per row: no exchange between threads).  The MMA warp keeps S
// two key tiles ahead: once P_r of tile j is ready it issues P_r V_j and then S_r of tile j + 2 into the
// buffer that P V has just read, so a softmax group finds its next S complete when it gets there, and the
// tensor pipe always has the other sub-tile's products to run.
//
// Roles: warp 0 TMA producer, warp 1 TMEM owner + MMA issue (converged warp, elected lane), warps 2-5
// softmax / epilogue of sub-tile 0, warps 6-9 of sub-tile 1.  Every wait is bounded; on expiry the CTA
// records a code in a global status word, drains and returns.
#include <cstring>
#include <type_traits>

#include "lca_common.cuh"
#include "tc_common.cuh"

namespace lca {
using namespace tc;

static __device__ int g_gqa2_status = 0;

namespace gq {
constexpr int ROWS = 128;                 // rows of one sub-tile (TMEM lanes)
constexpr int BN = 64;                    // keys per tile
constexpr int QCH = 128 * 128;            // bytes of one 64-column chunk of a 128-row query block (16 KB)
constexpr int KCH = BN * 128;             // bytes of one 64-column chunk of a key / value tile (8 KB)
constexpr int STAGES = 4;
constexpr int Q_BYTES = 2 * 2 * QCH;      // two sub-tiles x two chunks
constexpr int KV_STAGE = 2 * KCH;         // one key (or value) tile
constexpr int OFF_Q = 0, OFF_K = OFF_Q + Q_BYTES, OFF_V = OFF_K + STAGES * KV_STAGE, OFF_BAR = OFF_V + STAGES * KV_STAGE;
constexpr int OFF_MISC = OFF_BAR + 256;
constexpr int SMEM_BYTES = OFF_MISC + 64 + 1024;      // + slack to align the base to 1024 B
constexpr int TM_S = 0, TM_O = 256, TM_COLS = 512;    // S_r buffer u at TM_S + 128 r + 64 u, O_r at TM_O + 128 r
constexpr int THREADS = 320;
constexpr float RESCALE_THRESHOLD = 8.0f; // log2 units
constexpr int POLY_EVERY = 8;             // one exponential in POLY_EVERY of an interior tile goes to the FMA pipe (0: none; measured at config 5: none 1134, 1 in 16 1178, 1 in 8 1201, 1 in 6 1161, 1 in 4 1134, 1 in 2 1102 TFLOP/s)
static_assert(SMEM_BYTES <= 232448, "shared memory budget of one SM");
}  // namespace gq

struct Gqa2Params {
  CUtensorMap q, k, v, ck, cv;            // 3-D {d, heads, rows}: queries (box HB x TB), keys / values of the tokens and of the cache
  bf16* out; float* lse;
  int B, q_len, Hq, Hkv, L, g, w, cap;
  int HB, TB, n_blocks;                   // heads and tokens per sub-tile, 2*TB-token blocks per sequence
  int out_wide;
  float scale_log2, bias_log2;
  SeqTab tab;                             // ragged batch (tok_off != nullptr): q_len, L and cap are unused
};

template <bool WANT_LSE>
__global__ void __launch_bounds__(gq::THREADS, 1)
attn_gqa2_kernel(const __grid_constant__ Gqa2Params p) {
  using namespace gq;
  extern __shared__ unsigned char smem_dyn[];
  const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  unsigned char* base_ptr = smem_dyn + (base - smem_u32(smem_dyn));
  const uint32_t sQ = base + OFF_Q, sK = base + OFF_K, sV = base + OFF_V, bars = base + OFF_BAR;
  const uint32_t BAR_Q = bars;
  auto BAR_KFULL = [&](int s) { return bars + 8 * (1 + s); };                // STAGES each
  auto BAR_KEMPTY = [&](int s) { return bars + 8 * (1 + STAGES + s); };
  auto BAR_VFULL = [&](int s) { return bars + 8 * (1 + 2 * STAGES + s); };
  auto BAR_VEMPTY = [&](int s) { return bars + 8 * (1 + 3 * STAGES + s); };
  auto BAR_SFULL = [&](int r, int u) { return bars + 8 * (1 + 4 * STAGES + 2 * r + u); };   // S_r in buffer u is complete
  auto BAR_PFULL = [&](int r, int u) { return bars + 8 * (5 + 4 * STAGES + 2 * r + u); };   // P_r in buffer u has been written
  // P_r V of a tile is complete: one barrier per parity of the tile index, so that a waiter is never more than one
  // phase behind its barrier (a parity wait cannot tell phases two apart; P V of tile j - 2 is known to be complete
  // when S of tile j is, P V of tile j - 1 is not)
  auto BAR_ODONE = [&](int r, int u) { return bars + 8 * (9 + 4 * STAGES + 2 * r + u); };
  static_assert(8 * (13 + 4 * STAGES) <= 256, "barrier block");
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + OFF_MISC);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + OFF_MISC + 4);

  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;

  // ---- which rows, which key tiles (the same arithmetic in every role)
  const int hk = blockIdx.y, b = blockIdx.z;
  int q_len = p.q_len, qbase = b * p.q_len, kbase = b * p.L, cbase = b * p.cap, n_blocks = p.n_blocks;
  if (p.tab.tok_off) {                                       // ragged batch: this sequence's rows and length
    qbase = kbase = p.tab.tok_off[b];
    q_len = p.tab.tok_off[b + 1] - qbase;
    cbase = p.tab.cache_off[b];
    n_blocks = (q_len + 2 * p.TB - 1) / (2 * p.TB);
  }
  const int blk = n_blocks - 1 - (int)blockIdx.x;            // heaviest (latest) blocks first
  if (blk < 0) return;                                       // the grid covers the longest sequence (whole CTA leaves)
  const int t0 = blk * 2 * p.TB;                             // first token of the block
  const int t1 = min(t0 + 2 * p.TB, q_len) - 1;              // last valid token
  const int head0 = hk * p.HB;
  const int n_a_lo = reps_visible(t0, p.w, p.g), n_a_hi = reps_visible(t1, p.w, p.g);
  const int first_lo = n_a_lo * p.g;
  const int nA = (n_a_hi + BN - 1) / BN;
  const int nB = (t1 - first_lo + BN) / BN;
  const int n_tiles = nA + nB;                               // >= 1: every query sees at least itself

  if (threadIdx.x == 0) {
    mbar_init(BAR_Q, 1);
    for (int s = 0; s < STAGES; ++s) {
      mbar_init(BAR_KFULL(s), 1); mbar_init(BAR_KEMPTY(s), 1);
      mbar_init(BAR_VFULL(s), 1); mbar_init(BAR_VEMPTY(s), 1);
    }
    for (int r = 0; r < 2; ++r) {
      for (int u = 0; u < 2; ++u) { mbar_init(BAR_SFULL(r, u), 1); mbar_init(BAR_PFULL(r, u), 128); mbar_init(BAR_ODONE(r, u), 1); }
    }
    *abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32((const void*)tmem_slot), TM_COLS);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  auto fail = [&](int code) {
    atomicCAS(&g_gqa2_status, 0, code);
    *abort_flag = 1;
  };

  if (warp == 0) {
    // =============================================================== TMA producer
    if (lane == 0) {
      prefetch_tmap(&p.q); prefetch_tmap(&p.k); prefetch_tmap(&p.v);
      mbar_expect_tx(BAR_Q, Q_BYTES);
      for (int r = 0; r < 2; ++r) {
        const int qrow = qbase + t0 + r * p.TB;
        for (int c = 0; c < 2; ++c) tma_load_3d(sQ + (r * 2 + c) * QCH, &p.q, c * 64, head0, qrow, BAR_Q);
      }
      for (int j = 0; j < n_tiles; ++j) {
        const int s = j % STAGES, round = j / STAGES;
        const bool isA = j < nA;
        const int row = isA ? cbase + j * BN : kbase + first_lo + (j - nA) * BN;
        const CUtensorMap* mk = isA ? &p.ck : &p.k;
        const CUtensorMap* mv = isA ? &p.cv : &p.v;
        if (!mbar_wait(BAR_KEMPTY(s), (round & 1) ^ 1, abort_flag)) { fail(ERR_WAIT_KV_EMPTY); break; }
        mbar_expect_tx(BAR_KFULL(s), KV_STAGE);
        for (int c = 0; c < 2; ++c) tma_load_3d(sK + s * KV_STAGE + c * KCH, mk, c * 64, hk, row, BAR_KFULL(s));
        if (!mbar_wait(BAR_VEMPTY(s), (round & 1) ^ 1, abort_flag)) { fail(ERR_WAIT_KV_EMPTY); break; }
        mbar_expect_tx(BAR_VFULL(s), KV_STAGE);
        for (int c = 0; c < 2; ++c) tma_load_3d(sV + s * KV_STAGE + c * KCH, mv, c * 64, hk, row, BAR_VFULL(s));
      }
    }
  } else if (warp == 1) {
    // =============================================================== MMA issuer
    constexpr uint32_t IDESC_S = umma_idesc_bf16(ROWS, BN, false, false);
    constexpr uint32_t IDESC_PV = umma_idesc_bf16(ROWS, 128, false, true);
    const uint32_t leader = elect_one();
    bool ok = mbar_wait(BAR_Q, 0, abort_flag);
    if (!ok && leader) fail(ERR_WAIT_Q);
    const uint64_t qd0 = umma_desc_sw128(sQ, 16, 1024);
    auto issue_s = [&](int r, int j) {          // S_r = Q_r K_j^T into buffer j & 1 (the key stage has been waited for)
      const uint64_t kd0 = umma_desc_sw128(sK + (j % STAGES) * KV_STAGE, 16, 1024);
#pragma unroll
      for (int c = 0; c < 2; ++c) {
#pragma unroll
        for (int k = 0; k < 4; ++k)
          umma_ss_elected(leader, tmem + TM_S + 128 * r + 64 * (j & 1), desc_add(qd0, ((r * 2 + c) * QCH + k * 32) >> 4),
                          desc_add(kd0, (c * KCH + k * 32) >> 4), IDESC_S, (c > 0 || k > 0) ? 1u : 0u);
      }
      umma_commit_elected(leader, BAR_SFULL(r, j & 1));
    };
    auto issue_pv = [&](int r, int j) {         // O_r += P_r V_j (P_r and the value stage have been waited for)
      const uint64_t vd0 = umma_desc_sw128(sV + (j % STAGES) * KV_STAGE, KCH, 1024);
#pragma unroll
      for (int k = 0; k < BN / 16; ++k)
        umma_ts_elected(leader, tmem + TM_O + 128 * r, tmem + TM_S + 128 * r + 64 * (j & 1) + k * 8, desc_add(vd0, (k * 2048) >> 4),
                        IDESC_PV, (j > 0 || k > 0) ? 1u : 0u);
      umma_commit_elected(leader, BAR_ODONE(r, j & 1));
    };
    // S of the first two key tiles for both sub-tiles
    for (int j = 0; ok && j < 2 && j < n_tiles; ++j) {
      ok = mbar_wait(BAR_KFULL(j), 0, abort_flag);
      if (!ok) { if (leader) fail(ERR_WAIT_KV_FULL); break; }
      tc_fence_after();
      issue_s(0, j);
      issue_s(1, j);
      umma_commit_elected(leader, BAR_KEMPTY(j));
    }
    // Tile j: for each sub-tile in turn, P_r V_j and then S_r of tile j + 2 into the buffer P_r occupied (the
    // tensor pipe executes one thread's instructions in issue order).
    for (int j = 0; ok && j < n_tiles; ++j) {
      const int s = j % STAGES, round = j / STAGES;
      const bool more = j + 2 < n_tiles;
      const int s2 = (j + 2) % STAGES, round2 = (j + 2) / STAGES;
#pragma unroll
      for (int r = 0; r < 2; ++r) {
        ok = mbar_wait(BAR_PFULL(r, j & 1), (j >> 1) & 1, abort_flag);
        if (!ok) { if (leader) fail(ERR_WAIT_P_FULL); break; }
        if (r == 0) {
          ok = mbar_wait(BAR_VFULL(s), round & 1, abort_flag);
          if (!ok) { if (leader) fail(ERR_WAIT_KV_FULL); break; }
        }
        tc_fence_after();
        issue_pv(r, j);
        if (r == 1) umma_commit_elected(leader, BAR_VEMPTY(s));
        if (more) {
          if (r == 0) {
            ok = mbar_wait(BAR_KFULL(s2), round2 & 1, abort_flag);
            if (!ok) { if (leader) fail(ERR_WAIT_KV_FULL); break; }
            tc_fence_after();
          }
          issue_s(r, j + 2);
          if (r == 1) umma_commit_elected(leader, BAR_KEMPTY(s2));
        }
      }
    }
  } else {
    // =============================================================== softmax / epilogue, one thread per query row
    const int r = warp >= 6 ? 1 : 0;              // sub-tile
    const int quarter = warp & 3;                 // a warp may only touch the 32 TMEM lanes of its quarter
    const int row = quarter * 32 + lane;          // row inside the sub-tile
    const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
    const uint32_t s_tm = tmem + lane_base + TM_S + 128 * r, o_tm = tmem + lane_base + TM_O + 128 * r;
    const int tl = row / p.HB, hl = row % p.HB;
    const int t_row = t0 + r * p.TB + tl;
    const bool row_valid = t_row < q_len;
    const int n_a_row = reps_visible(min(t_row, q_len - 1), p.w, p.g);
    const int first_row = n_a_row * p.g;
    float m_ref = -INFINITY, l_sum = 0.f;
    bool ok = true;
    for (int j = 0; j < n_tiles; ++j) {
      const int u = j & 1;                        // S / P buffer of this tile
      if (ok) {
        ok = mbar_wait(BAR_SFULL(r, u), (j >> 1) & 1, abort_flag);
        if (!ok && lane == 0) fail(ERR_WAIT_S_FULL);
      }
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;                             // abort_flag is set: every other role drains as well
      tc_fence_after();
      uint32_t sr[2][32];
      tmem_ld32(s_tm + 64 * u, sr[0]);
      tmem_ld32(s_tm + 64 * u + 32, sr[1]);
      const bool isA = j < nA;
      const int key0 = isA ? j * BN : first_lo + (j - nA) * BN;
      bool need_mask;
      int lo, hi;                                  // visible columns of this row: lo <= c <= hi
      if (isA) { lo = 0; hi = n_a_row - key0 - 1; need_mask = key0 + BN > n_a_lo; }
      else { lo = first_row - key0; hi = t_row - key0; need_mask = (key0 < n_a_hi * p.g) || (key0 + BN - 1 > t0); }
      const bool plain = !need_mask && !(isA && p.bias_log2 != 0.f);
      tmem_wait_ld();
      float tmax;
      if (plain) {
        // interior tile: the raw products stay in sr; the (positive) scale is applied to the maximum here and
        // folded into the exponent's multiply-add below.  Three-input maxima, four independent chains.
        float tm0 = -INFINITY, tm1 = -INFINITY, tm2 = -INFINITY, tm3 = -INFINITY;
#pragma unroll
        for (int q = 0; q < 2; ++q) {
#pragma unroll
          for (int i = 0; i < 32; i += 8) {
            tm0 = max3(tm0, __uint_as_float(sr[q][i]), __uint_as_float(sr[q][i + 1]));
            tm1 = max3(tm1, __uint_as_float(sr[q][i + 2]), __uint_as_float(sr[q][i + 3]));
            tm2 = max3(tm2, __uint_as_float(sr[q][i + 4]), __uint_as_float(sr[q][i + 5]));
            tm3 = max3(tm3, __uint_as_float(sr[q][i + 6]), __uint_as_float(sr[q][i + 7]));
          }
        }
        tmax = fmaxf(fmaxf(tm0, tm1), fmaxf(tm2, tm3)) * p.scale_log2;
      } else {
        // boundary tile: scale, bias and mask with selects only
        const float bias = isA ? p.bias_log2 : 0.f;
        const int lo_m = need_mask ? lo : -(1 << 30), hi_m = need_mask ? hi : (1 << 30);
        float tm[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
        for (int q = 0; q < 2; ++q) {
#pragma unroll
          for (int i = 0; i < 32; ++i) {
            const int c = q * 32 + i;
            float sc = fmaf(__uint_as_float(sr[q][i]), p.scale_log2, bias);
            sc = ((c >= lo_m) & (c <= hi_m)) ? sc : -INFINITY;
            sr[q][i] = __float_as_uint(sc);
            tm[i & 3] = fmaxf(tm[i & 3], sc);
          }
        }
        tmax = fmaxf(fmaxf(tm[0], tm[1]), fmaxf(tm[2], tm[3]));
      }
      // running maximum: O_r is rescaled only when it grows by more than the threshold
      bool need = false;
      float factor = 1.f;
      if (j == 0) m_ref = tmax;
      else if (tmax > m_ref + RESCALE_THRESHOLD) { need = true; factor = exp2f(m_ref - tmax); }
      if (__any_sync(0xffffffffu, need)) {
        ok = mbar_wait(BAR_ODONE(r, (j - 1) & 1), ((j - 1) >> 1) & 1, abort_flag);       // P_r V of tile j - 1 has landed in O_r
        if (!ok && lane == 0) fail(ERR_WAIT_O_DONE);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) break;
        tc_fence_after();
#pragma unroll 1
        for (int q = 0; q < 4; ++q) {
          uint32_t o[32];
          tmem_ld32(o_tm + q * 32, o);
          tmem_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * factor);
          tmem_st32(o_tm + q * 32, o);
        }
        if (need) { l_sum *= factor; m_ref = tmax; }
      }
      const float m_use = (m_ref == -INFINITY) ? 0.f : m_ref;
      // Probabilities, packed two per word, written back over the first 32 columns of the S buffer (A operand of
      // P V).  Scale and row sum work on pairs of fp32 values (one instruction per pair).
      const float e_mul = plain ? p.scale_log2 : 1.f;          // sr holds raw products (plain) or scaled logits
      const uint64_t mul2 = pack_f32x2(e_mul, e_mul), sub2 = pack_f32x2(-m_use, -m_use);
      uint64_t rs2 = pack_f32x2(0.f, 0.f);
      uint32_t pk[32];
      auto exps = [&](auto interior) {
        constexpr bool INTERIOR = decltype(interior)::value;
#pragma unroll
        for (int i = 0; i < 32; ++i) {
          float a0, a1;
          unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(sr[i >> 4][(2 * i) & 31]), __uint_as_float(sr[i >> 4][(2 * i + 1) & 31])), mul2, sub2), a0, a1);
          // interior tiles (every logit finite): one exponential in POLY_EVERY on the FMA pipe, the others on the
          // special-function unit, so that the two pipes share the work
          const bool poly = INTERIOR && POLY_EVERY > 0 && (2 * i) % (POLY_EVERY > 0 ? POLY_EVERY : 1) == 0;
          const float p0 = poly ? exp2_fma(a0) : exp2f(a0);
          const float p1 = exp2f(a1);
          pk[i] = pack_bf16x2(p0, p1);
          rs2 = add_f32x2(rs2, pack_f32x2(p0, p1));
        }
      };
      if (plain) exps(std::true_type{}); else exps(std::false_type{});
      tmem_st32(s_tm + 64 * u, pk);
      {
        float r0, r1;
        unpack_f32x2(rs2, r0, r1);
        l_sum += r0 + r1;
      }
      tmem_wait_st();
      tc_fence_before();
      mbar_arrive(BAR_PFULL(r, u));
    }
    // ---- epilogue: O_r / l -> bf16 -> global
    if (ok) {
      ok = mbar_wait(BAR_ODONE(r, (n_tiles - 1) & 1), ((n_tiles - 1) >> 1) & 1, abort_flag);
      if (!ok && lane == 0) fail(ERR_WAIT_O_DONE);
      ok = __all_sync(0xffffffffu, ok);
    }
    if (ok) {
      tc_fence_after();
      const float inv = l_sum > 0.f ? 1.f / l_sum : 0.f;
      const size_t orow = ((size_t)qbase + t_row) * p.Hq + head0 + hl;
      bf16* dst = p.out + orow * 128;
#pragma unroll 1
      for (int q = 0; q < 4; ++q) {
        uint32_t o[32];
        tmem_ld32(o_tm + q * 32, o);
        tmem_wait_ld();
        if (row_valid) {
#pragma unroll
          for (int v = 0; v < 2; ++v) {
            uint32_t wv[8];
#pragma unroll
            for (int e = 0; e < 8; ++e)
              wv[e] = pack_bf16x2(__uint_as_float(o[16 * v + 2 * e]) * inv, __uint_as_float(o[16 * v + 2 * e + 1]) * inv);
            st_global_32B(dst + q * 32 + 16 * v, wv, p.out_wide != 0);
          }
        }
      }
      if (WANT_LSE && row_valid)
        p.lse[orow] = l_sum > 0.f ? (m_ref + log2f(l_sum)) * 0.6931471805599453f : -INFINITY;
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
    tmem_dealloc(tmem, TM_COLS);
  }
}

// ----------------------------------------------------------------------------------- host
bool make_tensor_map_3d(CUtensorMap* map, const void* ptr, int d, int heads, long long rows, int box_heads, int box_rows);

bool attn_gqa2_supported(const AttnProblem& a) {
  if (a.decode || a.variant != LCA_VARIANT_GQA || a.d_sem != 128 || a.d_pos != 128) return false;
  const int rep = a.n_q_heads / a.n_kv_heads;
  return rep >= 1 && rep <= 128 && 128 % rep == 0;
}

int attn_gqa2_launch(const AttnProblem& a) {
  using namespace gq;
  if (!attn_gqa2_supported(a)) return LCA_ERR_UNSUPPORTED_SHAPE;
  Gqa2Params p;
  memset(&p, 0, sizeof(p));
  const int rep = a.n_q_heads / a.n_kv_heads;
  p.HB = rep; p.TB = ROWS / rep;
  p.B = a.batch; p.q_len = a.q_len; p.Hq = a.n_q_heads; p.Hkv = a.n_kv_heads; p.L = a.seq_len;
  p.g = a.group_size; p.w = a.window; p.cap = a.cache_row_capacity;
  p.n_blocks = (a.q_len + 2 * p.TB - 1) / (2 * p.TB);
  p.scale_log2 = a.softmax_scale * 1.4426950408889634f;
  p.bias_log2 = a.rep_logit_bias * 1.4426950408889634f;
  p.out = (bf16*)a.out; p.lse = a.lse;
  p.out_wide = (reinterpret_cast<uintptr_t>(a.out) & 31u) == 0;
  long long qrows = (long long)a.batch * a.q_len, krows = (long long)a.batch * a.seq_len,
            crows = (long long)a.batch * a.cache_row_capacity;
  if (a.h_tok_off) {
    p.tab = a.tab;
    qrows = krows = a.h_tok_off[a.batch];
    crows = a.h_cache_off[a.batch];
  }
  bool ok = make_tensor_map_3d(&p.q, a.q_pos, 128, a.n_q_heads, qrows, p.HB, p.TB);
  ok = ok && make_tensor_map_3d(&p.k, a.kv_pos, 128, a.n_kv_heads, krows, 1, BN);
  ok = ok && make_tensor_map_3d(&p.v, a.kv_sem, 128, a.n_kv_heads, krows, 1, BN);
  // no group yet (m = 0): the cache maps are never used; describe the token arrays instead of a null pointer
  ok = ok && make_tensor_map_3d(&p.ck, a.cache_pos ? a.cache_pos : a.kv_pos, 128, a.n_kv_heads, a.cache_pos ? crows : krows, 1, BN);
  ok = ok && make_tensor_map_3d(&p.cv, a.cache_sem ? a.cache_sem : a.kv_sem, 128, a.n_kv_heads, a.cache_sem ? crows : krows, 1, BN);
  if (!ok) return LCA_ERR_CUDA;
  auto kern = a.lse ? attn_gqa2_kernel<true> : attn_gqa2_kernel<false>;
  if (cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) != cudaSuccess)
    return LCA_ERR_CUDA;
  dim3 grid(p.n_blocks, a.n_kv_heads, a.batch);
  kern<<<grid, THREADS, SMEM_BYTES, a.stream>>>(p);
  note_launch();
  return cudaGetLastError() == cudaSuccess ? LCA_OK : LCA_ERR_CUDA;
}

int attn_gqa2_take_status() {
  int st = 0;
  if (cudaMemcpyFromSymbol(&st, g_gqa2_status, sizeof(int)) != cudaSuccess) return -1;
  if (st != 0) {
    int zero = 0;
    cudaMemcpyToSymbol(g_gqa2_status, &zero, sizeof(int));
  }
  return st;
}

}  // namespace lca
