// MLA-shaped (d_c = 512, d_R = 64) attention over the condensed context on CTA pairs.
//
// The absorbed MLA shape does not fit one SM: 128 query rows x 512 fp32 output columns is the
// whole of tensor memory, and a 128 x 576 bf16 query tile is 144 KB of shared memory.  So two
// CTAs of a cluster share one tile of 128 query rows (TB tokens x HB heads) and issue
// tcgen05.mma with cta_group::2:
//   * each CTA holds 64 of the query rows (72 KB) and, per tile of 128 keys, 64 of the keys with
//     all 576 columns (B operand of S = Q K^T is split by keys) and all 128 keys of 256 of the
//     512 value columns (B operand of O += P V is split by output columns);
//   * S lands as 128 lanes x 64 columns per CTA (lanes 0-63: keys 0-63, lanes 64-127: keys
//     64-127 of the CTA's 64 rows), O as 128 lanes x 256 columns;
//   * softmax threads (one per lane) exchange the row maximum of the two key halves through
//     shared memory, write P as bf16 into a 128-byte-swizzled shared tile (A operand of PV)
//     and signal the even CTA, whose MMA warp issues every tcgen05.mma for the pair.
// Everything else (tile walk over representatives then local tokens, boundary-only masks, lazy
// rescale of O, bounded waits with a status word) follows the single-CTA kernel.
//
// A CTA pair is persistent: it takes work items (tiles of 128 query rows) from the heaviest (latest
// tokens) down in a fixed stride.  Barriers and tensor memory are set up once; the query tile of the
// next item is fetched as soon as the last S product of the current one has completed, and its first
// products run while the softmax threads still normalise and store the current output.
//
// The one software signal between the two CTAs ("P of the odd CTA is complete") is forwarded by a relay
// thread with mbarrier.arrive.relaxed.cluster after it has acquired the local arrivals of the writers (whose
// stores were followed by fence.proxy.async).  That the even CTA's next tcgen05.mma then sees the odd CTA's P
// is an argument about the hardware's behaviour, not a guarantee of the PTX memory model; the test that runs the
// 128K configuration twice and compares every output bit is its check and has to stay.
#include <algorithm>
#include <cstring>
#include <vector>

#include "lca_common.cuh"
#include "tc_common.cuh"

namespace lca {
using namespace tc;

static __device__ int g_tc2_status = 0;

namespace pair {
constexpr int BN = 128;                 // keys per tile (64 per CTA for S)
constexpr int NKC = 9;                  // 64-column key chunks: 8 latent + 1 rope
// The key part of a tile is one buffer, filled and released in NKG pieces, so that the refill of a piece
// starts while S = Q K^T still reads the others.  S takes the chunks in the order rope, latent 0..7; piece p
// covers positions [piece_begin(p), piece_begin(p + 1)) of that order.
constexpr int NKG = 2;                  // two pieces: rope chunk + latent chunks 0-3, latent chunks 4-7
__host__ __device__ constexpr int piece_begin(int p) { return p == 0 ? 0 : p == 1 ? 5 : 9; }
constexpr int KBOX = 4;                 // latent column chunks brought by one TMA request of the key part
constexpr int VBOX = 2;                 // column chunks brought by one request of the value part
constexpr int QCH = 64 * 128;           // bytes of one query chunk  (64 rows)
constexpr int KCH = 64 * 128;           // bytes of one key chunk    (64 keys)
constexpr int VCH = 64 * 128;           // bytes of one value chunk  (64 keys x 64 columns)
constexpr int PCH = 64 * 128;           // bytes of one P chunk      (64 rows x 64 keys)
constexpr int Q_BYTES = NKC * QCH, K_BYTES = NKC * KCH, V_BYTES = 8 * VCH, P_BYTES = 2 * PCH;
constexpr int OFF_Q = 0, OFF_K = OFF_Q + Q_BYTES, OFF_V = OFF_K + K_BYTES, OFF_P = OFF_V + V_BYTES;
constexpr int OFF_BAR = OFF_P + P_BYTES;
constexpr int OFF_MISC = OFF_BAR + 256, OFF_RED = OFF_BAR + 512;
constexpr int SMEM_BYTES = OFF_BAR + 512 + 3 * 128 * 4;     // 231424
constexpr int TM_S0 = 0, TM_S1 = 64, TM_O = 128, TM_COLS = 512;
constexpr int THREADS = 224;            // warps: 0 K/Q loads, 1 MMA + TMEM, 2-5 softmax, 6 V loads
constexpr float RESCALE_THRESHOLD = 8.0f;
static_assert(SMEM_BYTES <= 232448, "shared memory budget of one SM");
}  // namespace pair

struct Tc2Params {
  CUtensorMap q_sem, q_pos;       // queries, box of 64 rows
  CUtensorMap k_pos, c_pos;       // rope keys of the tokens / of the condensed cache, box of 64 rows
  CUtensorMap k_sem, c_sem;       // latents seen as (64 columns, rows, chunks): box of 64 rows x KBOX chunks
  CUtensorMap k_val, c_val;       // the same memory, box of 64 rows x VBOX chunks
  bf16* out; float* lse;
  DecodeLayout dl;                // decode: which rows of a sequence's cache take part (packed or ring layout)
  int B, q_len, H, L, g, w, cap, decode;
  int HB, TB, n_tok_tiles, n_head_blocks;
  int out_wide;                   // out is 32-byte aligned: 256-bit stores
  long long n_items;              // query tiles x head blocks x batch
  // ragged prefill batch: (sequence, token tile) of every entry, heaviest first, and the sequences' first rows;
  // item idx is head block idx % n_head_blocks of entry idx / n_head_blocks.  nullptr: uniform batch.
  const int2* entries;
  SeqTab tab;
  float scale_log2, bias_log2;
  // Split decode (few sequences): the key tiles of all (sequence, head block) units form one line that is cut into
  // equal ranges, one per CTA pair; a range that does not hold a whole unit leaves an unnormalised partial result
  // (O, row maximum, row sum) in `partial`, merged by decode_combine_kernel.  split = 0: one unit per work item.
  int split;
  float* partial;                 // [slots][PARTIAL_FLOATS]
};
constexpr int PARTIAL_FLOATS = 128 * 512 + 2 * 128;     // O of 128 rows, then (maximum, sum) per row

// One work item = one tile of 128 query rows (split decode: a range of its key tiles); the same arithmetic in every
// role of both CTAs.
struct Item {
  int b, head0, t0, t1, len;      // sequence, first head, first / last token of the tile, length of the sequence
  int qbase, kbase, cbase;        // row of the sequence's first token in the query / token arrays, of its first cache row
  int n_a_lo, n_a_hi, first_lo, nA, n_tiles;
  int j0;                         // split decode: first key tile of the range (0 otherwise)
  int slot;                       // split decode: >= 0 where the range is only a part of its unit
};
__device__ __forceinline__ Item make_item(const Tc2Params& p, long long idx) {
  Item it;
  int tile;
  if (p.entries) {
    const int2 e = p.entries[idx / p.n_head_blocks];
    it.b = e.x; tile = e.y;
    it.head0 = (int)(idx % p.n_head_blocks) * p.HB;
    it.qbase = it.kbase = p.tab.tok_off[it.b];
    it.len = p.tab.tok_off[it.b + 1] - it.qbase;
    it.cbase = p.tab.cache_off[it.b];
  } else {
    // heaviest query tiles (latest tokens) first; batch and head block vary fastest
    const long long per_tile = (long long)p.n_head_blocks * p.B;
    tile = p.n_tok_tiles - 1 - (int)(idx / per_tile);
    const int rem = (int)(idx % per_tile);
    it.b = rem / p.n_head_blocks;
    it.head0 = (rem % p.n_head_blocks) * p.HB;
    it.len = p.q_len;
    it.qbase = it.b * p.q_len; it.kbase = it.b * p.L; it.cbase = it.b * p.cap;
  }
  it.t0 = tile * p.TB;
  it.t1 = min(it.t0 + p.TB, it.len) - 1;
  it.j0 = 0; it.slot = -1;
  int nB;
  if (p.decode) {
    it.n_a_hi = it.n_a_lo = decode_span(p.dl, it.b).rows_end;
    it.first_lo = 0; nB = 0;
  } else {
    it.n_a_lo = reps_visible(it.t0, p.w, p.g);
    it.n_a_hi = reps_visible(it.t1, p.w, p.g);
    it.first_lo = it.n_a_lo * p.g;
    nB = (it.t1 - it.first_lo + pair::BN) / pair::BN;
  }
  it.nA = (it.n_a_hi + pair::BN - 1) / pair::BN;
  it.n_tiles = it.nA + nB;
  return it;
}

// Key tiles of decode unit u = (sequence, head block), head block fastest.
__device__ __forceinline__ int unit_tiles(const Tc2Params& p, int u) {
  const int rows = decode_span(p.dl, u / p.n_head_blocks).rows_end;
  return (rows + pair::BN - 1) / pair::BN;
}
// Ranges (one per pair, `q` tiles long) that touch a unit of n > 0 tiles starting at tile `off` of the line.
__device__ __forceinline__ int unit_ranges(long long off, int n, long long q) {
  return (int)((off + n - 1) / q - off / q) + 1;
}

// The walk of one role over the work items of its CTA pair.  Every role of both CTAs runs the same walk.
struct Walk {
  long long idx, stride;          // one unit / tile per item: next item, number of pairs
  long long cur, end, q, off;     // split decode: next tile of the line, end of this pair's range, range length,
  int u, slot_base, n_units;      //   first tile of unit u, first partial slot of unit u
  long long pair_id;
};
// Split decode: where the range of this pair starts, found once per CTA by one warp (units in chunks of 32, prefix
// sums by shuffles) and left in shared memory for every role: {q, cur, end, off, u, slot_base}.
__device__ __forceinline__ void split_start(const Tc2Params& p, long long pair_id, long long n_pairs, int lane, volatile int* dst) {
  const int n_units = p.B * p.n_head_blocks;
  int total = 0;
  for (int u0 = 0; u0 < n_units; u0 += 32) {
    const int n = u0 + lane < n_units ? unit_tiles(p, u0 + lane) : 0;
    total += __reduce_add_sync(0xffffffffu, n);
  }
  const int q = total > 0 ? (int)((total + n_pairs - 1) / n_pairs) : 1;
  const int cur = (int)min(pair_id * q, (long long)total), end = min(total, cur + q);
  int off = 0, slot_base = 0, u_found = n_units, off_found = total, slot_found = 0;
  for (int u0 = 0; u0 < n_units && u_found == n_units; u0 += 32) {
    const int n = u0 + lane < n_units ? unit_tiles(p, u0 + lane) : 0;
    int incl = n;                                            // inclusive prefix of the tile counts
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const int t = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += t; }
    const int my_off = off + incl - n;
    const int r = n > 0 ? unit_ranges(my_off, n, q) : 0;
    int rincl = r;                                           // inclusive prefix of the range counts
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const int t = __shfl_up_sync(0xffffffffu, rincl, o); if (lane >= o) rincl += t; }
    const bool holds = n > 0 && my_off <= cur && cur < my_off + n;
    const unsigned who = __ballot_sync(0xffffffffu, holds);
    if (who) {
      const int src = __ffs(who) - 1;
      u_found = u0 + src;
      off_found = __shfl_sync(0xffffffffu, my_off, src);
      slot_found = slot_base + __shfl_sync(0xffffffffu, rincl - r, src);
    }
    off += __shfl_sync(0xffffffffu, incl, 31);
    slot_base += __shfl_sync(0xffffffffu, rincl, 31);
  }
  if (lane == 0) { dst[0] = q; dst[1] = cur; dst[2] = end; dst[3] = off_found; dst[4] = u_found; dst[5] = slot_found; }
}
__device__ __forceinline__ void walk_init(const Tc2Params& p, Walk& w, long long pair_id, long long n_pairs, const volatile int* start) {
  w.idx = pair_id; w.stride = n_pairs; w.pair_id = pair_id;
  if (!p.split) return;
  w.n_units = p.B * p.n_head_blocks;
  w.q = start[0]; w.cur = start[1]; w.end = start[2]; w.off = start[3]; w.u = start[4]; w.slot_base = start[5];
}
__device__ __forceinline__ bool walk_next(const Tc2Params& p, Walk& w, Item& it) {
  if (!p.split) {
    if (w.idx >= p.n_items) return false;
    it = make_item(p, w.idx);
    w.idx += w.stride;
    return true;
  }
  if (w.cur >= w.end) return false;
  int n = unit_tiles(p, w.u);
  while (n == 0) { ++w.u; n = unit_tiles(p, w.u); }          // cur < total: a unit with tiles follows
  const int j0 = (int)(w.cur - w.off);
  const int j1 = (int)min((long long)n, j0 + (w.end - w.cur));
  it.b = w.u / p.n_head_blocks;
  it.head0 = (w.u % p.n_head_blocks) * p.HB;
  it.len = 1; it.t0 = 0; it.t1 = 0;
  it.qbase = it.b * p.q_len; it.kbase = 0; it.cbase = it.b * p.cap;
  it.n_a_hi = it.n_a_lo = decode_span(p.dl, it.b).rows_end;
  it.first_lo = 0;
  it.j0 = j0; it.nA = it.n_tiles = j1 - j0;
  it.slot = (j0 == 0 && j1 == n) ? -1 : w.slot_base + (int)(w.pair_id - w.off / w.q);
  w.cur += j1 - j0;
  if (j1 == n) { w.slot_base += unit_ranges(w.off, n, w.q); w.off += n; ++w.u; }
  return true;
}

// Decode only: tile j of the item contains cache rows at or behind the sequence's valid row count.
__device__ __forceinline__ bool ragged_decode_tile(const Tc2Params& p, const Item& it, int j) {
  return p.decode && (it.j0 + j + 1) * pair::BN > it.n_a_hi;
}

// RING: decode over the ring layout of the cache (rows of condensed tokens inside the ring are masked out, the
// representatives' bias applies from row R on); a separate instantiation so that the prefill code stays as it is.
template <bool RING>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(pair::THREADS, 1)
attn_tc2_kernel(const __grid_constant__ Tc2Params p) {
  using namespace pair;
  extern __shared__ __align__(1024) unsigned char smem[];
  const uint32_t base = smem_u32(smem);
  const uint32_t sQ = base + OFF_Q, sK = base + OFF_K, sV = base + OFF_V, sP = base + OFF_P;
  const uint32_t bars = base + OFF_BAR;
  // One buffer for the key part of a tile (nine 64-column chunks) and one for each 64-key half of
  // its value part: a buffer is refilled with the next tile's data as soon as the MMAs that read it
  // have completed, so the loads of tile j+1 run underneath the remaining MMAs of tile j.  Tiles are
  // counted through all items of the pair (jt), which is what every per-tile barrier phase follows;
  // the per-item barriers (Q, QFREE, OLAST, OFREE, OLOCAL) follow the count of non-empty items.
  const uint32_t BAR_Q = bars, BAR_SFULL0 = bars + 8, BAR_SFULL1 = bars + 16, BAR_PFULL = bars + 24,
                 BAR_ODONE = bars + 32;
  auto BAR_KFULL = [&](int c) { return bars + 40 + 8 * c; };            // NKG (room for 9)
  auto BAR_KEMPTY = [&](int c) { return bars + 40 + 72 + 8 * c; };      // NKG (room for 9)
  auto BAR_VFULL = [&](int h) { return bars + 40 + 144 + 8 * h; };      // 2
  auto BAR_VEMPTY = [&](int h) { return bars + 40 + 160 + 8 * h; };     // 2
  auto BAR_VLOC = [&](int h) { return bars + 40 + 16 + 8 * h; };        // 2: odd CTA, value part of a ragged decode tile
  const uint32_t BAR_PLOCAL = bars + 224;        // odd CTA: its 128 softmax threads -> its relay thread
  const uint32_t BAR_QFREE = bars + 216;         // last S of an item done: the query tile may be replaced
  const uint32_t BAR_OLAST = bars + 232;         // last P V of an item done: O is complete
  const uint32_t BAR_OFREE = bars + 240;         // O has been read out by both CTAs: the next item may overwrite it
  const uint32_t BAR_OLOCAL = bars + 248;        // odd CTA: O read out by its 128 threads -> its relay thread
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + OFF_MISC);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + OFF_MISC + 4);
  volatile float* red = reinterpret_cast<volatile float*>(smem + OFF_RED);    // [3][128]: maxima of even / odd tiles, row sums

  // the warp index through a shuffle: provably warp-uniform, so the role branches below are uniform branches
  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();       // 0 = even CTA: issues the MMAs, owns the "full" barriers

  const long long pair_id = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    mbar_init(BAR_Q, 1);
    for (int c = 0; c < NKG; ++c) { mbar_init(BAR_KFULL(c), 1); mbar_init(BAR_KEMPTY(c), 1); }
    for (int h = 0; h < 2; ++h) { mbar_init(BAR_VFULL(h), 1); mbar_init(BAR_VEMPTY(h), 1); mbar_init(BAR_VLOC(h), 1); }
    mbar_init(BAR_SFULL0, 1); mbar_init(BAR_SFULL1, 1);
    mbar_init(BAR_PFULL, 129); mbar_init(BAR_ODONE, 1);     // 128 threads of the even CTA + the odd CTA's relay
    mbar_init(BAR_PLOCAL, 128);
    mbar_init(BAR_QFREE, 1); mbar_init(BAR_OLAST, 1); mbar_init(BAR_OFREE, 129); mbar_init(BAR_OLOCAL, 128);
    *abort_flag = (base & 1023u) ? 1 : 0;
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc_pair(smem_u32((const void*)tmem_slot), TM_COLS);
    tmem_relinquish_pair();
  }
  volatile int* split_state = reinterpret_cast<volatile int*>(smem + OFF_MISC + 32);   // [6], split decode only
  if (p.split && warp == 0) split_start(p, pair_id, n_pairs, lane, split_state);
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();                              // both CTAs' barriers are initialised
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;

  auto fail = [&](int code) {
    atomicCAS(&g_tc2_status, 0, code);
    *abort_flag = 1;
  };
  if (threadIdx.x == 0 && (base & 1023u)) atomicCAS(&g_tc2_status, 0, 100);

  // rows of this CTA inside the pair tile: global row rg = 64*rank + rl = tl*HB + hl
  const int row0 = 64 * (int)rank;

  if (warp == 0) {
    // =============================================== producer: Q of each item, then the key part of each tile
    if (lane == 0 && !*abort_flag) {
      const uint32_t q_bar = mapa_u32(BAR_Q, 0);
      uint32_t jt = 0, n_item = 0;
      bool good = true;
      Walk wk;
      walk_init(p, wk, pair_id, n_pairs, split_state);
      Item it;
      while (good && walk_next(p, wk, it)) {
        if (it.n_tiles == 0) continue;             // nothing to attend to (decode with an empty cache): no loads, no phases
        // the query tile may be replaced once the last S of the previous item has completed
        if (!mbar_wait(BAR_QFREE, (n_item & 1) ^ 1, abort_flag)) { fail(ERR_WAIT_Q); break; }
        if (rank == 0) mbar_expect_tx(BAR_Q, 2 * Q_BYTES);
        const int qtok = it.qbase + it.t0 + row0 / p.HB, qhead = it.head0 + row0 % p.HB;
        for (int c = 0; c < 8; ++c) tma_load_3d_pair(sQ + c * QCH, &p.q_sem, c * 64, qhead, qtok, q_bar);
        tma_load_3d_pair(sQ + 8 * QCH, &p.q_pos, 0, qhead, qtok, q_bar);
        ++n_item;
        for (int j = 0; good && j < it.n_tiles; ++j, ++jt) {
          const bool isA = j < it.nA;
          const int row = (isA ? it.cbase + (it.j0 + j) * BN : it.kbase + it.first_lo + (j - it.nA) * BN) + 64 * (int)rank;
          const CUtensorMap* ms = isA ? &p.c_sem : &p.k_sem;
          const CUtensorMap* mp = isA ? &p.c_pos : &p.k_pos;
          if (p.decode) {
            // Decode: every sequence streams its own cache from HBM (in prefill the pairs share the stream through
            // L2).  Ask for the key rows into L2 before waiting for the buffer, so that the load below finds them there.
            for (int c = 0; c < 8; c += KBOX) tma_prefetch_l2_3d(&p.c_sem, 0, row, c);
            tma_prefetch_l2_3d(&p.c_pos, 0, 0, row);
          }
          for (int gk = 0; gk < NKG; ++gk) {
            if (!mbar_wait(BAR_KEMPTY(gk), (jt & 1) ^ 1, abort_flag)) { fail(ERR_WAIT_KV_EMPTY); good = false; break; }
            const int pos0 = piece_begin(gk), pos1 = piece_begin(gk + 1);
            if (rank == 0) mbar_expect_tx(BAR_KFULL(gk), 2 * (pos1 - pos0) * KCH);
            const uint32_t k_bar = mapa_u32(BAR_KFULL(gk), 0);
            if (pos0 == 0) tma_load_3d_pair(sK + 8 * KCH, mp, 0, 0, row, k_bar);
            for (int c = max(pos0 - 1, 0); c < pos1 - 1; c += KBOX) tma_load_3d_pair(sK + c * KCH, ms, 0, row, c, k_bar);
          }
        }
      }
    }
  } else if (warp == 6) {
    // =============================================== producer: the value part of each tile
    if (lane == 0 && !*abort_flag) {
      uint32_t jt = 0;
      bool good = true;
      Walk wk;
      walk_init(p, wk, pair_id, n_pairs, split_state);
      Item it;
      while (good && walk_next(p, wk, it)) {
        for (int j = 0; good && j < it.n_tiles; ++j, ++jt) {
          const bool isA = j < it.nA;
          const int row = isA ? it.cbase + (it.j0 + j) * BN : it.kbase + it.first_lo + (j - it.nA) * BN;
          const CUtensorMap* mv = isA ? &p.c_val : &p.k_val;
          // Decode, last tile of a sequence whose valid rows end inside it: the rows behind them may hold anything
          // (0 x NaN would reach O), so the softmax threads of each CTA zero them in their own value buffers before
          // they release P.  They must see the data land first: the odd CTA's copies then complete on a barrier of
          // its own, and the even CTA's barrier expects the even CTA's bytes only.
          const bool ragged = ragged_decode_tile(p, it, j);
          for (int kh = 0; kh < 2; ++kh) {            // keys [64*kh, 64*kh+64) of the tile
            if (!mbar_wait(BAR_VEMPTY(kh), (jt & 1) ^ 1, abort_flag)) { fail(ERR_WAIT_KV_EMPTY); good = false; break; }
            uint32_t v_bar;
            if (ragged && rank == 1) {
              mbar_expect_tx(BAR_VLOC(kh), 4 * VCH);
              v_bar = BAR_VLOC(kh);
            } else {
              if (rank == 0) mbar_expect_tx(BAR_VFULL(kh), (ragged ? 1 : 2) * 4 * VCH);
              v_bar = mapa_u32(BAR_VFULL(kh), 0);
            }
            // output columns of this CTA: [128*rank, +128) of the first 256, then of the second 256
            for (int i = 0; i < 4; i += VBOX) {
              const int chunk = (i >> 1) * 4 + 2 * (int)rank + (i & 1);
              tma_load_3d_pair(sV + (kh * 4 + i) * VCH, mv, 0, row + 64 * kh, chunk, v_bar);
            }
          }
        }
      }
    }
  } else if (warp == 1) {
    // =============================================== MMA issuer (even CTA only)
    // The whole warp walks the loop (every lane polls the barriers); one elected lane issues.
    if (rank == 0 && !*abort_flag) {
      const uint32_t leader = elect_one();
      constexpr uint32_t IDESC_S = umma_idesc_bf16(128, BN, false, false);
      constexpr uint32_t IDESC_PV = umma_idesc_bf16(128, 256, false, true);
      // The shared-memory descriptors are built once and only their start-address field (low word)
      // is advanced per instruction.
      const uint64_t qd0 = umma_desc_sw128(sQ, 16, 1024), kd0 = umma_desc_sw128(sK, 16, 1024);
      const uint64_t pd0 = umma_desc_sw128(sP, 16, 1024), vd0 = umma_desc_sw128(sV, VCH, 1024);
      uint32_t jt = 0, n_item = 0;                  // tiles issued so far (all items), non-empty items started
      bool ok = true;
      // P V of a tile is issued after S of the next one (so that S runs while the softmax threads work);
      // the tile whose P V is still to be issued:
      bool pending = false, pend_first = false, pend_last = false;
      uint32_t pend_t = 0, pend_item = 0;
      auto issue_pending_pv = [&]() -> bool {
        const uint32_t t = pend_t;
        pending = false;
        if (pend_first && pend_item > 0) {
          // O of the previous item has been read out by the epilogue threads of both CTAs
          if (!mbar_wait(BAR_OFREE, (pend_item - 1) & 1, abort_flag)) { if (leader) fail(ERR_WAIT_O_DONE); return false; }
        }
        if (!mbar_wait(BAR_PFULL, t & 1, abort_flag)) { if (leader) fail(ERR_WAIT_P_FULL); return false; }
#pragma unroll
        for (int kh = 0; kh < 2; ++kh) {
          if (!mbar_wait(BAR_VFULL(kh), t & 1, abort_flag)) { if (leader) fail(ERR_WAIT_KV_FULL); return false; }
          tc_fence_after();
          // descriptors differ from the precomputed bases only in the 16-byte-unit start address
#pragma unroll
          for (int n2 = 0; n2 < 2; ++n2) {
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              const uint64_t ad = desc_add(pd0, (kh * PCH + k * 32) >> 4);
              const uint64_t bd = desc_add(vd0, ((kh * 4 + n2 * 2) * VCH + k * 2048) >> 4);
              umma_ss_pair_elected(leader, tmem + TM_O + n2 * 128, ad, bd, IDESC_PV, (!pend_first || kh > 0 || k > 0) ? 1u : 0u);
            }
          }
          umma_commit_pair_elected(leader, BAR_VEMPTY(kh), 3);
        }
        umma_commit_pair_elected(leader, BAR_ODONE, 3);
        if (pend_last) umma_commit_pair_elected(leader, BAR_OLAST, 3);      // one phase per item, for the epilogue
        return true;
      };
      Walk wk;
      walk_init(p, wk, pair_id, n_pairs, split_state);
      Item it;
      while (ok && walk_next(p, wk, it)) {
        if (it.n_tiles == 0) continue;
        for (int j = 0; ok && j < it.n_tiles; ++j, ++jt) {
          // In the middle of an item S of tile j goes before P V of tile j - 1.  At an item boundary the
          // last P V of the previous item goes first: nothing else can run until the new query tile is in.
          const bool pv_first = (j == 0);
          if (pv_first) {
            if (pending) ok = issue_pending_pv();
            if (ok) {
              ok = mbar_wait(BAR_Q, n_item & 1, abort_flag);
              if (!ok && leader) fail(ERR_WAIT_Q);
            }
            if (!ok) break;
          }
          const uint32_t stm = tmem + ((jt & 1) ? TM_S1 : TM_S0);
#pragma unroll
          for (int gk = 0; gk < NKG; ++gk) {
            ok = mbar_wait(BAR_KFULL(gk), jt & 1, abort_flag);
            if (!ok) { if (leader) fail(ERR_WAIT_KV_FULL); break; }
            tc_fence_after();
#pragma unroll
            for (int pos = piece_begin(gk); pos < piece_begin(gk + 1); ++pos) {
              const int c = pos == 0 ? 8 : pos - 1;               // the rope chunk goes first
#pragma unroll
              for (int k = 0; k < 4; ++k) {
                const uint64_t ad = desc_add(qd0, (c * QCH + k * 32) >> 4);
                const uint64_t bd = desc_add(kd0, (c * KCH + k * 32) >> 4);
                umma_ss_pair_elected(leader, stm, ad, bd, IDESC_S, (c != 8 || k > 0) ? 1u : 0u);
              }
            }
            umma_commit_pair_elected(leader, BAR_KEMPTY(gk), 3);
          }
          if (!ok) break;
          umma_commit_pair_elected(leader, (jt & 1) ? BAR_SFULL1 : BAR_SFULL0, 3);
          if (j + 1 == it.n_tiles) umma_commit_pair_elected(leader, BAR_QFREE, 3);     // last S of the item is in flight
          if (!pv_first && pending) ok = issue_pending_pv();
          pending = true; pend_t = jt; pend_first = (j == 0); pend_last = (j + 1 == it.n_tiles); pend_item = n_item;
        }
        ++n_item;
      }
      if (ok && pending) issue_pending_pv();
    }
    // =============================================== relay (odd CTA): "P complete" / "O read out" -> even CTA
    // A release-arrive on a barrier of the other CTA stalls its thread for 1000-2000 cycles.  The odd CTA's
    // softmax threads therefore arrive on barriers of their own CTA and this otherwise idle thread forwards
    // one relaxed arrival per tile and one per item: it has observed the threads' arrivals (acquire), their
    // writes of P (followed by a proxy fence) and reads of O (followed by tcgen05.wait) are complete, and the
    // consumer is this SM's own tensor core, started by an instruction that the even CTA issues afterwards.
    if (rank == 1 && lane == 0 && !*abort_flag) {
      const uint32_t pfull_addr = mapa_u32(BAR_PFULL, 0), ofree_addr = mapa_u32(BAR_OFREE, 0);
      uint32_t jt = 0, n_item = 0;
      bool good = true;
      Walk wk;
      walk_init(p, wk, pair_id, n_pairs, split_state);
      Item it;
      while (good && walk_next(p, wk, it)) {
        if (it.n_tiles == 0) continue;
        for (int j = 0; j < it.n_tiles; ++j, ++jt) {
          if (!mbar_wait(BAR_PLOCAL, jt & 1, abort_flag)) { fail(ERR_WAIT_P_FULL); good = false; break; }
          mbar_arrive_cluster_relaxed(pfull_addr);
        }
        if (!good) break;
        if (!mbar_wait(BAR_OLOCAL, n_item & 1, abort_flag)) { fail(ERR_WAIT_O_DONE); break; }
        mbar_arrive_cluster_relaxed(ofree_addr);
        ++n_item;
      }
    }
  } else {
    // =============================================== softmax / epilogue: 128 threads, one per TMEM lane
    const int quarter = warp & 3;
    const int ln = quarter * 32 + lane;           // TMEM lane
    const int rl = ln & 63, half = ln >> 6;       // row inside this CTA, key half of the tile
    const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
    const int rg = row0 + rl;
    const int tl = rg / p.HB, hl = rg % p.HB;
    volatile int* fail_word = reinterpret_cast<volatile int*>(smem + OFF_MISC + 16);   // [3], softmax threads only
    if (ln < 3) fail_word[ln] = 0;
    asm volatile("bar.sync 1, 128;" ::: "memory");
    // All 128 threads execute exactly one named barrier per tile and one per item, whatever happens: a
    // thread whose wait expired marks the fail word before the barrier and everybody leaves after it.
    bool ok = !*abort_flag;
    uint32_t jt = 0, n_item = 0, n_ragged = 0;   // tiles / non-empty items / ragged decode tiles of this pair so far
    Walk wk;
    walk_init(p, wk, pair_id, n_pairs, split_state);
    Item it;
    while (ok && walk_next(p, wk, it)) {
    const int head0 = it.head0, t0 = it.t0, nA = it.nA, n_tiles = it.n_tiles;
    const int n_a_lo = it.n_a_lo, n_a_hi = it.n_a_hi, first_lo = it.first_lo;
    const int t_row = t0 + tl;
    const bool row_valid = t_row <= it.t1;
    int n_a_row, bias_rows, first_row;
    DecodeSpan sp = {};
    if (p.decode) { sp = decode_span(p.dl, it.b); n_a_row = n_a_hi; bias_rows = sp.bias_hi; first_row = 0; }
    else { n_a_row = reps_visible(min(t_row, it.len - 1), p.w, p.g); bias_rows = n_a_row; first_row = n_a_row * p.g; }
    float m_ref = -INFINITY, l_sum = 0.f;
    bool all_left = false;                       // every one of the 128 threads left the tile loop at a barrier
    for (int j = 0; j < n_tiles; ++j, ++jt) {
      if (ok) {
        ok = mbar_wait((jt & 1) ? BAR_SFULL1 : BAR_SFULL0, (jt >> 1) & 1, abort_flag);
        if (!ok && lane == 0) fail(ERR_WAIT_S_FULL);
      }
      ok = __all_sync(0xffffffffu, ok);
      const uint32_t stm = tmem + lane_base + ((jt & 1) ? TM_S1 : TM_S0);
      uint32_t sr[2][32];
      float tmax = -INFINITY;
      bool plain = false;
      const bool isA = j < nA;
      const int tile_key0 = isA ? (it.j0 + j) * BN : first_lo + (j - nA) * BN;
      const int key0 = tile_key0 + 64 * half;     // first key of this thread's 64 columns
      if (ok) {
        tc_fence_after();
        tmem_ld32(stm, sr[0]);
        tmem_ld32(stm + 32, sr[1]);
        tmem_wait_ld();
        bool need_mask;
        int lo, hi;
        if (isA) { lo = 0; hi = n_a_row - key0 - 1; need_mask = tile_key0 + BN > n_a_lo; }
        else { lo = first_row - key0; hi = t_row - key0; need_mask = (tile_key0 < n_a_hi * p.g) || (tile_key0 + BN - 1 > t0); }
        const int blim = isA ? bias_rows - key0 : 0;
        bool tile_bias = isA && p.bias_log2 != 0.f;
        if constexpr (RING) {
          need_mask = need_mask || (tile_key0 < sp.inv_hi && tile_key0 + BN > sp.inv_lo);
          tile_bias = tile_bias && tile_key0 < sp.bias_hi && tile_key0 + BN > sp.bias_lo;
        }
        plain = !need_mask && !tile_bias;
        if (plain) {
          // interior tile: the raw products stay in sr, the (positive) scale is applied to the maximum
          // here and folded into the exponent's multiply-add below
          float t0m = -INFINITY, t1m = -INFINITY, t2m = -INFINITY, t3m = -INFINITY;    // four short chains, three-input maxima
#pragma unroll
          for (int i = 0; i < 32; i += 4) {
            t0m = max3(t0m, __uint_as_float(sr[0][i]), __uint_as_float(sr[0][i + 1]));
            t1m = max3(t1m, __uint_as_float(sr[0][i + 2]), __uint_as_float(sr[0][i + 3]));
            t2m = max3(t2m, __uint_as_float(sr[1][i]), __uint_as_float(sr[1][i + 1]));
            t3m = max3(t3m, __uint_as_float(sr[1][i + 2]), __uint_as_float(sr[1][i + 3]));
          }
          tmax = fmaxf(fmaxf(t0m, t1m), fmaxf(t2m, t3m)) * p.scale_log2;
        } else {
          // boundary tile: scale, bias and mask with selects only (per-element branches cost ~25 cycles
          // each here), four short maximum chains
          const float bias = tile_bias ? p.bias_log2 : 0.f;
          const int lo_m = need_mask ? lo : -(1 << 30), hi_m = need_mask ? hi : (1 << 30);
          // ring layout: columns [ilo, ilo + ispan) are condensed tokens still in their rows, [blo, blo + bspan) representatives
          const int ilo = sp.inv_lo - key0, blo = sp.bias_lo - key0;
          const unsigned ispan = (unsigned)(sp.inv_hi - sp.inv_lo), bspan = (unsigned)(sp.bias_hi - sp.bias_lo);
          float tm[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
          for (int q = 0; q < 2; ++q) {
#pragma unroll
            for (int i = 0; i < 32; ++i) {
              const int c = q * 32 + i;
              float s;
              if constexpr (RING) {
                s = fmaf(__uint_as_float(sr[q][i]), p.scale_log2, (unsigned)(c - blo) < bspan ? bias : 0.f);
                s = ((c >= lo_m) & (c <= hi_m) & !((unsigned)(c - ilo) < ispan)) ? s : -INFINITY;
              } else {
                s = fmaf(__uint_as_float(sr[q][i]), p.scale_log2, c < blim ? bias : 0.f);
                s = ((c >= lo_m) & (c <= hi_m)) ? s : -INFINITY;
              }
              sr[q][i] = __float_as_uint(s);
              tm[i & 3] = fmaxf(tm[i & 3], s);
            }
          }
          tmax = fmaxf(fmaxf(tm[0], tm[1]), fmaxf(tm[2], tm[3]));
        }
      } else {
        fail_word[jt & 1] = 1;
      }
      // the two key halves of a row live in different warps: combine their maxima
      red[(jt & 1) * 128 + ln] = tmax;
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (fail_word[jt & 1]) { ok = false; all_left = true; break; }          // uniform over the 128 threads
      tmax = fmaxf(tmax, red[(jt & 1) * 128 + (ln ^ 64)]);
      bool need = false;
      float factor = 1.f;
      if (j == 0) m_ref = tmax;
      else if (tmax > m_ref + RESCALE_THRESHOLD) { need = true; factor = exp2f(m_ref - tmax); }
      // The probabilities depend only on S and the (new) reference maximum: compute and pack them
      // while P V of the previous tile is still running, then wait, rescale O if needed, and store.
      const float m_new = need ? tmax : m_ref;
      const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
      const float e_mul = plain ? p.scale_log2 : 1.f;       // sr holds raw products (plain) or scaled logits
      // scale and row sum work on pairs of fp32 values (one instruction per pair)
      const uint64_t mul2 = pack_f32x2(e_mul, e_mul), sub2 = pack_f32x2(-m_use, -m_use);
      uint64_t rs2 = pack_f32x2(0.f, 0.f);
      uint32_t pk[32];
#pragma unroll
      for (int i = 0; i < 32; ++i) {
        const int c = 2 * i;
        float a0, a1;
        unpack_f32x2(fma_f32x2(pack_f32x2(__uint_as_float(sr[c >> 5][c & 31]), __uint_as_float(sr[(c + 1) >> 5][(c + 1) & 31])), mul2, sub2), a0, a1);
        const float p0 = exp2f(a0), p1 = exp2f(a1);
        pk[i] = pack_bf16x2(p0, p1);
        rs2 = add_f32x2(rs2, pack_f32x2(p0, p1));
      }
      if (j >= 1) {
        // P (one buffer) and O are free once P_{j-1} V_{j-1} has completed
        ok = mbar_wait(BAR_ODONE, (jt - 1) & 1, abort_flag);
        if (!ok && lane == 0) fail(ERR_WAIT_O_DONE);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) continue;                                   // reported at the next tile's barrier
        tc_fence_after();
      }
      if (__any_sync(0xffffffffu, need)) {
#pragma unroll 1                                   // rare path: kept small (the kernel is sensitive to its code size)
        for (int q = 0; q < 8; ++q) {
          uint32_t o[32];
          tmem_ld32(tmem + lane_base + TM_O + q * 32, o);
          tmem_wait_ld();
#pragma unroll
          for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * factor);
          tmem_st32(tmem + lane_base + TM_O + q * 32, o);
        }
        tmem_wait_st();
      }
      if (need) { l_sum *= factor; m_ref = tmax; }
      if (ragged_decode_tile(p, it, j)) {
        // rows >= first_bad of this tile are not part of the sequence: zero them in this CTA's value buffers
        // (their probabilities are exactly 0, but 0 x NaN is not)
        bool vok = true;
#pragma unroll
        for (int kh = 0; kh < 2; ++kh)
          vok = vok && mbar_wait(rank == 0 ? BAR_VFULL(kh) : BAR_VLOC(kh), (rank == 0 ? jt : n_ragged) & 1, abort_flag);
        if (!vok && lane == 0) fail(ERR_WAIT_KV_FULL);
        ok = __all_sync(0xffffffffu, vok);
        if (!ok) continue;                                   // reported at the next tile's barrier
        ++n_ragged;
        const int first_bad = n_a_hi - (it.j0 + j) * BN;     // 1 .. 127
        for (int x = ln; x < (BN - first_bad) * 32; x += 128) {
          const int kr = first_bad + (x >> 5), chunk = (x >> 3) & 3, piece = x & 7;
          const uint32_t a = sV + ((kr >> 6) * 4 + chunk) * VCH + (kr & 63) * 128 + piece * 16;
          asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(a), "r"(0) : "memory");
        }
      }
      const uint32_t prow = sP + half * PCH + rl * 128;
#pragma unroll
      for (int s8 = 0; s8 < 8; ++s8) {             // 16-byte slot s8 holds keys 8*s8 .. 8*s8+7
        const uint32_t a = prow + ((s8 ^ (rl & 7)) << 4);
        asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a), "r"(pk[4 * s8]), "r"(pk[4 * s8 + 1]), "r"(pk[4 * s8 + 2]), "r"(pk[4 * s8 + 3]) : "memory");
      }
      {
        float r0, r1;
        unpack_f32x2(rs2, r0, r1);
        l_sum += r0 + r1;
      }
      fence_proxy_async_smem();                   // P is read by the tensor core (async proxy)
      tc_fence_before();
      mbar_arrive(rank == 0 ? BAR_PFULL : BAR_PLOCAL);
    }
    if (all_left) break;
    // ---- epilogue of the item (a warp whose last wait expired still takes the barrier below)
    if (n_tiles > 0) {
      if (ok) ok = mbar_wait(BAR_OLAST, n_item & 1, abort_flag);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok && lane == 0) fail(ERR_WAIT_O_DONE);
      if (!ok) fail_word[2] = 1;
      // total row sum = sum over both key halves
      red[2 * 128 + ln] = l_sum;
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (fail_word[2]) { ok = false; break; }                 // uniform over the 128 threads
    }
    const float l_tot = n_tiles > 0 ? l_sum + red[2 * 128 + (ln ^ 64)] : 0.f;
    {
      tc_fence_after();
      const float inv = (n_tiles > 0 && l_tot > 0.f) ? 1.f / l_tot : 0.f;
      const size_t orow = ((size_t)it.qbase + t_row) * p.H + head0 + hl;
      bf16* dst = p.out + orow * 512;
#pragma unroll 1                                   // once per item: kept small
      for (int q = 0; q < 8; ++q) {
        uint32_t o[32];
        if (n_tiles > 0) { tmem_ld32(tmem + lane_base + TM_O + q * 32, o); tmem_wait_ld(); }
        else {
#pragma unroll
          for (int i = 0; i < 32; ++i) o[i] = 0;
        }
        if (q == 7 && n_tiles > 0) {
          // every column of O is in registers: the next item may overwrite the accumulator
          tc_fence_before();
          mbar_arrive(rank == 0 ? BAR_OFREE : BAR_OLOCAL);
        }
        // TMEM columns [0,128): output columns 128*half + c ; [128,256): 256 + 128*half + (c-128)
        const int col = (q >> 2) * 256 + 128 * half + (q & 3) * 32;
        if (row_valid && it.slot >= 0) {
          // a part of the unit's key tiles: the unnormalised accumulator goes to the partial slot (fp32)
          float* pd = p.partial + (size_t)it.slot * PARTIAL_FLOATS + (size_t)rg * 512 + col;
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            uint32_t w[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) w[e] = o[8 * v + e];
            st_global_32B(pd + 8 * v, w, true);
          }
        } else if (row_valid) {
          // 32 bytes per store: every lane writes whole sectors of its own row
#pragma unroll
          for (int v = 0; v < 2; ++v) {
            uint32_t w[8];
#pragma unroll
            for (int e = 0; e < 8; ++e)
              w[e] = pack_bf16x2(__uint_as_float(o[16 * v + 2 * e]) * inv, __uint_as_float(o[16 * v + 2 * e + 1]) * inv);
            st_global_32B(dst + col + 16 * v, w, p.out_wide != 0);
          }
        }
      }
      if (row_valid && half == 0 && it.slot >= 0) {
        float* ml = p.partial + (size_t)it.slot * PARTIAL_FLOATS + 128 * 512 + 2 * rg;
        ml[0] = m_ref; ml[1] = l_tot;
      } else if (p.lse && row_valid && half == 0)
        p.lse[orow] = (n_tiles > 0 && l_tot > 0.f) ? (m_ref + log2f(l_tot)) * 0.6931471805599453f : -INFINITY;
    }
    if (n_tiles > 0) ++n_item;
    }   // items
    tc_fence_before();
  }
  // ---- teardown
  if (*abort_flag && (warp == 0 || warp == 6) && lane == 0) {
    const long long t0c = clock64();
    while (clock64() - t0c < 2000000ll) { __nanosleep(1000); }
  }
  __syncthreads();
  cluster_sync_all();                              // the peer is done with this CTA's memory and TMEM
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc_pair(tmem, TM_COLS);
  }
}

// Split decode, second step: one CTA of 128 threads per (unit, head): four output columns per thread.  Units whose
// key tiles were all taken by one pair are complete already; units without any valid row get zeros (lse = -inf);
// the others are merged from their partial results in range order:
//     out = sum_s O_s 2^(m_s - M) / sum_s l_s 2^(m_s - M),   M = max_s m_s.
__global__ void __launch_bounds__(128) decode_combine_kernel(const Tc2Params p, int n_pairs) {
  const int u = blockIdx.x / p.HB, hl = blockIdx.x % p.HB, lane = threadIdx.x & 31;
  const int n_units = p.B * p.n_head_blocks;
  // every warp repeats the scan over the units (chunks of 32, prefix sums by shuffles): tiles before unit u, slots before it
  int total = 0;
  for (int u0 = 0; u0 < n_units; u0 += 32) total += __reduce_add_sync(0xffffffffu, u0 + lane < n_units ? unit_tiles(p, u0 + lane) : 0);
  const int q = total > 0 ? (total + n_pairs - 1) / n_pairs : 1;
  int off = 0, slot_base = 0, my_slot = 0, n_seg = 0;
  for (int u0 = 0; u0 <= u; u0 += 32) {
    const int nn = u0 + lane < n_units ? unit_tiles(p, u0 + lane) : 0;
    int incl = nn;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const int t = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += t; }
    const int r = nn > 0 ? unit_ranges(off + incl - nn, nn, q) : 0;
    int rincl = r;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) { const int t = __shfl_up_sync(0xffffffffu, rincl, o); if (lane >= o) rincl += t; }
    if (u < u0 + 32) {
      const int src = u - u0;
      n_seg = __shfl_sync(0xffffffffu, r, src);
      my_slot = slot_base + __shfl_sync(0xffffffffu, rincl - r, src);
    }
    off += __shfl_sync(0xffffffffu, incl, 31);
    slot_base += __shfl_sync(0xffffffffu, rincl, 31);
  }
  if (n_seg == 1) return;
  const int b = u / p.n_head_blocks, head0 = (u % p.n_head_blocks) * p.HB;
  const int c4 = threadIdx.x;                               // columns 4 c4 .. 4 c4 + 3
  const size_t orow = (size_t)b * p.H + head0 + hl;         // q_len = 1
  const float* base = p.partial + (size_t)my_slot * PARTIAL_FLOATS;
  float M = -INFINITY;
  for (int sgm = 0; sgm < n_seg; ++sgm) M = fmaxf(M, base[(size_t)sgm * PARTIAL_FLOATS + 128 * 512 + 2 * hl]);
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  float Lsum = 0.f;
#pragma unroll 4
  for (int sgm = 0; sgm < n_seg; ++sgm) {
    const float* ps = base + (size_t)sgm * PARTIAL_FLOATS;
    const float ms = ps[128 * 512 + 2 * hl], ls = ps[128 * 512 + 2 * hl + 1];
    const float4 o = *reinterpret_cast<const float4*>(ps + (size_t)hl * 512 + 4 * c4);
    const float f = (ms == -INFINITY) ? 0.f : exp2f(ms - M);
    acc.x = fmaf(o.x, f, acc.x); acc.y = fmaf(o.y, f, acc.y); acc.z = fmaf(o.z, f, acc.z); acc.w = fmaf(o.w, f, acc.w);
    Lsum = fmaf(ls, f, Lsum);
  }
  const float inv = Lsum > 0.f ? 1.f / Lsum : 0.f;
  uint2 w;
  w.x = pack_bf16x2(acc.x * inv, acc.y * inv); w.y = pack_bf16x2(acc.z * inv, acc.w * inv);
  *reinterpret_cast<uint2*>(p.out + orow * 512 + 4 * c4) = w;
  if (p.lse && c4 == 0) p.lse[orow] = Lsum > 0.f ? (M + log2f(Lsum)) * 0.6931471805599453f : -INFINITY;
}

// ----------------------------------------------------------------------------------- host
bool make_tensor_map_3d(CUtensorMap* map, const void* ptr, int d, int heads, long long rows, int box_heads, int box_rows);
bool make_tensor_map_chunks(CUtensorMap* map, const void* ptr, int chunks, long long rows, int box_rows, int box_chunks);

// Entries of a ragged batch behind the sequence table: one (sequence, tile) pair per token tile.
size_t attn_tc2_ragged_workspace_bytes(int batch, int longest, int n_q_heads) {
  const int TB = n_q_heads >= 128 ? 1 : 128 / n_q_heads;
  return seq_table_bytes(batch) + (size_t)batch * ((size_t)(longest + TB - 1) / TB) * sizeof(int2);
}

bool attn_tc2_supported(const AttnProblem& a) {
  if (a.variant != LCA_VARIANT_MLA || a.d_sem != 512 || a.d_pos != 64 || a.n_kv_heads != 1) return false;
  const int H = a.n_q_heads;
  if (H >= 128) return H % 128 == 0;
  return H >= 1 && (128 % H) == 0;      // each CTA of the pair takes whole tokens
}

// CTA pairs that can be resident at once on the current device (one CTA per SM by shared memory): the size
// of the persistent grid.  Asked from the occupancy calculator once per device; half the SM count otherwise.
static int resident_pairs();
// Split decode is used while the (sequence, head block) units number at most half the resident CTA pairs: cutting the
// line of key tiles into equal ranges costs a partial result per cut (256 KB written and read again) and a second
// launch, about 30 us in all at 64 sequences x 40 tiles, which only pays where whole units would leave more than
// half of the pairs idle.  The workspace holds one partial result per unit and per pair at most.
static bool decode_splits(int batch, int n_q_heads) {
  const int units = batch * (n_q_heads >= 128 ? n_q_heads / 128 : 1);
  return 2 * units <= resident_pairs();
}
size_t attn_tc2_decode_workspace_bytes(int batch, int n_q_heads) {
  if (!decode_splits(batch, n_q_heads)) return 0;
  const size_t units = (size_t)batch * (n_q_heads >= 128 ? n_q_heads / 128 : 1);
  return (units + (size_t)resident_pairs()) * PARTIAL_FLOATS * sizeof(float);
}

static int resident_pairs() {
  static int cached[64];
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) dev = 0;
  if (cached[dev] > 0) return cached[dev];
  int n = 0;
  cudaLaunchConfig_t cfg;
  memset(&cfg, 0, sizeof(cfg));
  cfg.gridDim = dim3(2 * 1024); cfg.blockDim = dim3(pair::THREADS); cfg.dynamicSmemBytes = pair::SMEM_BYTES;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeClusterDimension;
  attr.val.clusterDim.x = 2; attr.val.clusterDim.y = 1; attr.val.clusterDim.z = 1;
  cfg.attrs = &attr; cfg.numAttrs = 1;
  if (cudaFuncSetAttribute(attn_tc2_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, pair::SMEM_BYTES) != cudaSuccess ||
      cudaOccupancyMaxActiveClusters(&n, attn_tc2_kernel<false>, &cfg) != cudaSuccess || n <= 0) {
    cudaGetLastError();
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 2) sms = 148;   // no device: a B200
    n = sms / 2;
  }
  cached[dev] = n;
  return n;
}

int attn_tc2_launch(const AttnProblem& a) {
  using namespace pair;
  if (!attn_tc2_supported(a)) return LCA_ERR_UNSUPPORTED_SHAPE;
  Tc2Params p;
  memset(&p, 0, sizeof(p));
  const int H = a.n_q_heads;
  p.HB = H >= 128 ? 128 : H;
  p.TB = 128 / p.HB;
  p.B = a.batch; p.q_len = a.q_len; p.H = H; p.L = a.seq_len; p.g = a.group_size; p.w = a.window;
  p.cap = a.cache_row_capacity; p.decode = a.decode;
  p.dl = DecodeLayout{a.cache_rows, a.ring_n_rep, a.ring_n_tok, a.cache_row_capacity, a.n_rep_bias, a.window + a.group_size, a.group_size};
  p.n_tok_tiles = (a.q_len + p.TB - 1) / p.TB;
  p.n_head_blocks = H >= 128 ? H / 128 : 1;
  p.n_items = (long long)p.n_tok_tiles * p.n_head_blocks * a.batch;
  long long qrows = (long long)a.batch * a.q_len, krows = (long long)a.batch * a.seq_len,
            crows = (long long)a.batch * a.cache_row_capacity;
  if (a.h_tok_off) {
    // ragged batch: one entry per (sequence, token tile), heaviest (most key tiles) first, uploaded behind the table
    std::vector<int2> entries;
    std::vector<int> weight;
    for (int b = 0; b < a.batch; ++b) {
      const int len = a.h_tok_off[b + 1] - a.h_tok_off[b];
      for (int tile = 0; tile * p.TB < len; ++tile) {
        const int t0 = tile * p.TB, t1 = std::min(t0 + p.TB, len) - 1;
        const int n_lo = reps_visible(t0, p.w, p.g), n_hi = reps_visible(t1, p.w, p.g);
        entries.push_back(make_int2(b, tile));
        weight.push_back((n_hi + BN - 1) / BN + (t1 - n_lo * p.g + BN) / BN);
      }
    }
    std::vector<int> order(entries.size());
    for (size_t i = 0; i < order.size(); ++i) order[i] = (int)i;
    std::stable_sort(order.begin(), order.end(), [&](int x, int y) { return weight[x] > weight[y]; });
    std::vector<int2> sorted(entries.size());
    for (size_t i = 0; i < order.size(); ++i) sorted[i] = entries[order[i]];
    int2* d_entries = reinterpret_cast<int2*>(static_cast<char*>(a.ws) + seq_table_bytes(a.batch));
    if (!sorted.empty() &&
        cudaMemcpyAsync(d_entries, sorted.data(), sorted.size() * sizeof(int2), cudaMemcpyHostToDevice, a.stream) != cudaSuccess)
      return LCA_ERR_CUDA;
    p.entries = d_entries; p.tab = a.tab;
    p.n_items = (long long)sorted.size() * p.n_head_blocks;
    qrows = krows = a.h_tok_off[a.batch];
    crows = a.h_cache_off[a.batch];
  }
  p.scale_log2 = a.softmax_scale * 1.4426950408889634f;
  p.bias_log2 = a.rep_logit_bias * 1.4426950408889634f;
  p.out = (bf16*)a.out; p.lse = a.lse;
  p.out_wide = (reinterpret_cast<uintptr_t>(a.out) & 31u) == 0;
  const int hbc = p.HB >= 64 ? 64 : p.HB, tbc = 64 / hbc;
  bool ok = make_tensor_map_3d(&p.q_sem, a.q_sem, 512, H, qrows, hbc, tbc);
  ok = ok && make_tensor_map_3d(&p.q_pos, a.q_pos, 64, H, qrows, hbc, tbc);
  ok = ok && make_tensor_map_3d(&p.k_pos, a.kv_pos, 64, 1, krows, 1, 64);
  ok = ok && make_tensor_map_3d(&p.c_pos, a.cache_pos, 64, 1, crows, 1, 64);
  ok = ok && make_tensor_map_chunks(&p.k_sem, a.kv_sem, 8, krows, 64, KBOX);
  ok = ok && make_tensor_map_chunks(&p.c_sem, a.cache_sem, 8, crows, 64, KBOX);
  ok = ok && make_tensor_map_chunks(&p.k_val, a.kv_sem, 8, krows, 64, VBOX);
  ok = ok && make_tensor_map_chunks(&p.c_val, a.cache_sem, 8, crows, 64, VBOX);
  if (!ok) return LCA_ERR_CUDA;
  const bool ring = a.decode && a.ring_n_tok != nullptr;
  if (cudaFuncSetAttribute(ring ? attn_tc2_kernel<true> : attn_tc2_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           SMEM_BYTES) != cudaSuccess)
    return LCA_ERR_CUDA;
  long long n_pairs = p.n_items < resident_pairs() ? p.n_items : resident_pairs();
  if (n_pairs <= 0) return LCA_OK;
  if (a.decode && decode_splits(a.batch, H)) {
    // every pair takes an equal share of all key tiles; ranges that cut a unit leave partial results in the workspace
    if (a.ws_bytes < attn_tc2_decode_workspace_bytes(a.batch, H)) return LCA_ERR_WORKSPACE_TOO_SMALL;
    if (!a.ws || (reinterpret_cast<uintptr_t>(a.ws) & 31u)) return LCA_ERR_MISALIGNED;
    p.split = 1; p.partial = static_cast<float*>(a.ws);
    n_pairs = resident_pairs();
  }
  dim3 grid((unsigned)(2 * n_pairs));
  if (ring) attn_tc2_kernel<true><<<grid, THREADS, SMEM_BYTES, a.stream>>>(p);
  else attn_tc2_kernel<false><<<grid, THREADS, SMEM_BYTES, a.stream>>>(p);
  note_launch();
  if (p.split) {
    decode_combine_kernel<<<dim3((unsigned)(a.batch * p.n_head_blocks * p.HB)), 128, 0, a.stream>>>(p, (int)n_pairs);
    note_launch();
  }
  return cudaGetLastError() == cudaSuccess ? LCA_OK : LCA_ERR_CUDA;
}

int attn_tc2_take_status() {
  int st = 0;
  if (cudaMemcpyFromSymbol(&st, g_tc2_status, sizeof(int)) != cudaSuccess) return -1;
  if (st != 0) {
    int zero = 0;
    cudaMemcpyToSymbol(g_tc2_status, &zero, sizeof(int));
  }
  return st;
}

}  // namespace lca
