// MLA-shaped (d_c = 512, d_R = 64) attention over the condensed context on CTA pairs.
//
// The absorbed MLA shape does not fit one SM: 128 query rows x 512 fp32 output columns is the
// whole of tensor memory, and a 128 x 576 bf16 query tile is 144 KB of shared memory.  So two
// CTAs of a cluster share one tile of 128 query rows (TB tokens x HB heads) and issue
// tcgen05.mma with cta_group::2 and M = 128: each CTA owns 64 of the rows, and a 64 x N result
// is laid out over all 128 tensor-memory lanes (lanes 0-63 hold columns 0..N/2-1, lanes 64-127
// hold columns N/2..N-1).  With N = 256 such an instruction keeps the whole data path of both
// SMs busy (N = 128 runs at half rate), so both contractions use N = 256:
//   S = Q K^T  per tile of 256 keys: the B operand is split by keys, each CTA stages 128 keys
//              x 576 columns as nine 16 KB chunks of 64 columns;
//   O += P V   per 64 keys and 256 output columns: the B operand is split by output columns,
//              each CTA stages 64 keys x 128 columns (16 KB) per group of four instructions.
// At full tensor rate these blocks amount to ~56 bytes per clock and SM, more than a TMA unit
// moves with tiled copies of a row-major tensor (35-40 B/clk measured) -- the fill of shared
// memory, not the tensor core, bounds this kernel.  So a small pre-pass (retile_kernel) rewrites
// the key/value stream once into "images": 8 KB blocks of 64 keys x 64 columns already in the
// 128-byte-swizzled order the tensor core reads, stored [column chunk][key block] so that every
// block the main kernel needs is one or two contiguous pieces fetched with plain bulk copies
// (cp.async.bulk, ~46 B/clk measured for 16 KB pieces).  Key images are stored [column chunk]
// [key block] (a chunk of 128 keys is 16 KB contiguous), value images [key block][column chunk]
// (64 keys x 128 columns are 16 KB contiguous).  All blocks travel through ONE ring of 16 KB
// slots in exactly the order in which the MMA warp consumes them (S of tile j+1, then P V of
// tile j).
//
// Signalling inside the pair.  Warp 1 of the even CTA issues every MMA.  What the tensor core
// signals (tcgen05.commit, multicast to both CTAs) costs no thread time.  A thread's arrive on
// a barrier of the OTHER CTA, however, stalls that thread for about a microsecond, so no
// producer or softmax thread ever does one: every thread arrives on barriers of its own CTA,
// and the lanes of warp 1 of the odd CTA (idle otherwise) each watch one of those barriers and
// forward its completions to a twin barrier in the even CTA.
//
// Tensor memory: two S buffers of 128 columns and O in 256 columns.  Softmax threads (one per
// lane) take the row maximum over the two key halves through shared memory, write P as bf16
// into a 128-byte-swizzled shared tile (the A operand of P V) in four chunks of 64 keys, each
// with its own full / free barrier, and rescale O only when the running maximum grew by more
// than 2^8.
//
// A CTA pair is persistent: it walks query tiles from the heaviest (latest tokens) down, and the
// query tile of the next work item is loaded as soon as the last S of the current one is done,
// so the epilogue of one item overlaps the first products of the next.
// Every wait is bounded; on expiry the CTA records a code in a global status word, drains and
// returns.
#include <cstring>

#include "lca_common.cuh"
#include "tc_common.cuh"

namespace lca {
using namespace tc;

static __device__ int g_tc2_status = 0;

#ifdef LCA_TC2_TRACE
// Debug build only: clock64 stamps of the first CTA pair, per key tile and pipeline event.
static __device__ long long g_trace[2 * 128 * 24];
#define TRACE(slot, j) do { if (blockIdx.x < 2 && (j) < 128) g_trace[((int)rank * 128 + (int)(j)) * 24 + (slot)] = clock64(); } while (0)
#define TRACE_ADD(slot, j, v) do { if (blockIdx.x < 2 && (j) < 128) g_trace[((int)rank * 128 + (int)(j)) * 24 + (slot)] += (v); } while (0)
#else
#define TRACE(slot, j) do { } while (0)
#define TRACE_ADD(slot, j, v) do { } while (0)
#endif

namespace pair {
constexpr int BN = 256;                 // keys per S tile (128 per CTA)
constexpr int NKC = 9;                  // 64-column key chunks: 8 latent + 1 rope
constexpr int NPC = 4;                  // 64-key chunks of P / value blocks per tile
constexpr int BOX = 64 * 128;           // bytes of one image / TMA box: 64 rows x 64 bf16
constexpr int SLOT = 2 * BOX;           // ring slot: K chunk [128 keys x 64 cols] or V block [64 keys x 128 cols]
constexpr int NSLOT = 7;
constexpr int BLOCKS_PER_TILE = NKC + 2 * NPC;
constexpr int QCH = BOX, PCH = BOX;
constexpr int Q_BYTES = NKC * QCH, P_BYTES = NPC * PCH;
constexpr int OFF_Q = 0, OFF_RING = OFF_Q + Q_BYTES, OFF_P = OFF_RING + NSLOT * SLOT;
constexpr int OFF_BAR = OFF_P + P_BYTES;
constexpr int OFF_MISC = OFF_BAR + 512, OFF_RED = OFF_BAR + 1024;
constexpr int SMEM_BYTES = OFF_RED + 3 * 128 * 4;
constexpr int TM_S0 = 0, TM_S1 = 128, TM_O = 256, TM_COLS = 512;
constexpr int THREADS = 192;            // warps: 0 copy producer, 1 MMA + TMEM (odd CTA: relay), 2-5 softmax
constexpr int PAD_KEY_BLOCKS = 4;       // a tile may start up to 255 keys before the end of its stream
constexpr float RESCALE_THRESHOLD = 8.0f;
static_assert(SMEM_BYTES <= 232448, "shared memory budget of one SM");
}  // namespace pair

struct Tc2Params {
  CUtensorMap q_sem, q_pos;       // queries, box of 64 rows
  const unsigned char* images;    // retiled key/value stream, see retile_kernel
  long long seq_image_bytes;      // bytes of one sequence's images (token keys, rep keys, token values, rep values)
  int nkb_tok, nkb_rep;           // 64-key blocks per column chunk in the two image sets
  bf16* out; float* lse;
  int B, q_len, H, L, g, w, cap;
  int HB, TB, n_tok_tiles, n_head_blocks;
  long long n_items;              // query tiles x head blocks x batch
  float scale_log2, bias_log2;
};

// ------------------------------------------------------------------------------- retiling
// images of sequence b: key images [9 chunks][nkb_tok key blocks][8 KB] from kv_sem / kv_pos, then
// [9][nkb_rep][8 KB] from the first m rows of cache_sem / cache_pos, then the value images
// [nkb_tok][8 chunks][8 KB] and [nkb_rep][8][8 KB] (the same blocks of the latent columns in
// the other order).  Inside a block, key r
// (0..63) occupies bytes [128 r, 128 r + 128) and its 16-byte piece ch sits at position
// ch ^ (r & 7): the layout a TMA box with 128-byte swizzle would have.  Keys past the end of the
// stream are zero.  grid (key blocks, 9, 2 * B), 512 threads = 64 keys x 8 pieces.
struct RetileArgs {
  const bf16* kv_sem; const bf16* kv_pos; const bf16* cache_sem; const bf16* cache_pos;
  unsigned char* images; long long seq_image_bytes;
  int L, m, cap, nkb_tok, nkb_rep;
};
__global__ void __launch_bounds__(512) retile_kernel(RetileArgs a) {
  const int kb = blockIdx.x, c = blockIdx.y, b = blockIdx.z >> 1, rep = blockIdx.z & 1;
  const int nkb = rep ? a.nkb_rep : a.nkb_tok;
  if (kb >= nkb) return;
  const int r = threadIdx.x >> 3, ch = threadIdx.x & 7;
  const long long key = (long long)kb * 64 + r;
  const int n_keys = rep ? a.m : a.L;
  uint4 v = make_uint4(0u, 0u, 0u, 0u);
  if (key < n_keys) {
    const long long row = (long long)b * (rep ? a.cap : a.L) + key;
    const bf16* src = c < 8 ? (rep ? a.cache_sem : a.kv_sem) + row * 512 + c * 64 + ch * 8
                            : (rep ? a.cache_pos : a.kv_pos) + row * 64 + ch * 8;
    v = *reinterpret_cast<const uint4*>(src);
  }
  unsigned char* seq = a.images + (long long)b * a.seq_image_bytes;
  const int off = r * 128 + ((ch ^ (r & 7)) << 4);
  unsigned char* kdst = seq + ((long long)(rep ? 9 * a.nkb_tok : 0) + (long long)c * nkb + kb) * pair::BOX;
  *reinterpret_cast<uint4*>(kdst + off) = v;
  if (c < 8) {
    unsigned char* vdst = seq + (9ll * (a.nkb_tok + a.nkb_rep) + (long long)(rep ? 8 * a.nkb_tok : 0) + (long long)kb * 8 + c) * pair::BOX;
    *reinterpret_cast<uint4*>(vdst + off) = v;
  }
}

// One work item = one tile of 128 query rows; identical arithmetic in every role of both CTAs.
struct Item {
  int b, head0, t0, t1;
  int n_a_lo, n_a_hi, first_lo, nA, n_tiles;
};
__device__ __forceinline__ Item make_item(const Tc2Params& p, long long idx) {
  Item it;
  // heaviest query tiles (latest tokens) first; batch and head block vary fastest
  const long long per_tile = (long long)p.n_head_blocks * p.B;
  const int tile = p.n_tok_tiles - 1 - (int)(idx / per_tile);
  const int rem = (int)(idx % per_tile);
  it.b = rem / p.n_head_blocks;
  it.head0 = (rem % p.n_head_blocks) * p.HB;
  it.t0 = tile * p.TB;
  it.t1 = min(it.t0 + p.TB, p.q_len) - 1;
  it.n_a_lo = reps_visible(it.t0, p.w, p.g);
  it.n_a_hi = reps_visible(it.t1, p.w, p.g);
  it.first_lo = (it.n_a_lo * p.g) & ~63;          // local tiles start on an image boundary
  it.nA = (it.n_a_hi + pair::BN - 1) / pair::BN;
  it.n_tiles = it.nA + (it.t1 - it.first_lo + pair::BN) / pair::BN;
  return it;
}

__device__ __forceinline__ void bulk_load(uint32_t smem_dst, const void* src, uint32_t bytes, uint32_t bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(pair::THREADS, 1)
attn_tc2_kernel(const __grid_constant__ Tc2Params p) {
  using namespace pair;
  extern __shared__ __align__(1024) unsigned char smem[];
  const uint32_t base = smem_u32(smem);
  const uint32_t sQ = base + OFF_Q, sRing = base + OFF_RING, sP = base + OFF_P;
  const uint32_t bars = base + OFF_BAR;
  // Barriers that threads of both CTAs arrive on live in the even CTA (rank 0), which issues
  // every MMA; barriers signalled by tcgen05.commit exist in both CTAs.
  const uint32_t BAR_QFULL = bars, BAR_QFREE = bars + 8, BAR_ODONE = bars + 16, BAR_OFREE = bars + 24,
                 BAR_OREADY = bars + 48 + 24 * NSLOT + 16 * NPC, BAR_OLAST = BAR_OREADY + 8,
                 BAR_OREADY_PEER = BAR_OREADY + 16, BAR_OFREE_PEER = BAR_OREADY + 24;
  auto BAR_PFULL_PEER = [&](int c) { return BAR_OREADY + 32 + 8 * c; };   // NPC, even CTA: the odd CTA's P chunk is written
  auto BAR_SFULL = [&](int i) { return bars + 32 + 8 * i; };              // 2
  auto BAR_FULL = [&](int s) { return bars + 48 + 8 * s; };               // NSLOT, own copies landed
  auto BAR_EMPTY = [&](int s) { return bars + 48 + 8 * NSLOT + 8 * s; };  // NSLOT
  auto BAR_PEER = [&](int s) { return bars + 48 + 16 * NSLOT + 8 * s; };  // NSLOT, even CTA: the odd CTA's copies landed
  auto BAR_PFULL = [&](int c) { return bars + 48 + 24 * NSLOT + 8 * c; };             // NPC
  auto BAR_PFREE = [&](int c) { return bars + 48 + 24 * NSLOT + 8 * NPC + 8 * c; };   // NPC
  static_assert(80 + 24 * NSLOT + 24 * NPC <= 512, "barrier area");
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(smem + OFF_MISC);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(smem + OFF_MISC + 4);
  volatile float* red = reinterpret_cast<volatile float*>(smem + OFF_RED);    // [3][128]

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const long long pair_id = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

  if (threadIdx.x == 0) {
    mbar_init(BAR_QFULL, 1); mbar_init(BAR_QFREE, 1); mbar_init(BAR_ODONE, 1); mbar_init(BAR_OFREE, 128);
    mbar_init(BAR_OREADY, 128); mbar_init(BAR_OLAST, 1); mbar_init(BAR_OREADY_PEER, 1); mbar_init(BAR_OFREE_PEER, 1);
    mbar_init(BAR_SFULL(0), 1); mbar_init(BAR_SFULL(1), 1);
    for (int s = 0; s < NSLOT; ++s) { mbar_init(BAR_FULL(s), 1); mbar_init(BAR_EMPTY(s), 1); mbar_init(BAR_PEER(s), 1); }
    for (int c = 0; c < NPC; ++c) { mbar_init(BAR_PFULL(c), 64); mbar_init(BAR_PFREE(c), 1); mbar_init(BAR_PFULL_PEER(c), 1); }
    *abort_flag = (base & 1023u) ? 1 : 0;
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc_pair(smem_u32((const void*)tmem_slot), TM_COLS);
    tmem_relinquish_pair();
  }
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

  const int row0 = 64 * (int)rank;                 // rows of this CTA inside the pair tile

  if (warp == 0) {
    // =============================================== producer: Q of each item, then the ring
    if (lane == 0 && !*abort_flag) {
      const uint32_t q_bar = mapa_u32(BAR_QFULL, 0);
      uint32_t ring_i = 0;                          // blocks pushed so far
      uint32_t n_item = 0;
      bool good = true;
      auto push = [&](const unsigned char* src) -> bool {        // one block = 16 KB contiguous
        const uint32_t s = ring_i % NSLOT, round = ring_i / NSLOT;
#ifdef LCA_TC2_TRACE
        const long long tw = clock64();
#endif
        if (!mbar_wait(BAR_EMPTY(s), (round & 1) ^ 1, abort_flag)) { fail(ERR_WAIT_KV_EMPTY); return false; }
#ifdef LCA_TC2_TRACE
        TRACE_ADD(16, ring_i / BLOCKS_PER_TILE, clock64() - tw);          // producer: cycles waiting for a free slot
        if (ring_i % BLOCKS_PER_TILE == 0) TRACE(17, ring_i / BLOCKS_PER_TILE);   // first block of the tile issued
        if (ring_i % BLOCKS_PER_TILE == 9) TRACE(18, ring_i / BLOCKS_PER_TILE);   // first value block issued
#endif
        mbar_expect_tx(BAR_FULL(s), SLOT);
        bulk_load(sRing + s * SLOT, src, SLOT, BAR_FULL(s));
        ++ring_i;
        return true;
      };
      for (long long idx = pair_id; good && idx < p.n_items; idx += n_pairs, ++n_item) {
        const Item it = make_item(p, idx);
        // the query tile may be replaced once the last S of the previous item has been computed
        if (!mbar_wait(BAR_QFREE, (n_item & 1) ^ 1, abort_flag)) { fail(ERR_WAIT_Q); break; }
        if (rank == 0) mbar_expect_tx(BAR_QFULL, 2 * Q_BYTES);
        const int qtok = it.b * p.q_len + it.t0 + row0 / p.HB, qhead = it.head0 + row0 % p.HB;
        for (int c = 0; c < 8; ++c) tma_load_3d_pair(sQ + c * QCH, &p.q_sem, c * 64, qhead, qtok, q_bar);
        tma_load_3d_pair(sQ + 8 * QCH, &p.q_pos, 0, qhead, qtok, q_bar);
        const unsigned char* seq = p.images + (long long)it.b * p.seq_image_bytes;
        const long long vbase = 9ll * (p.nkb_tok + p.nkb_rep);     // value images follow the key images
        auto push_keys = [&](int j) -> bool {      // nine chunks of this CTA's 128 keys
          const bool isA = j < it.nA;
          const int nkb = isA ? p.nkb_rep : p.nkb_tok;
          const int kb = (isA ? j * BN : it.first_lo + (j - it.nA) * BN) / 64 + 2 * (int)rank;
          for (int c = 0; c < NKC; ++c)
            if (!push(seq + ((long long)(isA ? 9 * p.nkb_tok : 0) + (long long)c * nkb + kb) * BOX)) return false;
          return true;
        };
        auto push_values = [&](int j) -> bool {    // per 64 keys: this CTA's 128 columns of each 256
          const bool isA = j < it.nA;
          const int kb0 = (isA ? j * BN : it.first_lo + (j - it.nA) * BN) / 64;
          for (int c = 0; c < NPC; ++c)
            for (int n2 = 0; n2 < 2; ++n2)
              if (!push(seq + (vbase + (long long)(isA ? 8 * p.nkb_tok : 0) + (long long)(kb0 + c) * 8 + 4 * n2 + 2 * (int)rank) * BOX)) return false;
          return true;
        };
        good = push_keys(0);
        for (int j = 0; good && j < it.n_tiles; ++j) {
          if (j + 1 < it.n_tiles) good = push_keys(j + 1);
          if (good) good = push_values(j);
        }
      }
    }
  } else if (warp == 1 && rank == 1) {
    // =============================================== odd CTA: forward barrier completions to the even CTA
    // lane l < NSLOT: ring slot l is full;  NSLOT..NSLOT+3: P chunk written;  then: O looked at; O read.
    if (lane < NSLOT + NPC + 2 && !*abort_flag) {
      long long n_tiles_total = 0, n_items_mine = 0;
      for (long long idx = pair_id; idx < p.n_items; idx += n_pairs) { n_tiles_total += make_item(p, idx).n_tiles; ++n_items_mine; }
      uint32_t local, remote;
      long long count;
      bool relaxed = false;
      if (lane < NSLOT) {
        local = BAR_FULL(lane); remote = BAR_PEER(lane);
        const long long blocks = n_tiles_total * BLOCKS_PER_TILE;
        count = blocks > lane ? (blocks - lane + NSLOT - 1) / NSLOT : 0;
        relaxed = true;          // the data was written by the copy engine, not by threads
      } else if (lane < NSLOT + NPC) {
        local = BAR_PFULL(lane - NSLOT); remote = BAR_PFULL_PEER(lane - NSLOT); count = n_tiles_total;
      } else if (lane == NSLOT + NPC) {
        local = BAR_OREADY; remote = BAR_OREADY_PEER; count = n_tiles_total;
      } else {
        local = BAR_OFREE; remote = BAR_OFREE_PEER; count = n_items_mine;
      }
      remote = mapa_u32(remote, 0);
      for (long long k = 0; k < count; ++k) {
        if (!mbar_wait(local, (uint32_t)(k & 1), abort_flag)) { fail(ERR_WAIT_PEER); break; }
        if (relaxed) asm volatile("mbarrier.arrive.relaxed.cluster.shared::cluster.b64 _, [%0];" ::"r"(remote) : "memory");
        else mbar_arrive_cluster(remote);
      }
    }
  } else if (warp == 1) {
    // =============================================== MMA issuer (even CTA)
    if (lane == 0 && !*abort_flag) {
      constexpr uint32_t IDESC = umma_idesc_bf16(128, 256, false, false);      // S: K-major A and B
      constexpr uint32_t IDESC_PV = umma_idesc_bf16(128, 256, false, true);    // PV: B is MN-major
      uint32_t ring_i = 0, n_item = 0, s_count = 0, pv_count = 0;
      bool ok = true;
#ifdef LCA_TC2_TRACE
      long long trace_wait = 0;
#endif
      auto wait_slot = [&]() -> uint32_t {
        const uint32_t s = ring_i % NSLOT, round = ring_i / NSLOT;
#ifdef LCA_TC2_TRACE
        const long long tw = clock64();
#endif
        if (!mbar_wait(BAR_FULL(s), round & 1, abort_flag) || !mbar_wait(BAR_PEER(s), round & 1, abort_flag)) {
          fail(ERR_WAIT_KV_FULL); ok = false;
        }
#ifdef LCA_TC2_TRACE
        trace_wait += clock64() - tw;
#endif
        tc_fence_after();
        ++ring_i;
        return s;
      };
      auto issue_s = [&]() {                       // S(s_count) = Q K^T into buffer s_count & 1
        const uint32_t stm = tmem + ((s_count & 1) ? TM_S1 : TM_S0);
        TRACE(0, s_count);
#ifdef LCA_TC2_TRACE
        trace_wait = 0;
#endif
        for (int c = 0; ok && c < NKC; ++c) {
          const uint32_t s = wait_slot();
          if (!ok) break;
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            const uint64_t ad = umma_desc_sw128(sQ + c * QCH + k * 32, 16, 1024);
            const uint64_t bd = umma_desc_sw128(sRing + s * SLOT + k * 32, 16, 1024);
            umma_ss_pair(stm, ad, bd, IDESC, (c > 0 || k > 0) ? 1u : 0u);
          }
          umma_commit_pair(BAR_EMPTY(s), 3);
        }
        if (ok) umma_commit_pair(BAR_SFULL(s_count & 1), 3);
        TRACE(1, s_count);
#ifdef LCA_TC2_TRACE
        TRACE_ADD(7, s_count, trace_wait);
#endif
        ++s_count;
      };
      auto issue_pv = [&](bool first_of_item, bool last_of_item) {    // O += P V for tile pv_count
        // every softmax thread of the pair has finished looking at (and possibly rescaling) O
        TRACE(2, pv_count);
        if (!mbar_wait(BAR_OREADY, pv_count & 1, abort_flag) || !mbar_wait(BAR_OREADY_PEER, pv_count & 1, abort_flag)) {
          fail(ERR_WAIT_P_FULL); ok = false; return;
        }
        TRACE(3, pv_count);
#ifdef LCA_TC2_TRACE
        trace_wait = 0;
#endif
        for (int c = 0; ok && c < NPC; ++c) {
          if (!mbar_wait(BAR_PFULL(c), pv_count & 1, abort_flag) || !mbar_wait(BAR_PFULL_PEER(c), pv_count & 1, abort_flag)) {
            fail(ERR_WAIT_P_FULL); ok = false; break;
          }
          if (c == 0) TRACE(4, pv_count);
          if (c == 3) TRACE(5, pv_count);
          tc_fence_after();
          for (int n2 = 0; ok && n2 < 2; ++n2) {
            const uint32_t s = wait_slot();
            if (!ok) break;
#pragma unroll
            for (int k = 0; k < 4; ++k) {
              const uint64_t ad = umma_desc_sw128(sP + c * PCH + k * 32, 16, 1024);
              const uint64_t bd = umma_desc_sw128(sRing + s * SLOT + k * 2048, BOX, 1024);
              umma_ss_pair(tmem + TM_O + n2 * 128, ad, bd, IDESC_PV, (!first_of_item || c > 0 || k > 0) ? 1u : 0u);
            }
            umma_commit_pair(BAR_EMPTY(s), 3);
          }
          if (ok) umma_commit_pair(BAR_PFREE(c), 3);
        }
        if (ok) umma_commit_pair(BAR_ODONE, 3);
        if (ok && last_of_item) umma_commit_pair(BAR_OLAST, 3);     // one phase per item, for the epilogue
        TRACE(6, pv_count);
#ifdef LCA_TC2_TRACE
        TRACE_ADD(8, pv_count, trace_wait);
#endif
        ++pv_count;
      };
      for (long long idx = pair_id; ok && idx < p.n_items; idx += n_pairs, ++n_item) {
        const Item it = make_item(p, idx);
        if (!mbar_wait(BAR_QFULL, n_item & 1, abort_flag)) { fail(ERR_WAIT_Q); break; }
        tc_fence_after();
        issue_s();
        for (int j = 0; ok && j < it.n_tiles; ++j) {
          if (j + 1 < it.n_tiles) issue_s();
          if (ok && j + 1 >= it.n_tiles) umma_commit_pair(BAR_QFREE, 3);     // last S of the item is in flight
          if (ok && j == 0 && n_item > 0) {
            // O of the previous item must have been read by the epilogue of both CTAs
            if (!mbar_wait(BAR_OFREE, (n_item - 1) & 1, abort_flag) || !mbar_wait(BAR_OFREE_PEER, (n_item - 1) & 1, abort_flag)) {
              fail(ERR_WAIT_O_DONE); ok = false; break;
            }
            tc_fence_after();
          }
          if (ok) issue_pv(j == 0, j + 1 == it.n_tiles);
        }
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
    volatile int* fail_word = reinterpret_cast<volatile int*>(smem + OFF_MISC + 16);   // [2], softmax threads only
    if (ln < 2) fail_word[ln] = 0;
    asm volatile("bar.sync 1, 128;" ::: "memory");
    // All 128 threads execute exactly one named barrier per tile, whatever happens: a thread whose
    // wait expired marks the tile's fail word before the barrier and everybody leaves after it.
    bool ok = !*abort_flag;
    uint32_t jt = 0;                               // tiles processed so far (all items)
    uint32_t n_item = 0;
    for (long long idx = pair_id; idx < p.n_items; idx += n_pairs, ++n_item) {
      const Item it = make_item(p, idx);
      const int t_row = it.t0 + tl;
      const bool row_valid = t_row <= it.t1;
      const int n_a_row = reps_visible(min(t_row, p.q_len - 1), p.w, p.g);
      const int first_row = n_a_row * p.g;
      float m_ref = -INFINITY, l_sum = 0.f;
      for (int j = 0; j < it.n_tiles; ++j, ++jt) {
        if (ln == 64) TRACE(9, jt);
        if (ok) {
          ok = mbar_wait(BAR_SFULL(jt & 1), (jt >> 1) & 1, abort_flag);
          if (!ok && lane == 0) fail(ERR_WAIT_S_FULL);
        }
        if (ln == 64) TRACE(10, jt);
        ok = __all_sync(0xffffffffu, ok);
        const uint32_t stm = tmem + lane_base + ((jt & 1) ? TM_S1 : TM_S0);
        const bool isA = j < it.nA;
        const int tile_key0 = isA ? j * BN : it.first_lo + (j - it.nA) * BN;
        const int key0 = tile_key0 + 128 * half;    // first key of this thread's 128 columns
        bool plain;                                 // no mask and no bias anywhere in this tile
        int lo, hi;                                 // visible columns of this thread: lo <= c <= hi
        if (isA) {
          lo = 0; hi = n_a_row - key0 - 1;
          plain = (tile_key0 + BN <= it.n_a_lo) && p.bias_log2 == 0.f;
        } else {
          lo = first_row - key0; hi = t_row - key0;
          plain = (tile_key0 >= it.n_a_hi * p.g) && (tile_key0 + BN - 1 <= it.t0);
        }
        const float bias = isA ? p.bias_log2 : 0.f;
        auto logit = [&](uint32_t raw, int c) -> float {      // general path: scale, bias, mask
          float s = fmaf(__uint_as_float(raw), p.scale_log2, bias);
          return (c < lo || c > hi) ? -INFINITY : s;
        };
        float tmax = -INFINITY;
        if (ok) {
          tc_fence_after();
#pragma unroll
          for (int q = 0; q < 4; ++q) {
            uint32_t sr[32];
            tmem_ld32(stm + q * 32, sr);
            tmem_wait_ld();
            if (plain) {
#pragma unroll
              for (int i = 0; i < 32; ++i) tmax = fmaxf(tmax, __uint_as_float(sr[i]));
            } else {
#pragma unroll
              for (int i = 0; i < 32; ++i) tmax = fmaxf(tmax, logit(sr[i], q * 32 + i));
            }
          }
          if (plain) tmax *= p.scale_log2;            // the scale is positive
        } else {
          fail_word[jt & 1] = 1;
        }
        // the two key halves of a row live in different warps: combine their maxima
        red[(jt & 1) * 128 + ln] = tmax;
        asm volatile("bar.sync 1, 128;" ::: "memory");
        if (fail_word[jt & 1]) { ok = false; continue; }      // uniform over the 128 threads
        tmax = fmaxf(tmax, red[(jt & 1) * 128 + (ln ^ 64)]);
        if (ln == 64) TRACE(11, jt);
        bool need = false;
        float factor = 1.f;
        if (j == 0) m_ref = tmax;
        else if (tmax > m_ref + RESCALE_THRESHOLD) { need = true; factor = exp2f(m_ref - tmax); }
        if (__any_sync(0xffffffffu, need)) {
          // O may be rescaled once every P V issued so far has completed (the next one waits for P)
          ok = mbar_wait(BAR_ODONE, (jt - 1) & 1, abort_flag);
          if (!ok && lane == 0) fail(ERR_WAIT_O_DONE);
          ok = __all_sync(0xffffffffu, ok);
          if (!ok) continue;                                  // reported at the next tile's barrier
          tc_fence_after();
#pragma unroll
          for (int q = 0; q < 8; ++q) {
            uint32_t o[32];
            tmem_ld32(tmem + lane_base + TM_O + q * 32, o);
            tmem_wait_ld();
#pragma unroll
            for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * factor);
            tmem_st32(tmem + lane_base + TM_O + q * 32, o);
          }
          tmem_wait_st();
          tc_fence_before();
        }
        if (need) { l_sum *= factor; m_ref = tmax; }
        const float m_use = (m_ref == -INFINITY) ? 0.f : m_ref;
        float rs = 0.f;
#pragma unroll
        for (int q = 0; q < 4; ++q) {               // 32 keys per step, P chunk pc holds 64 keys
          const int pc = half * 2 + (q >> 1);
          if ((q & 1) == 0 && jt > 0) {
            // the chunk is free once the P V of the previous tile has consumed it
            ok = mbar_wait(BAR_PFREE(pc), (jt - 1) & 1, abort_flag);
            if (!ok && lane == 0) fail(ERR_WAIT_P_FULL);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
          }
          // This thread is done with O for this tile.  Signalled only here, after the P V of the
          // previous tile has been seen to progress, so the barrier can never run a phase ahead
          // of the MMA warp's wait.
          if (q == 0) mbar_arrive(BAR_OREADY);
          if (ln == 64 && q == 0) TRACE(12, jt);
          if (ln == 64 && q == 2) TRACE(13, jt);
          uint32_t sr[32];
          tmem_ld32(stm + q * 32, sr);
          tmem_wait_ld();
          const uint32_t prow = sP + pc * PCH + rl * 128;
#pragma unroll
          for (int s4 = 0; s4 < 4; ++s4) {           // 16-byte slot holds 8 keys
            uint32_t pk[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const int e = s4 * 8 + 2 * i;
              float p0, p1;
              if (plain) {
                p0 = exp2f(fmaf(__uint_as_float(sr[e]), p.scale_log2, -m_use));
                p1 = exp2f(fmaf(__uint_as_float(sr[e + 1]), p.scale_log2, -m_use));
              } else {
                p0 = exp2f(logit(sr[e], q * 32 + e) - m_use);
                p1 = exp2f(logit(sr[e + 1], q * 32 + e + 1) - m_use);
              }
              rs += p0 + p1;
              pk[i] = pack_bf16x2(p0, p1);
            }
            const int s8 = (q & 1) * 4 + s4;
            const uint32_t a = prow + ((s8 ^ (rl & 7)) << 4);
            asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(a), "r"(pk[0]), "r"(pk[1]), "r"(pk[2]), "r"(pk[3]) : "memory");
          }
          if (q & 1) {
            fence_proxy_async_smem();               // P is read by the tensor core (async proxy)
            tc_fence_before();
            mbar_arrive(BAR_PFULL(pc));
          }
        }
        l_sum += rs;
        if (ln == 64) TRACE(14, jt);
      }
      // ---- epilogue of the item
      if (ok) {
        ok = mbar_wait(BAR_OLAST, n_item & 1, abort_flag);
        if (!ok && lane == 0) fail(ERR_WAIT_O_DONE);
      }
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) fail_word[0] = fail_word[1] = 1;
      // total row sum = sum over both key halves
      red[2 * 128 + ln] = l_sum;
      asm volatile("bar.sync 1, 128;" ::: "memory");
      if (fail_word[0]) { ok = false; break; }
      const float l_tot = l_sum + red[2 * 128 + (ln ^ 64)];
      tc_fence_after();
      const float inv = (it.n_tiles > 0 && l_tot > 0.f) ? 1.f / l_tot : 0.f;
      const size_t orow = ((size_t)it.b * p.q_len + t_row) * p.H + it.head0 + hl;
      bf16* dst = p.out + orow * 512;
#pragma unroll
      for (int q = 0; q < 8; ++q) {
        uint32_t o[32];
        tmem_ld32(tmem + lane_base + TM_O + q * 32, o);
        tmem_wait_ld();
        if (q == 7) {                                // O has been read: the next item may overwrite it
          tc_fence_before();
          mbar_arrive(BAR_OFREE);
        }
        if (row_valid) {
          // TMEM columns [0,128): output columns 128*half + c ; [128,256): 256 + 128*half + (c-128)
          const int col = (q >> 2) * 256 + 128 * half + (q & 3) * 32;
          uint4* d4 = reinterpret_cast<uint4*>(dst + col);
#pragma unroll
          for (int v = 0; v < 4; ++v) {
            uint4 w;
            w.x = pack_bf16x2(__uint_as_float(o[8 * v + 0]) * inv, __uint_as_float(o[8 * v + 1]) * inv);
            w.y = pack_bf16x2(__uint_as_float(o[8 * v + 2]) * inv, __uint_as_float(o[8 * v + 3]) * inv);
            w.z = pack_bf16x2(__uint_as_float(o[8 * v + 4]) * inv, __uint_as_float(o[8 * v + 5]) * inv);
            w.w = pack_bf16x2(__uint_as_float(o[8 * v + 6]) * inv, __uint_as_float(o[8 * v + 7]) * inv);
            d4[v] = w;
          }
        }
      }
      if (p.lse && row_valid && half == 0)
        p.lse[orow] = (l_tot > 0.f) ? (m_ref + log2f(l_tot)) * 0.6931471805599453f : -INFINITY;
    }
    tc_fence_before();
  }
  // ---- teardown: let straggling bulk copies land if the CTA gave up, then free TMEM
  if (*abort_flag && warp == 0 && lane == 0) {
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

// ----------------------------------------------------------------------------------- host
bool make_tensor_map_3d(CUtensorMap* map, const void* ptr, int d, int heads, long long rows, int box_heads, int box_rows);

bool attn_tc2_supported(const AttnProblem& a) {
  if (a.variant != LCA_VARIANT_MLA || a.d_sem != 512 || a.d_pos != 64 || a.n_kv_heads != 1) return false;
  if (a.decode) return false;
  const int H = a.n_q_heads;
  if (H >= 128) return H % 128 == 0;
  return H >= 1 && (128 % H) == 0;      // each CTA of the pair takes whole tokens
}

static int sm_count() {
  static int n = 0;
  if (n == 0) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
      n = 148;
  }
  return n;
}

// 64-key image blocks per column chunk of the token stream and of the representatives
static void image_blocks(const AttnProblem& a, int* nkb_tok, int* nkb_rep, int* m_out) {
  int64_t m, k;
  partition(a.seq_len, a.window, a.group_size, &m, &k);
  *nkb_tok = (a.seq_len + 63) / 64 + pair::PAD_KEY_BLOCKS;
  *nkb_rep = m > 0 ? (int)((m + 63) / 64) + pair::PAD_KEY_BLOCKS : 0;
  *m_out = (int)m;
}

size_t attn_tc2_workspace_bytes(const AttnProblem& a) {
  int nt, nr, m;
  image_blocks(a, &nt, &nr, &m);
  return (size_t)a.batch * 17 * ((size_t)nt + nr) * pair::BOX;
}

int attn_tc2_launch(const AttnProblem& a) {
  using namespace pair;
  if (!attn_tc2_supported(a)) return LCA_ERR_UNSUPPORTED_SHAPE;
  Tc2Params p;
  memset(&p, 0, sizeof(p));
  const int H = a.n_q_heads;
  int m;
  image_blocks(a, &p.nkb_tok, &p.nkb_rep, &m);
  p.seq_image_bytes = 17ll * (p.nkb_tok + p.nkb_rep) * BOX;
  p.images = (const unsigned char*)a.ws;
  p.HB = H >= 128 ? 128 : H;
  p.TB = 128 / p.HB;
  p.B = a.batch; p.q_len = a.q_len; p.H = H; p.L = a.seq_len; p.g = a.group_size; p.w = a.window;
  p.cap = a.cache_row_capacity;
  p.n_tok_tiles = (a.q_len + p.TB - 1) / p.TB;
  p.n_head_blocks = H >= 128 ? H / 128 : 1;
  p.n_items = (long long)p.n_tok_tiles * p.n_head_blocks * a.batch;
  p.scale_log2 = a.softmax_scale * 1.4426950408889634f;
  p.bias_log2 = a.rep_logit_bias * 1.4426950408889634f;
  p.out = (bf16*)a.out; p.lse = a.lse;
  const int hbc = p.HB >= 64 ? 64 : p.HB, tbc = 64 / hbc;
  const long long qrows = (long long)a.batch * a.q_len;
  bool ok = make_tensor_map_3d(&p.q_sem, a.q_sem, 512, H, qrows, hbc, tbc);
  ok = ok && make_tensor_map_3d(&p.q_pos, a.q_pos, 64, H, qrows, hbc, tbc);
  if (!ok) return LCA_ERR_CUDA;

  RetileArgs r;
  r.kv_sem = (const bf16*)a.kv_sem; r.kv_pos = (const bf16*)a.kv_pos;
  r.cache_sem = (const bf16*)a.cache_sem; r.cache_pos = (const bf16*)a.cache_pos;
  r.images = (unsigned char*)a.ws; r.seq_image_bytes = p.seq_image_bytes;
  r.L = a.seq_len; r.m = m; r.cap = a.cache_row_capacity; r.nkb_tok = p.nkb_tok; r.nkb_rep = p.nkb_rep;
  retile_kernel<<<dim3((unsigned)p.nkb_tok, 9, 2 * a.batch), 512, 0, a.stream>>>(r);
  note_launch();

  if (cudaFuncSetAttribute(attn_tc2_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) != cudaSuccess)
    return LCA_ERR_CUDA;
  long long pairs = sm_count() / 2;
  if (pairs > p.n_items) pairs = p.n_items;
  if (pairs < 1) pairs = 1;
  attn_tc2_kernel<<<dim3((unsigned)(2 * pairs)), THREADS, SMEM_BYTES, a.stream>>>(p);
  note_launch();
  return cudaGetLastError() == cudaSuccess ? LCA_OK : LCA_ERR_CUDA;
}

#ifdef LCA_TC2_TRACE
extern "C" int lca_debug_read_trace(long long* dst) {
  return cudaMemcpyFromSymbol(dst, g_trace, sizeof(long long) * 2 * 128 * 24) == cudaSuccess ? 0 : -1;
}
#endif

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
