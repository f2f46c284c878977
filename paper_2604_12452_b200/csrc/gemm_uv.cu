// Value up-projection of the latent attention output (Alg. 1, "v_rep = c_rep W^UV"; Sec. 4.3: in the
// absorbed form the attention runs in the latent space and W^UV is applied to its result, once per
// query and head):   out_v[t, h, :] = attn_latent[t, h, :] W^UV[h]      ([512] x [512, 128] per row).
//
// Per head this is a [T, 512] x [512, 128] product whose operands are read once: 102 flop per byte, below
// the ridge of the machine, so the kernel is laid out for HBM streaming rather than tensor throughput.  One
// CTA owns 128 tokens of one head: TMA brings the latent tile in eight 64-column chunks (16 KB, 128-byte
// swizzle) together with the matching 64 x 128 slice of W^UV (16 KB, L2-resident: every token tile of the
// head reads it again) through a three-stage ring; one tcgen05.mma chain (M 128, N 128, K 16 x 32)
// accumulates in tensor memory; four warps convert the accumulator to bf16 and store 32 bytes per
// instruction.  Two CTAs fit an SM (96 KB of shared memory, 128 TMEM columns each), so the prologue and
// the epilogue of one overlap the main loop of the other.
#include <cstring>

#include "lca_common.cuh"
#include "tc_common.cuh"

namespace lca {
using namespace tc;

static __device__ int g_uv_status = 0;

namespace uv {
constexpr int DC = 512, DV = 128, BM = 128, KC = 64;       // latent width, value width, tokens per CTA, K per stage
constexpr int NKC = DC / KC;                                // 8 stages' worth of K per tile
constexpr int A_BYTES = BM * KC * 2, B_BYTES = KC * DV * 2; // 16 KB each
constexpr int STAGE = A_BYTES + B_BYTES, STAGES = 3;
constexpr int OFF_BAR = STAGES * STAGE, OFF_MISC = OFF_BAR + 64;
constexpr int SMEM_BYTES = OFF_MISC + 16 + 1024;            // + slack to align the base to 1024 B
constexpr int THREADS = 192;                                // warp 0 loads, warp 1 MMA + TMEM, warps 2-5 epilogue
}  // namespace uv

struct UvParams {
  CUtensorMap a;          // latent [T, H, 512] as {512, H, T}, box {64, 1, 128}
  CUtensorMap w;          // W^UV [H, 512, 128] as {128, 512, H}, box {64, 64, 1}
  bf16* out;              // [T, H, 128]
  long long T;
  int H, out_wide;
};

__global__ void __launch_bounds__(uv::THREADS, 2)
latent_to_value_kernel(const __grid_constant__ UvParams p) {
  using namespace uv;
  extern __shared__ unsigned char smem_dyn[];
  const uint32_t base = (smem_u32(smem_dyn) + 1023u) & ~1023u;
  unsigned char* base_ptr = smem_dyn + (base - smem_u32(smem_dyn));
  const uint32_t bars = base + OFF_BAR;
  auto BAR_FULL = [&](int s) { return bars + 8 * s; };
  auto BAR_EMPTY = [&](int s) { return bars + 8 * (STAGES + s); };
  const uint32_t BAR_DONE = bars + 8 * (2 * STAGES);
  volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(base_ptr + OFF_MISC);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(base_ptr + OFF_MISC + 4);
  const int warp = __shfl_sync(0xffffffffu, (int)(threadIdx.x >> 5), 0), lane = threadIdx.x & 31;
  // heads vary fastest over the grid: CTAs that run at the same time read neighbouring 1 KB pieces of the same token rows
  const int h = (int)(blockIdx.x % (unsigned)p.H);
  const long long t0 = (long long)(blockIdx.x / (unsigned)p.H) * BM;

  if (threadIdx.x == 0) {
    for (int s = 0; s < STAGES; ++s) { mbar_init(BAR_FULL(s), 1); mbar_init(BAR_EMPTY(s), 1); }
    mbar_init(BAR_DONE, 1);
    *abort_flag = 0;
    fence_mbar_init();
  }
  if (warp == 1) {
    tmem_alloc(smem_u32((const void*)tmem_slot), 128);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem = *tmem_slot;
  auto fail = [&](int code) {
    atomicCAS(&g_uv_status, 0, code);
    *abort_flag = 1;
  };

  if (warp == 0) {
    if (lane == 0) {
      prefetch_tmap(&p.a); prefetch_tmap(&p.w);
      for (int kc = 0; kc < NKC; ++kc) {
        const int s = kc % STAGES, round = kc / STAGES;
        if (!mbar_wait(BAR_EMPTY(s), (round & 1) ^ 1, abort_flag)) { fail(ERR_WAIT_KV_EMPTY); break; }
        mbar_expect_tx(BAR_FULL(s), STAGE);
        const uint32_t sa = base + s * STAGE, sb = sa + A_BYTES;
        tma_load_3d(sa, &p.a, kc * KC, h, (int)t0, BAR_FULL(s));                       // 128 tokens x 64 latent columns
        for (int n = 0; n < 2; ++n) tma_load_3d(sb + n * (KC * 128), &p.w, n * 64, kc * KC, h, BAR_FULL(s));   // 64 k-rows x 64 value columns
      }
    }
  } else if (warp == 1) {
    constexpr uint32_t IDESC = umma_idesc_bf16(BM, DV, false, true);      // A K-major, B (W^UV slice) N-major
    const uint32_t leader = elect_one();
    bool ok = true;
    for (int kc = 0; ok && kc < NKC; ++kc) {
      const int s = kc % STAGES, round = kc / STAGES;
      ok = mbar_wait(BAR_FULL(s), round & 1, abort_flag);
      if (!ok) { if (leader) fail(ERR_WAIT_KV_FULL); break; }
      tc_fence_after();
      const uint32_t sa = base + s * STAGE, sb = sa + A_BYTES;
      const uint64_t ad0 = umma_desc_sw128(sa, 16, 1024), bd0 = umma_desc_sw128(sb, KC * 128, 1024);
#pragma unroll
      for (int k = 0; k < KC / 16; ++k)
        umma_ss_elected(leader, tmem, desc_add(ad0, (k * 32) >> 4), desc_add(bd0, (k * 2048) >> 4), IDESC, (kc > 0 || k > 0) ? 1u : 0u);
      umma_commit_elected(leader, BAR_EMPTY(s));
    }
    if (ok) umma_commit_elected(leader, BAR_DONE);
  } else {
    const int quarter = warp & 3;
    const int row = quarter * 32 + lane;
    const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
    bool ok = mbar_wait(BAR_DONE, 0, abort_flag);
    if (!ok && lane == 0) fail(ERR_WAIT_O_DONE);
    ok = __all_sync(0xffffffffu, ok);
    if (ok) {
      tc_fence_after();
      const long long t = t0 + row;
      bf16* dst = p.out + ((size_t)t * p.H + h) * DV;
#pragma unroll 1
      for (int q = 0; q < 4; ++q) {
        uint32_t o[32];
        tmem_ld32(tmem + lane_base + q * 32, o);
        tmem_wait_ld();
        if (t < p.T) {
#pragma unroll
          for (int v = 0; v < 2; ++v) {
            uint32_t wv[8];
#pragma unroll
            for (int e = 0; e < 8; ++e)
              wv[e] = pack_bf16x2(__uint_as_float(o[16 * v + 2 * e]), __uint_as_float(o[16 * v + 2 * e + 1]));
            st_global_32B(dst + q * 32 + 16 * v, wv, p.out_wide != 0);
          }
        }
      }
    }
    tc_fence_before();
  }
  if (*abort_flag && warp == 0 && lane == 0) {
    const long long t0c = clock64();
    while (clock64() - t0c < 2000000ll) { __nanosleep(1000); }
  }
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem, 128);
  }
}

// ----------------------------------------------------------------------------------- host
bool make_tensor_map_3d(CUtensorMap* map, const void* ptr, int d, int heads, long long rows, int box_heads, int box_rows);

int latent_to_value_launch(const void* latent, const void* w_uv, void* out, long long n_tokens, int n_heads,
                           int d_latent, int d_v, cudaStream_t stream) {
  using namespace uv;
  if (d_latent != DC || d_v != DV) return LCA_ERR_UNSUPPORTED_SHAPE;
  if (n_tokens > 0x7fffff00ll) return LCA_ERR_UNSUPPORTED_SHAPE;        // TMA row coordinates are 32-bit
  UvParams p;
  memset(&p, 0, sizeof(p));
  p.out = (bf16*)out; p.T = n_tokens; p.H = n_heads;
  p.out_wide = (reinterpret_cast<uintptr_t>(out) & 31u) == 0;
  bool ok = make_tensor_map_3d(&p.a, latent, DC, n_heads, n_tokens, 1, BM);
  // W^UV [H, 512, 128]: the same helper with (d, "heads", rows) = (128, 512, H): box 64 columns x 64 k-rows x 1 head
  ok = ok && make_tensor_map_3d(&p.w, w_uv, DV, DC, n_heads, KC, 1);
  if (!ok) return LCA_ERR_CUDA;
  if (cudaFuncSetAttribute(latent_to_value_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES) != cudaSuccess)
    return LCA_ERR_CUDA;
  const long long n_ctas = ((n_tokens + BM - 1) / BM) * n_heads;
  if (n_ctas > 0x7fffffffll) return LCA_ERR_UNSUPPORTED_SHAPE;
  dim3 grid((unsigned)n_ctas);
  latent_to_value_kernel<<<grid, THREADS, SMEM_BYTES, stream>>>(p);
  note_launch();
  return cudaGetLastError() == cudaSuccess ? LCA_OK : LCA_ERR_CUDA;
}

int latent_to_value_take_status() {
  int st = 0;
  if (cudaMemcpyFromSymbol(&st, g_uv_status, sizeof(int)) != cudaSuccess) return -1;
  if (st != 0) {
    int zero = 0;
    cudaMemcpyToSymbol(g_uv_status, &zero, sizeof(int));
  }
  return st;
}

}  // namespace lca
