// sc_masked_weight_grad: the fast circuit's weight gradient of one linear layer from masked activations
// (Section 3.1; Algorithm 1 lines 4-5):  G = dY^T (X . M) * 65536 / round(keep * 65536),  M the shared-PRF mask.
//
// Two launches on the caller's stream: the mask pass (sc_apply_prf_mask, X -> Xm, one HBM pass over the activation)
// and a dense bf16 GEMM over the token dimension on the tensor cores. The mask is applied once, not inside the GEMM's
// operand load: every activation tile is an operand of all row tiles of the output, so hashing at load time would
// repeat the same work rows/128 times and turn a tensor-bound kernel into an issue-bound one.
//
// GEMM: G[rows x cols] = scale * A^T B with A = dY (tokens x rows) and B = Xm (tokens x cols), both row-major, i.e.
// both operands are MN-major for the tensor core (the contraction index is the slow one in memory). Persistent blocks,
// tiles ordered so that the smaller of the two operands is the one the blocks running side by side have in common (it
// stays in L2; the larger one is streamed once), K advancing 64 tokens per pipeline stage. Two kernels:
//   wgrad_pair_kernel   outputs of at least 256 x 256: clusters of two SMs on 256 x 256 tiles, tcgen05 cta_group::2
//   wgrad_kernel        anything smaller: one block per 128 x 256 tile
// Warp roles in both: warp 0 TMA producer (64 x 64 boxes, 128-byte swizzle), warp 1 tcgen05.mma kind::f16 issuer with
// fp32 accumulators in two 256-column TMEM buffers, warps 2-5 epilogue (TMEM -> registers -> scale -> bf16 or fp32 ->
// global). Every mbarrier wait is bounded; a wait that runs out latches the time-out bit in *status_dev and the block
// winds down.
#include <cuda.h>

#include <cstdlib>

#include "sc_internal.cuh"
#include "sc_ptx.cuh"

namespace sc {
namespace {

constexpr int kWgBM = 128, kWgBN = 256, kWgBK = 64, kWgStages = 4;
constexpr int kWgBox = 64 * kWgBK * 2;                     // one 64 (MN) x 64 (K) bf16 box: 8 KB
constexpr int kWgABytes = (kWgBM / 64) * kWgBox;           // 16 KB
constexpr int kWgBBytes = (kWgBN / 64) * kWgBox;           // 32 KB
constexpr int kWgStageBytes = kWgABytes + kWgBBytes;       // 48 KB

struct WgBars {
  uint64_t full[kWgStages], empty[kWgStages];
  uint64_t acc_full[2], acc_empty[2];
  uint32_t tmem_slot;
  int abort_flag;
  int never_flag;
};

// MN-major bf16 operand, 128-byte swizzle: atoms of 64 (MN, contiguous 128 bytes) x 8 (K rows); consecutive K groups
// of 8 rows are 1024 bytes apart (SBO), consecutive 64-wide MN blocks `lbo` bytes apart.
__device__ __forceinline__ uint64_t umma_desc_mn_bf16(uint32_t saddr, uint32_t lbo) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo >> 4) << 16) | ((uint64_t)(1024 >> 4) << 32) |
         ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}
// bf16 x bf16 -> fp32, both operands MN-major, M = 128.
__device__ __forceinline__ uint32_t umma_idesc_bf16_mn(int N) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (1u << 16) | ((uint32_t)(N >> 3) << 17) |
         ((uint32_t)(128 >> 4) << 24);
}

__global__ void __launch_bounds__(192, 1)
wgrad_kernel(const __grid_constant__ CUtensorMap map_dy, const __grid_constant__ CUtensorMap map_x, void* __restrict__ G,
             int out_f32, int tokens, int rows, int cols, float scale, int n_fastest, unsigned* status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  WgBars* bars = reinterpret_cast<WgBars*>(smem + kWgStages * kWgStageBytes);
  volatile int* abort_flag = &bars->abort_flag;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int tiles_m = (rows + kWgBM - 1) / kWgBM, tiles_n = (cols + kWgBN - 1) / kWgBN;
  const int tiles = tiles_m * tiles_n;
  const int kchunks = (tokens + kWgBK - 1) / kWgBK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kWgStages; ++s) { mbar_init(&bars->full[s], 1); mbar_init(&bars->empty[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&bars->acc_full[a], 1); mbar_init(&bars->acc_empty[a], 4); }
    bars->abort_flag = 0;
    bars->never_flag = 0;
    fence_barrier_init();
    fence_proxy_async();
  }
  if (warp == 1) tmem_alloc(&bars->tmem_slot, 512);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      uint32_t it = 0;
      bool dead = false;
      for (int tile = blockIdx.x; tile < tiles && !dead; tile += gridDim.x) {
        const int tm = n_fastest ? tile / tiles_n : tile % tiles_m, tn = n_fastest ? tile % tiles_n : tile / tiles_m;
        for (int kc = 0; kc < kchunks; ++kc, ++it) {
          const int s = it % kWgStages;
          if (!mbar_wait(&bars->empty[s], ((it / kWgStages) & 1) ^ 1, abort_flag)) { dead = true; break; }
          uint8_t* st = smem + (size_t)s * kWgStageBytes;
          mbar_expect_tx(&bars->full[s], kWgStageBytes);
          // tokens past the end and rows / columns past the edge come in as zeros
          for (int b = 0; b < kWgBM / 64; ++b)
            tma_load_2d(st + b * kWgBox, &map_dy, &bars->full[s], tm * kWgBM + b * 64, kc * kWgBK);
          for (int b = 0; b < kWgBN / 64; ++b)
            tma_load_2d(st + kWgABytes + b * kWgBox, &map_x, &bars->full[s], tn * kWgBN + b * 64, kc * kWgBK);
        }
      }
      if (dead) {
        if (status) atomicOr(status, kDevTimeout);
        *abort_flag = 1;
        for (uint32_t u = it > (uint32_t)kWgStages ? it - kWgStages : 0; u < it; ++u)
          mbar_wait(&bars->full[u % kWgStages], (u / kWgStages) & 1, &bars->never_flag);
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = umma_idesc_bf16_mn(kWgBN);
      uint32_t it = 0, t = 0;
      bool dead = false;
      for (int tile = blockIdx.x; tile < tiles && !dead; tile += gridDim.x, ++t) {
        const uint32_t ab = t & 1;
        if (!mbar_wait(&bars->acc_empty[ab], ((t >> 1) & 1) ^ 1, abort_flag)) { dead = true; break; }
        tc_fence_after();
        const uint32_t d = tmem_base + ab * kWgBN;
        for (int kc = 0; kc < kchunks; ++kc, ++it) {
          const int s = it % kWgStages;
          if (!mbar_wait(&bars->full[s], (it / kWgStages) & 1, abort_flag)) { dead = true; break; }
          tc_fence_after();
          const uint32_t a0 = smem_u32(smem + (size_t)s * kWgStageBytes), b0 = a0 + kWgABytes;
#pragma unroll
          for (int k = 0; k < kWgBK / 16; ++k) {   // 16 tokens = two 8-row K groups = 2048 bytes per step
            umma_bf16(d, umma_desc_mn_bf16(a0 + k * 2048, kWgBox), umma_desc_mn_bf16(b0 + k * 2048, kWgBox), idesc,
                      (kc | k) != 0);
          }
          umma_commit(&bars->empty[s]);
        }
        if (dead) break;
        umma_commit(&bars->acc_full[ab]);
      }
      if (dead) {
        if (status) atomicOr(status, kDevTimeout);
        *abort_flag = 1;
      }
    }
    __syncwarp();
  } else {
    const int q = warp & 3;
    uint32_t t = 0;
    bool dead = false;
    for (int tile = blockIdx.x; tile < tiles && !dead; tile += gridDim.x, ++t) {
      const int tm = n_fastest ? tile / tiles_n : tile % tiles_m, tn = n_fastest ? tile % tiles_n : tile / tiles_m;
      const uint32_t ab = t & 1;
      if (!mbar_wait(&bars->acc_full[ab], (t >> 1) & 1, abort_flag)) { dead = true; break; }
      tc_fence_after();
      const int row = tm * kWgBM + q * 32 + lane;
      const uint32_t d = tmem_base + ab * kWgBN + ((uint32_t)(q * 32) << 16);
      for (int c = 0; c < kWgBN; c += 16) {
        float v[16];
        tmem_ld16(d + c, v);
        tmem_ld_wait();
        const int col = tn * kWgBN + c;
        if (row < rows && col < cols) {
#pragma unroll
          for (int j = 0; j < 16; ++j) v[j] *= scale;
          if (out_f32) {
            float* o = static_cast<float*>(G) + (size_t)row * cols + col;
#pragma unroll
            for (int j = 0; j < 16; j += 8) {
              if (col + j < cols) {     // cols is a multiple of 8
                *reinterpret_cast<float4*>(o + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                *reinterpret_cast<float4*>(o + j + 4) = make_float4(v[j + 4], v[j + 5], v[j + 6], v[j + 7]);
              }
            }
          } else {
            bf16* o = static_cast<bf16*>(G) + (size_t)row * cols + col;
#pragma unroll
            for (int j = 0; j < 16; j += 8) {
              if (col + j < cols) {
                const __nv_bfloat162 p0 = __floats2bfloat162_rn(v[j], v[j + 1]), p1 = __floats2bfloat162_rn(v[j + 2], v[j + 3]);
                const __nv_bfloat162 p2 = __floats2bfloat162_rn(v[j + 4], v[j + 5]), p3 = __floats2bfloat162_rn(v[j + 6], v[j + 7]);
                *reinterpret_cast<uint4*>(o + j) =
                    make_uint4(*reinterpret_cast<const uint32_t*>(&p0), *reinterpret_cast<const uint32_t*>(&p1),
                               *reinterpret_cast<const uint32_t*>(&p2), *reinterpret_cast<const uint32_t*>(&p3));
              }
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&bars->acc_empty[ab]);
    }
    if (dead && lane == 0) {
      if (status) atomicOr(status, kDevTimeout);
      *abort_flag = 1;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, 512);
}

// -----------------------------------------------------------------------------------------------------------------
// The same GEMM with two blocks (a cluster of two SMs) on one 256 x 256 tile: tcgen05.mma cta_group::2. Block t of the
// pair loads rows t*128.. of the dY tile and columns t*128.. of the Xm tile, i.e. half the activation tile each, and the
// tensor cores of both SMs read the two halves, so per SM and stage 32 KB go into shared memory instead of 48 KB for
// the same number of flops; with one block per tile the tensor pipe waits for shared memory (75% busy). Block 0 (the
// leader) issues the MMAs for both; its full barriers collect the bytes of both blocks' loads; its commits arrive on
// the empty and accumulator barriers of both blocks; the epilogue warps of both blocks release the accumulator
// through the leader's barrier. No multicast loads anywhere.
// -----------------------------------------------------------------------------------------------------------------
constexpr int kW2Stages = 6;
constexpr int kW2ABytes = 2 * kWgBox, kW2BBytes = 2 * kWgBox;          // 128 rows of dY^T, 128 columns of Xm per block
constexpr int kW2StageBytes = kW2ABytes + kW2BBytes;                   // 32 KB per block and stage

struct W2Bars {
  uint64_t full[kW2Stages], empty[kW2Stages];
  uint64_t acc_full[2], acc_empty[2];
  uint64_t drain;                // abort path only: the leader's MMAs in flight have finished
  uint32_t tmem_slot;
  int abort_flag;
  int never_flag;
};

__device__ __forceinline__ uint32_t umma_idesc_bf16_mn_pair(int N) {   // M = 256 over the two blocks
  return (1u << 4) | (1u << 7) | (1u << 10) | (1u << 15) | (1u << 16) | ((uint32_t)(N >> 3) << 17) |
         ((uint32_t)(256 >> 4) << 24);
}

// The kernel is also the library's general "A^T B" GEMM (sc::launch_tn_gemm): up to three operand pairs are contracted
// one after the other into the same accumulator (a split-precision product: hi*hi + lo*hi + hi*lo), the epilogue can
// add a multiple of the identity and can write the result as fp32, as bf16, or as a bf16 hi/lo pair.
struct TnMaps {
  CUtensorMap a[3], b[3];
};
struct TnEpilogue {
  void* out;        // out_mode 0: bf16, 1: fp32, 2: bf16 hi part of a hi/lo pair
  void* out_lo;     // out_mode 2: the lo part
  int out_mode;
  float scale;      // result = scale * sum + diag * I
  float diag;
};

// GEN = false is the plain weight-gradient GEMM (one operand pair, bf16 or fp32 output): every generalisation below
// folds away at compile time, so that path costs exactly what it did before the kernel was generalised.
template <bool GEN>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(192, 1)
wgrad_pair_kernel(const __grid_constant__ TnMaps maps, int nseg_arg, TnEpilogue epi, int tokens, int rows, int cols,
                  int n_fastest, unsigned* status) {
  const int nseg = GEN ? nseg_arg : 1;
  void* __restrict__ G = epi.out;
  const int out_f32 = epi.out_mode == 1;
  const float scale = epi.scale;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  W2Bars* bars = reinterpret_cast<W2Bars*>(smem + kW2Stages * kW2StageBytes);
  volatile int* abort_flag = &bars->abort_flag;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const int tiles_m = (rows + 255) / 256, tiles_n = (cols + 255) / 256;
  const int tiles = tiles_m * tiles_n;
  const int kchunks = (tokens + kWgBK - 1) / kWgBK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kW2Stages; ++s) { mbar_init(&bars->full[s], 1); mbar_init(&bars->empty[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&bars->acc_full[a], 1); mbar_init(&bars->acc_empty[a], 8); }
    mbar_init(&bars->drain, 1);
    bars->abort_flag = 0;
    bars->never_flag = 0;
    fence_barrier_init();
    fence_proxy_async();
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&bars->tmem_slot)), "r"(512u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();            // the peer's barriers exist before anything is sent to them
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      uint32_t it = 0;
      bool dead = false;
      for (int tile = pair; tile < tiles && !dead; tile += n_pairs) {
        const int tm = n_fastest ? tile / tiles_n : tile % tiles_m, tn = n_fastest ? tile % tiles_n : tile / tiles_m;
        for (int kk = 0, seg = 0, kc = 0; kk < kchunks * nseg; ++kk, ++it, ++kc) {
          if (GEN && kc == kchunks) { kc = 0; ++seg; }
          const int s = it % kW2Stages;
          if (!mbar_wait(&bars->empty[s], ((it / kW2Stages) & 1) ^ 1, abort_flag)) { dead = true; break; }
          uint8_t* st = smem + (size_t)s * kW2StageBytes;
          if (rank == 0) mbar_expect_tx(&bars->full[s], 2 * kW2StageBytes);      // both blocks' bytes
          const uint32_t leader_bar = map_to_rank(smem_u32(&bars->full[s]), 0);
          for (int b = 0; b < 2; ++b)
            tma_load_2d_pair(st + b * kWgBox, &maps.a[GEN ? seg : 0], leader_bar, tm * 256 + (int)rank * 128 + b * 64, kc * kWgBK);
          for (int b = 0; b < 2; ++b)
            tma_load_2d_pair(st + kW2ABytes + b * kWgBox, &maps.b[GEN ? seg : 0], leader_bar, tn * 256 + (int)rank * 128 + b * 64,
                             kc * kWgBK);
        }
      }
      if (dead) {
        if (status) atomicOr(status, kDevTimeout);
        *abort_flag = 1;
        // Let the copies in flight land before the pair's shared memory goes away. The bytes of both blocks are counted
        // on the leader's barriers, so the leader waits (bounded) for the stages it armed; the other block cannot see
        // its own copies land and instead idles for a grace period far longer than a copy takes. Both blocks then
        // meet in the cluster barrier at the end of the kernel, so neither leaves before the leader has drained.
        if (rank == 0) {
          for (uint32_t u = it > (uint32_t)kW2Stages ? it - kW2Stages : 0; u < it; ++u)
            mbar_wait(&bars->full[u % kW2Stages], (u / kW2Stages) & 1, &bars->never_flag);
        } else {
          for (int i = 0; i < 64; ++i) __nanosleep(1000);
        }
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    if (lane == 0 && rank == 0) {
      const uint32_t idesc = umma_idesc_bf16_mn_pair(256);
      uint32_t it = 0, t = 0;
      bool dead = false;
      for (int tile = pair; tile < tiles && !dead; tile += n_pairs, ++t) {
        const uint32_t ab = t & 1;
        if (!mbar_wait(&bars->acc_empty[ab], ((t >> 1) & 1) ^ 1, abort_flag)) { dead = true; break; }
        tc_fence_after();
        const uint32_t d = tmem_base + ab * 256;
        for (int kc = 0; kc < kchunks * nseg; ++kc, ++it) {
          const int s = it % kW2Stages;
          if (!mbar_wait(&bars->full[s], (it / kW2Stages) & 1, abort_flag)) { dead = true; break; }
          tc_fence_after();
          const uint32_t a0 = smem_u32(smem + (size_t)s * kW2StageBytes), b0 = a0 + kW2ABytes;
#pragma unroll
          for (int k = 0; k < kWgBK / 16; ++k)
            umma_bf16_pair(d, umma_desc_mn_bf16(a0 + k * 2048, kWgBox), umma_desc_mn_bf16(b0 + k * 2048, kWgBox), idesc,
                           (kc | k) != 0);
          umma_commit_pair(&bars->empty[s]);
        }
        if (dead) break;
        umma_commit_pair(&bars->acc_full[ab]);
      }
      if (dead) {
        if (status) atomicOr(status, kDevTimeout);
        *abort_flag = 1;
        // MMAs already issued still read shared memory and write TMEM of both blocks: wait (bounded) until they are done
        asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];"
                     ::"r"(smem_u32(&bars->drain)) : "memory");
        mbar_wait(&bars->drain, 0, &bars->never_flag);
      }
    }
    __syncwarp();
  } else {
    const int q = warp & 3;
    uint32_t t = 0;
    bool dead = false;
    for (int tile = pair; tile < tiles && !dead; tile += n_pairs, ++t) {
      const int tm = n_fastest ? tile / tiles_n : tile % tiles_m, tn = n_fastest ? tile % tiles_n : tile / tiles_m;
      const uint32_t ab = t & 1;
      if (!mbar_wait(&bars->acc_full[ab], (t >> 1) & 1, abort_flag)) { dead = true; break; }
      tc_fence_after();
      const int row = tm * 256 + (int)rank * 128 + q * 32 + lane;
      const uint32_t d = tmem_base + ab * 256 + ((uint32_t)(q * 32) << 16);
      for (int c = 0; c < 256; c += 16) {
        float v[16];
        tmem_ld16(d + c, v);
        tmem_ld_wait();
        const int col = tn * 256 + c;
        if (row < rows && col < cols) {
#pragma unroll
          for (int j = 0; j < 16; ++j) v[j] *= scale;
          if (GEN && epi.diag != 0.f && row >= col && row < col + 16) {
#pragma unroll
            for (int j = 0; j < 16; ++j) v[j] += (col + j == row) ? epi.diag : 0.f;    // static indices: v stays in registers
          }
          if (GEN && epi.out_mode == 2) {        // bf16 hi/lo pair: hi = rn(v), lo = rn(v - hi)
            bf16* oh = static_cast<bf16*>(G) + (size_t)row * cols + col;
            bf16* ol = static_cast<bf16*>(epi.out_lo) + (size_t)row * cols + col;
#pragma unroll
            for (int j = 0; j < 16; j += 8) {
              if (col + j < cols) {
                uint32_t hw[4], lw[4];
#pragma unroll
                for (int e = 0; e < 4; ++e) {
                  const float x0 = v[j + 2 * e], x1 = v[j + 2 * e + 1];
                  const __nv_bfloat162 h2 = __floats2bfloat162_rn(x0, x1);
                  const __nv_bfloat162 l2 = __floats2bfloat162_rn(x0 - __low2float(h2), x1 - __high2float(h2));
                  hw[e] = *reinterpret_cast<const uint32_t*>(&h2);
                  lw[e] = *reinterpret_cast<const uint32_t*>(&l2);
                }
                *reinterpret_cast<uint4*>(oh + j) = make_uint4(hw[0], hw[1], hw[2], hw[3]);
                *reinterpret_cast<uint4*>(ol + j) = make_uint4(lw[0], lw[1], lw[2], lw[3]);
              }
            }
          } else if (out_f32) {
            float* o = static_cast<float*>(G) + (size_t)row * cols + col;
#pragma unroll
            for (int j = 0; j < 16; j += 8) {
              if (col + j < cols) {
                *reinterpret_cast<float4*>(o + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
                *reinterpret_cast<float4*>(o + j + 4) = make_float4(v[j + 4], v[j + 5], v[j + 6], v[j + 7]);
              }
            }
          } else {
            bf16* o = static_cast<bf16*>(G) + (size_t)row * cols + col;
#pragma unroll
            for (int j = 0; j < 16; j += 8) {
              if (col + j < cols) {
                const __nv_bfloat162 p0 = __floats2bfloat162_rn(v[j], v[j + 1]), p1 = __floats2bfloat162_rn(v[j + 2], v[j + 3]);
                const __nv_bfloat162 p2 = __floats2bfloat162_rn(v[j + 4], v[j + 5]), p3 = __floats2bfloat162_rn(v[j + 6], v[j + 7]);
                *reinterpret_cast<uint4*>(o + j) =
                    make_uint4(*reinterpret_cast<const uint32_t*>(&p0), *reinterpret_cast<const uint32_t*>(&p1),
                               *reinterpret_cast<const uint32_t*>(&p2), *reinterpret_cast<const uint32_t*>(&p3));
              }
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(map_to_rank(smem_u32(&bars->acc_empty[ab]), 0));   // the leader's barrier
    }
    if (dead && lane == 0) {
      if (status) atomicOr(status, kDevTimeout);
      *abort_flag = 1;
    }
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();            // nothing of the peer is touched after this
  if (warp == 1)
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
        q != cudaDriverEntryPointSuccess)
      p = nullptr;
    return reinterpret_cast<EncodeTiledFn>(p);
  }();
  return fn;
}

// tokens x width bf16 row-major -> boxes of 64 (width) x 64 (tokens), 128-byte swizzle
bool encode_mn(CUtensorMap* out, const void* base, int64_t tokens, int64_t width) {
  EncodeTiledFn enc = encode_fn();
  if (!enc) return false;
  cuuint64_t dims[2] = {(cuuint64_t)width, (cuuint64_t)tokens};
  cuuint64_t strides[1] = {(cuuint64_t)width * 2};
  cuuint32_t box[2] = {64, (cuuint32_t)kWgBK};
  cuuint32_t estr[2] = {1, 1};
  return enc(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

// C[M x N] = scale * sum_seg A_seg^T B_seg + diag * I on the tensor cores (pairs of SMs, 256 x 256 tiles).
// A_seg: K x M bf16 row-major, B_seg: K x N bf16 row-major (the contraction index is the slow one in memory).
// out_mode 0: bf16 C; 1: fp32 C; 2: C as a bf16 hi/lo pair (out, out_lo). M, N >= 256, multiples of 8; any K.
sc_status launch_tn_gemm(const void* const* A_segs, const void* const* B_segs, int nseg, int64_t K, int64_t M, int64_t N,
                         void* out, void* out_lo, int out_mode, float scale, float diag, unsigned* status,
                         cudaStream_t s) {
  if (nseg < 1 || nseg > 3 || M < 256 || N < 256 || (M % 8) || (N % 8) || K < 1) return SC_ERR_SHAPE;
  TnMaps maps;
  for (int i = 0; i < 3; ++i) {
    const int j = i < nseg ? i : 0;
    if (!encode_mn(&maps.a[i], A_segs[j], K, M) || !encode_mn(&maps.b[i], B_segs[j], K, N)) return SC_ERR_CUDA;
  }
  int dev = 0, n_sm = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n_sm < 2)
    return SC_ERR_CUDA;
  const size_t smem2 = (size_t)kW2Stages * kW2StageBytes + sizeof(W2Bars) + 1024;
  if (cudaFuncSetAttribute(wgrad_pair_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem2) != cudaSuccess)
    return SC_ERR_CUDA;
  const long long tiles2 = ((M + 255) / 256) * ((N + 255) / 256);
  const int n_pairs = tiles2 < n_sm / 2 ? (int)tiles2 : n_sm / 2;
  const TnEpilogue epi{out, out_lo, out_mode, scale, diag};
  wgrad_pair_kernel<true><<<2 * n_pairs, 192, smem2, s>>>(maps, nseg, epi, (int)K, (int)M, (int)N, M >= N ? 1 : 0, status);
  ++g_kernel_launches;
  return cudaGetLastError() == cudaSuccess ? SC_OK : SC_ERR_CUDA;
}

}  // namespace sc

using namespace sc;

extern "C" sc_status sc_masked_weight_grad(const void* dY_dev, const void* X_dev, void* Xm_dev, void* G_dev,
                                           int out_dtype, int64_t tokens, int64_t rows, int64_t cols, float keep,
                                           uint64_t seed, uint32_t layer, uint64_t step, void* status_dev,
                                           void* stream) {
  if (!dY_dev || !X_dev || !Xm_dev || !G_dev) return SC_ERR_INVALID_ARG;
  if (tokens <= 0 || rows <= 0 || cols <= 0 || tokens > (1 << 30) || rows > (1 << 30) || cols > (1 << 30))
    return SC_ERR_INVALID_ARG;
  if ((rows % 8) != 0 || (cols % 8) != 0) return SC_ERR_SHAPE;              // 16-byte row strides for TMA
  if (out_dtype != SC_DTYPE_BF16 && out_dtype != SC_DTYPE_FP32) return SC_ERR_DTYPE;
  if (!(keep > 0.f) || keep > 1.f) return SC_ERR_INVALID_ARG;
  const uintptr_t al = reinterpret_cast<uintptr_t>(dY_dev) | reinterpret_cast<uintptr_t>(X_dev) |
                       reinterpret_cast<uintptr_t>(Xm_dev) | reinterpret_cast<uintptr_t>(G_dev);
  if (al & 15) return SC_ERR_ALIGNMENT;
  cudaStream_t s = static_cast<cudaStream_t>(stream);

  // Algorithm 1 line 4: Xm = X . M (unscaled; the 1 / keep goes into the GEMM's fp32 epilogue)
  sc_status st = sc_apply_prf_mask(X_dev, Xm_dev, tokens, cols, keep, seed, layer, step, 0, stream);
  if (st != SC_OK) return st;
  long thr = lroundf(keep * 65536.f);
  if (thr < 1) thr = 1;
  if (thr > 65536) thr = 65536;
  const float scale = 65536.f / (float)thr;

  CUtensorMap map_dy, map_x;
  if (!encode_mn(&map_dy, dY_dev, tokens, rows) || !encode_mn(&map_x, Xm_dev, tokens, cols)) return SC_ERR_CUDA;
  int dev = 0, n_sm = 0;
  if (cudaGetDevice(&dev) != cudaSuccess ||
      cudaDeviceGetAttribute(&n_sm, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess)
    return SC_ERR_CUDA;
  const size_t smem = (size_t)kWgStages * kWgStageBytes + sizeof(WgBars) + 1024;
  if (cudaFuncSetAttribute(wgrad_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess)
    return SC_ERR_CUDA;
  static const bool pair_off = getenv("SC_WGRAD_ONE_CTA") != nullptr;       // test hook: force the one-block-per-tile kernel
  const long long tiles2 = ((rows + 255) / 256) * ((cols + 255) / 256);
  if (!pair_off && rows >= 256 && cols >= 256 && n_sm >= 2) {
    // pairs of SMs on 256 x 256 tiles (tcgen05 cta_group::2)
    const size_t smem2 = (size_t)kW2Stages * kW2StageBytes + sizeof(W2Bars) + 1024;
    if (cudaFuncSetAttribute(wgrad_pair_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem2) != cudaSuccess)
      return SC_ERR_CUDA;
    const int n_pairs = tiles2 < n_sm / 2 ? (int)tiles2 : n_sm / 2;
    TnMaps maps;
    maps.a[0] = map_dy; maps.b[0] = map_x;
    const TnEpilogue epi{G_dev, nullptr, out_dtype == SC_DTYPE_FP32 ? 1 : 0, scale, 0.f};
    wgrad_pair_kernel<false><<<2 * n_pairs, 192, smem2, s>>>(maps, 1, epi, (int)tokens, (int)rows, (int)cols,
                                                             rows >= cols ? 1 : 0, static_cast<unsigned*>(status_dev));
  } else {
    const long long tiles = ((rows + kWgBM - 1) / kWgBM) * ((cols + kWgBN - 1) / kWgBN);
    const int grid = tiles < n_sm ? (int)tiles : n_sm;
    wgrad_kernel<<<grid, 192, smem, s>>>(map_dy, map_x, G_dev, out_dtype == SC_DTYPE_FP32, (int)tokens, (int)rows,
                                         (int)cols, scale, rows >= cols ? 1 : 0, static_cast<unsigned*>(status_dev));
  }
  ++g_kernel_launches;
  return cudaGetLastError() == cudaSuccess ? SC_OK : SC_ERR_CUDA;
}
