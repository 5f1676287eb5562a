// Tensor-core (tcgen05 / TMEM / TMA) kernels of the spectral-correction step for sm_100a.
//
//   project_kernel        T = G (Vhi + Vlo)              streaming GEMM over the masked gradient, N = rank
//   pass_kernel           Y = M B / Z = M^T B         sweeps over the anchor momentum (tf32), range finder
//   fused_update_stream_kernel   G_proj = clip * (alpha_s G + (Uhi + Ulo)(Chi + Clo)^T), then AdamW, one HBM pass
//
// Operands: G is bf16 as given; the fp32 factors are carried as a sum of two bf16 numbers (hi + lo), so
// the products lose nothing that matters at the 2e-3 tolerance. All MMA operands sit in shared memory in
// the K-major, 128-byte-swizzled layout that both TMA (SWIZZLE_128B) and the UMMA descriptors understand.
// Every wait on an mbarrier is bounded; when a wait runs out the kernel latches an error bit, drains what
// it has in flight, frees its TMEM and returns.
#include <cuda.h>

#include "sc_internal.cuh"
#include "sc_ptx.cuh"

namespace sc {

constexpr int kMapsPerMat = 29;
constexpr int kPerCallMaps = 7;   // the first seven are rebuilt whenever the caller's buffers move
enum { MAP_G = 0,    // masked gradient, bf16, box 64 x 128 (MMA A operand of the projection)
       MAP_G32,      // masked gradient, bf16, box 32 x 128, 64-byte swizzle (streaming tile of the fused update)
       MAP_W, MAP_M1, MAP_M2,   // fp32 weights and AdamW moments, box 32 x 128, 128-byte swizzle (load and store)
       MAP_WB,       // bf16 weight copy, box 32 x 128, 64-byte swizzle (store only)
       MAP_MS,       // slow EMA of the dual-EMA optimizer, fp32, same box as MAP_M1 (a copy of MAP_M1 when unused)
       MAP_VTHI, MAP_VTLO, MAP_UHI, MAP_ULO, MAP_CTHI, MAP_CTLO,
       MAP_CT64HI, MAP_CT64LO,   // C^T with a 64 x 64 box (N = 64 tiles of the streaming update)
       MAP_M_K,      // anchor momentum as a K-major A operand: box 32 floats x 128 rows
       MAP_M_MN,     // anchor momentum as an MN-major A operand: box 32 floats x 32 rows (one swizzle atom column)
       MAP_Y, MAP_Z, MAP_OMEGA,  // m x lp, n x lp, n x lp row-major fp32 as MN-major B operands: box 32 x 32
       MAP_Y2, MAP_Z2,           // the scratch twins of Y and Z (a single-round Cholesky QR leaves its result there)
       MAP_GANC32,               // anchor gradient, bf16, box 32 x 128, 64-byte swizzle (rebuilt per anchor call)
       MAP_M_F32,                // anchor momentum as plain fp32 (box 32 x 128): load and store of the fused EMA sweep
       MAP_U_MN, MAP_T,          // fp32 U (m x rp) and T (m x rp) as MN-major panels: X = U^T T on the tensor cores
       MAP_SPARE,
       MAP_VTHI_H, MAP_VTLO_H };   // V^T hi / lo with a box of rp / 2 rows: one block's half of the B operand of a pair
constexpr int kTileBytes = 128 * 128;   // 128 rows x 64 bf16

// =====================================================================================================
// T = G V  (per 128-row tile of G and per K slice).  Warp 0: TMA producer. Warp 1: MMA issuer (owns TMEM).
// Warps 2-5: epilogue, TMEM -> registers -> global.
// =====================================================================================================
__global__ void __launch_bounds__(192, 2)
project_kernel(const MatDev* __restrict__ tab, const int* __restrict__ idx, const CUtensorMap* __restrict__ maps,
               int m, int n, int rp, int cps, int stages, uint32_t tmem_cols, unsigned* status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const int stage_bytes = kTileBytes + 2 * rp * 128;
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + (size_t)stages * stage_bytes);
  uint64_t* empty = full + stages;
  uint64_t* accum = empty + stages;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(accum + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  volatile int* never_flag = abort_flag + 1;   // stays 0: lets the drain below wait although abort is set

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int inst = blockIdx.z;
  const MatDev& md = tab[idx[inst]];
  const CUtensorMap* mp = maps + (size_t)md.inst * kMapsPerMat;
  const int row0 = blockIdx.x * 128;
  const int nchunks = (n + 63) >> 6;
  const int c0 = blockIdx.y * cps;
  const int my_chunks = min(cps, nchunks - c0);

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    mbar_init(accum, 1);
    *abort_flag = 0;
    *never_flag = 0;
    fence_barrier_init();
    fence_proxy_async();
  }
  if (warp == 1) tmem_alloc(tmem_slot, tmem_cols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_d = *tmem_slot;

  if (warp == 0 && lane == 0) {
    tensormap_acquire(mp + MAP_G); tensormap_acquire(mp + MAP_VTHI); tensormap_acquire(mp + MAP_VTLO);
    int issued = 0;
    for (int i = 0; i < my_chunks; ++i, ++issued) {
      const int s = i % stages;
      if (!mbar_wait(&empty[s], ((i / stages) & 1) ^ 1, abort_flag)) { atomicOr(status, kDevTimeout); *abort_flag = 1; break; }
      uint8_t* st = smem + (size_t)s * stage_bytes;
      mbar_expect_tx(&full[s], (uint32_t)stage_bytes);
      const int x = (c0 + i) * 64;
      tma_load_2d(st, mp + MAP_G, &full[s], x, row0);
      tma_load_2d(st + kTileBytes, mp + MAP_VTHI, &full[s], x, 0);
      tma_load_2d(st + kTileBytes + rp * 128, mp + MAP_VTLO, &full[s], x, 0);
    }
    if (*abort_flag) {   // let copies already in flight land before the block's shared memory goes away
      for (int i = max(0, issued - stages); i < issued; ++i) mbar_wait(&full[i % stages], (i / stages) & 1, never_flag);
    }
  } else if (warp == 1 && lane == 0) {
    const uint32_t idesc = umma_idesc_bf16(rp);
    for (int i = 0; i < my_chunks; ++i) {
      const int s = i % stages;
      if (!mbar_wait(&full[s], (i / stages) & 1, abort_flag)) { atomicOr(status, kDevTimeout); *abort_flag = 1; break; }
      tc_fence_after();
      const uint32_t a = smem_u32(smem + (size_t)s * stage_bytes);
      const uint32_t bh = a + kTileBytes, bl = bh + rp * 128;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const uint64_t ad = umma_desc_k128(a + k * 32);
        umma_bf16(tmem_d, ad, umma_desc_k128(bh + k * 32), idesc, (i | k) != 0);
        umma_bf16(tmem_d, ad, umma_desc_k128(bl + k * 32), idesc, 1);
      }
      umma_commit(&empty[s]);
    }
    umma_commit(accum);
  } else if (warp >= 2) {
    const int q = warp & 3;
    const int row = row0 + q * 32 + lane;
    bool ok = mbar_wait(accum, 0, abort_flag);
    if (!ok && lane == 0) { atomicOr(status, kDevTimeout); *abort_flag = 1; }
    ok = __all_sync(0xffffffffu, ok) && !*abort_flag;
    tc_fence_after();
    if (ok) {
      float* Trow = md.T + ((size_t)blockIdx.y * m + row) * rp;
      for (int c = 0; c < rp; c += 16) {
        float v[16];
        tmem_ld16(tmem_d + ((uint32_t)(q * 32) << 16) + c, v);
        tmem_ld_wait();
        if (row < m) {
#pragma unroll
          for (int j = 0; j < 16; j += 4)
            *reinterpret_cast<float4*>(Trow + c + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_d, tmem_cols);
}

// =====================================================================================================
// The same projection on PAIRS of SMs (a cluster of two blocks, tcgen05.mma cta_group::2, M = 256): each block streams
// its own 128 rows of G, but only HALF of every V^T tile (rp / 2 rows of the hi and of the lo part); the tensor cores of
// both SMs read the two halves. With one block per tile every 16 KB tile of G came with a full hi + lo V^T tile out
// of L2 and the kernel was bound by what TMA can bring into an SM (10.6 TB/s in all, half of it V^T); here the V^T
// share is halved. Block 0 of a pair issues the MMAs; its barriers collect both blocks' bytes and its commits arrive in
// both blocks. No multicast loads.
// =====================================================================================================
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(192, 2)
project_pair_kernel(const MatDev* __restrict__ tab, const int* __restrict__ idx, const CUtensorMap* __restrict__ maps,
                    int m, int n, int rp, int cps, int stages, uint32_t tmem_cols, unsigned* status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const int half_b = (rp / 2) * 128;                          // bytes of one block's half of V^T hi (or lo) per stage
  const int stage_bytes = kTileBytes + 2 * half_b;
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + (size_t)stages * stage_bytes);
  uint64_t* empty = full + stages;
  uint64_t* accum = empty + stages;
  uint64_t* drain = accum + 1;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(drain + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  volatile int* never_flag = abort_flag + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const MatDev& md = tab[idx[blockIdx.z]];
  const CUtensorMap* mp = maps + (size_t)md.inst * kMapsPerMat;
  const int row0 = (blockIdx.x >> 1) * 256 + (int)rank * 128;
  const int nchunks = (n + 63) >> 6;
  const int c0 = blockIdx.y * cps;
  const int my_chunks = min(cps, nchunks - c0);

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    mbar_init(accum, 1);
    mbar_init(drain, 1);
    *abort_flag = 0;
    *never_flag = 0;
    fence_barrier_init();
    fence_proxy_async();
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(tmem_cols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();            // the peer's barriers exist before anything is sent to them
  tc_fence_after();
  const uint32_t tmem_d = *tmem_slot;

  if (warp == 0 && lane == 0) {
    tensormap_acquire(mp + MAP_G); tensormap_acquire(mp + MAP_VTHI_H); tensormap_acquire(mp + MAP_VTLO_H);
    int issued = 0;
    bool dead = false;
    for (int i = 0; i < my_chunks; ++i, ++issued) {
      const int s = i % stages;
      if (!mbar_wait(&empty[s], ((i / stages) & 1) ^ 1, abort_flag)) { dead = true; break; }
      uint8_t* st = smem + (size_t)s * stage_bytes;
      if (rank == 0) mbar_expect_tx(&full[s], 2u * (uint32_t)stage_bytes);      // both blocks' bytes
      const uint32_t leader_bar = map_to_rank(smem_u32(&full[s]), 0);
      const int x = (c0 + i) * 64;
      tma_load_2d_pair(st, mp + MAP_G, leader_bar, x, row0);
      tma_load_2d_pair(st + kTileBytes, mp + MAP_VTHI_H, leader_bar, x, (int)rank * (rp / 2));
      tma_load_2d_pair(st + kTileBytes + half_b, mp + MAP_VTLO_H, leader_bar, x, (int)rank * (rp / 2));
    }
    if (dead) {
      atomicOr(status, kDevTimeout);
      *abort_flag = 1;
      // the bytes of both blocks are counted on the leader's barriers: the leader waits (bounded) for the stages it
      // armed, the other block idles for a grace period; both then meet in the cluster barrier at the end
      if (rank == 0) {
        for (int i = max(0, issued - stages); i < issued; ++i) mbar_wait(&full[i % stages], (i / stages) & 1, never_flag);
      } else {
        for (int i = 0; i < 64; ++i) __nanosleep(1000);
      }
    }
  } else if (warp == 1 && lane == 0 && rank == 0) {
    const uint32_t idesc = umma_idesc_bf16_pair(rp);
    bool dead = false;
    for (int i = 0; i < my_chunks; ++i) {
      const int s = i % stages;
      if (!mbar_wait(&full[s], (i / stages) & 1, abort_flag)) { dead = true; break; }
      tc_fence_after();
      const uint32_t a = smem_u32(smem + (size_t)s * stage_bytes);
      const uint32_t bh = a + kTileBytes, bl = bh + half_b;
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const uint64_t ad = umma_desc_k128(a + k * 32);
        umma_bf16_pair(tmem_d, ad, umma_desc_k128(bh + k * 32), idesc, (i | k) != 0);
        umma_bf16_pair(tmem_d, ad, umma_desc_k128(bl + k * 32), idesc, 1);
      }
      umma_commit_pair(&empty[s]);
    }
    if (!dead) {
      umma_commit_pair(accum);
    } else {
      atomicOr(status, kDevTimeout);
      *abort_flag = 1;
      // MMAs already issued still read both blocks' shared memory: wait (bounded) until they are done
      asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(drain)) : "memory");
      mbar_wait(drain, 0, never_flag);
    }
  } else if (warp >= 2) {
    const int q = warp & 3;
    const int row = row0 + q * 32 + lane;
    bool ok = my_chunks <= 0 || mbar_wait(accum, 0, abort_flag);
    if (!ok && lane == 0) { atomicOr(status, kDevTimeout); *abort_flag = 1; }
    ok = __all_sync(0xffffffffu, ok) && !*abort_flag;
    tc_fence_after();
    if (ok) {
      float* Trow = md.T + ((size_t)blockIdx.y * m + row) * rp;
      for (int c = 0; c < rp; c += 16) {
        float v[16];
        if (my_chunks > 0) {
          tmem_ld16(tmem_d + ((uint32_t)(q * 32) << 16) + c, v);
          tmem_ld_wait();
        } else {
#pragma unroll
          for (int j = 0; j < 16; ++j) v[j] = 0.f;
        }
        if (row < m) {
#pragma unroll
          for (int j = 0; j < 16; j += 4)
            *reinterpret_cast<float4*>(Trow + c + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();            // nothing of the peer is touched after this
  if (warp == 1)
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_d), "r"(tmem_cols) : "memory");
}

// =====================================================================================================
// One sweep over the anchor momentum for the range finder, tf32 tensor cores, fp32 operands read as they are:
//   TRANS = false:  OUT[m x lp] = M  * B,   B = Omega or Z (n x lp row-major)
//   TRANS = true :  OUT[n x lp] = M^T * B,  B = Y (m x lp row-major)
// K advances 32 per pipeline stage. B is always an MN-major operand (its rows are the K index): lp/32 swizzle
// atoms of 32 K-rows x 128 bytes. A is K-major for M (rows of M are rows of OUT) and MN-major for M^T (columns
// of M are rows of OUT: 4 atoms of 32 K-rows x 128 bytes). Same warp roles as project_kernel.
// =====================================================================================================
__device__ __forceinline__ void umma_tf32(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
      : "memory");
}
// MN-major operand of 32-bit elements: the only layout the tensor core takes is the 128-byte swizzle with
// 32-byte atomicity (32-byte chunks of a 128-byte row XORed with the row index mod 4; TMA writes it with
// SWIZZLE_128B_ATOM_32B). Atoms are 4 K-rows x 128 bytes; consecutive atoms along MN are `lbo` bytes apart,
// consecutive 4-row K groups 512 bytes apart.
__device__ __forceinline__ uint64_t umma_desc_mn128(uint32_t saddr, uint32_t lbo) {
  return (uint64_t)((saddr & 0x3FFFFu) >> 4) | ((uint64_t)(lbo >> 4) << 16) | ((uint64_t)(512 >> 4) << 32) |
         ((uint64_t)1 << 46) | ((uint64_t)1 << 61);
}
__device__ __forceinline__ uint32_t umma_idesc_tf32(int N, int a_mn, int b_mn) {
  return (1u << 4) | (2u << 7) | (2u << 10) | ((uint32_t)a_mn << 15) | ((uint32_t)b_mn << 16) |
         ((uint32_t)(N >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
}

// A operand held in tensor memory: lane = row of the 128-row tile, one 32-bit column = two consecutive bf16 along K,
// so a K step of 16 is 8 columns. tcgen05.cp moves exactly such a slab (128 rows x 256 bits) from a shared-memory
// tile described like an MMA operand into tensor memory; issued by the MMA thread it is ordered with its MMAs.
__device__ __forceinline__ void tmem_cp_128x256b(uint32_t taddr, uint64_t sdesc) {
  asm volatile("tcgen05.cp.cta_group::1.128x256b [%0], %1;" ::"r"(taddr), "l"(sdesc) : "memory");
}
__device__ __forceinline__ void umma_bf16_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
  asm volatile(
      "{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], %2, %3, p;\n\t}"
      ::"r"(d_tmem), "r"(a_tmem), "l"(bdesc), "r"(idesc), "r"(acc)
      : "memory");
}

constexpr int kPassK = 32;                       // K per stage
constexpr int kAtomBytes = kPassK * 128;         // one MN-major atom column: 32 K-rows x 128 bytes

struct PassArgs {
  int a_map, b_map;     // tensor maps of the A source (K-major box 32 x 128, or MN-major box 32 x 32) and of B (MN-major)
  int same_ab;          // A and B are the same panel (Gram matrix): load it once, both descriptors point at it
  int out_off;          // MatDev field of the output (or of the partial-sum buffer when the K range is split)
  int rows_out;         // valid output rows
  int kdim;             // contraction length
  int ncols;            // MMA N = B panel width, a multiple of 32
  int ncols_valid;      // columns written (multiple of 16)
  int ldo;              // output row stride in floats
  int cps;              // K chunks (of 32) per K slice; blockIdx.y selects the slice
  int stages;
  uint32_t tmem_cols;
};

template <bool TRANS>
__global__ void __launch_bounds__(192, 2)
pass_kernel(const MatDev* __restrict__ tab, const int* __restrict__ idx, const CUtensorMap* __restrict__ maps,
            PassArgs pa, unsigned* status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const int stages = pa.stages;
  const int b_bytes = pa.same_ab ? 0 : (pa.ncols / 32) * kAtomBytes;
  const int stage_bytes = kTileBytes + b_bytes;
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + (size_t)stages * stage_bytes);
  uint64_t* empty = full + stages;
  uint64_t* accum = empty + stages;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(accum + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);
  volatile int* never_flag = abort_flag + 1;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const MatDev& md = tab[idx[blockIdx.z]];
  const CUtensorMap* mp = maps + (size_t)md.inst * kMapsPerMat;
  const int row0 = blockIdx.x * 128;
  const int nchunks_all = (pa.kdim + kPassK - 1) / kPassK;
  const int c0 = blockIdx.y * pa.cps;
  const int nchunks = min(pa.cps, nchunks_all - c0);      // <= 0 for a trailing K slice with nothing in it: writes zeros

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) { mbar_init(&full[s], 1); mbar_init(&empty[s], 1); }
    mbar_init(accum, 1);
    *abort_flag = 0;
    *never_flag = 0;
    fence_barrier_init();
    fence_proxy_async();
  }
  if (warp == 1) tmem_alloc(tmem_slot, pa.tmem_cols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_d = *tmem_slot;

  if (warp == 0 && lane == 0) {
    const CUtensorMap* amap = mp + pa.a_map;
    const CUtensorMap* bmap = mp + pa.b_map;
    tensormap_acquire(amap); tensormap_acquire(bmap);
    int issued = 0;
    for (int i = 0; i < nchunks; ++i, ++issued) {
      const int s = i % stages;
      if (!mbar_wait(&empty[s], ((i / stages) & 1) ^ 1, abort_flag)) { atomicOr(status, kDevTimeout); *abort_flag = 1; break; }
      uint8_t* st = smem + (size_t)s * stage_bytes;
      mbar_expect_tx(&full[s], (uint32_t)stage_bytes);
      const int k0 = (c0 + i) * kPassK;
      if (!TRANS) {
        tma_load_2d(st, amap, &full[s], k0, row0);                                    // 128 rows x 32 floats
      } else {
#pragma unroll
        for (int a = 0; a < 4; ++a) tma_load_2d(st + a * kAtomBytes, amap, &full[s], row0 + 32 * a, k0);
      }
      if (!pa.same_ab)
        for (int a = 0; a < pa.ncols / 32; ++a) tma_load_2d(st + kTileBytes + a * kAtomBytes, bmap, &full[s], 32 * a, k0);
    }
    if (*abort_flag)
      for (int i = max(0, issued - stages); i < issued; ++i) mbar_wait(&full[i % stages], (i / stages) & 1, never_flag);
  } else if (warp == 1 && lane == 0) {
    const uint32_t idesc = umma_idesc_tf32(pa.ncols, TRANS ? 1 : 0, 1);
    for (int i = 0; i < nchunks; ++i) {
      const int s = i % stages;
      if (!mbar_wait(&full[s], (i / stages) & 1, abort_flag)) { atomicOr(status, kDevTimeout); *abort_flag = 1; break; }
      tc_fence_after();
      const uint32_t a = smem_u32(smem + (size_t)s * stage_bytes);
      const uint32_t b = pa.same_ab ? a : a + kTileBytes;
#pragma unroll
      for (int k = 0; k < kPassK / 8; ++k) {
        const uint64_t ad = TRANS ? umma_desc_mn128(a + k * 1024, kAtomBytes) : umma_desc_k128(a + k * 32);
        umma_tf32(tmem_d, ad, umma_desc_mn128(b + k * 1024, kAtomBytes), idesc, (i | k) != 0);
      }
      umma_commit(&empty[s]);
    }
    if (nchunks > 0) umma_commit(accum);
  } else if (warp >= 2) {
    const int q = warp & 3;
    const int row = row0 + q * 32 + lane;
    bool ok = nchunks <= 0 || mbar_wait(accum, 0, abort_flag);
    if (!ok && lane == 0) { atomicOr(status, kDevTimeout); *abort_flag = 1; }
    ok = __all_sync(0xffffffffu, ok) && !*abort_flag;
    tc_fence_after();
    if (ok) {
      float* out = *reinterpret_cast<float* const*>(reinterpret_cast<const char*>(&md) + pa.out_off) +
                   ((size_t)blockIdx.y * pa.rows_out + row) * pa.ldo;
      for (int c = 0; c < pa.ncols_valid; c += 16) {
        float v[16];
        if (nchunks > 0) {
          tmem_ld16(tmem_d + ((uint32_t)(q * 32) << 16) + c, v);
          tmem_ld_wait();
        } else {
#pragma unroll
          for (int j = 0; j < 16; ++j) v[j] = 0.f;
        }
        if (row < pa.rows_out) {
#pragma unroll
          for (int j = 0; j < 16; j += 4)
            *reinterpret_cast<float4*>(out + c + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_d, pa.tmem_cols);
}

// =====================================================================================================
// First sweep of the range finder fused with the anchor EMA (Eq. 1): the block streams its 128 rows of the OLD
// momentum and of the bf16 anchor gradient, four warps form M_new = beta M + (1 - beta) G_anc in shared memory,
// one thread sends the tile back with a TMA store while the MMA warp consumes the same tile for Y = M_new B.
// The momentum is read once and written once for Eq. 1 and this sweep together.
//   warp 0 producer | warp 1 MMA | warps 2-5 transform, later epilogue | warp 6 store
// =====================================================================================================
constexpr int kGancTile = 128 * 32 * 2;   // bf16, 128 rows x 32 columns

__global__ void __launch_bounds__(224, 2)
ema_pass_kernel(const MatDev* __restrict__ tab, const int* __restrict__ idx, const CUtensorMap* __restrict__ maps,
                int b_map, int m, int n, int lp, int stages, uint32_t tmem_cols, float beta, unsigned* status) {
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const int b_bytes = (lp / 32) * kAtomBytes;
  const int stage_bytes = kTileBytes + kGancTile + b_bytes;
  uint64_t* full = reinterpret_cast<uint64_t*>(smem + (size_t)stages * stage_bytes);
  uint64_t* ready = full + stages;
  uint64_t* empty = ready + stages;
  uint64_t* accum = empty + stages;
  uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(accum + 1);
  volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const MatDev& md = tab[idx[blockIdx.z]];
  const CUtensorMap* mp = maps + (size_t)md.inst * kMapsPerMat;
  const int row0 = blockIdx.x * 128;
  const int nchunks = (n + kPassK - 1) / kPassK;

  if (threadIdx.x == 0) {
    for (int s = 0; s < stages; ++s) { mbar_init(&full[s], 1); mbar_init(&ready[s], 4); mbar_init(&empty[s], 2); }
    mbar_init(accum, 1);
    *abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async();
  }
  if (warp == 1) tmem_alloc(tmem_slot, tmem_cols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_d = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      const CUtensorMap* bmap = mp + b_map;
      tensormap_acquire(mp + MAP_M_F32); tensormap_acquire(mp + MAP_GANC32); tensormap_acquire(bmap);
      int issued = 0;
      for (int i = 0; i < nchunks; ++i, ++issued) {
        const int s = i % stages;
        if (!mbar_wait(&empty[s], ((i / stages) & 1) ^ 1, abort_flag)) { atomicOr(status, kDevTimeout); *abort_flag = 1; break; }
        uint8_t* st = smem + (size_t)s * stage_bytes;
        mbar_expect_tx(&full[s], (uint32_t)stage_bytes);
        const int k0 = i * kPassK;
        tma_load_2d(st, mp + MAP_M_F32, &full[s], k0, row0);
        tma_load_2d(st + kTileBytes, mp + MAP_GANC32, &full[s], k0, row0);
        for (int a = 0; a < lp / 32; ++a)
          tma_load_2d(st + kTileBytes + kGancTile + a * kAtomBytes, bmap, &full[s], 32 * a, k0);
      }
      if (*abort_flag) {   // let the copies already in flight land before the block's shared memory goes away
        volatile int never = 0;
        for (int i = max(0, issued - stages); i < issued; ++i) mbar_wait(&full[i % stages], (i / stages) & 1, &never);
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    if (lane == 0) {
      const uint32_t idesc = umma_idesc_tf32(lp, 0, 1);
      for (int i = 0; i < nchunks; ++i) {
        const int s = i % stages;
        if (!mbar_wait(&ready[s], (i / stages) & 1, abort_flag)) { atomicOr(status, kDevTimeout); *abort_flag = 1; break; }
        tc_fence_after();
        const uint32_t a = smem_u32(smem + (size_t)s * stage_bytes);
        const uint32_t b = a + kTileBytes + kGancTile;
#pragma unroll
        for (int k = 0; k < kPassK / 8; ++k)
          umma_tf32(tmem_d, umma_desc_k128(a + k * 32), umma_desc_mn128(b + k * 1024, kAtomBytes), idesc, (i | k) != 0);
        umma_commit(&empty[s]);
      }
      umma_commit(accum);
    }
    __syncwarp();
  } else if (warp == 6) {
    if (lane == 0) {
      tensormap_acquire(mp + MAP_M_F32);
      for (int i = 0; i < nchunks; ++i) {
        const int s = i % stages;
        if (!mbar_wait(&ready[s], (i / stages) & 1, abort_flag)) { atomicOr(status, kDevTimeout); *abort_flag = 1; break; }
        tma_store_2d(mp + MAP_M_F32, smem + (size_t)s * stage_bytes, i * kPassK, row0);
        tma_store_commit();
        tma_store_wait_read<0>();
        mbar_arrive(&empty[s]);
      }
      tma_store_wait_all();
    }
    __syncwarp();
  } else {
    // transform warps: one row per thread, 32 columns per chunk
    const int q = warp & 3;
    const int r = q * 32 + lane;
    const float omb = 1.f - beta;
    bool dead = false;
    for (int i = 0; i < nchunks; ++i) {
      const int s = i % stages;
      if (!mbar_wait(&full[s], (i / stages) & 1, abort_flag)) { dead = true; break; }
      uint8_t* st = smem + (size_t)s * stage_bytes;
      float4* Ms = reinterpret_cast<float4*>(st);
      const uint4* Gs = reinterpret_cast<const uint4*>(st + kTileBytes);
#pragma unroll
      for (int cg = 0; cg < 4; ++cg) {
        const uint4 graw = Gs[r * 4 + (cg ^ ((r >> 1) & 3))];
        const uint32_t gw[4] = {graw.x, graw.y, graw.z, graw.w};
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          const int fidx = r * 8 + ((2 * cg + h) ^ (r & 7));
          float4 mv = Ms[fidx];
          const __nv_bfloat162 g01 = *reinterpret_cast<const __nv_bfloat162*>(&gw[2 * h]);
          const __nv_bfloat162 g23 = *reinterpret_cast<const __nv_bfloat162*>(&gw[2 * h + 1]);
          mv.x = fmaf(beta, mv.x, omb * __low2float(g01));
          mv.y = fmaf(beta, mv.y, omb * __high2float(g01));
          mv.z = fmaf(beta, mv.z, omb * __low2float(g23));
          mv.w = fmaf(beta, mv.w, omb * __high2float(g23));
          Ms[fidx] = mv;
        }
      }
      fence_proxy_async();          // the new tile must be visible to the MMA and to the TMA store
      __syncwarp();
      if (lane == 0) mbar_arrive(&ready[s]);
    }
    // epilogue: Y rows from the accumulator
    bool ok = !dead && mbar_wait(accum, 0, abort_flag);
    if (!ok && lane == 0) { atomicOr(status, kDevTimeout); *abort_flag = 1; }
    ok = __all_sync(0xffffffffu, ok) && !*abort_flag;
    tc_fence_after();
    if (ok) {
      const int row = row0 + r;
      float* out = md.Y + (size_t)row * lp;
      for (int c = 0; c < lp; c += 16) {
        float v[16];
        tmem_ld16(tmem_d + ((uint32_t)(q * 32) << 16) + c, v);
        tmem_ld_wait();
        if (row < m) {
#pragma unroll
          for (int j = 0; j < 16; j += 4)
            *reinterpret_cast<float4*>(out + c + j) = make_float4(v[j], v[j + 1], v[j + 2], v[j + 3]);
        }
      }
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_d, tmem_cols);
}

// =====================================================================================================
// AdamW on four elements of G_proj = clip * (alpha_s * G + R), R = the low-rank part from the tensor cores.
// =====================================================================================================
// Square root and quotient without the special-case branches of the IEEE expansions: those branches end the
// basic block after every element, so the sixteen element chains of a thread would run one after another.
// sqrt.approx is within 1 ulp; the quotient takes the hardware reciprocal (1 ulp) and one residual correction,
// which leaves it within 1 ulp of the rounded quotient. den >= eps > 0 and vo >= 0 always hold here.
__device__ __forceinline__ float sqrt_nobranch(float x) {
  float y;
  asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float div_nobranch(float a, float b) {
  float r;
  asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(b));
  const float q = a * r;
  return fmaf(fmaf(-b, q, a), r, q);
}

__device__ __forceinline__ void adamw4(const StepScalars& s, float clip, const float g_raw[4], const float4& r,
                                       float4& w, float4& m1, float4& m2, float4& gp) {
  const float rr[4] = {r.x, r.y, r.z, r.w};
  float* W = &w.x; float* M1 = &m1.x; float* M2 = &m2.x; float* GP = &gp.x;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const float g = clip * fmaf(s.alpha_s, g_raw[j], rr[j]);
    const float mo = fmaf(s.beta1, M1[j], s.one_m_beta1 * g);
    const float vo = fmaf(s.beta2, M2[j], s.one_m_beta2 * g * g);
    const float den = fmaf(sqrt_nobranch(vo), s.inv_sqrt_bc2, s.eps);
    W[j] = fmaf(-s.step_size, div_nobranch(mo, den), W[j] * s.decay);
    M1[j] = mo; M2[j] = vo; GP[j] = g;
  }
}

// The same four elements under the dual-EMA optimizer: the slow average ms of G_proj (decay beta3, no bias correction)
// joins the bias-corrected fast average in the numerator.
__device__ __forceinline__ void ademamix4(const StepScalars& s, float clip, const float g_raw[4], const float4& r,
                                          float4& w, float4& m1, float4& m2, float4& ms, float4& gp) {
  const float rr[4] = {r.x, r.y, r.z, r.w};
  float* W = &w.x; float* M1 = &m1.x; float* M2 = &m2.x; float* MS = &ms.x; float* GP = &gp.x;
#pragma unroll
  for (int j = 0; j < 4; ++j) {
    const float g = clip * fmaf(s.alpha_s, g_raw[j], rr[j]);
    const float mo = fmaf(s.beta1, M1[j], s.one_m_beta1 * g);
    const float so = fmaf(s.beta3, MS[j], s.one_m_beta3 * g);
    const float vo = fmaf(s.beta2, M2[j], s.one_m_beta2 * g * g);
    const float den = fmaf(sqrt_nobranch(vo), s.inv_sqrt_bc2, s.eps);
    W[j] = W[j] * s.decay - div_nobranch(fmaf(s.lr_mix, so, s.step_size * mo), den);
    M1[j] = mo; M2[j] = vo; MS[j] = so; GP[j] = g;
  }
}

// =====================================================================================================
// Fused correction + AdamW, streaming form: no thread touches global memory for the state.
//   Persistent blocks (one per SM) draw work items (matrix, 128-row panel, one 64-column tile) from a counter.
//   warp 0   producer: TMA loads of the MMA operands (U panel, C^T tile) and of the streaming units
//            (128 rows x 32 columns of W, m, v fp32 and G bf16) into a 3-stage ring
//   warp 1   MMA issuer: R = (Uhi + Ulo)(Chi + Clo)^T for a 128 x 64 tile into one of two TMEM accumulators
//   warps 2-9  consumers, one thread per (row, half unit): R from TMEM, W/m/v/G from swizzled shared memory,
//            blend + AdamW, results written back in place; one elected thread sends the unit out with TMA stores
//            and hands the stage back once those stores have read it.
// UT = true (ranks above 64, i.e. more than one 64-wide K chunk): the U panel of a work item lives in TENSOR memory.
// With U in shared memory every 128 x 64 tile re-fetched 32 KB of U per K chunk from L2, and at rank 128 / 256 that
// traffic (12 / 24 B per element on top of the 28 streamed) made the kernel bound by what TMA can bring into the SM.
// Here a work item is a run of four column tiles of one row panel: the producer sends the panel's U chunks once per
// item through the 16 KB operand slots, the MMA thread copies them into tensor memory (tcgen05.cp, rk columns beside
// the two accumulators) and every tile of the item takes its A operand from there; only the C^T chunks (16 KB each)
// are fetched per tile.
// MIX = true is the dual-EMA optimizer: a fourth fp32 array (the slow average) travels with every unit, so a stage
// is 72 KB and only two fit beside the operands. With two stages a stage has to go back to the producer as soon as
// its stores have read it, so a warp of its own (warp 10) issues the stores and waits for them, instead of a
// consumer thread that would stall its warp.
// =====================================================================================================
constexpr int kUnitW = 32;                                   // columns per streaming unit
constexpr int kTileN = 64;                                   // columns per MMA tile (2 units)
constexpr int kUnitF32 = 128 * kUnitW * 4;                   // 16 KB: one fp32 array of a unit
constexpr int kUnitBf16 = 128 * kUnitW * 2;                  // 8 KB
constexpr int kStreamStages = 3;                             // most stages any variant uses (sizes the barrier arrays)
constexpr int kOpndU = 2 * kTileBytes;                       // U hi + lo, 128 rows x 64 bf16 each
constexpr int kOpndC = 2 * (kTileN * 128);                   // C^T hi + lo, 64 rows x 64 bf16 each
constexpr int kOpSlot = 16 * 1024;      // UT: one operand slot = a 128 x 64 bf16 tile of U (hi or lo), or C^T hi + lo (2 x 8 KB)
constexpr int kMaxOpSlots = 6;
template <bool MIX, bool UT = false>
struct StreamCfg {
  static constexpr int kF32 = MIX ? 4 : 3;                              // fp32 arrays per unit: W, m, v (, slow m)
  // Measured for UT on the 70B-shaped slice at rank 128 (update kernel against the HBM peak): three stages and three
  // operand slots 0.894, the same with the store warp 0.904, two stages with six slots and the store warp 0.859, two
  // stages with six slots without it 0.70 (one 14336 x 4096 matrix at rank 256: 0.81 / 0.81 / 0.83 / 0.64).
  static constexpr int kStages = MIX ? 2 : 3;
  static constexpr int kStageBytes = kF32 * kUnitF32 + kUnitBf16;      // 56 KB / 72 KB
  static constexpr int kOps = (UT && MIX) ? 4 : 3;                      // operand slots (UT); what fits beside the stages
  static constexpr int kSmem = kStages * kStageBytes + (UT ? kOps * kOpSlot : kOpndU + kOpndC);
  static constexpr bool kStoreWarpOn = MIX || UT;                       // a warp of its own sends the units out
  static constexpr int kStoreWarp = 10;
};
// warps: 0 producer, 1 MMA, 2-9 consumers, then one store warp (MIX, UT)
template <bool MIX, bool UT>
constexpr int stream_threads() { return 320 + ((MIX || UT) ? 32 : 0); }

// Work items are handed out by an atomic counter: blocks do not run at the same speed (the slowest of a static split
// finished 7% after the median), so each block's producer draws the next item when it needs one and passes the index
// to the MMA issuer and the consumers through a small ring in shared memory. The producer can be at most three
// units, i.e. fewer than kItemSlots items, ahead of the consumers, so a slot is never rewritten while still in use.
constexpr int kItemSlots = 8;

struct StreamBars {
  uint64_t full[kStreamStages], empty[kStreamStages];
  uint64_t opnd_full, opnd_empty;
  uint64_t op_full[kMaxOpSlots], op_empty[kMaxOpSlots];      // UT only: ring of 16 KB operand slots
  uint64_t acc_full[2], acc_empty[2];
  uint64_t item_ready[kItemSlots];
  uint64_t store_ready[kStreamStages];   // store-warp variants: the consumers have finished a unit, the store warp may send it
  int item_slot[kItemSlots];
  uint32_t tmem_slot;
  int abort_flag;
};

struct StreamGeom {
  int m, n, rp;
  int row_tiles, col_tiles, csplit, tiles_per_chunk, n_items;
};

__device__ __forceinline__ void decode_item(const StreamGeom& g, int item, int& inst, int& rt, int& ct0, int& ct1) {
  const int per_inst = g.row_tiles * g.csplit;
  inst = item / per_inst;
  const int rem = item - inst * per_inst;
  rt = rem / g.csplit;
  const int ch = rem - rt * g.csplit;
  ct0 = ch * g.tiles_per_chunk;
  ct1 = min(g.col_tiles, ct0 + g.tiles_per_chunk);
}

template <bool MIX, bool UT>
__global__ void __launch_bounds__(stream_threads<MIX, UT>(), 1)
fused_update_stream_kernel(const MatDev* __restrict__ tab, const int* __restrict__ idx,
                           const CUtensorMap* __restrict__ maps, StreamGeom g, StepScalars sc,
                           const float* __restrict__ clip_ptr, unsigned* status, unsigned* work_counter) {
  constexpr int kStages = StreamCfg<MIX, UT>::kStages, kStreamStageBytes = StreamCfg<MIX, UT>::kStageBytes;
  constexpr int kStreamSmem = StreamCfg<MIX, UT>::kSmem, kF32 = StreamCfg<MIX, UT>::kF32;
  constexpr int kOps = StreamCfg<MIX, UT>::kOps;
  constexpr bool SW = StreamCfg<MIX, UT>::kStoreWarpOn;
  extern __shared__ uint8_t smem_raw[];
  uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint8_t* opnd = smem + kStages * kStreamStageBytes;
  StreamBars* bars = reinterpret_cast<StreamBars*>(smem + kStreamSmem);
  volatile int* abort_flag = &bars->abort_flag;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int nch = (g.rp + 63) >> 6;

  if (threadIdx.x == 0) {
    for (int s = 0; s < kStreamStages; ++s) {
      mbar_init(&bars->full[s], 1); mbar_init(&bars->empty[s], 1); mbar_init(&bars->store_ready[s], 1);
    }
    mbar_init(&bars->opnd_full, 1);
    mbar_init(&bars->opnd_empty, 1);
    for (int k = 0; k < kMaxOpSlots; ++k) { mbar_init(&bars->op_full[k], 1); mbar_init(&bars->op_empty[k], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&bars->acc_full[a], 1); mbar_init(&bars->acc_empty[a], 8); }
    for (int k = 0; k < kItemSlots; ++k) mbar_init(&bars->item_ready[k], 1);
    bars->abort_flag = 0;
    fence_barrier_init();
    fence_proxy_async();
  }
  // UT: the two accumulators plus rk columns for the U panel (hi: rk / 2 columns, lo: rk / 2), a power of two
  const uint32_t tmem_cols = !UT ? 2 * kTileN : (2 * kTileN + nch * 64 <= 256 ? 256u : 512u);
  if (warp == 1) tmem_alloc(&bars->tmem_slot, tmem_cols);
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = bars->tmem_slot;

  if (warp == 0) {
    if (lane == 0) {
      // ------------------------------------------------------------------ producer
      uint32_t unit_it = 0, op_it = 0;
      int last_inst = -1, last_panel = -1;
      bool dead = false;
      uint32_t item_it = 0;
      int next_item = (int)atomicAdd(work_counter, 1u);
      while (!dead) {
        const int item = next_item < g.n_items ? next_item : -1;
        volatile int* slot = &bars->item_slot[item_it % kItemSlots];
        *slot = item;
        mbar_arrive(&bars->item_ready[item_it % kItemSlots]);   // release: the slot is visible to whoever sees this phase
        ++item_it;
        if (item < 0) break;
        next_item = (int)atomicAdd(work_counter, 1u);           // drawn one item ahead, so its latency is hidden
        int inst, rt, ct0, ct1;
        decode_item(g, item, inst, rt, ct0, ct1);
        const MatDev& md = tab[idx[inst]];
        const CUtensorMap* mp = maps + (size_t)md.inst * kMapsPerMat;
        if (inst != last_inst) {
          tensormap_acquire(mp + MAP_UHI); tensormap_acquire(mp + MAP_ULO);
          tensormap_acquire(mp + MAP_CT64HI); tensormap_acquire(mp + MAP_CT64LO);
          tensormap_acquire(mp + MAP_W); tensormap_acquire(mp + MAP_M1); tensormap_acquire(mp + MAP_M2);
          tensormap_acquire(mp + MAP_G32);
          if (MIX) tensormap_acquire(mp + MAP_MS);
          last_inst = inst;
          last_panel = -1;
        }
        const int row0 = rt * 128;
        for (int ct = ct0; ct < ct1 && !dead; ++ct) {
          if (UT) {
            // operand slots in the order the MMA thread consumes them: at the start of an item U hi and U lo of every
            // K chunk, then for every tile its C^T chunks. (A thread of its own for these loads was measured and
            // dropped: no gain on the 70B-shaped set, slower on a single matrix.)
            const int n_u = ct == ct0 ? 2 * nch : 0;
            for (int j = 0; j < n_u + nch && !dead; ++j, ++op_it) {
              const int sl = op_it % kOps;
              if (!mbar_wait(&bars->op_empty[sl], ((op_it / kOps) & 1) ^ 1, abort_flag)) { dead = true; break; }
              uint8_t* dst = opnd + sl * kOpSlot;
              mbar_expect_tx(&bars->op_full[sl], kOpSlot);
              if (j < n_u) {
                tma_load_2d(dst, mp + ((j & 1) ? MAP_ULO : MAP_UHI), &bars->op_full[sl], (j >> 1) * 64, row0);
              } else {
                const int kc = j - n_u;
                tma_load_2d(dst, mp + MAP_CT64HI, &bars->op_full[sl], kc * 64, ct * kTileN);
                tma_load_2d(dst + kTileN * 128, mp + MAP_CT64LO, &bars->op_full[sl], kc * 64, ct * kTileN);
              }
            }
          }
          for (int kc = 0; !UT && kc < nch; ++kc, ++op_it) {
            if (!mbar_wait(&bars->opnd_empty, (op_it & 1) ^ 1, abort_flag)) { dead = true; break; }
            const bool load_u = nch > 1 || last_panel != rt;
            mbar_expect_tx(&bars->opnd_full, kOpndC + (load_u ? kOpndU : 0));
            if (load_u) {
              tma_load_2d(opnd, mp + MAP_UHI, &bars->opnd_full, kc * 64, row0);
              tma_load_2d(opnd + kTileBytes, mp + MAP_ULO, &bars->opnd_full, kc * 64, row0);
            }
            tma_load_2d(opnd + kOpndU, mp + MAP_CT64HI, &bars->opnd_full, kc * 64, ct * kTileN);
            tma_load_2d(opnd + kOpndU + kTileN * 128, mp + MAP_CT64LO, &bars->opnd_full, kc * 64, ct * kTileN);
          }
          if (dead) break;
          last_panel = rt;
          const int units = (g.n - ct * kTileN > kUnitW) ? 2 : 1;
          for (int u = 0; u < units; ++u, ++unit_it) {
            const int s = unit_it % kStages;
            if (!mbar_wait(&bars->empty[s], ((unit_it / kStages) & 1) ^ 1, abort_flag)) { dead = true; break; }
            uint8_t* st = smem + (size_t)s * kStreamStageBytes;
            const int x = ct * kTileN + u * kUnitW;
            mbar_expect_tx(&bars->full[s], kStreamStageBytes);
            tma_load_2d(st, mp + MAP_W, &bars->full[s], x, row0);
            tma_load_2d(st + kUnitF32, mp + MAP_M1, &bars->full[s], x, row0);
            tma_load_2d(st + 2 * kUnitF32, mp + MAP_M2, &bars->full[s], x, row0);
            if (MIX) tma_load_2d(st + 3 * kUnitF32, mp + MAP_MS, &bars->full[s], x, row0);
            tma_load_2d(st + kF32 * kUnitF32, mp + MAP_G32, &bars->full[s], x, row0);
          }
        }
      }
      if (dead) {
        atomicOr(status, kDevTimeout);
        *abort_flag = 1;
        // let the copies already in flight land before this block's shared memory goes away (bounded waits)
        volatile int never = 0;
        for (uint32_t u = unit_it > (uint32_t)kStages ? unit_it - kStages : 0; u < unit_it; ++u)
          mbar_wait(&bars->full[u % kStages], (u / kStages) & 1, &never);
        if (!UT && op_it > 0) mbar_wait(&bars->opnd_full, (op_it - 1) & 1, &never);
        if (UT)
          for (uint32_t u = op_it > (uint32_t)kOps ? op_it - kOps : 0; u < op_it; ++u)
            mbar_wait(&bars->op_full[u % kOps], (u / kOps) & 1, &never);
      }
    }
    __syncwarp();
  } else if (warp == 1) {
    if (lane == 0) {
      // ------------------------------------------------------------------ MMA issuer
      const uint32_t idesc = umma_idesc_bf16(kTileN);
      const uint32_t uh = smem_u32(opnd), ul = uh + kTileBytes, ch = uh + kOpndU, cl = ch + kTileN * 128;
      uint32_t op_it = 0, t = 0;
      bool dead = false;
      for (uint32_t item_it = 0; !dead; ++item_it) {
        if (!mbar_wait(&bars->item_ready[item_it % kItemSlots], (item_it / kItemSlots) & 1, abort_flag)) { dead = true; break; }
        const int item = *reinterpret_cast<volatile int*>(&bars->item_slot[item_it % kItemSlots]);
        if (item < 0) break;
        int inst, rt, ct0, ct1;
        decode_item(g, item, inst, rt, ct0, ct1);
        for (int ct = ct0; ct < ct1 && !dead; ++ct, ++t) {
          const uint32_t ab = t & 1;
          if (!mbar_wait(&bars->acc_empty[ab], ((t >> 1) & 1) ^ 1, abort_flag)) { dead = true; break; }
          tc_fence_after();
          const uint32_t d = tmem_base + ab * kTileN;
          if (UT) {
            const uint32_t u_hi = tmem_base + 2 * kTileN, u_lo = u_hi + nch * 32;    // nch * 32 columns = rk / 2
            const int n_u = ct == ct0 ? 2 * nch : 0;
            for (int j = 0; j < n_u + nch && !dead; ++j, ++op_it) {
              const int sl = op_it % kOps;
              if (!mbar_wait(&bars->op_full[sl], (op_it / kOps) & 1, abort_flag)) { dead = true; break; }
              tc_fence_after();
              const uint32_t sa = uh + sl * kOpSlot;
              if (j < n_u) {        // a U chunk: four K steps of 16 into tensor memory
                const uint32_t dst = ((j & 1) ? u_lo : u_hi) + (j >> 1) * 32;
#pragma unroll
                for (int k = 0; k < 4; ++k) tmem_cp_128x256b(dst + k * 8, umma_desc_k128(sa + k * 32));
              } else {
                const int kc = j - n_u;
                const int ksteps = min(64, g.rp - kc * 64) >> 4;
                const uint32_t sb = sa + kTileN * 128;
                for (int k = 0; k < ksteps; ++k) {
                  const uint32_t ah = u_hi + (kc * 4 + k) * 8, al = u_lo + (kc * 4 + k) * 8;
                  const uint64_t bh = umma_desc_k128(sa + k * 32), bl = umma_desc_k128(sb + k * 32);
                  umma_bf16_ts(d, ah, bh, idesc, (kc | k) != 0);
                  umma_bf16_ts(d, ah, bl, idesc, 1);
                  umma_bf16_ts(d, al, bh, idesc, 1);
                }
              }
              umma_commit(&bars->op_empty[sl]);
            }
          }
          for (int kc = 0; !UT && kc < nch; ++kc, ++op_it) {
            if (!mbar_wait(&bars->opnd_full, op_it & 1, abort_flag)) { dead = true; break; }
            tc_fence_after();
            const int ksteps = min(64, g.rp - kc * 64) >> 4;
            for (int k = 0; k < ksteps; ++k) {
              const uint64_t ah = umma_desc_k128(uh + k * 32), al = umma_desc_k128(ul + k * 32);
              const uint64_t bh = umma_desc_k128(ch + k * 32), bl = umma_desc_k128(cl + k * 32);
              umma_bf16(d, ah, bh, idesc, (kc | k) != 0);
              umma_bf16(d, ah, bl, idesc, 1);
              umma_bf16(d, al, bh, idesc, 1);
            }
            umma_commit(&bars->opnd_empty);
          }
          if (dead) break;
          umma_commit(&bars->acc_full[ab]);
        }
      }
      if (dead) { atomicOr(status, kDevTimeout); *abort_flag = 1; }
    }
    __syncwarp();
  } else if (warp >= 2 && warp < 10) {
    // -------------------------------------------------------------------- consumers
    const int q = warp & 3, h = (warp - 2) >> 2;
    const int r = q * 32 + lane;                 // row inside the 128-row panel
    const bool leader = warp == 2 && lane == 0;
    const float clip = *clip_ptr;
    uint32_t unit_it = 0, t = 0;
    int last_inst = -1;
    bool dead = false;
    for (uint32_t item_it = 0; !dead; ++item_it) {
      if (!mbar_wait(&bars->item_ready[item_it % kItemSlots], (item_it / kItemSlots) & 1, abort_flag)) { dead = true; break; }
      const int item = *reinterpret_cast<volatile int*>(&bars->item_slot[item_it % kItemSlots]);
      if (item < 0) break;
      int inst, rt, ct0, ct1;
      decode_item(g, item, inst, rt, ct0, ct1);
      const MatDev& md = tab[idx[inst]];
      const CUtensorMap* mp = maps + (size_t)md.inst * kMapsPerMat;
      if (!SW && leader && inst != last_inst) {
        tensormap_acquire(mp + MAP_W); tensormap_acquire(mp + MAP_M1); tensormap_acquire(mp + MAP_M2);
        tensormap_acquire(mp + MAP_WB);
      }
      last_inst = inst;
      const int row0 = rt * 128;
      float* gp_dbg = md.gproj_dbg;
      const bool has_wb = md.Wb != nullptr;
      for (int ct = ct0; ct < ct1 && !dead; ++ct, ++t) {
        const uint32_t ab = t & 1;
        if (!mbar_wait(&bars->acc_full[ab], (t >> 1) & 1, abort_flag)) { dead = true; break; }
        tc_fence_after();
        const int units = (g.n - ct * kTileN > kUnitW) ? 2 : 1;
        for (int u = 0; u < units; ++u, ++unit_it) {
          const int s = unit_it % kStages;
          if (!mbar_wait(&bars->full[s], (unit_it / kStages) & 1, abort_flag)) { dead = true; break; }
          uint8_t* st = smem + (size_t)s * kStreamStageBytes;
          float rv[16];
          tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + ab * kTileN + u * kUnitW + h * 16, rv);
          tmem_ld_wait();
          float4* Ws = reinterpret_cast<float4*>(st);
          float4* M1s = reinterpret_cast<float4*>(st + kUnitF32);
          float4* M2s = reinterpret_cast<float4*>(st + 2 * kUnitF32);
          float4* MSs = reinterpret_cast<float4*>(st + 3 * kUnitF32);   // MIX only
          uint4* Gs = reinterpret_cast<uint4*>(st + kF32 * kUnitF32);
          // all of this thread's 16 elements are read first, so that the 16 AdamW chains are independent work for
          // the scheduler; results go back in place afterwards
          int fidx[4], gidx[2];
          float4 w[4], m1[4], m2[4], ms[4], gp[4];
          uint4 graw[2];
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            gidx[j] = r * 4 + ((2 * h + j) ^ ((r >> 1) & 3));
            graw[j] = Gs[gidx[j]];
          }
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            fidx[i] = r * 8 + ((4 * h + i) ^ (r & 7));
            w[i] = Ws[fidx[i]]; m1[i] = M1s[fidx[i]]; m2[i] = M2s[fidx[i]];
            if (MIX) ms[i] = MSs[fidx[i]];
          }
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const uint4& gq = graw[i >> 1];
            const uint32_t lo = (i & 1) ? gq.z : gq.x, hi = (i & 1) ? gq.w : gq.y;
            const __nv_bfloat162 g01 = *reinterpret_cast<const __nv_bfloat162*>(&lo);
            const __nv_bfloat162 g23 = *reinterpret_cast<const __nv_bfloat162*>(&hi);
            const float g4[4] = {__low2float(g01), __high2float(g01), __low2float(g23), __high2float(g23)};
            const float4 rr = make_float4(rv[4 * i], rv[4 * i + 1], rv[4 * i + 2], rv[4 * i + 3]);
            if (MIX) ademamix4(sc, clip, g4, rr, w[i], m1[i], m2[i], ms[i], gp[i]);
            else adamw4(sc, clip, g4, rr, w[i], m1[i], m2[i], gp[i]);
          }
          float gout[16];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            Ws[fidx[i]] = w[i]; M1s[fidx[i]] = m1[i]; M2s[fidx[i]] = m2[i];
            if (MIX) MSs[fidx[i]] = ms[i];
            gout[4 * i] = gp[i].x; gout[4 * i + 1] = gp[i].y; gout[4 * i + 2] = gp[i].z; gout[4 * i + 3] = gp[i].w;
          }
#pragma unroll
          for (int j = 0; j < 2; ++j) {
            const __nv_bfloat162 b0 = __floats2bfloat162_rn(w[2 * j].x, w[2 * j].y), b1 = __floats2bfloat162_rn(w[2 * j].z, w[2 * j].w);
            const __nv_bfloat162 b2 = __floats2bfloat162_rn(w[2 * j + 1].x, w[2 * j + 1].y), b3 = __floats2bfloat162_rn(w[2 * j + 1].z, w[2 * j + 1].w);
            Gs[gidx[j]] = make_uint4(*reinterpret_cast<const uint32_t*>(&b0), *reinterpret_cast<const uint32_t*>(&b1),
                                     *reinterpret_cast<const uint32_t*>(&b2), *reinterpret_cast<const uint32_t*>(&b3));
          }
          const int x = ct * kTileN + u * kUnitW;
          if (gp_dbg) {   // test hook: plain stores, one row per thread
            const int row = row0 + r, col = x + h * 16;
            if (row < g.m)
#pragma unroll
              for (int e = 0; e < 16; ++e)
                if (col + e < g.n) gp_dbg[(size_t)row * g.n + col + e] = gout[e];
          }
          fence_proxy_async();
          consumer_barrier();
          if (SW) {
            if (leader) mbar_arrive(&bars->store_ready[s]);       // the store warp sends the unit and frees the stage
          } else if (leader) {
            tma_store_2d(mp + MAP_W, st, x, row0);
            tma_store_2d(mp + MAP_M1, st + kUnitF32, x, row0);
            tma_store_2d(mp + MAP_M2, st + 2 * kUnitF32, x, row0);
            if (has_wb) tma_store_2d(mp + MAP_WB, st + 3 * kUnitF32, x, row0);
            tma_store_commit();
            // hand the previous unit's stage back once its stores have finished reading shared memory
            tma_store_wait_read<1>();
            if (unit_it > 0) mbar_arrive(&bars->empty[(unit_it - 1) % kStages]);
          }
        }
        if (dead) break;
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(&bars->acc_empty[ab]);
      }
    }
    if (dead && lane == 0) { atomicOr(status, kDevTimeout); *abort_flag = 1; }
    if (!SW && leader) tma_store_wait_all();
  } else if (SW && warp == StreamCfg<MIX, UT>::kStoreWarp) {
    // -------------------------------------------------------------------- store warp (dual-EMA and UT variants)
    if (lane == 0) {
      uint32_t unit_it = 0;
      int last_inst = -1;
      bool dead = false;
      for (uint32_t item_it = 0; !dead; ++item_it) {
        if (!mbar_wait(&bars->item_ready[item_it % kItemSlots], (item_it / kItemSlots) & 1, abort_flag)) { dead = true; break; }
        const int item = *reinterpret_cast<volatile int*>(&bars->item_slot[item_it % kItemSlots]);
        if (item < 0) break;
        int inst, rt, ct0, ct1;
        decode_item(g, item, inst, rt, ct0, ct1);
        const MatDev& md = tab[idx[inst]];
        const CUtensorMap* mp = maps + (size_t)md.inst * kMapsPerMat;
        if (inst != last_inst) {
          tensormap_acquire(mp + MAP_W); tensormap_acquire(mp + MAP_M1); tensormap_acquire(mp + MAP_M2);
          if (MIX) tensormap_acquire(mp + MAP_MS);
          tensormap_acquire(mp + MAP_WB);
          last_inst = inst;
        }
        const int row0 = rt * 128;
        const bool has_wb = md.Wb != nullptr;
        for (int ct = ct0; ct < ct1 && !dead; ++ct) {
          const int units = (g.n - ct * kTileN > kUnitW) ? 2 : 1;
          for (int u = 0; u < units; ++u, ++unit_it) {
            const int s = unit_it % kStages;
            if (!mbar_wait(&bars->store_ready[s], (unit_it / kStages) & 1, abort_flag)) { dead = true; break; }
            uint8_t* st = smem + (size_t)s * kStreamStageBytes;
            const int x = ct * kTileN + u * kUnitW;
            tma_store_2d(mp + MAP_W, st, x, row0);
            tma_store_2d(mp + MAP_M1, st + kUnitF32, x, row0);
            tma_store_2d(mp + MAP_M2, st + 2 * kUnitF32, x, row0);
            if (MIX) tma_store_2d(mp + MAP_MS, st + 3 * kUnitF32, x, row0);
            if (has_wb) tma_store_2d(mp + MAP_WB, st + kF32 * kUnitF32, x, row0);
            tma_store_commit();
            tma_store_wait_read<0>();          // the stage is free as soon as the stores have read it
            mbar_arrive(&bars->empty[s]);
          }
        }
      }
      if (dead) { atomicOr(status, kDevTimeout); *abort_flag = 1; }
      tma_store_wait_all();
    }
    __syncwarp();
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) tmem_dealloc(tmem_base, tmem_cols);
}

// A wait that nothing will ever satisfy, with a caller-chosen small poll limit: exercises the path by which a
// bounded wait reports through the status word (the block gives up, latches the bit and returns normally).
__global__ void wait_probe_kernel(int max_polls, unsigned* status) {
  __shared__ uint64_t bar;
  if (threadIdx.x == 0) {
    mbar_init(&bar, 1);
    fence_barrier_init();
    bool done = false;
    for (int it = 0; it < max_polls && !done; ++it) done = mbar_try_wait(&bar, 0);
    if (!done) atomicOr(status, kDevTimeout);
  }
}

// ---------------------------------------------------------------------------------------------- host
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
static EncodeTiledFn g_encode = nullptr;

bool tc_shape_supported(int64_t m, int64_t n, int rp) {
  return rp >= 16 && rp <= 256 && (n % 8) == 0 && m >= 1 && n >= 64;
}

size_t tc_tmaps_bytes(int count) { return (size_t)count * kMapsPerMat * sizeof(CUtensorMap); }

sc_status tc_init() {
  if (!g_encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess || !fn ||
        qres != cudaDriverEntryPointSuccess)
      return SC_ERR_CUDA;
    g_encode = reinterpret_cast<EncodeTiledFn>(fn);
  }
  // per device: the opt-in shared-memory sizes (cheap, so simply repeated for every plan)
  if (cudaFuncSetAttribute(project_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024) != cudaSuccess ||
      cudaFuncSetAttribute(project_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024) != cudaSuccess ||
      cudaFuncSetAttribute(fused_update_stream_kernel<false, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           StreamCfg<false>::kSmem + (int)sizeof(StreamBars) + 1024) != cudaSuccess ||
      cudaFuncSetAttribute(fused_update_stream_kernel<true, false>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           StreamCfg<true>::kSmem + (int)sizeof(StreamBars) + 1024) != cudaSuccess ||
      cudaFuncSetAttribute(fused_update_stream_kernel<false, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           StreamCfg<false, true>::kSmem + (int)sizeof(StreamBars) + 1024) != cudaSuccess ||
      cudaFuncSetAttribute(fused_update_stream_kernel<true, true>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                           StreamCfg<true, true>::kSmem + (int)sizeof(StreamBars) + 1024) != cudaSuccess ||
      cudaFuncSetAttribute(ema_pass_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024) != cudaSuccess ||
      cudaFuncSetAttribute(pass_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024) != cudaSuccess ||
      cudaFuncSetAttribute(pass_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 220 * 1024) != cudaSuccess)
    return SC_ERR_CUDA;
  return SC_OK;
}

// Row-major matrix [outer][inner] -> 2-D tiled map.
static bool encode2d(CUtensorMap* out, CUtensorMapDataType dt, int elem_bytes, const void* base, uint64_t inner,
                     uint64_t outer, uint64_t row_stride_elems, uint32_t box_inner, uint32_t box_rows,
                     CUtensorMapSwizzle swz) {
  cuuint64_t dims[2] = {inner, outer};
  cuuint64_t strides[1] = {row_stride_elems * (uint64_t)elem_bytes};
  cuuint32_t box[2] = {box_inner, box_rows};
  cuuint32_t estr[2] = {1, 1};
  return g_encode(out, dt, 2, const_cast<void*>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, swz,
                  CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
// bf16, 64-element (128-byte) rows, 128-byte swizzle: K-major MMA operand tiles.
static bool encode_bf16(CUtensorMap* out, const void* base, uint64_t inner, uint64_t outer, uint64_t row_stride_elems,
                        uint32_t box_rows) {
  return encode2d(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, base, inner, outer, row_stride_elems, 64, box_rows,
                  CU_TENSOR_MAP_SWIZZLE_128B);
}
// fp32 read as tf32, 32-element (128-byte) rows; MN-major operands need the 32-byte-atom flavour of the swizzle.
static bool encode_tf32(CUtensorMap* out, const void* base, uint64_t inner, uint64_t outer, uint32_t box_rows,
                        bool mn_major) {
  return encode2d(out, CU_TENSOR_MAP_DATA_TYPE_TFLOAT32, 4, base, inner, outer, inner, 32, box_rows,
                  mn_major ? CU_TENSOR_MAP_SWIZZLE_128B_ATOM_32B : CU_TENSOR_MAP_SWIZZLE_128B);
}

// (Re)encode the tensor maps of a class and copy them to the device. The source is pageable host memory,
// so the runtime has taken its copy of the bytes when cudaMemcpy2DAsync returns.
sc_status tc_encode_class(sc_plan* p, ShapeClass& c, bool static_part, bool per_call_part) {
  const int cnt = (int)c.mats.size();
  const int rp = p->rp, rk = p->rk, lp = p->lp;
  std::vector<CUtensorMap> maps((size_t)cnt * kMapsPerMat);
  CUtensorMap* dev = static_cast<CUtensorMap*>(c.tmaps);
  for (int i = 0; i < cnt; ++i) {
    const MatDev& md = p->host_tab[c.mats[i]];
    CUtensorMap* mp = &maps[(size_t)i * kMapsPerMat];
    bool ok = true;
    if (per_call_part) {
      const CUtensorMapDataType f32 = CU_TENSOR_MAP_DATA_TYPE_FLOAT32, b16 = CU_TENSOR_MAP_DATA_TYPE_BFLOAT16;
      ok = ok && encode_bf16(mp + MAP_G, md.G, c.n, c.m, c.n, 128);
      ok = ok && encode2d(mp + MAP_G32, b16, 2, md.G, c.n, c.m, c.n, 32, 128, CU_TENSOR_MAP_SWIZZLE_64B);
      ok = ok && encode2d(mp + MAP_W, f32, 4, md.W, c.n, c.m, c.n, 32, 128, CU_TENSOR_MAP_SWIZZLE_128B);
      ok = ok && encode2d(mp + MAP_M1, f32, 4, md.m1, c.n, c.m, c.n, 32, 128, CU_TENSOR_MAP_SWIZZLE_128B);
      ok = ok && encode2d(mp + MAP_M2, f32, 4, md.m2, c.n, c.m, c.n, 32, 128, CU_TENSOR_MAP_SWIZZLE_128B);
      ok = ok && encode2d(mp + MAP_WB, b16, 2, md.Wb ? (const void*)md.Wb : md.G, c.n, c.m, c.n, 32, 128,
                          CU_TENSOR_MAP_SWIZZLE_64B);
      ok = ok && encode2d(mp + MAP_MS, f32, 4, md.ms ? md.ms : md.m1, c.n, c.m, c.n, 32, 128, CU_TENSOR_MAP_SWIZZLE_128B);
      if (!ok) return SC_ERR_CUDA;
    }
    if (static_part) {
      ok = ok && encode_bf16(mp + MAP_VTHI, md.Vthi, c.n, rp, c.n, rp);
      ok = ok && encode_bf16(mp + MAP_VTLO, md.Vtlo, c.n, rp, c.n, rp);
      ok = ok && encode_bf16(mp + MAP_VTHI_H, md.Vthi, c.n, rp, c.n, rp / 2);
      ok = ok && encode_bf16(mp + MAP_VTLO_H, md.Vtlo, c.n, rp, c.n, rp / 2);
      ok = ok && encode_bf16(mp + MAP_UHI, md.Uhi, rk, c.m, rk, 128);
      ok = ok && encode_bf16(mp + MAP_ULO, md.Ulo, rk, c.m, rk, 128);
      ok = ok && encode_bf16(mp + MAP_CTHI, md.Cthi, rk, c.n, rk, 128);
      ok = ok && encode_bf16(mp + MAP_CTLO, md.Ctlo, rk, c.n, rk, 128);
      ok = ok && encode_bf16(mp + MAP_CT64HI, md.Cthi, rk, c.n, rk, kTileN);
      ok = ok && encode_bf16(mp + MAP_CT64LO, md.Ctlo, rk, c.n, rk, kTileN);
      ok = ok && encode_tf32(mp + MAP_M_K, md.Manc, c.n, c.m, 128, false);
      ok = ok && encode_tf32(mp + MAP_M_MN, md.Manc, c.n, c.m, kPassK, true);
      ok = ok && encode_tf32(mp + MAP_Y, md.Y, lp, c.m, kPassK, true);
      ok = ok && encode_tf32(mp + MAP_Z, md.Z, lp, c.n, kPassK, true);
      ok = ok && encode_tf32(mp + MAP_OMEGA, md.omega, lp, c.n, kPassK, true);
      ok = ok && encode2d(mp + MAP_M_F32, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, md.Manc, c.n, c.m, c.n, 32, 128,
                          CU_TENSOR_MAP_SWIZZLE_128B);
      ok = ok && encode_tf32(mp + MAP_U_MN, md.U, rp, c.m, kPassK, true);
      ok = ok && encode_tf32(mp + MAP_T, md.T, rp, c.m, kPassK, true);
      ok = ok && encode_tf32(mp + MAP_Y2, md.Y2, lp, c.m, kPassK, true);
      ok = ok && encode_tf32(mp + MAP_Z2, md.Z2, lp, c.n, kPassK, true);
      if (!ok) return SC_ERR_CUDA;
    }
  }
  const size_t pitch = kMapsPerMat * sizeof(CUtensorMap);
  if (per_call_part &&
      cudaMemcpy2DAsync(dev, pitch, maps.data(), pitch, kPerCallMaps * sizeof(CUtensorMap), cnt, cudaMemcpyHostToDevice,
                        p->stream) != cudaSuccess)
    return SC_ERR_CUDA;
  if (static_part &&
      cudaMemcpy2DAsync(dev + kPerCallMaps, pitch, maps.data() + kPerCallMaps, pitch,
                        (kMapsPerMat - kPerCallMaps) * sizeof(CUtensorMap), cnt, cudaMemcpyHostToDevice,
                        p->stream) != cudaSuccess)
    return SC_ERR_CUDA;
  return SC_OK;
}

// Two blocks per SM when three stages of each fit (their prologues and epilogues then overlap the other block's
// streaming); otherwise one block with as many stages as fit.
static int stages_for(int stage_bytes, int max_one_block) {
  if (2 * stage_bytes + 2048 <= 110 * 1024) {
    const int s = (110 * 1024 - 2048) / stage_bytes;
    return s > 4 ? 4 : s;
  }
  const int s = (200 * 1024) / stage_bytes;
  return s > max_one_block ? max_one_block : (s < 2 ? 2 : s);
}
static int project_stages(int rp) { return stages_for(kTileBytes + 2 * rp * 128, 6); }

sc_status tc_launch_project(sc_plan* p, ShapeClass& c, const int* idx, int count) {
  const int rp = p->rp, m = (int)c.m, n = (int)c.n;
  const int nchunks = (n + 63) / 64;
  const int cps = (nchunks + c.ksplit - 1) / c.ksplit;
  const int stages = project_stages(rp);
  const size_t smem = (size_t)stages * (kTileBytes + 2 * rp * 128) + 1024 + 256;
  uint32_t cols = 32;
  while ((int)cols < rp) cols <<= 1;
  if (m >= 256 && !p->no_pair_project) {
    // pairs of SMs on 256-row tiles, each block loading half of every V^T tile
    const int stage_b = kTileBytes + rp * 128;
    const int st2 = stages_for(stage_b, 6);
    const size_t smem2 = (size_t)st2 * stage_b + 1024 + 256;
    dim3 grid2(2 * ((m + 255) / 256), c.ksplit, count);
    project_pair_kernel<<<grid2, 192, smem2, p->stream>>>(p->dev_tab, idx, static_cast<const CUtensorMap*>(c.tmaps), m, n,
                                                          rp, cps, st2, cols, p->status_dev);
    ++g_kernel_launches;
    return cuda_ok(cudaGetLastError());
  }
  dim3 grid((m + 127) / 128, c.ksplit, count);
  project_kernel<<<grid, 192, smem, p->stream>>>(p->dev_tab, idx, static_cast<const CUtensorMap*>(c.tmaps), m, n, rp,
                                                 cps, stages, cols, p->status_dev);
  ++g_kernel_launches;
  return cuda_ok(cudaGetLastError());
}

sc_status tc_launch_wait_probe(sc_plan* p, int max_polls) {
  wait_probe_kernel<<<1, 32, 0, p->stream>>>(max_polls, p->status_dev);
  ++g_kernel_launches;
  return cuda_ok(cudaGetLastError());
}

// Tensor maps of the anchor gradients of one call (the matrices listed in ids), copied to the device.
sc_status tc_encode_anchor(sc_plan* p, ShapeClass& c, const std::vector<int>& ids) {
  CUtensorMap* dev = static_cast<CUtensorMap*>(c.tmaps);
  for (int id : ids) {
    const MatDev& md = p->host_tab[id];
    CUtensorMap tm;
    if (!encode2d(&tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, md.Ganc, c.n, c.m, c.n, 32, 128, CU_TENSOR_MAP_SWIZZLE_64B))
      return SC_ERR_CUDA;
    // pageable source: the runtime has taken its copy when this returns
    if (cudaMemcpyAsync(dev + (size_t)md.inst * kMapsPerMat + MAP_GANC32, &tm, sizeof(tm), cudaMemcpyHostToDevice,
                        p->stream) != cudaSuccess)
      return SC_ERR_CUDA;
  }
  return SC_OK;
}

// Eq. 1 fused with the first sweep: M <- beta M + (1 - beta) G_anc and Y <- M_new B in one pass over M.
sc_status tc_launch_ema_pass(sc_plan* p, ShapeClass& c, const int* idx, int count, int b_field_off) {
  const int lp = p->lp, m = (int)c.m, n = (int)c.n;
  const int stage_bytes = kTileBytes + kGancTile + (lp / 32) * kAtomBytes;
  const int stages = stages_for(stage_bytes, 6);
  const size_t smem = (size_t)stages * stage_bytes + 1024 + 512;
  uint32_t cols = 32;
  while ((int)cols < lp) cols <<= 1;
  int b_map;
  if (b_field_off == (int)offsetof(MatDev, omega_t) || b_field_off == (int)offsetof(MatDev, omega)) b_map = MAP_OMEGA;
  else if (b_field_off == (int)offsetof(MatDev, Z2)) b_map = MAP_Z2;
  else return SC_ERR_INVALID_ARG;
  dim3 grid((m + 127) / 128, 1, count);
  ema_pass_kernel<<<grid, 224, smem, p->stream>>>(p->dev_tab, idx, static_cast<const CUtensorMap*>(c.tmaps), b_map, m, n,
                                                  lp, stages, cols, p->hp.beta_anc, p->status_dev);
  ++g_kernel_launches;
  return cuda_ok(cudaGetLastError());
}

static uint32_t tmem_cols_for(int n) {
  uint32_t cols = 32;
  while ((int)cols < n) cols <<= 1;
  return cols;
}

static int panel_map(int field_off) {
  if (field_off == (int)offsetof(MatDev, omega_t) || field_off == (int)offsetof(MatDev, omega)) return MAP_OMEGA;
  if (field_off == (int)offsetof(MatDev, Y)) return MAP_Y;
  if (field_off == (int)offsetof(MatDev, Y2)) return MAP_Y2;
  if (field_off == (int)offsetof(MatDev, Z)) return MAP_Z;
  if (field_off == (int)offsetof(MatDev, Z2)) return MAP_Z2;
  return -1;
}

// One sweep over the anchor momentum: transposed ? Z <- M^T B : Y <- M B, with B one of the n x lp / m x lp buffers.
sc_status tc_launch_pass(sc_plan* p, ShapeClass& c, const int* idx, int count, bool transposed, int b_field_off) {
  const int lp = p->lp, m = (int)c.m, n = (int)c.n;
  PassArgs pa{};
  pa.a_map = transposed ? MAP_M_MN : MAP_M_K;
  pa.b_map = panel_map(b_field_off);
  if (pa.b_map < 0) return SC_ERR_INVALID_ARG;
  pa.out_off = transposed ? (int)offsetof(MatDev, Z) : (int)offsetof(MatDev, Y);
  pa.rows_out = transposed ? n : m;
  pa.kdim = transposed ? m : n;
  pa.ncols = lp; pa.ncols_valid = lp; pa.ldo = lp;
  // few output tiles (a plan with one or two matrices): split the contraction over K slices into spart, add them up
  const int slices = transposed ? c.sweep_split_t : c.sweep_split_n;
  const int nchunks = (pa.kdim + kPassK - 1) / kPassK;
  pa.cps = (nchunks + slices - 1) / slices;
  const int out_final = pa.out_off;
  if (slices > 1) pa.out_off = (int)offsetof(MatDev, spart);
  const int stage_bytes = kTileBytes + (lp / 32) * kAtomBytes;
  pa.stages = stages_for(stage_bytes, 8);
  pa.tmem_cols = tmem_cols_for(lp);
  const size_t smem = (size_t)pa.stages * stage_bytes + 1024 + 256;
  const CUtensorMap* maps = static_cast<const CUtensorMap*>(c.tmaps);
  dim3 grid((pa.rows_out + 127) / 128, slices, count);
  if (transposed) pass_kernel<true><<<grid, 192, smem, p->stream>>>(p->dev_tab, idx, maps, pa, p->status_dev);
  else pass_kernel<false><<<grid, 192, smem, p->stream>>>(p->dev_tab, idx, maps, pa, p->status_dev);
  ++g_kernel_launches;
  if (slices > 1)
    launch_sum_slices(p->dev_tab, idx, count, (int)offsetof(MatDev, spart), out_final, pa.rows_out * lp, slices, p->stream);
  return cuda_ok(cudaGetLastError());
}

// part[slice] = A^T B over the rows of K slice `slice`, for tall panels A (rows x ca) and B (rows x cb) given by
// their tensor maps; the caller adds the slices. a_map == b_map computes a Gram matrix from one load of the panel.
sc_status tc_launch_atb(sc_plan* p, ShapeClass& c, const int* idx, int count, int a_map, int b_map, int part_off,
                        int rows, int ca, int cb, int slices) {
  PassArgs pa{};
  pa.a_map = a_map; pa.b_map = b_map;
  pa.same_ab = a_map == b_map && ca <= 128 && cb <= 128;   // one 128-column tile holds the whole panel
  pa.out_off = part_off;
  pa.rows_out = ca;
  pa.kdim = rows;
  pa.ncols = (cb + 31) / 32 * 32; pa.ncols_valid = cb; pa.ldo = cb;
  const int nchunks = (rows + kPassK - 1) / kPassK;
  pa.cps = (nchunks + slices - 1) / slices;
  const int stage_bytes = kTileBytes + (pa.same_ab ? 0 : (pa.ncols / 32) * kAtomBytes);
  pa.stages = stages_for(stage_bytes, 8);
  pa.tmem_cols = tmem_cols_for(pa.ncols);
  const size_t smem = (size_t)pa.stages * stage_bytes + 1024 + 256;
  dim3 grid((ca + 127) / 128, slices, count);
  pass_kernel<true><<<grid, 192, smem, p->stream>>>(p->dev_tab, idx, static_cast<const CUtensorMap*>(c.tmaps), pa,
                                                     p->status_dev);
  ++g_kernel_launches;
  return cuda_ok(cudaGetLastError());
}

// Gram matrix partials of one of the Y / Y2 / Z / Z2 panels (lp columns) into gpart.
sc_status tc_launch_gram(sc_plan* p, ShapeClass& c, const int* idx, int count, int panel_field_off, int rows, int slices) {
  const int pm = panel_map(panel_field_off);
  if (pm < 0 || pm == MAP_OMEGA) return SC_ERR_INVALID_ARG;
  return tc_launch_atb(p, c, idx, count, pm, pm, (int)offsetof(MatDev, gpart), rows, p->lp, p->lp, slices);
}

// X partials: xpart[slice] = U^T T over the rows of the slice.
sc_status tc_launch_xpart(sc_plan* p, ShapeClass& c, const int* idx, int count, int slices) {
  return tc_launch_atb(p, c, idx, count, MAP_U_MN, MAP_T, (int)offsetof(MatDev, xpart), (int)c.m, p->rp, p->rp, slices);
}

sc_status tc_launch_epilogue(sc_plan* p, ShapeClass& c, const int* idx, int count, const StepScalars& sc) {
  const int m = (int)c.m, n = (int)c.n;
  const int n_sm = p->n_sm > 0 ? p->n_sm : 148;
  StreamGeom g;
  g.m = m; g.n = n; g.rp = p->rp;
  g.row_tiles = (m + 127) / 128;
  g.col_tiles = (n + kTileN - 1) / kTileN;
  // one 128 x 64 tile per item, neighbouring tiles next to each other in the item order: blocks that run side by side
  // then touch the same rows of DRAM, and the atomic hand-out has something to balance with. Measured on the 8B set,
  // update time per step for 1 / 2 / 4 / 8 tiles per item: 31.1 / 31.5 / 32.6 / 35.0 ms (the U panel that each item
  // reloads from L2 costs less than the locality lost with longer items).
  // Ranks above 64 keep the U panel of an item in tensor memory: an item is then a run of four tiles that share it.
  // Measured (update kernel against the HBM peak): the 70B-shaped set at rank 128 with runs of 1 (U re-fetched per tile)
  // / 2 / 3 / 4 / 8 tiles: 0.85 / 0.91 / 0.90 / 0.89 / 0.84; one 14336 x 4096 matrix at rank 256 with runs of 1 / 2 / 3:
  // 0.69 / 0.78 / 0.81. A single matrix at rank 128 is already at 0.93 with one tile per item (few items, all blocks on
  // one matrix) and loses with longer items, so it keeps that.
  const int ut_tiles = p->ut_tiles > 0 ? p->ut_tiles : (p->rp > 128 ? 3 : 2);
  const long long items_ut = (long long)count * g.row_tiles * ((g.col_tiles + ut_tiles - 1) / ut_tiles);
  const bool ut = p->rp > 64 && !p->no_tmem_u && (p->rp > 128 || items_ut >= 32ll * n_sm || p->ut_tiles > 0);
  g.tiles_per_chunk = ut ? ut_tiles : 1;
  g.csplit = (g.col_tiles + g.tiles_per_chunk - 1) / g.tiles_per_chunk;
  g.n_items = count * g.row_tiles * g.csplit;
  const int grid = g.n_items < n_sm ? g.n_items : n_sm;
  if (cudaMemsetAsync(p->work_dev, 0, sizeof(unsigned), p->stream) != cudaSuccess) return SC_ERR_CUDA;
  const CUtensorMap* maps = static_cast<const CUtensorMap*>(c.tmaps);
  const size_t smem_mix = StreamCfg<true>::kSmem + sizeof(StreamBars) + 1024;
  const size_t smem_adam = StreamCfg<false>::kSmem + sizeof(StreamBars) + 1024;
#define SC_LAUNCH_UPDATE(MIXV, UTV, SMEM)                                                                       \
  fused_update_stream_kernel<MIXV, UTV><<<grid, stream_threads<MIXV, UTV>(), SMEM, p->stream>>>(                \
      p->dev_tab, idx, maps, g, sc, p->clip_dev, p->status_dev, p->work_dev)
  const size_t smem_mix_ut = StreamCfg<true, true>::kSmem + sizeof(StreamBars) + 1024;
  const size_t smem_adam_ut = StreamCfg<false, true>::kSmem + sizeof(StreamBars) + 1024;
  if (sc.mix && ut) SC_LAUNCH_UPDATE(true, true, smem_mix_ut);
  else if (sc.mix) SC_LAUNCH_UPDATE(true, false, smem_mix);
  else if (ut) SC_LAUNCH_UPDATE(false, true, smem_adam_ut);
  else SC_LAUNCH_UPDATE(false, false, smem_adam);
#undef SC_LAUNCH_UPDATE
  ++g_kernel_launches;
  return cuda_ok(cudaGetLastError());
}

}  // namespace sc
