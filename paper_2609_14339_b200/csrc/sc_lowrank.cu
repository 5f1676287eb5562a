// Low-rank gradient compressor with error feedback (DP-compression appendix, "Low-rank factorization (F3)"): rank-1..8
// factors from one subspace-iteration step per gradient.
//
//     M = G + E            P = M Q_prev            P_hat = orth(P)            Q = M^T P_hat            E <- M - P_hat Q^T
//
// With rho <= 8 there are at most 16 flops per byte of the matrix, so every pass is bound by HBM and runs on the CUDA cores
// with 128-bit accesses: no tensor cores here. Three passes over the matrix:
//   phase A  reads G (and E), writes M into E, forms P                      lowrank_mq_kernel        (2 + 4 + 4 B/element)
//   phase B  orthonormalises P (Cholesky QR twice, one block), reads M, forms Q   lowrank_mtp_kernel  (4 B/element)
//   phase C  reads M, writes E = M - P_hat Q^T                               lowrank_residual_kernel  (4 + 4 B/element)
// All sums over rows or columns are two-stage in a fixed order (no float atomics), so results are reproducible.
#include "sc_internal.cuh"

namespace {

using sc::bf16;
constexpr int kMaxRho = 8;
constexpr int kRowsPerBlockA = 8;        // phase A: one warp per row
constexpr int kChunkA = 1024;            // columns of Q staged in shared memory at a time
constexpr int kColsPerBlock = 1024;      // phases B and C: 256 threads x 4 columns
constexpr int kSlabRows = 128;           // rows of P_hat staged in shared memory at a time (phases B and C)
constexpr int kMaxSlabs = 4096;

inline size_t align256(size_t x) { return (x + 255) / 256 * 256; }

struct Layout {          // carve-up of the caller's workspace
  size_t qpart, q_slabs, total;
};

int slabs_for(int64_t rows, int64_t cols) {
  const int64_t col_blocks = (cols + kColsPerBlock - 1) / kColsPerBlock;
  int64_t s = (4 * 148 + col_blocks - 1) / col_blocks;            // about four blocks per SM
  const int64_t most = (rows + 15) / 16;                           // at least 16 rows per slab
  if (s > most) s = most;
  if (s > kMaxSlabs) s = kMaxSlabs;
  return (int)(s < 1 ? 1 : s);
}

Layout layout_for(int64_t rows, int64_t cols, int rho) {
  Layout L{};
  size_t off = 0;
  L.q_slabs = (size_t)slabs_for(rows, cols);
  L.qpart = off;     off = align256(off + L.q_slabs * (size_t)cols * rho * sizeof(float));
  L.total = off;
  return L;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Four consecutive elements of the gradient as floats.
template <bool G_BF16>
__device__ __forceinline__ float4 load_g4(const void* G, size_t off) {
  if (G_BF16) {
    const uint2 raw = *reinterpret_cast<const uint2*>(static_cast<const bf16*>(G) + off);
    const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162*>(&raw.x);
    const __nv_bfloat162 b = *reinterpret_cast<const __nv_bfloat162*>(&raw.y);
    return make_float4(__low2float(a), __high2float(a), __low2float(b), __high2float(b));
  }
  return *reinterpret_cast<const float4*>(static_cast<const float*>(G) + off);
}

// Phase A. M[i, :] = G[i, :] + E[i, :] (written back into E), P[i, :] = M[i, :] Q_prev.
// A persistent grid (a multiple of the SM count, so there is no partly filled last wave); warp w of block b owns rows
// b * 8 + w, + 8 * gridDim.x, ... . The block walks over the columns in chunks of kChunkA: the chunk of Q_prev is staged
// once in shared memory, transposed (rho rows of kChunkA columns) so that a lane's four consecutive columns are one
// conflict-free 128-bit read per factor, then every warp runs that chunk of each of its rows and adds the chunk's
// contribution to P (the same lane of the same warp every time, chunks in order: deterministic).
template <int RHO, bool G_BF16>
__global__ void __launch_bounds__(32 * kRowsPerBlockA)
lowrank_mq_kernel(const void* __restrict__ G, float* __restrict__ E, const float* __restrict__ Qprev,
                  float* __restrict__ P, int rows, int cols) {
  __shared__ __align__(16) float Qs[RHO][kChunkA];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int row_first = blockIdx.x * kRowsPerBlockA + warp, row_step = gridDim.x * kRowsPerBlockA;
  for (int c0 = 0; c0 < cols; c0 += kChunkA) {
    const int cw = min(kChunkA, cols - c0);
    __syncthreads();
    for (int e = threadIdx.x; e < cw * RHO; e += blockDim.x) {      // Q_prev is cols x RHO row-major: coalesced reads
      const int j = e / RHO, k = e - j * RHO;
      Qs[k][j] = Qprev[(size_t)(c0 + j) * RHO + k];
    }
    __syncthreads();
    for (int row = row_first; row < rows; row += row_step) {
      float acc[RHO];
#pragma unroll
      for (int k = 0; k < RHO; ++k) acc[k] = 0.f;
      // Four column groups of 128 per trip, all loads first: the in-place write of M into E would otherwise pin every
      // load of the next group behind the store of the previous one (same array, the compiler cannot tell them apart).
      constexpr int kBatch = 4;
      for (int j0 = lane * 4; j0 < cw; j0 += 128 * kBatch) {
        float4 mv[kBatch];
#pragma unroll
        for (int b = 0; b < kBatch; ++b) {
          const int j = j0 + 128 * b;
          mv[b] = j < cw ? load_g4<G_BF16>(G, (size_t)row * cols + c0 + j) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        if (E) {
          float4 ev[kBatch];
#pragma unroll
          for (int b = 0; b < kBatch; ++b) {
            const int j = j0 + 128 * b;
            ev[b] = j < cw ? *reinterpret_cast<const float4*>(E + (size_t)row * cols + c0 + j) : make_float4(0.f, 0.f, 0.f, 0.f);
          }
#pragma unroll
          for (int b = 0; b < kBatch; ++b) {
            const int j = j0 + 128 * b;
            mv[b].x += ev[b].x; mv[b].y += ev[b].y; mv[b].z += ev[b].z; mv[b].w += ev[b].w;
            if (j < cw) *reinterpret_cast<float4*>(E + (size_t)row * cols + c0 + j) = mv[b];
          }
        }
#pragma unroll
        for (int b = 0; b < kBatch; ++b) {
          const int j = j0 + 128 * b;
          if (j >= cw) continue;
#pragma unroll
          for (int k = 0; k < RHO; ++k) {
            const float4 q = *reinterpret_cast<const float4*>(&Qs[k][j]);
            acc[k] = fmaf(mv[b].x, q.x, acc[k]); acc[k] = fmaf(mv[b].y, q.y, acc[k]);
            acc[k] = fmaf(mv[b].z, q.z, acc[k]); acc[k] = fmaf(mv[b].w, q.w, acc[k]);
          }
        }
      }
#pragma unroll
      for (int k = 0; k < RHO; ++k) {
        const float v = warp_sum(acc[k]);
        if (lane == 0) P[(size_t)row * RHO + k] = (c0 == 0 ? 0.f : P[(size_t)row * RHO + k]) + v;
      }
    }
  }
}

// P_hat = orth(P) in one block: Cholesky QR twice. Each round: Gram matrix of the rows x rho panel (per-thread partial
// sums over a fixed row assignment, then a fixed-order tree over the block), Cholesky factor Gram = R^T R and R^-1 by
// one thread, P <- P R^-1. A column whose pivot has cancelled to less than 1e-6 of its own squared norm (remainder
// below 1e-3 of the column's norm) lies in the span of the earlier columns to single precision: it is dropped (its
// column of R^-1 is zero). The panel is a few hundred KB at most and stays in L2 between the rounds.
constexpr int kOrthThreads = 1024;

template <int kMaxRho>      // instantiated per rho, so that every loop below has exactly rho trips
__global__ void __launch_bounds__(kOrthThreads) lowrank_orth_kernel(float* __restrict__ P, int rows, int rho) {
  __shared__ float part[kOrthThreads / 32][kMaxRho * kMaxRho];
  __shared__ float Gm[kMaxRho][kMaxRho], R[kMaxRho][kMaxRho], Ri[kMaxRho][kMaxRho];
  const int t = threadIdx.x, warp = t >> 5, lane = t & 31;
  for (int round = 0; round < 2; ++round) {
    float g[kMaxRho * kMaxRho];
#pragma unroll
    for (int e = 0; e < kMaxRho * kMaxRho; ++e) g[e] = 0.f;
    for (int i = t; i < rows; i += kOrthThreads) {
      float p[kMaxRho];
#pragma unroll
      for (int k = 0; k < kMaxRho; ++k) p[k] = k < rho ? P[(size_t)i * rho + k] : 0.f;
#pragma unroll
      for (int a = 0; a < kMaxRho; ++a)
#pragma unroll
        for (int b = a; b < kMaxRho; ++b) g[a * kMaxRho + b] = fmaf(p[a], p[b], g[a * kMaxRho + b]);
    }
#pragma unroll
    for (int a = 0; a < kMaxRho; ++a)
#pragma unroll
      for (int b = a; b < kMaxRho; ++b) {
        const float s = warp_sum(g[a * kMaxRho + b]);
        if (lane == 0) part[warp][a * kMaxRho + b] = s;
      }
    __syncthreads();
    if (t < kMaxRho * kMaxRho) {
      const int a = t / kMaxRho, b = t % kMaxRho;
      if (a <= b) {
        float s = 0.f;
        for (int w = 0; w < kOrthThreads / 32; ++w) s += part[w][t];
        Gm[a][b] = s; Gm[b][a] = s;
      }
    }
    __syncthreads();
    if (t == 0) {
      for (int j = 0; j < rho; ++j)
        for (int i = 0; i < rho; ++i) { R[j][i] = 0.f; Ri[j][i] = 0.f; }
      for (int j = 0; j < rho; ++j) {
        float s = Gm[j][j];
        for (int k = 0; k < j; ++k) s -= R[k][j] * R[k][j];
        const bool ok = Gm[j][j] > 0.f && s > 1e-6f * Gm[j][j];
        const float rjj = ok ? sqrtf(s) : 0.f, inv = ok ? 1.f / rjj : 0.f;
        R[j][j] = rjj;
        for (int i = j + 1; i < rho; ++i) {
          float v = Gm[j][i];
          for (int k = 0; k < j; ++k) v -= R[k][j] * R[k][i];
          R[j][i] = v * inv;
        }
        Ri[j][j] = inv;
      }
      // inverse of the upper-triangular factor, column by column (dropped columns stay zero)
      for (int c = 0; c < rho; ++c) {
        if (Ri[c][c] == 0.f) continue;
        for (int i = c - 1; i >= 0; --i) {
          float s = 0.f;
          for (int k = i + 1; k <= c; ++k) s += R[i][k] * Ri[k][c];
          Ri[i][c] = -s * Ri[i][i];
        }
      }
    }
    __syncthreads();
    for (int i = t; i < rows; i += kOrthThreads) {
      float p[kMaxRho];
#pragma unroll
      for (int k = 0; k < kMaxRho; ++k) p[k] = k < rho ? P[(size_t)i * rho + k] : 0.f;
#pragma unroll
      for (int c = 0; c < kMaxRho; ++c) {
        float s = 0.f;
#pragma unroll
        for (int k = 0; k < kMaxRho; ++k)
          if (k <= c && c < rho) s = fmaf(p[k], Ri[k][c], s);
        if (c < rho) P[(size_t)i * rho + c] = s;
      }
    }
    __syncthreads();     // the same thread re-reads its own rows next round; the barrier orders the shared arrays
  }
}

// Phase B. qpart[slab][j][:] = sum over the slab's rows i of M[i, j] P_hat[i, :]. A thread owns four consecutive columns.
template <int RHO, bool M_BF16>
__global__ void __launch_bounds__(256)
lowrank_mtp_kernel(const void* __restrict__ M, const float* __restrict__ Phat, float* __restrict__ qpart, int rows,
                   int cols, int rows_per_slab) {
  __shared__ float Ps[kSlabRows][RHO];
  const int j = blockIdx.x * kColsPerBlock + threadIdx.x * 4;
  const bool live = j < cols;
  const int r_lo = blockIdx.y * rows_per_slab, r_hi = min(rows, r_lo + rows_per_slab);
  float acc[4][RHO];
#pragma unroll
  for (int e = 0; e < 4; ++e)
#pragma unroll
    for (int k = 0; k < RHO; ++k) acc[e][k] = 0.f;
  for (int r0 = r_lo; r0 < r_hi; r0 += kSlabRows) {
    const int nr = min(kSlabRows, r_hi - r0);
    __syncthreads();
    for (int e = threadIdx.x; e < nr * RHO; e += blockDim.x) Ps[e / RHO][e % RHO] = Phat[(size_t)r0 * RHO + e];
    __syncthreads();
    if (!live) continue;
#pragma unroll 4
    for (int i = 0; i < nr; ++i) {
      const float4 mv = load_g4<M_BF16>(M, (size_t)(r0 + i) * cols + j);
#pragma unroll
      for (int k = 0; k < RHO; ++k) {
        const float p = Ps[i][k];
        acc[0][k] = fmaf(mv.x, p, acc[0][k]); acc[1][k] = fmaf(mv.y, p, acc[1][k]);
        acc[2][k] = fmaf(mv.z, p, acc[2][k]); acc[3][k] = fmaf(mv.w, p, acc[3][k]);
      }
    }
  }
  if (live) {
    float* out = qpart + ((size_t)blockIdx.y * cols + j) * RHO;
#pragma unroll
    for (int e = 0; e < 4; ++e)
#pragma unroll
      for (int k = 0; k < RHO; ++k) out[e * RHO + k] = acc[e][k];
  }
}

__global__ void __launch_bounds__(256) lowrank_qsum_kernel(const float* __restrict__ qpart, float* __restrict__ Q,
                                                           int64_t numel, int slabs) {
  const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= numel) return;
  float s = 0.f;
  for (int k = 0; k < slabs; ++k) s += qpart[(size_t)k * numel + e];
  Q[e] = s;
}

// Phase C. E[i, j] = M[i, j] - sum_k P_hat[i, k] Q[j, k], in place on the buffer that holds M.
template <int RHO>
__global__ void __launch_bounds__(256)
lowrank_residual_kernel(float* __restrict__ E, const float* __restrict__ Phat, const float* __restrict__ Q, int rows,
                        int cols, int rows_per_slab) {
  __shared__ float Ps[kSlabRows][RHO];
  const int j = blockIdx.x * kColsPerBlock + threadIdx.x * 4;
  const bool live = j < cols;
  const int r_lo = blockIdx.y * rows_per_slab, r_hi = min(rows, r_lo + rows_per_slab);
  float q[4][RHO];
#pragma unroll
  for (int e = 0; e < 4; ++e)
#pragma unroll
    for (int k = 0; k < RHO; ++k) q[e][k] = live ? Q[(size_t)(j + e) * RHO + k] : 0.f;
  for (int r0 = r_lo; r0 < r_hi; r0 += kSlabRows) {
    const int nr = min(kSlabRows, r_hi - r0);
    __syncthreads();
    for (int e = threadIdx.x; e < nr * RHO; e += blockDim.x) Ps[e / RHO][e % RHO] = Phat[(size_t)r0 * RHO + e];
    __syncthreads();
    if (!live) continue;
    // four rows per trip, loads first (the in-place stores would otherwise hold the next row's load back)
    for (int i0 = 0; i0 < nr; i0 += 4) {
      float4 mv[4];
#pragma unroll
      for (int b = 0; b < 4; ++b)
        mv[b] = i0 + b < nr ? *reinterpret_cast<const float4*>(E + (size_t)(r0 + i0 + b) * cols + j) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
      for (int b = 0; b < 4; ++b) {
        if (i0 + b >= nr) continue;
        float lo[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
        for (int k = 0; k < RHO; ++k) {
          const float p = Ps[i0 + b][k];
          lo[0] = fmaf(p, q[0][k], lo[0]); lo[1] = fmaf(p, q[1][k], lo[1]);
          lo[2] = fmaf(p, q[2][k], lo[2]); lo[3] = fmaf(p, q[3][k], lo[3]);
        }
        mv[b].x -= lo[0]; mv[b].y -= lo[1]; mv[b].z -= lo[2]; mv[b].w -= lo[3];
        *reinterpret_cast<float4*>(E + (size_t)(r0 + i0 + b) * cols + j) = mv[b];
      }
    }
  }
}

template <int RHO>
void launch_phase_a(const void* G, bool g_bf16, float* E, const float* Q, float* P, int rows, int cols, cudaStream_t s) {
  // Measured on 14336 x 4096: one row per warp at a time beats four (0.18 ms against 0.25 ms).
  const int want = (rows + kRowsPerBlockA - 1) / kRowsPerBlockA;
  const int blocks = want < 148 * 8 ? want : 148 * 8;          // eight blocks of 256 threads are resident per SM
  if (g_bf16) lowrank_mq_kernel<RHO, true><<<blocks, 32 * kRowsPerBlockA, 0, s>>>(G, E, Q, P, rows, cols);
  else lowrank_mq_kernel<RHO, false><<<blocks, 32 * kRowsPerBlockA, 0, s>>>(G, E, Q, P, rows, cols);
}
template <int RHO>
void launch_mtp(const void* M, bool m_bf16, const float* P, float* qpart, int rows, int cols, int slabs, int rps,
                cudaStream_t s) {
  dim3 grid((cols + kColsPerBlock - 1) / kColsPerBlock, slabs);
  if (m_bf16) lowrank_mtp_kernel<RHO, true><<<grid, 256, 0, s>>>(M, P, qpart, rows, cols, rps);
  else lowrank_mtp_kernel<RHO, false><<<grid, 256, 0, s>>>(M, P, qpart, rows, cols, rps);
}
template <int RHO>
void launch_residual(float* E, const float* P, const float* Q, int rows, int cols, int slabs, int rps, cudaStream_t s) {
  dim3 grid((cols + kColsPerBlock - 1) / kColsPerBlock, slabs);
  lowrank_residual_kernel<RHO><<<grid, 256, 0, s>>>(E, P, Q, rows, cols, rps);
}

#define DISPATCH_RHO(rho, CALL)                                        \
  switch (rho) {                                                       \
    case 1: { constexpr int R = 1; CALL; break; }                      \
    case 2: { constexpr int R = 2; CALL; break; }                      \
    case 3: { constexpr int R = 3; CALL; break; }                      \
    case 4: { constexpr int R = 4; CALL; break; }                      \
    case 5: { constexpr int R = 5; CALL; break; }                      \
    case 6: { constexpr int R = 6; CALL; break; }                      \
    case 7: { constexpr int R = 7; CALL; break; }                      \
    default: { constexpr int R = 8; CALL; break; }                     \
  }

}  // namespace

extern "C" size_t sc_lowrank_workspace_bytes(int64_t rows, int64_t cols, int rho) {
  if (rows <= 0 || cols <= 0 || rho < 1 || rho > kMaxRho || rows > (1 << 24) || cols > (1 << 24)) return 0;
  return layout_for(rows, cols, rho).total;
}

extern "C" sc_status sc_lowrank_compress(const void* G_dev, int grad_dtype, void* E_dev, void* P_dev, void* Q_dev,
                                         int64_t rows, int64_t cols, int rho, int phases, void* workspace,
                                         size_t workspace_bytes, void* stream) {
  if (!G_dev || !P_dev || !Q_dev || !workspace) return SC_ERR_INVALID_ARG;
  if (grad_dtype != SC_DTYPE_BF16 && grad_dtype != SC_DTYPE_FP32) return SC_ERR_DTYPE;
  if (rho < 1 || rho > kMaxRho || phases < 1 || phases > 7) return SC_ERR_INVALID_ARG;
  if (rows <= 0 || cols <= 0 || (cols % 4) != 0 || rho > rows || rho > cols) return SC_ERR_SHAPE;
  if (rows > (1 << 24) || cols > (1 << 24)) return SC_ERR_TOO_LARGE;
  const uintptr_t bits = reinterpret_cast<uintptr_t>(G_dev) | reinterpret_cast<uintptr_t>(E_dev) |
                         reinterpret_cast<uintptr_t>(P_dev) | reinterpret_cast<uintptr_t>(Q_dev);
  if ((bits & 15u) || (reinterpret_cast<uintptr_t>(workspace) & 255u)) return SC_ERR_ALIGNMENT;
  const Layout L = layout_for(rows, cols, rho);
  if (workspace_bytes < L.total) return SC_ERR_WORKSPACE;
  char* ws = static_cast<char*>(workspace);
  float* qpart = reinterpret_cast<float*>(ws + L.qpart);
  float* E = static_cast<float*>(E_dev);
  float* P = static_cast<float*>(P_dev);
  float* Q = static_cast<float*>(Q_dev);
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const bool g_bf16 = grad_dtype == SC_DTYPE_BF16;
  const int m = (int)rows, n = (int)cols;
  const int slabs = (int)L.q_slabs;
  const int rps = ((m + slabs - 1) / slabs + 15) / 16 * 16;
  long long launches = 0;

  if (phases & 1) {        // A: M = G + E (kept in E), P = M Q_prev
    DISPATCH_RHO(rho, launch_phase_a<R>(G_dev, g_bf16, E, Q, P, m, n, s));
    ++launches;
  }
  if (phases & 2) {        // B: P_hat = orth(P) by Cholesky QR, twice; Q = M^T P_hat
    DISPATCH_RHO(rho, (lowrank_orth_kernel<R><<<1, kOrthThreads, 0, s>>>(P, m, rho)));
    ++launches;
    const void* Msrc = E ? static_cast<const void*>(E) : G_dev;
    const bool m_bf16 = E ? false : g_bf16;
    DISPATCH_RHO(rho, launch_mtp<R>(Msrc, m_bf16, P, qpart, m, n, slabs, rps, s));
    const int64_t numel = (int64_t)n * rho;
    lowrank_qsum_kernel<<<(unsigned)((numel + 255) / 256), 256, 0, s>>>(qpart, Q, numel, slabs);
    launches += 2;
  }
  if ((phases & 4) && E) {  // C: E = M - P_hat Q^T
    DISPATCH_RHO(rho, launch_residual<R>(E, P, Q, m, n, slabs, rps, s));
    ++launches;
  }
  sc::g_kernel_launches += launches;
  return cudaGetLastError() == cudaSuccess ? SC_OK : SC_ERR_CUDA;
}

extern "C" sc_status sc_lowrank_init_q(void* Q_dev, int64_t cols, int rho, uint64_t seed, void* stream) {
  if (!Q_dev || cols <= 0 || rho < 1 || rho > kMaxRho) return SC_ERR_INVALID_ARG;
  sc::launch_sketch_rowmajor(static_cast<float*>(Q_dev), cols, rho, seed, static_cast<cudaStream_t>(stream));
  return cudaGetLastError() == cudaSuccess ? SC_OK : SC_ERR_CUDA;
}
