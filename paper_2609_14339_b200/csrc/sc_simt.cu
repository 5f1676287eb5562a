// CUDA-core (fp32) kernels of the spectral-correction step.
//
// These serve (a) every small, latency-bound piece of the method (Cholesky and Jacobi factorisations of
// l x l matrices, the r x r filter, norms) for all plans and (b) the large contractions too when the plan
// runs on the fp32 engine (fp32 gradients, shapes the tensor-core kernels do not take).
// Kernels are launched once per shape class; blockIdx.z selects the matrix through idx[] and the table.
#include <cooperative_groups.h>

#include <algorithm>

#include "sc_internal.cuh"

namespace sc {

template <typename T>
__device__ __forceinline__ T* field(const MatDev& md, int off) {
  return *reinterpret_cast<T* const*>(reinterpret_cast<const char*>(&md) + off);
}

__device__ __forceinline__ void split2(float x, bf16& hi, bf16& lo) {
  hi = __float2bfloat16_rn(x);
  lo = __float2bfloat16_rn(x - __bfloat162float(hi));
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// =====================================================================================================
// Batched tiled GEMM  C = alpha * op(A) * op(B), fp32 accumulate, with an optional fused AdamW epilogue.
// =====================================================================================================
constexpr int BM = 128, BN = 64, BK = 16;   // block tile; each of the 256 threads owns 8 rows x 4 columns

struct EpiStore {};
struct EpiAdamW {
  StepScalars sc;
  const float* clip;
  int g_bf16;
};

template <bool kAdamW>
__global__ void __launch_bounds__(256) gemm_kernel(GemmArgs a, EpiAdamW epi) {
  __shared__ __align__(16) float As[BK][BM + 4];
  __shared__ __align__(16) float Bs[BK][BN + 4];
  const MatDev& md = a.tab[a.idx[blockIdx.z]];
  const float* A = field<const float>(md, a.offA);
  const bf16* Ab = reinterpret_cast<const bf16*>(A);
  const float* B = field<const float>(md, a.offB);
  const int row0 = blockIdx.y * BM, col0 = blockIdx.x * BN;
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  float acc[8][4] = {};
  for (int k0 = 0; k0 < a.K; k0 += BK) {
    for (int e = tid; e < BM * BK; e += 256) {
      int r, k;
      if (!a.transA) { r = e / BK; k = e % BK; } else { k = e / BM; r = e % BM; }
      const int gr = row0 + r, gk = k0 + k;
      float v = 0.f;
      if (gr < a.M && gk < a.K) {
        const size_t off = a.transA ? (size_t)gk * a.lda + gr : (size_t)gr * a.lda + gk;
        v = a.a_bf16 ? __bfloat162float(Ab[off]) : A[off];
      }
      As[k][r] = v;
    }
    for (int e = tid; e < BN * BK; e += 256) {
      int c, k;
      if (!a.transB) { k = e / BN; c = e % BN; } else { c = e / BK; k = e % BK; }
      const int gc = col0 + c, gk = k0 + k;
      float v = 0.f;
      if (gc < a.N && gk < a.K) v = a.transB ? B[(size_t)gc * a.ldb + gk] : B[(size_t)gk * a.ldb + gc];
      Bs[k][c] = v;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < BK; ++k) {
      const float4 a0 = *reinterpret_cast<const float4*>(&As[k][ty * 8]);
      const float4 a1 = *reinterpret_cast<const float4*>(&As[k][ty * 8 + 4]);
      const float4 b0 = *reinterpret_cast<const float4*>(&Bs[k][tx * 4]);
      const float av[8] = {a0.x, a0.y, a0.z, a0.w, a1.x, a1.y, a1.z, a1.w};
      const float bv[4] = {b0.x, b0.y, b0.z, b0.w};
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    __syncthreads();
  }
  if (!kAdamW) {
    float* C = field<float>(md, a.offC);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int gr = row0 + ty * 8 + i;
      if (gr >= a.M) continue;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int gc = col0 + tx * 4 + j;
        if (gc < a.N) {
          float val = a.alpha * acc[i][j];
          if (a.beta_c != 0.f) val = fmaf(a.beta_c, C[(size_t)gr * a.ldc + gc], val);
          C[(size_t)gr * a.ldc + gc] = val;
          if (a.offHi) {   // also the bf16 hi/lo pair the tensor-core kernels read
            bf16 hi, lo;
            split2(val, hi, lo);
            field<bf16>(md, a.offHi)[(size_t)gr * a.ld_split + gc] = hi;
            field<bf16>(md, a.offLo)[(size_t)gr * a.ld_split + gc] = lo;
          }
        }
      }
    }
  } else {
    // acc = (U C)[i][j], the low-rank part (already carrying (1-alpha)*scale); blend, clip, AdamW.
    const float clip = *epi.clip;
    const StepScalars& s = epi.sc;
    const float* Gf = reinterpret_cast<const float*>(md.G);
    const bf16* Gb = reinterpret_cast<const bf16*>(md.G);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      const int gr = row0 + ty * 8 + i;
      if (gr >= a.M) continue;
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const int gc = col0 + tx * 4 + j;
        if (gc >= a.N) continue;
        const size_t o = (size_t)gr * a.N + gc;
        const float graw = epi.g_bf16 ? __bfloat162float(Gb[o]) : Gf[o];
        const float g = clip * fmaf(s.alpha_s, graw, acc[i][j]);
        const float mo = fmaf(s.beta1, md.m1[o], s.one_m_beta1 * g);
        const float vo = fmaf(s.beta2, md.m2[o], s.one_m_beta2 * g * g);
        const float den = fmaf(sqrtf(vo), s.inv_sqrt_bc2, s.eps);
        float w;
        if (s.mix) {     // dual EMA: the slow average of G_proj joins the numerator, not bias-corrected
          const float mslow = fmaf(s.beta3, md.ms[o], s.one_m_beta3 * g);
          md.ms[o] = mslow;
          w = md.W[o] * s.decay - fmaf(s.lr_mix, mslow, s.step_size * mo) / den;
        } else {
          w = fmaf(-s.step_size, mo / den, md.W[o] * s.decay);
        }
        md.m1[o] = mo;
        md.m2[o] = vo;
        md.W[o] = w;
        if (md.Wb) md.Wb[o] = __float2bfloat16_rn(w);
        if (md.gproj_dbg) md.gproj_dbg[o] = g;
      }
    }
  }
}

// =====================================================================================================
// Tall-skinny product  C = alpha * A * op(B) [+ beta_c * C]  for row-major fp32 A (M x K, K a few dozen to a
// few hundred): the shape of Y R^-1, U = Q Ub, V = Qb Wb and C^T = V Xs^T. A is streamed once through a
// two-deep ring of 128 x 32 chunks filled by cp.async (16 bytes per copy when base, row stride and K allow
// it, 4 bytes otherwise); B is small, comes from L2 and is prefetched into registers one chunk ahead.
// Thread (ty, tx) owns rows ty + 16 i (i < 8) and columns 4 tx .. 4 tx + 3; the sum over k runs in
// increasing k with one fmaf per term, exactly like gemm_kernel, so both give the same bits.
// =====================================================================================================
constexpr int TS_BM = 128, TS_BN = 64, TS_KC = 32;
constexpr int TS_AP = TS_KC + 4;   // row pitch of the A chunk (floats): 16-byte rows, no bank conflicts on float4 reads
constexpr int TS_BP = TS_BN + 4;
constexpr int TS_SMEM = (2 * TS_BM * TS_AP + 2 * TS_KC * TS_BP) * (int)sizeof(float);

__device__ __forceinline__ void cp_async16(float* dst, const float* src, bool valid) {
  const uint32_t d = (uint32_t)__cvta_generic_to_shared(dst);
  const int bytes = valid ? 16 : 0;   // 0 source bytes: the 16 destination bytes are zero-filled
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(d), "l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ void cp_async4(float* dst, const float* src, bool valid) {
  const uint32_t d = (uint32_t)__cvta_generic_to_shared(dst);
  const int bytes = valid ? 4 : 0;
  asm volatile("cp.async.ca.shared.global [%0], [%1], 4, %2;" ::"r"(d), "l"(src), "r"(bytes) : "memory");
}

__global__ void __launch_bounds__(256, 2) tsgemm_kernel(GemmArgs a) {
  extern __shared__ __align__(16) float ts_smem[];
  float(*As)[TS_BM][TS_AP] = reinterpret_cast<float(*)[TS_BM][TS_AP]>(ts_smem);
  float(*Bs)[TS_KC][TS_BP] = reinterpret_cast<float(*)[TS_KC][TS_BP]>(ts_smem + 2 * TS_BM * TS_AP);
  const MatDev& md = a.tab[a.idx[blockIdx.z]];
  const float* __restrict__ A = field<const float>(md, a.offA);
  const float* __restrict__ B = field<const float>(md, a.offB);
  const int row0 = blockIdx.y * TS_BM, col0 = blockIdx.x * TS_BN;
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  const bool vec = ((reinterpret_cast<uintptr_t>(A) & 15) == 0) && (a.lda % 4 == 0) && (a.K % 4 == 0);
  const int nchunks = (a.K + TS_KC - 1) / TS_KC;

  auto issue_a = [&](int stage, int k0) {
    if (vec) {
#pragma unroll
      for (int j = 0; j < (TS_BM * TS_KC / 4) / 256; ++j) {
        const int e = tid + 256 * j, r = e >> 3, q = e & 7;
        const int gr = row0 + r, gk = k0 + 4 * q;
        const bool ok = gr < a.M && gk < a.K;
        cp_async16(&As[stage][r][4 * q], ok ? A + (size_t)gr * a.lda + gk : A, ok);
      }
    } else {
      for (int e = tid; e < TS_BM * TS_KC; e += 256) {
        const int r = e / TS_KC, k = e % TS_KC;
        const int gr = row0 + r, gk = k0 + k;
        const bool ok = gr < a.M && gk < a.K;
        cp_async4(&As[stage][r][k], ok ? A + (size_t)gr * a.lda + gk : A, ok);
      }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  float breg[TS_KC * TS_BN / 256];
  auto load_b = [&](int k0) {
#pragma unroll
    for (int j = 0; j < TS_KC * TS_BN / 256; ++j) {
      const int e = tid + 256 * j;
      int k, c;
      if (!a.transB) { k = e / TS_BN; c = e % TS_BN; } else { c = e / TS_KC; k = e % TS_KC; }
      const int gk = k0 + k, gc = col0 + c;
      float v = 0.f;
      if (gk < a.K && gc < a.N) v = a.transB ? B[(size_t)gc * a.ldb + gk] : B[(size_t)gk * a.ldb + gc];
      breg[j] = v;
    }
  };
  auto store_b = [&](int stage) {
#pragma unroll
    for (int j = 0; j < TS_KC * TS_BN / 256; ++j) {
      const int e = tid + 256 * j;
      int k, c;
      if (!a.transB) { k = e / TS_BN; c = e % TS_BN; } else { c = e / TS_KC; k = e % TS_KC; }
      Bs[stage][k][c] = breg[j];
    }
  };

  float acc[8][4] = {};
  issue_a(0, 0);
  load_b(0);
  store_b(0);
  for (int c = 0; c < nchunks; ++c) {
    const int st = c & 1;
    const bool more = c + 1 < nchunks;
    if (more) {
      issue_a(st ^ 1, (c + 1) * TS_KC);
      load_b((c + 1) * TS_KC);
      asm volatile("cp.async.wait_group 1;" ::: "memory");
    } else {
      asm volatile("cp.async.wait_group 0;" ::: "memory");
    }
    __syncthreads();
#pragma unroll
    for (int kq = 0; kq < TS_KC / 4; ++kq) {
      float4 av[8];
#pragma unroll
      for (int i = 0; i < 8; ++i) av[i] = *reinterpret_cast<const float4*>(&As[st][i * 16 + ty][4 * kq]);
#pragma unroll
      for (int kk = 0; kk < 4; ++kk) {
        const float4 b = *reinterpret_cast<const float4*>(&Bs[st][4 * kq + kk][tx * 4]);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          const float x = kk == 0 ? av[i].x : kk == 1 ? av[i].y : kk == 2 ? av[i].z : av[i].w;
          acc[i][0] = fmaf(x, b.x, acc[i][0]);
          acc[i][1] = fmaf(x, b.y, acc[i][1]);
          acc[i][2] = fmaf(x, b.z, acc[i][2]);
          acc[i][3] = fmaf(x, b.w, acc[i][3]);
        }
      }
    }
    __syncthreads();
    if (more) store_b(st ^ 1);
  }

  float* C = field<float>(md, a.offC);
  bf16* Chi = a.offHi ? field<bf16>(md, a.offHi) : nullptr;
  bf16* Clo = a.offHi ? field<bf16>(md, a.offLo) : nullptr;
  const int gc0 = col0 + tx * 4;
  const bool vec_c = ((reinterpret_cast<uintptr_t>(C) & 15) == 0) && (a.ldc % 4 == 0) && gc0 + 3 < a.N;
  const bool vec_split = Chi && ((reinterpret_cast<uintptr_t>(Chi) & 7) == 0) && ((reinterpret_cast<uintptr_t>(Clo) & 7) == 0) &&
                         (a.ld_split % 4 == 0);
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int gr = row0 + i * 16 + ty;
    if (gr >= a.M) continue;
    float val[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) val[j] = a.alpha * acc[i][j];
    float* crow = C + (size_t)gr * a.ldc;
    if (Chi && a.split_only) {
      // nobody reads the fp32 result (the tensor-core update takes the bf16 pair)
    } else if (vec_c) {
      if (a.beta_c != 0.f) {
        const float4 o = *reinterpret_cast<const float4*>(crow + gc0);
        val[0] = fmaf(a.beta_c, o.x, val[0]); val[1] = fmaf(a.beta_c, o.y, val[1]);
        val[2] = fmaf(a.beta_c, o.z, val[2]); val[3] = fmaf(a.beta_c, o.w, val[3]);
      }
      *reinterpret_cast<float4*>(crow + gc0) = make_float4(val[0], val[1], val[2], val[3]);
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        if (gc0 + j >= a.N) continue;
        if (a.beta_c != 0.f) val[j] = fmaf(a.beta_c, crow[gc0 + j], val[j]);
        crow[gc0 + j] = val[j];
      }
    }
    if (Chi) {
      bf16 hi[4], lo[4];
#pragma unroll
      for (int j = 0; j < 4; ++j) split2(val[j], hi[j], lo[j]);
      const size_t o = (size_t)gr * a.ld_split + gc0;
      if (vec_split && gc0 + 3 < a.N) {            // four columns as one 8-byte store each
        uint2 ph, pl;
        ph.x = (uint32_t)__bfloat16_as_ushort(hi[0]) | ((uint32_t)__bfloat16_as_ushort(hi[1]) << 16);
        ph.y = (uint32_t)__bfloat16_as_ushort(hi[2]) | ((uint32_t)__bfloat16_as_ushort(hi[3]) << 16);
        pl.x = (uint32_t)__bfloat16_as_ushort(lo[0]) | ((uint32_t)__bfloat16_as_ushort(lo[1]) << 16);
        pl.y = (uint32_t)__bfloat16_as_ushort(lo[2]) | ((uint32_t)__bfloat16_as_ushort(lo[3]) << 16);
        *reinterpret_cast<uint2*>(Chi + o) = ph;
        *reinterpret_cast<uint2*>(Clo + o) = pl;
      } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) {
          if (gc0 + j >= a.N) continue;
          Chi[o + j] = hi[j];
          Clo[o + j] = lo[j];
        }
      }
    }
  }
}

void launch_gemm(const GemmArgs& a, int count, cudaStream_t s) {
  if (count <= 0 || a.M <= 0 || a.N <= 0) return;
  if (!a.transA && !a.a_bf16) {
    static const cudaError_t attr = cudaFuncSetAttribute(tsgemm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, TS_SMEM);
    (void)attr;
    dim3 grid((a.N + TS_BN - 1) / TS_BN, (a.M + TS_BM - 1) / TS_BM, count);
    tsgemm_kernel<<<grid, 256, TS_SMEM, s>>>(a);
  } else {
    dim3 grid((a.N + BN - 1) / BN, (a.M + BM - 1) / BM, count);
    gemm_kernel<false><<<grid, 256, 0, s>>>(a, EpiAdamW{});
  }
  ++g_kernel_launches;
}

void launch_epilogue_simt(const MatDev* tab, const int* idx, int count, int m, int n, int rp, int g_bf16,
                          const StepScalars& sc, const float* clip, cudaStream_t s) {
  if (count <= 0) return;
  GemmArgs a{};
  a.tab = tab; a.idx = idx;
  a.offA = offsetof(MatDev, U); a.offB = offsetof(MatDev, Ct); a.offC = 0;
  a.M = m; a.N = n; a.K = rp;
  a.lda = rp; a.ldb = rp; a.ldc = n;
  a.transA = 0; a.transB = 1; a.a_bf16 = 0; a.alpha = 1.f;
  EpiAdamW e{sc, clip, g_bf16};
  dim3 grid((n + BN - 1) / BN, (m + BM - 1) / BM, count);
  gemm_kernel<true><<<grid, 256, 0, s>>>(a, e);
  ++g_kernel_launches;
}

// =====================================================================================================
// Tall-skinny Gram-type product  C = A^T B  (A: rows x ca, B: rows x cb, both row-major) split over the
// rows: block s of the grid reduces its slice of rows into part[s] (ca x cb), a second kernel adds the
// slices in a fixed order. Used for X = U^T T and for the Gram matrices of the Cholesky QR.
// =====================================================================================================
template <int MT>
__global__ void __launch_bounds__(256) atb_kernel(const MatDev* tab, const int* idx, int offA, int offB, int offPart,
                                                  int rows, int ca, int cb, int lda, int ldb, int rows_per_split,
                                                  int b_slices) {
  constexpr int TS = 16 * MT;          // output tile edge
  __shared__ __align__(16) float As[32][TS + 4];
  __shared__ __align__(16) float Bs[32][TS + 4];
  const MatDev& md = tab[idx[blockIdx.z]];
  const float* A = field<const float>(md, offA);
  const float* B = field<const float>(md, offB);
  float* part = field<float>(md, offPart) + (size_t)blockIdx.x * ca * cb;
  const int tiles_b = (cb + TS - 1) / TS;
  const int i0 = (blockIdx.y / tiles_b) * TS, j0 = (blockIdx.y % tiles_b) * TS;
  const int r_lo = blockIdx.x * rows_per_split, r_hi = min(rows, r_lo + rows_per_split);
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  float acc[MT][MT] = {};
  for (int r0 = r_lo; r0 < r_hi; r0 += 32) {
    for (int e = tid; e < 32 * TS; e += 256) {
      const int rr = e / TS, c = e % TS;
      const int gr = r0 + rr;
      As[rr][c] = (gr < r_hi && i0 + c < ca) ? A[(size_t)gr * lda + i0 + c] : 0.f;
      float bval = 0.f;
      if (gr < r_hi && j0 + c < cb) {
        // B may arrive as several K-slice partials of the projection (fixed-order sum)
        const size_t o = (size_t)gr * ldb + j0 + c;
        bval = B[o];
        for (int sl = 1; sl < b_slices; ++sl) bval += B[(size_t)sl * rows * ldb + o];
      }
      Bs[rr][c] = bval;
    }
    __syncthreads();
#pragma unroll 8
    for (int rr = 0; rr < 32; ++rr) {
      float av[MT], bv[MT];
#pragma unroll
      for (int i = 0; i < MT; ++i) av[i] = As[rr][ty * MT + i];     // contiguous: compiles to 128-bit loads
#pragma unroll
      for (int j = 0; j < MT; ++j) bv[j] = Bs[rr][tx * MT + j];
#pragma unroll
      for (int i = 0; i < MT; ++i)
#pragma unroll
        for (int j = 0; j < MT; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < MT; ++i)
#pragma unroll
    for (int j = 0; j < MT; ++j) {
      const int gi = i0 + ty * MT + i, gj = j0 + tx * MT + j;
      if (gi < ca && gj < cb) part[(size_t)gi * cb + gj] = acc[i][j];
    }
}

__global__ void __launch_bounds__(256) sum_slices_kernel(const MatDev* tab, const int* idx, int offPart, int offOut,
                                                         int numel, int nsplit) {
  const MatDev& md = tab[idx[blockIdx.z]];
  const float* part = field<const float>(md, offPart);
  float* out = field<float>(md, offOut);
  for (int e = blockIdx.x * 256 + threadIdx.x; e < numel; e += gridDim.x * 256) {
    float t = 0.f;
    for (int s = 0; s < nsplit; ++s) t += part[(size_t)s * numel + e];
    out[e] = t;
  }
}

// Row slices of an A^T B product over `rows` rows when `count` matrices share the launch: about 1024 rows per
// slice for batched launches, finer (down to 128 rows) when few matrices would otherwise leave most SMs idle.
int atb_splits(int rows, int count) {
  int s = (rows + 1023) / 1024;
  const int want = (2 * 148 + count - 1) / (count > 0 ? count : 1);
  if (s < want) s = want;
  const int finest = (rows + 127) / 128;
  if (s > finest) s = finest;
  if (s > kAtbMaxSplits) s = kAtbMaxSplits;
  return s < 1 ? 1 : s;
}

void launch_atb(const MatDev* tab, const int* idx, int count, int offA, int offB, int offPart, int offOut, int rows,
                int ca, int cb, int lda, int ldb, int nsplit, cudaStream_t s, int b_slices, bool sum_here) {
  if (count <= 0 || ca <= 0 || cb <= 0) return;
  const int rps = ((rows + nsplit - 1) / nsplit + 31) / 32 * 32;
  const int big = ca > cb ? ca : cb;
  const int mt = big <= 16 ? 1 : big <= 32 ? 2 : big <= 64 ? 4 : 8;
  const int ts = 16 * mt;
  dim3 grid(nsplit, ((ca + ts - 1) / ts) * ((cb + ts - 1) / ts), count);
  switch (mt) {
    case 1: atb_kernel<1><<<grid, 256, 0, s>>>(tab, idx, offA, offB, offPart, rows, ca, cb, lda, ldb, rps, b_slices); break;
    case 2: atb_kernel<2><<<grid, 256, 0, s>>>(tab, idx, offA, offB, offPart, rows, ca, cb, lda, ldb, rps, b_slices); break;
    case 4: atb_kernel<4><<<grid, 256, 0, s>>>(tab, idx, offA, offB, offPart, rows, ca, cb, lda, ldb, rps, b_slices); break;
    default: atb_kernel<8><<<grid, 256, 0, s>>>(tab, idx, offA, offB, offPart, rows, ca, cb, lda, ldb, rps, b_slices); break;
  }
  ++g_kernel_launches;
  if (!sum_here) return;     // the consumer adds the row slices itself
  launch_sum_slices(tab, idx, count, offPart, offOut, ca * cb, nsplit, s);
}

// The same sum for many slices: 64 elements per block, the slices dealt to 16 groups of threads (group g adds slices
// g, g + 16, ... in increasing order), the 16 group sums added in group order. Fixed order, so reproducible.
__global__ void __launch_bounds__(1024) sum_slices_wide_kernel(const MatDev* tab, const int* idx, int offPart, int offOut,
                                                              int numel, int nsplit) {
  __shared__ float red[16][64];
  const MatDev& md = tab[idx[blockIdx.z]];
  const float* part = field<const float>(md, offPart);
  float* out = field<float>(md, offOut);
  const int el = threadIdx.x & 63, g = threadIdx.x >> 6;
  const int e = blockIdx.x * 64 + el;
  float t = 0.f;
  if (e < numel) {
#pragma unroll 8
    for (int s = g; s < nsplit; s += 16) t += part[(size_t)s * numel + e];
  }
  red[g][el] = t;
  __syncthreads();
  if (g == 0 && e < numel) {
    float a = red[0][el];
#pragma unroll
    for (int k = 1; k < 16; ++k) a += red[k][el];
    out[e] = a;
  }
}

void launch_sum_slices(const MatDev* tab, const int* idx, int count, int offPart, int offOut, int numel, int nsplit,
                       cudaStream_t s) {
  if (count <= 0 || numel <= 0) return;
  if (nsplit >= 32) {
    sum_slices_wide_kernel<<<dim3((numel + 63) / 64, 1, count), 1024, 0, s>>>(tab, idx, offPart, offOut, numel, nsplit);
    ++g_kernel_launches;
    return;
  }
  sum_slices_kernel<<<dim3((numel + 255) / 256 < 592 ? (numel + 255) / 256 : 592, 1, count), 256, 0, s>>>(
      tab, idx, offPart, offOut, numel, nsplit);
  ++g_kernel_launches;
}

// =====================================================================================================
// Eq. 1: anchor momentum  M <- beta M + (1 - beta) G_anc
// =====================================================================================================
__global__ void __launch_bounds__(256) ema_kernel(const MatDev* tab, const int* idx, int64_t numel, int g_bf16,
                                                  float beta) {
  const MatDev& md = tab[idx[blockIdx.z]];
  float* M = md.Manc;
  const float omb = 1.f - beta;
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  const int64_t t0 = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if ((numel & 3) == 0) {
    const int64_t n4 = numel >> 2;
    float4* M4 = reinterpret_cast<float4*>(M);
    for (int64_t i = t0; i < n4; i += stride) {
      float4 mv = M4[i];
      float g0, g1, g2, g3;
      if (g_bf16) {
        const uint2 raw = reinterpret_cast<const uint2*>(md.Ganc)[i];
        const __nv_bfloat162 a = *reinterpret_cast<const __nv_bfloat162*>(&raw.x);
        const __nv_bfloat162 b = *reinterpret_cast<const __nv_bfloat162*>(&raw.y);
        g0 = __low2float(a); g1 = __high2float(a); g2 = __low2float(b); g3 = __high2float(b);
      } else {
        const float4 gv = reinterpret_cast<const float4*>(md.Ganc)[i];
        g0 = gv.x; g1 = gv.y; g2 = gv.z; g3 = gv.w;
      }
      mv.x = fmaf(beta, mv.x, omb * g0); mv.y = fmaf(beta, mv.y, omb * g1);
      mv.z = fmaf(beta, mv.z, omb * g2); mv.w = fmaf(beta, mv.w, omb * g3);
      M4[i] = mv;
    }
  } else {
    for (int64_t i = t0; i < numel; i += stride) {
      const float g = g_bf16 ? __bfloat162float(reinterpret_cast<const bf16*>(md.Ganc)[i])
                             : reinterpret_cast<const float*>(md.Ganc)[i];
      M[i] = fmaf(beta, M[i], omb * g);
    }
  }
}

void launch_ema(const MatDev* tab, const int* idx, int count, int64_t numel, int g_bf16, float beta, cudaStream_t s) {
  if (count <= 0) return;
  int64_t blocks = (numel / 4 + 255) / 256;
  if (blocks > 148 * 8) blocks = 148 * 8;
  if (blocks < 1) blocks = 1;
  ema_kernel<<<dim3((unsigned)blocks, 1, count), 256, 0, s>>>(tab, idx, numel, g_bf16, beta);
  ++g_kernel_launches;
}

// =====================================================================================================
// Counter-based Rademacher sketch: Omega[j][c] = +1 / -1 from the top bit of a 64-bit hash of (seed, j, c).
//   counter = j * 2^10 + c ; h = mix(seed ^ ((counter + 1) * 0x9E3779B97F4A7C15)), mix = SplitMix64 finaliser.
// =====================================================================================================
__device__ __forceinline__ float sketch_entry(uint64_t seed, uint64_t j, uint64_t c) {
  uint64_t x = seed ^ (((j << 10) + c + 1ull) * 0x9E3779B97F4A7C15ull);
  x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
  x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
  x = x ^ (x >> 31);
  return (x >> 63) ? -1.f : 1.f;
}

__global__ void sketch_t_kernel(float* omega_t, int lp, int l, int64_t n, uint64_t seed) {
  const int64_t j = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int c = blockIdx.y;
  if (j >= n || c >= lp) return;
  omega_t[(size_t)c * n + j] = c < l ? sketch_entry(seed, (uint64_t)j, (uint64_t)c) : 0.f;
}

void launch_sketch(float* omega_t, int lp, int l, int64_t n, uint64_t seed, cudaStream_t s) {
  if (lp <= 0) return;
  sketch_t_kernel<<<dim3((unsigned)((n + 255) / 256), lp), 256, 0, s>>>(omega_t, lp, l, n, seed);
  ++g_kernel_launches;
}

__global__ void sketch_rm_kernel(float* omega, int64_t rows, int width, uint64_t seed) {
  const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= rows * width) return;
  omega[e] = sketch_entry(seed, (uint64_t)(e / width), (uint64_t)(e % width));
}

// Row-major n x lp copy of the sketch, columns l..lp-1 zero.
__global__ void sketch_padded_kernel(float* omega, int64_t rows, int lp, int l, uint64_t seed) {
  const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= rows * lp) return;
  const int c = (int)(e % lp);
  omega[e] = c < l ? sketch_entry(seed, (uint64_t)(e / lp), (uint64_t)c) : 0.f;
}

void launch_sketch_padded(float* omega, int64_t rows, int lp, int l, uint64_t seed, cudaStream_t s) {
  const int64_t tot = rows * lp;
  if (tot <= 0) return;
  sketch_padded_kernel<<<(unsigned)((tot + 255) / 256), 256, 0, s>>>(omega, rows, lp, l, seed);
  ++g_kernel_launches;
}

// Start block of a warm range finder: Z2[:, :rank] = previous V, Z2[:, rank:l] = sketch columns, rest zero.
__global__ void warm_start_kernel(const MatDev* tab, const int* idx, int n, int lp, int l, int rp, int rank,
                                  uint64_t seed) {
  const MatDev& md = tab[idx[blockIdx.z]];
  const int64_t stride = (int64_t)gridDim.x * blockDim.x, tot = (int64_t)n * lp;
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < tot; e += stride) {
    const int64_t j = e / lp;
    const int c = (int)(e % lp);
    float v = 0.f;
    if (c < rank) v = md.V[(size_t)j * rp + c];
    else if (c < l) v = sketch_entry(seed, (uint64_t)j, (uint64_t)c);
    md.Z2[e] = v;
  }
}

void launch_warm_start(const MatDev* tab, const int* idx, int count, int n, int lp, int l, int rp, int rank,
                       uint64_t seed, cudaStream_t s) {
  if (count <= 0 || lp <= 0) return;
  const int64_t tot = (int64_t)n * lp;
  const int blocks = (int)((tot + 255) / 256 < 592 ? (tot + 255) / 256 : 592);
  warm_start_kernel<<<dim3(blocks, 1, count), 256, 0, s>>>(tab, idx, n, lp, l, rp, rank, seed);
  ++g_kernel_launches;
}

void launch_sketch_rowmajor(float* omega, int64_t rows, int width, uint64_t seed, cudaStream_t s) {
  const int64_t tot = rows * width;
  if (tot <= 0) return;
  sketch_rm_kernel<<<(unsigned)((tot + 255) / 256), 256, 0, s>>>(omega, rows, width, seed);
  ++g_kernel_launches;
}

// =====================================================================================================
// Cholesky factor of the Gram matrix (gram = R^T R, R upper) and its inverse, one block per matrix.
// A pivot that has cancelled to (numerically) nothing marks a column that lies in the span of the earlier
// ones: that direction is dropped (its column of R^-1 is zero) instead of dividing by ~0.
// =====================================================================================================
// kSmem (the only form launched): the factor and its inverse are built in shared memory (2 lp^2 floats, lp <= 128) and
// copied out at the end. Larger factors (lp <= 256) go through chol_packed_kernel below.
template <bool kSmem>
__global__ void __launch_bounds__(256) chol_kernel(const MatDev* tab, const int* idx, int lp, int offR) {
  extern __shared__ __align__(16) float chol_smem[];
  __shared__ float invd[kMaxRank];
  __shared__ float piv_inv;
  const MatDev& md = tab[idx[blockIdx.x]];
  const float* G = md.gram;     // redirected to shared memory below when kSmem
  float* Rg = field<float>(md, offR);
  float* Rig = md.rinv;
  float* R = kSmem ? chol_smem : Rg;
  float* Ri = kSmem ? chol_smem + (size_t)lp * lp : Rig;
  const int t = threadIdx.x;
  if (kSmem) {
    // the Gram matrix comes into shared memory once (into the array that will hold the inverse, which is written only
    // after the factor is complete), so that no column step waits for a global load
    for (int e = t; e < lp * lp; e += 256) Ri[e] = md.gram[e];
    G = Ri;
    __syncthreads();
  }
  for (int j = 0; j < lp; ++j) {
    const int i = t;
    float s = 0.f;
    if (i >= j && i < lp) {
      // four independent partial sums: the dot product is a latency chain otherwise. fp32 is enough: the Gram
      // matrix itself was accumulated in fp32, and the second Cholesky QR round repairs what is lost here.
      float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
      int k = 0;
      for (; k + 3 < j; k += 4) {
        s0 = fmaf(R[(size_t)k * lp + j], R[(size_t)k * lp + i], s0);
        s1 = fmaf(R[(size_t)(k + 1) * lp + j], R[(size_t)(k + 1) * lp + i], s1);
        s2 = fmaf(R[(size_t)(k + 2) * lp + j], R[(size_t)(k + 2) * lp + i], s2);
        s3 = fmaf(R[(size_t)(k + 3) * lp + j], R[(size_t)(k + 3) * lp + i], s3);
      }
      for (; k < j; ++k) s0 = fmaf(R[(size_t)k * lp + j], R[(size_t)k * lp + i], s0);
      s = G[(size_t)j * lp + i] - ((s0 + s1) + (s2 + s3));
    }
    if (i == j) {
      const float gjj = G[(size_t)j * lp + j];
      const bool ok = (s > 1e-6f * gjj) && (gjj > 0.f);
      const float rjj = ok ? sqrtf(s) : 0.f;
      piv_inv = ok ? 1.f / rjj : 0.f;
      invd[j] = piv_inv;
      R[(size_t)j * lp + j] = rjj;
    }
    __syncthreads();
    if (i > j && i < lp) R[(size_t)j * lp + i] = s * piv_inv;
    if (i < j) R[(size_t)j * lp + i] = 0.f;
    __syncthreads();
  }
  // inverse of the upper-triangular factor, one column per thread
  const int c = t;
  if (c < lp) {
    for (int i = lp - 1; i > c; --i) Ri[(size_t)i * lp + c] = 0.f;
    Ri[(size_t)c * lp + c] = invd[c];
    for (int i = c - 1; i >= 0; --i) {
      float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
      int k = i + 1;
      for (; k + 3 <= c; k += 4) {
        s0 = fmaf(R[(size_t)i * lp + k], Ri[(size_t)k * lp + c], s0);
        s1 = fmaf(R[(size_t)i * lp + k + 1], Ri[(size_t)(k + 1) * lp + c], s1);
        s2 = fmaf(R[(size_t)i * lp + k + 2], Ri[(size_t)(k + 2) * lp + c], s2);
        s3 = fmaf(R[(size_t)i * lp + k + 3], Ri[(size_t)(k + 3) * lp + c], s3);
      }
      for (; k <= c; ++k) s0 = fmaf(R[(size_t)i * lp + k], Ri[(size_t)k * lp + c], s0);
      Ri[(size_t)i * lp + c] = -((s0 + s1) + (s2 + s3)) * invd[i];
    }
  }
  if (kSmem) {
    __syncthreads();
    for (int e = t; e < lp * lp; e += 256) { Rg[e] = R[e]; Rig[e] = Ri[e]; }
  }
}

// The same factorisation for 128 < lp <= 256, still on-chip: two full lp x lp arrays no longer fit in one SM's shared
// memory, so the upper triangle is kept PACKED (lp (lp + 1) / 2 floats, 129 KB at lp = 256) and everything happens in
// place: the Gram matrix is loaded into the packed array, row j of the factor overwrites row j of the Gram matrix (it
// is the last use of that row), the factor is copied out, and then the packed array is inverted in place column by
// column (x_j = -R^-1[0:j, 0:j] R[0:j, j] / r_jj uses only the already inverted leading block and column j itself).
// One thread per column, lp <= 256 threads.
__device__ __forceinline__ int tri_off(int j, int lp) { return j * lp - (j * (j - 1)) / 2; }   // start of packed row j

__global__ void __launch_bounds__(256) chol_packed_kernel(const MatDev* tab, const int* idx, int lp, int offR) {
  extern __shared__ __align__(16) float tri[];                 // packed upper triangle, row j: entries (j, j..lp-1)
  __shared__ float invd[kMaxRank];
  __shared__ float colj[kMaxRank];
  __shared__ int roff[kMaxRank];                                // roff[k] + c = position of element (k, c), c >= k
  __shared__ float piv_inv;
  const MatDev& md = tab[idx[blockIdx.x]];
  float* Rg = field<float>(md, offR);
  float* Rig = md.rinv;
  const int t = threadIdx.x;
  if (t < lp) roff[t] = tri_off(t, lp) - t;
  __syncthreads();
  for (int e = t; e < lp * lp; e += 256) {                      // coalesced read of the Gram matrix, upper part kept
    const int j = e / lp, i = e - j * lp;
    if (i >= j) tri[roff[j] + i] = md.gram[e];
  }
  __syncthreads();
  // factor: R[j][i] = (G[j][i] - sum_{k<j} R[k][j] R[k][i]) / r_jj, in place
  for (int j = 0; j < lp; ++j) {
    const int i = t;
    float s = 0.f;
    if (i >= j && i < lp) {
      float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
      int k = 0;
      for (; k + 3 < j; k += 4) {
        const int o0 = roff[k], o1 = roff[k + 1], o2 = roff[k + 2], o3 = roff[k + 3];
        s0 = fmaf(tri[o0 + j], tri[o0 + i], s0); s1 = fmaf(tri[o1 + j], tri[o1 + i], s1);
        s2 = fmaf(tri[o2 + j], tri[o2 + i], s2); s3 = fmaf(tri[o3 + j], tri[o3 + i], s3);
      }
      for (; k < j; ++k) { const int o = roff[k]; s0 = fmaf(tri[o + j], tri[o + i], s0); }
      s = tri[roff[j] + i] - ((s0 + s1) + (s2 + s3));
    }
    if (i == j) {
      const float gjj = tri[roff[j] + j];
      const bool ok = (s > 1e-6f * gjj) && (gjj > 0.f);
      const float rjj = ok ? sqrtf(s) : 0.f;
      piv_inv = ok ? 1.f / rjj : 0.f;
      invd[j] = piv_inv;
    }
    __syncthreads();
    if (i == j) tri[roff[j] + j] = piv_inv > 0.f ? 1.f / piv_inv : 0.f;
    if (i > j && i < lp) tri[roff[j] + i] = s * piv_inv;
    __syncthreads();
  }
  // copy the factor out (full lp x lp, zeros below the diagonal)
  for (int e = t; e < lp * lp; e += 256) {
    const int j = e / lp, i = e - j * lp;
    Rg[e] = i >= j ? tri[roff[j] + i] : 0.f;
  }
  __syncthreads();
  // in-place inverse, column by column
  for (int j = 0; j < lp; ++j) {
    if (t < j) colj[t] = tri[roff[t] + j];                        // R[0:j, j], about to be overwritten
    __syncthreads();
    if (t < j) {
      // x_t = -(sum_{k=t}^{j-1} Rinv[t][k] R[k][j]) / r_jj ; row t of the inverted block is packed row t, entries t..j-1
      const int o = roff[t];
      float s0 = 0.f, s1 = 0.f, s2 = 0.f, s3 = 0.f;
      int k = t;
      for (; k + 3 < j; k += 4) {
        s0 = fmaf(tri[o + k], colj[k], s0); s1 = fmaf(tri[o + k + 1], colj[k + 1], s1);
        s2 = fmaf(tri[o + k + 2], colj[k + 2], s2); s3 = fmaf(tri[o + k + 3], colj[k + 3], s3);
      }
      for (; k < j; ++k) s0 = fmaf(tri[o + k], colj[k], s0);
      tri[o + j] = -((s0 + s1) + (s2 + s3)) * invd[j];
    } else if (t == j) {
      tri[roff[j] + j] = invd[j];
    }
    __syncthreads();
  }
  for (int e = t; e < lp * lp; e += 256) {
    const int j = e / lp, i = e - j * lp;
    Rig[e] = i >= j ? tri[roff[j] + i] : 0.f;
  }
}

void launch_chol(const MatDev* tab, const int* idx, int count, int lp, int offR, cudaStream_t s) {
  if (count <= 0 || lp <= 0) return;
  if (lp <= 128) {
    const size_t smem = (size_t)2 * lp * lp * sizeof(float);
    cudaFuncSetAttribute(chol_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 2 * 128 * 128 * 4);
    chol_kernel<true><<<count, 256, smem, s>>>(tab, idx, lp, offR);
  } else {
    const size_t smem = ((size_t)lp * (lp + 1) / 2) * sizeof(float);
    cudaFuncSetAttribute(chol_packed_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (256 * 257 / 2) * 4);
    chol_packed_kernel<<<count, 256, smem, s>>>(tab, idx, lp, offR);
  }
  ++g_kernel_launches;
}

// =====================================================================================================
// One-sided Jacobi SVD of the small factor, one block per matrix.
//   racc = R (lp x lp) with B^T = Qb R, hence B = R^T Qb^T. Row j of R is column j of K = R^T, so the
//   buffer is read as lp contiguous columns. Right rotations J orthogonalise the columns: K J = Ub S.
//   Output (sorted by descending singular value, leading `rank` kept, padded to rp with zeros):
//     sv, d (Eq. 2), ub = Ub (lp x rp), wb = J (lp x rp).
// =====================================================================================================
constexpr int kJacobiThreads = 512;

template <bool kSmem>
__global__ void __launch_bounds__(kJacobiThreads) jacobi_kernel(const MatDev* tab, const int* idx, int lp, int rp,
                                                                int rank, float tau_p) {
  extern __shared__ __align__(16) float jac_smem[];   // kSmem (the only form launched): both l x l work arrays live here
                                                      // (lp <= 128); larger factors go through jacobi_cluster_kernel
  __shared__ float nrm[kMaxRank];
  __shared__ int order[kMaxRank];
  __shared__ int rotated;
  const MatDev& md = tab[idx[blockIdx.x]];
  float* Kc = kSmem ? jac_smem : md.jk;
  float* Jc = kSmem ? jac_smem + (size_t)lp * lp : md.jv;
  const float* R = md.racc;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarp = kJacobiThreads / 32;
  for (int e = tid; e < lp * lp; e += kJacobiThreads) {
    Kc[e] = R[e];
    Jc[e] = (e / lp == e % lp) ? 1.f : 0.f;
  }
  __syncthreads();
  const int half = lp / 2;
  for (int sweep = 0; sweep < 16; ++sweep) {
    if (tid == 0) rotated = 0;
    __syncthreads();
    for (int rd = 0; rd < lp - 1; ++rd) {
      for (int pi = warp; pi < half; pi += nwarp) {
        int p, q;
        if (pi == 0) { p = lp - 1; q = rd; }
        else { p = (rd + pi) % (lp - 1); q = (rd - pi + (lp - 1)) % (lp - 1); }
        float* kp = Kc + (size_t)p * lp; float* kq = Kc + (size_t)q * lp;
        float a = 0.f, b = 0.f, c = 0.f;
        for (int i = lane; i < lp; i += 32) {
          const float x = kp[i], y = kq[i];
          a = fmaf(x, x, a); b = fmaf(y, y, b); c = fmaf(x, y, c);
        }
        a = warp_sum(a); b = warp_sum(b); c = warp_sum(c);
        const float lim = sqrtf(a) * sqrtf(b);
        if (!(fabsf(c) > 1e-7f * lim) || lim == 0.f) continue;
        if (fabsf(c) > 4e-6f * lim && lane == 0) rotated = 1;   // below this the fp32 dot product is noise
        const float zeta = (b - a) / (2.f * c);
        const float tt = copysignf(1.f, zeta) / (fabsf(zeta) + sqrtf(1.f + zeta * zeta));
        const float cs = rsqrtf(1.f + tt * tt), sn = cs * tt;
        float* jp = Jc + (size_t)p * lp; float* jq = Jc + (size_t)q * lp;
        for (int i = lane; i < lp; i += 32) {
          const float x = kp[i], y = kq[i];
          kp[i] = cs * x - sn * y; kq[i] = sn * x + cs * y;
          const float u = jp[i], w = jq[i];
          jp[i] = cs * u - sn * w; jq[i] = sn * u + cs * w;
        }
      }
      __syncthreads();
    }
    if (!rotated) break;
    __syncthreads();
  }
  // column norms = singular values
  for (int j = warp; j < lp; j += nwarp) {
    float a = 0.f;
    for (int i = lane; i < lp; i += 32) { const float x = Kc[(size_t)j * lp + i]; a = fmaf(x, x, a); }
    a = warp_sum(a);
    if (lane == 0) nrm[j] = sqrtf(a);
  }
  __syncthreads();
  // rank of each column by counting (stable for ties)
  for (int j = tid; j < lp; j += kJacobiThreads) {
    int rk = 0;
    const float sj = nrm[j];
    for (int k = 0; k < lp; ++k) rk += (nrm[k] > sj) || (nrm[k] == sj && k < j);
    order[rk] = j;
  }
  __syncthreads();
  const float smax = nrm[order[0]];
  for (int k = tid; k < rp; k += kJacobiThreads) {
    float s = (k < rank && k < lp) ? nrm[order[k]] : 0.f;
    if (!(s > 1e-7f * smax)) s = 0.f;
    md.sv[k] = s;
    md.d[k] = (s + tau_p > 0.f) ? s / (s + tau_p) : 0.f;
  }
  for (int e = tid; e < lp * rp; e += kJacobiThreads) {
    const int i = e / rp, k = e % rp;
    float u = 0.f, w = 0.f;
    if (k < rank && k < lp) {
      const int j = order[k];
      const float s = nrm[j];
      if (s > 1e-7f * smax) { u = Kc[(size_t)j * lp + i] / s; w = Jc[(size_t)j * lp + i]; }
    }
    md.ub[e] = u;
    md.wb[e] = w;
  }
}

// The same SVD for 128 < lp <= 256, still on-chip: the two lp x lp work arrays (512 KB at lp = 256) are spread over the
// shared memory of a CLUSTER of four blocks, lp / 4 columns of each array per block. A warp that rotates columns p and
// q reaches them through distributed shared memory (plain loads and stores on addresses mapped into the owning block;
// no multicast), rounds are separated by cluster barriers, and the "did anything rotate" flag lives in block 0.
// Block 0 writes the results; the others wait in a final cluster barrier so that their shared memory stays alive.
constexpr int kJacobiClusterThreads = 1024;     // 4 x 32 warps = one warp per column pair of a round at lp = 256

__global__ void __cluster_dims__(4, 1, 1) __launch_bounds__(kJacobiClusterThreads)
jacobi_cluster_kernel(const MatDev* tab, const int* idx, int lp, int rp, int rank, float tau_p) {
  constexpr int kJacobiThreads = kJacobiClusterThreads;
  namespace cg = cooperative_groups;
  extern __shared__ __align__(16) float jc_smem[];
  __shared__ float nrm[kMaxRank];
  __shared__ int order[kMaxRank];
  __shared__ int rotated;
  cg::cluster_group cluster = cg::this_cluster();
  const int crank = (int)cluster.block_rank();
  const MatDev& md = tab[idx[blockIdx.x >> 2]];
  const int cols_per = lp >> 2;                        // lp is a multiple of 32
  float* Kl = jc_smem;                                 // this block's columns of K = R^T ...
  float* Jl = jc_smem + (size_t)cols_per * lp;         // ... and of the accumulated rotations
  const float* R = md.racc;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5, nwarp = kJacobiThreads / 32;
  for (int e = tid; e < cols_per * lp; e += kJacobiThreads) {
    const int c = crank * cols_per + e / lp, i = e % lp;
    Kl[e] = R[(size_t)c * lp + i];
    Jl[e] = (c == i) ? 1.f : 0.f;
  }
  if (tid == 0) rotated = 0;
  cluster.sync();
  auto kcol = [&](int c) { return cluster.map_shared_rank(Kl + (size_t)(c % cols_per) * lp, c / cols_per); };
  auto jcol = [&](int c) { return cluster.map_shared_rank(Jl + (size_t)(c % cols_per) * lp, c / cols_per); };
  int* rot0 = cluster.map_shared_rank(&rotated, 0);
  float* nrm0 = cluster.map_shared_rank(nrm, 0);
  const int half = lp / 2, gw = crank * nwarp + warp, gwarps = 4 * nwarp;
  for (int sweep = 0; sweep < 16; ++sweep) {
    for (int rd = 0; rd < lp - 1; ++rd) {
      for (int pi = gw; pi < half; pi += gwarps) {
        int p, q;
        if (pi == 0) { p = lp - 1; q = rd; }
        else { p = (rd + pi) % (lp - 1); q = (rd - pi + (lp - 1)) % (lp - 1); }
        float* kp = kcol(p); float* kq = kcol(q);
        float* jp = jcol(p); float* jq = jcol(q);
        // both columns of K and of J come into registers first (lp / 32 <= 8 elements per lane each): all the
        // distributed-shared-memory loads of a pair are in flight together instead of one round trip per element
        float x[8], y[8], u[8], w[8];
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const int i = lane + 32 * e;
          const bool in = i < lp;
          x[e] = in ? kp[i] : 0.f; y[e] = in ? kq[i] : 0.f;
          u[e] = in ? jp[i] : 0.f; w[e] = in ? jq[i] : 0.f;
        }
        float a = 0.f, b = 0.f, c = 0.f;
#pragma unroll
        for (int e = 0; e < 8; ++e) { a = fmaf(x[e], x[e], a); b = fmaf(y[e], y[e], b); c = fmaf(x[e], y[e], c); }
        a = warp_sum(a); b = warp_sum(b); c = warp_sum(c);
        const float lim = sqrtf(a) * sqrtf(b);
        if (!(fabsf(c) > 1e-7f * lim) || lim == 0.f) continue;
        if (fabsf(c) > 4e-6f * lim && lane == 0) *rot0 = 1;     // below this the fp32 dot product is noise
        const float zeta = (b - a) / (2.f * c);
        const float tt = copysignf(1.f, zeta) / (fabsf(zeta) + sqrtf(1.f + zeta * zeta));
        const float cs = rsqrtf(1.f + tt * tt), sn = cs * tt;
#pragma unroll
        for (int e = 0; e < 8; ++e) {
          const int i = lane + 32 * e;
          if (i < lp) {
            kp[i] = cs * x[e] - sn * y[e]; kq[i] = sn * x[e] + cs * y[e];
            jp[i] = cs * u[e] - sn * w[e]; jq[i] = sn * u[e] + cs * w[e];
          }
        }
      }
      cluster.sync();
    }
    const int any = *rot0;          // the same value in every thread of the cluster: written before the barrier above
    cluster.sync();                 // everyone has read it before block 0 clears it
    if (!any) break;
    if (crank == 0 && tid == 0) rotated = 0;
    cluster.sync();
  }
  // column norms = singular values, into block 0
  for (int j = warp; j < cols_per; j += nwarp) {
    float a = 0.f;
    for (int i = lane; i < lp; i += 32) { const float x = Kl[(size_t)j * lp + i]; a = fmaf(x, x, a); }
    a = warp_sum(a);
    if (lane == 0) nrm0[crank * cols_per + j] = sqrtf(a);
  }
  cluster.sync();
  if (crank == 0) {
    for (int j = tid; j < lp; j += kJacobiThreads) {      // rank of each column by counting (stable for ties)
      int rk = 0;
      const float sj = nrm[j];
      for (int k = 0; k < lp; ++k) rk += (nrm[k] > sj) || (nrm[k] == sj && k < j);
      order[rk] = j;
    }
    __syncthreads();
    const float smax = nrm[order[0]];
    for (int k = tid; k < rp; k += kJacobiThreads) {
      float s = (k < rank && k < lp) ? nrm[order[k]] : 0.f;
      if (!(s > 1e-7f * smax)) s = 0.f;
      md.sv[k] = s;
      md.d[k] = (s + tau_p > 0.f) ? s / (s + tau_p) : 0.f;
    }
    for (int e = tid; e < lp * rp; e += kJacobiThreads) {
      const int i = e / rp, k = e % rp;
      float u = 0.f, w = 0.f;
      if (k < rank && k < lp) {
        const int j = order[k];
        const float s = nrm[j];
        if (s > 1e-7f * smax) { u = kcol(j)[i] / s; w = jcol(j)[i]; }
      }
      md.ub[e] = u;
      md.wb[e] = w;
    }
  }
  cluster.sync();                   // nobody leaves while block 0 may still be reading its columns
}

void launch_jacobi(const MatDev* tab, const int* idx, int count, int lp, int rp, int rank, float tau_p,
                   cudaStream_t s) {
  if (count <= 0 || lp <= 0 || rp <= 0) return;
  if (lp <= 128) {
    const size_t smem = (size_t)2 * lp * lp * sizeof(float);
    cudaFuncSetAttribute(jacobi_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, 2 * 128 * 128 * 4);
    jacobi_kernel<true><<<count, kJacobiThreads, smem, s>>>(tab, idx, lp, rp, rank, tau_p);
  } else {
    const size_t smem = (size_t)2 * (lp / 4) * lp * sizeof(float);
    cudaFuncSetAttribute(jacobi_cluster_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 2 * 64 * 256 * 4);
    jacobi_cluster_kernel<<<count * 4, kJacobiClusterThreads, smem, s>>>(tab, idx, lp, rp, rank, tau_p);
  }
  ++g_kernel_launches;
}

// Eq. 2 from stored singular values (used after a basis import).
__global__ void filter_weights_kernel(const MatDev* tab, const int* idx, int rp, int rank, float tau_p) {
  const MatDev& md = tab[idx[blockIdx.x]];
  for (int k = threadIdx.x; k < rp; k += blockDim.x) {
    const float s = k < rank ? md.sv[k] : 0.f;
    md.d[k] = (s + tau_p > 0.f) ? s / (s + tau_p) : 0.f;
  }
}

void launch_filter_weights(const MatDev* tab, const int* idx, int count, int rp, int rank, float tau_p,
                           cudaStream_t s) {
  if (count <= 0 || rp <= 0) return;
  filter_weights_kernel<<<count, 256, 0, s>>>(tab, idx, rp, rank, tau_p);
  ++g_kernel_launches;
}

// =====================================================================================================
// bf16 hi/lo splits of the basis: U ~= Uhi + Ulo (m x rp), V^T ~= Vthi + Vtlo (rp x n, transposed).
// =====================================================================================================
// blockIdx.y == 0: U (m x rp fp32) -> Uhi, Ulo (row stride rk; columns rp..rk-1 stay zero), four columns per thread.
// blockIdx.y == 1: V (n x rp fp32) -> Vthi, Vtlo = the TRANSPOSE (rp x n) through 32 x 32 shared-memory tiles, so that
// both the reads (along the rank index) and the writes (along n) are coalesced.
__global__ void __launch_bounds__(256) split_basis_kernel(const MatDev* tab, const int* idx, int m, int n, int rp,
                                                          int rk) {
  const MatDev& md = tab[idx[blockIdx.z]];
  if (blockIdx.y == 0) {
    const int q = rp >> 2;                                     // rp is a multiple of 16
    const int64_t nu4 = (int64_t)m * q;
    for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < nu4; e += (int64_t)gridDim.x * blockDim.x) {
      const int64_t i = e / q;
      const int k = (int)(e - i * q) * 4;
      const float4 u = *reinterpret_cast<const float4*>(md.U + i * rp + k);
      bf16 h[4], l[4];
      split2(u.x, h[0], l[0]); split2(u.y, h[1], l[1]); split2(u.z, h[2], l[2]); split2(u.w, h[3], l[3]);
      *reinterpret_cast<uint2*>(md.Uhi + i * rk + k) = *reinterpret_cast<const uint2*>(h);
      *reinterpret_cast<uint2*>(md.Ulo + i * rk + k) = *reinterpret_cast<const uint2*>(l);
    }
  } else {
    __shared__ float tile[32][33];
    const int tx = threadIdx.x & 31, ty = threadIdx.x >> 5;    // 32 x 8 threads
    const int ktiles = rp >> 5 ? (rp + 31) >> 5 : 1, jtiles = (n + 31) >> 5;
    for (int t = blockIdx.x; t < ktiles * jtiles; t += gridDim.x) {
      const int j0 = (t / ktiles) * 32, k0 = (t % ktiles) * 32;
      __syncthreads();
      for (int r = ty; r < 32; r += 8) {
        const int j = j0 + r, k = k0 + tx;
        tile[r][tx] = (j < n && k < rp) ? md.V[(size_t)j * rp + k] : 0.f;
      }
      __syncthreads();
      for (int r = ty; r < 32; r += 8) {
        const int k = k0 + r, j = j0 + tx;
        if (k < rp && j < n) split2(tile[tx][r], md.Vthi[(size_t)k * n + j], md.Vtlo[(size_t)k * n + j]);
      }
    }
  }
}

void launch_split_basis(const MatDev* tab, const int* idx, int count, int m, int n, int rp, int rk, cudaStream_t s) {
  if (count <= 0 || rp <= 0) return;
  const int64_t work = std::max<int64_t>((int64_t)m * rp / 4, (int64_t)((n + 31) / 32) * ((rp + 31) / 32) * 256);
  const int blocks = (int)std::min<int64_t>((work + 255) / 256, 592);
  split_basis_kernel<<<dim3(blocks, 2, count), 256, 0, s>>>(tab, idx, m, n, rp, rk);
  ++g_kernel_launches;
}

// =====================================================================================================
// ||G||_F^2 in two fixed-order stages (no float atomics): kSqnormBlocks partials per matrix.
// =====================================================================================================
__global__ void __launch_bounds__(256) sqnorm_kernel(const MatDev* tab, const int* idx, int64_t numel, int g_bf16) {
  __shared__ float red[8];
  const MatDev& md = tab[idx[blockIdx.z]];
  const int64_t per = (numel + kSqnormBlocks - 1) / kSqnormBlocks;
  const int64_t lo = per * blockIdx.x, hi = (lo + per < numel) ? lo + per : numel;
  float acc = 0.f;
  for (int64_t i = lo + threadIdx.x; i < hi; i += 256) {
    const float g = g_bf16 ? __bfloat162float(reinterpret_cast<const bf16*>(md.G)[i])
                           : reinterpret_cast<const float*>(md.G)[i];
    acc = fmaf(g, g, acc);
  }
  acc = warp_sum(acc);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = 0.f;
    for (int w = 0; w < 8; ++w) t += red[w];
    md.sqpart[blockIdx.x] = t;
  }
}

void launch_sqnorm(const MatDev* tab, const int* idx, int count, int64_t numel, int g_bf16, cudaStream_t s) {
  if (count <= 0) return;
  sqnorm_kernel<<<dim3(kSqnormBlocks, 1, count), 256, 0, s>>>(tab, idx, numel, g_bf16);
  ++g_kernel_launches;
}

// =====================================================================================================
// The r x r filter: Xs = coef * D X D (coef = (1-alpha)*scale), and the per-matrix statistics.
//   stats[0] = ||g||^2, stats[1] = ||X||^2 (scaled), stats[2] = ||G_proj||^2 (closed form), stats[3] = sum d^2
// =====================================================================================================
__global__ void __launch_bounds__(1024) xs_kernel(const MatDev* tab, const int* idx, int rp, int rank, int x_slices,
                                                 float scale, float alpha, unsigned* status) {
  __shared__ float red[5][32];
  const int nt = blockDim.x;             // 256 threads, 1024 from rank 64 on (one block per matrix either way)
  const MatDev& md = tab[idx[blockIdx.x]];
  float sx = 0.f, s1 = 0.f, s2 = 0.f;
  const int numel = rp * rp;
  // four elements per thread at a time, so that their loads (and the slices' loads) are in flight together
  for (int e0 = threadIdx.x; e0 < numel; e0 += 4 * nt) {
    float xr[4] = {0.f, 0.f, 0.f, 0.f};
    if (x_slices > 0) {                   // X = sum of the row-slice partials of U^T T, in slice order
      for (int sl = 0; sl < x_slices; ++sl) {
        const float* ps = md.xpart + (size_t)sl * numel;
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          const int e = e0 + nt * u;
          if (e < numel) xr[u] += ps[e];
        }
      }
    } else {                              // already summed by a separate launch
#pragma unroll
      for (int u = 0; u < 4; ++u) {
        const int e = e0 + nt * u;
        if (e < numel) xr[u] = md.X[e];
      }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      const int e = e0 + nt * u;
      if (e >= numel) break;
      const int i = e / rp, j = e % rp;
      if (x_slices > 0) md.X[e] = xr[u];
      const float x = xr[u] * scale;
      const float dd = (i < rank && j < rank) ? md.d[i] * md.d[j] : 0.f;
      md.Xs[e] = (1.f - alpha) * dd * x;
      sx = fmaf(x, x, sx);
      s1 = fmaf(dd * x, x, s1);
      s2 = fmaf(dd * dd * x, x, s2);
    }
  }
  // ||g||^2 from its block partials and sum d^2, one term per thread; all five sums by warp, then in warp order
  const int tid = threadIdx.x;
  float gg = tid < kSqnormBlocks ? md.sqpart[tid] : 0.f;
  float re = tid < rank ? md.d[tid] * md.d[tid] : 0.f;
  sx = warp_sum(sx); s1 = warp_sum(s1); s2 = warp_sum(s2); gg = warp_sum(gg); re = warp_sum(re);
  if ((tid & 31) == 0) {
    const int w = tid >> 5;
    red[0][w] = sx; red[1][w] = s1; red[2][w] = s2; red[3][w] = gg; red[4][w] = re;
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    float tx = 0.f, t1 = 0.f, t2 = 0.f;
    gg = 0.f; re = 0.f;
    for (int w = 0; w < nt / 32; ++w) { tx += red[0][w]; t1 += red[1][w]; t2 += red[2][w]; gg += red[3][w]; re += red[4][w]; }
    gg *= scale * scale;
    md.stats[0] = gg;
    md.stats[1] = tx;
    md.stats[2] = alpha * alpha * gg + 2.f * alpha * (1.f - alpha) * t1 + (1.f - alpha) * (1.f - alpha) * t2;
    md.stats[3] = re;
    // a NaN or Inf anywhere in the gradient reaches X = U^T G V (or ||g||^2): latch it for the host
    if (!isfinite(tx) || !isfinite(gg)) atomicOr(status, kDevNonfinite);
  }
}

void launch_xs(const MatDev* tab, const int* idx, int count, int rp, int rank, int x_slices, float scale, float alpha,
               unsigned* status, cudaStream_t s) {
  if (count <= 0) return;
  xs_kernel<<<count, rp >= 64 ? 1024 : 256, 0, s>>>(tab, idx, rp, rank, x_slices, scale, alpha, status);
  ++g_kernel_launches;
}

// =====================================================================================================
// The r x r filter and C^T = V Xs^T in one launch (padded rank up to 128). Every block forms Xs = coef * D X D in
// shared memory from the summed X (16 to 64 KB out of L2) and multiplies its 64 rows of V by Xs^T; block 0 of a matrix
// also writes Xs and the statistics, exactly as xs_kernel does. The sum over the rank index runs in increasing order
// with one fmaf per term, like tsgemm_kernel, so C^T has the same bits as from the two separate launches.
// CPT = rp / 16 columns of C^T per thread.
// =====================================================================================================
template <int CPT>
__global__ void __launch_bounds__(256) filter_ct_kernel(const MatDev* tab, const int* idx, int rank, int n, int rk,
                                                        float scale, float alpha, unsigned* status) {
  constexpr int RP = 16 * CPT, XP = RP + 1, VP = RP + 4, RB = 64;
  extern __shared__ __align__(16) float fct_smem[];
  float* Vs = fct_smem;                  // [RB][VP]
  float* Xs = fct_smem + RB * VP;        // [RP][XP]
  __shared__ float red[5][8];
  static_assert(kSqnormBlocks <= 256, "one partial of ||g||^2 per thread");
  const MatDev& md = tab[idx[blockIdx.z]];
  const bool lead = blockIdx.x == 0;
  const int tid = threadIdx.x, row0 = blockIdx.x * RB;
  // every global load of a phase is issued before its first use (the kernel is a chain of load latencies otherwise)
  __shared__ float ds[RP];
  if (tid < RP) ds[tid] = tid < rank ? md.d[tid] : 0.f;
  constexpr int NV = RB * (RP / 4) / 256;          // float4 loads of V per thread (= CPT)
  float4 vreg[NV];
#pragma unroll
  for (int u = 0; u < NV; ++u) {
    const int e = tid + 256 * u, r = e / (RP / 4), q = e % (RP / 4);
    vreg[u] = make_float4(0.f, 0.f, 0.f, 0.f);
    if (row0 + r < n) vreg[u] = *reinterpret_cast<const float4*>(md.V + (size_t)(row0 + r) * RP + 4 * q);
  }
  constexpr int NX = RP * RP / 256;                // elements of X per thread (= CPT^2)
  constexpr int XB = NX < 16 ? NX : 16;            // loaded in batches of up to 16
  float sx = 0.f, s1 = 0.f, s2 = 0.f;
  float xr[XB];
#pragma unroll
  for (int u = 0; u < XB; ++u) xr[u] = md.X[tid + 256 * u];
#pragma unroll
  for (int u = 0; u < NV; ++u) {
    const int e = tid + 256 * u, r = e / (RP / 4), q = e % (RP / 4);
    *reinterpret_cast<float4*>(Vs + r * VP + 4 * q) = vreg[u];
  }
  __syncthreads();                                 // ds
  for (int b0 = 0; b0 < NX; b0 += XB) {
    float xn[XB];
    if (b0 + XB < NX) {
#pragma unroll
      for (int u = 0; u < XB; ++u) xn[u] = (b0 + XB + u < NX) ? md.X[tid + 256 * (b0 + XB + u)] : 0.f;
    }
#pragma unroll
    for (int u = 0; u < XB; ++u) {
      if (b0 + u >= NX) break;
      const int e = tid + 256 * (b0 + u);
      const int i = e / RP, j = e % RP;
      const float x = xr[u] * scale;
      const float dd = ds[i] * ds[j];              // zero beyond the rank
      const float xs = (1.f - alpha) * dd * x;
      Xs[i * XP + j] = xs;
      if (lead) {
        md.Xs[e] = xs;
        sx = fmaf(x, x, sx);
        s1 = fmaf(dd * x, x, s1);
        s2 = fmaf(dd * dd * x, x, s2);
      }
    }
    if (b0 + XB < NX) {
#pragma unroll
      for (int u = 0; u < XB; ++u) xr[u] = xn[u];
    }
  }
  if (lead) {
    // ||g||^2 from its block partials and sum d^2, one term per thread; all five sums by warp, then in warp order
    float gg = tid < kSqnormBlocks ? md.sqpart[tid] : 0.f;
    float re = tid < rank ? md.d[tid] * md.d[tid] : 0.f;
    sx = warp_sum(sx); s1 = warp_sum(s1); s2 = warp_sum(s2); gg = warp_sum(gg); re = warp_sum(re);
    if ((tid & 31) == 0) {
      const int w = tid >> 5;
      red[0][w] = sx; red[1][w] = s1; red[2][w] = s2; red[3][w] = gg; red[4][w] = re;
    }
  }
  __syncthreads();
  if (lead && tid == 0) {
    float tx = 0.f, t1 = 0.f, t2 = 0.f, gg = 0.f, re = 0.f;
    for (int w = 0; w < 8; ++w) { tx += red[0][w]; t1 += red[1][w]; t2 += red[2][w]; gg += red[3][w]; re += red[4][w]; }
    gg *= scale * scale;
    md.stats[0] = gg;
    md.stats[1] = tx;
    md.stats[2] = alpha * alpha * gg + 2.f * alpha * (1.f - alpha) * t1 + (1.f - alpha) * (1.f - alpha) * t2;
    md.stats[3] = re;
    if (!isfinite(tx) || !isfinite(gg)) atomicOr(status, kDevNonfinite);
  }
  // rows ty + 16 i (i < 4), columns CPT tx .. CPT tx + CPT - 1
  const int ty = tid >> 4, tx = tid & 15;
  float acc[4][CPT];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < CPT; ++j) acc[i][j] = 0.f;
#pragma unroll 4
  for (int b = 0; b < RP; ++b) {
    float xv[CPT], vv[4];
#pragma unroll
    for (int j = 0; j < CPT; ++j) xv[j] = Xs[(tx * CPT + j) * XP + b];
#pragma unroll
    for (int i = 0; i < 4; ++i) vv[i] = Vs[(ty + 16 * i) * VP + b];
#pragma unroll
    for (int i = 0; i < 4; ++i)
#pragma unroll
      for (int j = 0; j < CPT; ++j) acc[i][j] = fmaf(vv[i], xv[j], acc[i][j]);
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int gr = row0 + ty + 16 * i;
    if (gr >= n) continue;
    if (md.Cthi) {          // the tensor-core update takes the bf16 pair (nobody reads the fp32 copy then)
      bf16 hi[CPT], lo[CPT];
#pragma unroll
      for (int j = 0; j < CPT; ++j) split2(1.f * acc[i][j], hi[j], lo[j]);
      const size_t o = (size_t)gr * rk + tx * CPT;
      if (CPT % 4 == 0) {   // four columns as one 8-byte store (rk is a multiple of 64)
#pragma unroll
        for (int j = 0; j < CPT; j += 4) {
          uint2 ph, pl;
          ph.x = (uint32_t)__bfloat16_as_ushort(hi[j]) | ((uint32_t)__bfloat16_as_ushort(hi[j + 1]) << 16);
          ph.y = (uint32_t)__bfloat16_as_ushort(hi[j + 2]) | ((uint32_t)__bfloat16_as_ushort(hi[j + 3]) << 16);
          pl.x = (uint32_t)__bfloat16_as_ushort(lo[j]) | ((uint32_t)__bfloat16_as_ushort(lo[j + 1]) << 16);
          pl.y = (uint32_t)__bfloat16_as_ushort(lo[j + 2]) | ((uint32_t)__bfloat16_as_ushort(lo[j + 3]) << 16);
          *reinterpret_cast<uint2*>(md.Cthi + o + j) = ph;
          *reinterpret_cast<uint2*>(md.Ctlo + o + j) = pl;
        }
      } else {
#pragma unroll
        for (int j = 0; j < CPT; ++j) { md.Cthi[o + j] = hi[j]; md.Ctlo[o + j] = lo[j]; }
      }
    } else {
#pragma unroll
      for (int j = 0; j < CPT; ++j) md.Ct[(size_t)gr * RP + tx * CPT + j] = 1.f * acc[i][j];
    }
  }
}

bool filter_ct_supported(int rp) { return rp >= 16 && rp <= 128 && rp % 16 == 0; }

template <int CPT>
static void launch_filter_ct_t(const MatDev* tab, const int* idx, int count, int rank, int n, int rk, float scale,
                               float alpha, unsigned* status, cudaStream_t s) {
  constexpr int RP = 16 * CPT;
  constexpr size_t smem = ((size_t)64 * (RP + 4) + (size_t)RP * (RP + 1)) * sizeof(float);
  static const cudaError_t attr =
      cudaFuncSetAttribute(filter_ct_kernel<CPT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  (void)attr;
  filter_ct_kernel<CPT><<<dim3((n + 63) / 64, 1, count), 256, smem, s>>>(tab, idx, rank, n, rk, scale, alpha, status);
}

void launch_filter_ct(const MatDev* tab, const int* idx, int count, int rp, int rank, int n, int rk, float scale,
                      float alpha, unsigned* status, cudaStream_t s) {
  if (count <= 0 || !filter_ct_supported(rp)) return;
  switch (rp / 16) {
    case 1: launch_filter_ct_t<1>(tab, idx, count, rank, n, rk, scale, alpha, status, s); break;
    case 2: launch_filter_ct_t<2>(tab, idx, count, rank, n, rk, scale, alpha, status, s); break;
    case 3: launch_filter_ct_t<3>(tab, idx, count, rank, n, rk, scale, alpha, status, s); break;
    case 4: launch_filter_ct_t<4>(tab, idx, count, rank, n, rk, scale, alpha, status, s); break;
    case 5: launch_filter_ct_t<5>(tab, idx, count, rank, n, rk, scale, alpha, status, s); break;
    case 6: launch_filter_ct_t<6>(tab, idx, count, rank, n, rk, scale, alpha, status, s); break;
    case 7: launch_filter_ct_t<7>(tab, idx, count, rank, n, rk, scale, alpha, status, s); break;
    default: launch_filter_ct_t<8>(tab, idx, count, rank, n, rk, scale, alpha, status, s); break;
  }
  ++g_kernel_launches;
}

// Global-norm clip factor over all matrices, summed in matrix order by one thread block.
__global__ void clip_kernel(const MatDev* tab, int n_mats, float max_norm, float* clip) {
  __shared__ float red[256];
  float acc = 0.f;
  for (int i = threadIdx.x; i < n_mats; i += 256) acc += tab[i].stats[2];
  red[threadIdx.x] = acc;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = 0.f;
    for (int i = 0; i < 256; ++i) t += red[i];
    const float nrm = sqrtf(t);
    *clip = (max_norm > 0.f && nrm > max_norm) ? max_norm / nrm : 1.f;
  }
}

void launch_clip(const MatDev* tab, int n_mats, float max_norm, float* clip, cudaStream_t s) {
  clip_kernel<<<1, 256, 0, s>>>(tab, n_mats, max_norm, clip);
  ++g_kernel_launches;
}

// Copies between a dense rows x cols matrix and its zero-padded rows x cols_dst copy (basis import/export).
__global__ void pad_copy_kernel(float* dst, int ldd, const float* src, int lds, int rows, int cols, int cols_dst) {
  const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= (int64_t)rows * cols_dst) return;
  const int i = (int)(e / cols_dst), j = (int)(e % cols_dst);
  dst[(size_t)i * ldd + j] = j < cols ? src[(size_t)i * lds + j] : 0.f;
}

void launch_pad_copy(float* dst, int ldd, const float* src, int lds, int rows, int cols, int cols_dst,
                     cudaStream_t s) {
  const int64_t tot = (int64_t)rows * cols_dst;
  if (tot <= 0) return;
  pad_copy_kernel<<<(unsigned)((tot + 255) / 256), 256, 0, s>>>(dst, ldd, src, lds, rows, cols, cols_dst);
  ++g_kernel_launches;
}

void launch_unpad_copy(float* dst, int ldd, const float* src, int lds, int rows, int cols, cudaStream_t s) {
  launch_pad_copy(dst, ldd, src, lds, rows, cols, cols, s);
}

// Sum of split-K partials of T (fixed order): T[0] <- sum_s T[s]. 128-bit accesses (numel is a multiple of 16), the
// loads of all slices of an element issued together.
__global__ void reduce_partials_kernel(const MatDev* tab, const int* idx, int64_t numel4, int ksplit) {
  const MatDev& md = tab[idx[blockIdx.z]];
  float4* T4 = reinterpret_cast<float4*>(md.T);
  const int64_t stride = (int64_t)gridDim.x * blockDim.x;
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < numel4; e += stride) {
    float4 v[8];
#pragma unroll
    for (int s = 0; s < 8; ++s)
      if (s < ksplit) v[s] = T4[(size_t)s * numel4 + e];
    float4 t = v[0];
#pragma unroll
    for (int s = 1; s < 8; ++s)
      if (s < ksplit) { t.x += v[s].x; t.y += v[s].y; t.z += v[s].z; t.w += v[s].w; }
    T4[e] = t;
  }
}

void launch_reduce_partials(const MatDev* tab, const int* idx, int count, int64_t numel, int ksplit, cudaStream_t s) {
  if (count <= 0 || ksplit <= 1) return;
  const int64_t numel4 = numel / 4;      // rows x padded rank, the padded rank a multiple of 16
  int blocks = (int)((numel4 + 255) / 256 < 1184 ? (numel4 + 255) / 256 : 1184);
  reduce_partials_kernel<<<dim3(blocks, 1, count), 256, 0, s>>>(tab, idx, numel4, ksplit);
  ++g_kernel_launches;
}

}  // namespace sc
