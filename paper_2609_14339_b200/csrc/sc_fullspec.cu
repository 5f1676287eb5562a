// Full-spectrum soft filter: the main-text form of Section 3.2 ("Filtering d_i = s_i / (s_i + tau_p)"), in which the soft
// weights apply to ALL singular directions of the anchor momentum and there is no rank cut. With M = U S V^T:
//
//     P_U = U diag(d) U^T = A (A + tau I)^-1,  A = (M M^T)^(1/2)       P_V = V diag(d) V^T = B (B + tau I)^-1,  B = (M^T M)^(1/2)
//     G_filt = P_U G P_V          G_proj = alpha g + (1 - alpha) G_filt          (Eq. 3)
//
// On anchor arrival (refresh) the two soft projectors are built without an eigen-decomposition, by matrix products only:
// a coupled Newton-Schulz iteration for the square root of the Gram matrix, then a Newton-Schulz iteration for
// (S + tau I)^-1, then P = I - tau (S + tau I)^-1. These products run in fp64 on the CUDA cores: the square root turns a
// perturbation eps of the Gram matrix into sqrt(eps) on the directions near its null space (d is not Lipschitz in the
// eigenvalue at 0), so fp32 products (eps ~ 1e-7) would already leave weights of order 1e-3..1e-2 on directions that
// should get none. Every optimizer step then costs two dense contractions on the tensor cores,
//     T1^T = G^T P_U   (n x m)        F = (1 - alpha) scale * T1 P_V   (m x n)
// with the fp32 factors carried as bf16 hi + lo pairs (split-precision products accumulated in TMEM), followed by one
// elementwise AdamW pass.
#include <math.h>

#include <algorithm>
#include <utility>

#include "sc_internal.cuh"

namespace sc {
namespace {

inline size_t align256(size_t x) { return (x + 255) / 256 * 256; }

// ------------------------------------------------------------------------------------------ fp64 products
// C (M x N, fp64) = alpha * op(A) op(B) + diag * I.  op(A) is M x K: A[i * lda + k], or A[k * lda + i] when TA.
// op(B) is K x N: B[k * ldb + j], or B[j * ldb + k] when TB.  Inputs fp32 (the anchor momentum) or fp64.
// 128 x 128 tile per block of 256 threads, 8 x 8 per thread as pairs of rows and columns interleaved across the tile (rows
// 2 ty + {0, 1} + 32 i, columns 2 tx + {0, 1} + 32 j), so that every shared-memory read is a 16-byte one that the lanes
// of a warp either share or read side by side. K advances 16 per stage; the next stage's global loads are in flight
// while the current one multiplies, and land in the other half of the double buffer.
constexpr int DBM = 128, DBN = 128, DBK = 16;
constexpr int DPA = DBM + 2, DPB = DBN + 2;          // row pitch in doubles (even: 16-byte rows)
constexpr size_t kDgemmSmem = (size_t)2 * DBK * (DPA + DPB) * sizeof(double);

template <typename TIn, bool TA, bool TB>
__global__ void __launch_bounds__(256)
dgemm_kernel(const TIn* __restrict__ A, const TIn* __restrict__ B, double* __restrict__ C, int M, int N, int K, int lda,
             int ldb, int ldc, double alpha, double diag, int sym) {
  // sym: the product is symmetric (a Gram matrix, or two commuting symmetric factors): only the tiles on and above the
  // diagonal are computed and each is also written transposed
  if (sym && blockIdx.x < blockIdx.y) return;
  extern __shared__ __align__(16) double dsm[];
  double* As = dsm;                                  // [2][DBK][DPA]
  double* Bs = dsm + 2 * DBK * DPA;                  // [2][DBK][DPB]
  const int row0 = blockIdx.y * DBM, col0 = blockIdx.x * DBN;
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  constexpr int NA = DBM * DBK / 256, NB = DBN * DBK / 256;   // 8 and 8 elements per thread and stage
  double ra[NA], rb[NB];
  auto fetch = [&](int k0) {
#pragma unroll
    for (int u = 0; u < NA; ++u) {
      const int e = tid + 256 * u;
      int r, k;
      if (!TA) { r = e / DBK; k = e % DBK; } else { k = e / DBM; r = e % DBM; }
      const int gr = row0 + r, gk = k0 + k;
      ra[u] = (gr < M && gk < K) ? (double)(TA ? A[(size_t)gk * lda + gr] : A[(size_t)gr * lda + gk]) : 0.0;
    }
#pragma unroll
    for (int u = 0; u < NB; ++u) {
      const int e = tid + 256 * u;
      int c, k;
      if (!TB) { k = e / DBN; c = e % DBN; } else { c = e / DBK; k = e % DBK; }
      const int gc = col0 + c, gk = k0 + k;
      rb[u] = (gc < N && gk < K) ? (double)(TB ? B[(size_t)gc * ldb + gk] : B[(size_t)gk * ldb + gc]) : 0.0;
    }
  };
  auto stash = [&](int buf) {
    double* as = As + buf * DBK * DPA;
    double* bs = Bs + buf * DBK * DPB;
#pragma unroll
    for (int u = 0; u < NA; ++u) {
      const int e = tid + 256 * u;
      int r, k;
      if (!TA) { r = e / DBK; k = e % DBK; } else { k = e / DBM; r = e % DBM; }
      as[k * DPA + r] = ra[u];
    }
#pragma unroll
    for (int u = 0; u < NB; ++u) {
      const int e = tid + 256 * u;
      int c, k;
      if (!TB) { k = e / DBN; c = e % DBN; } else { c = e / DBK; k = e % DBK; }
      bs[k * DPB + c] = rb[u];
    }
  };
  double acc[8][8];
#pragma unroll
  for (int i = 0; i < 8; ++i)
#pragma unroll
    for (int j = 0; j < 8; ++j) acc[i][j] = 0.0;
  fetch(0);
  stash(0);
  __syncthreads();
  const int nk = (K + DBK - 1) / DBK;
  for (int t = 0; t < nk; ++t) {
    const int buf = t & 1;
    if (t + 1 < nk) fetch((t + 1) * DBK);
    const double* as = As + buf * DBK * DPA + 2 * ty;
    const double* bs = Bs + buf * DBK * DPB + 2 * tx;
#pragma unroll
    for (int k = 0; k < DBK; ++k) {
      double av[8], bv[8];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const double2 a2 = *reinterpret_cast<const double2*>(as + k * DPA + 32 * i);
        const double2 b2 = *reinterpret_cast<const double2*>(bs + k * DPB + 32 * i);
        av[2 * i] = a2.x; av[2 * i + 1] = a2.y;
        bv[2 * i] = b2.x; bv[2 * i + 1] = b2.y;
      }
#pragma unroll
      for (int i = 0; i < 8; ++i)
#pragma unroll
        for (int j = 0; j < 8; ++j) acc[i][j] = fma(av[i], bv[j], acc[i][j]);
    }
    if (t + 1 < nk) stash(buf ^ 1);      // the other buffer: nobody reads it during this stage
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 8; ++i) {
    const int gr = row0 + 2 * ty + 32 * (i >> 1) + (i & 1);
    if (gr >= M) continue;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
      const int gc = col0 + 2 * tx + 32 * (j >> 1) + (j & 1);
      if (gc >= N) continue;
      const double v = alpha * acc[i][j] + (gr == gc ? diag : 0.0);
      C[(size_t)gr * ldc + gc] = v;
      if (sym && blockIdx.x != blockIdx.y) C[(size_t)gc * ldc + gr] = v;
    }
  }
}

template <typename TIn, bool TA, bool TB>
void dgemm(const TIn* A, const TIn* B, double* C, int M, int N, int K, int lda, int ldb, int ldc, double alpha,
           double diag, cudaStream_t s, bool sym = false) {
  static const cudaError_t attr = cudaFuncSetAttribute(dgemm_kernel<TIn, TA, TB>,
                                                        cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kDgemmSmem);
  (void)attr;
  dim3 grid((N + DBN - 1) / DBN, (M + DBM - 1) / DBM);
  dgemm_kernel<TIn, TA, TB><<<grid, 256, kDgemmSmem, s>>>(A, B, C, M, N, K, lda, ldb, ldc, alpha, diag,
                                                          sym && M == N ? 1 : 0);
  ++g_kernel_launches;
}

// Frobenius norm of a k x k fp64 matrix into *out: per-block partial sums, the last step by one block in a fixed order.
constexpr int kNormBlocks = 256;
__global__ void __launch_bounds__(256) sqsum_part_kernel(const double* __restrict__ X, int64_t numel, double* part) {
  __shared__ double sh[256];
  double s = 0.0;
  for (int64_t e = (int64_t)blockIdx.x * 256 + threadIdx.x; e < numel; e += (int64_t)gridDim.x * 256) s = fma(X[e], X[e], s);
  sh[threadIdx.x] = s;
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if ((int)threadIdx.x < o) sh[threadIdx.x] += sh[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) part[blockIdx.x] = sh[0];
}
__global__ void sqsum_final_kernel(const double* part, int n, double* out) {
  double s = 0.0;
  for (int i = 0; i < n; ++i) s += part[i];
  *out = sqrt(s);
}

// Y = A / ||A||_F, Z = I   (an all-zero A gives Y = 0)
__global__ void __launch_bounds__(256) ns_init_kernel(const double* __restrict__ A, const double* __restrict__ normA,
                                                      double* __restrict__ Y, double* __restrict__ Z, int k) {
  const double c = *normA, inv = c > 0.0 ? 1.0 / c : 0.0;
  const int64_t numel = (int64_t)k * k;
  for (int64_t e = (int64_t)blockIdx.x * 256 + threadIdx.x; e < numel; e += (int64_t)gridDim.x * 256) {
    Y[e] = A[e] * inv;
    Z[e] = (e / k == e % k) ? 1.0 : 0.0;
  }
}
// After the square root: B = sqrt(c) Y + tau I (in place on Y), X = I / (sqrt(c) ||Y||_F + tau)
__global__ void __launch_bounds__(256) inv_init_kernel(double* __restrict__ YB, double* __restrict__ X,
                                                       const double* __restrict__ normA, const double* __restrict__ normY,
                                                       double tau, int k) {
  const double rc = sqrt(*normA), x0 = 1.0 / (rc * (*normY) + tau);
  const int64_t numel = (int64_t)k * k;
  for (int64_t e = (int64_t)blockIdx.x * 256 + threadIdx.x; e < numel; e += (int64_t)gridDim.x * 256) {
    const bool dg = (e / k == e % k);
    YB[e] = rc * YB[e] + (dg ? tau : 0.0);
    X[e] = dg ? x0 : 0.0;
  }
}
// P = I - tau X as a bf16 hi/lo pair (the symmetric part, so that P^T = P holds exactly for the step's A^T B products)
__global__ void __launch_bounds__(256) soft_projector_out_kernel(const double* __restrict__ X, double tau, int k,
                                                                 bf16* __restrict__ hi, bf16* __restrict__ lo) {
  const int64_t numel = (int64_t)k * k;
  for (int64_t e = (int64_t)blockIdx.x * 256 + threadIdx.x; e < numel; e += (int64_t)gridDim.x * 256) {
    const int i = (int)(e / k), j = (int)(e % k);
    const double x = 0.5 * (X[e] + X[(size_t)j * k + i]);
    const float p = (float)((i == j ? 1.0 : 0.0) - tau * x);
    const bf16 h = __float2bfloat16_rn(p);
    hi[e] = h;
    lo[e] = __float2bfloat16_rn(p - __bfloat162float(h));
  }
}

// Elementwise AdamW on G_proj = clip * (alpha_s * G + F), F = the filtered part (already carrying (1 - alpha) * scale).
__global__ void __launch_bounds__(256)
fs_adamw_kernel(const bf16* __restrict__ G, const float* __restrict__ F, float* __restrict__ W, float* __restrict__ m1,
                float* __restrict__ m2, bf16* __restrict__ Wb, float* __restrict__ gdbg, int64_t numel, StepScalars s,
                const float* __restrict__ clip_ptr) {
  const float clip = *clip_ptr;
  for (int64_t e = ((int64_t)blockIdx.x * 256 + threadIdx.x) * 4; e < numel; e += (int64_t)gridDim.x * 1024) {
    const uint2 graw = *reinterpret_cast<const uint2*>(G + e);
    const __nv_bfloat162 g01 = *reinterpret_cast<const __nv_bfloat162*>(&graw.x);
    const __nv_bfloat162 g23 = *reinterpret_cast<const __nv_bfloat162*>(&graw.y);
    const float gr[4] = {__low2float(g01), __high2float(g01), __low2float(g23), __high2float(g23)};
    const float4 f4 = *reinterpret_cast<const float4*>(F + e);
    float4 w4 = *reinterpret_cast<const float4*>(W + e), a4 = *reinterpret_cast<const float4*>(m1 + e),
           b4 = *reinterpret_cast<const float4*>(m2 + e);
    const float fr[4] = {f4.x, f4.y, f4.z, f4.w};
    float* w = &w4.x; float* a = &a4.x; float* b = &b4.x;
    float gp[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float g = clip * fmaf(s.alpha_s, gr[j], fr[j]);
      const float mo = fmaf(s.beta1, a[j], s.one_m_beta1 * g);
      const float vo = fmaf(s.beta2, b[j], s.one_m_beta2 * g * g);
      const float den = fmaf(sqrtf(vo), s.inv_sqrt_bc2, s.eps);
      w[j] = fmaf(-s.step_size, mo / den, w[j] * s.decay);
      a[j] = mo; b[j] = vo; gp[j] = g;
    }
    *reinterpret_cast<float4*>(W + e) = w4;
    *reinterpret_cast<float4*>(m1 + e) = a4;
    *reinterpret_cast<float4*>(m2 + e) = b4;
    if (Wb) {
      const __nv_bfloat162 o0 = __floats2bfloat162_rn(w[0], w[1]), o1 = __floats2bfloat162_rn(w[2], w[3]);
      *reinterpret_cast<uint2*>(Wb + e) = make_uint2(*reinterpret_cast<const uint32_t*>(&o0), *reinterpret_cast<const uint32_t*>(&o1));
    }
    if (gdbg) *reinterpret_cast<float4*>(gdbg + e) = make_float4(gp[0], gp[1], gp[2], gp[3]);
  }
}

int grid_for(int64_t numel) {
  const int64_t b = (numel + 255) / 256;
  return (int)(b < 148 * 8 ? b : 148 * 8);
}

}  // namespace

// ------------------------------------------------------------------------------------------ layout
// Per matrix (persistent): P_U (m x m) and P_V (n x n) as bf16 hi/lo pairs. Shared by all matrices (one matrix is
// processed at a time): five k x k fp64 work matrices (k = the largest dimension of any matrix), the norm partials,
// T1^T (n x m, bf16 hi/lo) and F (m x n fp32).
size_t fs_layout(sc_plan* p, char* base) {
  size_t off = 0;
  auto take = [&](size_t bytes) { char* q = base ? base + off : nullptr; off = align256(off + bytes); return q; };
  int64_t kmax = 0, emax = 0;
  for (const auto& sh : p->shapes) {
    kmax = std::max(kmax, std::max(sh.rows, sh.cols));
    emax = std::max(emax, sh.rows * sh.cols);
  }
  if (base) p->fs.mats.resize(p->n_mats);
  for (int i = 0; i < p->n_mats; ++i) {
    const size_t m = (size_t)p->shapes[i].rows, n = (size_t)p->shapes[i].cols;
    bf16* a = reinterpret_cast<bf16*>(take(m * m * 2)); bf16* b = reinterpret_cast<bf16*>(take(m * m * 2));
    bf16* c = reinterpret_cast<bf16*>(take(n * n * 2)); bf16* d = reinterpret_cast<bf16*>(take(n * n * 2));
    if (base) p->fs.mats[i] = FsMat{a, b, c, d};
  }
  double* w[5];
  for (int j = 0; j < 5; ++j) w[j] = reinterpret_cast<double*>(take((size_t)kmax * kmax * sizeof(double)));
  double* part = reinterpret_cast<double*>(take((kNormBlocks + 8) * sizeof(double)));
  bf16* t1hi = reinterpret_cast<bf16*>(take((size_t)emax * 2)); bf16* t1lo = reinterpret_cast<bf16*>(take((size_t)emax * 2));
  float* F = reinterpret_cast<float*>(take((size_t)emax * 4));
  if (base) {
    for (int j = 0; j < 5; ++j) p->fs.work[j] = w[j];
    p->fs.part = part; p->fs.scal = part + kNormBlocks; p->fs.T1hi = t1hi; p->fs.T1lo = t1lo; p->fs.F = F;
  }
  return off;
}

// One soft projector: P = f(Gram) with Gram = M M^T (left = true, k = m) or M^T M (k = n), written as a bf16 hi/lo pair.
static void fs_build_projector(sc_plan* p, const float* M, int m, int n, bool left, bf16* hi, bf16* lo) {
  cudaStream_t s = p->stream;
  const int k = left ? m : n;
  double* A = p->fs.work[0]; double* Y = p->fs.work[1]; double* Z = p->fs.work[2]; double* T = p->fs.work[3];
  double* Y2 = p->fs.work[4];
  double* normA = p->fs.scal; double* normY = p->fs.scal + 1;
  const int64_t numel = (int64_t)k * k;
  const int g = grid_for(numel);
  if (left) dgemm<float, false, true>(M, M, A, k, k, n, n, n, k, 1.0, 0.0, s, true);      // M M^T
  else dgemm<float, true, false>(M, M, A, k, k, m, n, n, k, 1.0, 0.0, s, true);           // M^T M
  sqsum_part_kernel<<<kNormBlocks, 256, 0, s>>>(A, numel, p->fs.part);
  sqsum_final_kernel<<<1, 1, 0, s>>>(p->fs.part, kNormBlocks, normA);
  ns_init_kernel<<<g, 256, 0, s>>>(A, normA, Y, Z, k);
  g_kernel_launches += 3;
  // square root: T = (3 I - Z Y) / 2 ; Y <- Y T ; Z <- T Z.  A (no longer needed) is the second ping-pong buffer for Z.
  // Y, Z and T are polynomials in the same symmetric matrix: they commute, so every product here is symmetric. Only the
  // upper tiles of Z Y are computed (and of both products of the inverse iteration below). Y T and T Z are computed in
  // full: a Gram matrix with a null space (more columns than rows) makes Z grow like 1.5^k there, and writing the upper
  // tiles of Y T into the lower half mixes Y T with T Y, which feeds their rounding-level commutator back through that
  // growth (measured: NaN after 24 iterations).
  double* Z2 = A;
  for (int it = 0; it < p->hp.fs_sqrt_iters; ++it) {
    dgemm<double, false, false>(Z, Y, T, k, k, k, k, k, k, -0.5, 1.5, s, true);
    dgemm<double, false, false>(Y, T, Y2, k, k, k, k, k, k, 1.0, 0.0, s);
    dgemm<double, false, false>(T, Z, Z2, k, k, k, k, k, k, 1.0, 0.0, s);
    std::swap(Y, Y2); std::swap(Z, Z2);
  }
  sqsum_part_kernel<<<kNormBlocks, 256, 0, s>>>(Y, numel, p->fs.part);
  sqsum_final_kernel<<<1, 1, 0, s>>>(p->fs.part, kNormBlocks, normY);
  // inverse of B = S + tau I: X <- X (2 I - B X).  B overwrites Y; X, R and the ping-pong buffer reuse Z, T, Z2.
  double* B = Y; double* X = Z; double* R = T; double* X2 = Z2;
  inv_init_kernel<<<g, 256, 0, s>>>(B, X, normA, normY, (double)p->hp.tau_p, k);
  g_kernel_launches += 3;
  for (int it = 0; it < p->hp.fs_inv_iters; ++it) {
    dgemm<double, false, false>(B, X, R, k, k, k, k, k, k, -1.0, 2.0, s, true);
    dgemm<double, false, false>(X, R, X2, k, k, k, k, k, k, 1.0, 0.0, s, true);
    std::swap(X, X2);
  }
  soft_projector_out_kernel<<<g, 256, 0, s>>>(X, (double)p->hp.tau_p, k, hi, lo);
  ++g_kernel_launches;
}

sc_status fs_refresh(sc_plan* p, int mat) {
  const MatDev& md = p->host_tab[mat];
  const FsMat& f = p->fs.mats[mat];
  fs_build_projector(p, md.Manc, md.m, md.n, true, f.PUhi, f.PUlo);
  fs_build_projector(p, md.Manc, md.m, md.n, false, f.PVhi, f.PVlo);
  return cuda_ok(cudaGetLastError());
}

// F = filt_scale * P_U G P_V for one matrix (zero before the first anchor has arrived: G_proj = alpha g then).
sc_status fs_step_filter(sc_plan* p, int mat, float filt_scale) {
  const MatDev& md = p->host_tab[mat];
  const FsMat& f = p->fs.mats[mat];
  cudaStream_t s = p->stream;
  const int64_t m = md.m, n = md.n;
  sc_status st;
  if (p->has_basis[mat]) {
    // T1^T (n x m) = G^T P_U: contraction over the m rows of G; P_U as hi + lo
    const void* a1[3] = {md.G, md.G, md.G};
    const void* b1[3] = {f.PUhi, f.PUlo, f.PUhi};
    if ((st = launch_tn_gemm(a1, b1, 2, m, n, m, p->fs.T1hi, p->fs.T1lo, 2, 1.f, 0.f, p->status_dev, s)) != SC_OK) return st;
    // F (m x n) = filt_scale * T1 P_V: contraction over n; both factors as hi + lo (hi hi + lo hi + hi lo)
    const void* a2[3] = {p->fs.T1hi, p->fs.T1lo, p->fs.T1hi};
    const void* b2[3] = {f.PVhi, f.PVhi, f.PVlo};
    if ((st = launch_tn_gemm(a2, b2, 3, n, m, n, p->fs.F, nullptr, 1, filt_scale, 0.f, p->status_dev, s)) != SC_OK) return st;
  } else {
    if (cudaMemsetAsync(p->fs.F, 0, (size_t)(m * n) * sizeof(float), s) != cudaSuccess) return SC_ERR_CUDA;
  }
  return SC_OK;
}

// Eq. 3 and AdamW, elementwise, on the F that fs_step_filter left for this matrix.
sc_status fs_step_update(sc_plan* p, int mat, const StepScalars& sc) {
  const MatDev& md = p->host_tab[mat];
  cudaStream_t s = p->stream;
  const int64_t m = md.m, n = md.n;
  fs_adamw_kernel<<<grid_for((m * n + 3) / 4), 256, 0, s>>>(static_cast<const bf16*>(md.G), p->fs.F, md.W, md.m1, md.m2, md.Wb,
                                                            md.gproj_dbg, m * n, sc, p->clip_dev);
  ++g_kernel_launches;
  return cuda_ok(cudaGetLastError());
}

}  // namespace sc
