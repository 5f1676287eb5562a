// sc_project_static: the projection X = U^T G V for one matrix, for callers that cannot provide scratch.
//
// Some users of this library have no way to hand over a workspace: an optimizer hook that runs after a
// framework's caching allocator has claimed all of HBM (a raw cudaMalloc then fails or fragments the pool),
// or a monitoring path that must never take the allocator's lock or trigger the device-wide synchronisation
// that cudaMalloc / cudaFree imply. For them the intermediate T = G V and the row-slice partials of U^T T live
// in one fixed, file-scope device array. The price: a hard size limit, and all calls share that one array.
#include <mutex>

#include "sc_internal.cuh"

namespace {

constexpr size_t kStaticScratchFloats = size_t(2) << 20;   // 8 MiB, resident on every device that loads the library
constexpr int kMaxDevices = 64;
constexpr int kSlices = 16;                                 // row slices of U^T T (fixed-order two-stage sum)

static __device__ __align__(256) float g_static_scratch[kStaticScratchFloats];

// Device address of g_static_scratch per device. In host code the array's name is only a handle for
// cudaGetSymbolAddress; it is not something a kernel may be given.
float* g_scratch_addr[kMaxDevices] = {};
std::mutex g_scratch_mutex;

constexpr int TM = 64, TN = 64, TK = 16;

// C[z] = op(A) B over the K range of slice z. A is M x K (or K x M when transA), fp32 or bf16; B is K x N fp32.
__global__ void __launch_bounds__(256)
static_gemm_kernel(const void* __restrict__ Av, int a_bf16, int transA, const float* __restrict__ B,
                   float* __restrict__ C, int M, int N, int K, int lda, int ldb, int ldc, int k_per_slice) {
  __shared__ float As[TK][TM + 1];
  __shared__ float Bs[TK][TN + 1];
  const float* A = static_cast<const float*>(Av);
  const __nv_bfloat16* Ab = static_cast<const __nv_bfloat16*>(Av);
  const int k_lo = blockIdx.z * k_per_slice, k_hi = min(K, k_lo + k_per_slice);
  float* Cz = C + (size_t)blockIdx.z * M * ldc;
  const int row0 = blockIdx.y * TM, col0 = blockIdx.x * TN;
  const int tid = threadIdx.x, ty = tid >> 4, tx = tid & 15;
  float acc[4][4] = {};
  for (int k0 = k_lo; k0 < k_hi; k0 += TK) {
    for (int e = tid; e < TM * TK; e += 256) {
      int r, k;
      if (!transA) { r = e / TK; k = e % TK; } else { k = e / TM; r = e % TM; }
      const int gr = row0 + r, gk = k0 + k;
      float v = 0.f;
      if (gr < M && gk < k_hi) {
        const size_t off = transA ? (size_t)gk * lda + gr : (size_t)gr * lda + gk;
        v = a_bf16 ? __bfloat162float(Ab[off]) : A[off];
      }
      As[k][r] = v;
    }
    for (int e = tid; e < TN * TK; e += 256) {
      const int k = e / TN, c = e % TN;
      const int gc = col0 + c, gk = k0 + k;
      Bs[k][c] = (gc < N && gk < k_hi) ? B[(size_t)gk * ldb + gc] : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int k = 0; k < TK; ++k) {
      float av[4], bv[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) av[i] = As[k][ty * 4 + i];
#pragma unroll
      for (int j = 0; j < 4; ++j) bv[j] = Bs[k][tx * 4 + j];
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(av[i], bv[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int gr = row0 + ty * 4 + i, gc = col0 + tx * 4 + j;
      if (gr < M && gc < N) Cz[(size_t)gr * ldc + gc] = acc[i][j];
    }
}

__global__ void static_sum_kernel(const float* __restrict__ part, float* __restrict__ out, int numel, int slices) {
  const int e = blockIdx.x * blockDim.x + threadIdx.x;
  if (e >= numel) return;
  float t = 0.f;
  for (int s = 0; s < slices; ++s) t += part[(size_t)s * numel + e];
  out[e] = t;
}

}  // namespace

extern "C" sc_status sc_project_static(const void* G_dev, int grad_dtype, const void* U_dev, const void* V_dev,
                                       int64_t rows, int64_t cols, int rank, void* X_dev, void* stream) {
  if (!G_dev || !U_dev || !V_dev || !X_dev) return SC_ERR_INVALID_ARG;
  if (grad_dtype != SC_DTYPE_BF16 && grad_dtype != SC_DTYPE_FP32) return SC_ERR_DTYPE;
  if (rows <= 0 || cols <= 0 || rank <= 0 || rank > rows || rank > cols) return SC_ERR_SHAPE;
  if (rank > sc::kMaxRank || rows > (1 << 24) || cols > (1 << 24)) return SC_ERR_TOO_LARGE;
  const size_t need = (size_t)rows * rank + (size_t)kSlices * rank * rank;
  if (need > kStaticScratchFloats) return SC_ERR_TOO_LARGE;   // rows*rank + 16*rank^2 floats must fit in 8 MiB

  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess) return SC_ERR_CUDA;
  if (dev < 0 || dev >= kMaxDevices) return SC_ERR_INVALID_ARG;
  float* scratch = nullptr;
  {
    // First call on this device: look the array's device address up (with this device current) and keep it.
    std::lock_guard<std::mutex> lock(g_scratch_mutex);
    if (!g_scratch_addr[dev]) {
      void* p = nullptr;
      if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) return SC_ERR_CUDA;
      g_scratch_addr[dev] = static_cast<float*>(p);
    }
    scratch = g_scratch_addr[dev];
  }
  cudaStream_t s = static_cast<cudaStream_t>(stream);
  const int m = (int)rows, n = (int)cols, r = rank;
  float* T = scratch;                         // rows x rank, fully written below before it is read
  float* part = scratch + (size_t)rows * r;   // kSlices x rank x rank, fully written below before it is read
  // T = G V
  static_gemm_kernel<<<dim3((r + TN - 1) / TN, (m + TM - 1) / TM, 1), 256, 0, s>>>(
      G_dev, grad_dtype == SC_DTYPE_BF16, 0, static_cast<const float*>(V_dev), T, m, r, n, n, r, r, n);
  ++sc::g_kernel_launches;
  // part[z] = U[rows of slice z]^T T[rows of slice z]; X = sum_z part[z]
  const int per = ((m + kSlices - 1) / kSlices + TK - 1) / TK * TK;
  const int slices = (m + per - 1) / per;
  static_gemm_kernel<<<dim3((r + TN - 1) / TN, (r + TM - 1) / TM, slices), 256, 0, s>>>(
      U_dev, 0, 1, T, part, r, r, m, r, r, r, per);
  ++sc::g_kernel_launches;
  static_sum_kernel<<<(r * r + 255) / 256, 256, 0, s>>>(part, static_cast<float*>(X_dev), r * r, slices);
  ++sc::g_kernel_launches;
  return cudaGetLastError() == cudaSuccess ? SC_OK : SC_ERR_CUDA;
}
