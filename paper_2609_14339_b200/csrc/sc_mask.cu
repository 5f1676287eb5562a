// In-graph activation masking from a shared pseudo-random function (Section 3.1; Algorithm 1 line 4,
// M_l = g(l, t, B, S, H)): h~ = h * M (optionally / keep). One pass over the activation, bf16 in, bf16 out.
//
// The mask is a pure function of (seed, layer, step, token, feature), so every pipeline stage can regenerate it
// and nothing is transmitted. Specification (the fp64 oracle implements the same on its own):
//   row key   k_t = low 32 bits of mix64(seed ^ ((layer * 2^40 + step) * G) ^ (t + 1) * 0xD1B54A32D192ED03),
//             mix64 = SplitMix64 finaliser, G = 0x9E3779B97F4A7C15
//   pair hash h   = lowbias32(k_t + (j / 2) * 0x9E3779B9)
//   element j keeps its value iff its 16 bits (low half of h for even j, high half for odd j) < round(keep * 65536)
//
// The weight gradient dY^T h~ that follows is a plain dense GEMM; the mask is NOT regenerated inside that GEMM's
// operand load on purpose: each activation tile is reused by every row tile of the output (112 times for a
// 14336-row weight), so hashing there would repeat the same work 112 times and make the GEMM issue-bound.
#include "sc_internal.cuh"

namespace {

__device__ __forceinline__ uint64_t mix64(uint64_t x) {
  x = (x ^ (x >> 30)) * 0xBF58476D1CE4E5B9ull;
  x = (x ^ (x >> 27)) * 0x94D049BB133111EBull;
  return x ^ (x >> 31);
}
__device__ __forceinline__ uint32_t lowbias32(uint32_t x) {
  x ^= x >> 16; x *= 0x21F0AAADu;
  x ^= x >> 15; x *= 0x735A2D97u;
  x ^= x >> 15;
  return x;
}

// One thread handles 8 consecutive features (16 bytes) of one token; features must be a multiple of 8.
__global__ void __launch_bounds__(256) prf_mask_kernel(const uint4* __restrict__ in, uint4* __restrict__ out,
                                                       int64_t tokens, int chunks_per_row, uint64_t base, uint32_t thr,
                                                       float scale, int do_scale) {
  const int64_t total = tokens * chunks_per_row;
  for (int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; e < total; e += (int64_t)gridDim.x * blockDim.x) {
    const int64_t t = e / chunks_per_row;
    const int c = (int)(e - t * chunks_per_row);
    const uint32_t key = (uint32_t)mix64(base ^ (((uint64_t)t + 1ull) * 0xD1B54A32D192ED03ull));
    uint4 v = __ldcs(in + e);
    uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const uint32_t h = lowbias32(key + (uint32_t)(c * 4 + i) * 0x9E3779B9u);
      const uint32_t m = ((h & 0xFFFFu) < thr ? 0x0000FFFFu : 0u) | ((h >> 16) < thr ? 0xFFFF0000u : 0u);
      uint32_t x = w[i] & m;
      if (do_scale) {
        __nv_bfloat162 b = *reinterpret_cast<__nv_bfloat162*>(&x);
        const float2 f = __bfloat1622float2(b);
        b = __floats2bfloat162_rn(f.x * scale, f.y * scale);
        x = *reinterpret_cast<uint32_t*>(&b);
      }
      w[i] = x;
    }
    __stcs(out + e, make_uint4(w[0], w[1], w[2], w[3]));
  }
}

// Exactly-K-per-token variant: one block per token. Composite keys (hash << 16 | j) are distinct, so the K smallest
// are found exactly by a radix select over their 48 bits, most significant byte first: in each of six rounds the
// block histograms the current byte of the keys that still match the prefix and keeps the bin the K-th key falls in.
__global__ void __launch_bounds__(256) prf_exact_k_kernel(const sc::bf16* __restrict__ in, sc::bf16* __restrict__ out,
                                                          int features, int K, uint64_t base, float scale,
                                                          int do_scale) {
  __shared__ unsigned hist[256];
  __shared__ unsigned long long prefix_s;
  __shared__ unsigned remaining_s;
  const int64_t t = blockIdx.x;
  const uint32_t key = (uint32_t)mix64(base ^ (((uint64_t)t + 1ull) * 0xD1B54A32D192ED03ull));
  unsigned long long prefix = 0;      // the leading bytes of the K-th smallest key found so far
  unsigned remaining = (unsigned)K;   // its rank among the keys that share this prefix (1-based)
  for (int round = 0; round < 6; ++round) {
    const int shift = 40 - 8 * round;
    hist[threadIdx.x] = 0;
    __syncthreads();
    for (int j = threadIdx.x; j < features; j += 256) {
      const unsigned long long c = ((unsigned long long)lowbias32(key + (uint32_t)j * 0x9E3779B9u) << 16) | (unsigned)j;
      if (round == 0 || (c >> (shift + 8)) == prefix) atomicAdd(&hist[(unsigned)(c >> shift) & 255u], 1u);
    }
    __syncthreads();
    if (threadIdx.x == 0) {
      unsigned acc = 0;
      int b = 0;
      for (; b < 256; ++b) {
        if (acc + hist[b] >= remaining) break;
        acc += hist[b];
      }
      prefix_s = (prefix << 8) | (unsigned)b;
      remaining_s = remaining - acc;
    }
    __syncthreads();
    prefix = prefix_s;
    remaining = remaining_s;
    __syncthreads();
  }
  // prefix is now the K-th smallest composite key: keep everything at or below it
  const sc::bf16 zero = __float2bfloat16_rn(0.f);
  for (int j = threadIdx.x; j < features; j += 256) {
    const unsigned long long c = ((unsigned long long)lowbias32(key + (uint32_t)j * 0x9E3779B9u) << 16) | (unsigned)j;
    const size_t o = (size_t)t * features + j;
    sc::bf16 v = in[o];
    if (c > prefix) v = zero;
    else if (do_scale) v = __float2bfloat16_rn(__bfloat162float(v) * scale);
    out[o] = v;
  }
}

}  // namespace

extern "C" sc_status sc_apply_prf_mask_exact_k(const void* X_dev, void* out_dev, int64_t tokens, int64_t features,
                                               float keep, uint64_t seed, uint32_t layer, uint64_t step, int rescale,
                                               void* stream) {
  if (!X_dev || !out_dev) return SC_ERR_INVALID_ARG;
  if (tokens <= 0 || features <= 0) return SC_ERR_SHAPE;
  if (features > 65536 || tokens > (1ll << 31) - 1) return SC_ERR_TOO_LARGE;
  if (!(keep > 0.f && keep <= 1.f)) return SC_ERR_INVALID_ARG;
  long K = lroundf(keep * (float)features);
  K = K < 1 ? 1 : (K > features ? (long)features : K);
  const uint64_t base = seed ^ ((((uint64_t)layer << 40) + step) * 0x9E3779B97F4A7C15ull);
  prf_exact_k_kernel<<<(unsigned)tokens, 256, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const sc::bf16*>(X_dev), static_cast<sc::bf16*>(out_dev), (int)features, (int)K, base,
      (float)features / (float)K, rescale != 0);
  ++sc::g_kernel_launches;
  return cudaGetLastError() == cudaSuccess ? SC_OK : SC_ERR_CUDA;
}

extern "C" sc_status sc_apply_prf_mask(const void* X_dev, void* out_dev, int64_t tokens, int64_t features, float keep,
                                       uint64_t seed, uint32_t layer, uint64_t step, int rescale, void* stream) {
  if (!X_dev || !out_dev) return SC_ERR_INVALID_ARG;
  if (tokens <= 0 || features <= 0 || (features % 8) != 0) return SC_ERR_SHAPE;
  if (!(keep > 0.f && keep <= 1.f)) return SC_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(X_dev) | reinterpret_cast<uintptr_t>(out_dev)) & 15u) return SC_ERR_ALIGNMENT;
  long thr = lroundf(keep * 65536.f);
  thr = thr < 1 ? 1 : (thr > 65536 ? 65536 : thr);
  const uint64_t base = seed ^ ((((uint64_t)layer << 40) + step) * 0x9E3779B97F4A7C15ull);
  const int chunks = (int)(features / 8);
  const int64_t total = tokens * chunks;
  int64_t blocks = (total + 255) / 256;
  if (blocks > 148 * 16) blocks = 148 * 16;
  prf_mask_kernel<<<(unsigned)blocks, 256, 0, static_cast<cudaStream_t>(stream)>>>(
      static_cast<const uint4*>(X_dev), static_cast<uint4*>(out_dev), tokens, chunks, base, (uint32_t)thr,
      65536.f / (float)thr, rescale != 0);
  ++sc::g_kernel_launches;
  return cudaGetLastError() == cudaSuccess ? SC_OK : SC_ERR_CUDA;
}
