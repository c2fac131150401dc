// Tokens whose keys are strongly anti-correlated with the rest (the augmented BalanceKV of
// Section 4.3, which keeps such tokens exactly and runs the standard procedure on the others).
// The paper names neither the measure nor a threshold; here a token of an appended block is
// preserved when the cosine between its key and the mean key of the block is at most tau:
//   <k_j, kbar> <= tau ||k_j|| ||kbar||,   kbar = (1/n) sum_j k_j   (per stream and block).
// Three kernels: column sums of K over chunks of 256 rows, their fixed-order total (the mean and its
// squared norm), and the class of every row (0 = preserved, 1 = the rest) as the routing pass's
// forced slot.  Everything is fp32 with a fixed summation order, so a run is reproducible.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "common.cuh"

namespace bkv {

namespace {

constexpr int kSumRows = 256;       // rows per CTA of the column sums
constexpr int kRowsPerBlock = 64;

__device__ inline float key_at(const void* K, size_t idx, bool bf16) {
  return bf16 ? __bfloat162float(static_cast<const __nv_bfloat16*>(K)[idx]) : static_cast<const float*>(K)[idx];
}

// grid (chunks of kSumRows rows, streams), d threads: thread e sums column e over the chunk's rows.
__global__ void anticorr_colsum_kernel(const void* __restrict__ K, int n, int d, int n_chunks, int bf16, float* __restrict__ partial) {
  const int sl = blockIdx.y, chunk = blockIdx.x, e = threadIdx.x;
  const int r0 = chunk * kSumRows, r1 = min(n, r0 + kSumRows);
  float s = 0.f;
  for (int r = r0; r < r1; ++r) s += key_at(K, ((size_t)sl * n + r) * d + e, bf16 != 0);
  partial[((size_t)sl * n_chunks + chunk) * d + e] = s;
}

// grid (streams), d threads (a multiple of 32): mean[sl][e], and mean[sl][d] = ||mean||^2.
__global__ void anticorr_mean_kernel(const float* __restrict__ partial, int n, int d, int n_chunks, float* __restrict__ mean) {
  __shared__ float wsum[4];
  const int sl = blockIdx.x, e = threadIdx.x;
  float s = 0.f;
  for (int c = 0; c < n_chunks; ++c) s += partial[((size_t)sl * n_chunks + c) * d + e];
  const float m = s / (float)n;
  mean[(size_t)sl * (d + 1) + e] = m;
  const float w = warp_sum(m * m);
  if ((e & 31) == 0) wsum[e >> 5] = w;
  __syncthreads();
  if (e == 0) {
    float t = 0.f;
    for (int i = 0; i < d / 32; ++i) t += wsum[i];
    mean[(size_t)sl * (d + 1) + d] = t;
  }
}

// grid (row groups, streams), 256 threads; `chunks` lanes (16-byte pieces of a row) share a row.
template <bool kBf16>
__global__ void __launch_bounds__(256)
anticorr_class_kernel(const void* __restrict__ K, int n, int d, int chunks, float tau, const float* __restrict__ mean,
                      int8_t* __restrict__ cls) {
  const int sl = blockIdx.y;
  const int rows_per_pass = blockDim.x / chunks;
  const int row_in = threadIdx.x / chunks, piece = threadIdx.x % chunks;
  const float* mu = mean + (size_t)sl * (d + 1);
  const float m2 = mu[d];
  const int per = kBf16 ? 8 : 4;                 // elements of a 16-byte piece
  const int row_end = min(n, (int)(blockIdx.x + 1) * kRowsPerBlock);
  for (int r0 = blockIdx.x * kRowsPerBlock; r0 < row_end; r0 += rows_per_pass) {
    const int r = r0 + row_in;
    float dot = 0.f, k2 = 0.f;
    if (r < row_end) {
      float x[8];
      const char* row = static_cast<const char*>(K) + ((size_t)sl * n + r) * d * (kBf16 ? 2 : 4);
      if constexpr (kBf16) load8<true>(row, piece * 8, x);
      else {
        const float4 v = *reinterpret_cast<const float4*>(reinterpret_cast<const float*>(row) + piece * 4);
        x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
      }
      for (int i = 0; i < per; ++i) {
        dot = fmaf(x[i], mu[piece * per + i], dot);
        k2 = fmaf(x[i], x[i], k2);
      }
    }
    for (int o = chunks / 2; o > 0; o >>= 1) {
      dot += __shfl_xor_sync(0xffffffffu, dot, o);
      k2 += __shfl_xor_sync(0xffffffffu, k2, o);
    }
    if (r < row_end && piece == 0) {
      const float scale = sqrtf(k2 * m2);
      const bool keep = scale > 0.f ? dot <= tau * scale : 0.f <= tau;     // a zero key or mean: cosine 0
      cls[(size_t)sl * n + r] = keep ? 0 : 1;
    }
  }
}

}  // namespace

size_t anticorr_scratch_floats(int n_sl, int n, int d) {
  return (size_t)n_sl * ((size_t)((n + kSumRows - 1) / kSumRows) * d + d + 1);
}

// cls[n_sl][n] = 0 for the rows of K ([n_sl][n][d]) to preserve, 1 for the rest.  scratch:
// anticorr_scratch_floats(n_sl, n, d) floats.
cudaError_t launch_anticorr_classes(const Geom& G, const void* K, int n_sl, int n, float tau, float* scratch, int8_t* cls,
                                    cudaStream_t st) {
  const int d = G.d, n_chunks = (n + kSumRows - 1) / kSumRows;
  float* partial = scratch;
  float* mean = scratch + (size_t)n_sl * n_chunks * d;
  anticorr_colsum_kernel<<<dim3(n_chunks, n_sl), d, 0, st>>>(K, n, d, n_chunks, G.is_bf16, partial);
  anticorr_mean_kernel<<<n_sl, d, 0, st>>>(partial, n, d, n_chunks, mean);
  const int chunks = d * (G.is_bf16 ? 2 : 4) / 16;
  dim3 grid((n + kRowsPerBlock - 1) / kRowsPerBlock, n_sl);
  if (G.is_bf16) anticorr_class_kernel<true><<<grid, 256, 0, st>>>(K, n, d, chunks, tau, mean, cls);
  else anticorr_class_kernel<false><<<grid, 256, 0, st>>>(K, n, d, chunks, tau, mean, cls);
  return cudaGetLastError();
}

}  // namespace bkv
