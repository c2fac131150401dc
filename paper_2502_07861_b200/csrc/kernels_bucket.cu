// Value-norm buckets of BalanceKV (Algorithm 1, the bucketing step and the erasure of small-norm
// buckets): token j goes to the MergeAndReduce instance of the index i with 2^(i-1) < ||v_j|| <= 2^i,
// instances whose bucket satisfies 2^i <= rho * v_max are erased.  Three kernels: squared value
// norms + running maximum, a stable partition of the block's tokens by bucket (one CTA per
// stream), and the copy of every kept row into the level-0 set of its bucket's instance.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "common.cuh"

namespace bkv {

namespace {

constexpr int kScanThreads = 1024;
constexpr int kRowsPerBlock = 64;

template <bool kBf16>
__device__ inline float sumsq_piece(const uint4& v) {
  float s = 0.f;
  if constexpr (kBf16) {
    const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 f = __bfloat1622float2(h[i]);
      s = fmaf(f.x, f.x, s);
      s = fmaf(f.y, f.y, s);
    }
  } else {
    const float* f = reinterpret_cast<const float*>(&v);
#pragma unroll
    for (int i = 0; i < 4; ++i) s = fmaf(f[i], f[i], s);
  }
  return s;
}

// ||v_j||^2 of every row of the block (chunks = 16-byte pieces of a row: 8, 16 or 32 lanes share
// a row) and the maximum per stream.  grid (row groups, streams), 256 threads.
template <bool kBf16>
__global__ void __launch_bounds__(256)
bucket_norms_kernel(const void* __restrict__ V, int n, int chunks, float* __restrict__ ns, unsigned* __restrict__ vmax2_bits) {
  const int sl = blockIdx.y;
  const int rows_per_pass = blockDim.x / chunks;
  const int row_in = threadIdx.x / chunks, piece = threadIdx.x % chunks;
  const uint4* src = reinterpret_cast<const uint4*>(V) + (size_t)sl * n * chunks;
  float mx = 0.f;
  const int row_end = min(n, (int)(blockIdx.x + 1) * kRowsPerBlock);
  for (int r0 = blockIdx.x * kRowsPerBlock; r0 < row_end; r0 += rows_per_pass) {
    const int r = r0 + row_in;
    float s = 0.f;
    if (r < row_end) s = sumsq_piece<kBf16>(src[(size_t)r * chunks + piece]);
    for (int o = chunks / 2; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (r < row_end && piece == 0) ns[(size_t)sl * n + r] = s;
    mx = fmaxf(mx, s);
  }
  mx = warp_max(mx);
  // squared norms are >= 0, so their bit patterns order like the values
  if ((threadIdx.x & 31) == 0 && mx > 0.f) atomicMax(vmax2_bits + sl, __float_as_uint(mx));
}

// The bucket index of a squared norm: the smallest i with 4^i >= ns (ns > 0).
__device__ inline int bucket_of(float ns) {
  int e;
  const float m = frexpf(ns, &e);            // ns = m * 2^e, m in [0.5, 1)
  const int a = (m == 0.5f) ? e - 1 : e;     // smallest integer >= log2(ns)
  return (a + 1) >> 1;                       // ceil(a / 2), also for negative a
}

// Stable partition of a stream's block by bucket.  One CTA per stream; thread x owns the
// contiguous tokens [x*per, (x+1)*per).  Writes, per token, its slot (or -1) and its rank among
// the block's tokens of the same slot; per stream, the counts and the erase decision.
__global__ void __launch_bounds__(kScanThreads)
bucket_scan_kernel(const float* __restrict__ ns, int n, int n_buckets, int i_top, float rho2,
                   const BucketIn* __restrict__ in, const unsigned* __restrict__ vmax2_bits, int8_t* __restrict__ slot,
                   int32_t* __restrict__ rank, BucketOut* __restrict__ out) {
  __shared__ int warp_tot[kMaxBuckets][kScanThreads / 32];
  __shared__ int tot[kMaxBuckets];
  const int sl = blockIdx.x;
  const float vmax2 = fmaxf(in[sl].prev_vmax2, __uint_as_float(vmax2_bits[sl]));
  // largest erased index: 4^i <= rho^2 * v_max^2
  int erase_max = INT32_MIN;
  const float thr = rho2 * vmax2;
  if (thr > 0.f) {
    int e;
    frexpf(thr, &e);                         // log2(thr) in [e-1, e)
    erase_max = (e - 1) >> 1;                // floor((e-1)/2)
  }
  erase_max = max(erase_max, in[sl].prev_erase_max);
  const int per = (n + kScanThreads - 1) / kScanThreads;
  const int j0 = min(n, (int)threadIdx.x * per), j1 = min(n, j0 + per);
  const float* x = ns + (size_t)sl * n;
  int cnt[kMaxBuckets];
#pragma unroll
  for (int b = 0; b < kMaxBuckets; ++b) cnt[b] = 0;
  int dropped = 0, above = 0;
  for (int j = j0; j < j1; ++j) {
    const float v = x[j];
    int b = -1;
    if (v > 0.f) {
      const int i = bucket_of(v);
      if (i > i_top) ++above;
      else if (i > erase_max && i_top - i < n_buckets) b = i_top - i;
    }
    if (b < 0) ++dropped;
#pragma unroll
    for (int bb = 0; bb < kMaxBuckets; ++bb) cnt[bb] += (bb == b);
    slot[(size_t)sl * n + j] = (int8_t)b;
  }
  // exclusive prefix of the per-thread counts, bucket by bucket
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int excl[kMaxBuckets];
#pragma unroll
  for (int b = 0; b < kMaxBuckets; ++b) {
    int v = cnt[b];
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int u = __shfl_up_sync(0xffffffffu, v, o);
      if (lane >= o) v += u;
    }
    excl[b] = v - cnt[b];
    if (lane == 31) warp_tot[b][warp] = v;
  }
  __syncthreads();
  if (warp < kMaxBuckets) {
    int v = warp_tot[warp][lane];
    const int own = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int u = __shfl_up_sync(0xffffffffu, v, o);
      if (lane >= o) v += u;
    }
    warp_tot[warp][lane] = v - own;
    if (lane == 31) tot[warp] = v;
  }
  __syncthreads();
#pragma unroll
  for (int b = 0; b < kMaxBuckets; ++b) excl[b] += warp_tot[b][warp];
  for (int j = j0; j < j1; ++j) {
    const int b = slot[(size_t)sl * n + j];
    int r = 0;
#pragma unroll
    for (int bb = 0; bb < kMaxBuckets; ++bb)
      if (bb == b) r = excl[bb]++;
    rank[(size_t)sl * n + j] = r;
  }
  dropped = warp_sum_int(dropped);
  above = warp_sum_int(above);
  if (threadIdx.x == 0) { out[sl].dropped = 0; out[sl].above = 0; }
  __syncthreads();
  if (lane == 0) {
    if (dropped) atomicAdd(&out[sl].dropped, dropped);
    if (above) atomicAdd(&out[sl].above, above);
  }
  if (threadIdx.x == 0) {
    for (int b = 0; b < kMaxBuckets; ++b) out[sl].count[b] = tot[b];
    out[sl].erase_max = erase_max;
    out[sl].vmax2 = vmax2;
  }
}

// Copies every kept row of the block to its instance: row `rank` after the level-0 rows the
// instance already holds, with its position in the instance's stream and its squared norms.
// grid (row groups, streams), 256 threads; chunks lanes share a row.
template <bool kBf16>
__global__ void __launch_bounds__(256)
bucket_scatter_kernel(Geom G, Arena A, const void* __restrict__ Ksrc, const void* __restrict__ Vsrc, int n, int chunks,
                      int n_buckets, const int8_t* __restrict__ slot, const int32_t* __restrict__ rank,
                      const float* __restrict__ ns, const BucketDst* __restrict__ dst) {
  const int sl = blockIdx.y;
  const int rows_per_pass = blockDim.x / chunks;
  const int row_in = threadIdx.x / chunks, piece = threadIdx.x % chunks;
  const uint4* sK = reinterpret_cast<const uint4*>(Ksrc) + (size_t)sl * n * chunks;
  const uint4* sV = reinterpret_cast<const uint4*>(Vsrc) + (size_t)sl * n * chunks;
  uint4* dK = reinterpret_cast<uint4*>(A.K);
  uint4* dV = reinterpret_cast<uint4*>(A.V);
  const int row_end = min(n, (int)(blockIdx.x + 1) * kRowsPerBlock);
  for (int r0 = blockIdx.x * kRowsPerBlock; r0 < row_end; r0 += rows_per_pass) {
    const int r = r0 + row_in;
    const int b = r < row_end ? slot[(size_t)sl * n + r] : -1;
    float k2 = 0.f;
    int64_t row = 0;
    int rk = 0;
    if (b >= 0) {
      const BucketDst D = dst[sl * n_buckets + b];
      rk = rank[(size_t)sl * n + r];
      row = D.dst_row + rk;
      const uint4 kk = sK[(size_t)r * chunks + piece];
      const uint4 vv = sV[(size_t)r * chunks + piece];
      dK[(size_t)row * chunks + piece] = kk;
      dV[(size_t)row * chunks + piece] = vv;
      k2 = sumsq_piece<kBf16>(kk);
      if (piece == 0) A.idx[row] = D.idx0 + rk;
    }
    for (int o = chunks / 2; o > 0; o >>= 1) k2 += __shfl_xor_sync(0xffffffffu, k2, o);
    if (b >= 0 && piece == 0 && A.nrm) A.nrm[row] = make_float2(k2, ns[(size_t)sl * n + r]);
  }
  if (blockIdx.x == 0 && threadIdx.x < n_buckets) {
    const BucketDst D = dst[sl * n_buckets + threadIdx.x];
    if (D.stream >= 0) A.seg[(size_t)D.stream * (G.T + 1)].len = D.new_len;
  }
}

}  // namespace

cudaError_t launch_bucket_route(const Geom& G, const void* V, int n_sl, int n, int n_buckets, int i_top, float rho2,
                                const BucketIn* in, unsigned* vmax2_bits, float* ns, int8_t* slot, int32_t* rank,
                                BucketOut* out, cudaStream_t st) {
  const int chunks = G.d * (G.is_bf16 ? 2 : 4) / 16;
  cudaError_t e = cudaMemsetAsync(vmax2_bits, 0, sizeof(unsigned) * n_sl, st);
  if (e != cudaSuccess) return e;
  dim3 grid((n + kRowsPerBlock - 1) / kRowsPerBlock, n_sl);
  if (G.is_bf16) bucket_norms_kernel<true><<<grid, 256, 0, st>>>(V, n, chunks, ns, vmax2_bits);
  else bucket_norms_kernel<false><<<grid, 256, 0, st>>>(V, n, chunks, ns, vmax2_bits);
  bucket_scan_kernel<<<n_sl, kScanThreads, 0, st>>>(ns, n, n_buckets, i_top, rho2, in, vmax2_bits, slot, rank, out);
  return cudaGetLastError();
}

cudaError_t launch_bucket_scatter(const Geom& G, const Arena& A, const void* K, const void* V, int n_sl, int n,
                                  int n_buckets, const int8_t* slot, const int32_t* rank, const float* ns,
                                  const BucketDst* dst, cudaStream_t st) {
  const int chunks = G.d * (G.is_bf16 ? 2 : 4) / 16;
  dim3 grid((n + kRowsPerBlock - 1) / kRowsPerBlock, n_sl);
  if (G.is_bf16) bucket_scatter_kernel<true><<<grid, 256, 0, st>>>(G, A, K, V, n, chunks, n_buckets, slot, rank, ns, dst);
  else bucket_scatter_kernel<false><<<grid, 256, 0, st>>>(G, A, K, V, n, chunks, n_buckets, slot, rank, ns, dst);
  return cudaGetLastError();
}

}  // namespace bkv
