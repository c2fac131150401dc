// Value-norm buckets of BalanceKV (Algorithm 1, the bucketing step and the erasure of small-norm
// buckets): token j goes to the MergeAndReduce instance of the index i with 2^(i-1) < ||v_j|| <= 2^i,
// instances whose bucket satisfies 2^i <= rho * v_max are erased.  Four kernels: squared value
// norms + running maximum; a stable partition of the block's tokens by bucket in two parts (ranks
// inside chunks of 2048 tokens, then the prefix over a stream's chunks); and the copy of every
// kept row into the level-0 set of its bucket's instance.
#include <cuda_bf16.h>
#include <cuda_runtime.h>

#include <cstdint>

#include "common.cuh"

namespace bkv {

namespace {

constexpr int kScanThreads = 256;
constexpr int kScanChunk = 2048;               // tokens per CTA of the partition's first part
constexpr int kCountCols = kMaxBuckets + 2;    // per-slot counts, dropped, above
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
// a row) and the maximum per stream.  grid (row groups, streams), 256 threads; a thread's loads of
// all passes are issued before the first is reduced.
template <bool kBf16>
__global__ void __launch_bounds__(256)
bucket_norms_kernel(const void* __restrict__ V, int n, int chunks, float* __restrict__ ns, unsigned* __restrict__ vmax2_bits) {
  const int sl = blockIdx.y;
  const int rows_per_pass = blockDim.x / chunks;         // 32, 16 or 8
  const int row_in = threadIdx.x / chunks, piece = threadIdx.x % chunks;
  const uint4* src = reinterpret_cast<const uint4*>(V) + (size_t)sl * n * chunks;
  const int row0 = blockIdx.x * kRowsPerBlock;
  const int row_end = min(n, row0 + kRowsPerBlock);
  constexpr int kMaxPasses = kRowsPerBlock / 8;
  uint4 v[kMaxPasses];
#pragma unroll
  for (int u = 0; u < kMaxPasses; ++u) {
    const int r = row0 + u * rows_per_pass + row_in;
    v[u] = make_uint4(0u, 0u, 0u, 0u);
    if (u * rows_per_pass < kRowsPerBlock && r < row_end) v[u] = src[(size_t)r * chunks + piece];
  }
  float mx = 0.f;
#pragma unroll
  for (int u = 0; u < kMaxPasses; ++u) {
    if (u * rows_per_pass >= kRowsPerBlock) break;       // block-uniform
    const int r = row0 + u * rows_per_pass + row_in;
    float s = sumsq_piece<kBf16>(v[u]);
    for (int o = chunks / 2; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    if (r < row_end && piece == 0) ns[(size_t)sl * n + r] = s;
    mx = fmaxf(mx, s);
  }
  mx = warp_max(mx);
  __shared__ float warp_mx[8];
  if ((threadIdx.x & 31) == 0) warp_mx[threadIdx.x >> 5] = mx;
  __syncthreads();
  if (threadIdx.x == 0) {
#pragma unroll
    for (int w = 1; w < 8; ++w) mx = fmaxf(mx, warp_mx[w]);
    // squared norms are >= 0, so their bit patterns order like the values; one atomic per CTA,
    // and none once the stream's maximum is already at least this large
    const unsigned bits = __float_as_uint(mx);
    if (bits > *reinterpret_cast<volatile unsigned*>(vmax2_bits + sl)) atomicMax(vmax2_bits + sl, bits);
  }
}

// The bucket index of a squared norm: the smallest i with 4^i >= ns (ns > 0).
__device__ inline int bucket_of(float ns) {
  int e;
  const float m = frexpf(ns, &e);            // ns = m * 2^e, m in [0.5, 1)
  const int a = (m == 0.5f) ? e - 1 : e;     // smallest integer >= log2(ns)
  return (a + 1) >> 1;                       // ceil(a / 2), also for negative a
}

// The largest erased bucket index after the block: 4^i <= rho^2 * v_max^2 (INT32_MIN: none).
__device__ inline int erase_index(float rho2, const BucketIn& in, unsigned vmax2_bits) {
  const float vmax2 = fmaxf(in.prev_vmax2, __uint_as_float(vmax2_bits));
  int erase_max = INT32_MIN;
  const float thr = rho2 * vmax2;
  if (thr > 0.f) {
    int e;
    frexpf(thr, &e);                         // log2(thr) in [e-1, e)
    erase_max = (e - 1) >> 1;                // floor((e-1)/2)
  }
  return max(erase_max, in.prev_erase_max);
}

// Stable partition of a stream's block by bucket, first part.  grid (chunks of kScanChunk tokens,
// streams), 256 threads; warp w owns the contiguous tokens [w*256, (w+1)*256) of the chunk and
// walks them 32 at a time (ballots give the rank among equal slots).  Writes, per token, its slot
// (or -1) and its rank among the chunk's tokens of the same slot; per chunk, the counts.
__global__ void __launch_bounds__(kScanThreads)
bucket_scan_kernel(const float* __restrict__ ns, int n, int n_chunks, int n_buckets, int i_top, float rho2,
                   const BucketIn* __restrict__ in, const unsigned* __restrict__ vmax2_bits, int8_t* __restrict__ slot,
                   int32_t* __restrict__ rank, int32_t* __restrict__ chunk_cnt, const int8_t* __restrict__ forced) {
  constexpr int kWarps = kScanThreads / 32, kRounds = kScanChunk / kScanThreads;
  __shared__ int warp_tot[kCountCols][kWarps];
  const int sl = blockIdx.y, chunk = blockIdx.x;
  const int erase_max = erase_index(rho2, in[sl], vmax2_bits[sl]);
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const unsigned lt = (1u << lane) - 1u;
  const size_t base = (size_t)sl * n;
  const int j0 = chunk * kScanChunk + warp * (kScanChunk / kWarps);
  float x[kRounds];
#pragma unroll
  for (int u = 0; u < kRounds; ++u) {
    const int j = j0 + u * 32 + lane;
    x[u] = j < n ? ns[base + j] : -1.f;
  }
  int run[kCountCols];                                   // warp-uniform running counts: slots, dropped, above
#pragma unroll
  for (int b = 0; b < kCountCols; ++b) run[b] = 0;
  int my_slot[kRounds], my_rank[kRounds];
#pragma unroll
  for (int u = 0; u < kRounds; ++u) {
    int b = -3;                                          // past the end of the block
    if (x[u] >= 0.f && forced) {
      b = forced[base + j0 + u * 32 + lane];             // the slot was decided elsewhere (not by the value norm)
    } else if (x[u] >= 0.f) {
      b = kMaxBuckets;                                   // dropped
      if (x[u] > 0.f) {
        const int i = bucket_of(x[u]);
        if (i > i_top) b = kMaxBuckets + 1;              // above the highest slot
        else if (i > erase_max && i_top - i < n_buckets) b = i_top - i;
      }
    }
    my_slot[u] = b;
    my_rank[u] = 0;
#pragma unroll
    for (int bb = 0; bb < kCountCols; ++bb) {
      const unsigned m = __ballot_sync(0xffffffffu, b == bb);
      if (b == bb) my_rank[u] = run[bb] + __popc(m & lt);
      run[bb] += __popc(m);
    }
  }
  if (lane == 0) {
#pragma unroll
    for (int bb = 0; bb < kCountCols; ++bb) warp_tot[bb][warp] = run[bb];
  }
  __syncthreads();
#pragma unroll
  for (int u = 0; u < kRounds; ++u) {
    const int j = j0 + u * 32 + lane;
    const int b = my_slot[u];
    if (j < n) {
      int off = 0;
      if (b >= 0 && b < kMaxBuckets)
        for (int w = 0; w < warp; ++w) off += warp_tot[b][w];
      slot[base + j] = (int8_t)(b < kMaxBuckets ? b : -1);
      rank[base + j] = off + my_rank[u];
    }
  }
  if (threadIdx.x < kCountCols) {
    int t = 0;
    for (int w = 0; w < kWarps; ++w) t += warp_tot[threadIdx.x][w];
    chunk_cnt[((size_t)sl * n_chunks + chunk) * kCountCols + threadIdx.x] = t;
  }
}

// Second part: per stream, the exclusive prefix of the chunks' counts (in place) and the totals.
// grid (streams), kCountCols warps: warp b scans column b, 32 chunks at a time.
__global__ void __launch_bounds__(kCountCols * 32)
bucket_prefix_kernel(int n_chunks, float rho2, const BucketIn* __restrict__ in, const unsigned* __restrict__ vmax2_bits,
                     int32_t* __restrict__ chunk_cnt, BucketOut* __restrict__ out) {
  const int sl = blockIdx.x, col = threadIdx.x >> 5, lane = threadIdx.x & 31;
  int32_t* c = chunk_cnt + (size_t)sl * n_chunks * kCountCols + col;
  int carry = 0;
  for (int c0 = 0; c0 < n_chunks; c0 += 32) {
    const int i = c0 + lane;
    const int own = i < n_chunks ? c[(size_t)i * kCountCols] : 0;
    int v = own;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const int u = __shfl_up_sync(0xffffffffu, v, o);
      if (lane >= o) v += u;
    }
    if (i < n_chunks) c[(size_t)i * kCountCols] = carry + v - own;
    carry += __shfl_sync(0xffffffffu, v, 31);
  }
  if (lane == 0) {
    if (col < kMaxBuckets) out[sl].count[col] = carry;
    else if (col == kMaxBuckets) out[sl].dropped = carry;
    else out[sl].above = carry;
  }
  if (threadIdx.x == 0) {
    out[sl].erase_max = erase_index(rho2, in[sl], vmax2_bits[sl]);
    out[sl].vmax2 = fmaxf(in[sl].prev_vmax2, __uint_as_float(vmax2_bits[sl]));
  }
}

// Copies every kept row of the block to its instance: row `rank` after the level-0 rows the
// instance already holds, with its position in the instance's stream and its squared norms.
// grid (row groups, streams), 256 threads; chunks lanes share a row.
template <bool kBf16>
__global__ void __launch_bounds__(256)
bucket_scatter_kernel(Geom G, Arena A, const void* __restrict__ Ksrc, const void* __restrict__ Vsrc, int n, int chunks,
                      int n_buckets, const int8_t* __restrict__ slot, const int32_t* __restrict__ rank,
                      const int32_t* __restrict__ chunk_base, int n_chunks, const float* __restrict__ ns,
                      const BucketDst* __restrict__ dst) {
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
      rk = rank[(size_t)sl * n + r] + chunk_base[((size_t)sl * n_chunks + r / kScanChunk) * kCountCols + b];
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

int bucket_scan_chunks(int n) { return (n + kScanChunk - 1) / kScanChunk; }
size_t bucket_chunk_count_ints(int n_sl, int n) { return (size_t)n_sl * bucket_scan_chunks(n) * kCountCols; }

cudaError_t launch_bucket_route(const Geom& G, const void* V, int n_sl, int n, int n_buckets, int i_top, float rho2,
                                const BucketIn* in, unsigned* vmax2_bits, float* ns, int8_t* slot, int32_t* rank,
                                int32_t* chunk_cnt, BucketOut* out, const int8_t* forced_slot, cudaStream_t st) {
  const int chunks = G.d * (G.is_bf16 ? 2 : 4) / 16;
  cudaError_t e = cudaMemsetAsync(vmax2_bits, 0, sizeof(unsigned) * n_sl, st);
  if (e != cudaSuccess) return e;
  dim3 grid((n + kRowsPerBlock - 1) / kRowsPerBlock, n_sl);
  if (G.is_bf16) bucket_norms_kernel<true><<<grid, 256, 0, st>>>(V, n, chunks, ns, vmax2_bits);
  else bucket_norms_kernel<false><<<grid, 256, 0, st>>>(V, n, chunks, ns, vmax2_bits);
  const int n_chunks = bucket_scan_chunks(n);
  bucket_scan_kernel<<<dim3(n_chunks, n_sl), kScanThreads, 0, st>>>(ns, n, n_chunks, n_buckets, i_top, rho2, in, vmax2_bits,
                                                                   slot, rank, chunk_cnt, forced_slot);
  bucket_prefix_kernel<<<n_sl, kCountCols * 32, 0, st>>>(n_chunks, rho2, in, vmax2_bits, chunk_cnt, out);
  return cudaGetLastError();
}

cudaError_t launch_bucket_scatter(const Geom& G, const Arena& A, const void* K, const void* V, int n_sl, int n,
                                  int n_buckets, const int8_t* slot, const int32_t* rank, const int32_t* chunk_base,
                                  const float* ns, const BucketDst* dst, cudaStream_t st) {
  const int chunks = G.d * (G.is_bf16 ? 2 : 4) / 16;
  const int n_chunks = bucket_scan_chunks(n);
  dim3 grid((n + kRowsPerBlock - 1) / kRowsPerBlock, n_sl);
  if (G.is_bf16)
    bucket_scatter_kernel<true><<<grid, 256, 0, st>>>(G, A, K, V, n, chunks, n_buckets, slot, rank, chunk_base, n_chunks, ns, dst);
  else
    bucket_scatter_kernel<false><<<grid, 256, 0, st>>>(G, A, K, V, n, chunks, n_buckets, slot, rank, chunk_base, n_chunks, ns, dst);
  return cudaGetLastError();
}

}  // namespace bkv
