// Strict-half selection and stream compaction of one SoftmaxBalance call.
//
// Algorithm 2 outputs the smaller sign class (ties: the +1 class); the paper's
// implementation note (Appendix B, "strictly select n/2 embeddings") fixes the output size
// at exactly t/2: the class is completed with the latest tokens of the other class.
// Survivors keep their stream order, move to the next level's set (Algorithm 3,
// C^{i+1} <- C^{i+1} + SoftmaxBalance(C^i)) and thereby double their weight.
//
// Grid: (calls, t/2 / 64).  Every CTA recomputes the call's keep mask from the t sign
// bytes (cheap) and copies its own 64 survivor rows of K and V with 16-byte accesses.
#include "common.cuh"

namespace bkv {

namespace {

constexpr int kThreads = 256;
constexpr int kRowsPerCta = 64;

__device__ inline int block_exclusive_scan(int v, int* warp_sums, int& total) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  int inc = v;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int n = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += n;
  }
  __syncthreads();  // protect warp_sums from the previous use
  if (lane == 31) warp_sums[warp] = inc;
  __syncthreads();
  int base = 0, tot = 0;
#pragma unroll
  for (int w = 0; w < kThreads / 32; ++w) {
    const int s = warp_sums[w];
    if (w < warp) base += s;
    tot += s;
  }
  total = tot;
  return base + inc - v;
}

__global__ void __launch_bounds__(kThreads)
compact_kernel(Geom G, Arena A, const CallDesc* __restrict__ calls, const int8_t* __restrict__ eta) {
  extern __shared__ int kept_pos[];  // [t/2]
  __shared__ int warp_sums[kThreads / 32];
  const CallDesc C = calls[blockIdx.x];
  const int t = G.t, half = t / 2;
  const int ipt = (t + kThreads - 1) / kThreads;   // consecutive items per thread
  const int j0 = threadIdx.x * ipt;
  const int8_t* e = eta + (size_t)blockIdx.x * t;

  int plus = 0;
  for (int i = 0; i < ipt; ++i) { const int j = j0 + i; if (j < t) plus += e[j] > 0; }
  int total_plus;
  const int plus_before = block_exclusive_scan(plus, warp_sums, total_plus);
  const int keep_sign = (total_plus <= t - total_plus) ? 1 : -1;
  const int have = keep_sign > 0 ? total_plus : t - total_plus;
  const int other_total = t - have;
  const int first_other_kept = other_total - (half - have);   // rank (in stream order) from which the other class is kept
  // rank of this thread's first item inside the other class
  int other_rank = keep_sign > 0 ? (min(j0, t) - plus_before) : plus_before;
  int keep_cnt = 0;
  unsigned mask = 0;   // ipt <= 32
  for (int i = 0; i < ipt; ++i) {
    const int j = j0 + i;
    if (j >= t) break;
    const bool mine = (e[j] > 0) == (keep_sign > 0);
    bool keep = mine;
    if (!mine) { keep = other_rank >= first_other_kept; ++other_rank; }
    if (keep) { mask |= 1u << i; ++keep_cnt; }
  }
  int total_keep;
  int pos = block_exclusive_scan(keep_cnt, warp_sums, total_keep);
  for (int i = 0; i < ipt; ++i)
    if (mask & (1u << i)) kept_pos[pos++] = j0 + i;
  __syncthreads();

  const int esz = G.is_bf16 ? 2 : 4;
  const int chunks = G.d * esz / 16;
  const int o0 = blockIdx.y * kRowsPerCta;
  const int rows = min(kRowsPerCta, half - o0);
  const int per_row = 2 * chunks;
  for (int i = threadIdx.x; i < rows * per_row; i += kThreads) {
    const int o = o0 + i / per_row;
    const int rem = i % per_row;
    const int which = rem / chunks, ch = rem % chunks;
    const char* src = static_cast<const char*>(which ? A.V : A.K) + (size_t)(C.src_row + kept_pos[o]) * G.d * esz;
    char* dst = static_cast<char*>(which ? A.V : A.K) + (size_t)(C.dst_row + o) * G.d * esz;
    reinterpret_cast<uint4*>(dst)[ch] = reinterpret_cast<const uint4*>(src)[ch];
  }
  for (int i = threadIdx.x; i < rows; i += kThreads) {
    A.idx[C.dst_row + o0 + i] = A.idx[C.src_row + kept_pos[o0 + i]];
    if (A.nrm) A.nrm[C.dst_row + o0 + i] = A.nrm[C.src_row + kept_pos[o0 + i]];
  }
}

}  // namespace

cudaError_t launch_compact(const Geom& G, const Arena& A, const CallDesc* calls, int n_calls, int level,
                           const int8_t* eta, cudaStream_t st) {
  if (n_calls <= 0) return cudaSuccess;
  const int half = G.t / 2;
  dim3 grid(n_calls, (half + kRowsPerCta - 1) / kRowsPerCta);
  (void)level;
  compact_kernel<<<grid, kThreads, sizeof(int) * half, st>>>(G, A, calls, eta);
  return cudaGetLastError();
}

}  // namespace bkv
