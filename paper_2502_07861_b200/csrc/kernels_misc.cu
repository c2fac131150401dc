// Data-movement and reduction helpers of the BalanceKV library:
//   append / level load   (Algorithm 3: C^0 <- C^0 + {k_j, v_j})
//   level-0 remainder move
//   per-call radii r_key^2, r_value^2 (inputs of Algorithm 2) and the optional key shift
#include "common.cuh"

namespace bkv {

namespace {

constexpr int kCopyRows = 64;  // rows handled by one CTA of the copy kernels

// Copies rows of 16-byte chunks: dst[r][c] = src[r][c].
__device__ inline void copy_rows(uint4* __restrict__ dst, const uint4* __restrict__ src, int rows, int chunks) {
  const int total = rows * chunks;
  for (int i = threadIdx.x; i < total; i += blockDim.x) dst[i] = src[i];
}

template <bool kBf16>
__device__ inline float sumsq16(const uint4& v) {
  float s = 0.f;
  if (kBf16) {
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

// Copies rows of K and V and records (||k||^2, ||v||^2) of every row: the radii of Algorithm 2
// (r_key, r_value of a call) then need the norms only, not the rows.  `chunks` (16-byte pieces
// of a row: 8, 16 or 32) consecutive lanes share a row; blockDim is a multiple of 32.
template <bool kBf16>
__device__ inline void copy_rows_norm(uint4* __restrict__ dK, const uint4* __restrict__ sK, uint4* __restrict__ dV,
                                      const uint4* __restrict__ sV, float2* __restrict__ nrm, int rows, int chunks) {
  const int total = rows * chunks;
  // four rounds of loads are issued before the first is consumed (the copy is latency bound)
  for (int i0 = 0; i0 < total; i0 += 4 * blockDim.x) {    // whole warps take part in the shuffles
    uint4 a[4], b[4];
    int idx[4];
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      idx[u] = i0 + u * blockDim.x + threadIdx.x;
      if (idx[u] < total) { a[u] = sK[idx[u]]; b[u] = sV[idx[u]]; }
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
      if (i0 + u * (int)blockDim.x >= total) break;       // block-uniform
      const int i = idx[u];
      float k2 = 0.f, v2 = 0.f;
      if (i < total) {
        dK[i] = a[u];
        dV[i] = b[u];
        k2 = sumsq16<kBf16>(a[u]);
        v2 = sumsq16<kBf16>(b[u]);
      }
      for (int o = chunks / 2; o > 0; o >>= 1) {
        k2 += __shfl_xor_sync(0xffffffffu, k2, o);
        v2 += __shfl_xor_sync(0xffffffffu, v2, o);
      }
      if (i < total && i % chunks == 0) nrm[i / chunks] = make_float2(k2, v2);
    }
  }
}

__device__ inline void copy_rows_kv(const Geom& G, const Arena& A, size_t dst_b, int64_t dst_row, const void* Ksrc,
                                    const void* Vsrc, size_t src_b, int rows) {
  const int esz = G.is_bf16 ? 2 : 4;
  const int chunks = G.d * esz / 16;
  uint4* dK = reinterpret_cast<uint4*>(static_cast<char*>(A.K) + dst_b);
  uint4* dV = reinterpret_cast<uint4*>(static_cast<char*>(A.V) + dst_b);
  const uint4* sK = reinterpret_cast<const uint4*>(static_cast<const char*>(Ksrc) + src_b);
  const uint4* sV = reinterpret_cast<const uint4*>(static_cast<const char*>(Vsrc) + src_b);
  if (A.nrm && chunks <= 32) {
    if (G.is_bf16) copy_rows_norm<true>(dK, sK, dV, sV, A.nrm + dst_row, rows, chunks);
    else copy_rows_norm<false>(dK, sK, dV, sV, A.nrm + dst_row, rows, chunks);
  } else {
    copy_rows(dK, sK, rows, chunks);
    copy_rows(dV, sV, rows, chunks);
  }
}

__global__ void __launch_bounds__(256)
append_kernel(Geom G, Arena A, const AppendDesc* __restrict__ descs, const void* __restrict__ Ksrc,
              const void* __restrict__ Vsrc, const int32_t* __restrict__ idx_src) {
  const AppendDesc D = descs[blockIdx.x];
  const int row0 = blockIdx.y * kCopyRows;
  if (row0 < D.n) {
    const int rows = min(kCopyRows, D.n - row0);
    const int esz = G.is_bf16 ? 2 : 4;
    const size_t dst_b = (size_t)(D.dst_row + row0) * G.d * esz;
    const size_t src_b = ((size_t)D.src_off + (size_t)row0 * G.d) * esz;
    copy_rows_kv(G, A, dst_b, D.dst_row + row0, Ksrc, Vsrc, src_b, rows);
    for (int i = threadIdx.x; i < rows; i += blockDim.x)
      A.idx[D.dst_row + row0 + i] = idx_src ? idx_src[D.src_off / G.d + row0 + i] : D.idx0 + row0 + i;
  }
  if (blockIdx.y == 0 && threadIdx.x == 0) A.seg[(size_t)D.stream * (G.T + 1) + D.level].len = D.new_len;
}

// Append for a layer whose streams are in lockstep (same level-0 fill): the per-stream
// descriptor is implied by the block index, so no descriptor array travels to the device.
__global__ void __launch_bounds__(256)
append_uniform_kernel(Geom G, Arena A, int layer, int level, int rel_row, int idx0, int n, int new_len,
                      const void* __restrict__ Ksrc, const void* __restrict__ Vsrc, const int32_t* __restrict__ idx_src) {
  const int sl = blockIdx.x;                                 // seq * H + head
  const int stream = ((sl / G.H) * G.L + layer) * G.H + (sl % G.H);
  const int64_t dst_row = (int64_t)stream * G.rows_per_stream + G.region_off[level] + rel_row;
  const int row0 = blockIdx.y * kCopyRows;
  if (row0 < n) {
    const int rows = min(kCopyRows, n - row0);
    const int esz = G.is_bf16 ? 2 : 4;
    const size_t dst_b = (size_t)(dst_row + row0) * G.d * esz;
    const size_t src_b = ((size_t)sl * n + row0) * G.d * esz;
    copy_rows_kv(G, A, dst_b, dst_row + row0, Ksrc, Vsrc, src_b, rows);
    for (int i = threadIdx.x; i < rows; i += blockDim.x)
      A.idx[dst_row + row0 + i] = idx_src ? idx_src[(size_t)sl * n + row0 + i] : idx0 + row0 + i;
  }
  if (blockIdx.y == 0 && threadIdx.x == 0) A.seg[(size_t)stream * (G.T + 1) + level].len = new_len;
}

__global__ void __launch_bounds__(256)
move_kernel(Geom G, Arena A, const MoveDesc* __restrict__ descs) {
  const MoveDesc D = descs[blockIdx.x];
  const int row0 = blockIdx.y * kCopyRows;
  if (row0 < D.n) {
    const int rows = min(kCopyRows, D.n - row0);
    const int esz = G.is_bf16 ? 2 : 4;
    const int chunks = G.d * esz / 16;
    const size_t dst_b = (size_t)(D.dst_row + row0) * G.d * esz;
    const size_t src_b = (size_t)(D.src_row + row0) * G.d * esz;
    copy_rows(reinterpret_cast<uint4*>(static_cast<char*>(A.K) + dst_b),
              reinterpret_cast<const uint4*>(static_cast<const char*>(A.K) + src_b), rows, chunks);
    copy_rows(reinterpret_cast<uint4*>(static_cast<char*>(A.V) + dst_b),
              reinterpret_cast<const uint4*>(static_cast<const char*>(A.V) + src_b), rows, chunks);
    for (int i = threadIdx.x; i < rows; i += blockDim.x) {
      A.idx[D.dst_row + row0 + i] = A.idx[D.src_row + row0 + i];
      if (A.nrm) A.nrm[D.dst_row + row0 + i] = A.nrm[D.src_row + row0 + i];
    }
  }
}

__global__ void seg_update_kernel(Arena A, const SegUpdate* __restrict__ ups, int n) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) A.seg[ups[i].index] = Seg{ups[i].start, ups[i].len};
}

// Column means of the call's keys, one CTA per call, thread e owns column e
// (fixed summation order, so the result is reproducible).
template <bool kBf16>
__global__ void mean_kernel(Geom G, Arena A, const CallDesc* __restrict__ calls, float* __restrict__ mean) {
  const CallDesc C = calls[blockIdx.x];
  const int e = threadIdx.x;
  if (e >= G.d) return;
  float s = 0.f;
  for (int j = 0; j < G.t; ++j) {
    const size_t off = (size_t)(C.src_row + j) * G.d + e;
    s += kBf16 ? __bfloat162float(static_cast<const __nv_bfloat16*>(A.K)[off]) : static_cast<const float*>(A.K)[off];
  }
  mean[(size_t)blockIdx.x * G.d + e] = s / (float)G.t;
}

// r_key^2 = max_j ||k_j - mean||^2, r_value^2 = max_j ||v_j||^2 over the call's tokens,
// and the per-token shift a_j = <k_j, mean> - ||mean||^2/2, with which
// <k_i - mean, k_j - mean> = <k_i, k_j> - a_i - a_j.
template <bool kBf16>
__global__ void __launch_bounds__(256)
radii_kernel(Geom G, Arena A, const CallDesc* __restrict__ calls, CallStat* __restrict__ stats,
             const float* __restrict__ mean, float* __restrict__ tok_shift) {
  const CallDesc C = calls[blockIdx.x];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int esz = kBf16 ? 2 : 4;
  float mk = 0.f, mv = 0.f;
  const float* mu = mean ? mean + (size_t)blockIdx.x * G.d : nullptr;
  float mu2 = 0.f;
  if (mu) {
    for (int e = lane; e < G.d; e += 32) mu2 += mu[e] * mu[e];
    mu2 = warp_sum(mu2);
  }
  // d / 8 lanes share a row (8 elements each): with d = 128 a warp works on two rows at a time
  const int lpr = G.d / 8 < 32 ? G.d / 8 : 32;     // lanes per row
  const int rpw = 32 / lpr;                        // rows per warp step
  const int sub = lane / lpr, l0 = lane % lpr;
  const int row_end = min(G.t, (int)(blockIdx.y + 1) * 64);
  for (int r = blockIdx.y * 64 + warp * rpw + sub; r - sub < row_end; r += 8 * rpw) {
    const bool live = r < row_end;
    const char* krow = static_cast<const char*>(A.K) + (size_t)(C.src_row + (live ? r : 0)) * G.d * esz;
    const char* vrow = static_cast<const char*>(A.V) + (size_t)(C.src_row + (live ? r : 0)) * G.d * esz;
    float sk = 0.f, sv = 0.f, sm = 0.f;
    for (int e = l0 * 8; e < G.d; e += lpr * 8) {
      float a[8], b[8];
      load8<kBf16>(krow, e, a);
      load8<kBf16>(vrow, e, b);
#pragma unroll
      for (int i = 0; i < 8; ++i) {
        sk = fmaf(a[i], a[i], sk);
        sv = fmaf(b[i], b[i], sv);
        if (mu) sm = fmaf(a[i], mu[e + i], sm);
      }
    }
    for (int o = lpr / 2; o > 0; o >>= 1) {
      sk += __shfl_xor_sync(0xffffffffu, sk, o);
      sv += __shfl_xor_sync(0xffffffffu, sv, o);
      if (mu) sm += __shfl_xor_sync(0xffffffffu, sm, o);
    }
    if (mu) {
      const float shift = sm - 0.5f * mu2;
      sk = fmaxf(sk - 2.f * shift, 0.f);
      if (live && l0 == 0) tok_shift[(size_t)blockIdx.x * G.t + r] = shift;
    }
    if (live) { mk = fmaxf(mk, sk); mv = fmaxf(mv, sv); }
  }
  mk = warp_max(mk); mv = warp_max(mv);
  __shared__ float smk[8], smv[8];
  if (lane == 0) { smk[warp] = mk; smv[warp] = mv; }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < 8; ++w) { mk = fmaxf(mk, smk[w]); mv = fmaxf(mv, smv[w]); }
    // non-negative floats order like their bit patterns
    atomicMax(reinterpret_cast<int*>(&stats[blockIdx.x].rk2), __float_as_int(mk));
    atomicMax(reinterpret_cast<int*>(&stats[blockIdx.x].rv2), __float_as_int(mv));
  }
}

// r_key^2, r_value^2 of a call from the stored row norms: one CTA per call.
__global__ void __launch_bounds__(256)
radii_norms_kernel(Geom G, Arena A, const CallDesc* __restrict__ calls, CallStat* __restrict__ stats) {
  const CallDesc C = calls[blockIdx.x];
  float mk = 0.f, mv = 0.f;
  for (int j = threadIdx.x; j < G.t; j += 256) {
    const float2 n = A.nrm[C.src_row + j];
    mk = fmaxf(mk, n.x);
    mv = fmaxf(mv, n.y);
  }
  mk = warp_max(mk); mv = warp_max(mv);
  __shared__ float smk[8], smv[8];
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (lane == 0) { smk[warp] = mk; smv[warp] = mv; }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < 8; ++w) { mk = fmaxf(mk, smk[w]); mv = fmaxf(mv, smv[w]); }
    CallStat S{};
    S.rk2 = mk; S.rv2 = mv;
    stats[blockIdx.x] = S;
  }
}

__global__ void fill_weights_kernel(float* w, int n, float value) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i < n) w[i] = value;
}

}  // namespace

cudaError_t launch_append(const Geom& G, const Arena& A, const AppendDesc* descs, int n_desc, int max_rows,
                          const void* Ksrc, const void* Vsrc, const int32_t* idx_src, cudaStream_t st) {
  if (n_desc <= 0) return cudaSuccess;
  dim3 grid(n_desc, (max_rows + kCopyRows - 1) / kCopyRows);
  if (grid.y == 0) grid.y = 1;
  append_kernel<<<grid, 256, 0, st>>>(G, A, descs, Ksrc, Vsrc, idx_src);
  return cudaGetLastError();
}

cudaError_t launch_append_uniform(const Geom& G, const Arena& A, int layer, int level, int rel_row, int idx0, int n,
                                  int new_len, const void* Ksrc, const void* Vsrc, const int32_t* idx_src,
                                  cudaStream_t st) {
  dim3 grid(G.B * G.H, (n + kCopyRows - 1) / kCopyRows);
  append_uniform_kernel<<<grid, n >= 16 ? 256 : 64, 0, st>>>(G, A, layer, level, rel_row, idx0, n, new_len, Ksrc, Vsrc, idx_src);
  return cudaGetLastError();
}

cudaError_t launch_move(const Geom& G, const Arena& A, const MoveDesc* descs, int n_desc, int max_rows,
                        cudaStream_t st) {
  if (n_desc <= 0) return cudaSuccess;
  dim3 grid(n_desc, (max_rows + kCopyRows - 1) / kCopyRows);
  if (grid.y == 0) grid.y = 1;
  move_kernel<<<grid, 256, 0, st>>>(G, A, descs);
  return cudaGetLastError();
}

// stats must hold n_calls entries; tok_shift n_calls * t floats (+ n_calls * d floats of
// mean scratch behind it) when key centering is on, else it may be null.
cudaError_t launch_radii(const Geom& G, const Arena& A, const CallDesc* calls, int n_calls, CallStat* stats,
                         float* tok_shift, cudaStream_t st) {
  if (n_calls <= 0) return cudaSuccess;
  if (!G.center_keys && A.nrm) {     // the norms were recorded when the rows were written
    radii_norms_kernel<<<n_calls, 256, 0, st>>>(G, A, calls, stats);
    return cudaGetLastError();
  }
  cudaError_t e = cudaMemsetAsync(stats, 0, sizeof(CallStat) * (size_t)n_calls, st);
  if (e != cudaSuccess) return e;
  float* mean = nullptr;
  if (G.center_keys) {
    mean = tok_shift + (size_t)n_calls * G.t;
    if (G.is_bf16) mean_kernel<true><<<n_calls, 128, 0, st>>>(G, A, calls, mean);
    else mean_kernel<false><<<n_calls, 128, 0, st>>>(G, A, calls, mean);
  }
  dim3 grid(n_calls, (G.t + 63) / 64);
  if (G.is_bf16) radii_kernel<true><<<grid, 256, 0, st>>>(G, A, calls, stats, mean, tok_shift);
  else radii_kernel<false><<<grid, 256, 0, st>>>(G, A, calls, stats, mean, tok_shift);
  return cudaGetLastError();
}

cudaError_t launch_seg_update(const Arena& A, const SegUpdate* ups, int n, cudaStream_t st) {
  if (n <= 0) return cudaSuccess;
  seg_update_kernel<<<(n + 255) / 256, 256, 0, st>>>(A, ups, n);
  return cudaGetLastError();
}

cudaError_t launch_fill_weights(float* w, int n, float value, cudaStream_t st) {
  if (n <= 0) return cudaSuccess;
  fill_weights_kernel<<<(n + 255) / 256, 256, 0, st>>>(w, n, value);
  return cudaGetLastError();
}

}  // namespace bkv
