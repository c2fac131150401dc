// Split-K decode attention over the weighted compressed cache.
//
//   out = sum_i w_i e^{<k_i,q>/sqrt d} v_i / sum_i w_i e^{<k_i,q>/sqrt d},   w_i = 2^level(i)
//
// i.e. the output ratio of Algorithm 1 / the estimator of Theorem 3.3 over the sets
// C^T..C^0 of one stream (Eq. (1) when every token sits in C^0).  In base 2 the weight is an
// exact integer added to the logit: l_i = <k_i,q> log2(e)/sqrt d + level(i).
//
// Grid (streams of the layer, splits).  A CTA walks its share of the stream's 16 KB tiles
// (K and V rows are contiguous per level, so a tile is one linear bulk copy per tensor)
// through a 3-stage shared-memory ring filled by cp.async.bulk + mbarrier.  Each warp keeps
// private online-softmax state (max, sum, accumulator) for all g query heads of the KV
// head: 8 lanes share a token for the q.k dot product, then every lane owns D/32 output
// columns for p.v.  Warps merge through shared memory, splits through a global scratch
// and a ticket counter (the last CTA of a stream combines; nobody waits).
#include "common.cuh"

namespace bkv {

namespace {

constexpr int kThreads = 256;
constexpr int kWarps = 8;
constexpr int kStages = 3;
constexpr int kTileBytes = 16384;          // per tensor per stage
constexpr int kMaxDevices = 64;
constexpr long long kWaitCycles = 100000000LL;    // about 50 ms: a bulk copy that has not landed by then never will

__device__ inline uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ inline void mbar_init(uint64_t* bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ inline void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ inline bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// Bounded wait: gives up after kWaitCycles and reports failure.
__device__ inline bool mbar_wait(uint64_t* bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (clock64() - t0 > kWaitCycles) return false;
  }
  return true;
}
__device__ inline void bulk_load(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

struct TileRef {
  int64_t row;   // first arena row
  int rows;      // valid rows
  int level;
};

template <int TN>
__device__ inline TileRef locate_tile(int tile, const int* lvl_tiles, const Seg* seg, int T, int64_t stream_base,
                                      const int32_t* region_off) {
  // levels are visited from T down to 0
  TileRef r{0, 0, 0};
  for (int l = T; l >= 0; --l) {
    const int nt = lvl_tiles[l];
    if (tile < nt) {
      r.level = l;
      r.row = stream_base + region_off[l] + seg[l].start + (int64_t)tile * TN;
      r.rows = min(TN, seg[l].len - tile * TN);
      return r;
    }
    tile -= nt;
  }
  return r;
}

template <bool kBf16, int D, int GQ>
__global__ void __launch_bounds__(kThreads, 2)
decode_kernel(Geom G, Arena A, int layer, const void* __restrict__ q, void* __restrict__ out,
              float* __restrict__ part, unsigned* __restrict__ tickets, int* __restrict__ status) {
  constexpr int esz = kBf16 ? 2 : 4;
  constexpr int TN = kTileBytes / (D * esz);      // tokens per tile
  constexpr int DPL = D / 8;                      // dims per lane in the q.k phase
  constexpr int CPL = D / 32;                     // output columns per lane
  constexpr int PS = D + 2;                       // partial row: acc[D], max, sum

  extern __shared__ __align__(128) unsigned char smem_raw[];
  unsigned char* tiles = smem_raw;                                   // kStages * 2 * kTileBytes
  uint64_t* full = reinterpret_cast<uint64_t*>(smem_raw + kStages * 2 * kTileBytes);
  __shared__ int lvl_tiles[kMaxLevels + 1];
  __shared__ Seg seg_s[kMaxLevels + 1];
  __shared__ int is_last_s;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int sl = blockIdx.x;                       // stream inside the layer: seq * H + head
  const int seq = sl / G.H, head = sl % G.H;
  const int stream = (seq * G.L + layer) * G.H + head;
  const int splits = gridDim.y, split = blockIdx.y;
  const int64_t stream_base = (int64_t)stream * G.rows_per_stream;

  if (tid <= G.T) {
    const Seg s = A.seg[(size_t)stream * (G.T + 1) + tid];
    seg_s[tid] = s;
    lvl_tiles[tid] = (s.len + TN - 1) / TN;
  }
  if (tid == 0) {
    for (int s = 0; s < kStages; ++s) mbar_init(&full[s], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  __syncthreads();
  int n_tiles = 0;
  for (int l = 0; l <= G.T; ++l) n_tiles += lvl_tiles[l];
  const int t_begin = (int)((long long)n_tiles * split / splits);
  const int t_end = (int)((long long)n_tiles * (split + 1) / splits);
  const int my_tiles = t_end - t_begin;

  // query of this lane's dims for the g heads of the KV head, pre-scaled by log2(e)/sqrt d
  const int sub = lane & 7, grp = lane >> 3;
  float qr[GQ][DPL];
  {
    const float sc = 1.4426950408889634f * G.inv_sqrt_d;
#pragma unroll
    for (int h = 0; h < GQ; ++h) {
      const size_t off = ((size_t)seq * (G.H * GQ) + head * GQ + h) * D;
#pragma unroll
      for (int i = 0; i < DPL; i += 8) {
        float v[8];
        load8<kBf16>(static_cast<const char*>(q) + off * esz, sub * DPL + i, v);
#pragma unroll
        for (int k = 0; k < 8; ++k) qr[h][i + k] = v[k] * sc;
      }
    }
  }

  auto issue = [&](int i) {   // thread 0 only
    const TileRef tr = locate_tile<TN>(t_begin + i, lvl_tiles, seg_s, G.T, stream_base, G.region_off);
    const int s = i % kStages;
    const uint32_t bytes = (uint32_t)tr.rows * D * esz;
    mbar_expect_tx(&full[s], 2 * bytes);
    bulk_load(tiles + (size_t)s * 2 * kTileBytes, static_cast<const char*>(A.K) + (size_t)tr.row * D * esz, bytes, &full[s]);
    bulk_load(tiles + (size_t)s * 2 * kTileBytes + kTileBytes, static_cast<const char*>(A.V) + (size_t)tr.row * D * esz, bytes, &full[s]);
  };
  if (tid == 0)
    for (int i = 0; i < min(kStages, my_tiles); ++i) issue(i);

  float m_run[GQ], l_run[GQ], acc[GQ][CPL];
#pragma unroll
  for (int h = 0; h < GQ; ++h) {
    m_run[h] = -INFINITY; l_run[h] = 0.f;
#pragma unroll
    for (int c = 0; c < CPL; ++c) acc[h][c] = 0.f;
  }

  bool failed = false;
  for (int i = 0; i < my_tiles; ++i) {
    const int s = i % kStages;
    const bool arrived = __all_sync(0xffffffffu, mbar_wait(&full[s], (uint32_t)((i / kStages) & 1)));
    TileRef tr = locate_tile<TN>(t_begin + i, lvl_tiles, seg_s, G.T, stream_base, G.region_off);
    const unsigned char* Kt = tiles + (size_t)s * 2 * kTileBytes;
    const unsigned char* Vt = Kt + kTileBytes;
    const float lvl = (float)tr.level;
    if (!arrived) tr.rows = 0;   // skip the tile; the CTA agrees on the failure below
#pragma unroll 1
    for (int base = warp * 4; base < tr.rows; base += 4 * kWarps) {
      const int tok = base + grp;
      const bool valid = tok < tr.rows;
      // ---- q.k: 8 lanes per token
      float dot[GQ];
#pragma unroll
      for (int h = 0; h < GQ; ++h) dot[h] = 0.f;
#pragma unroll
      for (int i8 = 0; i8 < DPL; i8 += 8) {
        float kf[8];
        load8<kBf16>(Kt + (size_t)(valid ? tok : 0) * D * esz, sub * DPL + i8, kf);
#pragma unroll
        for (int h = 0; h < GQ; ++h)
#pragma unroll
          for (int k = 0; k < 8; ++k) dot[h] = fmaf(qr[h][i8 + k], kf[k], dot[h]);
      }
      float mx_new[GQ];
      bool grew = false;
#pragma unroll
      for (int h = 0; h < GQ; ++h) {
        float v = dot[h];
        v += __shfl_xor_sync(0xffffffffu, v, 1);
        v += __shfl_xor_sync(0xffffffffu, v, 2);
        v += __shfl_xor_sync(0xffffffffu, v, 4);
        v = valid ? v + lvl : -INFINITY;
        dot[h] = v;
        float mx = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, 8));
        mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 16));
        mx_new[h] = fmaxf(m_run[h], mx);
        grew |= mx_new[h] > m_run[h];
      }
      if (grew) {   // warp-uniform
#pragma unroll
        for (int h = 0; h < GQ; ++h) {
          const float a = exp2f(m_run[h] - mx_new[h]);   // m_run = -inf -> 0; mx_new is finite here
          l_run[h] *= a;
#pragma unroll
          for (int c = 0; c < CPL; ++c) acc[h][c] *= a;
          m_run[h] = mx_new[h];
        }
      }
      float p[GQ];
#pragma unroll
      for (int h = 0; h < GQ; ++h) {
        p[h] = valid ? exp2f(dot[h] - m_run[h]) : 0.f;
        if (sub == 0) l_run[h] += p[h];      // one lane per token carries the sum
      }
      // ---- p.v: every lane owns CPL columns
#pragma unroll
      for (int tk = 0; tk < 4; ++tk) {
        if (base + tk < tr.rows) {   // warp-uniform
          float vf[CPL];
          const unsigned char* vrow = Vt + (size_t)(base + tk) * D * esz;
          if constexpr (kBf16) {
            if constexpr (CPL == 4) {
              const uint2 w = *reinterpret_cast<const uint2*>(vrow + lane * 8);
              vf[0] = bf16_lo(w.x); vf[1] = bf16_hi(w.x); vf[2] = bf16_lo(w.y); vf[3] = bf16_hi(w.y);
            } else {
              const uint32_t w = *reinterpret_cast<const uint32_t*>(vrow + lane * 4);
              vf[0] = bf16_lo(w); vf[1] = bf16_hi(w);
            }
          } else {
            if constexpr (CPL == 4) {
              const float4 w = *reinterpret_cast<const float4*>(vrow + lane * 16);
              vf[0] = w.x; vf[1] = w.y; vf[2] = w.z; vf[3] = w.w;
            } else {
              const float2 w = *reinterpret_cast<const float2*>(vrow + lane * 8);
              vf[0] = w.x; vf[1] = w.y;
            }
          }
#pragma unroll
          for (int h = 0; h < GQ; ++h) {
            const float ph = __shfl_sync(0xffffffffu, p[h], tk * 8);
#pragma unroll
            for (int c = 0; c < CPL; ++c) acc[h][c] = fmaf(ph, vf[c], acc[h][c]);
          }
        }
      }
    }
    // stage s fully consumed; the same barrier makes a timed-out wait a CTA-wide decision
    if (__syncthreads_or(!arrived)) { failed = true; break; }
    if (tid == 0 && i + kStages < my_tiles) issue(i + kStages);
  }
  if (failed) {
    if (lane == 0) atomicCAS(status, kStatusOk, kStatusWaitTimeout);
  }
  __syncthreads();

  // ---- merge the 8 warps through shared memory (the tile ring is idle now)
  float* mrg = reinterpret_cast<float*>(tiles);        // [kWarps][GQ][PS]
#pragma unroll
  for (int h = 0; h < GQ; ++h) {
    float l = l_run[h];
    l += __shfl_xor_sync(0xffffffffu, l, 8);
    l += __shfl_xor_sync(0xffffffffu, l, 16);
    l = __shfl_sync(0xffffffffu, l, 0);
    float* row = mrg + ((size_t)warp * GQ + h) * PS;
#pragma unroll
    for (int c = 0; c < CPL; ++c) row[lane * CPL + c] = acc[h][c];
    if (lane == 0) { row[D] = m_run[h]; row[D + 1] = l; }
  }
  __syncthreads();
  float* my_part = part + ((size_t)sl * splits + split) * GQ * PS;
  for (int i = tid; i < GQ * D; i += kThreads) {
    const int h = i / D, c = i % D;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) M = fmaxf(M, mrg[((size_t)w * GQ + h) * PS + D]);
    float o = 0.f, L = 0.f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
      const float* row = mrg + ((size_t)w * GQ + h) * PS;
      const float sc = row[D] == -INFINITY ? 0.f : exp2f(row[D] - M);
      o = fmaf(row[c], sc, o);
      L = fmaf(row[D + 1], sc, L);
    }
    my_part[h * PS + c] = o;
    if (c == 0) { my_part[h * PS + D] = M; my_part[h * PS + D + 1] = L; }
  }
  // ---- ticket: the last CTA of the stream combines the splits
  __threadfence();
  __syncthreads();
  if (tid == 0) {
    const unsigned old = atomicAdd(&tickets[sl], 1u);
    is_last_s = old == (unsigned)(splits - 1);
  }
  __syncthreads();
  if (!is_last_s) return;
  __threadfence();
  const float* sp = part + (size_t)sl * splits * GQ * PS;
  for (int i = tid; i < GQ * D; i += kThreads) {
    const int h = i / D, c = i % D;
    float M = -INFINITY;
    for (int s = 0; s < splits; ++s) M = fmaxf(M, __ldcg(sp + ((size_t)s * GQ + h) * PS + D));
    float o = 0.f, L = 0.f;
    for (int s = 0; s < splits; ++s) {
      const float* row = sp + ((size_t)s * GQ + h) * PS;
      const float ms = __ldcg(row + D);
      const float sc = ms == -INFINITY ? 0.f : exp2f(ms - M);
      o = fmaf(__ldcg(row + c), sc, o);
      L = fmaf(__ldcg(row + D + 1), sc, L);
    }
    const float r = L > 0.f ? o / L : 0.f;
    const size_t off = ((size_t)seq * (G.H * GQ) + head * GQ + h) * D + c;
    if constexpr (kBf16) static_cast<__nv_bfloat16*>(out)[off] = __float2bfloat16_rn(r);
    else static_cast<float*>(out)[off] = r;
  }
  if (tid == 0) tickets[sl] = 0;   // ready for the next launch
}

template <bool kBf16, int D, int GQ>
cudaError_t launch_t(const Geom& G, const Arena& A, int layer, const void* q, void* out, float* scratch,
                     int splits, int* status, cudaStream_t st) {
  auto kern = decode_kernel<kBf16, D, GQ>;
  const size_t smem = (size_t)kStages * 2 * kTileBytes + kStages * sizeof(uint64_t);
  // the attribute belongs to the (kernel, device) pair: once per device that launches this instance
  static bool configured[kMaxDevices] = {};
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices || !configured[dev]) {
    e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    if (dev >= 0 && dev < kMaxDevices) configured[dev] = true;
  }
  const int n_sl = G.B * G.H;
  unsigned* tickets = reinterpret_cast<unsigned*>(scratch);
  float* part = scratch + ((n_sl + 63) / 64) * 64;
  dim3 grid(n_sl, splits);
  kern<<<grid, kThreads, smem, st>>>(G, A, layer, q, out, part, tickets, status);
  return cudaGetLastError();
}

template <bool kBf16, int D>
cudaError_t launch_g(const Geom& G, const Arena& A, int layer, const void* q, void* out, float* scratch,
                     int splits, int* status, cudaStream_t st) {
  switch (G.g) {
    case 1: return launch_t<kBf16, D, 1>(G, A, layer, q, out, scratch, splits, status, st);
    case 2: return launch_t<kBf16, D, 2>(G, A, layer, q, out, scratch, splits, status, st);
    case 3: return launch_t<kBf16, D, 3>(G, A, layer, q, out, scratch, splits, status, st);
    case 4: return launch_t<kBf16, D, 4>(G, A, layer, q, out, scratch, splits, status, st);
    case 5: return launch_t<kBf16, D, 5>(G, A, layer, q, out, scratch, splits, status, st);
    case 6: return launch_t<kBf16, D, 6>(G, A, layer, q, out, scratch, splits, status, st);
    case 7: return launch_t<kBf16, D, 7>(G, A, layer, q, out, scratch, splits, status, st);
    case 8: return launch_t<kBf16, D, 8>(G, A, layer, q, out, scratch, splits, status, st);
  }
  return cudaErrorInvalidValue;
}

}  // namespace

// Scratch layout: ticket counters (zero-initialised once by the owner; self-resetting),
// then per (stream, split, head) partial rows of D+2 floats.
size_t decode_scratch_bytes(const Geom& G, int splits) {
  const size_t n_sl = (size_t)G.B * G.H;
  return sizeof(float) * (((n_sl + 63) / 64) * 64 + n_sl * splits * G.g * (G.d + 8));   // rows of d + 8 floats cover both decode kernels' layouts
}

cudaError_t launch_decode(const Geom& G, const Arena& A, int layer, const void* q, void* out, float* scratch,
                          int splits, int* status, cudaStream_t st) {
  if (G.d == 128) return G.is_bf16 ? launch_g<true, 128>(G, A, layer, q, out, scratch, splits, status, st)
                                   : launch_g<false, 128>(G, A, layer, q, out, scratch, splits, status, st);
  if (G.d == 64) return G.is_bf16 ? launch_g<true, 64>(G, A, layer, q, out, scratch, splits, status, st)
                                  : launch_g<false, 64>(G, A, layer, q, out, scratch, splits, status, st);
  return cudaErrorInvalidValue;
}

}  // namespace bkv
