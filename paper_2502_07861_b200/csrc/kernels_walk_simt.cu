// SoftmaxBalance (Algorithm 2) on CUDA cores: one CTA per call.
//
// For every token j of the call, in stream order,
//   S_j   = sum_{i<j} eta_i * Ghat_ij,   Ghat_ij = exp((<k_i,k_j> - r_key^2)/sqrt d) <v_i,v_j> / r_value^2
//         = y^T eta / R^2 of Algorithm 2 (kernel identity from the proof of Theorem 3.2),
//   eta_j = +1 iff u_j < 1/2 - S_j/(2c)   <=>   S_j < c (1 - 2 u_j),
// with u_j the Philox uniform of (seed, layer, head, call ordinal, level, j).
//
// The kernel never materialises Ghat in global memory: 64-row panels of K and V are staged
// in shared memory as fp32, 64x64 tiles of Ghat are formed with FFMA, off-diagonal tiles are
// folded into the panel's partial correlations with the (already final) signs of earlier
// panels, and the diagonal tile is consumed by a one-warp sequential walk in which lane l
// owns token l of a 32-token group and the signs travel by warp shuffle.
// All accumulation is fp32 in a fixed order, so two runs give identical bits.
#include "common.cuh"

namespace bkv {

namespace {

constexpr int kPanel = 64;
constexpr int kThreads = 256;

template <int D>
struct SimtSmem {
  static constexpr int kStride = D + 4;
  static constexpr size_t panel_floats = (size_t)kPanel * kStride;
  static size_t bytes(int t) {
    return sizeof(float) * (4 * panel_floats + (size_t)kPanel * (kPanel + 1) + kPanel + 3 * (size_t)t);
  }
};

template <bool kBf16, int D>
__device__ inline void load_panel(float* __restrict__ dst, const void* __restrict__ base, int64_t row0) {
  constexpr int kStride = D + 4;
  constexpr int chunks = D / 8;
  const int esz = kBf16 ? 2 : 4;
  for (int i = threadIdx.x; i < kPanel * chunks; i += kThreads) {
    const int r = i / chunks, c = i % chunks;
    float v[8];
    load8<kBf16>(static_cast<const char*>(base) + (size_t)(row0 + r) * D * esz, c * 8, v);
    float4* o = reinterpret_cast<float4*>(dst + r * kStride + c * 8);
    o[0] = make_float4(v[0], v[1], v[2], v[3]);
    o[1] = make_float4(v[4], v[5], v[6], v[7]);
  }
}

template <bool kBf16, int D>
__global__ void __launch_bounds__(kThreads, 1)
walk_simt_kernel(Geom G, Arena A, const CallDesc* __restrict__ calls, int level,
                 const CallStat* __restrict__ stats, const float* __restrict__ tok_shift,
                 int8_t* __restrict__ eta_out, int8_t* __restrict__ dbg_eta, float* __restrict__ dbg_S,
                 float* __restrict__ dbg_p, unsigned long long* __restrict__ fail_count) {
  constexpr int kStride = D + 4;
  extern __shared__ __align__(16) float smem[];
  float* Kr = smem;
  float* Vr = Kr + kPanel * kStride;
  float* Kc = Vr + kPanel * kStride;
  float* Vc = Kc + kPanel * kStride;
  float* Gs = Vc + kPanel * kStride;               // [64][65]
  float* s_row = Gs + kPanel * (kPanel + 1);       // [64]
  float* eta_s = s_row + kPanel;                   // [t]
  float* thr_s = eta_s + G.t;                      // [t]
  float* shift_s = thr_s + G.t;                    // [t]

  const int call = blockIdx.x;
  const CallDesc C = calls[call];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int t = G.t;
  const int head = C.stream % G.H;
  const int layer = (C.stream / G.H) % G.L;
  const int seq = C.stream / (G.H * G.L);
  const float rk2 = G.fixed_rk2 > 0.f ? G.fixed_rk2 : stats[call].rk2;
  const float rv2 = G.fixed_rv2 > 0.f ? G.fixed_rv2 : stats[call].rv2;
  const float inv_rv2 = rv2 > 0.f ? 1.0f / rv2 : 0.f;
  const float scale = 1.4426950408889634f * G.inv_sqrt_d;
  const float c = G.c;

  for (int j = tid; j < t; j += kThreads) {
    const float u = walk_uniform(G.seed + (uint64_t)seq, layer, head, C.ordinal, level, j);
    thr_s[j] = c * (1.0f - 2.0f * u);
    shift_s[j] = tok_shift ? tok_shift[(size_t)call * t + j] : 0.f;
  }

  const int ty = tid >> 4, tx = tid & 15;
  int fails = 0;
  for (int r = 0; r < t / kPanel; ++r) {
    __syncthreads();  // previous panel fully consumed
    load_panel<kBf16, D>(Kr, A.K, C.src_row + (int64_t)r * kPanel);
    load_panel<kBf16, D>(Vr, A.V, C.src_row + (int64_t)r * kPanel);
    if (tid < kPanel) s_row[tid] = 0.f;
    for (int cp = 0; cp <= r; ++cp) {
      if (cp < r) {
        load_panel<kBf16, D>(Kc, A.K, C.src_row + (int64_t)cp * kPanel);
        load_panel<kBf16, D>(Vc, A.V, C.src_row + (int64_t)cp * kPanel);
      }
      __syncthreads();
      const float* Kcol = cp < r ? Kc : Kr;
      const float* Vcol = cp < r ? Vc : Vr;
      // ---- 64x64 tile: thread (ty,tx) owns rows ty+16a, cols tx+16b
      float kk[4][4], vv[4][4];
#pragma unroll
      for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) { kk[a][b] = 0.f; vv[a][b] = 0.f; }
#pragma unroll 2
      for (int e = 0; e < D; e += 4) {
        float4 kr[4], kc[4], vr[4], vc[4];
#pragma unroll
        for (int a = 0; a < 4; ++a) {
          kr[a] = *reinterpret_cast<const float4*>(Kr + (ty + 16 * a) * kStride + e);
          vr[a] = *reinterpret_cast<const float4*>(Vr + (ty + 16 * a) * kStride + e);
          kc[a] = *reinterpret_cast<const float4*>(Kcol + (tx + 16 * a) * kStride + e);
          vc[a] = *reinterpret_cast<const float4*>(Vcol + (tx + 16 * a) * kStride + e);
        }
#pragma unroll
        for (int a = 0; a < 4; ++a)
#pragma unroll
          for (int b = 0; b < 4; ++b) {
            kk[a][b] = fmaf(kr[a].x, kc[b].x, kk[a][b]);
            kk[a][b] = fmaf(kr[a].y, kc[b].y, kk[a][b]);
            kk[a][b] = fmaf(kr[a].z, kc[b].z, kk[a][b]);
            kk[a][b] = fmaf(kr[a].w, kc[b].w, kk[a][b]);
            vv[a][b] = fmaf(vr[a].x, vc[b].x, vv[a][b]);
            vv[a][b] = fmaf(vr[a].y, vc[b].y, vv[a][b]);
            vv[a][b] = fmaf(vr[a].z, vc[b].z, vv[a][b]);
            vv[a][b] = fmaf(vr[a].w, vc[b].w, vv[a][b]);
          }
      }
#pragma unroll
      for (int a = 0; a < 4; ++a)
#pragma unroll
        for (int b = 0; b < 4; ++b) {
          const int row = ty + 16 * a, col = tx + 16 * b;
          const float ex = (kk[a][b] - shift_s[r * kPanel + row] - shift_s[cp * kPanel + col] - rk2) * scale;
          Gs[row * (kPanel + 1) + col] = exp2f(ex) * (vv[a][b] * inv_rv2);
        }
      __syncthreads();
      if (cp < r) {
        // fold the tile into the panel's partial correlations: 4 threads per row
        const int row = tid >> 2, part = tid & 3;
        float acc = 0.f;
#pragma unroll
        for (int q = 0; q < 16; ++q) {
          const int col = part * 16 + q;
          acc = fmaf(Gs[row * (kPanel + 1) + col], eta_s[cp * kPanel + col], acc);
        }
        acc += __shfl_xor_sync(0xffffffffu, acc, 1);
        acc += __shfl_xor_sync(0xffffffffu, acc, 2);
        if (part == 0) s_row[row] += acc;
      } else if (warp == 0) {
        // the sequential walk over the panel's 64 tokens, 32 at a time
        for (int grp = 0; grp < 2; ++grp) {
          const int row = grp * 32 + lane;
          const int jg = r * kPanel + row;
          float S = s_row[row];
          if (grp == 1) {
#pragma unroll
            for (int col = 0; col < 32; ++col) S = fmaf(Gs[row * (kPanel + 1) + col], eta_s[r * kPanel + col], S);
          }
          float g[32];
#pragma unroll
          for (int j = 0; j < 32; ++j) g[j] = j < lane ? Gs[row * (kPanel + 1) + grp * 32 + j] : 0.f;
          const float thr = thr_s[jg];
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            const float dec = S < thr ? 1.0f : -1.0f;
            const float ej = __shfl_sync(0xffffffffu, dec, j);
            S = fmaf(ej, g[j], S);   // g[j] = 0 once this lane's token is decided
          }
          const float my_eta = S < thr ? 1.0f : -1.0f;
          eta_s[jg] = my_eta;
          if (fabsf(S) > c) ++fails;   // FAIL of Algorithm 2: counted, decision already clamped
          if (C.dbg_off >= 0) {
            dbg_S[C.dbg_off + jg] = S;
            dbg_p[C.dbg_off + jg] = 0.5f - fminf(fmaxf(S, -c), c) / (2.0f * c);
          }
          __syncwarp();
        }
      }
    }
  }
  __syncthreads();
  for (int j = tid; j < t; j += kThreads) {
    const int8_t e = eta_s[j] > 0.f ? 1 : -1;
    eta_out[(size_t)call * t + j] = e;
    if (C.dbg_off >= 0) dbg_eta[C.dbg_off + j] = e;
  }
  if (warp == 0) {
    fails = (int)__reduce_add_sync(0xffffffffu, (unsigned)fails);
    if (lane == 0 && fails) atomicAdd(fail_count, (unsigned long long)fails);
  }
}

template <bool kBf16, int D>
cudaError_t launch_one(const Geom& G, const Arena& A, const CallDesc* calls, int n_calls, int level,
                       const CallStat* stats, const float* tok_shift, int8_t* eta, int8_t* dbg_eta, float* dbg_S,
                       float* dbg_p, unsigned long long* fail_count, cudaStream_t st) {
  const size_t smem = SimtSmem<D>::bytes(G.t);
  auto kern = walk_simt_kernel<kBf16, D>;
  cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (e != cudaSuccess) return e;
  kern<<<n_calls, kThreads, smem, st>>>(G, A, calls, level, stats, tok_shift, eta, dbg_eta, dbg_S, dbg_p, fail_count);
  return cudaGetLastError();
}

}  // namespace

int walk_simt_supported(int d) { return d == 64 || d == 128; }

size_t walk_simt_smem_bytes(int d, int t) { return d == 64 ? SimtSmem<64>::bytes(t) : SimtSmem<128>::bytes(t); }

cudaError_t launch_walk_simt(const Geom& G, const Arena& A, const CallDesc* calls, int n_calls, int level,
                             const CallStat* stats, const float* tok_shift, int8_t* eta, int8_t* dbg_eta,
                             float* dbg_S, float* dbg_p, unsigned long long* fail_count, cudaStream_t st) {
  if (n_calls <= 0) return cudaSuccess;
  if (G.d == 128) {
    return G.is_bf16 ? launch_one<true, 128>(G, A, calls, n_calls, level, stats, tok_shift, eta, dbg_eta, dbg_S, dbg_p, fail_count, st)
                     : launch_one<false, 128>(G, A, calls, n_calls, level, stats, tok_shift, eta, dbg_eta, dbg_S, dbg_p, fail_count, st);
  }
  if (G.d == 64) {
    return G.is_bf16 ? launch_one<true, 64>(G, A, calls, n_calls, level, stats, tok_shift, eta, dbg_eta, dbg_S, dbg_p, fail_count, st)
                     : launch_one<false, 64>(G, A, calls, n_calls, level, stats, tok_shift, eta, dbg_eta, dbg_S, dbg_p, fail_count, st);
  }
  return cudaErrorInvalidValue;
}

}  // namespace bkv
