// Shared device/host declarations of the BalanceKV CUDA library (sm_100a).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace bkv {

constexpr int kMaxLevels = 8;      // T <= 8
constexpr int kMaxGroup = 8;       // query heads per KV head

// One SoftmaxBalance call (Algorithm 2) of a batched launch.
struct CallDesc {
  int64_t src_row;        // first row of the call's t tokens in the arena
  int64_t dst_row;        // first row the t/2 survivors are written to
  int64_t dbg_off;        // element offset of the call's debug record, or -1
  int32_t stream;         // (seq * L + layer) * H + head
  int32_t ordinal;        // call ordinal inside its level (Philox coordinate)
};

// One append (or level load) of a batched launch.
struct AppendDesc {
  int64_t dst_row;    // first destination row in the arena
  int64_t src_off;    // element offset of the first source row in the caller's tensor
  int32_t stream;
  int32_t n;          // rows
  int32_t idx0;       // original position of the first row (when no index array is given)
  int32_t level;      // segment to update
  int32_t new_len;    // segment length after the copy
  int32_t pad;
};

// Value-norm buckets (Algorithm 1): per-stream input and result of the routing pass, and the
// destination of one (stream, bucket) pair in the arena.
constexpr int kMaxBuckets = 8;
struct BucketIn {
  float prev_vmax2;        // v_max^2 over the stream's earlier blocks
  int32_t prev_erase_max;  // largest bucket index erased so far (INT32_MIN: none)
};
struct BucketOut {
  int32_t count[kMaxBuckets];  // tokens of the block per slot
  int32_t dropped;             // zero values, erased buckets, indices below the lowest slot
  int32_t above;               // tokens above the highest slot (the block is then refused)
  int32_t erase_max;           // largest erased bucket index after the block
  float vmax2;                 // v_max^2 after the block
};
struct BucketDst {
  int64_t dst_row;    // arena row that receives the slot's first token of the block
  int32_t idx0;       // that token's position in the instance's stream
  int32_t stream;     // instance's stream (segment table row); -1: nothing to update
  int32_t new_len;    // level-0 length after the block
  int32_t pad;
};

// One move of a stream's level-0 remainder to the front of its region.
struct MoveDesc {
  int64_t src_row, dst_row;
  int32_t stream, n;
};

struct SegUpdate {  // seg[index] = {start, len}
  int32_t index, start, len, pad;
};

struct Seg {  // one level of one stream: rows [start, start+len) of the level's region
  int32_t start, len;
};

// Per-call radii of Algorithm 2 and the key shift.
struct CallStat {
  float rk2, rv2;    // r_key^2, r_value^2
};

// Geometry shared by every kernel.
struct Geom {
  int32_t d, t, T, H, L, B, g;
  int32_t is_bf16;
  int64_t rows_per_stream;            // R
  int32_t region_off[kMaxLevels + 1]; // first row of level l's region inside a stream
  float inv_sqrt_d;
  float c;                            // walk constant, single precision
  float fixed_rk2, fixed_rv2;         // > 0: fixed radii
  uint64_t seed;
  int32_t center_keys;
};

enum DeviceStatus : int { kStatusOk = 0, kStatusWaitTimeout = 1, kStatusBadIndex = 2 };

// ------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al., SC'11), from its published definition.
// ------------------------------------------------------------------------------------
__host__ __device__ inline void philox4x32_10(uint32_t k0, uint32_t k1, uint32_t c0, uint32_t c1,
                                              uint32_t c2, uint32_t c3, uint32_t out[4]) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    if (r > 0) { k0 += 0x9E3779B9u; k1 += 0xBB67AE85u; }
    const uint64_t p0 = (uint64_t)0xD2511F53u * c0;
    const uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
    const uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
    const uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
    c1 = (uint32_t)p1; c3 = (uint32_t)p0; c0 = n0; c2 = n2;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// 24-bit uniform of the walk's coin for token j of call (layer, head, ordinal, level).
__host__ __device__ inline float walk_uniform(uint64_t seed, int layer, int head, int ordinal, int level, int j) {
  uint32_t r[4];
  philox4x32_10((uint32_t)seed, (uint32_t)(seed >> 32), (uint32_t)j, (uint32_t)ordinal, (uint32_t)level,
                ((uint32_t)layer << 16) | ((uint32_t)head & 0xffffu), r);
  return (float)(r[0] >> 8) * (1.0f / 16777216.0f);
}

// ------------------------------------------------------------------------------------
// element access
// ------------------------------------------------------------------------------------
__device__ inline float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ inline float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }

// Load 8 consecutive elements starting at element index `e` (multiple of 8) of a row.
template <bool kBf16>
__device__ inline void load8(const void* row, int e, float out[8]) {
  if constexpr (kBf16) {
    const uint4 w = *reinterpret_cast<const uint4*>(reinterpret_cast<const __nv_bfloat16*>(row) + e);
    out[0] = bf16_lo(w.x); out[1] = bf16_hi(w.x); out[2] = bf16_lo(w.y); out[3] = bf16_hi(w.y);
    out[4] = bf16_lo(w.z); out[5] = bf16_hi(w.z); out[6] = bf16_lo(w.w); out[7] = bf16_hi(w.w);
  } else {
    const float4 a = *reinterpret_cast<const float4*>(reinterpret_cast<const float*>(row) + e);
    const float4 b = *reinterpret_cast<const float4*>(reinterpret_cast<const float*>(row) + e + 4);
    out[0] = a.x; out[1] = a.y; out[2] = a.z; out[3] = a.w;
    out[4] = b.x; out[5] = b.y; out[6] = b.z; out[7] = b.w;
  }
}

__device__ inline float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ inline int warp_sum_int(int v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ inline float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// ------------------------------------------------------------------------------------
// launchers (implemented in the kernel files)
// ------------------------------------------------------------------------------------
struct Arena {
  void* K;          // [n_streams * R, d]
  void* V;
  int32_t* idx;     // [n_streams * R] original token position
  Seg* seg;         // [n_streams, T+1]
  float2* nrm;      // [n_streams * R] (||k||^2, ||v||^2) of every stored row, written with the row (null: not kept)
};

cudaError_t launch_append(const Geom& G, const Arena& A, const AppendDesc* descs, int n_desc, int max_rows,
                          const void* Ksrc, const void* Vsrc, const int32_t* idx_src, cudaStream_t st);
cudaError_t launch_append_uniform(const Geom& G, const Arena& A, int layer, int level, int rel_row, int idx0, int n,
                                  int new_len, const void* Ksrc, const void* Vsrc, const int32_t* idx_src,
                                  cudaStream_t st);
cudaError_t launch_move(const Geom& G, const Arena& A, const MoveDesc* descs, int n_desc, int max_rows,
                        cudaStream_t st);
cudaError_t launch_radii(const Geom& G, const Arena& A, const CallDesc* calls, int n_calls, CallStat* stats,
                         float* tok_shift, cudaStream_t st);
cudaError_t launch_walk_simt(const Geom& G, const Arena& A, const CallDesc* calls, int n_calls, int level,
                             const CallStat* stats, const float* tok_shift, int8_t* eta, int8_t* dbg_eta,
                             float* dbg_S, float* dbg_p, unsigned long long* fail_count, cudaStream_t st);
cudaError_t launch_walk_tc(const Geom& G, const Arena& A, const CallDesc* calls, int n_calls, int level,
                           const CallStat* stats, const float* tok_shift, int8_t* eta, int8_t* dbg_eta,
                           float* dbg_S, float* dbg_p, unsigned long long* fail_count, int* status,
                           const void* tmap_k, const void* tmap_v, cudaStream_t st);
cudaError_t launch_compact(const Geom& G, const Arena& A, const CallDesc* calls, int n_calls, int level,
                           const int8_t* eta, cudaStream_t st);
size_t decode_scratch_bytes(const Geom& G, int splits);
cudaError_t launch_decode(const Geom& G, const Arena& A, int layer, const void* q, void* out, float* scratch,
                          int splits, int* status, cudaStream_t st);
cudaError_t launch_fill_weights(float* w, int n, float value, cudaStream_t st);
cudaError_t launch_seg_update(const Arena& A, const SegUpdate* ups, int n, cudaStream_t st);
int bucket_scan_chunks(int n);
size_t bucket_chunk_count_ints(int n_sl, int n);   // ints of the per-chunk count table of the routing pass
cudaError_t launch_bucket_route(const Geom& G, const void* V, int n_sl, int n, int n_buckets, int i_top, float rho2,
                                const BucketIn* in, unsigned* vmax2_bits, float* ns, int8_t* slot, int32_t* rank,
                                int32_t* chunk_cnt, BucketOut* out, const int8_t* forced_slot, cudaStream_t st);
size_t anticorr_scratch_floats(int n_sl, int n, int d);
cudaError_t launch_anticorr_classes(const Geom& G, const void* K, int n_sl, int n, float tau, float* scratch, int8_t* cls,
                                    cudaStream_t st);
cudaError_t launch_bucket_scatter(const Geom& G, const Arena& A, const void* K, const void* V, int n_sl, int n,
                                  int n_buckets, const int8_t* slot, const int32_t* rank, const int32_t* chunk_base,
                                  const float* ns, const BucketDst* dst, cudaStream_t st);
int walk_simt_supported(int d);
size_t walk_simt_smem_bytes(int d, int t);

}  // namespace bkv
