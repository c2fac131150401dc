// Split-K decode attention over the weighted compressed cache, bf16 / d = 128, on tensor cores.
//
//   out = sum_i w_i e^{<k_i,q>/sqrt d} v_i / sum_i w_i e^{<k_i,q>/sqrt d},   w_i = 2^level(i)
//
// (output ratio of Algorithm 1 / estimator of Theorem 3.3 over the sets C^T..C^0 of a stream;
// Eq. (1) when every token sits in C^0).  The g <= 8 query heads of a KV head form the rows of a
// 16-row MMA tile, so q.K^T and p.V each cost one mma.sync.m16n8k16 per 8 tokens x 16 dims: at
// g = 5 the CUDA-core formulation needs ~65 instructions per token and is issue bound far below
// HBM speed, this one needs ~6.
//
// Grid (streams of the layer, splits), 4 warps.  A CTA walks its share of the stream's 64-token
// tiles through a 3-stage ring filled by TMA (tensor maps over the K and V arenas, boxes of
// 64 dims x 64 rows, 128-byte swizzle, so ldmatrix reads are bank-conflict free).  Warp w owns
// tokens 16w..16w+15 of a tile and keeps a private online softmax (running max, sum, 16 x 128
// accumulator) in registers; warps merge through shared memory, splits through a global scratch
// and a ticket counter (the last CTA of a stream combines; nobody waits).
// Fused decode step: with k_new / v_new given, the launch also appends one token per stream
// (Algorithm 3's C^0 <- C^0 + {(k_j, v_j)}).  The new token never goes through the tiles: the
// combining CTA scores it in fp32, adds it as one more partial (weight 1) and only then writes
// its row, its position and the stream's new level-0 length, after every CTA of the stream has
// taken its ticket, i.e. has finished reading the old segment table.
// Rows of a tile beyond a segment's end are masked in the scores; their V rows are whatever the
// arena holds there (zero-initialised at creation or finite older rows) times an exact zero.
#include <cuda.h>

#include "common.cuh"

namespace bkv {

namespace {

constexpr int kThreads = 128;
constexpr int kWarps = 4;
constexpr int kStages = 3;
constexpr int kTN = 64;                      // tokens per tile
constexpr int kD = 128;
constexpr uint32_t kHalf = kTN * 128;        // bytes of one [64 tokens][64 dims] bf16 box
constexpr uint32_t kTensorBytes = 2 * kHalf; // K (or V) tile: two boxes
constexpr uint32_t kStageBytes = 2 * kTensorBytes;
constexpr long long kWaitCycles = 4000000000LL;
constexpr int PS = kD + 4;                   // partial row: acc[D], max, sum, 2 pad (rows stay 16-byte aligned)

struct DecodeMaps {
  CUtensorMap k, v;
};

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
__device__ inline bool mbar_wait(uint64_t* bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (clock64() - t0 > kWaitCycles) return false;
  }
  return true;
}
__device__ inline void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y) : "memory");
}
__device__ inline void ldsm_x4(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ inline void ldsm_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
  asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0, %1, %2, %3}, [%4];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ inline void mma_bf16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
      : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ inline uint32_t pack_bf16(float lo, float hi) {
  const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<const uint32_t*>(&v);
}
// Byte offset of (token row, 16-byte chunk of dims) inside a K or V tile: two 64-dim boxes of
// 64 rows x 128 bytes, chunk index XORed with (row % 8) by the 128-byte swizzle.
__device__ inline uint32_t tile_off(int token, int chunk16) {   // chunk16 in [0, 16)
  return (uint32_t)(chunk16 >> 3) * kHalf + (uint32_t)token * 128u + (uint32_t)(((chunk16 & 7) ^ (token & 7)) << 4);
}

// One appended token per stream of the layer (lockstep fill): source rows [B*H, d] and where they go.
struct StepAppend {
  const __nv_bfloat16* k_new;   // nullptr: plain decode
  const __nv_bfloat16* v_new;
  int rel_row, idx0, new_len;   // row inside the level-0 region, original position, new level-0 length
  // Un-normalised result instead of the ratio (both nullptr: ratio in `out`): per query head
  // sum_i w_i e^{l_i - M} v_i as fp32 [B, H g, d] and (M, sum_i w_i e^{l_i - M}) as fp32 [B, H g, 2],
  // M the largest base-2 logit incl. log2 w_i.  Algorithm 1 divides the numerator of one
  // MergeAndReduce instance by the denominator of another; this is one such part.
  float* raw_acc;
  float* raw_ml;
  int keys_only;                // 1: only (M, sum) are wanted (a denominator instance): V is neither loaded nor multiplied
  // Segment table of the layer's streams when they are all alike (the host mirrors it): saves the
  // dependent global read at the start of a latency-bound launch.  n_seg = 0: read the table.
  int n_seg;
  Seg seg[kMaxLevels + 1];
  // One launch over several layer slots (decode merged over slots): blockIdx.z selects the slot.
  // n_slots = 0: a launch over the one slot `layer`.  z_stride: 4-byte words between the scratch
  // blocks (tickets, partial rows) of consecutive slots; raw_acc / raw_ml advance by one
  // [B, H g, d] / [B, H g, 2] block per slot; bit z of keys_mask = keys_only of slot z.
  int n_slots;
  int slot_layer[8];
  unsigned keys_mask;
  unsigned z_stride;
};

struct TileRef {
  int64_t row;
  int rows, level;
};
__device__ inline TileRef locate_tile(int tile, const int* lvl_tiles, const Seg* seg, int T, int64_t stream_base,
                                      const int32_t* region_off) {
  TileRef r{0, 0, 0};
  for (int l = T; l >= 0; --l) {
    const int nt = lvl_tiles[l];
    if (tile < nt) {
      r.level = l;
      r.row = stream_base + region_off[l] + seg[l].start + (int64_t)tile * kTN;
      r.rows = min(kTN, seg[l].len - tile * kTN);
      return r;
    }
    tile -= nt;
  }
  return r;
}

__global__ void __launch_bounds__(kThreads, 2)
decode_mma_kernel(Geom G, Arena A, int layer, const __nv_bfloat16* __restrict__ q, __nv_bfloat16* __restrict__ out,
                  float* __restrict__ part_base, unsigned* __restrict__ tickets_base, int* __restrict__ status,
                  const StepAppend ap, const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV) {
  float* part = part_base;
  unsigned* tickets = tickets_base;
  float* raw_acc = ap.raw_acc;
  float* raw_ml = ap.raw_ml;
  int keys_only = ap.keys_only;
  if (ap.n_slots) {
    const int z = blockIdx.z;
    layer = ap.slot_layer[z];
    keys_only = (int)((ap.keys_mask >> z) & 1u);
    part += (size_t)z * ap.z_stride;
    tickets += (size_t)z * ap.z_stride;
    raw_acc += (size_t)z * G.B * G.H * G.g * kD;
    raw_ml += (size_t)z * G.B * G.H * G.g * 2;
  }
  extern __shared__ unsigned char smem_raw[];
  unsigned char* tiles = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* full = reinterpret_cast<uint64_t*>(tiles + kStages * kStageBytes);
  __shared__ int lvl_tiles[kMaxLevels + 1];
  __shared__ Seg seg_s[kMaxLevels + 1];
  __shared__ int is_last_s;

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int g = G.g;
  const int sl = blockIdx.x;
  const int seq = sl / G.H, head = sl % G.H;
  const int stream = (seq * G.L + layer) * G.H + head;
  const int splits = gridDim.y, split = blockIdx.y;
  const int64_t stream_base = (int64_t)stream * G.rows_per_stream;

  // Launched with programmatic stream serialization, this grid may become resident while the
  // previous kernel of the stream is still finishing (the launch latency overlaps its tail);
  // nothing that kernel wrote is touched before the wait below.  Without the launch attribute
  // both instructions do nothing.
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  if (tid == 0) {
    for (int s = 0; s <= kStages; ++s) mbar_init(&full[s], 1);       // full[kStages]: the combine's bulk copy
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmK) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmV) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  asm volatile("griddepcontrol.wait;" ::: "memory");
  if (tid <= G.T) {
    const Seg s = ap.n_seg ? ap.seg[tid] : A.seg[(size_t)stream * (G.T + 1) + tid];
    seg_s[tid] = s;
    lvl_tiles[tid] = (s.len + kTN - 1) / kTN;
  }
  __syncthreads();
  int n_tiles = 0;
  for (int l = 0; l <= G.T; ++l) n_tiles += lvl_tiles[l];
  const int t_begin = (int)((long long)n_tiles * split / splits);
  const int t_end = (int)((long long)n_tiles * (split + 1) / splits);
  const int my_tiles = t_end - t_begin;

  auto issue = [&](int i) {   // thread 0 only
    const TileRef tr = locate_tile(t_begin + i, lvl_tiles, seg_s, G.T, stream_base, G.region_off);
    unsigned char* st = tiles + (size_t)(i % kStages) * kStageBytes;
    uint64_t* bar = &full[i % kStages];
    mbar_expect_tx(bar, keys_only ? kTensorBytes : kStageBytes);
    tma_load_2d(st, &tmK, 0, (int)tr.row, bar);
    tma_load_2d(st + kHalf, &tmK, 64, (int)tr.row, bar);
    if (!keys_only) {
      tma_load_2d(st + kTensorBytes, &tmV, 0, (int)tr.row, bar);
      tma_load_2d(st + kTensorBytes + kHalf, &tmV, 64, (int)tr.row, bar);
    }
  };
  if (tid == 0)
    for (int i = 0; i < min(kStages, my_tiles); ++i) issue(i);

  // A fragments of the query tile: row = query head of the group (rows >= g are zero)
  const int qrow = lane >> 2, qcol = (lane & 3) * 2;
  uint32_t qa[8][4];
  {
    const __nv_bfloat16* qp = q + ((size_t)seq * (G.H * g) + (size_t)head * g + qrow) * kD;
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
      uint32_t lo = 0, hi = 0;
      if (qrow < g) {
        lo = *reinterpret_cast<const uint32_t*>(qp + ks * 16 + qcol);
        hi = *reinterpret_cast<const uint32_t*>(qp + ks * 16 + 8 + qcol);
      }
      qa[ks][0] = lo; qa[ks][1] = 0; qa[ks][2] = hi; qa[ks][3] = 0;
    }
  }
  const float sc = 1.4426950408889634f * G.inv_sqrt_d;

  float o[16][4];
#pragma unroll
  for (int n = 0; n < 16; ++n) { o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f; }
  float m_run = -INFINITY, l_run = 0.f;      // of row qrow, over this thread's columns

  // ldmatrix row addresses of this lane (see the fragment layouts of mma.m16n8k16)
  const int mi = lane >> 3, mr = lane & 7;
  const int k_tok = warp * 16 + (mi >> 1) * 8 + mr, k_chunk = mi & 1;     // K: x4 = (tok 0-7 | 8-15) x (dims lo | hi)
  const int v_tok = warp * 16 + (mi & 1) * 8 + mr, v_chunk = mi >> 1;     // V (transposed): x4 = (dims lo | hi) x (tok 0-7 | 8-15)

  bool failed = false;
  for (int i = 0; i < my_tiles; ++i) {
    const int s = i % kStages;
    const bool arrived = __all_sync(0xffffffffu, mbar_wait(&full[s], (uint32_t)((i / kStages) & 1)));
    const TileRef tr = locate_tile(t_begin + i, lvl_tiles, seg_s, G.T, stream_base, G.region_off);
    const uint32_t Kt = smem_u32(tiles + (size_t)s * kStageBytes), Vt = Kt + kTensorBytes;
    if (arrived && warp * 16 < tr.rows) {
      // ---- scores of the 16 tokens of this warp: S[16 x 16] = Q K^T
      float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
      for (int ks = 0; ks < 8; ++ks) {
        uint32_t kb[4];
        ldsm_x4(Kt + tile_off(k_tok, ks * 2 + k_chunk), kb);
        mma_bf16(s0, qa[ks], kb[0], kb[1]);
        mma_bf16(s1, qa[ks], kb[2], kb[3]);
      }
      // this thread: row qrow, tokens tcol, tcol+1 (s0) and tcol+8, tcol+9 (s1)
      const int tcol = warp * 16 + qcol;
      const float lvl = (float)tr.level;
      float x0 = tcol < tr.rows ? fmaf(s0[0], sc, lvl) : -INFINITY;
      float x1 = tcol + 1 < tr.rows ? fmaf(s0[1], sc, lvl) : -INFINITY;
      float x2 = tcol + 8 < tr.rows ? fmaf(s1[0], sc, lvl) : -INFINITY;
      float x3 = tcol + 9 < tr.rows ? fmaf(s1[1], sc, lvl) : -INFINITY;
      float mx = fmaxf(fmaxf(x0, x1), fmaxf(x2, x3));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 1));
      mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, 2));
      const float m_new = fmaxf(m_run, mx);                   // finite: token 16 w of the tile is valid
      if (__any_sync(0xffffffffu, m_new > m_run)) {
        const float a = exp2f(m_run - m_new);                 // m_run = -inf -> 0
        l_run *= a;
#pragma unroll
        for (int n = 0; n < 16; ++n) { o[n][0] *= a; o[n][1] *= a; }
        m_run = m_new;
      }
      x0 = exp2f(x0 - m_run); x1 = exp2f(x1 - m_run); x2 = exp2f(x2 - m_run); x3 = exp2f(x3 - m_run);
      l_run += (x0 + x1) + (x2 + x3);
      // the probabilities enter the second MMA as bf16: split them into a high and a low part
      // (p = hi + lo to 16 bits) so that the output error stays that of the final rounding
      const uint32_t ph[4] = {pack_bf16(x0, x1), 0u, pack_bf16(x2, x3), 0u};
      const uint32_t pl[4] = {pack_bf16(x0 - bf16_lo(ph[0]), x1 - bf16_hi(ph[0])), 0u,
                              pack_bf16(x2 - bf16_lo(ph[2]), x3 - bf16_hi(ph[2])), 0u};
      // ---- O[16 x 128] += P[16 x 16] V[16 x 128]
      if (!keys_only)
#pragma unroll
      for (int nb = 0; nb < 8; ++nb) {
        uint32_t vb[4];
        ldsm_x4_trans(Vt + tile_off(v_tok, nb * 2 + v_chunk), vb);
        mma_bf16(o[2 * nb], ph, vb[0], vb[1]);
        mma_bf16(o[2 * nb], pl, vb[0], vb[1]);
        mma_bf16(o[2 * nb + 1], ph, vb[2], vb[3]);
        mma_bf16(o[2 * nb + 1], pl, vb[2], vb[3]);
      }
    }
    // stage s fully consumed; the same barrier makes a timed-out wait a CTA-wide decision
    if (__syncthreads_or(!arrived)) { failed = true; break; }
    if (tid == 0 && i + kStages < my_tiles) issue(i + kStages);
  }
  if (failed && tid == 0) atomicCAS(status, kStatusOk, kStatusWaitTimeout);
  __syncthreads();

  // ---- merge the 4 warps through shared memory (the tile ring is idle now)
  float* mrg = reinterpret_cast<float*>(tiles);        // [kWarps][g][PS]
  {
    float l = l_run;
    l += __shfl_xor_sync(0xffffffffu, l, 1);
    l += __shfl_xor_sync(0xffffffffu, l, 2);
    if (qrow < g) {
      float* rowp = mrg + ((size_t)warp * g + qrow) * PS;
#pragma unroll
      for (int n = 0; n < 16; ++n) { rowp[n * 8 + qcol] = o[n][0]; rowp[n * 8 + qcol + 1] = o[n][1]; }
      if ((lane & 3) == 0) { rowp[kD] = m_run; rowp[kD + 1] = l; }
    }
  }
  __syncthreads();
  // With a single split the CTA's partial is the stream's result: it stays in shared memory (behind
  // the merge buffer) and the ticket, the fences and the staging copy are skipped.
  constexpr uint32_t kSingleOff = 32768;
  const bool single = splits == 1;
  float* my_part = single ? reinterpret_cast<float*>(tiles + kSingleOff) : part + ((size_t)sl * splits + split) * g * PS;
  for (int i = tid; i < g * kD; i += kThreads) {
    const int h = i / kD, c = i % kD;
    float M = -INFINITY;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) M = fmaxf(M, mrg[((size_t)w * g + h) * PS + kD]);
    float acc = 0.f, L = 0.f;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
      const float* rowp = mrg + ((size_t)w * g + h) * PS;
      const float f = rowp[kD] == -INFINITY ? 0.f : exp2f(rowp[kD] - M);
      acc = fmaf(rowp[c], f, acc);
      L = fmaf(rowp[kD + 1], f, L);
    }
    my_part[h * PS + c] = acc;
    if (c == 0) { my_part[h * PS + kD] = M; my_part[h * PS + kD + 1] = L; }
  }
  // ---- ticket: the last CTA of the stream combines the splits
  if (!single) {
    __threadfence();
    __syncthreads();
    if (tid == 0) {
      const unsigned old = atomicAdd(&tickets[sl], 1u);
      is_last_s = old == (unsigned)(splits - 1);
    }
    __syncthreads();
    if (!is_last_s) return;
    __threadfence();
  } else {
    __syncthreads();
  }
  // Combine: first the (max, sum) pairs of all splits in one round of loads, then every thread
  // sums its output columns over the splits with independent loads.
  const float* sp = part + (size_t)sl * splits * g * PS;   // 16-byte aligned: rows of PS * 4 = 528 bytes
  float* cm = reinterpret_cast<float*>(tiles);            // [splits][g] max, later the scale factors
  float* cl = cm + 64 * kMaxGroup;                        // [splits][g] sums
  float* cM = cl + 64 * kMaxGroup;                        // [g] overall max
  float* cL = cM + kMaxGroup;                             // [g] overall sum
  float* cN = cL + kMaxGroup;                             // [g] factor of the appended token
  // All partial rows of the stream are contiguous.  If they fit, one bulk copy brings them into
  // the idle tile ring (a single round trip); otherwise they are read from global memory.
  constexpr uint32_t kStageOff = 8192;                     // behind cm, cl, cM, cL, cN
  const uint32_t part_bytes = (uint32_t)splits * g * PS * sizeof(float);
  const bool staged = single || part_bytes <= kStages * kStageBytes - kStageOff;
  const float* sp_s = reinterpret_cast<const float*>(tiles + (single ? kSingleOff : kStageOff));
  if (ap.k_new) {
    // append (every CTA of the stream has taken its ticket, so nobody reads the old segment table
    // any more): one 256-byte row of K and of V, the position, the new length of C^0.  Done first,
    // so that the writes drain while the partials are combined.
    const size_t dst_row = (size_t)stream_base + G.region_off[0] + ap.rel_row;
    if (warp == 0) {                                          // lanes 0-15: the row of K, lanes 16-31: the row of V
      const __nv_bfloat16* src = (lane < 16 ? ap.k_new : ap.v_new) + (size_t)sl * kD;
      __nv_bfloat16* dstp = static_cast<__nv_bfloat16*>(lane < 16 ? A.K : A.V) + dst_row * kD;
      const uint4 v = reinterpret_cast<const uint4*>(src)[lane & 15];
      reinterpret_cast<uint4*>(dstp)[lane & 15] = v;
      float s2 = 0.f;                                         // ||k||^2 / ||v||^2 travel with the row
      const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&v);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float2 f = __bfloat1622float2(h2[i]);
        s2 = fmaf(f.x, f.x, s2);
        s2 = fmaf(f.y, f.y, s2);
      }
#pragma unroll
      for (int o = 8; o > 0; o >>= 1) s2 += __shfl_xor_sync(0xffffffffu, s2, o);
      const float v2 = __shfl_sync(0xffffffffu, s2, 16);
      if (lane == 0 && A.nrm) A.nrm[dst_row] = make_float2(s2, v2);
    } else if (tid == 32) {
      A.idx[dst_row] = ap.idx0;
      A.seg[(size_t)stream * (G.T + 1)].len = ap.new_len;
    }
  }
  // the appended token's operands are requested now, so that their latency overlaps the staging:
  // per lane 4 dims of <q_h, k_new> for this warp's (up to two) heads, and this thread's first
  // four columns of v_new
  float dot_pre[2] = {0.f, 0.f};
  uint2 vn_pre = make_uint2(0u, 0u);
  if (ap.k_new) {
    const uint2 kn = *reinterpret_cast<const uint2*>(ap.k_new + (size_t)sl * kD + 4 * lane);
    const __nv_bfloat162 k01 = *reinterpret_cast<const __nv_bfloat162*>(&kn.x), k23 = *reinterpret_cast<const __nv_bfloat162*>(&kn.y);
#pragma unroll
    for (int hh = 0; hh < 2; ++hh) {
      const int h = warp + kWarps * hh;
      if (h < g) {
        const uint2 qv = *reinterpret_cast<const uint2*>(q + ((size_t)seq * (G.H * g) + (size_t)head * g + h) * kD + 4 * lane);
        const __nv_bfloat162 q01 = *reinterpret_cast<const __nv_bfloat162*>(&qv.x), q23 = *reinterpret_cast<const __nv_bfloat162*>(&qv.y);
        float d = __bfloat162float(q01.x) * __bfloat162float(k01.x);
        d = fmaf(__bfloat162float(q01.y), __bfloat162float(k01.y), d);
        d = fmaf(__bfloat162float(q23.x), __bfloat162float(k23.x), d);
        d = fmaf(__bfloat162float(q23.y), __bfloat162float(k23.y), d);
        dot_pre[hh] = d;
      }
    }
    if (tid < g * (kD / 4)) vn_pre = *reinterpret_cast<const uint2*>(ap.v_new + (size_t)sl * kD + (tid % (kD / 4)) * 4);
  }
  if (staged && !single) {
    if (tid == 0) {
      // earlier generic-proxy accesses to this shared memory and the other CTAs' global writes
      // (acquired above) come before the async-proxy copy
      asm volatile("fence.proxy.async;" ::: "memory");
      mbar_expect_tx(&full[kStages], part_bytes);
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                   ::"r"(smem_u32(tiles + kStageOff)), "l"(sp), "r"(part_bytes), "r"(smem_u32(&full[kStages])) : "memory");
    }
    const bool landed = mbar_wait(&full[kStages], 0u);
    if (__syncthreads_or(!landed)) {
      if (tid == 0) { atomicCAS(status, kStatusOk, kStatusWaitTimeout); tickets[sl] = 0; }
      return;
    }
  }
  if (staged) sp = sp_s;
  for (int i = tid; i < splits * g; i += kThreads) {
    const float* rowp = sp + (size_t)i * PS;
    cm[i] = staged ? rowp[kD] : __ldcg(rowp + kD);
    cl[i] = staged ? rowp[kD + 1] : __ldcg(rowp + kD + 1);
  }
  __syncthreads();
  for (int h = warp; h < g; h += kWarps) {     // one warp per head, lanes over the (<= 64) splits
    const int s0 = lane, s1 = lane + 32;
    const float m0 = s0 < splits ? cm[s0 * g + h] : -INFINITY, m1 = s1 < splits ? cm[s1 * g + h] : -INFINITY;
    const float M = warp_max(fmaxf(m0, m1));
    const float f0 = m0 == -INFINITY ? 0.f : exp2f(m0 - M), f1 = m1 == -INFINITY ? 0.f : exp2f(m1 - M);
    float L = (s0 < splits ? cl[s0 * g + h] * f0 : 0.f) + (s1 < splits ? cl[s1 * g + h] * f1 : 0.f);
    L = warp_sum(L);
    if (!ap.k_new) {
      if (s0 < splits) cm[s0 * g + h] = f0;
      if (s1 < splits) cm[s1 * g + h] = f1;
    }
    float fN = 0.f;
    if (ap.k_new) {
      // the appended token: level 0, weight 1; <q, k_new> in fp32, 4 dims per lane
      const float x = warp_sum(h < kWarps ? dot_pre[0] : dot_pre[1]) * sc;
      const float M2 = fmaxf(M, x);
      const float fS = M == -INFINITY ? 0.f : exp2f(M - M2);
      fN = exp2f(x - M2);
      if (s0 < splits) cm[s0 * g + h] = f0 * fS;
      if (s1 < splits) cm[s1 * g + h] = f1 * fS;
      if (lane == 0) { cM[h] = M2; cL[h] = fmaf(L, fS, fN); cN[h] = fN; }
    } else if (lane == 0) {
      cM[h] = M; cL[h] = L;
    }
  }
  __syncthreads();
  // every thread owns 4 consecutive output columns of one head; 8 splits' loads in flight
  const int n_items = g * (kD / 4);
  for (int i = tid; i < n_items; i += kThreads) {
    const int h = i / (kD / 4), c = (i % (kD / 4)) * 4;
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    if (staged) {
      // partial rows in shared memory: plain shared loads, four independent accumulators
      const float* base = sp_s + (size_t)h * PS + c;
      const float* fac = cm + h;
      float4 a0 = make_float4(0.f, 0.f, 0.f, 0.f), a1 = a0, a2 = a0, a3 = a0;
      int s = 0;
      for (; s + 4 <= splits; s += 4) {
        const float4 v0 = *reinterpret_cast<const float4*>(base + (size_t)(s + 0) * g * PS);
        const float4 v1 = *reinterpret_cast<const float4*>(base + (size_t)(s + 1) * g * PS);
        const float4 v2 = *reinterpret_cast<const float4*>(base + (size_t)(s + 2) * g * PS);
        const float4 v3 = *reinterpret_cast<const float4*>(base + (size_t)(s + 3) * g * PS);
        const float f0 = fac[(s + 0) * g], f1 = fac[(s + 1) * g], f2 = fac[(s + 2) * g], f3 = fac[(s + 3) * g];
        a0.x = fmaf(v0.x, f0, a0.x); a0.y = fmaf(v0.y, f0, a0.y); a0.z = fmaf(v0.z, f0, a0.z); a0.w = fmaf(v0.w, f0, a0.w);
        a1.x = fmaf(v1.x, f1, a1.x); a1.y = fmaf(v1.y, f1, a1.y); a1.z = fmaf(v1.z, f1, a1.z); a1.w = fmaf(v1.w, f1, a1.w);
        a2.x = fmaf(v2.x, f2, a2.x); a2.y = fmaf(v2.y, f2, a2.y); a2.z = fmaf(v2.z, f2, a2.z); a2.w = fmaf(v2.w, f2, a2.w);
        a3.x = fmaf(v3.x, f3, a3.x); a3.y = fmaf(v3.y, f3, a3.y); a3.z = fmaf(v3.z, f3, a3.z); a3.w = fmaf(v3.w, f3, a3.w);
      }
      for (; s < splits; ++s) {
        const float4 v0 = *reinterpret_cast<const float4*>(base + (size_t)s * g * PS);
        const float f0 = fac[s * g];
        a0.x = fmaf(v0.x, f0, a0.x); a0.y = fmaf(v0.y, f0, a0.y); a0.z = fmaf(v0.z, f0, a0.z); a0.w = fmaf(v0.w, f0, a0.w);
      }
      acc.x = (a0.x + a1.x) + (a2.x + a3.x); acc.y = (a0.y + a1.y) + (a2.y + a3.y);
      acc.z = (a0.z + a1.z) + (a2.z + a3.z); acc.w = (a0.w + a1.w) + (a2.w + a3.w);
    } else {
      for (int s = 0; s < splits; s += 8) {
        float4 v[8];
#pragma unroll
        for (int u = 0; u < 8; ++u)
          v[u] = s + u < splits ? __ldcg(reinterpret_cast<const float4*>(sp + ((size_t)(s + u) * g + h) * PS + c))
                                : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int u = 0; u < 8; ++u) {
          const float f = s + u < splits ? cm[(s + u) * g + h] : 0.f;
          acc.x = fmaf(v[u].x, f, acc.x); acc.y = fmaf(v[u].y, f, acc.y);
          acc.z = fmaf(v[u].z, f, acc.z); acc.w = fmaf(v[u].w, f, acc.w);
        }
      }
    }
    if (ap.k_new) {
      const float fN = cN[h];
      const uint2 vn = i == tid ? vn_pre : *reinterpret_cast<const uint2*>(ap.v_new + (size_t)sl * kD + c);
      const __nv_bfloat162 v01 = *reinterpret_cast<const __nv_bfloat162*>(&vn.x), v23 = *reinterpret_cast<const __nv_bfloat162*>(&vn.y);
      acc.x = fmaf(__bfloat162float(v01.x), fN, acc.x); acc.y = fmaf(__bfloat162float(v01.y), fN, acc.y);
      acc.z = fmaf(__bfloat162float(v23.x), fN, acc.z); acc.w = fmaf(__bfloat162float(v23.y), fN, acc.w);
    }
    if (raw_acc) {
      const size_t qh = (size_t)seq * (G.H * g) + (size_t)head * g + h;
      *reinterpret_cast<float4*>(raw_acc + qh * kD + c) = acc;
      if (c == 0) { raw_ml[2 * qh] = cM[h]; raw_ml[2 * qh + 1] = cL[h]; }
      continue;
    }
    const float inv = cL[h] > 0.f ? 1.0f / cL[h] : 0.f;
    __nv_bfloat162* o2 = reinterpret_cast<__nv_bfloat162*>(out + ((size_t)seq * (G.H * g) + (size_t)head * g + h) * kD + c);
    o2[0] = __floats2bfloat162_rn(acc.x * inv, acc.y * inv);
    o2[1] = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
  }
  if (tid == 0 && !single) tickets[sl] = 0;   // ready for the next launch
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

constexpr size_t kSmemBytes = 1024 + (size_t)kStages * kStageBytes + (kStages + 1) * sizeof(uint64_t);

}  // namespace

bool decode_mma_supported(const Geom& G) { return G.is_bf16 && G.d == kD && G.g <= 8; }

// Tensor maps over the K and V arenas viewed as [total_rows, 128] bf16, boxes of 64 dims x 64 rows.
cudaError_t decode_mma_prepare(const Geom& G, const Arena& A, int64_t total_rows, void** maps_out) {
  *maps_out = nullptr;
  if (!decode_mma_supported(G) || total_rows >= ((int64_t)1 << 31)) return cudaErrorNotSupported;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
  if (e != cudaSuccess) return e;
  if (!fn || qres != cudaDriverEntryPointSuccess) return cudaErrorNotSupported;
  EncodeTiledFn encode = reinterpret_cast<EncodeTiledFn>(fn);
  DecodeMaps* tm = new DecodeMaps();
  const cuuint64_t dims[2] = {(cuuint64_t)kD, (cuuint64_t)total_rows};
  const cuuint64_t strides[1] = {(cuuint64_t)kD * 2};
  const cuuint32_t box[2] = {64, (cuuint32_t)kTN};
  const cuuint32_t estr[2] = {1, 1};
  void* bases[2] = {A.K, A.V};
  CUtensorMap* maps[2] = {&tm->k, &tm->v};
  for (int i = 0; i < 2; ++i) {
    CUresult r = encode(maps[i], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, bases[i], dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { delete tm; return cudaErrorInvalidValue; }
  }
  e = cudaFuncSetAttribute(decode_mma_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
  if (e != cudaSuccess) { delete tm; return e; }
  *maps_out = tm;
  return cudaSuccess;
}

void decode_mma_release(void* maps) { delete static_cast<DecodeMaps*>(maps); }

cudaError_t launch_decode_step_mma(const Geom& G, const Arena& A, int layer, const void* q, void* out, float* scratch,
                                   int splits, int* status, const void* maps, const void* k_new, const void* v_new,
                                   int rel_row, int idx0, int new_len, const Seg* seg_hint, cudaStream_t st);

// Scratch layout of all launches (as for launch_decode): ticket counters, then (stream, split, head)
// partial rows.
// Un-normalised parts (see StepAppend::raw_acc) of the layer's streams, for decode merged over slots.
cudaError_t launch_decode_parts_mma(const Geom& G, const Arena& A, int layer, const void* q, float* raw_acc, float* raw_ml,
                                    float* scratch, int splits, int* status, const void* maps, int keys_only,
                                    cudaStream_t st) {
  if (!maps || !raw_acc || !raw_ml) return cudaErrorInvalidValue;
  const DecodeMaps* tm = static_cast<const DecodeMaps*>(maps);
  const int n_sl = G.B * G.H;
  unsigned* tickets = reinterpret_cast<unsigned*>(scratch);
  float* part = scratch + ((n_sl + 63) / 64) * 64;
  dim3 grid(n_sl, splits);
  const StepAppend ap{nullptr, nullptr, 0, 0, 0, raw_acc, raw_ml, keys_only, 0, {}, 0, {}, 0u, 0u};
  decode_mma_kernel<<<grid, kThreads, kSmemBytes, st>>>(G, A, layer, static_cast<const __nv_bfloat16*>(q), nullptr, part,
                                                        tickets, status, ap, tm->k, tm->v);
  return cudaGetLastError();
}

// The same for n_slots layer slots in one launch (grid z = slot): raw_acc / raw_ml hold one block per
// slot, scratch one block of z_stride_words 4-byte words per slot (laid out as for a single slot).
cudaError_t launch_decode_parts_mma_slots(const Geom& G, const Arena& A, const int* slot_layers, int n_slots,
                                          unsigned keys_mask, const void* q, float* raw_acc, float* raw_ml, float* scratch,
                                          size_t z_stride_words, int splits, int* status, const void* maps,
                                          cudaStream_t st) {
  if (!maps || !raw_acc || !raw_ml || n_slots < 1 || n_slots > 8 || z_stride_words > 0xffffffffull) return cudaErrorInvalidValue;
  const DecodeMaps* tm = static_cast<const DecodeMaps*>(maps);
  const int n_sl = G.B * G.H;
  unsigned* tickets = reinterpret_cast<unsigned*>(scratch);
  float* part = scratch + ((n_sl + 63) / 64) * 64;
  dim3 grid(n_sl, splits, n_slots);
  StepAppend ap{nullptr, nullptr, 0, 0, 0, raw_acc, raw_ml, 0, 0, {}, n_slots, {}, keys_mask, (unsigned)z_stride_words};
  for (int i = 0; i < n_slots; ++i) ap.slot_layer[i] = slot_layers[i];
  decode_mma_kernel<<<grid, kThreads, kSmemBytes, st>>>(G, A, slot_layers[0], static_cast<const __nv_bfloat16*>(q), nullptr,
                                                        part, tickets, status, ap, tm->k, tm->v);
  return cudaGetLastError();
}

// Ratio of merged parts: the value sums of the numerator slots over the weight sums of the
// denominator slots,
//   out = sum_p acc_p 2^{M_p - M*} / sum_r L_r 2^{M_r - M*},   M* the largest M involved
// (Algorithm 1's output ratio: the union of the numerator instances' sets above, the
// denominator instance's sets below; with the same slots on both sides, the estimator over the
// union of their caches).  parts: acc [n_parts][n_heads][d], ml [n_parts][n_heads][2]; num_mask /
// den_mask: bit p set = part p enters the numerator / the denominator.
__global__ void merged_ratio_kernel(const float* __restrict__ acc, const float* __restrict__ ml, int n_parts,
                                    unsigned num_mask, unsigned den_mask, __nv_bfloat16* __restrict__ out, int n_heads,
                                    int d) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n_heads * d) return;
  const int h = i / d;
  float M = -INFINITY;
  for (int p = 0; p < n_parts; ++p) M = fmaxf(M, ml[((size_t)p * n_heads + h) * 2]);
  float num = 0.f, den = 0.f;
  for (int p = 0; p < n_parts; ++p) {
    const float Mp = ml[((size_t)p * n_heads + h) * 2];
    if (Mp == -INFINITY) continue;                 // an empty slot
    const float f = exp2f(Mp - M);
    if ((num_mask >> p) & 1u) num = fmaf(acc[(size_t)p * n_heads * d + i], f, num);
    if ((den_mask >> p) & 1u) den = fmaf(ml[((size_t)p * n_heads + h) * 2 + 1], f, den);
  }
  out[i] = __float2bfloat16(den > 0.f ? num / den : 0.f);
}

cudaError_t launch_merged_ratio(const float* acc, const float* ml, int n_parts, unsigned num_mask, unsigned den_mask,
                                void* out, int n_heads, int d, cudaStream_t st) {
  const int n = n_heads * d;
  merged_ratio_kernel<<<(n + 255) / 256, 256, 0, st>>>(acc, ml, n_parts, num_mask, den_mask,
                                                       static_cast<__nv_bfloat16*>(out), n_heads, d);
  return cudaGetLastError();
}

// Decode attention fused with the append of one token per stream of the layer (k_new, v_new:
// [B*H, d] bf16; all streams of the layer have the same level-0 fill).  k_new == nullptr: plain decode.
cudaError_t launch_decode_step_mma(const Geom& G, const Arena& A, int layer, const void* q, void* out, float* scratch,
                                   int splits, int* status, const void* maps, const void* k_new, const void* v_new,
                                   int rel_row, int idx0, int new_len, const Seg* seg_hint, cudaStream_t st) {
  if (!maps) return cudaErrorInvalidValue;
  const DecodeMaps* tm = static_cast<const DecodeMaps*>(maps);
  const int n_sl = G.B * G.H;
  unsigned* tickets = reinterpret_cast<unsigned*>(scratch);
  float* part = scratch + ((n_sl + 63) / 64) * 64;
  dim3 grid(n_sl, splits);
  StepAppend ap{static_cast<const __nv_bfloat16*>(k_new), static_cast<const __nv_bfloat16*>(v_new), rel_row, idx0,
                new_len, nullptr, nullptr, 0, 0, {}, 0, {}, 0u, 0u};
  if (seg_hint) {
    ap.n_seg = G.T + 1;
    for (int l = 0; l <= G.T; ++l) ap.seg[l] = seg_hint[l];
  }
  // programmatic stream serialization: back-to-back decode steps overlap a launch with the
  // previous kernel's tail (see the kernel's prologue)
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(kThreads);
  cfg.dynamicSmemBytes = kSmemBytes;
  cfg.stream = st;
  cudaLaunchAttribute attr;
  attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr.val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = &attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, decode_mma_kernel, G, A, layer, static_cast<const __nv_bfloat16*>(q),
                            static_cast<__nv_bfloat16*>(out), part, tickets, status, ap, tm->k, tm->v);
}

}  // namespace bkv
