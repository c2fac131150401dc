// SoftmaxBalance (Algorithm 2) with the Gram tiles on the 5th-generation tensor cores.
//
// One CTA per call.  The call's t x t kernel matrix
//   Ghat_ij = exp((<k_i,k_j> - r_key^2)/sqrt d) <v_i,v_j> / r_value^2      (proof of Theorem 3.2)
// is visited in 128 x 128 tiles of its lower triangle, row panel by row panel.  For a tile,
// TMA brings the bf16 rows of K and V into 128B-swizzled shared memory, tcgen05.mma
// (bf16 x bf16 -> fp32) forms K_r K_c^T and V_r V_c^T in two TMEM accumulators, and four
// epilogue warpgroups (thread = row, 32 columns of the tile each) read them back with
// tcgen05.ld, apply exp2/scale/product and fold the tile into the row's running correlation
//   S_j = sum_{i<j} eta_i Ghat_ij
// with the signs of earlier panels.  The diagonal tile feeds the walk,
//   eta_j = +1  iff  u_j < 1/2 - S_j/(2c)  <=>  S_j < c (1 - 2 u_j),
// u_j the Philox uniform of (seed, layer, head, call ordinal, level, j).  eta_j depends only on
// eta_{<j}, so the sequential recurrence has a unique solution, and it is the fixed point of
// "decide every token of the panel from the current signs": all 512 epilogue threads keep their
// 32 entries of the diagonal tile in registers and repeat that sweep (two named-barrier exchanges
// per sweep) until no sign changes.  Sweep k makes at least token k final, so 129 sweeps always
// suffice; with small Ghat two or three do.
// TMEM is double buffered (2 x 256 columns); an epilogue hands its buffer back as soon as the
// accumulator values are in registers.  Each of the two products of a tile has its own issuing
// thread and its own barriers, so that one product's waits and commits overlap the other's
// MMAs.  Operands live in three 64 KB slots (K tile + V tile) that rotate roles: panel r keeps
// its rows in slot r % 3 and streams its column tiles through the other two, and the rows of
// panel r + 1 are fetched into the slot that panel r's column tiles leave first, so the next
// panel's first products are already in TMEM when the walk of the diagonal tile ends.
// Inside a slot every operand is two boxes of 64 dims with their own full/empty barriers: a box is
// refilled as soon as the four MMAs that read it have retired.
// Ghat never touches global memory.
//
// Every wait is bounded: a wait that runs out sets the abort flag and the status word, all
// roles leave their loops, TMEM is freed and the kernel returns.
#include <cuda.h>

#include "common.cuh"

namespace bkv {

namespace {

constexpr int kTile = 128;
constexpr int kEpiGroups = 4;              // epilogue + walk warpgroups: warps 0-15 (warp % 4 = TMEM lane quadrant)
constexpr int kEpiWarps = 4 * kEpiGroups;
constexpr int kTmaWarp = kEpiWarps, kMmaWarp = kEpiWarps + 1, kMmaWarpV = kEpiWarps + 2;   // TMA, MMA (K K^T), MMA (V V^T)
constexpr int kThreads = 32 * (kEpiWarps + 3);
constexpr uint32_t kHalfBytes = 16384;     // [128 rows][64 bf16] = one swizzle-atom column of a tile
constexpr uint32_t kTileBytes = 32768;     // [128 rows][128 bf16]
constexpr uint32_t kTmemCols = 512;
constexpr long long kWaitCycles = 100000000LL;   // about 50 ms; every wait here is on this CTA's own copies and MMAs

struct TensorMaps {
  CUtensorMap k, v;
};

__device__ inline uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ inline void mbar_init(uint64_t* bar, int count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ inline void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ inline void mbar_arrive(uint64_t* bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
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
__device__ inline int ld_acquire(const int* p) {
  int v;
  asm volatile("ld.acquire.cta.shared.s32 %0, [%1];" : "=r"(v) : "r"(smem_u32(p)) : "memory");
  return v;
}
__device__ inline void st_release(int* p, int v) {
  asm volatile("st.release.cta.shared.s32 [%0], %1;" ::"r"(smem_u32(p)), "r"(v) : "memory");
}
// Bounded wait on an mbarrier phase; false = gave up (abort flag set) or someone else aborted.
__device__ inline bool wait_bar(uint64_t* bar, uint32_t parity, int* abort_flag) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (ld_acquire(abort_flag)) return false;
    if (clock64() - t0 > kWaitCycles) { st_release(abort_flag, 1); return false; }
  }
  return true;
}
// Named barriers of the 512 epilogue threads (ids 1..3; id 0 is __syncthreads).  Every epilogue
// thread reaches every one of them whatever happened before (a failed wait only clears `ok`), so
// none of them can be left waiting.
__device__ inline void bar_sync(int id, int n) { asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(n) : "memory"); }
__device__ inline void bar_arrive(int id, int n) { asm volatile("bar.arrive %0, %1;" ::"r"(id), "r"(n) : "memory"); }
__device__ inline bool bar_red_or(int id, int n, bool pred) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 q, %3, 0;\n\t"
      "bar.red.or.pred p, %1, %2, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(r) : "r"(id), "r"(n), "r"((uint32_t)pred) : "memory");
  return r != 0;
}

__device__ inline void tma_load_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
      ::"r"(smem_u32(dst)), "l"(map), "r"(smem_u32(bar)), "r"(x), "r"(y) : "memory");
}

// Shared-memory matrix descriptor of a K-major, 128B-swizzled bf16 operand: rows of 128 bytes,
// 8-row groups 1024 bytes apart (stride byte offset), version 1, layout type SWIZZLE_128B.
// Only the low word depends on the address: (addr >> 4) in bits [0,14), leading byte offset 1
// (unused for swizzled K-major) in bits [16,30).  Stepping 16 elements along K adds 32 bytes,
// i.e. 2 to the low word; the second 64-column half of a tile sits kHalfBytes further.
constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);
__device__ inline uint32_t umma_desc_lo(uint32_t smem_addr) { return ((smem_addr & 0x3FFFFu) >> 4) | (1u << 16); }
// kind::f16 instruction descriptor: D fp32, A and B bf16, both K-major, M = N = 128.
constexpr uint32_t kInstrDesc = (1u << 4) | (1u << 7) | (1u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);

// A tcgen05.mma is issued at the rate the tensor core retires them, so every other instruction
// of the issuing thread is idle time of the pipe: descriptors come as ready-made words and the
// accumulate flag is a compile-time constant.
template <int kAccumulate>
__device__ inline void umma_bf16(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "mov.b64 da, {%1, %3};\n\t"
      "mov.b64 db, {%2, %3};\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %5, p;\n\t}"
      ::"r"(d_tmem), "r"(a_lo), "r"(b_lo), "r"(kDescHi), "n"(kAccumulate), "r"(kInstrDesc) : "memory");
}
// The 8 K-steps of one 128 x 128 x 128 product in two halves (dims 0..63, then 64..127, which sit
// kHalfBytes further): A and B tiles given by their descriptor low words.
__device__ inline void umma_tile_lo(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo) {
  umma_bf16<0>(d_tmem, a_lo, b_lo);
  umma_bf16<1>(d_tmem, a_lo + 2, b_lo + 2);
  umma_bf16<1>(d_tmem, a_lo + 4, b_lo + 4);
  umma_bf16<1>(d_tmem, a_lo + 6, b_lo + 6);
}
__device__ inline void umma_tile_hi(uint32_t d_tmem, uint32_t a_lo, uint32_t b_lo) {
  constexpr uint32_t kHalf = kHalfBytes >> 4;
  umma_bf16<1>(d_tmem, a_lo + kHalf, b_lo + kHalf);
  umma_bf16<1>(d_tmem, a_lo + kHalf + 2, b_lo + kHalf + 2);
  umma_bf16<1>(d_tmem, a_lo + kHalf + 4, b_lo + kHalf + 4);
  umma_bf16<1>(d_tmem, a_lo + kHalf + 6, b_lo + kHalf + 6);
}
__device__ inline void umma_commit(uint64_t* bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ inline void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ inline void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

// 32 consecutive fp32 columns of this warp's 32 TMEM lanes.
__device__ inline void tmem_ld32(uint32_t taddr, float (&v)[32]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr) : "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ inline void tmem_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

__device__ inline float fast_exp2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// 2^x for a pair of values on the FMA pipe (the special-function unit delivers 16 ex2 per clock
// and SM, which is as many cycles per tile as the tensor core needs for its MMAs; moving part of
// the exponentials here takes the unit off the critical path).  Cody-Waite: x = n + f with n the
// nearest integer (magic-number rounding) and f in [-1/2, 1/2]; 2^f by a degree-5 polynomial
// (coefficients from a Remez fit of 2^f on [-1/2, 1/2], relative error 7.5e-8; 2.3e-7 when
// evaluated in fp32); 2^n by adding n to the exponent field.  Valid for x in [-126, 126];
// smaller x are clamped (result ~1e-38 instead of 0).
__device__ inline float2 poly_exp2x2(float2 x) {
  const float kMagic = 12582912.0f;   // 1.5 * 2^23
  x.x = fmaxf(x.x, -126.0f);
  x.y = fmaxf(x.y, -126.0f);
  const float2 t = __fadd2_rn(x, make_float2(kMagic, kMagic));
  const float2 n = __fadd2_rn(t, make_float2(-kMagic, -kMagic));
  const float2 f = __ffma2_rn(n, make_float2(-1.0f, -1.0f), x);
  float2 p = make_float2(0x1.5c08e6p-10f, 0x1.5c08e6p-10f);
  p = __ffma2_rn(p, f, make_float2(0x1.3d0c52p-7f, 0x1.3d0c52p-7f));
  p = __ffma2_rn(p, f, make_float2(0x1.c6b6e4p-5f, 0x1.c6b6e4p-5f));
  p = __ffma2_rn(p, f, make_float2(0x1.ebf918p-3f, 0x1.ebf918p-3f));
  p = __ffma2_rn(p, f, make_float2(0x1.62e428p-1f, 0x1.62e428p-1f));
  p = __ffma2_rn(p, f, make_float2(0x1.000002p+0f, 0x1.000002p+0f));
  float2 r;
  r.x = __int_as_float(__float_as_int(p.x) + (__float_as_int(t.x) << 23));
  r.y = __int_as_float(__float_as_int(p.y) + (__float_as_int(t.y) << 23));
  return r;
}
// Of the 16 column pairs of a 32-column chunk, pairs with (index % 8) < kPolyOf8 take the
// polynomial path, the others the special-function unit.
constexpr int kPolyOf8 = 1;

struct Smem {
  // three operand slots first (1024-byte aligned for the 128B swizzle); a slot holds a K tile then a V tile
  static constexpr uint32_t kSlotBytes = 2 * kTileBytes;
  static constexpr uint32_t kTilesEnd = 3 * kSlotBytes;
};
constexpr int kMaxSweeps = kTile + 2;

// Output of Algorithm 2 completed to exactly t/2 tokens (the implementation note of Appendix B:
// "strictly select n/2"), and Algorithm 3's C^{i+1} <- C^{i+1} + SoftmaxBalance(C^i): the smaller
// sign class (ties: +1) plus the latest tokens of the other class, in stream order, copied to the
// call's destination rows with their positions and norms.  Runs at the tail of the call's CTA, whose
// operand slots are idle by then: `scratch` holds the kept positions.  The rows were read by this
// CTA microseconds ago and come from L2.  All kThreads threads take part.
__device__ inline void select_and_compact(const Geom& G, const Arena& A, const CallDesc& C, const int8_t* eta8, int* scratch) {
  const int t = G.t, half = t / 2;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  constexpr int kScan = 512;                       // scanning threads (warps 0-15)
  int* warp_sums = scratch;                        // [16] + [16]
  int* kept_pos = scratch + 64;                    // [t/2]
  const int ipt = (t + kScan - 1) / kScan;         // consecutive tokens per scanning thread (<= 8)
  const int j0 = tid * ipt;
  int plus = 0;
  if (tid < kScan)
    for (int i = 0; i < ipt; ++i) plus += (j0 + i < t && eta8[j0 + i] > 0) ? 1 : 0;
  // exclusive scan of `plus` over the scanning threads
  int inc = plus;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int n = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += n;
  }
  if (tid < kScan && lane == 31) warp_sums[warp] = inc;
  __syncthreads();
  int base = 0, total_plus = 0;
#pragma unroll
  for (int w = 0; w < kScan / 32; ++w) {
    const int sv = warp_sums[w];
    if (w < warp) base += sv;
    total_plus += sv;
  }
  const int plus_before = base + inc - plus;
  const int keep_sign = (total_plus <= t - total_plus) ? 1 : -1;
  const int have = keep_sign > 0 ? total_plus : t - total_plus;
  const int first_other_kept = (t - have) - (half - have);   // rank (in stream order) from which the other class is kept
  int other_rank = keep_sign > 0 ? (min(j0, t) - plus_before) : plus_before;
  int keep_cnt = 0;
  unsigned mask = 0;
  if (tid < kScan)
    for (int i = 0; i < ipt; ++i) {
      const int j = j0 + i;
      if (j >= t) break;
      const bool mine = (eta8[j] > 0) == (keep_sign > 0);
      bool keep = mine;
      if (!mine) { keep = other_rank >= first_other_kept; ++other_rank; }
      if (keep) { mask |= 1u << i; ++keep_cnt; }
    }
  inc = keep_cnt;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const int n = __shfl_up_sync(0xffffffffu, inc, o);
    if (lane >= o) inc += n;
  }
  if (tid < kScan && lane == 31) warp_sums[16 + warp] = inc;
  __syncthreads();
  int pos = inc - keep_cnt;
#pragma unroll
  for (int w = 0; w < kScan / 32; ++w)
    if (w < warp) pos += warp_sums[16 + w];
  if (tid < kScan)
    for (int i = 0; i < ipt; ++i)
      if (mask & (1u << i)) kept_pos[pos++] = j0 + i;
  __syncthreads();
  // copy: a survivor row of K and of V is 2 x 16 chunks of 16 bytes; eight loads in flight per thread.
  // (All CTAs of a wave reach this point together, so the copy runs at the chip's memory bandwidth
  // whichever engine moves the bytes; the bulk-copy engine was measured and is no faster.)
  const uint4* Ks = reinterpret_cast<const uint4*>(A.K) + (size_t)C.src_row * 16;
  const uint4* Vs = reinterpret_cast<const uint4*>(A.V) + (size_t)C.src_row * 16;
  uint4* Kd = reinterpret_cast<uint4*>(A.K) + (size_t)C.dst_row * 16;
  uint4* Vd = reinterpret_cast<uint4*>(A.V) + (size_t)C.dst_row * 16;
  const int items = half * 32;
  for (int i0 = tid; i0 < items; i0 += 8 * kThreads) {
    uint4 v[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int i = i0 + u * kThreads;
      if (i < items) {
        const int o = i >> 5, c = i & 31;
        v[u] = (c < 16 ? Ks : Vs)[(size_t)kept_pos[o] * 16 + (c & 15)];
      }
    }
#pragma unroll
    for (int u = 0; u < 8; ++u) {
      const int i = i0 + u * kThreads;
      if (i < items) {
        const int o = i >> 5, c = i & 31;
        (c < 16 ? Kd : Vd)[(size_t)o * 16 + (c & 15)] = v[u];
      }
    }
  }
  for (int o = tid; o < half; o += kThreads) {
    A.idx[C.dst_row + o] = A.idx[C.src_row + kept_pos[o]];
    if (A.nrm) A.nrm[C.dst_row + o] = A.nrm[C.src_row + kept_pos[o]];
  }
}

template <bool kCenter>
__global__ void __launch_bounds__(kThreads, 1)
walk_tc_kernel(Geom G, const CallDesc* __restrict__ calls, int level, const CallStat* __restrict__ stats,
               const float* __restrict__ tok_shift, int8_t* __restrict__ eta_out, int8_t* __restrict__ dbg_eta,
               float* __restrict__ dbg_S, float* __restrict__ dbg_p, unsigned long long* __restrict__ fail_count,
               int* __restrict__ status, const float2* __restrict__ row_norms, const Arena A,
               const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* sm = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  const int t = G.t, P = t / kTile;
  float* etas = reinterpret_cast<float*>(sm + Smem::kTilesEnd);          // [t] signs scaled by 1/r_value^2 (0 = undecided)
  float* xs = etas + t;                                                   // [3][128] partial correlations of column quarters 1..3
  float* xb = xs + (kEpiGroups - 1) * kTile;                              // [3][128] ... and of their sums of |Ghat|
  float* thr_s = xb + (kEpiGroups - 1) * kTile;                           // [t] decision thresholds c (1 - 2 u_j)
  int8_t* eta8 = reinterpret_cast<int8_t*>(thr_s + t);                    // [t] signs
  uint64_t* bars = reinterpret_cast<uint64_t*>(eta8 + t);                 // t is a multiple of 128
  // x = 0: the K K^T product, x = 1: the V V^T product
  // An operand tile travels as two boxes of 64 dims (h = 0, 1); a box is refilled as soon as the
  // four MMAs that read it are done, which lengthens the prefetch distance of the column ring.
  uint64_t* full = bars + 0;         // [x][3][h] box h of product x's operand landed in slot s: index 6 x + 2 s + h
  uint64_t* empty = bars + 12;       // [x][3][h] product x no longer reads that box -> producer
  uint64_t* xdone = bars + 24;       // [2] both products of the tile in TMEM buffer b finished (one arrival per product) -> epilogue
  uint64_t* tmem_empty = bars + 28;  // [2] all epilogue warps have drained buffer b
  uint32_t* tmem_ptr_s = reinterpret_cast<uint32_t*>(bars + 30);
  int* abort_flag = reinterpret_cast<int*>(tmem_ptr_s + 1);

  const int call = blockIdx.x;
  const CallDesc C = calls[call];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

  if (tid == 0) {
    for (int i = 0; i < 12; ++i) { mbar_init(full + i, 1); mbar_init(empty + i, 1); }
    for (int i = 0; i < 2; ++i) mbar_init(xdone + i, 2);
    for (int i = 0; i < 2; ++i) mbar_init(tmem_empty + i, kEpiWarps);       // one arrival per warp (lane 0 after __syncwarp)
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  for (int i = tid; i < t; i += kThreads) etas[i] = 0.f;
  if (warp == kMmaWarp) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_ptr_s)), "r"(kTmemCols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = *tmem_ptr_s;

  // Tiles are numbered in issue order i = 0, 1, ...: panel r contributes (r,0) .. (r,r).  Tile i
  // uses TMEM buffer i & 1.  Panel r reads its rows from slot r % 3 and column tile c from slot
  // (r + 1 + (c & 1)) % 3.  Loads happen in the order R0, R1, C(1,0), R2, C(2,0), C(2,1), R3, ...
  // (R = row panel), which is also the order in which the MMA threads first touch them, so both
  // sides count the uses of a slot alike.  Every barrier is waited on phase by phase by its one
  // kind of waiter, and each next phase depends on that waiter having passed, so a parity wait
  // can never be a phase behind.
  if (warp == kTmaWarp) {
    // ------------------------------------------------------------------ TMA producer
    if (lane == 0) {
      uint32_t used = 0, par = 0;        // per slot: loaded before; parity of the next wait on its empty barriers
      bool ok = true;
      auto load = [&](int slot, int tile_row) -> bool {
        const bool again = (used >> slot) & 1u;
        const uint32_t ph = (par >> slot) & 1u;
        used |= 1u << slot;
        if (again) par ^= 1u << slot;
        unsigned char* st = sm + (uint32_t)slot * Smem::kSlotBytes;
        const int y = (int)(C.src_row + (int64_t)tile_row * kTile);
#pragma unroll
        for (int h = 0; h < 2; ++h) {
          uint64_t* fk = full + 2 * slot + h;
          uint64_t* fv = full + 6 + 2 * slot + h;
          if (again && !wait_bar(empty + 2 * slot + h, ph, abort_flag)) return false;
          mbar_expect_tx(fk, kHalfBytes);
          tma_load_2d(st + h * kHalfBytes, &tmK, 64 * h, y, fk);
          if (again && !wait_bar(empty + 6 + 2 * slot + h, ph, abort_flag)) return false;
          mbar_expect_tx(fv, kHalfBytes);
          tma_load_2d(st + kTileBytes + h * kHalfBytes, &tmV, 64 * h, y, fv);
        }
        return true;
      };
      ok = load(0, 0);
      for (int r = 0; r < P && ok; ++r) {
        for (int c = 0; c < r && ok; ++c) ok = load((r + 1 + (c & 1)) % 3, c);
        if (ok && r + 1 < P) ok = load((r + 1) % 3, r + 1);
      }
    }
    __syncwarp();
  } else if (warp == kMmaWarp || warp == kMmaWarpV) {
    // ------------------------------------------------------------------ MMA issuers (K K^T and V V^T)
    if (lane == 0) {
      const int x = warp == kMmaWarpV ? 1 : 0;
      int i = 0;
      uint32_t par = 0;                  // per slot: parity of the next wait on its full barrier
      bool ok = true;
      const uint32_t slot0 = umma_desc_lo(smem_u32(sm + (x ? kTileBytes : 0u)));
      constexpr uint32_t kSlotDesc = Smem::kSlotBytes >> 4;
      for (int r = 0; r < P && ok; ++r) {
        const int rs = r % 3;
        if (!(ok = wait_bar(full + 6 * x + 2 * rs, (par >> rs) & 1u, abort_flag))) break;
        if (!(ok = wait_bar(full + 6 * x + 2 * rs + 1, (par >> rs) & 1u, abort_flag))) break;
        par ^= 1u << rs;
        const uint32_t arow = slot0 + (uint32_t)rs * kSlotDesc;
        for (int c = 0; c <= r; ++c, ++i) {
          const int buf = i & 1;
          if (!(ok = wait_bar(tmem_empty + buf, (uint32_t)(((i >> 1) & 1) ^ 1), abort_flag))) break;
          const int slot = c < r ? (r + 1 + (c & 1)) % 3 : rs;
          const uint32_t b = slot0 + (uint32_t)slot * kSlotDesc;
          const uint32_t d_tmem = tmem_base + (uint32_t)buf * 256u + (x ? 128u : 0u);
          const uint32_t ph = (par >> slot) & 1u;
          if (c < r) {
            if (!(ok = wait_bar(full + 6 * x + 2 * slot, ph, abort_flag))) break;
            par ^= 1u << slot;
          }
          tc_fence_after();
          umma_tile_lo(d_tmem, arow, b);
          umma_commit(empty + 6 * x + 2 * slot);       // a column slot's box after its tile, the row slot's after the diagonal tile
          if (c < r && !(ok = wait_bar(full + 6 * x + 2 * slot + 1, ph, abort_flag))) break;
          umma_tile_hi(d_tmem, arow, b);
          umma_commit(empty + 6 * x + 2 * slot + 1);
          umma_commit(xdone + buf);
        }
      }
    }
    __syncwarp();
  } else {
    // ------------------------------------------------------------------ four epilogue warpgroups
    // Every tile is drained by all groups: group wg takes columns 32 wg .. 32 wg + 31 of the tile
    // (thread = row) and keeps a partial running correlation of its row over those columns.
    const int wg = warp >> 2;
    const int q = warp & 3;                   // quarter of the panel = TMEM lane quadrant
    const int row = 32 * q + lane;
    const float scale = 1.4426950408889634f * G.inv_sqrt_d;
    const float cw = G.c;
    const uint32_t tlane = tmem_base + ((uint32_t)(32 * q) << 16) + (uint32_t)(32 * wg);
    const float* shift = kCenter ? tok_shift + (size_t)call * t : nullptr;
    int tile_it = 0, fails = 0;
    bool ok = true;

    // Ghat' (without 1/r_value^2) of two neighbouring columns, packed fp32
    auto ghat2 = [&](float k0, float k1, float v0, float v1, float nb, bool poly) -> float2 {
      const float2 ex = __ffma2_rn(make_float2(k0, k1), make_float2(scale, scale), make_float2(nb, nb));
      const float2 ee = poly ? poly_exp2x2(ex) : make_float2(fast_exp2(ex.x), fast_exp2(ex.y));
      return __fmul2_rn(ee, make_float2(v0, v1));
    };
    // acc += sum over this group's 32 columns of Ghat' * sign, from accumulator values in registers
    auto fold_regs = [&](const float (&dk)[32], const float (&dv)[32], const float* signs, int shift_base, float nb,
                         float acc) -> float {
      const float4* e4 = reinterpret_cast<const float4*>(signs);
      if constexpr (kCenter) {
#pragma unroll
        for (int x = 0; x < 8; ++x) {
          const float4 e = e4[x];
          const float ev[4] = {e.x, e.y, e.z, e.w};
#pragma unroll
          for (int y = 0; y < 4; ++y) {
            const int i = 4 * x + y;
            const float ex = fmaf(dk[i], scale, nb) - shift[shift_base + i] * scale;
            acc = fmaf(fast_exp2(ex) * dv[i], ev[y], acc);
          }
        }
        return acc;
      } else {
        float2 a2[2] = {make_float2(acc, 0.f), make_float2(0.f, 0.f)};
#pragma unroll
        for (int x = 0; x < 8; ++x) {
          const float4 e = e4[x];
#pragma unroll
          for (int h = 0; h < 2; ++h) {
            const int i = 4 * x + 2 * h, pair = 2 * x + h;
            const float2 g = ghat2(dk[i], dk[i + 1], dv[i], dv[i + 1], nb, (pair & 7) < kPolyOf8);
            a2[pair & 1] = __ffma2_rn(g, h ? make_float2(e.z, e.w) : make_float2(e.x, e.y), a2[pair & 1]);
          }
        }
        const float2 s2 = __fadd2_rn(a2[0], a2[1]);
        return s2.x + s2.y;
      }
    };

    constexpr int kEpiThreads = 32 * kEpiWarps;
    {
      // all coins of the call up front (the first tile is still on its way), off the walk's critical path
      const int head = C.stream % G.H, layer = (C.stream / G.H) % G.L, seq = C.stream / (G.H * G.L);
      for (int i = tid; i < t; i += kEpiThreads)
        thr_s[i] = cw * (1.0f - 2.0f * walk_uniform(G.seed + (uint64_t)seq, layer, head, C.ordinal, level, i));
      // r_key^2, r_value^2 of the call (inputs of Algorithm 2) = maxima of the stored row norms,
      // unless a separate kernel has put them (key centering changes them) or they are fixed
      if (row_norms) {
        float mk = 0.f, mv = 0.f;
        for (int i = tid; i < t; i += kEpiThreads) {
          const float2 n2 = row_norms[C.src_row + i];
          mk = fmaxf(mk, n2.x);
          mv = fmaxf(mv, n2.y);
        }
        mk = warp_max(mk); mv = warp_max(mv);
        if (lane == 0) { xs[2 * warp] = mk; xs[2 * warp + 1] = mv; }
      }
      bar_sync(3, kEpiThreads);
    }
    float rk2 = G.fixed_rk2, rv2 = G.fixed_rv2;
    if (row_norms) {
      float mk = 0.f, mv = 0.f;
#pragma unroll
      for (int w = 0; w < kEpiWarps; ++w) { mk = fmaxf(mk, xs[2 * w]); mv = fmaxf(mv, xs[2 * w + 1]); }
      if (rk2 <= 0.f) rk2 = mk;
      if (rv2 <= 0.f) rv2 = mv;
      bar_sync(3, kEpiThreads);                               // xs is reused by the first walk
    } else {
      if (rk2 <= 0.f) rk2 = stats[call].rk2;
      if (rv2 <= 0.f) rv2 = stats[call].rv2;
    }
    const float inv_rv2 = rv2 > 0.f ? 1.0f / rv2 : 0.f;
    // All waits of a panel come before its vote barrier (id 3); a thread whose wait timed out
    // skips to the vote, where everybody learns of it and leaves.  The sweep barriers (ids 1, 2)
    // come after the vote and contain no waits, so no thread can be left waiting at them.
    for (int r = 0; r < P; ++r) {
      const int j = r * kTile + row;                      // this thread's token in the panel
      float nb = -rk2 * scale;                            // exponent offset of this row
      if constexpr (kCenter) nb -= shift[j] * scale;
      float acc = 0.f;
      const int col0 = 32 * wg;
      const bool below = wg <= q;                         // warp-uniform: the warp has columns below the diagonal
      for (int c = 0; c < r && ok; ++c, ++tile_it) {
        const int buf = tile_it & 1;
        if (!(ok = wait_bar(xdone + buf, (uint32_t)((tile_it >> 1) & 1), abort_flag))) break;
        tc_fence_after();
        const uint32_t tb = tlane + (uint32_t)buf * 256u;
        // pull this group's 32 columns of both accumulators into registers and hand the TMEM
        // buffer back at once; the arithmetic then overlaps the next tiles' MMAs
        float dk[32], dv[32];
        tmem_ld32(tb, dk);
        tmem_ld32(tb + 128, dv);
        tmem_ld_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(tmem_empty + buf);
        // signs of panel c are final since its walk
        acc = fold_regs(dk, dv, etas + c * kTile + 32 * wg, c * kTile + 32 * wg, nb, acc);
      }
      // ---- diagonal tile
      const int buf = tile_it & 1;
      if (ok) ok = wait_bar(xdone + buf, (uint32_t)((tile_it >> 1) & 1), abort_flag);
      if (bar_red_or(3, kEpiThreads, !ok)) { ok = false; break; }          // uniform: everybody walks or everybody leaves
      ++tile_it;
      float g[32];
      {
        tc_fence_after();
        const uint32_t tb = tlane + (uint32_t)buf * 256u;
        float dk[32], dv[32];
        tmem_ld32(tb, dk);
        tmem_ld32(tb + 128, dv);
        tmem_ld_wait();
        tc_fence_before();
        __syncwarp();
        if (lane == 0) mbar_arrive(tmem_empty + buf);
        // Ghat' of this row against the strictly earlier tokens among this group's columns (none
        // for the warps above the diagonal)
#pragma unroll
        for (int i = 0; i < 32; i += 2) {
          float2 v = make_float2(0.f, 0.f);
          if (below) {
            if constexpr (kCenter) {
              v.x = fast_exp2(fmaf(dk[i], scale, nb) - shift[r * kTile + col0 + i] * scale) * dv[i];
              v.y = fast_exp2(fmaf(dk[i + 1], scale, nb) - shift[r * kTile + col0 + i + 1] * scale) * dv[i + 1];
            } else {
              v = ghat2(dk[i], dk[i + 1], dv[i], dv[i + 1], nb, false);
            }
          }
          g[i] = col0 + i < row ? v.x : 0.f;
          g[i + 1] = col0 + i + 1 < row ? v.y : 0.f;
        }
      }
      const float thr = thr_s[j];
      // The walk over the panel's 128 tokens by sweeps: group 0 owns the decisions, groups 1-3
      // supply the partial sums of their columns.  Undecided signs are stored as 0.
      const float4* e4 = reinterpret_cast<const float4*>(etas + r * kTile + col0);
      // In sweep 0 (all in-panel signs still 0, S = the earlier panels' part) a row whose distance
      // to its threshold exceeds sum_j |Ghat_ij| of its in-panel columns is already decided; if
      // that holds for every row (and no row can FAIL, and S is not recorded) one sweep suffices.
      float absum = 0.f;
      if (below) {
#pragma unroll
        for (int i = 0; i < 32; ++i) absum += fabsf(g[i]);
      }
      if (wg > 0) xb[(wg - 1) * kTile + row] = absum;
      bool plus = false;
      float S = 0.f;
#pragma unroll 1
      for (int sweep = 0; sweep < kMaxSweeps; ++sweep) {
        float part = acc;
        if (below) {
          float2 a2 = make_float2(acc, 0.f), b2 = make_float2(0.f, 0.f);
#pragma unroll
          for (int x = 0; x < 8; ++x) {
            const float4 e = e4[x];
            a2 = __ffma2_rn(make_float2(g[4 * x], g[4 * x + 1]), make_float2(e.x, e.y), a2);
            b2 = __ffma2_rn(make_float2(g[4 * x + 2], g[4 * x + 3]), make_float2(e.z, e.w), b2);
          }
          part = (a2.x + a2.y) + (b2.x + b2.y);
        }
        bool changed = false;
        if (wg > 0) {
          xs[(wg - 1) * kTile + row] = part;
          bar_arrive(1, kEpiThreads);
        } else {
          bar_sync(1, kEpiThreads);                       // all partial sums of this sweep are written
          S = (part + xs[row]) + (xs[kTile + row] + xs[2 * kTile + row]);
          const bool now = S < thr;
          if (sweep == 0) {
            const float bound = ((absum + xb[row]) + (xb[kTile + row] + xb[2 * kTile + row])) * inv_rv2;
            const float slack = 1e-5f * (fabsf(S) + bound) + 1e-30f;
            changed = C.dbg_off >= 0 || !(fabsf(S - thr) > bound + slack) || !(fabsf(S) + bound + slack < cw);
          } else {
            changed = now != plus;
          }
          plus = now;
          etas[j] = plus ? inv_rv2 : -inv_rv2;
        }
        if (!bar_red_or(2, kEpiThreads, changed)) break;  // all signs of this sweep are written; any change?
      }
      if (wg == 0) {
        eta8[j] = plus ? 1 : -1;
        if (fabsf(S) > cw) ++fails;                          // FAIL of Algorithm 2: counted; the decision is the clamped one
        if (C.dbg_off >= 0) {
          dbg_S[C.dbg_off + j] = S;
          dbg_p[C.dbg_off + j] = 0.5f - fminf(fmaxf(S, -cw), cw) / (2.0f * cw);
        }
      }
    }
    fails = (int)__reduce_add_sync(0xffffffffu, (unsigned)fails);
    if (lane == 0 && fails) atomicAdd(fail_count, (unsigned long long)fails);
  }

  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  if (*abort_flag) {
    if (tid == 0) atomicCAS(status, kStatusOk, kStatusWaitTimeout);
  } else {
    for (int i = tid; i < t; i += kThreads) {
      const int8_t e = eta8[i];
      eta_out[(size_t)call * t + i] = e;
      if (C.dbg_off >= 0) dbg_eta[C.dbg_off + i] = e;
    }
    if (A.K) select_and_compact(G, A, C, eta8, reinterpret_cast<int*>(sm));
  }
  if (warp == kMmaWarp) {
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

size_t tc_smem_bytes(int t) { return 1024 + Smem::kTilesEnd + (size_t)t * 9 + 2 * (kEpiGroups - 1) * kTile * 4 + 512; }

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

}  // namespace

bool walk_tc_supported(const Geom& G) {
  return G.is_bf16 && G.d == 128 && G.t % kTile == 0 && tc_smem_bytes(G.t) <= (size_t)227 * 1024;
}

// Encodes the two tensor maps (K and V arenas viewed as [total_rows, 128] bf16, boxes of
// 64 columns x 128 rows, 128-byte swizzle).
cudaError_t walk_tc_prepare(const Geom& G, const Arena& A, int64_t total_rows, void** tmaps_out) {
  *tmaps_out = nullptr;
  if (!walk_tc_supported(G)) return cudaErrorNotSupported;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
  if (e != cudaSuccess) return e;
  if (!fn || qres != cudaDriverEntryPointSuccess) return cudaErrorNotSupported;
  EncodeTiledFn encode = reinterpret_cast<EncodeTiledFn>(fn);
  TensorMaps* tm = new TensorMaps();
  const cuuint64_t dims[2] = {(cuuint64_t)G.d, (cuuint64_t)total_rows};
  const cuuint64_t strides[1] = {(cuuint64_t)G.d * 2};
  const cuuint32_t box[2] = {64, (cuuint32_t)kTile};
  const cuuint32_t estr[2] = {1, 1};
  void* bases[2] = {A.K, A.V};
  CUtensorMap* maps[2] = {&tm->k, &tm->v};
  for (int i = 0; i < 2; ++i) {
    CUresult r = encode(maps[i], CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, bases[i], dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) { delete tm; return cudaErrorInvalidValue; }
  }
  e = cudaFuncSetAttribute(walk_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tc_smem_bytes(G.t));
  if (e == cudaSuccess)
    e = cudaFuncSetAttribute(walk_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)tc_smem_bytes(G.t));
  if (e != cudaSuccess) { delete tm; return e; }
  *tmaps_out = tm;
  return cudaSuccess;
}

void walk_tc_release(void* tmaps) { delete static_cast<TensorMaps*>(tmaps); }

cudaError_t launch_walk_tc(const Geom& G, const Arena& A, const CallDesc* calls, int n_calls, int level,
                           const CallStat* stats, const float* tok_shift, int8_t* eta, int8_t* dbg_eta,
                           float* dbg_S, float* dbg_p, unsigned long long* fail_count, int* status,
                           const void* tmaps, const void* fuse_compaction, cudaStream_t st) {
  if (n_calls <= 0) return cudaSuccess;
  if (!tmaps) return cudaErrorInvalidValue;
  const TensorMaps* tm = static_cast<const TensorMaps*>(tmaps);
  const size_t smem = tc_smem_bytes(G.t);
  Arena Af = A;                       // K == nullptr: leave selection and compaction to the separate kernel
  if (!fuse_compaction) Af.K = nullptr;
  if (G.center_keys)
    walk_tc_kernel<true><<<n_calls, kThreads, smem, st>>>(G, calls, level, stats, tok_shift, eta, dbg_eta, dbg_S, dbg_p,
                                                          fail_count, status, G.center_keys ? nullptr : A.nrm, Af, tm->k, tm->v);
  else
    walk_tc_kernel<false><<<n_calls, kThreads, smem, st>>>(G, calls, level, stats, tok_shift, eta, dbg_eta, dbg_S, dbg_p,
                                                           fail_count, status, G.center_keys ? nullptr : A.nrm, Af, tm->k, tm->v);
  return cudaGetLastError();
}

}  // namespace bkv
