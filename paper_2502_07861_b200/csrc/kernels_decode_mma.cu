// Split-K decode attention over the weighted compressed cache, bf16 / d = 128, on tensor cores.
//
//   out = sum_i w_i e^{<k_i,q>/sqrt d} v_i / sum_i w_i e^{<k_i,q>/sqrt d},   w_i = 2^level(i)
//
// (output ratio of Algorithm 1 / estimator of Theorem 3.3 over the sets C^T..C^0 of a stream;
// Eq. (1) when every token sits in C^0).  The g <= 8 query heads of a KV head form the rows of a
// 8-column MMA operand, so K.q^T and V^T.p^T each cost one mma.sync.m16n8k16 per 16 tokens x 16 dims:
// at g = 5 the CUDA-core formulation needs ~65 instructions per token and is issue bound far below
// HBM speed, this one needs ~3.
//
// Grid (streams of the layer, splits [+ g - 1], slots), CTAs of four warps in two groups, two per SM.  A CTA
// walks its share of the stream's 64-token tiles through a 3-stage ring filled by TMA (tensor maps over the K
// and V arenas, boxes of 64 dims x 64 rows, 128-byte swizzle, so ldmatrix reads are bank-conflict free); the
// groups take tiles in turn.  Warp w of a group owns tokens 32w..32w+31 of a tile -- the tokens are the M
// dimension of both products -- and keeps a private online softmax (running max, sum, 128 x 8 accumulator)
// in registers; warps merge through shared memory, splits through a global scratch whose words are their own
// arrival flags: with more than one split, head 0 of a stream is combined by the CTA of its last split and
// head h > 0 by a CTA of its own (grid y = splits + h - 1), which polls the partial rows of its head.
// Fused decode step: with k_new / v_new given, the launch also appends one token per stream
// (Algorithm 3's C^0 <- C^0 + {(k_j, v_j)}).  The new token never goes through the tiles: the combining
// CTAs score it in fp32 and add it as one more partial (weight 1), and the combiner of head 0 writes its
// row, its position and the stream's new level-0 length once its polls have shown that every CTA of the
// stream is past its tiles, i.e. has finished reading the old segment table.
// Rows of a tile beyond a segment's end are masked in the scores; their V rows are whatever the
// arena holds there (zero-initialised at creation or finite older rows) times an exact zero.
#include <cuda.h>

#include "common.cuh"

namespace bkv {

namespace {

// Shape of a CTA: kGroups warp groups that take the CTA's tiles in turn, each warp of a group owning
// kTB blocks of 16 tokens of a 64-token tile; kStages tiles in flight; kCtasPerSm resident CTAs.
constexpr int kGroups = 2;
constexpr int kTB = 2;
constexpr int kStages = 3;
constexpr int kCtasPerSm = 2;
constexpr int kWarpTokens = 16 * kTB;
constexpr int kGroupWarps = 64 / kWarpTokens;
constexpr int kGroupThreads = 32 * kGroupWarps;
constexpr int kWarps = kGroups * kGroupWarps;
constexpr int kThreads = 32 * kWarps;
constexpr int kBars = kGroups * kStages;      // tile i: stage i % kStages, barrier i % kBars (a multiple of kStages and kGroups)
constexpr int kTN = 64;                      // tokens per tile
constexpr int kD = 128;
constexpr uint32_t kHalf = kTN * 128;        // bytes of one [64 tokens][64 dims] bf16 box
constexpr uint32_t kTensorBytes = 2 * kHalf; // K (or V) tile: two boxes
constexpr uint32_t kStageBytes = 2 * kTensorBytes;
constexpr long long kWaitCycles = 100000000LL;   // about 50 ms: a bulk copy that has not landed by then never will
constexpr int PS = kD + 4;                   // row of the in-CTA merge buffer: acc[D], max, sum, 2 pad (bank-conflict free)

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
// Transpose of an 8 x 8 matrix of 16-bit elements held one row pair per thread (row lane / 4,
// columns 2 (lane % 4) and the next): turns C-fragment rows into B-fragment columns.
__device__ inline uint32_t movm_trans(uint32_t a) {
  uint32_t d;
  asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
  return d;
}
__device__ inline float fast_exp2(float x) {     // -inf -> 0
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
// Accesses to the split-K scratch (see the combine).  Publishing stores and polling loads are relaxed operations at
// GPU scope -- never served by L1, and not a data race although nothing else orders them: each word validates itself.
constexpr uint32_t kEmptyWord = 0xffffffffu;
constexpr int kMaxSplits = 64;
static_assert(2 * kWarps <= 8, "the scratch holds 8 floats of (max, sum) copies per partial row (decode_scratch_bytes)");
static_assert(kThreads == kD, "the combine maps a warp to 32 output columns");
__device__ inline bool is_empty(float x) { return __float_as_uint(x) == kEmptyWord; }
// Plain loads as volatile asm statements: they keep their place among the polling loads, i.e. they are issued
// before the polls and not where their values are first used.
__device__ inline uint2 ld_early_v2(const void* p) {
  uint2 v;
  asm volatile("ld.global.v2.u32 {%0, %1}, [%2];" : "=r"(v.x), "=r"(v.y) : "l"(p) : "memory");
  return v;
}
__device__ inline uint4 ld_early_v4(const void* p) {
  uint4 v;
  asm volatile("ld.global.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p) : "memory");
  return v;
}
__device__ inline float4 ld_poll4(const float* p) {
  float4 v;
  asm volatile("ld.relaxed.gpu.global.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p) : "memory");
  return v;
}
__device__ inline float2 ld_poll2(const float* p) {
  float2 v;
  asm volatile("ld.relaxed.gpu.global.v2.f32 {%0, %1}, [%2];" : "=f"(v.x), "=f"(v.y) : "l"(p) : "memory");
  return v;
}
__device__ inline void st_scratch4(float* p, float4 v) {
  asm volatile("st.relaxed.gpu.global.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(v.x), "f"(v.y), "f"(v.z), "f"(v.w) : "memory");
}
__device__ inline void st_scratch2(float* p, float2 v) {
  asm volatile("st.relaxed.gpu.global.v2.f32 [%0], {%1, %2};" ::"l"(p), "f"(v.x), "f"(v.y) : "memory");
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
  // blocks (partial rows and their pairs) of consecutive slots; raw_acc / raw_ml advance by one
  // [B, H g, d] / [B, H g, 2] block per slot; bit z of keys_mask = keys_only of slot z.
  int n_slots;
  int slot_layer[8];
  unsigned keys_mask;
  unsigned z_stride;
  // 1: the library's previous launch on this CUDA stream was a decode launch of this context, so
  // the only arena rows that can still be in flight are the one row per stream that launch
  // appended.  Every other tile may then be fetched before the grid dependency is resolved (see
  // the kernel's prologue).  Needs the segment table as a parameter (n_seg > 0).
  int early;
  // The step's operands (q, k_new, v_new) arrive by a copy on another CUDA stream that no event ties to
  // this launch: the copy is followed by a copy of the word `in_expect` to *in_flag, and the kernel
  // waits (bounded) for that word before it reads them.  nullptr: the operands are ordered before the
  // launch in the usual way.
  const int* in_flag;
  int in_expect;
  // Splits of a stream's tiles.  With more than one the grid has g - 1 more CTAs per stream, which combine
  // the heads 1 .. g - 1 (see the kernel's combine).
  int splits;
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

// Named barrier of one warp group (ids 1, 2; id 0 is __syncthreads) that also votes: true if any
// of the group's threads passes a true predicate.
__device__ inline bool group_bar_or(int group, bool pred) {
  uint32_t r;
  asm volatile(
      "{\n\t.reg .pred p, q;\n\t"
      "setp.ne.u32 q, %3, 0;\n\t"
      "bar.red.or.pred p, %1, %2, q;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(r) : "r"(group + 1), "r"(kGroupThreads), "r"((uint32_t)pred) : "memory");
  return r != 0;
}

__global__ void __launch_bounds__(kThreads, kCtasPerSm)
decode_mma_kernel(Geom G, Arena A, int layer, const __nv_bfloat16* __restrict__ q, __nv_bfloat16* __restrict__ out,
                  float* __restrict__ part_base, int* __restrict__ status,
                  const StepAppend ap, const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV) {
  float* part = part_base;
  float* raw_acc = ap.raw_acc;
  float* raw_ml = ap.raw_ml;
  int keys_only = ap.keys_only;
  if (ap.n_slots) {
    const int z = blockIdx.z;
    layer = ap.slot_layer[z];
    keys_only = (int)((ap.keys_mask >> z) & 1u);
    part += (size_t)z * ap.z_stride;
    raw_acc += (size_t)z * G.B * G.H * G.g * kD;
    raw_ml += (size_t)z * G.B * G.H * G.g * 2;
  }
  extern __shared__ unsigned char smem_raw[];
  unsigned char* tiles = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
  uint64_t* full = reinterpret_cast<uint64_t*>(tiles + kStages * kStageBytes);
  __shared__ int lvl_tiles[kMaxLevels + 1];
  __shared__ Seg seg_s[kMaxLevels + 1];

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int group = warp / kGroupWarps, wq = warp % kGroupWarps;   // tile parity served, token quarter of the tile
  const int g = G.g;
  const int sl = blockIdx.x;
  const int seq = sl / G.H, head = sl % G.H;
  const int stream = (seq * G.L + layer) * G.H + head;
  const int splits = ap.splits, split = blockIdx.y;     // split >= splits: a combiner without tiles (see the combine)
  const int64_t stream_base = (int64_t)stream * G.rows_per_stream;
  // Merge and combine phases: the first work item of this warp, (head mh, way mw) with warp = mw g + mh.
  int mh = warp, mw = 0;
  if (g < kWarps)
    while (mh >= g) { mh -= g; ++mw; }

  // Launched with programmatic stream serialization, this grid may become resident while the
  // previous kernel of the stream is still finishing.  What precedes griddepcontrol.wait touches
  // nothing that kernel may still write: barrier set-up, and -- in a chain of decode launches
  // (ap.early) -- the fetch of this CTA's first tiles, except the stream's last tile, which holds the
  // row the previous step appended.  The dependents are released only after the wait, so at most
  // one earlier launch of the chain is ever in flight.  Without the launch attribute both
  // instructions do nothing.
  if (tid == 0) {
    for (int s = 0; s < kBars; ++s) mbar_init(&full[s], 1);
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmK) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(&tmV) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
  }
  // The step's operands are wanted right after the dependency resolves: ask for them in L2 now.  A
  // line fetched before its producer has written it is harmless, L2 being the point of coherence
  // (the producer's write updates that line; nothing is taken into L1 here).
  if (ap.in_flag) {
    // operands still in flight: nothing to ask for yet
  } else if (tid < 2 * g) {
    const char* qrow = reinterpret_cast<const char*>(q + ((size_t)seq * (G.H * g) + (size_t)head * g + (tid >> 1)) * kD);
    asm volatile("prefetch.global.L2 [%0];" ::"l"(qrow + 128 * (tid & 1)));
  } else if (ap.k_new && tid < 2 * g + 4) {
    const int k = tid - 2 * g;
    const char* row = reinterpret_cast<const char*>((k & 2 ? ap.v_new : ap.k_new) + (size_t)sl * kD);
    asm volatile("prefetch.global.L2 [%0];" ::"l"(row + 128 * (k & 1)));
  }
  const bool early = ap.early && ap.n_seg;
  if (!early) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
  }
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
  const int my_tiles = split < splits ? t_end - t_begin : 0;

  auto issue = [&](int i) {   // one thread
    const TileRef tr = locate_tile(t_begin + i, lvl_tiles, seg_s, G.T, stream_base, G.region_off);
    unsigned char* st = tiles + (size_t)(i % kStages) * kStageBytes;
    uint64_t* bar = &full[i % kBars];
    mbar_expect_tx(bar, keys_only ? kTensorBytes : kStageBytes);
    tma_load_2d(st, &tmK, 0, (int)tr.row, bar);
    tma_load_2d(st + kHalf, &tmK, 64, (int)tr.row, bar);
    if (!keys_only) {
      tma_load_2d(st + kTensorBytes, &tmV, 0, (int)tr.row, bar);
      tma_load_2d(st + kTensorBytes + kHalf, &tmV, 64, (int)tr.row, bar);
    }
  };
  int issued = 0;
  if (tid == 0) {
    const int lim = min(kStages, my_tiles);
    while (issued < lim && !(early && t_begin + issued == n_tiles - 1)) issue(issued++);
  }
  if (early) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    if (tid == 0)
      while (issued < min(kStages, my_tiles)) issue(issued++);
  }
  if (ap.in_flag) {
    // the copy engine writes the operands, then the flag word (two copies in stream order)
    if (tid == 0) {
      const long long t0 = clock64();
      while (*reinterpret_cast<const volatile int*>(ap.in_flag) != ap.in_expect) {
        if (clock64() - t0 > kWaitCycles) { atomicCAS(status, kStatusOk, kStatusWaitTimeout); break; }
      }
      __threadfence();
    }
    __syncthreads();
  }

  const float sc = 1.4426950408889634f * G.inv_sqrt_d;
  constexpr uint32_t kFacOff = 4352 + kWarps * kMaxGroup * 32 * 16 + 4096;   // = the single-split rows' place (never both)

  // ---- the end of a head's path, by all threads of a CTA (thread = output column): the appended token
  // joins as one more partial (level 0, weight 1, <q, k_new> in fp32), the ratio or the raw parts are
  // written, and with h == 0 the token's row goes into the cache.
  struct NewTok {
    uint2 kn;                  // 4 dims of k_new per lane
    uint2 qv[kMaxGroup];       // 4 dims of q per lane and head (one head: slot 0)
    uint2 vn;                  // lanes 0-7: the columns 32 warp + 4 lane .. + 3 of v_new
    uint4 row_new;             // last warp: lanes 0-15 a piece of the row of K, lanes 16-31 of V
  };
  // h < 0: the queries of all heads
  auto load_new = [&](int h) -> NewTok {
    NewTok nt;
    nt.kn = make_uint2(0u, 0u);
    nt.vn = make_uint2(0u, 0u);
    nt.row_new = make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
    for (int k = 0; k < kMaxGroup; ++k) nt.qv[k] = make_uint2(0u, 0u);
    if (ap.k_new) {
      nt.kn = ld_early_v2(ap.k_new + (size_t)sl * kD + 4 * lane);
      if (lane < 8) nt.vn = ld_early_v2(ap.v_new + (size_t)sl * kD + 32 * warp + 4 * lane);
      const __nv_bfloat16* qs = q + ((size_t)seq * (G.H * g) + (size_t)head * g) * kD + 4 * lane;
      if (h >= 0) {
        nt.qv[0] = ld_early_v2(qs + (size_t)h * kD);
      } else {
#pragma unroll
        for (int k = 0; k < kMaxGroup; ++k)
          if (k < g) nt.qv[k] = ld_early_v2(qs + (size_t)k * kD);
      }
      if (h <= 0 && warp == kWarps - 1)
        nt.row_new = ld_early_v4(reinterpret_cast<const uint4*>((lane < 16 ? ap.k_new : ap.v_new) + (size_t)sl * kD) + (lane & 15));
    }
    return nt;
  };
  // base-2 logit of the appended token for the head whose query sits in slot qslot (by a whole warp)
  auto score_new = [&](const NewTok& nt, int qslot) -> float {
    const uint2 qv = nt.qv[qslot];
    const __nv_bfloat162 k01 = *reinterpret_cast<const __nv_bfloat162*>(&nt.kn.x), k23 = *reinterpret_cast<const __nv_bfloat162*>(&nt.kn.y);
    const __nv_bfloat162 q01 = *reinterpret_cast<const __nv_bfloat162*>(&qv.x), q23 = *reinterpret_cast<const __nv_bfloat162*>(&qv.y);
    float dot = __bfloat162float(q01.x) * __bfloat162float(k01.x);
    dot = fmaf(__bfloat162float(q01.y), __bfloat162float(k01.y), dot);
    dot = fmaf(__bfloat162float(q23.x), __bfloat162float(k23.x), dot);
    dot = fmaf(__bfloat162float(q23.y), __bfloat162float(k23.y), dot);
    return warp_sum(dot) * sc;
  };
  // a: lanes 0-7 of every warp hold the sums of the output columns 32 warp + 4 lane .. + 3
  auto finish = [&](int h, float4 a, float M, float L, const NewTok& nt, float x) {
    if (ap.k_new) {
      const float Mn = fmaxf(M, x);
      const float f = M == -INFINITY ? 0.f : fast_exp2(M - Mn), fN = fast_exp2(x - Mn);
      const __nv_bfloat162 v01 = *reinterpret_cast<const __nv_bfloat162*>(&nt.vn.x), v23 = *reinterpret_cast<const __nv_bfloat162*>(&nt.vn.y);
      a.x = fmaf(__bfloat162float(v01.x), fN, a.x * f); a.y = fmaf(__bfloat162float(v01.y), fN, a.y * f);
      a.z = fmaf(__bfloat162float(v23.x), fN, a.z * f); a.w = fmaf(__bfloat162float(v23.y), fN, a.w * f);
      L = fmaf(L, f, fN);
      M = Mn;
    }
    const size_t qh = (size_t)seq * (G.H * g) + (size_t)head * g + h;
    if (lane < 8) {
      const int c = 32 * warp + 4 * lane;
      if (raw_acc) {
        *reinterpret_cast<float4*>(raw_acc + qh * kD + c) = a;
        if (c == 0) { raw_ml[2 * qh] = M; raw_ml[2 * qh + 1] = L; }
      } else {
        const float inv = L > 0.f ? 1.0f / L : 0.f;
        __nv_bfloat162 o01 = __floats2bfloat162_rn(a.x * inv, a.y * inv), o23 = __floats2bfloat162_rn(a.z * inv, a.w * inv);
        uint2 w;
        w.x = *reinterpret_cast<uint32_t*>(&o01);
        w.y = *reinterpret_cast<uint32_t*>(&o23);
        *reinterpret_cast<uint2*>(out + qh * kD + c) = w;
      }
    }
    if (ap.k_new && h == 0 && warp == kWarps - 1) {
      // append: one 256-byte row of K and of V, the position, the new length of C^0
      const size_t dst_row = (size_t)stream_base + G.region_off[0] + ap.rel_row;
      __nv_bfloat16* dstp = static_cast<__nv_bfloat16*>(lane < 16 ? A.K : A.V) + dst_row * kD;
      reinterpret_cast<uint4*>(dstp)[lane & 15] = nt.row_new;
      float s2 = 0.f;                                         // ||k||^2 / ||v||^2 travel with the row
      const __nv_bfloat162* h2 = reinterpret_cast<const __nv_bfloat162*>(&nt.row_new);
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        const float2 fv = __bfloat1622float2(h2[i]);
        s2 = fmaf(fv.x, fv.x, s2);
        s2 = fmaf(fv.y, fv.y, s2);
      }
#pragma unroll
      for (int o = 8; o > 0; o >>= 1) s2 += __shfl_xor_sync(0xffffffffu, s2, o);
      const float v2 = __shfl_sync(0xffffffffu, s2, 16);
      if (lane == 0 && A.nrm) A.nrm[dst_row] = make_float2(s2, v2);
      if (lane == 1) {
        A.idx[dst_row] = ap.idx0;
        A.seg[(size_t)stream * (G.T + 1)].len = ap.new_len;
      }
    }
  };
  // Combine head h of this CTA's stream (see the combine below).  Warp w sums the columns 32 w .. 32 w + 31,
  // a 128-byte line of every partial row: lane = (row group rg = lane / 8, 16-byte piece lane % 8), the lane
  // takes the rows rg, rg + 4, ... (vector loads and stores: a quarter of the memory instructions that a
  // lane per column would need), and the four row groups meet by two shuffle steps.
  auto combine_head = [&](int h) {
    const int rg = lane >> 3;
    const float* rows = part + ((size_t)sl * splits * g + h) * kD + 32 * warp + 4 * (lane & 7);        // row of split sp: + sp rstep
    const float* mls = part + (size_t)gridDim.x * splits * g * kD + (((size_t)sl * g + h) * kWarps + warp) * splits * 2;   // this warp's copies of the head's pairs, split by split: one line or two for a polling warp
    const size_t rstep = (size_t)g * kD, mstep = 2;
    const NewTok nt = load_new(h);              // in flight during the polls
    const float* mlp[2] = {mls + (size_t)lane * mstep, mls + (size_t)(lane + 32) * mstep};
    float2 ml[2];
#pragma unroll
    for (int e = 0; e < 2; ++e) ml[e] = lane + 32 * e < splits ? ld_poll2(mlp[e]) : make_float2(-INFINITY, 0.f);
    constexpr int kPer = kMaxSplits / 4;
    float4 v[kPer];
#pragma unroll
    for (int i = 0; i < kPer; ++i)
      if (rg + 4 * i < splits) v[i] = ld_poll4(rows + (size_t)(rg + 4 * i) * rstep);
    const float x_new = ap.k_new ? score_new(nt, 0) : 0.f;      // while the polls are in flight
    // A round re-reads everything that was still empty, all loads in flight together (words checked one
    // after the other would cost a round trip each).
    const long long t0 = clock64();
    bool ok = true;
    for (;;) {
      bool pending = false;
#pragma unroll
      for (int e = 0; e < 2; ++e)
        if (lane + 32 * e < splits && (is_empty(ml[e].x) || is_empty(ml[e].y))) {
          ml[e] = ld_poll2(mlp[e]);
          pending = true;
        }
#pragma unroll
      for (int i = 0; i < kPer; ++i)
        if (rg + 4 * i < splits && (is_empty(v[i].x) || is_empty(v[i].y) || is_empty(v[i].z) || is_empty(v[i].w))) {
          v[i] = ld_poll4(rows + (size_t)(rg + 4 * i) * rstep);
          pending = true;
        }
      if (!pending) break;
      if (clock64() - t0 > kWaitCycles) { ok = false; break; }
    }
    __syncwarp();
    const float M = warp_max(fmaxf(ml[0].x, ml[1].x));
    const float f0 = ml[0].x == -INFINITY ? 0.f : fast_exp2(ml[0].x - M);
    const float f1 = ml[1].x == -INFINITY ? 0.f : fast_exp2(ml[1].x - M);
    const float L = warp_sum(fmaf(ml[0].y, f0, ml[1].y * f1));
    // the factors of all splits through shared memory (behind the merge buffers, which other warps of the
    // last split's CTA may still be reading)
    float* fac = reinterpret_cast<float*>(tiles + kFacOff) + warp * kMaxSplits;
    fac[lane] = f0;
    fac[lane + 32] = f1;
    __syncwarp();
    float4 a = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
    for (int i = 0; i < kPer; ++i)
      if (rg + 4 * i < splits) {
        const float f = fac[rg + 4 * i];
        a.x = fmaf(v[i].x, f, a.x); a.y = fmaf(v[i].y, f, a.y); a.z = fmaf(v[i].z, f, a.z); a.w = fmaf(v[i].w, f, a.w);
      }
#pragma unroll
    for (int o = 8; o < 32; o <<= 1) {
      a.x += __shfl_xor_sync(0xffffffffu, a.x, o); a.y += __shfl_xor_sync(0xffffffffu, a.y, o);
      a.z += __shfl_xor_sync(0xffffffffu, a.z, o); a.w += __shfl_xor_sync(0xffffffffu, a.w, o);
    }
    finish(h, a, M, L, nt, x_new);
    // the empty pattern again, for the next launch (every warp has its own copy of the pairs, so nobody else
    // still wants these words)
    {
      const float e = __uint_as_float(kEmptyWord);
#pragma unroll
      for (int i = 0; i < kPer; ++i)
        if (rg + 4 * i < splits) st_scratch4(const_cast<float*>(rows + (size_t)(rg + 4 * i) * rstep), make_float4(e, e, e, e));
#pragma unroll
      for (int k = 0; k < 2; ++k)
        if (lane + 32 * k < splits) st_scratch2(const_cast<float*>(mlp[k]), make_float2(e, e));
    }
    if (!ok && lane == 0) atomicCAS(status, kStatusOk, kStatusWaitTimeout);
  };
  if (split >= splits) {                        // a CTA without tiles: the combiner of head split - splits + 1
    combine_head(split - splits + 1);
    return;
  }

  // B fragments of the query tile (k = dims, n = query head of the group; heads >= g are zero).
  // The tokens are the M dimension of both products (S^T = K Q^T, O^T = V^T P^T), so a warp spends
  // one mma.sync.m16n8k16 per 16 tokens x 16 dims instead of the two that a query-major tile
  // (16 rows, at most 8 of them used) needs.
  const int hq = lane >> 2, tq = lane & 3;         // C fragment: rows hq, hq + 8; columns 2 tq, 2 tq + 1
  // With g <= 4 the columns 4-7 of the operand repeat the heads 0-3: both halves compute the same scores, and
  // in the second product the columns 0-3 carry the high parts of the probabilities and the columns 4-7 their
  // low parts, so that one MMA does what takes two with more heads; the halves are added before the merge.
  const bool packed = g <= 4;
  uint32_t qb[8][2];
  {
    const int hr = packed ? hq & 3 : hq;
    const __nv_bfloat16* qp = q + ((size_t)seq * (G.H * g) + (size_t)head * g + hr) * kD;
#pragma unroll
    for (int ks = 0; ks < 8; ++ks) {
      uint32_t lo = 0, hi = 0;
      if (hr < g) {
        lo = *reinterpret_cast<const uint32_t*>(qp + ks * 16 + 2 * tq);
        hi = *reinterpret_cast<const uint32_t*>(qp + ks * 16 + 8 + 2 * tq);
      }
      qb[ks][0] = lo; qb[ks][1] = hi;
    }
  }

  // O^T of this warp's tokens: o[mb][j] = dim 16 mb + hq + 8 (j >> 1), query head 2 tq + (j & 1)
  float o[8][4];
#pragma unroll
  for (int n = 0; n < 8; ++n) { o[n][0] = o[n][1] = o[n][2] = o[n][3] = 0.f; }
  float m_run[2] = {-INFINITY, -INFINITY}, l_run[2] = {0.f, 0.f};   // heads 2 tq, 2 tq + 1; l over this thread's tokens

  // ldmatrix row addresses of this lane (see the fragment layouts of mma.m16n8k16), for the first of
  // the warp's kTB 16-token blocks
  const int mi = lane >> 3, mr = lane & 7;
  const int k_tok = wq * kWarpTokens + (mi & 1) * 8 + mr, k_chunk = mi >> 1;     // K (A operand): x4 = (tok 0-7 | 8-15) x (dims lo | hi)
  const int v_tok = wq * kWarpTokens + (mi >> 1) * 8 + mr, v_chunk = mi & 1;     // V (A operand, transposed): x4 = (dims lo | hi) x (tok 0-7 | 8-15)

  // The warp groups take tiles in turn (one group: every tile).  With the tiles already in shared
  // memory the loop is bound by the latency of its dependency chain (barrier, score MMAs, softmax
  // shuffles, value MMAs).  Tile i lives in stage i % kStages whichever group consumes it; the
  // group that frees a stage refills it.
  bool failed = false;
  for (int i = group; i < my_tiles; i += kGroups) {
    const int s = i % kStages;
    // Barrier i % kBars serves tiles i, i + kBars, ... only, all of them this group's: the phase
    // before the awaited one is a tile the group has consumed itself, so the parity wait cannot be
    // a phase off although the groups advance independently.  One lane polls (every poll of a
    // barrier is a serialised shared-memory access).
    bool arrived = true;
    if (lane == 0) arrived = mbar_wait(&full[i % kBars], (uint32_t)((i / kBars) & 1));
    arrived = __shfl_sync(0xffffffffu, arrived, 0);
    __syncwarp();                  // the polling lane's view of the landed tile, for the whole warp
    const TileRef tr = locate_tile(t_begin + i, lvl_tiles, seg_s, G.T, stream_base, G.region_off);
    const uint32_t Kt = smem_u32(tiles + (size_t)s * kStageBytes), Vt = Kt + kTensorBytes;
    if (arrived && wq * kWarpTokens < tr.rows) {
      // ---- scores of the warp's tokens against the group's heads: S^T[16 x 8] = K Q^T per block.
      // A dependent mma.sync waits for its predecessor's whole latency and the asm statements keep
      // their order: operand loads go first, and the MMAs form 4 chains per block issued in turn.
      float sa[kTB][4][4];
#pragma unroll
      for (int tb = 0; tb < kTB; ++tb)
#pragma unroll
        for (int c = 0; c < 4; ++c) { sa[tb][c][0] = sa[tb][c][1] = sa[tb][c][2] = sa[tb][c][3] = 0.f; }
#pragma unroll
      for (int kh = 0; kh < 2; ++kh) {
        uint32_t ka[4][kTB][4];
#pragma unroll
        for (int k4 = 0; k4 < 4; ++k4)
#pragma unroll
          for (int tb = 0; tb < kTB; ++tb) ldsm_x4(Kt + tile_off(k_tok + 16 * tb, (kh * 4 + k4) * 2 + k_chunk), ka[k4][tb]);
#pragma unroll
        for (int k4 = 0; k4 < 4; ++k4)
#pragma unroll
          for (int tb = 0; tb < kTB; ++tb) mma_bf16(sa[tb][k4], ka[k4][tb], qb[kh * 4 + k4][0], qb[kh * 4 + k4][1]);
      }
      // the value operands do not depend on the probabilities: their loads are in flight during the softmax
      uint32_t va[kTB][8][4];
      if (!keys_only) {
#pragma unroll
        for (int tb = 0; tb < kTB; ++tb)
#pragma unroll
          for (int mb = 0; mb < 8; ++mb) ldsm_x4_trans(Vt + tile_off(v_tok + 16 * tb, mb * 2 + v_chunk), va[tb][mb]);
      }
      // this thread: per block tb the tokens tok0 (x[tb][0], x[tb][1]) and tok0 + 8 (x[tb][2], x[tb][3]),
      // heads 2 tq (even index) and 2 tq + 1
      const float lvl = (float)tr.level;
      float x[kTB][4];
      float mx0 = -INFINITY, mx1 = -INFINITY;
#pragma unroll
      for (int tb = 0; tb < kTB; ++tb) {
        const int tok0 = wq * kWarpTokens + tb * 16 + hq;
#pragma unroll
        for (int j = 0; j < 4; ++j)
          x[tb][j] = tok0 + 8 * (j >> 1) < tr.rows
                         ? fmaf((sa[tb][0][j] + sa[tb][1][j]) + (sa[tb][2][j] + sa[tb][3][j]), sc, lvl) : -INFINITY;
        mx0 = fmaxf(mx0, fmaxf(x[tb][0], x[tb][2]));
        mx1 = fmaxf(mx1, fmaxf(x[tb][1], x[tb][3]));
      }
#pragma unroll
      for (int off = 4; off < 32; off <<= 1) {
        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, off));
        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, off));
      }
      const float mn0 = fmaxf(m_run[0], mx0), mn1 = fmaxf(m_run[1], mx1);   // finite: the warp's first token of the tile is valid
      if (__any_sync(0xffffffffu, mn0 > m_run[0] || mn1 > m_run[1])) {
        const float a0 = fast_exp2(m_run[0] - mn0), a1 = fast_exp2(m_run[1] - mn1);   // m_run = -inf -> 0
        l_run[0] *= a0; l_run[1] *= a1;
#pragma unroll
        for (int n = 0; n < 8; ++n) { o[n][0] *= a0; o[n][1] *= a1; o[n][2] *= a0; o[n][3] *= a1; }
        m_run[0] = mn0; m_run[1] = mn1;
      }
      // The probabilities enter the second MMA as bf16: split them into a high and a low part
      // (p = hi + lo to 16 bits) so that the output error stays that of the final rounding.  Each
      // packed register is a row of an 8 x 8 [token][head] matrix; the B operand wants [head][token].
      uint32_t bh[kTB][2], bl[kTB][2];
#pragma unroll
      for (int tb = 0; tb < kTB; ++tb) {
#pragma unroll
        for (int j = 0; j < 4; ++j) x[tb][j] = fast_exp2(x[tb][j] - m_run[j & 1]);
        l_run[0] += x[tb][0] + x[tb][2];
        l_run[1] += x[tb][1] + x[tb][3];
        const uint32_t ph0 = pack_bf16(x[tb][0], x[tb][1]), ph1 = pack_bf16(x[tb][2], x[tb][3]);
        const uint32_t pl0 = pack_bf16(x[tb][0] - bf16_lo(ph0), x[tb][1] - bf16_hi(ph0));
        const uint32_t pl1 = pack_bf16(x[tb][2] - bf16_lo(ph1), x[tb][3] - bf16_hi(ph1));
        if (packed) {                          // this thread's two columns: high parts (tq < 2) or low parts
          bh[tb][0] = movm_trans(tq < 2 ? ph0 : pl0); bh[tb][1] = movm_trans(tq < 2 ? ph1 : pl1);
          bl[tb][0] = bl[tb][1] = 0u;
        } else {
          bh[tb][0] = movm_trans(ph0); bh[tb][1] = movm_trans(ph1);
          bl[tb][0] = movm_trans(pl0); bl[tb][1] = movm_trans(pl1);
        }
      }
      // ---- O^T[128 x 8] += V^T[128 x 16 kTB] P^T[16 kTB x 8]: the high parts of a block, then its low
      // parts, so that no MMA follows its predecessor on the same accumulator
      if (!keys_only) {
        if (packed) {
#pragma unroll
          for (int tb = 0; tb < kTB; ++tb)
#pragma unroll
            for (int mb = 0; mb < 8; ++mb) mma_bf16(o[mb], va[tb][mb], bh[tb][0], bh[tb][1]);
        } else {
#pragma unroll
          for (int tb = 0; tb < kTB; ++tb) {
#pragma unroll
            for (int mb = 0; mb < 8; ++mb) mma_bf16(o[mb], va[tb][mb], bh[tb][0], bh[tb][1]);
#pragma unroll
            for (int mb = 0; mb < 8; ++mb) mma_bf16(o[mb], va[tb][mb], bl[tb][0], bl[tb][1]);
          }
        }
      }
    }
    // the group has consumed stage s; the same barrier makes a timed-out wait a group-wide decision
    if (group_bar_or(group, !arrived)) { failed = true; break; }
    if (tid == group * kGroupThreads && i + kStages < my_tiles) issue(i + kStages);
  }
  if (failed && lane == 0 && wq == 0) atomicCAS(status, kStatusOk, kStatusWaitTimeout);

  // ---- merge the warps through shared memory (after the barrier the tile ring is idle)
  float* mrg = reinterpret_cast<float*>(tiles);        // [kWarps][g][PS]
#pragma unroll
  for (int off = 4; off < 32; off <<= 1) {
    l_run[0] += __shfl_xor_sync(0xffffffffu, l_run[0], off);
    l_run[1] += __shfl_xor_sync(0xffffffffu, l_run[1], off);
  }
  if (packed) {                                // high + low halves: the columns 2 tq + e and 2 tq + e + 4
#pragma unroll
    for (int n = 0; n < 8; ++n)
#pragma unroll
      for (int j = 0; j < 4; ++j) o[n][j] += __shfl_xor_sync(0xffffffffu, o[n][j], 2);
  }
  __syncthreads();
#pragma unroll
  for (int e = 0; e < 2; ++e) {
    const int h = 2 * tq + e;
    if (h < g) {
      float* rowp = mrg + ((size_t)warp * g + h) * PS;
#pragma unroll
      for (int n = 0; n < 8; ++n) { rowp[16 * n + hq] = o[n][e]; rowp[16 * n + 8 + hq] = o[n][2 + e]; }
      if (hq == 0) { rowp[kD] = m_run[e]; rowp[kD + 1] = l_run[e]; }
    }
  }
  __syncthreads();
  // With a single split the CTA's partial is the stream's result: it stays in shared memory (behind
  // the merge buffers) and goes straight to the end of the heads' path.
  constexpr uint32_t kMrg2Off = kWarps * kMaxGroup * PS * 4;        // behind mrg: [ways][g][PS] first-level merges
  constexpr uint32_t kSingleOff = 4352 + kWarps * kMaxGroup * 32 * 16 + 4096;   // behind the merge buffers and the combine's tables
  const bool single = splits == 1;
  // Partial results: per (stream, split, head) a row of kD column sums, and behind all rows the
  // (max, sum) pairs.  Rows of 512 bytes keep the staging copy 128-byte aligned.
  const size_t n_rows_all = (size_t)gridDim.x * splits * g;
  float* my_acc = single ? reinterpret_cast<float*>(tiles + kSingleOff) : part + ((size_t)sl * splits + split) * g * kD;
  float* my_ml = single ? reinterpret_cast<float*>(tiles + kSingleOff) + kMaxGroup * kD
                        : part + n_rows_all * kD + (size_t)sl * g * kWarps * splits * 2;       // pair of (head, copy, split): + ((h kWarps + copy) splits + split) 2
  // Work items of the merge and combine phases: (head mh, way mw), item r = mw g + mh, ways =
  // max(1, warps / g); a warp takes items r = warp, warp + kWarps, ... (lane = 4 output columns).
  // The ways of a head share its rows: way mw takes the rows mw, mw + ways, ...
  const int ways = g >= kWarps ? 1 : kWarps / g;
  const int n_r = g * ways;
  if (ways > 1) {
    // two levels, so that no thread walks all warps' rows
    float* mrg2 = reinterpret_cast<float*>(tiles + kMrg2Off);
    if (warp < n_r) {
      float mv[kWarps], M = -INFINITY;
#pragma unroll
      for (int k = 0; k < kWarps; ++k) {
        const int w = mw + k * ways;
        mv[k] = w < kWarps ? mrg[((size_t)w * g + mh) * PS + kD] : -INFINITY;
        M = fmaxf(M, mv[k]);
      }
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
      float L = 0.f;
#pragma unroll
      for (int k = 0; k < kWarps; ++k) {
        const int w = mw + k * ways;
        if (w < kWarps && mv[k] != -INFINITY) {
          const float* rowp = mrg + ((size_t)w * g + mh) * PS;
          const float f = fast_exp2(mv[k] - M);
          const float4 v = *reinterpret_cast<const float4*>(rowp + 4 * lane);
          acc.x = fmaf(v.x, f, acc.x); acc.y = fmaf(v.y, f, acc.y); acc.z = fmaf(v.z, f, acc.z); acc.w = fmaf(v.w, f, acc.w);
          L = fmaf(rowp[kD + 1], f, L);
        }
      }
      float* dst = mrg2 + ((size_t)mw * g + mh) * PS;
      *reinterpret_cast<float4*>(dst + 4 * lane) = acc;
      if (lane == 0) { dst[kD] = M; dst[kD + 1] = L; }
    }
    __syncthreads();
    mrg = mrg2;                                 // the second level reads `ways` rows per head
  }
  {
    const int n_src = ways > 1 ? ways : kWarps;
    for (int h = warp; h < g; h += kWarps) {
      float M = -INFINITY;
      for (int k = 0; k < n_src; ++k) M = fmaxf(M, mrg[((size_t)k * g + h) * PS + kD]);
      float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
      float L = 0.f;
      for (int k = 0; k < n_src; ++k) {
        const float* rowp = mrg + ((size_t)k * g + h) * PS;
        const float mk = rowp[kD];
        const float f = mk == -INFINITY ? 0.f : fast_exp2(mk - M);
        const float4 v = *reinterpret_cast<const float4*>(rowp + 4 * lane);
        acc.x = fmaf(v.x, f, acc.x); acc.y = fmaf(v.y, f, acc.y); acc.z = fmaf(v.z, f, acc.z); acc.w = fmaf(v.w, f, acc.w);
        L = fmaf(rowp[kD + 1], f, L);
      }
      if (single) {
        *reinterpret_cast<float4*>(my_acc + h * kD + 4 * lane) = acc;
        if (lane == 0) *reinterpret_cast<float2*>(my_ml + 2 * h) = make_float2(M, L);
      } else {                                  // published: see the combine below
        st_scratch4(my_acc + h * kD + 4 * lane, acc);
        if (lane < kWarps) st_scratch2(my_ml + ((size_t)(h * kWarps + lane) * splits + split) * 2, make_float2(M, L));   // a copy per combining warp
      }
    }
  }
  // ---- combine.  No ticket, no fence and no staging copy: a word of the scratch is its own arrival flag.
  // Between launches every word of the partial rows holds kEmptyWord, a NaN pattern that arithmetic never
  // produces (results are canonical NaNs, and -inf is a legal maximum).  A CTA publishes its rows with relaxed
  // stores.  Head 0 of a stream is combined by the stream's CTA of the last split, head h > 0 by the CTA
  // (stream, splits + h - 1), which has no tiles: the g combiners of a stream run side by side on different
  // SMs, each polls the words of its head until none is empty, sums, and puts the empty pattern back for the
  // next launch.  CTAs are dispatched in index order, so everything a combiner waits for was dispatched
  // before it and never waits itself: the wait ends (and is bounded anyway).  The chain behind the last tile
  // is then one store and about one load through L2 instead of fence, ticket, fence and copy.
  if (single) {
    __syncthreads();                            // the rows in shared memory are complete
    const float* acc1 = reinterpret_cast<const float*>(tiles + kSingleOff);
    const float* ml1 = acc1 + kMaxGroup * kD;
    NewTok nt = load_new(-1);
#pragma unroll
    for (int h = 0; h < kMaxGroup; ++h)
      if (h < g)
        finish(h, *reinterpret_cast<const float4*>(acc1 + h * kD + 32 * warp + 4 * (lane & 7)), ml1[2 * h], ml1[2 * h + 1], nt,
               ap.k_new ? score_new(nt, h) : 0.f);
    return;
  }
  if (split == splits - 1) combine_head(0);
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

constexpr size_t kSmemBytes = 1024 + (size_t)kStages * kStageBytes + kBars * sizeof(uint64_t);

}  // namespace

bool decode_mma_supported(const Geom& G) { return G.is_bf16 && G.d == kD && G.g <= 8; }
int decode_mma_ctas_per_sm() { return kCtasPerSm; }

// CTAs per stream of a launch with `splits` splits: the combiners of the heads 1 .. g - 1 have CTAs of their own.
int decode_mma_ctas_per_stream(int g, int splits) { return splits > 1 ? splits + g - 1 : 1; }
static unsigned grid_y(const Geom& G, int splits) { return (unsigned)decode_mma_ctas_per_stream(G.g, splits); }

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
                                   int rel_row, int idx0, int new_len, const Seg* seg_hint, int early, const int* in_flag,
                                   int in_expect, cudaStream_t st);

// Scratch layout of all launches: the CUDA-core kernel's ticket counters (unused here), then (stream, split,
// head) rows of kD column sums, then per row kWarps copies of its (max, sum) pair.
// Un-normalised parts (see StepAppend::raw_acc) of the layer's streams, for decode merged over slots.
cudaError_t launch_decode_parts_mma(const Geom& G, const Arena& A, int layer, const void* q, float* raw_acc, float* raw_ml,
                                    float* scratch, int splits, int* status, const void* maps, int keys_only,
                                    cudaStream_t st) {
  if (!maps || !raw_acc || !raw_ml) return cudaErrorInvalidValue;
  const DecodeMaps* tm = static_cast<const DecodeMaps*>(maps);
  const int n_sl = G.B * G.H;
  float* part = scratch + ((n_sl + 63) / 64) * 64;
  dim3 grid(n_sl, grid_y(G, splits));
  const StepAppend ap{nullptr, nullptr, 0, 0, 0, raw_acc, raw_ml, keys_only, 0, {}, 0, {}, 0u, 0u, 0, nullptr, 0, splits};
  decode_mma_kernel<<<grid, kThreads, kSmemBytes, st>>>(G, A, layer, static_cast<const __nv_bfloat16*>(q), nullptr, part,
                                                        status, ap, tm->k, tm->v);
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
  float* part = scratch + ((n_sl + 63) / 64) * 64;
  dim3 grid(n_sl, grid_y(G, splits), n_slots);
  StepAppend ap{nullptr, nullptr, 0, 0, 0, raw_acc, raw_ml, 0, 0, {}, n_slots, {}, keys_mask, (unsigned)z_stride_words, 0, nullptr, 0, splits};
  for (int i = 0; i < n_slots; ++i) ap.slot_layer[i] = slot_layers[i];
  decode_mma_kernel<<<grid, kThreads, kSmemBytes, st>>>(G, A, slot_layers[0], static_cast<const __nv_bfloat16*>(q), nullptr,
                                                        part, status, ap, tm->k, tm->v);
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
                                   int rel_row, int idx0, int new_len, const Seg* seg_hint, int early, const int* in_flag,
                                   int in_expect, cudaStream_t st) {
  if (!maps) return cudaErrorInvalidValue;
  const DecodeMaps* tm = static_cast<const DecodeMaps*>(maps);
  const int n_sl = G.B * G.H;
  float* part = scratch + ((n_sl + 63) / 64) * 64;
  dim3 grid(n_sl, grid_y(G, splits));
  StepAppend ap{static_cast<const __nv_bfloat16*>(k_new), static_cast<const __nv_bfloat16*>(v_new), rel_row, idx0,
                new_len, nullptr, nullptr, 0, 0, {}, 0, {}, 0u, 0u, 0, nullptr, 0, splits};
  if (seg_hint) {
    ap.n_seg = G.T + 1;
    for (int l = 0; l <= G.T; ++l) ap.seg[l] = seg_hint[l];
    ap.early = early ? 1 : 0;
  }
  ap.in_flag = in_flag;
  ap.in_expect = in_expect;
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
                            static_cast<__nv_bfloat16*>(out), part, status, ap, tm->k, tm->v);
}

}  // namespace bkv
