// C ABI of the BalanceKV library: context, memory layout, launch scheduling.
// Every step of the hot path runs in the CUDA kernels of this directory; this file only
// validates arguments, keeps Algorithm 3's bookkeeping (sched.h) and enqueues launches.
#include <climits>
#include <cmath>
#include <cstdint>
#include <cstdio>
#include <cstring>
#include <new>
#include <utility>
#include <vector>

#include <cuda.h>

#include "../../include/balancekv.h"
#include "common.cuh"
#include "sched.h"

using namespace bkv;

namespace bkv {
bool walk_tc_supported(const Geom& G);
cudaError_t walk_tc_prepare(const Geom& G, const Arena& A, int64_t total_rows, void** tmaps_out);
void walk_tc_release(void* tmaps);
bool decode_mma_supported(const Geom& G);
int decode_mma_ctas_per_sm();
cudaError_t decode_mma_prepare(const Geom& G, const Arena& A, int64_t total_rows, void** maps_out);
void decode_mma_release(void* maps);
cudaError_t launch_decode_parts_mma(const Geom& G, const Arena& A, int layer, const void* q, float* raw_acc, float* raw_ml,
                                    float* scratch, int splits, int* status, const void* maps, int keys_only,
                                    cudaStream_t st);
cudaError_t launch_decode_parts_mma_slots(const Geom& G, const Arena& A, const int* slot_layers, int n_slots,
                                          unsigned keys_mask, const void* q, float* raw_acc, float* raw_ml, float* scratch,
                                          size_t z_stride_words, int splits, int* status, const void* maps,
                                          cudaStream_t st);
cudaError_t launch_merged_ratio(const float* acc, const float* ml, int n_parts, unsigned num_mask, unsigned den_mask,
                                void* out, int n_heads, int d, cudaStream_t st);
cudaError_t launch_decode_step_mma(const Geom& G, const Arena& A, int layer, const void* q, void* out, float* scratch,
                                   int splits, int* status, const void* maps, const void* k_new, const void* v_new,
                                   int rel_row, int idx0, int new_len, const Seg* seg_hint, int early, const int* in_flag,
                                   int in_expect, cudaStream_t st);
}  // namespace bkv

#define BKV_CUDA(expr)                                                                    \
  do {                                                                                    \
    cudaError_t _e = (expr);                                                              \
    if (_e != cudaSuccess) {                                                              \
      std::fprintf(stderr, "balancekv: %s failed: %s (%s:%d)\n", #expr, cudaGetErrorString(_e), \
                   __FILE__, __LINE__);                                                   \
      return _e == cudaErrorMemoryAllocation ? BALANCEKV_E_NOMEM : BALANCEKV_E_CUDA;      \
    }                                                                                     \
  } while (0)

// Split-K scratch of the decode kernels: ticket counters (CUDA-core kernel: zero, self-resetting), then
// the partial rows.  The tensor-core kernel uses a word of a partial row as its own arrival flag: between
// launches every such word holds the all-ones pattern, which the combining CTA restores after reading.
static cudaError_t init_decode_scratch(float* scratch, size_t bytes, size_t n_sl, cudaStream_t st) {
  const size_t ticket_bytes = ((n_sl + 63) / 64) * 64 * sizeof(unsigned);
  cudaError_t e = cudaMemsetAsync(scratch, 0xff, bytes, st);
  if (e == cudaSuccess) e = cudaMemsetAsync(scratch, 0, ticket_bytes < bytes ? ticket_bytes : bytes, st);
  return e;
}

struct balancekv_ctx {
  balancekv_config cfg{};
  Geom G{};
  Layout Lo{};
  Arena A{};
  int n_streams = 0, device = 0, sm_count = 148;
  int64_t total_rows = 0;
  std::vector<StreamState> st;
  size_t bytes_resident = 0;
  int esz = 2;

  // per-launch buffers
  int max_calls = 0;
  CallStat* d_stats = nullptr;
  float* d_tokshift = nullptr;
  int8_t* d_eta = nullptr;
  unsigned long long* d_fail = nullptr;
  int* d_status = nullptr;
  int* h_status = nullptr;       // pinned mirror of the status word, refreshed after every compress batch and by stats
  float* d_decode_scratch = nullptr;
  int max_splits = 1;
  int decode_slots = 148;        // CTAs of the decode kernel that are resident at once
  bool use_tc = false;
  void* tmaps = nullptr;
  void* decode_maps = nullptr;   // tensor maps of the tensor-core decode kernel (bf16, d = 128)

  // descriptor ring: two halves of pinned host memory mirrored on the device
  char* h_ring = nullptr;
  char* d_ring = nullptr;
  size_t ring_half = 0, ring_pos = 0;
  int ring_cur = 0;
  cudaEvent_t ring_ev[2]{};
  bool ring_ev_valid[2] = {false, false};

  // debug records
  bool debug = false;
  int8_t* dbg_eta = nullptr;
  float* dbg_S = nullptr;
  float* dbg_p = nullptr;
  int64_t dbg_calls_per_stream = 0;
  int64_t dbg_level_base[kMaxLevels + 1] = {};

  // inspection view
  void* view_K = nullptr;
  void* view_V = nullptr;
  float* view_w = nullptr;
  int32_t* view_idx = nullptr;
  int64_t view_cap = 0;

  // staging for the *_host entry points
  void* bounce_K = nullptr;
  void* bounce_V = nullptr;
  size_t bounce_bytes = 0;
  void* bounce_q = nullptr;
  void* bounce_out = nullptr;
  // stream_step_host: q | k_new | v_new of a step packed into one pinned slot, one copy to the device
  static constexpr int kStepSlots = 64;
  char* step_host = nullptr;            // pinned, kStepSlots slots
  char* step_dev_in = nullptr;          // q | k | v, kStepSlots slots as well
  cudaStream_t step_copy_stream = nullptr;   // the transfers run beside the caller's stream
  cudaEvent_t step_used_ev[kStepSlots] = {}; // the step's kernel has finished (its slots may be reused)
  void* step_dev_out = nullptr;
  size_t step_slot_bytes = 0;
  cudaEvent_t step_ev[kStepSlots] = {};
  unsigned long long step_count = 0;
  const int* step_flag = nullptr;       // set by stream_step_host for the launch that follows: arrival flag of its operands
  int step_expect = 0;
  void* write_value_fn = nullptr;       // cuStreamWriteValue32, if the driver offers it
  cudaEvent_t step_group_ev[4] = {};    // kernels of 16 consecutive host steps have finished (their slots may be reused)
  // two-instance estimator: un-normalised parts of the numerator and denominator instances, unit values
  float* two_acc = nullptr;             // [BALANCEKV_MAX_MERGE][B, Hq, d] value sums per merged slot
  float* two_ml = nullptr;              // [BALANCEKV_MAX_MERGE][B, Hq, 2] (max, sum) per merged slot
  float* two_scratch = nullptr;         // [BALANCEKV_MAX_MERGE] split-K scratch blocks (laid out like d_decode_scratch)
  size_t two_scratch_words = 0;         // 4-byte words per block
  void* unit_V = nullptr;               // rows (1, 0, ..., 0) for balancekv_stream_append_layer_keys
  size_t unit_rows = 0;

  int64_t tokens_appended = 0, calls_run = 0, kernels_launched = 0;
  std::vector<std::vector<int>> layer_stream_ids;

  // Chain of decode launches: true while the last work this context enqueued was a launch of the
  // tensor-core decode kernel on chain_stream.  The next decode launch on that stream may then fetch
  // cache tiles before its grid dependency resolves (only the previous launch can still be running,
  // and it writes one row per stream).  Every other enqueuing call breaks the chain.
  bool decode_chain = false;
  cudaStream_t chain_stream = nullptr;

  // value-norm buckets (Algorithm 1): running v_max^2 and the largest erased bucket index, indexed
  // by the stream of the first bucket slot; routing buffers sized for the largest block so far
  std::vector<float> bucket_vmax2;
  std::vector<int32_t> bucket_erase_max;
  float* bkt_ns = nullptr;
  int8_t* bkt_slot = nullptr;
  int32_t* bkt_rank = nullptr;
  unsigned* bkt_vmax_bits = nullptr;
  int32_t* bkt_chunk_cnt = nullptr;     // per (stream, chunk of the block): counts, then their prefix
  size_t bkt_chunk_ints = 0;
  BucketOut* bkt_out = nullptr;
  BucketOut* bkt_out_host = nullptr;    // pinned
  size_t bkt_rows = 0, bkt_streams = 0;
  int64_t bucket_dropped = 0;
  // preservation of anti-correlated keys: column sums / mean scratch and the class of every row
  float* acr_scratch = nullptr;
  int8_t* acr_cls = nullptr;
  size_t acr_floats = 0, acr_rows = 0;

  // optional per-class kernel timing
  unsigned profiling = 0;                   // bit per kernel class
  int prof_every[BALANCEKV_PROFILE_CLASSES] = {1, 1, 1, 1, 1, 1};
  unsigned long long prof_seen[BALANCEKV_PROFILE_CLASSES] = {0, 0, 0, 0, 0, 0};
  std::vector<cudaEvent_t> prof_ev;     // pairs
  std::vector<int> prof_class;
  size_t prof_used = 0;
};

namespace {
constexpr size_t kProfMax = 8192;
// Brackets one kernel-class launch with events while profiling is on.
struct ProfScope {
  balancekv_ctx* c; cudaStream_t st; bool on;
  ProfScope(balancekv_ctx* c_, int cls, cudaStream_t st_) : c(c_), st(st_), on(false) {
    if (((c->profiling >> cls) & 1u) && c->prof_seen[cls]++ % c->prof_every[cls] == 0 && c->prof_used < kProfMax) {
      on = true;
      c->prof_class[c->prof_used] = cls;
      cudaEventRecord(c->prof_ev[2 * c->prof_used], st);
    }
  }
  ~ProfScope() {
    if (on) { cudaEventRecord(c->prof_ev[2 * c->prof_used + 1], st); c->prof_used++; }
  }
};
}  // namespace

namespace {

template <typename T>
int dev_alloc(balancekv_ctx* c, T** p, size_t count) {
  const size_t bytes = std::max<size_t>(count * sizeof(T), 256);
  BKV_CUDA(cudaMalloc(reinterpret_cast<void**>(p), bytes));
  c->bytes_resident += bytes;
  return BALANCEKV_OK;
}

// Copies a host array into the descriptor ring and returns its device address.
int ring_push(balancekv_ctx* c, const void* data, size_t bytes, cudaStream_t st, void** dev) {
  const size_t need = (bytes + 255) & ~(size_t)255;
  if (need > c->ring_half) return BALANCEKV_E_NOMEM;
  if (c->ring_pos + need > c->ring_half) {
    BKV_CUDA(cudaEventRecord(c->ring_ev[c->ring_cur], st));
    c->ring_ev_valid[c->ring_cur] = true;
    c->ring_cur ^= 1;
    c->ring_pos = 0;
    if (c->ring_ev_valid[c->ring_cur]) BKV_CUDA(cudaEventSynchronize(c->ring_ev[c->ring_cur]));
  }
  const size_t off = (size_t)c->ring_cur * c->ring_half + c->ring_pos;
  std::memcpy(c->h_ring + off, data, bytes);
  BKV_CUDA(cudaMemcpyAsync(c->d_ring + off, c->h_ring + off, bytes, cudaMemcpyHostToDevice, st));
  c->ring_pos += need;
  *dev = c->d_ring + off;
  return BALANCEKV_OK;
}

int stream_id(const balancekv_ctx* c, int seq, int layer, int head) {
  return (seq * c->cfg.n_layers + layer) * c->cfg.n_kv_heads + head;
}

int64_t dbg_offset(const balancekv_ctx* c, int stream, int level, int64_t ordinal) {
  return ((int64_t)stream * c->dbg_calls_per_stream + c->dbg_level_base[level] + ordinal) * c->cfg.block;
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

// A bounded device-side wait that gave up sets the context's status word.  The host sees it through
// a pinned mirror (no synchronisation): once set, every call that would enqueue more work refuses.
bool timed_out(const balancekv_ctx* c) { return c->h_status && *static_cast<volatile int*>(c->h_status) == kStatusWaitTimeout; }

int check_config(const balancekv_config& f) {
  if (f.n_seqs < 1 || f.n_layers < 1 || f.n_kv_heads < 1 || f.n_q_heads < 1) return BALANCEKV_E_INVAL;
  if (f.n_layers > 65535 || f.n_kv_heads > 65535) return BALANCEKV_E_INVAL;
  if (f.n_q_heads % f.n_kv_heads) return BALANCEKV_E_INVAL;
  const int g = f.n_q_heads / f.n_kv_heads;
  if (g < 1 || g > kMaxGroup) return BALANCEKV_E_INVAL;
  if (f.head_dim != 64 && f.head_dim != 128) return BALANCEKV_E_INVAL;
  if (f.dtype != 0 && f.dtype != 1) return BALANCEKV_E_INVAL;
  if (f.block < 64 || f.block % 64 || f.block > 4096) return BALANCEKV_E_INVAL;
  if (f.levels < 0 || f.levels > kMaxLevels) return BALANCEKV_E_INVAL;
  if (f.max_tokens < 1 || f.recent_window < 0) return BALANCEKV_E_INVAL;
  if (f.gram_path < 0 || f.gram_path > 2) return BALANCEKV_E_INVAL;
  if (f.decode_splits < 0 || f.decode_splits > 64) return BALANCEKV_E_INVAL;
  return BALANCEKV_OK;
}

// Builds the per-stream region layout (rows) for the given parameters.
void build_layout(const balancekv_config& f, int max_pending, Layout& Lo) {
  const int t = f.block, T = f.levels, N = f.max_tokens;
  Lo.t = t; Lo.T = T; Lo.W = f.recent_window;
  if (T == 0) {
    Lo.cap0 = N; Lo.capT = 0;
    Lo.region_off[0] = 0;
    Lo.R = N;
    return;
  }
  const int64_t calls_top = (int64_t)N / ((int64_t)t << (T - 1));
  Lo.capT = (int32_t)std::max<int64_t>(calls_top * (t / 2), ((int64_t)N + (1 << T) - 1) >> T);
  Lo.cap0 = (int32_t)std::min<int64_t>((int64_t)max_pending + 2 * ((int64_t)t + f.recent_window),
                                       (int64_t)N + 2 * ((int64_t)t + f.recent_window));
  int64_t off = 0;
  Lo.region_off[T] = (int32_t)off; off += Lo.capT;
  for (int l = T - 1; l >= 1; --l) { Lo.region_off[l] = (int32_t)off; off += 2 * t; }
  Lo.region_off[0] = (int32_t)off; off += Lo.cap0;
  Lo.R = (off + 63) / 64 * 64;
}

}  // namespace

extern "C" {

const char* balancekv_strerror(int code) {
  switch (code) {
    case BALANCEKV_OK: return "ok";
    case BALANCEKV_E_INVAL: return "invalid argument";
    case BALANCEKV_E_NOMEM: return "capacity or memory exhausted";
    case BALANCEKV_E_STATE: return "call not valid in the current state";
    case BALANCEKV_E_CUDA: return "CUDA runtime error";
    case BALANCEKV_E_TIMEOUT: return "device-side wait timed out";
  }
  return "unknown error";
}

int balancekv_create(const balancekv_config* cfg, balancekv_ctx** out) {
  if (!cfg || !out) return BALANCEKV_E_INVAL;
  *out = nullptr;
  int rc = check_config(*cfg);
  if (rc) return rc;
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev == 0) return BALANCEKV_E_CUDA;
  balancekv_ctx* c = new (std::nothrow) balancekv_ctx();
  if (!c) return BALANCEKV_E_NOMEM;
  c->cfg = *cfg;
  const balancekv_config& f = c->cfg;
  BKV_CUDA(cudaGetDevice(&c->device));
  BKV_CUDA(cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, c->device));
  c->esz = f.dtype ? 2 : 4;
  const int t = f.block, T = f.levels, N = f.max_tokens;
  const int max_pending = f.max_pending > 0 ? std::min(f.max_pending, N) : N;
  build_layout(f, max_pending, c->Lo);
  c->n_streams = f.n_seqs * f.n_layers * f.n_kv_heads;
  c->st.assign(c->n_streams, StreamState());

  // most level-0 calls of one batched launch, and the ping-pong pools behind the streams
  const size_t row_bytes = (size_t)f.head_dim * c->esz;
  if (T > 0) {
    const size_t per_call = (size_t)(t / 2) * row_bytes * 2;          // K+V survivors of one call
    // Both pools together: up to 1 GiB, so that a batched launch spans many waves of CTAs (a launch of
    // 256 calls is 1.7 waves on 148 SMs: 86 % of its slots), but no more than the level-0 calls that can
    // be pending at once.
    const size_t budget = (size_t)1 << 30;
    int64_t mc = (int64_t)(budget / (2 * per_call));
    const int64_t pending_calls = (int64_t)c->n_streams * ((max_pending + t - 1) / t);
    mc = std::max<int64_t>(2, std::min<int64_t>(std::min<int64_t>(mc, pending_calls), 4096));
    c->max_calls = (int)mc;
    c->Lo.pool_pairs = T > 1 ? (mc + 1) / 2 : 0;
  }
  const int64_t stream_rows = (int64_t)c->n_streams * c->Lo.R;
  c->Lo.pool_row[0] = stream_rows;
  c->Lo.pool_row[1] = stream_rows + c->Lo.pool_pairs * t;
  c->total_rows = stream_rows + 2 * c->Lo.pool_pairs * t;

  Geom& G = c->G;
  G.d = f.head_dim; G.t = t; G.T = T; G.H = f.n_kv_heads; G.L = f.n_layers; G.B = f.n_seqs;
  G.g = f.n_q_heads / f.n_kv_heads;
  G.is_bf16 = f.dtype;
  G.rows_per_stream = c->Lo.R;
  for (int l = 0; l <= kMaxLevels; ++l) G.region_off[l] = c->Lo.region_off[l];
  G.inv_sqrt_d = (float)(1.0 / std::sqrt((double)f.head_dim));
  {
    // c = 30 log(n/delta), natural log, n = tokens of a call, delta = 1/N^2 by default
    const double delta = f.delta > 0 ? (double)f.delta : 1.0 / ((double)N * (double)N);
    const double cc = f.c_override > 0 ? (double)f.c_override : 30.0 * std::log((double)t / delta);
    G.c = (float)cc;
  }
  G.fixed_rk2 = f.r_key > 0 ? (float)((double)f.r_key * f.r_key) : 0.f;
  G.fixed_rv2 = f.r_value > 0 ? (float)((double)f.r_value * f.r_value) : 0.f;
  G.seed = f.seed;
  G.center_keys = f.center_keys ? 1 : 0;

  auto fail = [&](int code) { balancekv_destroy(c); return code; };
  if ((rc = dev_alloc(c, reinterpret_cast<char**>(&c->A.K), (size_t)c->total_rows * row_bytes))) return fail(rc);
  if ((rc = dev_alloc(c, reinterpret_cast<char**>(&c->A.V), (size_t)c->total_rows * row_bytes))) return fail(rc);
  if ((rc = dev_alloc(c, &c->A.idx, (size_t)c->total_rows))) return fail(rc);
  if ((rc = dev_alloc(c, &c->A.nrm, (size_t)c->total_rows))) return fail(rc);
  if (cudaMemset(c->A.nrm, 0, sizeof(float2) * (size_t)c->total_rows) != cudaSuccess) return fail(BALANCEKV_E_CUDA);
  if ((rc = dev_alloc(c, &c->A.seg, (size_t)c->n_streams * (T + 1)))) return fail(rc);
  if (cudaMemset(c->A.seg, 0, sizeof(Seg) * (size_t)c->n_streams * (T + 1)) != cudaSuccess) return fail(BALANCEKV_E_CUDA);
  // rows that were never written must hold finite numbers: tiles of the decode kernels may
  // cover rows past a segment's end, which are masked to weight zero but still multiplied
  if (cudaMemset(c->A.K, 0, (size_t)c->total_rows * row_bytes) != cudaSuccess) return fail(BALANCEKV_E_CUDA);
  if (cudaMemset(c->A.V, 0, (size_t)c->total_rows * row_bytes) != cudaSuccess) return fail(BALANCEKV_E_CUDA);
  if (T > 0) {
    if ((rc = dev_alloc(c, &c->d_stats, (size_t)c->max_calls))) return fail(rc);
    if ((rc = dev_alloc(c, &c->d_eta, (size_t)c->max_calls * t))) return fail(rc);
    if (G.center_keys && (rc = dev_alloc(c, &c->d_tokshift, (size_t)c->max_calls * (t + f.head_dim)))) return fail(rc);
  }
  if ((rc = dev_alloc(c, &c->d_fail, 1))) return fail(rc);
  if ((rc = dev_alloc(c, &c->d_status, 1))) return fail(rc);
  if (cudaMemset(c->d_fail, 0, 256) != cudaSuccess || cudaMemset(c->d_status, 0, 256) != cudaSuccess) return fail(BALANCEKV_E_CUDA);
  if (cudaMallocHost(reinterpret_cast<void**>(&c->h_status), 64) != cudaSuccess) return fail(BALANCEKV_E_NOMEM);
  *c->h_status = 0;
  {
    const int n_sl = f.n_seqs * f.n_kv_heads;
    const int per_sm = f.gram_path != 1 && decode_mma_supported(G) ? decode_mma_ctas_per_sm() : 2;
    c->decode_slots = per_sm * c->sm_count;                                 // CTAs of one wave
    c->max_splits = std::max(1, std::min(64, c->decode_slots / n_sl));      // rounding down keeps one wave
    if (f.decode_splits > 0) c->max_splits = std::min(64, f.decode_splits);
    const size_t sb = decode_scratch_bytes(G, c->max_splits);
    if ((rc = dev_alloc(c, reinterpret_cast<char**>(&c->d_decode_scratch), sb))) return fail(rc);
    if (init_decode_scratch(c->d_decode_scratch, sb, (size_t)G.B * G.H, nullptr) != cudaSuccess) return fail(BALANCEKV_E_CUDA);
    if (cudaStreamSynchronize(nullptr) != cudaSuccess) return fail(BALANCEKV_E_CUDA);
  }
  c->ring_half = (size_t)4 << 20;
  if (cudaMallocHost(reinterpret_cast<void**>(&c->h_ring), 2 * c->ring_half) != cudaSuccess) return fail(BALANCEKV_E_NOMEM);
  if ((rc = dev_alloc(c, &c->d_ring, 2 * c->ring_half))) return fail(rc);
  for (int i = 0; i < 2; ++i)
    if (cudaEventCreateWithFlags(&c->ring_ev[i], cudaEventDisableTiming) != cudaSuccess) return fail(BALANCEKV_E_CUDA);

  // The kernel family follows from the shape alone; a supported shape whose tensor maps cannot be
  // prepared is an error, never a quiet change of kernels.
  const bool rows_ok = c->total_rows < ((int64_t)1 << 31);
  if (f.gram_path != 1 && decode_mma_supported(G) && rows_ok) {
    if (decode_mma_prepare(G, c->A, c->total_rows, &c->decode_maps) != cudaSuccess) return fail(BALANCEKV_E_CUDA);
  }
  const bool tc_ok = walk_tc_supported(G) && rows_ok;
  if (f.gram_path == 2 && !tc_ok) return fail(BALANCEKV_E_INVAL);
  c->use_tc = T > 0 && tc_ok && f.gram_path != 1;
  if (c->use_tc && walk_tc_prepare(G, c->A, c->total_rows, &c->tmaps) != cudaSuccess) return fail(BALANCEKV_E_CUDA);
  if (T > 0 && !c->use_tc) {
    if (!walk_simt_supported(G.d)) return fail(BALANCEKV_E_INVAL);
    if (walk_simt_smem_bytes(G.d, t) > (size_t)227 * 1024) return fail(BALANCEKV_E_INVAL);
  }
  *out = c;
  return BALANCEKV_OK;
}

int balancekv_destroy(balancekv_ctx* c) {
  if (!c) return BALANCEKV_E_INVAL;
  cudaDeviceSynchronize();
  walk_tc_release(c->tmaps);
  decode_mma_release(c->decode_maps);
  void* ptrs[] = {c->A.K, c->A.V, c->A.idx, c->A.seg, c->A.nrm, c->d_stats, c->d_tokshift, c->d_eta, c->d_fail, c->d_status,
                  c->d_decode_scratch, c->d_ring, c->dbg_eta, c->dbg_S, c->dbg_p, c->view_K, c->view_V, c->view_w,
                  c->view_idx, c->bounce_K, c->bounce_V, c->bounce_q, c->bounce_out, c->step_dev_in, c->step_dev_out, c->two_acc, c->two_ml, c->two_scratch, c->unit_V};
  for (void* p : ptrs)
    if (p) cudaFree(p);
  void* bkt[] = {c->bkt_ns, c->bkt_slot, c->bkt_rank, c->bkt_vmax_bits, c->bkt_out, c->bkt_chunk_cnt, c->acr_scratch, c->acr_cls};
  for (void* p : bkt)
    if (p) cudaFree(p);
  if (c->bkt_out_host) cudaFreeHost(c->bkt_out_host);
  if (c->h_ring) cudaFreeHost(c->h_ring);
  if (c->h_status) cudaFreeHost(c->h_status);
  if (c->step_host) cudaFreeHost(c->step_host);
  if (c->step_copy_stream) cudaStreamDestroy(c->step_copy_stream);
  for (cudaEvent_t e : c->step_used_ev)
    if (e) cudaEventDestroy(e);
  for (cudaEvent_t e : c->step_group_ev)
    if (e) cudaEventDestroy(e);
  for (cudaEvent_t e : c->step_ev)
    if (e) cudaEventDestroy(e);
  for (int i = 0; i < 2; ++i)
    if (c->ring_ev[i]) cudaEventDestroy(c->ring_ev[i]);
  for (cudaEvent_t e : c->prof_ev) cudaEventDestroy(e);
  delete c;
  return BALANCEKV_OK;
}

// Appends (level 0) or loads (level T) n rows per listed stream from a caller tensor laid
// out as consecutive [n, d] blocks in the order of `streams`.
static int append_impl(balancekv_ctx* c, const std::vector<int>& streams, int level, const void* K, const void* V,
                       const int32_t* idx, int n, cudaStream_t st, int whole_layer = -1) {
  if (!K || !V || n < 0) return BALANCEKV_E_INVAL;
  if (!aligned16(K) || !aligned16(V)) return BALANCEKV_E_INVAL;
  if (n == 0) return BALANCEKV_OK;
  if (timed_out(c)) return BALANCEKV_E_TIMEOUT;
  c->decode_chain = false;
  const balancekv_config& f = c->cfg;
  const Layout& Lo = c->Lo;
  const int T = Lo.T;
  const int max_pending = T == 0 ? f.max_tokens : (f.max_pending > 0 ? std::min(f.max_pending, f.max_tokens) : f.max_tokens);
  for (int s : streams) {
    const StreamState& S = c->st[s];
    if (level == 0) {
      if (S.appended + n > f.max_tokens) return BALANCEKV_E_NOMEM;
      if (S.pending + n > max_pending) return BALANCEKV_E_NOMEM;
      if ((int64_t)S.start0 + S.len0 + n > Lo.cap0) return BALANCEKV_E_NOMEM;
    } else {
      if ((int64_t)S.lvl_len[T] + n > Lo.capT) return BALANCEKV_E_NOMEM;
    }
  }
  if (whole_layer >= 0) {
    // lockstep layer: every stream has the same fill, so the kernel derives the descriptors
    const StreamState& S0 = c->st[streams[0]];
    bool same = true;
    for (int s : streams) {
      const StreamState& S = c->st[s];
      same &= S.start0 == S0.start0 && S.len0 == S0.len0 && S.appended == S0.appended && S.lvl_len[T] == S0.lvl_len[T];
    }
    if (same) {
      const int rel = level == 0 ? S0.start0 + S0.len0 : S0.lvl_len[T];
      const int idx0 = level == 0 ? (int)S0.appended : S0.lvl_len[T];
      const int new_len = (level == 0 ? S0.len0 : S0.lvl_len[T]) + n;
      for (int s : streams) {
        StreamState& S = c->st[s];
        if (level == 0) { S.len0 += n; S.appended += n; S.pending += n; c->tokens_appended += n; }
        else S.lvl_len[T] += n;
      }
      ProfScope ps(c, 0, st);
      BKV_CUDA(launch_append_uniform(c->G, c->A, whole_layer, level, rel, idx0, n, new_len, K, V, idx, st));
      c->kernels_launched++;
      return BALANCEKV_OK;
    }
  }
  std::vector<AppendDesc> descs(streams.size());
  for (size_t i = 0; i < streams.size(); ++i) {
    const int s = streams[i];
    StreamState& S = c->st[s];
    AppendDesc& D = descs[i];
    D.src_off = (int64_t)i * n * f.head_dim;
    D.stream = s; D.n = n; D.level = level; D.pad = 0;
    if (level == 0) {
      D.dst_row = (int64_t)s * Lo.R + Lo.region_off[0] + S.start0 + S.len0;
      D.idx0 = (int32_t)S.appended;
      S.len0 += n; S.appended += n; S.pending += n;
      D.new_len = S.len0;
      c->tokens_appended += n;
    } else {
      D.dst_row = (int64_t)s * Lo.R + Lo.region_off[T] + S.lvl_len[T];
      D.idx0 = S.lvl_len[T];
      S.lvl_len[T] += n;
      D.new_len = S.lvl_len[T];
    }
  }
  void* d_descs = nullptr;
  int rc = ring_push(c, descs.data(), descs.size() * sizeof(AppendDesc), st, &d_descs);
  if (rc) return rc;
  {
    ProfScope ps(c, 0, st);
    BKV_CUDA(launch_append(c->G, c->A, static_cast<const AppendDesc*>(d_descs), (int)descs.size(), n, K, V, idx, st));
  }
  c->kernels_launched++;
  return BALANCEKV_OK;
}

int balancekv_stream_append(balancekv_ctx* c, int seq, int layer, int kv_head, const void* K_blk, const void* V_blk,
                            int n_tokens, void* stream) {
  if (!c) return BALANCEKV_E_INVAL;
  const balancekv_config& f = c->cfg;
  if (seq < 0 || seq >= f.n_seqs || layer < 0 || layer >= f.n_layers || kv_head < 0 || kv_head >= f.n_kv_heads)
    return BALANCEKV_E_INVAL;
  std::vector<int> s{stream_id(c, seq, layer, kv_head)};
  return append_impl(c, s, 0, K_blk, V_blk, nullptr, n_tokens, static_cast<cudaStream_t>(stream));
}

static const std::vector<int>& layer_streams(balancekv_ctx* c, int layer) {
  if (c->layer_stream_ids.empty()) c->layer_stream_ids.resize(c->cfg.n_layers);
  std::vector<int>& v = c->layer_stream_ids[layer];
  if (v.empty())
    for (int s = 0; s < c->cfg.n_seqs; ++s)
      for (int h = 0; h < c->cfg.n_kv_heads; ++h) v.push_back(stream_id(c, s, layer, h));
  return v;
}

int balancekv_stream_append_layer(balancekv_ctx* c, int layer, const void* K, const void* V, int n_tokens, void* stream) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers) return BALANCEKV_E_INVAL;
  return append_impl(c, layer_streams(c, layer), 0, K, V, nullptr, n_tokens, static_cast<cudaStream_t>(stream), layer);
}

int balancekv_stream_append_layer_host(balancekv_ctx* c, int layer, const void* K_host, const void* V_host,
                                       int n_tokens, void* stream) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers || !K_host || !V_host || n_tokens < 0) return BALANCEKV_E_INVAL;
  if (n_tokens == 0) return BALANCEKV_OK;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t bytes = (size_t)c->cfg.n_seqs * c->cfg.n_kv_heads * n_tokens * c->cfg.head_dim * c->esz;
  if (bytes > c->bounce_bytes) {
    BKV_CUDA(cudaStreamSynchronize(st));
    if (c->bounce_K) { cudaFree(c->bounce_K); cudaFree(c->bounce_V); c->bytes_resident -= 2 * c->bounce_bytes; }
    c->bounce_K = c->bounce_V = nullptr; c->bounce_bytes = 0;
    BKV_CUDA(cudaMalloc(&c->bounce_K, bytes));
    BKV_CUDA(cudaMalloc(&c->bounce_V, bytes));
    c->bounce_bytes = bytes; c->bytes_resident += 2 * bytes;
  }
  BKV_CUDA(cudaMemcpyAsync(c->bounce_K, K_host, bytes, cudaMemcpyHostToDevice, st));
  BKV_CUDA(cudaMemcpyAsync(c->bounce_V, V_host, bytes, cudaMemcpyHostToDevice, st));
  return append_impl(c, layer_streams(c, layer), 0, c->bounce_K, c->bounce_V, nullptr, n_tokens, st, layer);
}

int balancekv_cache_load_level(balancekv_ctx* c, int layer, int level, const void* K, const void* V,
                               const int32_t* orig_idx, int n_tokens, void* stream) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers) return BALANCEKV_E_INVAL;
  if (level != 0 && level != c->cfg.levels) return BALANCEKV_E_INVAL;
  return append_impl(c, layer_streams(c, layer), level, K, V, orig_idx, n_tokens, static_cast<cudaStream_t>(stream), layer);
}

// Runs one planned batch: per level radii -> walk -> selection/compaction, then the
// level-0 remainder moves and the segment-table update.
static int run_plan(balancekv_ctx* c, Plan& P, cudaStream_t st) {
  const Geom& G = c->G;
  c->decode_chain = false;
  // Every descriptor array of the batch (the calls of each level, the remainder moves, the segment
  // updates) travels in one transfer ahead of the first kernel, so that no copy sits between two
  // kernels of the batch; if they do not fit one half of the ring they go array by array.
  auto pad = [](size_t b) { return (b + 255) & ~(size_t)255; };
  size_t total = 0;
  for (int l = 0; l < G.T; ++l) {
    if (c->debug)
      for (CallDesc& d : P.levels[l]) d.dbg_off = dbg_offset(c, d.stream, l, d.ordinal);
    total += pad(P.levels[l].size() * sizeof(CallDesc));
  }
  const size_t off_moves = total;
  total += pad(P.moves.size() * sizeof(MoveDesc));
  const size_t off_segs = total;
  total += pad(P.segs.size() * sizeof(SegUpdate));
  char* d_all = nullptr;
  if (total > 0 && total <= c->ring_half) {
    std::vector<char> host(total);
    size_t off = 0;
    for (int l = 0; l < G.T; ++l) {
      const size_t b = P.levels[l].size() * sizeof(CallDesc);
      if (b) std::memcpy(host.data() + off, P.levels[l].data(), b);
      off += pad(b);
    }
    if (!P.moves.empty()) std::memcpy(host.data() + off_moves, P.moves.data(), P.moves.size() * sizeof(MoveDesc));
    if (!P.segs.empty()) std::memcpy(host.data() + off_segs, P.segs.data(), P.segs.size() * sizeof(SegUpdate));
    void* dv = nullptr;
    int rc = ring_push(c, host.data(), total, st, &dv);
    if (rc) return rc;
    d_all = static_cast<char*>(dv);
  }
  size_t off_level = 0;
  for (int l = 0; l < G.T; ++l) {
    std::vector<CallDesc>& calls = P.levels[l];
    const size_t level_base = off_level;
    off_level += pad(calls.size() * sizeof(CallDesc));
    if (calls.empty()) continue;
    for (size_t first = 0; first < calls.size(); first += c->max_calls) {
      const int n = (int)std::min<size_t>(c->max_calls, calls.size() - first);
      void* d_calls = d_all ? d_all + level_base + first * sizeof(CallDesc) : nullptr;
      if (!d_all) {
        int rc = ring_push(c, calls.data() + first, (size_t)n * sizeof(CallDesc), st, &d_calls);
        if (rc) return rc;
      }
      const CallDesc* dc = static_cast<const CallDesc*>(d_calls);
      // the tensor-core walk kernel takes the radii from the stored row norms itself
      const bool need_radii = (G.center_keys || G.fixed_rk2 <= 0.f || G.fixed_rv2 <= 0.f) &&
                              !(c->use_tc && !G.center_keys && c->A.nrm);
      if (need_radii) {
        ProfScope ps(c, 1, st);
        BKV_CUDA(launch_radii(G, c->A, dc, n, c->d_stats, c->d_tokshift, st));
        c->kernels_launched += 1 + (G.center_keys ? 1 : 0);
      }
      if (c->use_tc) {
        ProfScope ps(c, 2, st);
        BKV_CUDA(launch_walk_tc(G, c->A, dc, n, l, c->d_stats, c->d_tokshift, c->d_eta, c->dbg_eta, c->dbg_S,
                                c->dbg_p, c->d_fail, c->d_status, c->tmaps, c, st));   // selection + compaction fused at the tail
      } else {
        ProfScope ps(c, 2, st);
        BKV_CUDA(launch_walk_simt(G, c->A, dc, n, l, c->d_stats, c->d_tokshift, c->d_eta, c->dbg_eta, c->dbg_S,
                                  c->dbg_p, c->d_fail, st));
      }
      if (!c->use_tc) {
        ProfScope ps(c, 3, st);
        BKV_CUDA(launch_compact(G, c->A, dc, n, l, c->d_eta, st));
        c->kernels_launched++;
      }
      c->kernels_launched++;
      c->calls_run += n;
    }
  }
  if (!P.moves.empty()) {
    void* d_moves = d_all ? d_all + off_moves : nullptr;
    if (!d_all) {
      int rc = ring_push(c, P.moves.data(), P.moves.size() * sizeof(MoveDesc), st, &d_moves);
      if (rc) return rc;
    }
    ProfScope ps(c, 5, st);
    BKV_CUDA(launch_move(G, c->A, static_cast<const MoveDesc*>(d_moves), (int)P.moves.size(), P.max_move_rows, st));
    c->kernels_launched++;
  }
  if (!P.segs.empty()) {
    void* d_segs = d_all ? d_all + off_segs : nullptr;
    if (!d_all) {
      int rc = ring_push(c, P.segs.data(), P.segs.size() * sizeof(SegUpdate), st, &d_segs);
      if (rc) return rc;
    }
    ProfScope ps(c, 5, st);
    BKV_CUDA(launch_seg_update(c->A, static_cast<const SegUpdate*>(d_segs), (int)P.segs.size(), st));
    c->kernels_launched++;
  }
  // refresh the host's view of the status word behind the batch (4 bytes, no synchronisation)
  BKV_CUDA(cudaMemcpyAsync(c->h_status, c->d_status, sizeof(int), cudaMemcpyDeviceToHost, st));
  return BALANCEKV_OK;
}

static int compress_streams(balancekv_ctx* c, const std::vector<int>& streams, int T, cudaStream_t st) {
  if (T != c->cfg.levels) return BALANCEKV_E_INVAL;
  if (timed_out(c)) return BALANCEKV_E_TIMEOUT;
  for (int s : streams) c->st[s].pending = 0;
  if (T == 0) return BALANCEKV_OK;
  // greedy batches of at most max_calls level-0 calls
  std::vector<int64_t> left(streams.size());
  bool any = false;
  for (size_t i = 0; i < streams.size(); ++i) { left[i] = ready_blocks(c->Lo, c->st[streams[i]]); any |= left[i] > 0; }
  Plan P;
  while (any) {
    std::vector<std::pair<int, int>> runs;
    int budget = c->max_calls;
    any = false;
    for (size_t i = 0; i < streams.size() && budget > 0; ++i) {
      if (left[i] <= 0) continue;
      const int take = (int)std::min<int64_t>(left[i], budget);
      runs.emplace_back(streams[i], take);
      left[i] -= take; budget -= take;
    }
    for (size_t i = 0; i < streams.size(); ++i) any |= left[i] > 0;
    if (runs.empty()) break;
    if (!plan_batch(c->Lo, c->st.data(), runs, P)) return BALANCEKV_E_STATE;
    int rc = run_plan(c, P, st);
    if (rc) return rc;
  }
  return BALANCEKV_OK;
}

int balancekv_compress(balancekv_ctx* c, int T, void* stream) {
  if (!c) return BALANCEKV_E_INVAL;
  std::vector<int> all(c->n_streams);
  for (int i = 0; i < c->n_streams; ++i) all[i] = i;
  return compress_streams(c, all, T, static_cast<cudaStream_t>(stream));
}

int balancekv_compress_layer(balancekv_ctx* c, int layer, int T, void* stream) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers) return BALANCEKV_E_INVAL;
  return compress_streams(c, layer_streams(c, layer), T, static_cast<cudaStream_t>(stream));
}

// The layer's segment table as the host mirrors it, if all its streams hold the same segments
// (lockstep streams): out[l] = (start, len) of level l.  False if they differ.
static bool layer_seg_hint(balancekv_ctx* c, int layer, Seg* out) {
  const int T = c->cfg.levels;
  const std::vector<int>& streams = layer_streams(c, layer);
  const StreamState& S0 = c->st[streams[0]];
  for (int s : streams) {
    const StreamState& S = c->st[s];
    if (S.start0 != S0.start0 || S.len0 != S0.len0) return false;
    for (int l = 1; l <= T; ++l)
      if (S.lvl_len[l] != S0.lvl_len[l] || (l < T && S.lvl_base[l] != S0.lvl_base[l])) return false;
  }
  out[0] = Seg{S0.start0, S0.len0};
  for (int l = 1; l < T; ++l) out[l] = Seg{S0.lvl_base[l], S0.lvl_len[l]};
  if (T >= 1) out[T] = Seg{0, S0.lvl_len[T]};
  return true;
}

// Split-K factor of a decode launch over the layer's current caches.
// The tensor-core decode kernel adds g - 1 combining CTAs per stream to a launch with more than one split:
// the largest split factor <= splits whose grid over n_streams streams still fits one wave.
static int one_wave_splits(balancekv_ctx* c, int splits, int n_streams) {
  const int per_stream = c->decode_slots / std::max(1, n_streams);
  const int room = per_stream - (c->cfg.n_q_heads / c->cfg.n_kv_heads - 1);
  return std::max(1, std::min(splits, room));
}

static int pick_splits(balancekv_ctx* c, int layer) {
  const balancekv_config& f = c->cfg;
  int64_t max_rows = 0;
  for (int s = 0; s < f.n_seqs; ++s)
    for (int h = 0; h < f.n_kv_heads; ++h) {
      const StreamState& S = c->st[stream_id(c, s, layer, h)];
      int64_t rows = S.len0;
      for (int l = 1; l <= f.levels; ++l) rows += S.lvl_len[l];
      max_rows = std::max(max_rows, rows);
    }
  const int tile_tokens = 16384 / (f.head_dim * c->esz);
  const int64_t tiles = (max_rows + tile_tokens - 1) / tile_tokens + f.levels;
  int splits = (int)std::max<int64_t>(1, std::min<int64_t>(c->max_splits, (tiles + 1) / 2));
  // the fewest splits with the same number of tiles per CTA: the tile phase is as long, the combine shorter
  const int64_t tiles_per = std::max<int64_t>(1, (tiles + splits - 1) / splits);
  splits = (int)std::max<int64_t>(1, (tiles + tiles_per - 1) / tiles_per);
  if (c->decode_maps) splits = one_wave_splits(c, splits, c->cfg.n_seqs * c->cfg.n_kv_heads);
  if (f.decode_splits > 0) splits = std::min(f.decode_splits, c->max_splits);
  return splits;
}

int balancekv_decode_attn(balancekv_ctx* c, int layer, const void* q, void* out, void* stream) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers || !q || !out) return BALANCEKV_E_INVAL;
  if (!aligned16(q) || !aligned16(out)) return BALANCEKV_E_INVAL;
  if (timed_out(c)) return BALANCEKV_E_TIMEOUT;
  const int splits = pick_splits(c, layer);
  {
    ProfScope ps(c, 4, static_cast<cudaStream_t>(stream));
    if (c->decode_maps) {
      Seg hint[kMaxLevels + 1];
      const bool alike = layer_seg_hint(c, layer, hint);
      cudaStream_t st = static_cast<cudaStream_t>(stream);
      const int early = alike && c->decode_chain && c->chain_stream == st;
      BKV_CUDA(launch_decode_step_mma(c->G, c->A, layer, q, out, c->d_decode_scratch, splits, c->d_status, c->decode_maps,
                                      nullptr, nullptr, 0, 0, 0, alike ? hint : nullptr, early, nullptr, 0, st));
      c->decode_chain = true;
      c->chain_stream = st;
    } else
      BKV_CUDA(launch_decode(c->G, c->A, layer, q, out, c->d_decode_scratch, splits, c->d_status,
                             static_cast<cudaStream_t>(stream)));
  }
  c->kernels_launched++;
  return BALANCEKV_OK;
}

int balancekv_decode_attn_host(balancekv_ctx* c, int layer, const void* q_host, void* out_host, void* stream) {
  if (!c || !q_host || !out_host) return BALANCEKV_E_INVAL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t bytes = (size_t)c->cfg.n_seqs * c->cfg.n_q_heads * c->cfg.head_dim * c->esz;
  if (!c->bounce_q) {
    BKV_CUDA(cudaMalloc(&c->bounce_q, bytes));
    BKV_CUDA(cudaMalloc(&c->bounce_out, bytes));
    c->bytes_resident += 2 * bytes;
  }
  BKV_CUDA(cudaMemcpyAsync(c->bounce_q, q_host, bytes, cudaMemcpyHostToDevice, st));
  int rc = balancekv_decode_attn(c, layer, c->bounce_q, c->bounce_out, stream);
  if (rc) return rc;
  BKV_CUDA(cudaMemcpyAsync(out_host, c->bounce_out, bytes, cudaMemcpyDeviceToHost, st));
  return BALANCEKV_OK;
}

int balancekv_stream_append_layer_keys(balancekv_ctx* c, int layer, const void* K, int n_tokens, void* stream) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers || !K || n_tokens < 0) return BALANCEKV_E_INVAL;
  if (n_tokens == 0) return BALANCEKV_OK;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t rows = (size_t)c->cfg.n_seqs * c->cfg.n_kv_heads * n_tokens;
  if (rows > c->unit_rows) {   // (re)build the unit-value rows: the value "1" of Algorithm 1's denominator instance
    const size_t rb = (size_t)c->cfg.head_dim * c->esz;
    BKV_CUDA(cudaStreamSynchronize(st));
    if (c->unit_V) { cudaFree(c->unit_V); c->bytes_resident -= c->unit_rows * rb; }
    c->unit_V = nullptr; c->unit_rows = 0;
    BKV_CUDA(cudaMalloc(&c->unit_V, rows * rb));
    BKV_CUDA(cudaMemsetAsync(c->unit_V, 0, rows * rb, st));
    // element 0 of every row = 1.0 (bf16 0x3F80 / fp32 0x3F800000): a strided 2-D set of the high bytes
    if (c->esz == 2) {
      BKV_CUDA(cudaMemset2DAsync(static_cast<char*>(c->unit_V) + 1, rb, 0x3F, 1, rows, st));
      BKV_CUDA(cudaMemset2DAsync(c->unit_V, rb, 0x80, 1, rows, st));
    } else {
      BKV_CUDA(cudaMemset2DAsync(static_cast<char*>(c->unit_V) + 3, rb, 0x3F, 1, rows, st));
      BKV_CUDA(cudaMemset2DAsync(static_cast<char*>(c->unit_V) + 2, rb, 0x80, 1, rows, st));
    }
    c->unit_rows = rows; c->bytes_resident += rows * rb;
  }
  return append_impl(c, layer_streams(c, layer), 0, K, c->unit_V, nullptr, n_tokens, st, layer);
}

int balancekv_decode_attn_merged(balancekv_ctx* c, const int32_t* layers_num, int n_num, const int32_t* layers_den,
                                 int n_den, const void* q, void* out, void* stream) {
  if (!c || !q || !out || !layers_num || !layers_den || n_num < 1 || n_den < 1) return BALANCEKV_E_INVAL;
  if (!aligned16(q) || !aligned16(out)) return BALANCEKV_E_INVAL;
  if (!c->decode_maps) return BALANCEKV_E_INVAL;          // bf16, head_dim 128, group <= 8 only
  if (timed_out(c)) return BALANCEKV_E_TIMEOUT;
  c->decode_chain = false;
  // distinct slots in order of first appearance, with the sides they enter
  int slots[BALANCEKV_MAX_MERGE];
  unsigned num_mask = 0, den_mask = 0;
  int n_parts = 0;
  for (int side = 0; side < 2; ++side) {
    const int32_t* ls = side ? layers_den : layers_num;
    for (int i = 0; i < (side ? n_den : n_num); ++i) {
      if (ls[i] < 0 || ls[i] >= c->cfg.n_layers) return BALANCEKV_E_INVAL;
      int p = 0;
      while (p < n_parts && slots[p] != ls[i]) ++p;
      if (p == n_parts) {
        if (n_parts == BALANCEKV_MAX_MERGE) return BALANCEKV_E_INVAL;
        slots[n_parts++] = ls[i];
      }
      unsigned& mask = side ? den_mask : num_mask;
      if ((mask >> p) & 1u) return BALANCEKV_E_INVAL;      // a slot twice on one side
      mask |= 1u << p;
    }
  }
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int n_heads = c->cfg.n_seqs * c->cfg.n_q_heads, d = c->cfg.head_dim;
  if (!c->two_acc) {   // first call: buffers for the un-normalised parts (allocates)
    BKV_CUDA(cudaMalloc(reinterpret_cast<void**>(&c->two_acc), sizeof(float) * (size_t)n_heads * d * BALANCEKV_MAX_MERGE));
    BKV_CUDA(cudaMalloc(reinterpret_cast<void**>(&c->two_ml), sizeof(float) * (size_t)n_heads * 2 * BALANCEKV_MAX_MERGE));
    c->bytes_resident += sizeof(float) * (size_t)n_heads * (d + 2) * BALANCEKV_MAX_MERGE;
    // one split-K scratch block per slot, so that all slots go in one launch
    const size_t block_bytes = (decode_scratch_bytes(c->G, c->max_splits) + 255) & ~(size_t)255;
    BKV_CUDA(cudaMalloc(reinterpret_cast<void**>(&c->two_scratch), block_bytes * BALANCEKV_MAX_MERGE));
    for (int z = 0; z < BALANCEKV_MAX_MERGE; ++z)
      BKV_CUDA(init_decode_scratch(reinterpret_cast<float*>(reinterpret_cast<char*>(c->two_scratch) + block_bytes * z), block_bytes,
                                   (size_t)c->G.B * c->G.H, st));
    c->two_scratch_words = block_bytes / 4;
    c->bytes_resident += block_bytes * BALANCEKV_MAX_MERGE;
  }
  // One launch over all slots (grid z = slot).  The split factor is the largest any slot asks for,
  // bounded so that the whole grid stays within one wave where it can.
  int splits = 1;
  unsigned keys_mask = 0;
  for (int p = 0; p < n_parts; ++p) {
    splits = std::max(splits, pick_splits(c, slots[p]));
    if (!((num_mask >> p) & 1u)) keys_mask |= 1u << p;     // a slot that only enters the denominator: values are not read
  }
  const int n_sl = c->cfg.n_seqs * c->cfg.n_kv_heads;
  splits = one_wave_splits(c, splits, n_sl * n_parts);
  {
    ProfScope ps(c, 4, st);
    BKV_CUDA(launch_decode_parts_mma_slots(c->G, c->A, slots, n_parts, keys_mask, q, c->two_acc, c->two_ml, c->two_scratch,
                                           c->two_scratch_words, splits, c->d_status, c->decode_maps, st));
  }
  BKV_CUDA(launch_merged_ratio(c->two_acc, c->two_ml, n_parts, num_mask, den_mask, out, n_heads, d, st));
  c->kernels_launched += 2;
  return BALANCEKV_OK;
}

int balancekv_decode_attn_two(balancekv_ctx* c, int layer_num, int layer_den, const void* q, void* out, void* stream) {
  const int32_t n = layer_num, dn = layer_den;
  return balancekv_decode_attn_merged(c, &n, 1, &dn, 1, q, out, stream);
}

// True if balancekv_stream_step will serve this layer's step with the one fused launch.
static bool step_can_fuse(balancekv_ctx* c, int layer) {
  if (!c->decode_maps) return false;
  const balancekv_config& f = c->cfg;
  const Layout& Lo = c->Lo;
  const std::vector<int>& streams = layer_streams(c, layer);
  const int max_pending = Lo.T == 0 ? f.max_tokens : (f.max_pending > 0 ? std::min(f.max_pending, f.max_tokens) : f.max_tokens);
  const StreamState& S0 = c->st[streams[0]];
  for (int s : streams) {
    const StreamState& S = c->st[s];
    if (S.start0 != S0.start0 || S.len0 != S0.len0 || S.appended != S0.appended) return false;
    if (S.appended + 1 > f.max_tokens || S.pending + 1 > max_pending || (int64_t)S.start0 + S.len0 + 1 > Lo.cap0) return false;
  }
  return true;
}

int balancekv_stream_step(balancekv_ctx* c, int layer, const void* q, const void* k_new, const void* v_new, void* out,
                          void* stream) {
  if (c && timed_out(c)) return BALANCEKV_E_TIMEOUT;
  // One launch when the tensor-core decode kernel serves this context and the layer's streams are
  // in lockstep with room for the token: the kernel appends after attending (see its header).
  if (c && layer >= 0 && layer < c->cfg.n_layers && c->decode_maps && q && out && k_new && v_new && aligned16(q) &&
      aligned16(out) && aligned16(k_new) && aligned16(v_new)) {
    const balancekv_config& f = c->cfg;
    const Layout& Lo = c->Lo;
    const std::vector<int>& streams = layer_streams(c, layer);
    const int max_pending = Lo.T == 0 ? f.max_tokens : (f.max_pending > 0 ? std::min(f.max_pending, f.max_tokens) : f.max_tokens);
    const StreamState& S0 = c->st[streams[0]];
    bool fits = true;
    for (int s : streams) {
      const StreamState& S = c->st[s];
      fits &= S.start0 == S0.start0 && S.len0 == S0.len0 && S.appended == S0.appended;
      fits &= S.appended + 1 <= f.max_tokens && S.pending + 1 <= max_pending && (int64_t)S.start0 + S.len0 + 1 <= Lo.cap0;
    }
    if (fits) {
      const int splits = pick_splits(c, layer);
      Seg hint[kMaxLevels + 1];
      const bool alike = layer_seg_hint(c, layer, hint);       // the table before this step's append
      const int rel = S0.start0 + S0.len0, idx0 = (int)S0.appended, new_len = S0.len0 + 1;
      for (int s : streams) {
        StreamState& S = c->st[s];
        S.len0 += 1; S.appended += 1; S.pending += 1; c->tokens_appended += 1;
      }
      cudaStream_t st = static_cast<cudaStream_t>(stream);
      const int early = alike && c->decode_chain && c->chain_stream == st;
      ProfScope ps(c, 4, st);
      BKV_CUDA(launch_decode_step_mma(c->G, c->A, layer, q, out, c->d_decode_scratch, splits, c->d_status, c->decode_maps,
                                      k_new, v_new, rel, idx0, new_len, alike ? hint : nullptr, early, c->step_flag, c->step_expect, st));
      c->step_flag = nullptr;
      c->decode_chain = true;
      c->chain_stream = st;
      c->kernels_launched++;
      return BALANCEKV_OK;
    }
  }
  int rc = balancekv_stream_append_layer(c, layer, k_new, v_new, 1, stream);
  if (rc) return rc;
  return balancekv_decode_attn(c, layer, q, out, stream);
}

int balancekv_stream_step_host(balancekv_ctx* c, int layer, const void* q_host, const void* k_host, const void* v_host,
                               void* out_host, void* stream) {
  if (!c || layer < 0 || layer >= c->cfg.n_layers || !q_host || !k_host || !v_host || !out_host) return BALANCEKV_E_INVAL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t qb = (size_t)c->cfg.n_seqs * c->cfg.n_q_heads * c->cfg.head_dim * c->esz;
  const size_t kb = (size_t)c->cfg.n_seqs * c->cfg.n_kv_heads * c->cfg.head_dim * c->esz;
  const size_t payload = (qb + 2 * kb + 15) / 16 * 16;
  if (!c->step_host) {   // first call: staging buffers (allocates)
    c->step_slot_bytes = (payload + 16 + 255) / 256 * 256;          // q | k | v | arrival flag
    BKV_CUDA(cudaHostAlloc(reinterpret_cast<void**>(&c->step_host), c->step_slot_bytes * balancekv_ctx::kStepSlots,
                           cudaHostAllocDefault));
    std::memset(c->step_host, 0, c->step_slot_bytes * balancekv_ctx::kStepSlots);
    BKV_CUDA(cudaMalloc(reinterpret_cast<void**>(&c->step_dev_in), c->step_slot_bytes * balancekv_ctx::kStepSlots));
    BKV_CUDA(cudaMemset(c->step_dev_in, 0, c->step_slot_bytes * balancekv_ctx::kStepSlots));
    BKV_CUDA(cudaMalloc(&c->step_dev_out, qb));
    c->bytes_resident += c->step_slot_bytes * balancekv_ctx::kStepSlots + qb;
    for (cudaEvent_t& e : c->step_ev) BKV_CUDA(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
    for (cudaEvent_t& e : c->step_used_ev) BKV_CUDA(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
    for (cudaEvent_t& e : c->step_group_ev) BKV_CUDA(cudaEventCreateWithFlags(&e, cudaEventDisableTiming));
    if (!c->step_copy_stream) BKV_CUDA(cudaStreamCreateWithFlags(&c->step_copy_stream, cudaStreamNonBlocking));
    cudaDriverEntryPointQueryResult qres;
    void* fn = nullptr;
    if (cudaGetDriverEntryPoint("cuStreamWriteValue32", &fn, cudaEnableDefault, &qres) == cudaSuccess &&
        qres == cudaDriverEntryPointSuccess)
      c->write_value_fn = fn;
    else
      (void)cudaGetLastError();
  }
  // The three small inputs travel as one copy: packed into a pinned slot on the host, then one
  // host-to-device transfer into the slot's device twin on the library's copy stream, so that the
  // transfer of a step runs while the previous step's kernel does.  With the fused step kernel no event
  // ties the launch to the transfer (an event wait between two steps would keep the next step's CTAs
  // from becoming resident early): a second small copy writes an arrival word behind the operands and
  // the kernel waits, bounded, for that word.  Otherwise the step's kernels wait for the transfer
  // through an event.  A slot is reused only after the kernel that read it has finished (one event
  // per 16 steps).
  constexpr int kSlots = balancekv_ctx::kStepSlots, kGroup = kSlots / 4;
  const unsigned long long n = c->step_count++;
  const int slot = (int)(n % kSlots), group = slot / kGroup;
  if (n >= (unsigned long long)kSlots && slot % kGroup == 0) BKV_CUDA(cudaEventSynchronize(c->step_group_ev[group]));
  char* h = c->step_host + (size_t)slot * c->step_slot_bytes;
  char* dev_in = c->step_dev_in + (size_t)slot * c->step_slot_bytes;
  std::memcpy(h, q_host, qb);
  std::memcpy(h + qb, k_host, kb);
  std::memcpy(h + qb + kb, v_host, kb);
  const bool fused = step_can_fuse(c, layer);
  BKV_CUDA(cudaMemcpyAsync(dev_in, h, qb + 2 * kb, cudaMemcpyHostToDevice, c->step_copy_stream));
  if (fused) {
    const int expect = (int)((n + 1) & 0x7fffffffu);
    // the arrival word: a stream memory operation behind the transfer (a 16-byte copy where the driver has none)
    typedef CUresult (*WriteValueFn)(CUstream, CUdeviceptr, cuuint32_t, unsigned int);
    bool written = false;
    if (c->write_value_fn)
      written = reinterpret_cast<WriteValueFn>(c->write_value_fn)(c->step_copy_stream, (CUdeviceptr)(uintptr_t)(dev_in + payload),
                                                                  (cuuint32_t)expect, 0) == CUDA_SUCCESS;
    if (!written) {
      *reinterpret_cast<int*>(h + payload) = expect;
      BKV_CUDA(cudaMemcpyAsync(dev_in + payload, h + payload, 16, cudaMemcpyHostToDevice, c->step_copy_stream));
    }
    c->step_flag = reinterpret_cast<const int*>(dev_in + payload);
    c->step_expect = expect;
  } else {
    BKV_CUDA(cudaEventRecord(c->step_ev[slot], c->step_copy_stream));
    BKV_CUDA(cudaStreamWaitEvent(st, c->step_ev[slot], 0));
  }
  // A pinned (mapped) result buffer is written by the kernel itself: the 8 KB of a step then need
  // no transfer of their own.  Pageable memory goes through the device buffer and a copy.
  void* out_dev = nullptr;
  {
    cudaPointerAttributes at;
    if (cudaPointerGetAttributes(&at, out_host) == cudaSuccess && at.type == cudaMemoryTypeHost && at.devicePointer &&
        aligned16(at.devicePointer))
      out_dev = at.devicePointer;
    else
      (void)cudaGetLastError();
  }
  int rc = balancekv_stream_step(c, layer, dev_in, dev_in + qb, dev_in + qb + kb, out_dev ? out_dev : c->step_dev_out, stream);
  c->step_flag = nullptr;
  if (slot % kGroup == kGroup - 1) BKV_CUDA(cudaEventRecord(c->step_group_ev[group], st));
  if (rc) return rc;
  if (!out_dev) BKV_CUDA(cudaMemcpyAsync(out_host, c->step_dev_out, qb, cudaMemcpyDeviceToHost, st));
  return BALANCEKV_OK;
}

int balancekv_level_sizes(balancekv_ctx* c, int seq, int layer, int kv_head, int32_t* sizes) {
  if (!c || !sizes) return BALANCEKV_E_INVAL;
  const balancekv_config& f = c->cfg;
  if (seq < 0 || seq >= f.n_seqs || layer < 0 || layer >= f.n_layers || kv_head < 0 || kv_head >= f.n_kv_heads)
    return BALANCEKV_E_INVAL;
  const StreamState& S = c->st[stream_id(c, seq, layer, kv_head)];
  sizes[0] = S.len0;
  for (int l = 1; l <= f.levels; ++l) sizes[l] = S.lvl_len[l];
  return BALANCEKV_OK;
}

int balancekv_cache_view(balancekv_ctx* c, int seq, int layer, int kv_head, const void** K, const void** V,
                         const float** w, const int32_t** orig_idx, int* len) {
  if (!c) return BALANCEKV_E_INVAL;
  const balancekv_config& f = c->cfg;
  if (seq < 0 || seq >= f.n_seqs || layer < 0 || layer >= f.n_layers || kv_head < 0 || kv_head >= f.n_kv_heads)
    return BALANCEKV_E_INVAL;
  BKV_CUDA(cudaDeviceSynchronize());
  c->decode_chain = false;
  const int s = stream_id(c, seq, layer, kv_head);
  const StreamState& S = c->st[s];
  int64_t total = S.len0;
  for (int l = 1; l <= f.levels; ++l) total += S.lvl_len[l];
  if (total > c->view_cap) {
    void* old[] = {c->view_K, c->view_V, c->view_w, c->view_idx};
    for (void* p : old) if (p) cudaFree(p);
    c->view_K = c->view_V = nullptr; c->view_w = nullptr; c->view_idx = nullptr;
    const int64_t cap = std::max<int64_t>(total, 1024);
    const size_t rb = (size_t)f.head_dim * c->esz;
    BKV_CUDA(cudaMalloc(&c->view_K, cap * rb));
    BKV_CUDA(cudaMalloc(&c->view_V, cap * rb));
    BKV_CUDA(cudaMalloc(reinterpret_cast<void**>(&c->view_w), cap * sizeof(float)));
    BKV_CUDA(cudaMalloc(reinterpret_cast<void**>(&c->view_idx), cap * sizeof(int32_t)));
    c->view_cap = cap;
  }
  const size_t rb = (size_t)f.head_dim * c->esz;
  int64_t pos = 0;
  for (int l = f.levels; l >= 0; --l) {
    const int64_t n = l == 0 ? S.len0 : S.lvl_len[l];
    if (n == 0) continue;
    const int64_t start = l == 0 ? S.start0 : (l == f.levels ? 0 : S.lvl_base[l]);
    const int64_t row = (int64_t)s * c->Lo.R + c->Lo.region_off[l] + start;
    BKV_CUDA(cudaMemcpy(static_cast<char*>(c->view_K) + pos * rb, static_cast<char*>(c->A.K) + row * rb, n * rb, cudaMemcpyDeviceToDevice));
    BKV_CUDA(cudaMemcpy(static_cast<char*>(c->view_V) + pos * rb, static_cast<char*>(c->A.V) + row * rb, n * rb, cudaMemcpyDeviceToDevice));
    BKV_CUDA(cudaMemcpy(c->view_idx + pos, c->A.idx + row, n * sizeof(int32_t), cudaMemcpyDeviceToDevice));
    BKV_CUDA(launch_fill_weights(c->view_w + pos, (int)n, std::ldexp(1.0f, l), 0));
    pos += n;
  }
  BKV_CUDA(cudaDeviceSynchronize());
  if (K) *K = c->view_K;
  if (V) *V = c->view_V;
  if (w) *w = c->view_w;
  if (orig_idx) *orig_idx = c->view_idx;
  if (len) *len = (int)total;
  return BALANCEKV_OK;
}

int balancekv_debug_enable(balancekv_ctx* c, int on) {
  if (!c) return BALANCEKV_E_INVAL;
  if (!on) { c->debug = false; return BALANCEKV_OK; }
  if (c->cfg.levels == 0) return BALANCEKV_OK;
  if (!c->dbg_eta) {
    if (c->calls_run > 0) return BALANCEKV_E_STATE;
    const int64_t blocks = c->cfg.max_tokens / c->cfg.block;
    int64_t base = 0;
    for (int l = 0; l < c->cfg.levels; ++l) { c->dbg_level_base[l] = base; base += blocks >> l; }
    c->dbg_calls_per_stream = std::max<int64_t>(base, 1);
    const size_t n = (size_t)c->n_streams * c->dbg_calls_per_stream * c->cfg.block;
    int rc;
    if ((rc = dev_alloc(c, &c->dbg_eta, n))) return rc;
    if ((rc = dev_alloc(c, &c->dbg_S, n))) return rc;
    if ((rc = dev_alloc(c, &c->dbg_p, n))) return rc;
  }
  c->debug = true;
  return BALANCEKV_OK;
}

int balancekv_debug_call(balancekv_ctx* c, int seq, int layer, int kv_head, int level, int call_ordinal,
                         const int8_t** eta, const float** S, const float** p, int* m) {
  if (!c || !c->dbg_eta) return BALANCEKV_E_STATE;
  const balancekv_config& f = c->cfg;
  if (seq < 0 || seq >= f.n_seqs || layer < 0 || layer >= f.n_layers || kv_head < 0 || kv_head >= f.n_kv_heads)
    return BALANCEKV_E_INVAL;
  if (level < 0 || level >= f.levels) return BALANCEKV_E_INVAL;
  const int s = stream_id(c, seq, layer, kv_head);
  if (call_ordinal < 0 || call_ordinal >= c->st[s].calls_done[level]) return BALANCEKV_E_INVAL;
  const int64_t off = dbg_offset(c, s, level, call_ordinal);
  if (eta) *eta = c->dbg_eta + off;
  if (S) *S = c->dbg_S + off;
  if (p) *p = c->dbg_p + off;
  if (m) *m = f.block;
  return BALANCEKV_OK;
}

// Algorithm 1's bucketing step for the streams `heads` (pairs seq, kv_head) whose blocks lie
// consecutively in K, V.  Slot layer0 + b is the instance of bucket index i_top - b.
static int append_bucketed_impl(balancekv_ctx* c, const std::vector<std::pair<int, int>>& heads, int layer0,
                                int n_buckets, int i_top, const void* K, const void* V, int n, float rho,
                                int8_t* token_slot, int32_t* counts_host, cudaStream_t st, bool preserve = false,
                                float tau = 0.f) {
  const balancekv_config& f = c->cfg;
  const Layout& Lo = c->Lo;
  if (!K || !V || n < 1 || n > (1 << 22) || !aligned16(K) || !aligned16(V)) return BALANCEKV_E_INVAL;
  if (n_buckets < 1 || n_buckets > kMaxBuckets || layer0 < 0 || layer0 + n_buckets > f.n_layers) return BALANCEKV_E_INVAL;
  if (i_top < -60 || i_top > 60 || !(rho >= 0.f) || rho > 1.f) return BALANCEKV_E_INVAL;
  const int n_sl = (int)heads.size();
  if (n_sl < 1) return BALANCEKV_E_INVAL;
  if (timed_out(c)) return BALANCEKV_E_TIMEOUT;
  c->decode_chain = false;
  if (c->bucket_vmax2.empty()) {
    c->bucket_vmax2.assign(c->n_streams, 0.f);
    c->bucket_erase_max.assign(c->n_streams, INT32_MIN);
  }
  // routing buffers (grown with the largest block; the call synchronises the stream anyway)
  if ((size_t)n_sl * n > c->bkt_rows || (size_t)n_sl > c->bkt_streams || bucket_chunk_count_ints(n_sl, n) > c->bkt_chunk_ints) {
    BKV_CUDA(cudaStreamSynchronize(st));
    void* old[] = {c->bkt_ns, c->bkt_slot, c->bkt_rank, c->bkt_vmax_bits, c->bkt_out, c->bkt_chunk_cnt};
    for (void* p : old)
      if (p) cudaFree(p);
    if (c->bkt_out_host) cudaFreeHost(c->bkt_out_host);
    c->bkt_ns = nullptr; c->bkt_slot = nullptr; c->bkt_rank = nullptr; c->bkt_vmax_bits = nullptr; c->bkt_out = nullptr;
    c->bkt_out_host = nullptr; c->bkt_chunk_cnt = nullptr;
    c->bkt_chunk_ints = std::max(c->bkt_chunk_ints, bucket_chunk_count_ints(n_sl, n));
    BKV_CUDA(cudaMalloc(reinterpret_cast<void**>(&c->bkt_chunk_cnt), sizeof(int32_t) * c->bkt_chunk_ints));
    c->bkt_rows = std::max(c->bkt_rows, (size_t)n_sl * n);
    c->bkt_streams = std::max(c->bkt_streams, (size_t)n_sl);
    BKV_CUDA(cudaMalloc(reinterpret_cast<void**>(&c->bkt_ns), sizeof(float) * c->bkt_rows));
    BKV_CUDA(cudaMalloc(reinterpret_cast<void**>(&c->bkt_slot), c->bkt_rows));
    BKV_CUDA(cudaMalloc(reinterpret_cast<void**>(&c->bkt_rank), sizeof(int32_t) * c->bkt_rows));
    BKV_CUDA(cudaMalloc(reinterpret_cast<void**>(&c->bkt_vmax_bits), sizeof(unsigned) * c->bkt_streams));
    BKV_CUDA(cudaMalloc(reinterpret_cast<void**>(&c->bkt_out), sizeof(BucketOut) * c->bkt_streams));
    BKV_CUDA(cudaMallocHost(reinterpret_cast<void**>(&c->bkt_out_host), sizeof(BucketOut) * c->bkt_streams));
  }
  std::vector<BucketIn> in(n_sl);
  for (int i = 0; i < n_sl; ++i) {
    const int s0 = stream_id(c, heads[i].first, layer0, heads[i].second);
    in[i].prev_vmax2 = c->bucket_vmax2[s0];
    in[i].prev_erase_max = c->bucket_erase_max[s0];
  }
  void* d_in = nullptr;
  int rc = ring_push(c, in.data(), in.size() * sizeof(BucketIn), st, &d_in);
  if (rc) return rc;
  const int8_t* forced = nullptr;
  if (preserve) {
    // slot of every row from its key's cosine with the block's mean key instead of from its value norm
    const size_t need_f = anticorr_scratch_floats(n_sl, n, f.head_dim), need_c = (size_t)n_sl * n;
    if (need_f > c->acr_floats || need_c > c->acr_rows) {
      BKV_CUDA(cudaStreamSynchronize(st));
      if (c->acr_scratch) cudaFree(c->acr_scratch);
      if (c->acr_cls) cudaFree(c->acr_cls);
      c->acr_scratch = nullptr; c->acr_cls = nullptr;
      c->acr_floats = std::max(c->acr_floats, need_f);
      c->acr_rows = std::max(c->acr_rows, need_c);
      BKV_CUDA(cudaMalloc(reinterpret_cast<void**>(&c->acr_scratch), sizeof(float) * c->acr_floats));
      BKV_CUDA(cudaMalloc(reinterpret_cast<void**>(&c->acr_cls), c->acr_rows));
    }
    ProfScope ps(c, 0, st);
    BKV_CUDA(launch_anticorr_classes(c->G, K, n_sl, n, tau, c->acr_scratch, c->acr_cls, st));
    c->kernels_launched += 3;
    forced = c->acr_cls;
  }
  {
    ProfScope ps(c, 0, st);
    BKV_CUDA(launch_bucket_route(c->G, V, n_sl, n, n_buckets, i_top, rho * rho, static_cast<const BucketIn*>(d_in),
                                 c->bkt_vmax_bits, c->bkt_ns, c->bkt_slot, c->bkt_rank, c->bkt_chunk_cnt, c->bkt_out, forced, st));
  }
  c->kernels_launched += 3;
  BKV_CUDA(cudaMemcpyAsync(c->bkt_out_host, c->bkt_out, sizeof(BucketOut) * n_sl, cudaMemcpyDeviceToHost, st));
  BKV_CUDA(cudaStreamSynchronize(st));   // the counts decide the host bookkeeping of every instance
  const BucketOut* out = c->bkt_out_host;
  const int T = Lo.T;
  const int max_pending = T == 0 ? f.max_tokens : (f.max_pending > 0 ? std::min(f.max_pending, f.max_tokens) : f.max_tokens);
  for (int i = 0; i < n_sl; ++i) {
    if (out[i].above > 0) return BALANCEKV_E_INVAL;        // a value norm above 2^i_top: nothing was appended
    for (int b = 0; b < n_buckets; ++b) {
      const StreamState& S = c->st[stream_id(c, heads[i].first, layer0 + b, heads[i].second)];
      const int m = out[i].count[b];
      if (S.appended + m > f.max_tokens || S.pending + m > max_pending) return BALANCEKV_E_NOMEM;
      if ((int64_t)S.start0 + S.len0 + m > Lo.cap0) return BALANCEKV_E_NOMEM;
    }
  }
  std::vector<BucketDst> dst((size_t)n_sl * n_buckets);
  for (int i = 0; i < n_sl; ++i) {
    const int s0 = stream_id(c, heads[i].first, layer0, heads[i].second);
    c->bucket_vmax2[s0] = out[i].vmax2;
    c->bucket_erase_max[s0] = out[i].erase_max;
    c->bucket_dropped += out[i].dropped;
    for (int b = 0; b < n_buckets; ++b) {
      const int s = stream_id(c, heads[i].first, layer0 + b, heads[i].second);
      StreamState& S = c->st[s];
      BucketDst& D = dst[(size_t)i * n_buckets + b];
      D.pad = 0;
      if (i_top - b <= out[i].erase_max) {
        // "erase all MR-Numerator_i with 2^i <= rho * v_max": the instance forgets its sets
        if (S.appended > 0) {
          c->bucket_dropped += S.appended;
          S = StreamState();
          BKV_CUDA(cudaMemsetAsync(c->A.seg + (size_t)s * (T + 1), 0, sizeof(Seg) * (T + 1), st));
        }
        D.dst_row = 0; D.idx0 = 0; D.stream = -1; D.new_len = 0;
        continue;
      }
      const int m = out[i].count[b];
      D.dst_row = (int64_t)s * Lo.R + Lo.region_off[0] + S.start0 + S.len0;
      D.idx0 = (int32_t)S.appended;
      D.stream = m > 0 ? s : -1;
      S.len0 += m; S.appended += m; S.pending += m;
      D.new_len = S.len0;
      c->tokens_appended += m;
    }
  }
  void* d_dst = nullptr;
  rc = ring_push(c, dst.data(), dst.size() * sizeof(BucketDst), st, &d_dst);
  if (rc) return rc;
  {
    ProfScope ps(c, 0, st);
    BKV_CUDA(launch_bucket_scatter(c->G, c->A, K, V, n_sl, n, n_buckets, c->bkt_slot, c->bkt_rank, c->bkt_chunk_cnt,
                                   c->bkt_ns, static_cast<const BucketDst*>(d_dst), st));
  }
  c->kernels_launched++;
  if (token_slot)
    BKV_CUDA(cudaMemcpyAsync(token_slot, c->bkt_slot, (size_t)n_sl * n, cudaMemcpyDeviceToDevice, st));
  if (counts_host)
    for (int i = 0; i < n_sl; ++i) {
      int32_t* row = counts_host + (size_t)i * (n_buckets + 1);
      for (int b = 0; b < n_buckets; ++b) row[b] = out[i].count[b];
      row[n_buckets] = out[i].dropped;
    }
  return BALANCEKV_OK;
}

int balancekv_stream_append_bucketed(balancekv_ctx* c, int seq, int layer0, int n_buckets, int i_top, int kv_head,
                                     const void* K_blk, const void* V_blk, int n_tokens, float erase_ratio,
                                     int8_t* token_slot, int32_t* counts_host, void* stream) {
  if (!c || seq < 0 || seq >= c->cfg.n_seqs || kv_head < 0 || kv_head >= c->cfg.n_kv_heads) return BALANCEKV_E_INVAL;
  std::vector<std::pair<int, int>> heads{{seq, kv_head}};
  return append_bucketed_impl(c, heads, layer0, n_buckets, i_top, K_blk, V_blk, n_tokens, erase_ratio, token_slot,
                              counts_host, static_cast<cudaStream_t>(stream));
}

int balancekv_stream_append_layer_bucketed(balancekv_ctx* c, int layer0, int n_buckets, int i_top, const void* K,
                                           const void* V, int n_tokens, float erase_ratio, int8_t* token_slot,
                                           int32_t* counts_host, void* stream) {
  if (!c) return BALANCEKV_E_INVAL;
  std::vector<std::pair<int, int>> heads;
  for (int s = 0; s < c->cfg.n_seqs; ++s)
    for (int h = 0; h < c->cfg.n_kv_heads; ++h) heads.push_back({s, h});
  return append_bucketed_impl(c, heads, layer0, n_buckets, i_top, K, V, n_tokens, erase_ratio, token_slot, counts_host,
                              static_cast<cudaStream_t>(stream));
}

int balancekv_stream_append_layer_preserving(balancekv_ctx* c, int layer0, const void* K, const void* V, int n_tokens,
                                             float tau, int8_t* token_slot, int32_t* counts_host, void* stream) {
  if (!c || !(tau >= -1.f) || tau > 1.f) return BALANCEKV_E_INVAL;
  std::vector<std::pair<int, int>> heads;
  for (int s = 0; s < c->cfg.n_seqs; ++s)
    for (int h = 0; h < c->cfg.n_kv_heads; ++h) heads.push_back({s, h});
  return append_bucketed_impl(c, heads, layer0, 2, 0, K, V, n_tokens, 0.f, token_slot, counts_host,
                              static_cast<cudaStream_t>(stream), true, tau);
}

int balancekv_reset(balancekv_ctx* c, void* stream) {
  if (!c) return BALANCEKV_E_INVAL;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  c->decode_chain = false;
  for (StreamState& S : c->st) S = StreamState();
  c->bucket_vmax2.clear();
  c->bucket_erase_max.clear();
  BKV_CUDA(cudaMemsetAsync(c->A.seg, 0, sizeof(Seg) * (size_t)c->n_streams * (c->cfg.levels + 1), st));
  // a context that gave up on a device-side wait becomes usable again
  BKV_CUDA(cudaMemsetAsync(c->d_status, 0, sizeof(int), st));
  *c->h_status = 0;
  // a launch that gave up may have left partial rows behind
  BKV_CUDA(init_decode_scratch(c->d_decode_scratch, decode_scratch_bytes(c->G, c->max_splits), (size_t)c->G.B * c->G.H, st));
  if (c->two_scratch)
    for (int z = 0; z < BALANCEKV_MAX_MERGE; ++z)
      BKV_CUDA(init_decode_scratch(c->two_scratch + c->two_scratch_words * z, c->two_scratch_words * 4, (size_t)c->G.B * c->G.H, st));
  return BALANCEKV_OK;
}

int balancekv_profile_enable(balancekv_ctx* c, int on) {
  if (!c) return BALANCEKV_E_INVAL;
  if (on && c->prof_ev.empty()) {
    c->prof_ev.resize(2 * kProfMax);
    c->prof_class.resize(kProfMax);
    for (cudaEvent_t& e : c->prof_ev) BKV_CUDA(cudaEventCreate(&e));
  }
  c->profiling = on == 1 ? ~0u : static_cast<unsigned>(on) >> 1;   // bit `class` set: time that class
  return BALANCEKV_OK;
}

int balancekv_profile_sample(balancekv_ctx* c, int cls, int every) {
  if (!c || cls < 0 || cls >= BALANCEKV_PROFILE_CLASSES || every < 1) return BALANCEKV_E_INVAL;
  c->prof_every[cls] = every;
  c->prof_seen[cls] = 0;
  return BALANCEKV_OK;
}

int balancekv_profile_read(balancekv_ctx* c, double* out) {
  if (!c || !out) return BALANCEKV_E_INVAL;
  BKV_CUDA(cudaDeviceSynchronize());
  for (int i = 0; i < 2 * BALANCEKV_PROFILE_CLASSES; ++i) out[i] = 0.0;
  for (size_t i = 0; i < c->prof_used; ++i) {
    float ms = 0.f;
    BKV_CUDA(cudaEventElapsedTime(&ms, c->prof_ev[2 * i], c->prof_ev[2 * i + 1]));
    out[2 * c->prof_class[i]] += 1.0;
    out[2 * c->prof_class[i] + 1] += ms;
  }
  c->prof_used = 0;
  return BALANCEKV_OK;
}

int balancekv_stats(balancekv_ctx* c, balancekv_stats_t* out) {
  if (!c || !out) return BALANCEKV_E_INVAL;
  BKV_CUDA(cudaDeviceSynchronize());
  unsigned long long fails = 0;
  int status = 0;
  BKV_CUDA(cudaMemcpy(&fails, c->d_fail, sizeof(fails), cudaMemcpyDeviceToHost));
  BKV_CUDA(cudaMemcpy(&status, c->d_status, sizeof(status), cudaMemcpyDeviceToHost));
  int64_t stored = 0;
  for (const StreamState& S : c->st) {
    stored += S.len0;
    for (int l = 1; l <= c->cfg.levels; ++l) stored += S.lvl_len[l];
  }
  out->tokens_appended = c->tokens_appended;
  out->tokens_stored = stored;
  out->calls_run = c->calls_run;
  out->walk_fails = (int64_t)fails;
  out->device_status = status;
  out->bytes_resident = (int64_t)c->bytes_resident;
  out->kernels_launched = c->kernels_launched;
  out->walk_kernel = c->cfg.levels == 0 ? 0 : (c->use_tc ? 2 : 1);
  out->decode_kernel = c->decode_maps ? 2 : 1;
  if (c->h_status) *c->h_status = status;
  return status == kStatusWaitTimeout ? BALANCEKV_E_TIMEOUT : BALANCEKV_OK;
}

int balancekv_debug_set_status(balancekv_ctx* c, int value) {
  if (!c) return BALANCEKV_E_INVAL;
  BKV_CUDA(cudaDeviceSynchronize());
  BKV_CUDA(cudaMemcpy(c->d_status, &value, sizeof(int), cudaMemcpyHostToDevice));
  *c->h_status = value;
  return BALANCEKV_OK;
}

int balancekv_debug_scratch_used(balancekv_ctx* c, int64_t* words) {
  if (!c || !words) return BALANCEKV_E_INVAL;
  *words = 0;
  if (!c->decode_maps) return BALANCEKV_OK;          // the CUDA-core kernel keeps no state in its partial rows
  BKV_CUDA(cudaDeviceSynchronize());
  const size_t n_sl = (size_t)c->G.B * c->G.H;
  const size_t ticket_words = ((n_sl + 63) / 64) * 64;
  auto count = [&](const float* block, size_t bytes) -> int {
    std::vector<uint32_t> host(bytes / 4);
    if (cudaMemcpy(host.data(), block, host.size() * 4, cudaMemcpyDeviceToHost) != cudaSuccess) return BALANCEKV_E_CUDA;
    for (size_t i = ticket_words; i < host.size(); ++i) *words += host[i] != 0xffffffffu;
    return BALANCEKV_OK;
  };
  int rc = count(c->d_decode_scratch, decode_scratch_bytes(c->G, c->max_splits));
  if (rc == BALANCEKV_OK && c->two_scratch)
    for (int z = 0; z < BALANCEKV_MAX_MERGE && rc == BALANCEKV_OK; ++z)
      rc = count(c->two_scratch + c->two_scratch_words * z, c->two_scratch_words * 4);
  return rc;
}

int balancekv_plan_calls(int block, int levels, int recent_window, const int32_t* appended_after_event, int n_events,
                         int32_t* calls_out, int max_calls) {
  if (block < 2 || block % 2 || levels < 0 || levels > kMaxLevels || recent_window < 0 || !appended_after_event ||
      n_events < 0 || (!calls_out && max_calls > 0))
    return BALANCEKV_E_INVAL;
  Layout Lo;
  Lo.t = block; Lo.T = levels; Lo.W = recent_window;
  Lo.R = (int64_t)1 << 40;
  for (int l = 0; l <= levels; ++l) Lo.region_off[l] = l * (1 << 20);
  Lo.pool_row[0] = (int64_t)1 << 41; Lo.pool_row[1] = (int64_t)1 << 42;
  Lo.pool_pairs = (int64_t)1 << 30;
  StreamState S;
  int n_out = 0;
  Plan P;
  for (int e = 0; e < n_events; ++e) {
    if (appended_after_event[e] < S.appended) return BALANCEKV_E_INVAL;
    S.len0 += (int32_t)(appended_after_event[e] - S.appended);
    S.appended = appended_after_event[e];
    if (levels == 0) continue;
    const int64_t nb = ready_blocks(Lo, S);
    if (nb <= 0) continue;
    std::vector<std::pair<int, int>> runs{{0, (int)nb}};
    if (!plan_batch(Lo, &S, runs, P)) return BALANCEKV_E_STATE;
    // sequential order of Algorithm 3: block by block, climbing levels after each block
    std::vector<size_t> next(levels, 0);
    const int64_t first_block = S.calls_done[0] - nb;
    for (int64_t b = 0; b < nb; ++b) {
      int64_t beta = first_block + b + 1;
      for (int l = 0; l < levels; ++l) {
        if (next[l] >= P.levels[l].size()) break;
        const CallDesc& d = P.levels[l][next[l]++];
        if (n_out < max_calls) {
          calls_out[3 * n_out] = e; calls_out[3 * n_out + 1] = l; calls_out[3 * n_out + 2] = d.ordinal;
        }
        ++n_out;
        if (beta % 2) break;
        beta /= 2;
      }
    }
  }
  return n_out;
}

}  // extern "C"
