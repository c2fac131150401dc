/*
 * balancekv.h -- C ABI of the BalanceKV hot path on NVIDIA B200 (sm_100a).
 *
 * BalanceKV ("Streaming Attention Approximation via Discrepancy Theory") compresses the
 * key/value cache of every (sequence, layer, KV head) stream: batches of t tokens are
 * halved by SoftmaxBalance (Algorithm 2: a self-balancing walk over the pairwise kernel
 * exp(<k_i,k_j>/sqrt d) <v_i,v_j>), survivors double their weight and climb the
 * MergeAndReduce tree (Algorithm 3) up to level T, and decode attention is the ratio of
 * Algorithm 1's output step evaluated over the weighted sets C^0..C^T (Theorem 3.3's
 * estimator) -- here over one shared set for numerator and denominator.
 *
 * Conventions
 *   - Every call returns 0 (BALANCEKV_OK) or a negative error code; nothing throws.
 *   - Unless a parameter says "host", tensor pointers are DEVICE pointers owned by the
 *     caller, row-major and contiguous.  The library copies what it keeps and never
 *     frees or retains caller memory.
 *   - Work is enqueued asynchronously on the CUDA stream passed as `stream`
 *     (a cudaStream_t cast to void*; NULL = the default stream).  A context must be used
 *     from one host thread at a time, on the device that was current at create time.
 *   - dtype: 0 = float32, 1 = bfloat16 (keys, values, queries and outputs alike).
 *   - A "stream" below is one (sequence, layer, KV head) token stream of the paper's
 *     streaming formulation (Section 2.1); `stream` (void*) is the CUDA stream.
 *   - There is no CPU fallback: without a CUDA device every device call fails with
 *     BALANCEKV_E_CUDA.
 */
#ifndef BALANCEKV_H_
#define BALANCEKV_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define BALANCEKV_OK 0
#define BALANCEKV_E_INVAL (-1)   /* bad argument, shape, dtype or state                 */
#define BALANCEKV_E_NOMEM (-2)   /* a stream's capacity (or device memory) is exhausted */
#define BALANCEKV_E_STATE (-3)   /* call not valid in the context's current state       */
#define BALANCEKV_E_CUDA (-4)    /* a CUDA runtime call failed                          */
#define BALANCEKV_E_TIMEOUT (-5) /* a bounded device-side wait gave up                  */

typedef struct balancekv_ctx balancekv_ctx;

/* Parameters of Algorithms 1-3 (r, t, T, delta) plus the shape of the model. */
typedef struct balancekv_config {
  int32_t n_seqs;        /* B: sequences                                                      */
  int32_t n_layers;      /* L                                                                 */
  int32_t n_kv_heads;    /* H                                                                 */
  int32_t n_q_heads;     /* H*g, g = query heads per KV head (1..8)                           */
  int32_t head_dim;      /* d: 64 or 128                                                      */
  int32_t dtype;         /* 0 = float32, 1 = bfloat16                                         */
  int32_t block;         /* t: batch size of Algorithm 3 = tokens per SoftmaxBalance call;
                            multiple of 64                                                    */
  int32_t levels;        /* T >= 0: compression rate 2^-T; 0 keeps every token                */
  int32_t max_tokens;    /* N: most tokens a stream will ever receive; also delta's default   */
  int32_t max_pending;   /* most tokens appended to a stream between two compress calls;
                            <= 0 means N (always safe)                                        */
  int32_t recent_window; /* W >= 0: the newest W tokens of a stream never enter a call        */
  int32_t center_keys;   /* 1: subtract the call's mean key inside the kernel only
                            (the stored keys are untouched); 0 (default): off                 */
  int32_t gram_path;     /* 0 = automatic, 1 = CUDA-core (fp32 FMA) kernels for the walk and for
                            decode, 2 = tensor-core (tcgen05) walk kernel; 2 needs bf16,
                            d = 128, t multiple of 128                                         */
  int32_t decode_splits; /* > 0: split-K factor of decode attention (1..64); 0 = automatic         */
  uint64_t seed;         /* Philox key; sequence s uses seed + s                              */
  float delta;           /* failure probability of Algorithm 2; <= 0 means 1/N^2              */
  float c_override;      /* > 0: use this c instead of 30 ln(t/delta)                         */
  float r_key, r_value;  /* > 0: fixed radii of Algorithm 2; <= 0: per-call maxima            */
} balancekv_config;

typedef struct balancekv_stats_t {
  int64_t tokens_appended;    /* over all streams                                             */
  int64_t tokens_stored;      /* rows currently held (all levels, all streams)                */
  int64_t calls_run;          /* SoftmaxBalance calls executed                                */
  int64_t walk_fails;         /* times |y^T eta| exceeded c R^2 (counted, clamped, no error)  */
  int64_t device_status;      /* 0, or the first device-side error code                       */
  int64_t bytes_resident;     /* device memory owned by the context                           */
  int64_t kernels_launched;   /* kernels of this library launched so far                      */
  int64_t walk_kernel;        /* Algorithm 2's kernel: 0 none (T = 0), 1 CUDA cores (fp32 FMA),
                                 2 tensor cores (tcgen05); fixed at create time by the shape    */
  int64_t decode_kernel;      /* decode attention: 1 CUDA cores, 2 tensor cores (mma + TMA)    */
} balancekv_stats_t;

/* Allocate a context: all cache memory for n_seqs*n_layers*n_kv_heads streams.
 * E_INVAL on a bad field, E_NOMEM / E_CUDA if the device allocation fails.  The kernels that
 * serve the context follow from its shape (balancekv_stats reports them); if the tensor-core
 * kernels of a shape that has them cannot be prepared, the call fails with E_CUDA -- there is no
 * quiet change to other kernels.
 *
 * Device-side waits are bounded (about 50 ms).  One that gives up sets the context's status word:
 * balancekv_stats then returns BALANCEKV_E_TIMEOUT (after filling the record), and so does every
 * later call that would enqueue work once the host has seen the word (it is copied back behind
 * every compress batch); results computed after that point are not valid.  balancekv_reset clears
 * the condition. */
int balancekv_create(const balancekv_config* cfg, balancekv_ctx** out);
int balancekv_destroy(balancekv_ctx* ctx);

/* Algorithm 3, "C^0 <- C^0 + {k_j, v_j}": append n_tokens rows to one stream.
 * K_blk, V_blk: [n_tokens, head_dim].  No compression work happens here.
 * E_NOMEM if the stream would exceed max_tokens or its pending capacity. */
int balancekv_stream_append(balancekv_ctx* ctx, int seq, int layer, int kv_head, const void* K_blk,
                            const void* V_blk, int n_tokens, void* stream);

/* Same for every stream of one layer at once.
 * K, V: [n_seqs, n_kv_heads, n_tokens, head_dim]. */
int balancekv_stream_append_layer(balancekv_ctx* ctx, int layer, const void* K, const void* V,
                                  int n_tokens, void* stream);

/* As above with HOST buffers (pinned memory recommended): the copy to the device is
 * enqueued on `stream` through a staging buffer owned by the context, which the next
 * *_host call reuses (such calls must all be issued on the same CUDA stream). */
int balancekv_stream_append_layer_host(balancekv_ctx* ctx, int layer, const void* K_host,
                                       const void* V_host, int n_tokens, void* stream);

/* Algorithm 3's update step for every stream: run every SoftmaxBalance call that is ready
 * (a full batch of t eligible tokens in C^0, or two halves in C^i, i < T), level by level,
 * including the strict-half selection of the paper's implementation note (Appendix B).
 * T must equal config.levels (E_INVAL otherwise); T = 0 is a no-op. */
int balancekv_compress(balancekv_ctx* ctx, int T, void* stream);
/* Same, restricted to the streams of one layer. */
int balancekv_compress_layer(balancekv_ctx* ctx, int layer, int T, void* stream);

/* Algorithm 1's output ratio / Theorem 3.3's estimator for one layer:
 * out[s,h,:] = sum_i w_i e^{<k_i,q>/sqrt d} v_i / sum_i w_i e^{<k_i,q>/sqrt d} over every
 * stored token of the stream of (s, h / g), w_i = 2^level.  q, out: [n_seqs, n_q_heads,
 * head_dim] in the context's dtype.  With T = 0 this is Eq. (1) exactly. */
int balancekv_decode_attn(balancekv_ctx* ctx, int layer, const void* q, void* out, void* stream);

/* One step of the streaming problem of Section 2.1: the triple (q_j, k_j, v_j) of every
 * stream of a layer arrives, k_j, v_j join C^0 (Algorithm 3; decode-phase tokens stay
 * uncompressed until a later compress), and z_j is returned.  k_new, v_new: [n_seqs,
 * n_kv_heads, head_dim]; q, out as in balancekv_decode_attn.  Equivalent to
 * balancekv_stream_append_layer(.., 1) followed by balancekv_decode_attn. */
int balancekv_stream_step(balancekv_ctx* ctx, int layer, const void* q, const void* k_new, const void* v_new,
                          void* out, void* stream);
/* Same with HOST buffers for q, k_new, v_new and out.  The inputs are read by the CPU during
 * the call (packed into a pinned staging slot of the context and sent as one transfer on a copy
 * stream of the context, so that the transfer of a step overlaps the previous step's kernel), and the
 * caller may reuse them as soon as the call returns.  The fused step kernel is not tied to that
 * transfer by an event: an arrival word is written behind the operands on the copy stream and the
 * kernel waits for it (bounded like every device-side wait); where the step takes more than one
 * launch the launches wait for the transfer through an event.  out_host is written in stream order
 * (synchronise the stream before reading it): a pinned out_host is written by the kernel itself,
 * pageable memory through a device buffer and a copy.  The first call allocates the staging buffers. */
int balancekv_stream_step_host(balancekv_ctx* ctx, int layer, const void* q_host, const void* k_host,
                               const void* v_host, void* out_host, void* stream);

/* As above with HOST q and out: q is copied in, out copied back, both on `stream`;
 * the call returns without synchronising (synchronise the stream before reading out). */
int balancekv_decode_attn_host(balancekv_ctx* ctx, int layer, const void* q_host, void* out_host,
                               void* stream);

/* Decode attention for callers that must not allocate (the paper has no counterpart: this
 * is a deployment variant of balancekv_decode_attn, not a step of the method).
 *
 * Who needs it: code that runs where device allocation is off limits -- a serving loop that
 * cannot afford cudaMalloc's device-wide synchronisation, a plugin that only ever receives
 * buffers from its host framework, a process whose memory pool is fully committed.  Such a
 * caller cannot create a context (that allocates the cache), so it keeps the cache rows
 * itself and passes them in:
 *   K, V : [n_streams, cache_len, head_dim]   q, out : [n_streams, group, head_dim]
 * (device pointers, 16-byte aligned, dtype 0 = float32 / 1 = bfloat16).  In every stream the
 * first n_heavy rows carry weight 2^level and the remaining rows weight 1; out is
 * sum_i w_i e^{<k_i,q>/sqrt d} v_i / sum_i w_i e^{<k_i,q>/sqrt d}, the same arithmetic as
 * balancekv_decode_attn.
 *
 * The split-K scratch is a fixed 8 MiB array inside the library image (held by every GPU
 * that loads the library, until the process exits); the call performs no cudaMalloc, cudaFree
 * or other allocating call.  A problem whose scratch (256 bytes, a segment table of
 * n_streams * (level+1) * 8 bytes, n_streams ticket words rounded up to 64, and n_streams *
 * splits * group * (head_dim+8) * 4 bytes of partial rows, splits <= 64 chosen from the SM
 * count) exceeds the array is rejected with BALANCEKV_E_NOMEM and a message on stderr.  The
 * first call on a device -- of this function or of balancekv_decode_attn_static_status,
 * whichever host thread gets there first -- looks up the array's device address
 * (cudaGetSymbolAddress) and clears its status word with a synchronous memset; make that first
 * call outside any stream capture.  All calls share the array: the part a call uses is
 * re-initialised by the call itself, but two calls that overlap on the GPU (different CUDA
 * streams) race on it -- issue them on one stream. */
int balancekv_decode_attn_static(const void* K, const void* V, int n_streams, int cache_len, int n_heavy,
                                 int level, const void* q, void* out, int group, int head_dim, int dtype,
                                 void* stream);
/* The entry point above returns before its kernel has run, so a bounded device-side wait that
 * gives up cannot show in its return value; it sets a status word in the built-in array
 * instead, which this call copies to *status_host (0 = fine, 1 = a wait gave up since the last
 * read; the outputs of that launch are then not valid) and clears.  Allocates nothing;
 * synchronises `stream`.  The paper has no counterpart. */
int balancekv_decode_attn_static_status(int* status_host, void* stream);

/* Load an already-compressed set into level `level` of every stream of one layer
 * (weight 2^level, the weights of Theorem 3.3's estimator): K, V: [n_seqs, n_kv_heads,
 * n_tokens, head_dim]; orig_idx (may be NULL): [n_seqs, n_kv_heads, n_tokens] original
 * token positions.  level is 0 or T (else BALANCEKV_E_INVAL): the levels between hold exactly 0
 * or t/2 rows by construction and are only ever filled by balancekv_compress. */
int balancekv_cache_load_level(balancekv_ctx* ctx, int layer, int level, const void* K, const void* V,
                               const int32_t* orig_idx, int n_tokens, void* stream);

/* Inspection.  Gathers the stream's weighted set in the order C^T, ..., C^1, C^0
 * (ascending original position) into buffers owned by the context and returns DEVICE
 * pointers to them, valid until the next call on the context.  Synchronises the device.
 * Any output pointer may be NULL. */
int balancekv_cache_view(balancekv_ctx* ctx, int seq, int layer, int kv_head, const void** K,
                         const void** V, const float** w, const int32_t** orig_idx, int* len);

/* Host-side bookkeeping of one stream: sizes_host[0..T] = |C^0| .. |C^T| (Algorithm 3). */
int balancekv_level_sizes(balancekv_ctx* ctx, int seq, int layer, int kv_head, int32_t* sizes_host);

/* Record, for every later call, the signs eta, the running correlation
 * S_j = y^T eta / R^2 and the probability p_j of Algorithm 2.  Allocates the record
 * buffers; must be enabled before the first compress. */
int balancekv_debug_enable(balancekv_ctx* ctx, int on);
/* DEVICE pointers to the record of call (level, ordinal) of a stream, each [t]. */
int balancekv_debug_call(balancekv_ctx* ctx, int seq, int layer, int kv_head, int level,
                         int call_ordinal, const int8_t** eta, const float** S, const float** p,
                         int* m);

/* Forget every token of every stream (Algorithm 3's "initialize C^i to empty"); memory,
 * configuration and debug buffers are kept.  Enqueued on `stream`. */
int balancekv_reset(balancekv_ctx* ctx, void* stream);

/* Algorithm 1 with its separate denominator instance (MR-Denominator), without the value-norm
 * buckets.  The caller dedicates two layer slots of the context to one model layer: slot
 * `layer_num` receives (k_j, v_j) through the ordinary append calls, slot `layer_den` receives
 * (k_j, 1) through balancekv_stream_append_layer_keys (K: [n_seqs, n_kv_heads, n_tokens, head_dim]
 * device; the library supplies the unit value (1, 0, ..., 0), for which the pairwise kernel of
 * Algorithm 2 becomes exp(<k_i, k_j>/sqrt d)).  balancekv_compress then runs MergeAndReduce on
 * both, with independent coins (the coin's counter holds the slot index), and
 *   balancekv_decode_attn_two:  out = sum_l 2^l sum_{V^l} e^{<k,q>/sqrt d} v
 *                                   / sum_l 2^l sum_{K^l} e^{<k,q>/sqrt d}
 * (Algorithm 1's output ratio), V^l the sets of slot layer_num and K^l those of slot layer_den.
 * bf16, head_dim 128, group <= 8 only (else BALANCEKV_E_INVAL); q, out as balancekv_decode_attn.
 * The first call of either function allocates its buffers. */
int balancekv_stream_append_layer_keys(balancekv_ctx* ctx, int layer, const void* K, int n_tokens, void* stream);
int balancekv_decode_attn_two(balancekv_ctx* ctx, int layer_num, int layer_den, const void* q, void* out,
                              void* stream);

/* Decode over several layer slots at once:
 *   out = sum over the slots of layers_num of  sum_i w_i e^{<k_i,q>/sqrt d} v_i
 *       / sum over the slots of layers_den of  sum_i w_i e^{<k_i,q>/sqrt d}.
 * With the same slots on both sides this is the estimator of Theorem 3.3 over the union of their
 * caches -- e.g. the paper's single-layer experiments (Appendix B), which keep the first 256 tokens
 * exactly: one slot holds them and is never compressed (balancekv_compress_layer leaves the other
 * slots alone), a second slot runs BalanceKV on the rest with a recent window.  With different
 * slots it is Algorithm 1's output ratio (numerator instances above, e.g. one per value-norm bucket
 * that the caller routes tokens to; the denominator instance below).  At most
 * BALANCEKV_MAX_MERGE distinct slots, none twice on a side; bf16, head_dim 128, group <= 8 only
 * (else BALANCEKV_E_INVAL).  layers_* are host arrays.  The first call allocates its buffers. */
#define BALANCEKV_MAX_MERGE 8
int balancekv_decode_attn_merged(balancekv_ctx* ctx, const int32_t* layers_num, int n_num, const int32_t* layers_den,
                                 int n_den, const void* q, void* out, void* stream);

/* Algorithm 1's bucketing of the stream by value norm and its erasure of small-norm buckets.
 * Token j belongs to the bucket index i with 2^(i-1) < ||v_j||_2 <= 2^i (a norm that is an exact
 * power of two satisfies Algorithm 1's printed condition for two indices; the smaller is taken).
 * The caller dedicates n_buckets (1..8) consecutive layer slots to one model layer: slot
 * layer0 + b is the instance MR-Numerator_i of bucket i = i_top - b, so i_top >= log2 of the
 * largest value norm that will ever arrive.  The call routes every row of the block to its
 * instance (appended to that instance's C^0 in stream order, exactly as balancekv_stream_append
 * would; the stored original position is the position inside the instance's own stream),
 * updates the running maximum v_max of the value norms, and erases (empties, for good) every
 * instance with 2^i <= erase_ratio * v_max -- Algorithm 1 prints the factor
 * eps/(2n) e^{-r^2/sqrt d}, the proof of Theorem 1.1 uses eps/sqrt n; pass either, or 0 for no
 * erasure.  Rows that are dropped instead of stored: zero values, rows of an erased bucket, rows
 * below the lowest slot's bucket.  balancekv_compress then runs MergeAndReduce on every
 * instance with independent coins, and balancekv_decode_attn_merged over the slots (numerator)
 * and a balancekv_stream_append_layer_keys slot (denominator) is Algorithm 1's output ratio.
 *   K, V        [n_tokens, head_dim] of one stream (balancekv_stream_append_bucketed) or
 *               [n_seqs, n_kv_heads, n_tokens, head_dim] (.._layer_bucketed); device, 16-byte aligned
 *   token_slot  device, may be NULL: int8 per row in the layout of K without head_dim, the slot
 *               offset b the row went to, -1 if it was dropped
 *   counts_host host, may be NULL: per stream n_buckets + 1 numbers, the rows sent to each slot
 *               and the rows dropped
 * Norms are compared as fp32 squared norms.  The call SYNCHRONISES `stream` once (the per-bucket
 * counts drive the host bookkeeping of Algorithm 3) and may allocate routing buffers when a block
 * is larger than any before.  Errors: BALANCEKV_E_INVAL for bad arguments or a value norm above
 * 2^i_top (nothing is appended then), BALANCEKV_E_NOMEM when an instance would overflow. */
int balancekv_stream_append_bucketed(balancekv_ctx* ctx, int seq, int layer0, int n_buckets, int i_top, int kv_head,
                                     const void* K_blk, const void* V_blk, int n_tokens, float erase_ratio,
                                     int8_t* token_slot, int32_t* counts_host, void* stream);
int balancekv_stream_append_layer_bucketed(balancekv_ctx* ctx, int layer0, int n_buckets, int i_top, const void* K,
                                           const void* V, int n_tokens, float erase_ratio, int8_t* token_slot,
                                           int32_t* counts_host, void* stream);

/* The augmented BalanceKV of Section 4.3: tokens whose keys are strongly anti-correlated with the
 * rest are preserved exactly, the standard procedure runs on the others.  The paper gives neither
 * the measure nor a threshold; here token j of the appended block is preserved when the cosine
 * between its key and the block's mean key (per stream) is at most tau,
 *   <k_j, kbar> <= tau ||k_j|| ||kbar||,   -1 <= tau <= 1 (tau = -1 preserves nothing but exact
 * opposites; a zero key or mean counts as cosine 0),
 * compared in fp32.  The caller dedicates two consecutive layer slots to one model layer: slot
 * layer0 receives the preserved rows and is never compressed (use balancekv_compress_layer on slot
 * layer0 + 1 only), slot layer0 + 1 receives the rest in stream order and is an ordinary BalanceKV
 * stream.  balancekv_decode_attn_merged over both slots on both sides is the estimator of
 * Theorem 3.3 over the union: preserved tokens weigh 1, so the weights still sum to the tokens seen.
 * K, V: [n_seqs, n_kv_heads, n_tokens, head_dim] device; token_slot (device, may be NULL): int8 per
 * row, 0 = preserved, 1 = the rest; counts_host (host, may be NULL): per stream {preserved, rest,
 * dropped = 0}.  The stored original position of a row is its position in its slot's own stream.
 * Synchronises `stream` once, like the bucketed append.  Errors as for the bucketed append. */
int balancekv_stream_append_layer_preserving(balancekv_ctx* ctx, int layer0, const void* K, const void* V, int n_tokens,
                                             float tau, int8_t* token_slot, int32_t* counts_host, void* stream);

/* Kernel timing for roofline reports.  While enabled, every launch of the kernel classes
 * below is bracketed by CUDA events on its launch stream (at most 8192 launches between two
 * reads; later ones are not recorded).  balancekv_profile_read synchronises the device and
 * writes, per class, {launches, total milliseconds} into out_host[2*class + {0,1}], then
 * clears the record.  Classes: 0 append/load, 1 radii (inputs of Algorithm 2), 2 Gram tiles +
 * sign walk (Algorithm 2), 3 strict-half selection + compaction, 4 decode attention
 * (Algorithm 1's output ratio), 5 bookkeeping (remainder move, segment table).
 * `on`: 0 = off, 1 = every class, any other value = a mask with bit (1 + class) set for each
 * class to time.  balancekv_profile_sample makes the record of one class sparse: only every
 * `every`-th launch of it (counted from the call) is timed, which keeps the events out of the
 * way of a loop of microsecond-sized launches; read then reports the timed launches only. */
#define BALANCEKV_PROFILE_CLASSES 6
int balancekv_profile_enable(balancekv_ctx* ctx, int on);
int balancekv_profile_sample(balancekv_ctx* ctx, int kernel_class, int every);
int balancekv_profile_read(balancekv_ctx* ctx, double* out_host);

/* Testing aid: overwrite the context's device status word (0 = clear, 1 = a wait gave up), as a
 * kernel whose bounded wait ran out would.  Synchronises the device. */
int balancekv_debug_set_status(balancekv_ctx* ctx, int value);

/* Testing aid: the number of 4-byte words of the split-K decode scratch that do not hold the
 * "empty" pattern (Algorithm 1's output ratio is summed over splits through that scratch; the
 * tensor-core decode kernel uses each word as its own arrival flag and must leave every word
 * empty behind every launch).  0 for contexts on the CUDA-core decode kernel.  Synchronises the
 * device.  words: host pointer. */
int balancekv_debug_scratch_used(balancekv_ctx* ctx, int64_t* words);

/* Synchronises the device.  Returns BALANCEKV_E_TIMEOUT (record filled) if a device-side wait gave up. */
int balancekv_stats(balancekv_ctx* ctx, balancekv_stats_t* out);
const char* balancekv_strerror(int code);

/* Pure host bookkeeping of Algorithm 3 (no device needed): a stream holds
 * appended_after_event[e] tokens after its e-th append, and compress runs after every
 * append; writes the calls that fire, in launch order, as (event, level, ordinal)
 * triples.  Returns the number of calls (at most max_calls are written) or an error. */
int balancekv_plan_calls(int block, int levels, int recent_window, const int32_t* appended_after_event,
                         int n_events, int32_t* calls_out, int max_calls);

#ifdef __cplusplus
}
#endif
#endif /* BALANCEKV_H_ */
