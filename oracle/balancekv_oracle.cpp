// BalanceKV CPU oracle -- TEST INFRASTRUCTURE, NOT PART OF THE PRODUCT.
//
// A plain, slow, double-precision restatement of the method of
// "Streaming Attention Approximation via Discrepancy Theory" (BalanceKV):
//   * SoftmaxBalance (Algorithm 2): the self-balancing walk (Algorithm 4) run on the
//     implicit feature vectors phi(k_i) (x) v_i, whose inner product is the pairwise
//     kernel exp(<k_i,k_j>/sqrt d) <v_i,v_j> (proof of Theorem 3.2).
//   * the strict n/2 selection of the "Implementation Detail" paragraph of Appendix B,
//   * MergeAndReduce (Algorithm 3) with its estimator (Theorem 3.3),
//   * the attention definition Eq. (1) and the weighted estimator ratio of
//     Algorithm 1's output ratio, evaluated over one shared weighted set, and its two
//     un-normalised halves for the form with a separate denominator instance.
//
// It shares no code with the CUDA library: no common header, helper, table or
// constant generator.  Only tests, the smoke check and the bench's cpu_baseline /
// reference arm may call it.  Everything is double precision, std::exp, no blocking,
// no fusion, no reordering beyond what the algorithms state.
//
// Parity pins (see tests/test_oracle_*.py): Philox known-answer vectors; T=0 equals
// Eq. (1); weight-sum and level-size invariants; brute-force enumeration of the walk
// law for m<=16; closed forms of the kernel; the Theorem 3.2 bound with explicit c; the
// un-normalised sums against a direct evaluation and against the pinned ratio.
//
// Build: g++ -O2 -fopenmp -shared -fPIC balancekv_oracle.cpp -o libbalancekv_oracle.so

#include <cmath>
#include <cstdint>
#include <cstring>
#include <map>
#include <utility>
#include <vector>
#include <algorithm>
#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

// ---------------------------------------------------------------------------------
// Philox4x32-10 (Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as
// 1, 2, 3", SC'11): counter-based generator, written from its published definition.
// ---------------------------------------------------------------------------------
void philox4x32_10(const uint32_t key_in[2], const uint32_t ctr_in[4], uint32_t out[4]) {
  const uint64_t mult_a = 0xD2511F53ull, mult_b = 0xCD9E8D57ull;
  const uint32_t weyl_a = 0x9E3779B9u, weyl_b = 0xBB67AE85u;
  uint32_t x[4] = {ctr_in[0], ctr_in[1], ctr_in[2], ctr_in[3]};
  uint32_t k0 = key_in[0], k1 = key_in[1];
  for (int round = 0; round < 10; ++round) {
    if (round > 0) { k0 += weyl_a; k1 += weyl_b; }
    uint64_t pa = mult_a * (uint64_t)x[0];
    uint64_t pb = mult_b * (uint64_t)x[2];
    uint32_t y0 = (uint32_t)(pb >> 32) ^ x[1] ^ k0;
    uint32_t y1 = (uint32_t)pb;
    uint32_t y2 = (uint32_t)(pa >> 32) ^ x[3] ^ k1;
    uint32_t y3 = (uint32_t)pa;
    x[0] = y0; x[1] = y1; x[2] = y2; x[3] = y3;
  }
  for (int i = 0; i < 4; ++i) out[i] = x[i];
}

// The coin of Algorithm 2 ("+1 with probability p_j"): a 24-bit uniform in [0,1) drawn
// from the Philox stream keyed by (seed) at counter (token j, call ordinal, level,
// layer<<16 | head).
double walk_uniform(uint64_t seed, int layer, int head, int ordinal, int level, int j) {
  uint32_t key[2] = {(uint32_t)(seed & 0xffffffffull), (uint32_t)(seed >> 32)};
  uint32_t ctr[4] = {(uint32_t)j, (uint32_t)ordinal, (uint32_t)level,
                     ((uint32_t)layer << 16) | ((uint32_t)head & 0xffffu)};
  uint32_t r[4];
  philox4x32_10(key, ctr, r);
  return (double)(r[0] >> 8) * (1.0 / 16777216.0);
}

struct Params {
  int32_t d;            // head dimension
  int32_t t;            // batch size t of Algorithm 3 (tokens per call)
  int32_t T;            // number of levels (compression rate 2^-T)
  int32_t W;            // recent window kept exact
  int32_t center_keys;  // shift keys by the call's mean inside the kernel only
  int32_t layer, head;  // Philox coordinates
  int32_t max_tokens;   // N: enters the default delta = N^-2
  uint64_t seed;        // Philox key of this sequence
  double delta;         // <=0 -> 1/N^2
  double c_override;    // >0 -> use as c
  double r_key, r_value;  // >0 -> fixed radii, else per-call maxima
};

struct CallRecord {
  int level = 0, ordinal = 0, m = 0, fails = 0;
  double rk2 = 0, rv2 = 0, c = 0;
  std::vector<int32_t> idx;    // original token index of each in-call position
  std::vector<int8_t> eta;     // signs
  std::vector<double> S, p, u; // running correlation / probability / uniform per position
  std::vector<int32_t> kept;   // kept in-call positions, ascending (exactly m/2)
};

double dot(const double* a, const double* b, int d) {
  double s = 0.0;
  for (int e = 0; e < d; ++e) s += a[e] * b[e];
  return s;
}

// c = 30 log(n/delta) (Algorithm 2): natural log, n := tokens of this call,
// delta := 1/N^2 by default; rounded once to single precision so that a single-
// precision implementation can use the identical constant.
double walk_constant(const Params& P, int m) {
  if (P.c_override > 0) return (double)(float)P.c_override;
  double delta = P.delta > 0 ? P.delta : 1.0 / ((double)P.max_tokens * (double)P.max_tokens);
  double c = 30.0 * std::log((double)m / delta);
  return (double)(float)c;
}

// One SoftmaxBalance call (Algorithm 2) followed by the strict-half selection.
// K,V: [m,d] row-major.  forced: optional sign vector to follow instead of the coin
// (the probabilities and uniforms are still recorded) -- used for teacher-forced checks.
void softmax_balance(const Params& P, const double* K, const double* V, int m, int ordinal,
                     int level, const int8_t* forced, CallRecord& rec) {
  const int d = P.d;
  rec.level = level; rec.ordinal = ordinal; rec.m = m; rec.fails = 0;
  rec.eta.assign(m, 0); rec.S.assign(m, 0.0); rec.p.assign(m, 0.0); rec.u.assign(m, 0.0);

  // keys as seen by the kernel (optionally mean-shifted; stored keys are untouched)
  std::vector<double> Kc(K, K + (size_t)m * d);
  if (P.center_keys) {
    std::vector<double> mean(d, 0.0);
    for (int j = 0; j < m; ++j) for (int e = 0; e < d; ++e) mean[e] += Kc[(size_t)j * d + e];
    for (int e = 0; e < d; ++e) mean[e] /= (double)m;
    for (int j = 0; j < m; ++j) for (int e = 0; e < d; ++e) Kc[(size_t)j * d + e] -= mean[e];
  }
  // radii (inputs of Algorithm 2): tightest valid values unless fixed by the caller
  double rk2 = 0, rv2 = 0;
  if (P.r_key > 0) rk2 = P.r_key * P.r_key;
  else for (int j = 0; j < m; ++j) rk2 = std::max(rk2, dot(&Kc[(size_t)j * d], &Kc[(size_t)j * d], d));
  if (P.r_value > 0) rv2 = P.r_value * P.r_value;
  else for (int j = 0; j < m; ++j) rv2 = std::max(rv2, dot(V + (size_t)j * d, V + (size_t)j * d, d));
  const double c = walk_constant(P, m);
  rec.rk2 = rk2; rec.rv2 = rv2; rec.c = c;
  const double inv_sqrt_d = 1.0 / std::sqrt((double)d);

  // the walk (the loop of Algorithm 2), on the kernel divided by R^2 =
  // exp(r_key^2/sqrt d) r_value^2, i.e. y^T eta / R^2 compared with c
  for (int j = 0; j < m; ++j) {
    double S = 0.0;
    if (rv2 > 0) {
      for (int i = 0; i < j; ++i) {
        double kk = dot(&Kc[(size_t)i * d], &Kc[(size_t)j * d], d);
        double vv = dot(V + (size_t)i * d, V + (size_t)j * d, d);
        double g = std::exp((kk - rk2) * inv_sqrt_d) * (vv / rv2);
        S += (double)rec.eta[i] * g;
      }
    }
    rec.S[j] = S;
    double Sc = S;
    if (std::fabs(S) > c) { rec.fails++; Sc = S > 0 ? c : -c; }  // FAIL: counted, clamped
    double p = 0.5 - Sc / (2.0 * c);
    double u = walk_uniform(P.seed, P.layer, P.head, ordinal, level, j);
    rec.p[j] = p; rec.u[j] = u;
    int8_t sign = (u < p) ? 1 : -1;
    rec.eta[j] = forced ? forced[j] : sign;
  }

  // Algorithm 2's output step: the smaller sign class (ties -> +1) ...
  int plus = 0;
  for (int j = 0; j < m; ++j) plus += rec.eta[j] > 0;
  int minus = m - plus;
  int8_t keep_sign = (plus <= minus) ? 1 : -1;
  int have = keep_sign > 0 ? plus : minus;
  // ... completed to exactly m/2 with the latest tokens of the other class
  int need = m / 2 - have;
  std::vector<char> keep(m, 0);
  for (int j = 0; j < m; ++j) if (rec.eta[j] == keep_sign) keep[j] = 1;
  for (int j = m - 1; j >= 0 && need > 0; --j)
    if (rec.eta[j] != keep_sign) { keep[j] = 1; --need; }
  rec.kept.clear();
  for (int j = 0; j < m; ++j) if (keep[j]) rec.kept.push_back(j);
}

// One (sequence, layer, KV head) stream: MergeAndReduce (Algorithm 3).
struct Stream {
  Params P;
  std::vector<double> K, V;                 // every token ever appended, [n,d]
  int64_t n = 0;                            // tokens appended
  int64_t blocks_done = 0;                  // level-0 calls run so far (beta)
  int64_t consumed = 0;                     // tokens that left C^0 (= blocks_done * t)
  std::vector<std::vector<int32_t>> level;  // level[i] = original indices in C^i, i=1..T
  std::vector<CallRecord> calls;
  std::map<std::pair<int, int>, std::vector<int8_t>> forced;

  int run_call(const std::vector<int32_t>& idx, int lvl, int ordinal) {
    const int d = P.d, m = (int)idx.size();
    std::vector<double> Kb((size_t)m * d), Vb((size_t)m * d);
    for (int j = 0; j < m; ++j) {
      std::memcpy(&Kb[(size_t)j * d], &K[(size_t)idx[j] * d], sizeof(double) * d);
      std::memcpy(&Vb[(size_t)j * d], &V[(size_t)idx[j] * d], sizeof(double) * d);
    }
    calls.emplace_back();
    CallRecord& rec = calls.back();
    rec.idx = idx;
    auto it = forced.find({lvl, ordinal});
    const int8_t* f = (it != forced.end() && (int)it->second.size() == m) ? it->second.data() : nullptr;
    softmax_balance(P, Kb.data(), Vb.data(), m, ordinal, lvl, f, rec);
    return (int)calls.size() - 1;
  }

  // Run every call that is ready (the update step of Algorithm 3); returns calls run.
  int compress() {
    if (P.T <= 0) return 0;
    int ran = 0;
    const int t = P.t;
    for (;;) {
      int64_t eligible = std::max<int64_t>(0, n - P.W);
      if ((blocks_done + 1) * (int64_t)t > eligible) break;
      int64_t beta = blocks_done + 1;
      std::vector<int32_t> cur(t);
      for (int j = 0; j < t; ++j) cur[j] = (int32_t)(consumed + j);
      int64_t p = beta;
      int i = 0;
      // "while p is an integer and until i = T"
      for (;;) {
        int c = run_call(cur, i, (int)(p - 1));
        ++ran;
        const CallRecord& rec = calls[c];
        for (int pos : rec.kept) level[i + 1].push_back(rec.idx[pos]);
        ++i;
        if (i >= P.T) break;
        if (p % 2 != 0) break;
        p /= 2;
        cur = level[i];       // C^i holds exactly t tokens here (two halves)
        level[i].clear();
      }
      blocks_done = beta;
      consumed += t;
    }
    return ran;
  }

  // the weighted set in the order C^T, C^(T-1), ..., C^1, C^0 (ascending original index)
  void view(std::vector<int32_t>& idx, std::vector<double>& w) const {
    idx.clear(); w.clear();
    for (int i = P.T; i >= 1; --i)
      for (int32_t x : level[i]) { idx.push_back(x); w.push_back(std::ldexp(1.0, i)); }
    for (int64_t x = consumed; x < n; ++x) { idx.push_back((int32_t)x); w.push_back(1.0); }
  }
};

// z = sum_i w_i exp(<k_i,q>/sqrt d) v_i / sum_i w_i exp(<k_i,q>/sqrt d)
// (Algorithm 1's output ratio with one shared set; Eq. (1) when every w_i = 1),
// evaluated with the maximum logit subtracted.
void weighted_attention(const double* K, const double* V, const double* w, int64_t len, int d,
                        const double* q, double* out) {
  const double inv_sqrt_d = 1.0 / std::sqrt((double)d);
  std::vector<double> logit((size_t)len);
  double mx = -INFINITY;
  for (int64_t i = 0; i < len; ++i) {
    logit[i] = dot(K + i * d, q, d) * inv_sqrt_d + std::log(w ? w[i] : 1.0);
    mx = std::max(mx, logit[i]);
  }
  double Z = 0.0;
  std::vector<double> acc(d, 0.0);
  for (int64_t i = 0; i < len; ++i) {
    double e = std::exp(logit[i] - mx);
    Z += e;
    for (int c = 0; c < d; ++c) acc[c] += e * V[i * d + c];
  }
  for (int c = 0; c < d; ++c) out[c] = len > 0 ? acc[c] / Z : 0.0;
}

}  // namespace

extern "C" {

struct okv_params {
  int32_t d, t, T, W, center_keys, layer, head, max_tokens;
  uint64_t seed;
  double delta, c_override, r_key, r_value;
};

static Params to_params(const okv_params* p) {
  Params P;
  P.d = p->d; P.t = p->t; P.T = p->T; P.W = p->W; P.center_keys = p->center_keys;
  P.layer = p->layer; P.head = p->head; P.max_tokens = p->max_tokens; P.seed = p->seed;
  P.delta = p->delta; P.c_override = p->c_override; P.r_key = p->r_key; P.r_value = p->r_value;
  return P;
}

void okv_philox4x32_10(const uint32_t* key, const uint32_t* ctr, uint32_t* out) {
  philox4x32_10(key, ctr, out);
}

double okv_walk_uniform(uint64_t seed, int layer, int head, int ordinal, int level, int j) {
  return walk_uniform(seed, layer, head, ordinal, level, j);
}

double okv_walk_constant(const okv_params* p, int m) { return walk_constant(to_params(p), m); }

// Stand-alone SoftmaxBalance call.  forced may be null.  kept receives m/2 positions.
int okv_softmax_balance(const okv_params* p, const double* K, const double* V, int m, int ordinal,
                        int level, const int8_t* forced, int8_t* eta, double* S, double* prob,
                        double* u, int32_t* kept, double* stats /* rk2, rv2, c, fails */) {
  Params P = to_params(p);
  CallRecord rec;
  softmax_balance(P, K, V, m, ordinal, level, forced, rec);
  if (eta) std::memcpy(eta, rec.eta.data(), m);
  if (S) std::memcpy(S, rec.S.data(), sizeof(double) * m);
  if (prob) std::memcpy(prob, rec.p.data(), sizeof(double) * m);
  if (u) std::memcpy(u, rec.u.data(), sizeof(double) * m);
  if (kept) std::memcpy(kept, rec.kept.data(), sizeof(int32_t) * rec.kept.size());
  if (stats) { stats[0] = rec.rk2; stats[1] = rec.rv2; stats[2] = rec.c; stats[3] = rec.fails; }
  return (int)rec.kept.size();
}

void* okv_stream_new(const okv_params* p) {
  Stream* s = new Stream();
  s->P = to_params(p);
  s->level.assign((size_t)std::max(1, s->P.T + 1), {});
  return s;
}
void okv_stream_free(void* h) { delete (Stream*)h; }

int okv_stream_append(void* h, const double* K, const double* V, int n) {
  Stream* s = (Stream*)h;
  s->K.insert(s->K.end(), K, K + (size_t)n * s->P.d);
  s->V.insert(s->V.end(), V, V + (size_t)n * s->P.d);
  s->n += n;
  return 0;
}

int okv_stream_force_eta(void* h, int level, int ordinal, const int8_t* eta, int m) {
  Stream* s = (Stream*)h;
  s->forced[{level, ordinal}] = std::vector<int8_t>(eta, eta + m);
  return 0;
}

int okv_stream_compress(void* h) { return ((Stream*)h)->compress(); }

// OpenMP over independent streams only.
int okv_streams_compress(void** hs, int n) {
  int total = 0;
#pragma omp parallel for schedule(dynamic, 1) reduction(+ : total)
  for (int i = 0; i < n; ++i) total += ((Stream*)hs[i])->compress();
  return total;
}

int64_t okv_stream_len(void* h) {
  Stream* s = (Stream*)h;
  int64_t len = s->n - s->consumed;
  for (int i = 1; i <= s->P.T; ++i) len += (int64_t)s->level[i].size();
  return len;
}

// sizes[0..T]: |C^0| (everything at weight 1), |C^1|, ..., |C^T|
void okv_stream_level_sizes(void* h, int64_t* sizes) {
  Stream* s = (Stream*)h;
  sizes[0] = s->n - s->consumed;
  for (int i = 1; i <= s->P.T; ++i) sizes[i] = (int64_t)s->level[i].size();
}

void okv_stream_view(void* h, double* K, double* V, double* w, int32_t* idx) {
  Stream* s = (Stream*)h;
  std::vector<int32_t> ix; std::vector<double> ww;
  s->view(ix, ww);
  const int d = s->P.d;
  for (size_t i = 0; i < ix.size(); ++i) {
    if (K) std::memcpy(K + i * d, &s->K[(size_t)ix[i] * d], sizeof(double) * d);
    if (V) std::memcpy(V + i * d, &s->V[(size_t)ix[i] * d], sizeof(double) * d);
    if (w) w[i] = ww[i];
    if (idx) idx[i] = ix[i];
  }
}

int okv_stream_num_calls(void* h) { return (int)((Stream*)h)->calls.size(); }

void okv_stream_call_info(void* h, int c, int32_t* info /* level, ordinal, m, fails */,
                          double* stats /* rk2, rv2, c */) {
  const CallRecord& r = ((Stream*)h)->calls[c];
  info[0] = r.level; info[1] = r.ordinal; info[2] = r.m; info[3] = r.fails;
  stats[0] = r.rk2; stats[1] = r.rv2; stats[2] = r.c;
}

void okv_stream_call_data(void* h, int c, int32_t* idx, int8_t* eta, double* S, double* prob,
                          double* u, int32_t* kept) {
  const CallRecord& r = ((Stream*)h)->calls[c];
  if (idx) std::memcpy(idx, r.idx.data(), sizeof(int32_t) * r.m);
  if (eta) std::memcpy(eta, r.eta.data(), r.m);
  if (S) std::memcpy(S, r.S.data(), sizeof(double) * r.m);
  if (prob) std::memcpy(prob, r.p.data(), sizeof(double) * r.m);
  if (u) std::memcpy(u, r.u.data(), sizeof(double) * r.m);
  if (kept) std::memcpy(kept, r.kept.data(), sizeof(int32_t) * r.kept.size());
}

// Decode over the stream's weighted set for nq queries: q [nq,d] -> out [nq,d]
void okv_stream_decode(void* h, const double* q, int nq, double* out) {
  Stream* s = (Stream*)h;
  std::vector<int32_t> ix; std::vector<double> ww;
  s->view(ix, ww);
  const int d = s->P.d;
  std::vector<double> Kc(ix.size() * (size_t)d), Vc(ix.size() * (size_t)d);
  for (size_t i = 0; i < ix.size(); ++i) {
    std::memcpy(&Kc[i * d], &s->K[(size_t)ix[i] * d], sizeof(double) * d);
    std::memcpy(&Vc[i * d], &s->V[(size_t)ix[i] * d], sizeof(double) * d);
  }
  for (int a = 0; a < nq; ++a)
    weighted_attention(Kc.data(), Vc.data(), ww.data(), (int64_t)ix.size(), d, q + (size_t)a * d,
                       out + (size_t)a * d);
}

// Exact attention over every token appended so far (Eq. (1)).
void okv_stream_exact(void* h, const double* q, int nq, double* out) {
  Stream* s = (Stream*)h;
  for (int a = 0; a < nq; ++a)
    weighted_attention(s->K.data(), s->V.data(), nullptr, s->n, s->P.d, q + (size_t)a * s->P.d,
                       out + (size_t)a * s->P.d);
}

// Un-normalised weighted sums over explicit arrays (the two halves of Algorithm 1's output ratio,
// which takes its numerator from the sets V^l of one MergeAndReduce instance and its denominator
// from the sets K^l of another):  with m = max_i (<k_i,q>/sqrt d + ln w_i),
//   num[c] = sum_i w_i e^{<k_i,q>/sqrt d - m} v_i[c],   den = sum_i w_i e^{<k_i,q>/sqrt d - m},   logmax = m.
void okv_weighted_sums(const double* K, const double* V, const double* w, int64_t len, int d, const double* q,
                       int nq, double* num, double* den, double* logmax) {
  const double inv_sqrt_d = 1.0 / std::sqrt((double)d);
  for (int a = 0; a < nq; ++a) {
    const double* qa = q + (size_t)a * d;
    double mx = -INFINITY;
    for (int64_t i = 0; i < len; ++i)
      mx = std::max(mx, dot(K + i * d, qa, d) * inv_sqrt_d + std::log(w ? w[i] : 1.0));
    double Z = 0.0;
    for (int c = 0; c < d; ++c) num[(size_t)a * d + c] = 0.0;
    for (int64_t i = 0; i < len; ++i) {
      const double e = std::exp(dot(K + i * d, qa, d) * inv_sqrt_d + std::log(w ? w[i] : 1.0) - mx);
      Z += e;
      for (int c = 0; c < d; ++c) num[(size_t)a * d + c] += e * V[i * d + c];
    }
    den[a] = Z;
    logmax[a] = mx;
  }
}

// Weighted attention over explicit arrays: K,V [len,d], w [len] (null = all ones).
void okv_weighted_attn(const double* K, const double* V, const double* w, int64_t len, int d,
                       const double* q, int nq, double* out) {
#pragma omp parallel for schedule(dynamic, 1)
  for (int a = 0; a < nq; ++a)
    weighted_attention(K, V, w, len, d, q + (size_t)a * d, out + (size_t)a * d);
}

int okv_num_threads() {
  int n = 1;
#ifdef _OPENMP
#pragma omp parallel
  {
#pragma omp single
    n = omp_get_num_threads();
  }
#endif
  return n;
}

}  // extern "C"
