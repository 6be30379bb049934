// ORACLE -- TEST INFRASTRUCTURE ONLY.
//
// A plain, slow, obviously-correct CPU statement of speculative sampling
// (Chen et al., "Accelerating Large Language Model Decoding with Speculative
// Sampling"): Algorithm 1 (auto-regressive sampling), Algorithm 2 (speculative
// sampling), the modified rejection sampling scheme of the section of that
// name, and the decoder-only transformer the two models are instances of.
//
// Only the tests, the smoke check and the benchmark's CPU-baseline leg may
// call into this file.  It shares no code, header, table or constant with the
// CUDA library; it never includes or links anything from it.
//
// Numerics: logits, weights and the KV cache are read from their storage type
// (fp32, or bf16 widened exactly); every dot product, reduction, softmax,
// CDF and ratio is carried in double.  No blocking, fusion or reordering:
// sums run in index order.
//
// Notation follows the paper: q is the TARGET model, p is the DRAFT model,
// K is the lookahead, x~_t (here d_t, 0-based) are the draft tokens.
//
// Pins (what each function is checked against, in tests/ with -m "not gpu"):
//   philox            : published known-answer vectors (tests/golden/philox_kat.txt)
//   accept chain      : Theorem 1 closed forms, brute-force enumeration
//   sps loop          : exact end-to-end distribution on a vocab-16 pair, K=0 == Alg. 1
//   transformer       : PARITY UNPINNED BY THE PAPER (it prints no architecture
//                       values); pinned by cached == uncached forward, an
//                       independent numpy restatement, and invariances.
//   linear            : an independent float64 matrix product (fp32 and bf16 weights,
//                       ragged shapes), also at sizes where the rows are split over
//                       threads, where the result must equal the one-thread result bit for bit
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstdio>
#include <cstring>
#include <thread>
#include <vector>

// Rows of a large mat-vec are split over plain std::threads (no OpenMP runtime: the host process
// usually carries another one already).  Small problems run on the calling thread.
static int g_threads_override = 0;   // test hook (orc_set_threads): > 0 replaces the machine's thread count
static int hw_threads() {
  if (g_threads_override > 0) return g_threads_override;
  static const int n = [] {
    unsigned h = std::thread::hardware_concurrency();
    int v = h ? (int)h : 1;
    return v > 64 ? 64 : v;
  }();
  return n;
}
template <class F>
static void parallel_rows(int N, long long work_per_row, F fn) {
  const int T = hw_threads();
  if (T <= 1 || (long long)N * work_per_row < (1ll << 22)) { fn(0, N); return; }
  std::vector<std::thread> th;
  const int per = (N + T - 1) / T;
  for (int t = 0; t < T; ++t) {
    const int a = t * per, b = std::min(N, a + per);
    if (a >= b) break;
    th.emplace_back([=] { fn(a, b); });
  }
  for (auto& x : th) x.join();
}

// ---------------------------------------------------------------------------
// Random numbers.  Algorithm 2 draws r ~ U[0,1] and "samples" tokens without
// naming a generator; this build fixes a counter-based one so that two
// implementations can be compared token by token: Philox4x32-10 (Salmon et
// al., SC'11), key = (seed low, seed high), counter = (t, s, b, 0) with t the
// position inside the loop, s the loop index, b the sequence index.
// ---------------------------------------------------------------------------
static inline void philox_round(uint32_t c[4], const uint32_t k[2]) {
  const uint64_t p0 = (uint64_t)0xD2511F53u * c[0];
  const uint64_t p1 = (uint64_t)0xCD9E8D57u * c[2];
  const uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
  const uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
  const uint32_t n0 = hi1 ^ c[1] ^ k[0];
  const uint32_t n2 = hi0 ^ c[3] ^ k[1];
  c[0] = n0; c[1] = lo1; c[2] = n2; c[3] = lo0;
}

extern "C" void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  uint32_t c[4] = {ctr[0], ctr[1], ctr[2], ctr[3]};
  uint32_t k[2] = {key[0], key[1]};
  for (int r = 0; r < 10; ++r) {
    philox_round(c, k);
    k[0] += 0x9E3779B9u;
    k[1] += 0xBB67AE85u;
  }
  for (int i = 0; i < 4; ++i) out[i] = c[i];
}

// U(w) = (w >> 8) * 2^-24: a 24-bit grid in [0, 1), exact in fp32 and fp64.
static inline double u01(uint32_t w) { return (double)(w >> 8) * (1.0 / 16777216.0); }

// out[0] = u_draft (draw of x~_t from p_t), out[1] = u_acc (the r of
// Algorithm 2's accept test), out[2] = u_res (residual resample at t, or the
// extra-token draw when t == K).
extern "C" void orc_uniforms(uint64_t seed, uint32_t b, uint32_t s, uint32_t t, double out[3]) {
  const uint32_t ctr[4] = {t, s, b, 0u};
  const uint32_t key[2] = {(uint32_t)seed, (uint32_t)(seed >> 32)};
  uint32_t w[4];
  orc_philox4x32_10(ctr, key, w);
  out[0] = u01(w[0]); out[1] = u01(w[1]); out[2] = u01(w[2]);
}

// ---------------------------------------------------------------------------
// Distributions.
// ---------------------------------------------------------------------------
// softmax(l / T): subtract the maximum, exponentiate, divide by the sum.
// (Modified Rejection Sampling: a temperature changes both models'
// probabilities before the rejection scheme sees them.)
static void softmax_T(const float* logits, int V, double T, std::vector<double>& prob) {
  prob.resize(V);
  double mx = -INFINITY;
  for (int i = 0; i < V; ++i) mx = std::max(mx, (double)logits[i] / T);
  double sum = 0.0;
  for (int i = 0; i < V; ++i) { prob[i] = std::exp((double)logits[i] / T - mx); sum += prob[i]; }
  for (int i = 0; i < V; ++i) prob[i] /= sum;
}

// Top-k and nucleus (top-p) filtering.  The section Modified Rejection
// Sampling says that such sampling methods are handled by changing the
// probabilities first and applying the rejection scheme to the changed
// distributions; it names the methods and gives no formula.  This build's
// reading, applied to the draft and the target alike:
//   1. pr = softmax(l / T);
//   2. top-k (k >= 1; 0 = off): keep every token whose logit is at least the
//      k-th largest logit (tokens tied with the k-th are all kept);
//   3. nucleus (0 < top_p < 1; 1 = off), on what step 2 kept, mass Z_k: walk the
//      distinct logit values downwards adding the mass of each value's tokens;
//      stop at the first value where the running mass reaches top_p * Z_k, keep
//      that value and everything above it;
//   4. zero the rest and renormalise.
// Greedy decoding is top_k = 1.  *near_cut is set when the running mass passes
// top_p * Z_k within 1e-5 * Z_k on either side of the cut, i.e. when sums taken
// in another order or precision could legitimately cut one value earlier or later.
struct Filt { int top_k = 0; double top_p = 1.0; };

static void filtered_T(const float* logits, int V, double T, const Filt& f, std::vector<double>& prob, int* near_cut) {
  softmax_T(logits, V, T, prob);
  if (near_cut) *near_cut = 0;
  const bool use_k = f.top_k >= 1 && f.top_k < V, use_p = f.top_p < 1.0;
  if (!use_k && !use_p) return;
  std::vector<int> order(V);
  for (int i = 0; i < V; ++i) order[i] = i;
  std::stable_sort(order.begin(), order.end(), [&](int a, int b) { return logits[a] > logits[b]; });
  float cut = -INFINITY;            // keep logits >= cut
  int n_k = V;                      // how many tokens step 2 keeps (a prefix of `order`)
  if (use_k) {
    const float lk = logits[order[f.top_k - 1]];
    n_k = f.top_k;
    while (n_k < V && logits[order[n_k]] == lk) ++n_k;
    cut = lk;
  }
  if (use_p) {
    double Zk = 0.0;
    for (int j = 0; j < n_k; ++j) Zk += prob[order[j]];
    const double target = f.top_p * Zk, band = 1e-5 * Zk;
    double run = 0.0;
    int j = 0;
    while (j < n_k) {
      const float v = logits[order[j]];
      const double before = run;
      while (j < n_k && logits[order[j]] == v) run += prob[order[j++]];
      if (run >= target) {
        if (v > cut) cut = v;
        if (near_cut && ((run - target < band && j < n_k) || (before > 0.0 && target - before < band))) *near_cut = 1;
        break;
      }
    }
  }
  double Z = 0.0;
  for (int i = 0; i < V; ++i) { if (logits[i] < cut) prob[i] = 0.0; else Z += prob[i]; }
  for (int i = 0; i < V; ++i) prob[i] /= Z;
}

// Inverse-CDF draw on unnormalised weights, in index order: the smallest i
// whose inclusive running sum C_i exceeds u * C_{V-1}; if rounding leaves none,
// the largest i with w_i > 0.  *near_tie is set when u * total lies within
// 2e-6 * total of either edge of the chosen token's interval, i.e. when a sum
// taken in another order could legitimately pick a neighbour.
static int invcdf(const double* w, int V, double u, int* near_tie) {
  double total = 0.0;
  for (int i = 0; i < V; ++i) total += w[i];
  const double target = u * total;
  double c = 0.0;
  int pick = -1;
  double lo = 0.0, hi = 0.0;
  for (int i = 0; i < V; ++i) {
    const double c_prev = c;
    c += w[i];
    if (c > target) { pick = i; lo = c_prev; hi = c; break; }
  }
  if (pick < 0) {
    for (int i = V - 1; i >= 0; --i) if (w[i] > 0.0) { pick = i; break; }
    if (pick < 0) pick = V - 1;
    if (near_tie) *near_tie = 1;
    return pick;
  }
  if (near_tie) {
    const double band = 2e-6 * total;
    // the lower edge at 0 and the upper edge at total are not boundaries
    // between two tokens; every other edge is.
    const bool lo_close = (lo > 0.0) && (target - lo < band);
    const bool hi_close = (hi - target < band);
    *near_tie = (lo_close || hi_close) ? 1 : 0;
  }
  return pick;
}

// One token from softmax(logits / T) by inverse CDF (Algorithm 1's "Sample",
// and Algorithm 2's draft draw).
extern "C" int orc_sample_row(const float* logits, int V, double T, double u, int* near_tie) {
  std::vector<double> pr;
  softmax_T(logits, V, T, pr);
  return invcdf(pr.data(), V, u, near_tie);
}
// the same draw from the top-k / nucleus filtered distribution; *near_tie also covers a near cut
extern "C" int orc_sample_row_f(const float* logits, int V, double T, int top_k, double top_p, double u, int* near_tie) {
  std::vector<double> pr;
  Filt f; f.top_k = top_k; f.top_p = top_p;
  int nc = 0, nt = 0;
  filtered_T(logits, V, T, f, pr, &nc);
  const int tok = invcdf(pr.data(), V, u, &nt);
  if (near_tie) *near_tie = (nc || nt) ? 1 : 0;
  return tok;
}
extern "C" void orc_filtered(const float* logits, int V, double T, int top_k, double top_p, double* out, int* near_cut) {
  std::vector<double> pr;
  Filt f; f.top_k = top_k; f.top_p = top_p;
  filtered_T(logits, V, T, f, pr, near_cut);
  for (int i = 0; i < V; ++i) out[i] = pr[i];
}

extern "C" void orc_softmax(const float* logits, int V, double T, double* out) {
  std::vector<double> pr;
  softmax_T(logits, V, T, pr);
  for (int i = 0; i < V; ++i) out[i] = pr[i];
}

enum : uint32_t {
  ORC_RESAMPLED = 1u,       // a draft was rejected and a token drawn from the residual
  ORC_BONUS = 2u,           // all K drafts accepted, extra token drawn from q_{K+1}
  ORC_FALLBACK = 4u,        // rejected although sum max(0, q-p) == 0: drawn from q_t
  ORC_NEAR_ACCEPT = 256u,   // |u_acc - min(1, q/p)| < 1e-4 at some tested position
  ORC_NEAR_CDF = 512u,      // the resample / extra-token draw fell in a CDF edge band
  ORC_NEAR_CUT = 1024u      // a nucleus cut of a distribution this loop used was within its tie band
};

// Modified rejection sampling over one loop's K drafts (Algorithm 2, second
// for-loop and the extra-token line; section "Modified Rejection Sampling").
//   q_logits [K+1][V] target logits, row t scores draft t; row K is the extra token's
//   p_logits [K][V]   draft logits the drafts were drawn from
//   drafts   [K]
// Writes the emitted tokens (n_accepted drafts then one resampled or extra
// token) to out_tokens[0..n_accepted], -1 beyond; optional beta[K] receives
// sum_x min(p_t(x), q_t(x)) (Theorem 1's acceptance probability).
static void accept_chain_impl(const float* q_logits, const float* p_logits, const int32_t* drafts,
                              int K, int V, double T, const Filt& filt, uint64_t seed, uint32_t b, uint32_t s,
                              int32_t* out_tokens, int32_t* n_accepted, uint32_t* flags,
                              double* beta) {
  std::vector<double> q, p, r(V);
  uint32_t fl = 0;
  // q and p below are the distributions after temperature, top-k and nucleus
  auto softmax_T = [&](const float* lg, int V_, double T_, std::vector<double>& out) {
    int nc = 0;
    filtered_T(lg, V_, T_, filt, out, &nc);
    if (nc) fl |= ORC_NEAR_CUT;
  };
  int a = 0;
  for (int i = 0; i <= K; ++i) out_tokens[i] = -1;
  if (beta) {
    for (int t = 0; t < K; ++t) {
      softmax_T(q_logits + (size_t)t * V, V, T, q);
      softmax_T(p_logits + (size_t)t * V, V, T, p);
      double bsum = 0.0;
      for (int x = 0; x < V; ++x) bsum += std::min(p[x], q[x]);
      beta[t] = bsum;
    }
  }
  bool rejected = false;
  for (int t = 0; t < K; ++t) {
    double u[3];
    orc_uniforms(seed, b, s, (uint32_t)t, u);
    softmax_T(q_logits + (size_t)t * V, V, T, q);
    softmax_T(p_logits + (size_t)t * V, V, T, p);
    const int d = drafts[t];
    const double qd = q[d], pd = p[d];
    // accept with probability min(1, q(d)/p(d)); r < ... is strict.
    // p == 0 cannot happen for a token drawn from p in exact arithmetic; by
    // convention p == 0 and q > 0 accepts, 0/0 rejects.
    double ratio;
    if (pd > 0.0) ratio = std::min(1.0, qd / pd);
    else ratio = (qd > 0.0) ? 1.0 : 0.0;
    if (std::fabs(u[1] - ratio) < 1e-4) fl |= ORC_NEAR_ACCEPT;
    if (u[1] < ratio) {
      out_tokens[a++] = d;
      continue;
    }
    // rejected: x ~ (q - p)_+ = max(0, q - p) / sum max(0, q - p)
    double S = 0.0;
    for (int x = 0; x < V; ++x) { r[x] = std::max(0.0, q[x] - p[x]); S += r[x]; }
    int nt = 0;
    int tok;
    if (S > 0.0) {
      tok = invcdf(r.data(), V, u[2], &nt);
    } else {
      tok = invcdf(q.data(), V, u[2], &nt);
      fl |= ORC_FALLBACK;
    }
    if (nt) fl |= ORC_NEAR_CDF;
    fl |= ORC_RESAMPLED;
    out_tokens[a] = tok;
    rejected = true;
    break;
  }
  if (!rejected) {
    // every draft accepted: the (K+1)-th distribution gives one more token.
    double u[3];
    orc_uniforms(seed, b, s, (uint32_t)K, u);
    softmax_T(q_logits + (size_t)K * V, V, T, q);
    int nt = 0;
    out_tokens[a] = invcdf(q.data(), V, u[2], &nt);
    if (nt) fl |= ORC_NEAR_CDF;
    fl |= ORC_BONUS;
  }
  *n_accepted = a;
  *flags = fl;
}

extern "C" void orc_accept_chain(const float* q_logits, const float* p_logits, const int32_t* drafts,
                                 int K, int V, double T, uint64_t seed, uint32_t b, uint32_t s,
                                 int32_t* out_tokens, int32_t* n_accepted, uint32_t* flags,
                                 double* beta) {
  accept_chain_impl(q_logits, p_logits, drafts, K, V, T, Filt(), seed, b, s, out_tokens, n_accepted, flags, beta);
}
extern "C" void orc_accept_chain_f(const float* q_logits, const float* p_logits, const int32_t* drafts,
                                   int K, int V, double T, int top_k, double top_p, uint64_t seed, uint32_t b, uint32_t s,
                                   int32_t* out_tokens, int32_t* n_accepted, uint32_t* flags,
                                   double* beta) {
  Filt f; f.top_k = top_k; f.top_p = top_p;
  accept_chain_impl(q_logits, p_logits, drafts, K, V, T, f, seed, b, s, out_tokens, n_accepted, flags, beta);
}

// The same chain with the WRONG resampling rule (draw from q_t instead of the
// residual).  Its law is min(p,q) + (1-beta) q != q.  It exists only as the
// negative control that shows the distribution tests have power.
extern "C" void orc_accept_chain_wrong(const float* q_logits, const float* p_logits, const int32_t* drafts,
                                       int K, int V, double T, uint64_t seed, uint32_t b, uint32_t s,
                                       int32_t* out_tokens, int32_t* n_accepted) {
  std::vector<double> q, p;
  int a = 0;
  for (int i = 0; i <= K; ++i) out_tokens[i] = -1;
  for (int t = 0; t <= K; ++t) {
    double u[3];
    orc_uniforms(seed, b, s, (uint32_t)t, u);
    softmax_T(q_logits + (size_t)t * V, V, T, q);
    if (t < K) {
      softmax_T(p_logits + (size_t)t * V, V, T, p);
      const int d = drafts[t];
      const double ratio = p[d] > 0.0 ? std::min(1.0, q[d] / p[d]) : (q[d] > 0.0 ? 1.0 : 0.0);
      if (u[1] < ratio) { out_tokens[a++] = d; continue; }
    }
    out_tokens[a] = invcdf(q.data(), V, u[2], nullptr);
    break;
  }
  *n_accepted = a;
}

// ---------------------------------------------------------------------------
// Models.  A model maps rows (token, absolute position) to next-token logits,
// conditioning each row on every position before it (section "Conditional
// Scoring": K+1 sets of logits from one call equal the K+1 sequential ones).
// ---------------------------------------------------------------------------
struct OrcModel {
  int V = 0;
  virtual ~OrcModel() {}
  // logits may be null (prefill: only the cache is wanted)
  virtual void forward(const int32_t* tokens, const int32_t* positions, int M, float* logits) = 0;
};

// --- a lookup-table model for tiny vocabularies (used by the distribution pins).
// depth 0: context-free, logits depend on the absolute position only
//          (table [n_pos][V], row = position - pos0, clamped);
// depth D>0: logits depend on the last min(D, position - pos0 + 1) tokens after
//          the prompt; contexts longer than D use the last D tokens.
struct TableModel : OrcModel {
  int depth = 0, pos0 = 0, n_rows = 0;
  std::vector<float> table;
  std::vector<int32_t> seq;
  size_t ctx_index(int pos) const {
    // suffix after the prompt: tokens at positions pos0 .. pos  (length L = pos - pos0 + 1)
    int L = pos - pos0 + 1;
    if (L < 0) L = 0;
    if (L > depth) L = depth;
    // index of a length-L context: offset(L) + base-V number of the tokens
    size_t off = 0, pw = 1;
    for (int l = 0; l < L; ++l) { off += pw; pw *= (size_t)V; }
    size_t num = 0;
    for (int i = pos - L + 1; i <= pos; ++i) num = num * (size_t)V + (size_t)seq[i];
    return off + num;
  }
  void forward(const int32_t* tokens, const int32_t* positions, int M, float* logits) override {
    for (int m = 0; m < M; ++m) {
      const int pos = positions[m];
      if ((int)seq.size() <= pos) seq.resize(pos + 1, 0);
      seq[pos] = tokens[m];
      if (!logits) continue;
      size_t row;
      if (depth == 0) {
        int r = pos - pos0; if (r < 0) r = 0; if (r >= n_rows) r = n_rows - 1;
        row = (size_t)r;
      } else {
        row = ctx_index(pos);
      }
      std::memcpy(logits + (size_t)m * V, table.data() + row * V, sizeof(float) * V);
    }
  }
};

extern "C" OrcModel* orc_table_model_create(const float* table, int n_rows, int V, int depth, int pos0) {
  TableModel* m = new TableModel();
  m->V = V; m->depth = depth; m->pos0 = pos0; m->n_rows = n_rows;
  m->table.assign(table, table + (size_t)n_rows * V);
  return m;
}

// --- the transformer -------------------------------------------------------
// The paper fixes only d_model / heads / layers (Hyperparams table).  This
// build's reading: pre-RMSNorm decoder, multi-head attention with
// n_heads * d_head == d_model, rotary positions on adjacent pairs over the
// whole head, non-gated FFN with tanh-GeLU, no biases, untied (un)embedding.
struct TfLayer { const void *attn_norm, *ffn_norm, *wq, *wk, *wv, *wo, *w_up, *w_down; };

static inline double load_w(const void* base, size_t i, int dtype) {
  if (dtype == 0) return (double)((const float*)base)[i];
  uint32_t bits = (uint32_t)((const uint16_t*)base)[i] << 16;  // bf16 -> fp32, exact
  float f; std::memcpy(&f, &bits, 4);
  return (double)f;
}

// value as it is held in the KV cache (storage rounding is part of the model)
static inline float round_storage(double x, int dtype) {
  if (dtype == 0) return (float)x;
  if (x == 0.0 || !std::isfinite(x)) return (float)x;
  int e; std::frexp(x, &e);                 // |x| = m * 2^e, 0.5 <= m < 1
  const double quantum = std::ldexp(1.0, e - 8);   // bf16 keeps 8 significant bits
  return (float)(std::nearbyint(x / quantum) * quantum);  // round to nearest even
}

struct Transformer : OrcModel {
  int L = 0, d = 0, H = 0, dh = 0, dff = 0, dtype = 0, max_seq = 0;
  int Hkv = 0;           // key / value heads; query head h reads key / value head h / (H / Hkv)  (Hkv = H: one each)
  int cache_dtype = 0;   // storage type of cached keys / values; differs from the weights' for int8-weight models
  double eps = 1e-5, rope_base = 10000.0;
  const void *tok_embed = nullptr, *unembed = nullptr, *final_norm = nullptr;
  std::vector<TfLayer> layers;
  std::vector<float> kc, vc;  // [L][max_seq][Hkv * dh]
  // state of a layer-by-layer pass
  std::vector<double> x;      // [M][d]
  std::vector<int32_t> pos;
  int M = 0;

  // y[n] = sum_k W[n][k] v[k],  W row-major [N][D]
  void matvec(const void* W, const double* v, int N, int D, double* y) const {
    const int dt = dtype;
    parallel_rows(N, D, [=](int n0, int n1) {
      for (int n = n0; n < n1; ++n) {
        double acc = 0.0;
        const size_t base = (size_t)n * D;
        for (int k = 0; k < D; ++k) acc += load_w(W, base + k, dt) * v[k];
        y[n] = acc;
      }
    });
  }
  void rmsnorm(const double* v, const void* gain, double* out) const {
    double ss = 0.0;
    for (int j = 0; j < d; ++j) ss += v[j] * v[j];
    const double inv = 1.0 / std::sqrt(ss / d + eps);
    for (int j = 0; j < d; ++j) out[j] = (double)((const float*)gain)[j] * v[j] * inv;
  }
  static double gelu(double v) {
    return 0.5 * v * (1.0 + std::tanh(0.7978845608028654 * (v + 0.044715 * v * v * v)));
  }

  void begin(const int32_t* tokens, const int32_t* positions, int M_) {
    M = M_;
    x.assign((size_t)M * d, 0.0);
    pos.assign(positions, positions + M);
    for (int m = 0; m < M; ++m)
      for (int j = 0; j < d; ++j) x[(size_t)m * d + j] = load_w(tok_embed, (size_t)tokens[m] * d + j, dtype);
  }
  void begin_rows(const void* emb_rows, const int32_t* positions, int M_) {
    M = M_;
    x.assign((size_t)M * d, 0.0);
    pos.assign(positions, positions + M);
    for (size_t i = 0; i < (size_t)M * d; ++i) x[i] = load_w(emb_rows, i, dtype);
  }
  void layer(int l, const TfLayer& w) {
    const int dkv = Hkv * dh, group = H / Hkv;
    std::vector<double> h(d), qv(d), kv(dkv), vv(dkv), o(d), y(d), up(dff);
    float* kcl = kc.data() + (size_t)l * max_seq * dkv;
    float* vcl = vc.data() + (size_t)l * max_seq * dkv;
    // rows go in order, so row i sees the cache rows of rows <= i (in-block causality)
    for (int m = 0; m < M; ++m) {
      double* xm = x.data() + (size_t)m * d;
      const int p = pos[m];
      rmsnorm(xm, w.attn_norm, h.data());
      matvec(w.wq, h.data(), d, d, qv.data());
      matvec(w.wk, h.data(), dkv, d, kv.data());
      matvec(w.wv, h.data(), dkv, d, vv.data());
      for (int hd = 0; hd < H; ++hd) {
        for (int i = 0; i < dh / 2; ++i) {
          const double ang = (double)p * std::pow(rope_base, -2.0 * i / dh);
          const double c = std::cos(ang), s = std::sin(ang);
          double* a = qv.data() + hd * dh + 2 * i;
          double a0 = a[0], a1 = a[1];
          a[0] = a0 * c - a1 * s; a[1] = a0 * s + a1 * c;
          if (hd >= Hkv) continue;
          double* bb = kv.data() + hd * dh + 2 * i;
          a0 = bb[0]; a1 = bb[1];
          bb[0] = a0 * c - a1 * s; bb[1] = a0 * s + a1 * c;
        }
      }
      for (int j = 0; j < dkv; ++j) {
        kcl[(size_t)p * dkv + j] = round_storage(kv[j], cache_dtype);
        vcl[(size_t)p * dkv + j] = round_storage(vv[j], cache_dtype);
      }
      const double scale = 1.0 / std::sqrt((double)dh);
      for (int hd = 0; hd < H; ++hd) {
        const int hk = hd / group;   // the key / value head this query head shares
        std::vector<double> sc(p + 1);
        double mx = -INFINITY;
        for (int j = 0; j <= p; ++j) {
          double acc = 0.0;
          for (int i = 0; i < dh; ++i) acc += qv[hd * dh + i] * (double)kcl[(size_t)j * dkv + hk * dh + i];
          sc[j] = acc * scale;
          mx = std::max(mx, sc[j]);
        }
        double sum = 0.0;
        for (int j = 0; j <= p; ++j) { sc[j] = std::exp(sc[j] - mx); sum += sc[j]; }
        for (int i = 0; i < dh; ++i) {
          double acc = 0.0;
          for (int j = 0; j <= p; ++j) acc += sc[j] * (double)vcl[(size_t)j * dkv + hk * dh + i];
          o[hd * dh + i] = acc / sum;
        }
      }
      matvec(w.wo, o.data(), d, d, y.data());
      for (int j = 0; j < d; ++j) xm[j] += y[j];
      rmsnorm(xm, w.ffn_norm, h.data());
      matvec(w.w_up, h.data(), dff, d, up.data());
      for (int j = 0; j < dff; ++j) up[j] = gelu(up[j]);
      matvec(w.w_down, up.data(), d, dff, y.data());
      for (int j = 0; j < d; ++j) xm[j] += y[j];
    }
  }
  void end(float* logits, double* logits64) {
    std::vector<double> h(d), lg(V);
    for (int m = 0; m < M; ++m) {
      rmsnorm(x.data() + (size_t)m * d, final_norm, h.data());
      matvec(unembed, h.data(), V, d, lg.data());
      if (logits) for (int v = 0; v < V; ++v) logits[(size_t)m * V + v] = (float)lg[v];
      if (logits64) for (int v = 0; v < V; ++v) logits64[(size_t)m * V + v] = lg[v];
    }
  }
  void forward(const int32_t* tokens, const int32_t* positions, int M_, float* logits) override {
    begin(tokens, positions, M_);
    for (int l = 0; l < L; ++l) layer(l, layers[l]);
    if (logits) end(logits, nullptr);
  }
};

extern "C" OrcModel* orc_tf_create(int n_layers, int d_model, int n_heads, int d_head, int d_ff, int vocab,
                                   int dtype, double rms_eps, double rope_base, int max_seq) {
  if (n_heads * d_head != d_model || (d_head & 1)) return nullptr;
  Transformer* t = new Transformer();
  t->L = n_layers; t->d = d_model; t->H = n_heads; t->Hkv = n_heads; t->dh = d_head; t->dff = d_ff; t->V = vocab;
  t->dtype = dtype; t->cache_dtype = dtype; t->eps = rms_eps; t->rope_base = rope_base; t->max_seq = max_seq;
  t->layers.resize(n_layers);
  t->kc.assign((size_t)n_layers * max_seq * d_model, 0.f);
  t->vc.assign((size_t)n_layers * max_seq * d_model, 0.f);
  return t;
}
// fewer key / value heads than query heads (multi-query: 1; grouped: a divisor of n_heads); call before any pass
extern "C" int orc_tf_set_kv_heads(OrcModel* m, int n_kv_heads) {
  Transformer* t = static_cast<Transformer*>(m);
  if (n_kv_heads < 1 || t->H % n_kv_heads) return -1;
  t->Hkv = n_kv_heads;
  t->kc.assign((size_t)t->L * t->max_seq * n_kv_heads * t->dh, 0.f);
  t->vc.assign((size_t)t->L * t->max_seq * n_kv_heads * t->dh, 0.f);
  return 0;
}
extern "C" void orc_tf_set_cache_dtype(OrcModel* m, int cache_dtype) { static_cast<Transformer*>(m)->cache_dtype = cache_dtype; }
extern "C" void orc_tf_set_globals(OrcModel* m, const void* tok_embed, const void* unembed, const void* final_norm) {
  Transformer* t = static_cast<Transformer*>(m);
  t->tok_embed = tok_embed; t->unembed = unembed; t->final_norm = final_norm;
}
extern "C" void orc_tf_set_layer(OrcModel* m, int l, const void* attn_norm, const void* ffn_norm, const void* wq,
                                 const void* wk, const void* wv, const void* wo, const void* w_up,
                                 const void* w_down) {
  Transformer* t = static_cast<Transformer*>(m);
  t->layers[l] = TfLayer{attn_norm, ffn_norm, wq, wk, wv, wo, w_up, w_down};
}
// layer-by-layer pass: lets a caller hold one layer's weights at a time
extern "C" void orc_tf_begin_rows(OrcModel* m, const void* emb_rows, const int32_t* positions, int M) {
  static_cast<Transformer*>(m)->begin_rows(emb_rows, positions, M);
}
extern "C" void orc_tf_layer(OrcModel* m, int l, const void* attn_norm, const void* ffn_norm, const void* wq,
                             const void* wk, const void* wv, const void* wo, const void* w_up,
                             const void* w_down) {
  static_cast<Transformer*>(m)->layer(l, TfLayer{attn_norm, ffn_norm, wq, wk, wv, wo, w_up, w_down});
}
extern "C" void orc_tf_end(OrcModel* m, const void* final_norm, const void* unembed, float* logits, double* logits64) {
  Transformer* t = static_cast<Transformer*>(m);
  t->final_norm = final_norm; t->unembed = unembed;
  t->end(logits, logits64);
}
// the residual stream after the layers applied so far, [M][d]
extern "C" void orc_tf_hidden(OrcModel* m, double* out) {
  Transformer* t = static_cast<Transformer*>(m);
  std::memcpy(out, t->x.data(), sizeof(double) * t->x.size());
}
// cached keys / values of one layer at one position, [n_kv_heads * d_head] each
extern "C" void orc_tf_kv(OrcModel* m, int l, int position, float* k_out, float* v_out) {
  Transformer* t = static_cast<Transformer*>(m);
  const size_t dkv = (size_t)t->Hkv * t->dh;
  std::memcpy(k_out, t->kc.data() + ((size_t)l * t->max_seq + position) * dkv, sizeof(float) * dkv);
  std::memcpy(v_out, t->vc.data() + ((size_t)l * t->max_seq + position) * dkv, sizeof(float) * dkv);
}
extern "C" void orc_model_forward(OrcModel* m, const int32_t* tokens, const int32_t* positions, int M,
                                  float* logits) {
  m->forward(tokens, positions, M, logits);
}
extern "C" void orc_model_forward64(OrcModel* m, const int32_t* tokens, const int32_t* positions, int M,
                                    double* logits64) {
  Transformer* t = static_cast<Transformer*>(m);
  t->begin(tokens, positions, M);
  for (int l = 0; l < t->L; ++l) t->layer(l, t->layers[l]);
  t->end(nullptr, logits64);
}
extern "C" int orc_model_vocab(OrcModel* m) { return m->V; }
extern "C" void orc_model_destroy(OrcModel* m) { delete m; }

// ---------------------------------------------------------------------------
// The sampling loops.
// ---------------------------------------------------------------------------
struct OrcSps {
  OrcModel* target = nullptr;
  OrcModel* draft = nullptr;
  std::vector<int32_t> x;  // the sequence so far, x[0..n-1]
  int tlen = 0;            // target cache holds positions 0..tlen-1
  int dlen = 0;            // draft cache holds positions 0..dlen-1
  int V = 0;
  // what the last loop saw (for element-wise comparison with another implementation)
  std::vector<float> last_q, last_p;
  std::vector<int32_t> last_drafts;
  Filt filt;               // top-k / nucleus applied to both models' distributions
};

extern "C" OrcSps* orc_sps_create(OrcModel* target, OrcModel* draft) {
  OrcSps* c = new OrcSps();
  c->target = target; c->draft = draft; c->V = target->V;
  return c;
}
extern "C" void orc_sps_destroy(OrcSps* c) { delete c; }
extern "C" void orc_sps_set_sampling(OrcSps* c, int top_k, double top_p) { c->filt.top_k = top_k; c->filt.top_p = top_p; }

// Start from a prompt x_0..x_{P-1}: both caches take positions 0..P-2, so that
// the first loop feeds x_{P-1} (n = P).
extern "C" void orc_sps_reset(OrcSps* c, const int32_t* prompt, int P) {
  c->x.assign(prompt, prompt + P);
  std::vector<int32_t> pos(P);
  for (int i = 0; i < P; ++i) pos[i] = i;
  if (P > 1) {
    c->target->forward(prompt, pos.data(), P - 1, nullptr);
    if (c->draft) c->draft->forward(prompt, pos.data(), P - 1, nullptr);
  }
  c->tlen = P - 1; c->dlen = P - 1;
}
extern "C" int orc_sps_len(OrcSps* c) { return (int)c->x.size(); }
extern "C" void orc_sps_tokens(OrcSps* c, int32_t* out) { std::memcpy(out, c->x.data(), 4 * c->x.size()); }
extern "C" void orc_sps_last_logits(OrcSps* c, float* q_out, float* p_out, int32_t* drafts_out) {
  if (q_out) std::memcpy(q_out, c->last_q.data(), 4 * c->last_q.size());
  if (p_out && !c->last_p.empty()) std::memcpy(p_out, c->last_p.data(), 4 * c->last_p.size());
  if (drafts_out && !c->last_drafts.empty()) std::memcpy(drafts_out, c->last_drafts.data(), 4 * c->last_drafts.size());
}

// One iteration of Algorithm 2's while-loop (K >= 1), or of Algorithm 1's (K == 0).
// n is frozen at loop entry; accepted draft t lands at position n + t; n
// advances once, by n_accepted + 1, at the end.
// Returns the number of tokens emitted (n_accepted + 1) and writes them.
extern "C" int orc_sps_loop(OrcSps* c, int K, double T, uint64_t seed, uint32_t b, uint32_t s,
                            int32_t* out_tokens /*[K+1]*/, int32_t* n_accepted, uint32_t* flags,
                            uint32_t* draft_near_tie /* bit t set: draft draw t fell in a CDF edge band */) {
  const int V = c->V;
  const int n = (int)c->x.size();
  std::vector<int32_t> d(K);
  c->last_p.assign((size_t)K * V, 0.f);
  c->last_q.assign((size_t)(K + 1) * V, 0.f);
  uint32_t dnt = 0;
  // --- draft auto-regressively: d_t ~ p(. | x_0..x_{n-1}, d_0..d_{t-1})
  for (int t = 0; t < K; ++t) {
    // feed every token the draft has not cached yet, up to the newest one
    std::vector<int32_t> tok, pos;
    for (int i = c->dlen; i <= n - 1 + t; ++i) {
      tok.push_back(i < n ? c->x[i] : d[i - n]);
      pos.push_back(i);
    }
    std::vector<float> lg((size_t)tok.size() * V);
    c->draft->forward(tok.data(), pos.data(), (int)tok.size(), lg.data());
    c->dlen = n + t;
    const float* last = lg.data() + (size_t)(tok.size() - 1) * V;
    std::memcpy(c->last_p.data() + (size_t)t * V, last, sizeof(float) * V);
    double u[3];
    orc_uniforms(seed, b, s, (uint32_t)t, u);
    int nt = 0;
    d[t] = orc_sample_row_f(last, V, T, c->filt.top_k, c->filt.top_p, u[0], &nt);
    if (nt) dnt |= (1u << t);
  }
  // --- score: K+1 sets of target logits in one call over [x_{n-1}, d_0..d_{K-1}]
  {
    std::vector<int32_t> tok(K + 1), pos(K + 1);
    tok[0] = c->x[n - 1]; pos[0] = n - 1;
    for (int t = 0; t < K; ++t) { tok[t + 1] = d[t]; pos[t + 1] = n + t; }
    c->target->forward(tok.data(), pos.data(), K + 1, c->last_q.data());
  }
  c->last_drafts = d;
  // --- accept from left to right, resample or draw the extra token
  int a = 0;
  uint32_t fl = 0;
  accept_chain_impl(c->last_q.data(), c->last_p.data(), d.data(), K, V, T, c->filt, seed, b, s, out_tokens, &a, &fl, nullptr);
  for (int i = 0; i <= a; ++i) c->x.push_back(out_tokens[i]);
  // --- caches: nothing is undone, only the valid lengths move
  c->tlen = n + a;
  if (K > 0) c->dlen = std::min(n + a, n + K - 1);
  *n_accepted = a;
  *flags = fl;
  if (draft_near_tie) *draft_near_tie = dnt;
  return a + 1;
}

// Run loops until n_new tokens exist after the prompt; the last loop may
// overshoot and is truncated (T is a minimum length in Algorithm 2).
// loops_out: number of loops; hist_emitted[K+2]: how many loops emitted j tokens.
extern "C" int orc_sps_generate(OrcSps* c, const int32_t* prompt, int P, int n_new, int K, double T,
                                uint64_t seed, uint32_t b, uint32_t step0, int32_t* out_tokens,
                                int32_t* loops_out, int32_t* hist_emitted, uint32_t* any_flags) {
  orc_sps_reset(c, prompt, P);
  std::vector<int32_t> em(K + 1);
  int made = 0, loops = 0;
  uint32_t anyf = 0;
  if (hist_emitted) for (int i = 0; i < K + 2; ++i) hist_emitted[i] = 0;
  while (made < n_new) {
    int a; uint32_t fl, dnt;
    const int e = orc_sps_loop(c, K, T, seed, b, step0 + (uint32_t)loops, em.data(), &a, &fl, &dnt);
    if (hist_emitted) hist_emitted[e]++;
    anyf |= fl | (dnt ? ORC_NEAR_CDF : 0u);
    for (int i = 0; i < e && made < n_new; ++i) out_tokens[made++] = em[i];
    ++loops;
  }
  if (loops_out) *loops_out = loops;
  if (any_flags) *any_flags = anyf;
  return made;
}

// Adaptive lookahead.  The paper finds that the best K depends on the domain (the K trade-off figure and its
// discussion) and fixes K per experiment; choosing it on the fly is this build's addition.  The rule: K starts
// at (K_min + K_max) / 2; after a
// loop in which every draft was accepted it grows by one (up to K_max), after a loop in which the first draft
// was rejected it shrinks by one (down to K_min), otherwise it stays.  K only depends on the past, so every
// loop is still an exact iteration of Algorithm 2 and the output law is unchanged (Theorem 1 per loop).
static int next_K(int K, int accepted, int K_min, int K_max) {
  if (accepted == K) return std::min(K + 1, K_max);
  if (accepted == 0) return std::max(K - 1, K_min);
  return K;
}

extern "C" int orc_sps_generate_adaptive(OrcSps* c, const int32_t* prompt, int P, int n_new, int K_min, int K_max, double T,
                                         uint64_t seed, uint32_t b, uint32_t step0, int32_t* out_tokens,
                                         int32_t* loops_out, int32_t* draft_calls_out, uint32_t* any_flags) {
  orc_sps_reset(c, prompt, P);
  std::vector<int32_t> em(K_max + 1);
  int made = 0, loops = 0, K = (K_min + K_max) / 2, drafts = 0;
  uint32_t anyf = 0;
  while (made < n_new) {
    int a; uint32_t fl, dnt;
    const int e = orc_sps_loop(c, K, T, seed, b, step0 + (uint32_t)loops, em.data(), &a, &fl, &dnt);
    anyf |= fl | (dnt ? ORC_NEAR_CDF : 0u);
    for (int i = 0; i < e && made < n_new; ++i) out_tokens[made++] = em[i];
    drafts += K;
    K = next_K(K, a, K_min, K_max);
    ++loops;
  }
  if (loops_out) *loops_out = loops;
  if (draft_calls_out) *draft_calls_out = drafts;
  if (any_flags) *any_flags = anyf;
  return made;
}

// n_trials independent adaptive generations (trial i uses sequence index b0 + i); table models
extern "C" void orc_sps_trials_adaptive(OrcModel* target, OrcModel* draft, const int32_t* prompt, int P, int n_new,
                                        int K_min, int K_max, double T, uint64_t seed, uint32_t b0, int64_t n_trials,
                                        int32_t* out_tokens /*[n_trials][n_new]*/, int64_t* draft_calls_total) {
  OrcSps* c = orc_sps_create(target, draft);
  int64_t tot = 0;
  for (int64_t tr = 0; tr < n_trials; ++tr) {
    int32_t dc = 0;
    orc_sps_generate_adaptive(c, prompt, P, n_new, K_min, K_max, T, seed, b0 + (uint32_t)tr, 0u, out_tokens + tr * n_new,
                              nullptr, &dc, nullptr);
    tot += dc;
  }
  if (draft_calls_total) *draft_calls_total = tot;
  orc_sps_destroy(c);
}

// Many independent trials of "the first n_new tokens after a fixed prompt",
// trial i using sequence index b0 + i (so each trial has its own uniforms).
// Meant for table models, where a forward costs nothing.  wrong_rule != 0
// swaps in the negative-control chain.
static void sps_trials_impl(OrcModel* target, OrcModel* draft, const int32_t* prompt, int P, int n_new, int K,
                            double T, const Filt& filt, uint64_t seed, uint32_t b0, int64_t n_trials, int wrong_rule,
                            int32_t* out_tokens /*[n_trials][n_new]*/, int64_t* emitted_hist /*[K+2]*/,
                            int32_t* first_n_accepted /*[n_trials] or null*/,
                            uint32_t* first_flags /*[n_trials] or null*/,
                            uint32_t* all_flags = nullptr /*[n_trials] or null: flags of every loop of the trial, OR-ed,
                                                            a draft draw's near tie counted as ORC_NEAR_CDF*/) {
  const int V = target->V;
  for (int i = 0; i < K + 2; ++i) emitted_hist[i] = 0;
  OrcSps* c = orc_sps_create(target, draft);
  c->filt = filt;
  std::vector<int32_t> em(K + 1), d(K);
  for (int64_t tr = 0; tr < n_trials; ++tr) {
    const uint32_t b = b0 + (uint32_t)tr;
    int32_t* out = out_tokens + tr * n_new;
    if (!wrong_rule) {
      orc_sps_reset(c, prompt, P);
      int made = 0; uint32_t s = 0;
      if (all_flags) all_flags[tr] = 0u;
      while (made < n_new) {
        int a; uint32_t fl, dnt = 0;
        const int e = orc_sps_loop(c, K, T, seed, b, s, em.data(), &a, &fl, &dnt);
        if (s == 0 && first_n_accepted) first_n_accepted[tr] = a;
        if (s == 0 && first_flags) first_flags[tr] = fl;
        if (all_flags) all_flags[tr] |= fl | (dnt ? ORC_NEAR_CDF : 0u);
        ++s;
        emitted_hist[e]++;
        for (int i = 0; i < e && made < n_new; ++i) out[made++] = em[i];
      }
    } else {
      // same loop, wrong chain (negative control only)
      orc_sps_reset(c, prompt, P);
      int made = 0; uint32_t s = 0;
      std::vector<float> pl((size_t)K * V), ql((size_t)(K + 1) * V);
      while (made < n_new) {
        const int n = (int)c->x.size();
        for (int t = 0; t < K; ++t) {
          std::vector<int32_t> tok, pos;
          for (int i = c->dlen; i <= n - 1 + t; ++i) { tok.push_back(i < n ? c->x[i] : d[i - n]); pos.push_back(i); }
          std::vector<float> lg((size_t)tok.size() * V);
          draft->forward(tok.data(), pos.data(), (int)tok.size(), lg.data());
          c->dlen = n + t;
          std::memcpy(pl.data() + (size_t)t * V, lg.data() + (size_t)(tok.size() - 1) * V, 4 * V);
          double u[3]; orc_uniforms(seed, b, s, (uint32_t)t, u);
          d[t] = orc_sample_row(pl.data() + (size_t)t * V, V, T, u[0], nullptr);
        }
        std::vector<int32_t> tok(K + 1), pos(K + 1);
        tok[0] = c->x[n - 1]; pos[0] = n - 1;
        for (int t = 0; t < K; ++t) { tok[t + 1] = d[t]; pos[t + 1] = n + t; }
        target->forward(tok.data(), pos.data(), K + 1, ql.data());
        int a;
        orc_accept_chain_wrong(ql.data(), pl.data(), d.data(), K, V, T, seed, b, s, em.data(), &a);
        for (int i = 0; i <= a; ++i) c->x.push_back(em[i]);
        c->tlen = n + a;
        if (K > 0) c->dlen = std::min(n + a, n + K - 1);
        for (int i = 0; i <= a && made < n_new; ++i) out[made++] = em[i];
        ++s;
      }
    }
  }
  orc_sps_destroy(c);
}

extern "C" void orc_sps_trials(OrcModel* target, OrcModel* draft, const int32_t* prompt, int P, int n_new, int K,
                               double T, uint64_t seed, uint32_t b0, int64_t n_trials, int wrong_rule,
                               int32_t* out_tokens, int64_t* emitted_hist, int32_t* first_n_accepted, uint32_t* first_flags) {
  sps_trials_impl(target, draft, prompt, P, n_new, K, T, Filt(), seed, b0, n_trials, wrong_rule, out_tokens, emitted_hist,
                  first_n_accepted, first_flags);
}
// the same trials, also reporting per trial the flags of all its loops (which trials another implementation may
// legitimately decide differently)
extern "C" void orc_sps_trials_flagged(OrcModel* target, OrcModel* draft, const int32_t* prompt, int P, int n_new, int K,
                                       double T, uint64_t seed, uint32_t b0, int64_t n_trials, int32_t* out_tokens,
                                       int64_t* emitted_hist, uint32_t* all_flags) {
  sps_trials_impl(target, draft, prompt, P, n_new, K, T, Filt(), seed, b0, n_trials, 0, out_tokens, emitted_hist, nullptr, nullptr,
                  all_flags);
}
// the same with top-k / nucleus filtering of both models (not with the negative-control chain)
extern "C" void orc_sps_trials_f(OrcModel* target, OrcModel* draft, const int32_t* prompt, int P, int n_new, int K,
                                 double T, int top_k, double top_p, uint64_t seed, uint32_t b0, int64_t n_trials,
                                 int32_t* out_tokens, int64_t* emitted_hist, int32_t* first_n_accepted, uint32_t* first_flags) {
  Filt f; f.top_k = top_k; f.top_p = top_p;
  sps_trials_impl(target, draft, prompt, P, n_new, K, T, f, seed, b0, n_trials, 0, out_tokens, emitted_hist,
                  first_n_accepted, first_flags);
}

// Y[m][n] = sum_k X[m][k] W[n][k]: the linear layer by its definition, in double.
extern "C" void orc_linear(const void* W, int dtype, const float* X, int M, int N, int D, double* Y) {
  parallel_rows(N, (long long)D * M, [=](int n0, int n1) {
    for (int n = n0; n < n1; ++n)
      for (int m = 0; m < M; ++m) {
        double acc = 0.0;
        for (int k = 0; k < D; ++k) acc += load_w(W, (size_t)n * D + k, dtype) * (double)X[(size_t)m * D + k];
        Y[(size_t)m * N + n] = acc;
      }
  });
}

extern "C" int orc_num_threads() { return hw_threads(); }
// Test hook: n > 0 makes every later call split its rows over n threads (1 = the calling thread only), 0 goes
// back to the machine's count.  The arithmetic of a row does not depend on which thread runs it, so results
// must be identical for every n; a test checks exactly that.
extern "C" void orc_set_threads(int n) { g_threads_override = n > 64 ? 64 : n; }
// The inverse-CDF draw on given unnormalised weights (the "Sample" of Algorithms 1 and 2 under this build's
// reading), exposed so that its two degenerate exits can be pinned directly.
extern "C" int orc_invcdf(const double* w, int V, double u, int* near_tie) { return invcdf(w, V, u, near_tie); }
