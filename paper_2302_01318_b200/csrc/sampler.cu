// Sampling kernels: the inverse-CDF draw used for draft tokens, and the fused modified rejection
// sampler of Algorithm 2 (accept test, residual resample, extra token) -- one CTA per sequence,
// warp shuffles plus a block prefix sum over the vocabulary.
#include <limits.h>

#include <algorithm>
#include <cstdlib>

#include "common.cuh"

#define SAMPLER_THREADS 1024
#define SAMPLER_WARPS (SAMPLER_THREADS / 32)

struct ScanSmem {
  float warp_part[SAMPLER_WARPS];
  float total;
  int ired[SAMPLER_WARPS];
  int ires;
};

__device__ inline int block_min_int(int v, ScanSmem& sm) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  v = warp_min_int(v);
  __syncthreads();
  if (lane == 0) sm.ired[warp] = v;
  __syncthreads();
  if (warp == 0) {
    int x = (lane < (int)(blockDim.x >> 5)) ? sm.ired[lane] : INT_MAX;
    x = warp_min_int(x);
    if (lane == 0) sm.ires = x;
  }
  __syncthreads();
  return sm.ires;
}
__device__ inline int block_max_int(int v, ScanSmem& sm) { return -block_min_int(-v, sm); }

// Inverse-CDF draw in index order on unnormalised weights w(0..V-1): the smallest i whose inclusive
// running sum exceeds u * total; if rounding leaves none, the largest i with w(i) > 0.
// Thread t owns the contiguous chunk [t*c, (t+1)*c); chunk sums are combined by a warp scan and a
// scan of the warp totals, so the result does not depend on timing.  Returns the token to all threads.
template <class F>
__device__ int block_invcdf(F w, int V, float u, ScanSmem& sm, float* total_out) {
  const int tid = threadIdx.x, nt = blockDim.x, lane = tid & 31, warp = tid >> 5;
  const int chunk = (V + nt - 1) / nt;
  const int i0 = min(tid * chunk, V), i1 = min(i0 + chunk, V);
  float local = 0.f;
  for (int i = i0; i < i1; ++i) local += w(i);
  float incl = local;
#pragma unroll
  for (int o = 1; o < 32; o <<= 1) {
    const float v = __shfl_up_sync(0xffffffffu, incl, o);
    if (lane >= o) incl += v;
  }
  __syncthreads();
  if (lane == 31) sm.warp_part[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    const int nw = nt >> 5;
    const float v = (lane < nw) ? sm.warp_part[lane] : 0.f;
    float iv = v;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const float x = __shfl_up_sync(0xffffffffu, iv, o);
      if (lane >= o) iv += x;
    }
    if (lane < nw) sm.warp_part[lane] = iv - v;  // exclusive prefix of the warp
    if (lane == nw - 1) sm.total = iv;
  }
  __syncthreads();
  const float pre = sm.warp_part[warp] + (incl - local);
  const float total = sm.total;
  if (total_out) *total_out = total;
  const float target = u * total;
  int cand = INT_MAX;
  float c = pre;
  for (int i = i0; i < i1; ++i) {
    c += w(i);
    if (c > target) { cand = i; break; }
  }
  int tok = block_min_int(cand, sm);
  if (tok == INT_MAX) {
    int last = -1;
    for (int i = i0; i < i1; ++i) if (w(i) > 0.f) last = i;
    tok = block_max_int(last, sm);
    if (tok < 0) tok = V - 1;
  }
  return tok;
}

// Same draw when the weights already sit in shared memory (written once with coalesced global loads).
// Element i lives at ws[i + (i >> 5)]: the one-word skew per 32 elements makes the chunk-order reads
// (thread t walks i = t*c .. t*c + c - 1) conflict-free.
__device__ __forceinline__ int skew(int i) { return i + (i >> 5); }
__device__ int block_invcdf_smem(const float* ws, int V, float u, ScanSmem& sm, float* total_out) {
  auto w = [&](int i) { return ws[skew(i)]; };
  return block_invcdf(w, V, u, sm, total_out);
}

__device__ inline float block_max_f(float v, float* s_part, float* s_out) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  v = warp_max(v);
  __syncthreads();
  if (lane == 0) s_part[warp] = v;
  __syncthreads();
  if (warp == 0) {
    float x = (lane < (int)(blockDim.x >> 5)) ? s_part[lane] : -INFINITY;
    x = warp_max(x);
    if (lane == 0) *s_out = x;
  }
  __syncthreads();
  return *s_out;
}
__device__ inline float block_sum_f(float v, float* s_part, float* s_out) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  v = warp_sum(v);
  __syncthreads();
  if (lane == 0) s_part[warp] = v;
  __syncthreads();
  if (warp == 0) {
    float x = (lane < (int)(blockDim.x >> 5)) ? s_part[lane] : 0.f;
    x = warp_sum(x);
    if (lane == 0) *s_out = x;
  }
  __syncthreads();
  return *s_out;
}

// ------------------------------------------------------------------------------------------------
// Top-k and nucleus filtering.  The section Modified Rejection Sampling says that nucleus, top-k and
// temperature are handled by changing the probabilities first and running the rejection scheme on the
// changed distributions; it gives no formulas.  Here a row keeps every token whose logit is at least a cut:
//   top-k   : the cut is the k-th largest logit (tokens tied with it stay);
//   nucleus : over what top-k kept, mass Z_k, the largest logit value v such that the tokens with logit
//             >= v hold at least top_p * Z_k.
// Both are "the largest key whose upper tail reaches a target", the key being the order-preserving bit
// pattern of the fp32 logit and the tail a token count (top-k) or a weight mass (nucleus).  The key is
// built from its top bit down, two bits per step: the block evaluates the tail at the three candidate
// keys and keeps the largest that still reaches the target.  No sort, no atomics: a thread holds the keys
// of its 32 tokens (tid, tid + 1024, ...) in registers, the weights sit in shared memory, and every sum
// runs in a fixed order (thread, warp butterfly, butterfly over the warps), so results are reproducible.
// (A radix descent with shared-memory histograms was 5-10 times slower: the digits of real logits fall in
// a handful of bins and the adds to them serialise.)
// ------------------------------------------------------------------------------------------------
#define CUT_ELEMS 32   // tokens per thread held in registers: rows up to 32 * 1024 tokens
struct CutSmem {
  float f[2][3][SAMPLER_WARPS];
  int i[2][3][SAMPLER_WARPS];
};

__device__ __forceinline__ uint32_t order_key(float f) {   // unsigned order of keys == order of the floats
  const uint32_t b = __float_as_uint(f);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float order_key_inv(uint32_t k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}

// sums of three per-thread values over the block, the same bits in every thread; `slot` alternates
// between consecutive calls so that one barrier per call is enough
__device__ __forceinline__ void block_total3(float (&v)[3], CutSmem& cs, int slot) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int c = 0; c < 3; ++c) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v[c] += __shfl_xor_sync(0xffffffffu, v[c], o);
    if (lane == 0) cs.f[slot][c][warp] = v[c];
  }
  __syncthreads();
#pragma unroll
  for (int c = 0; c < 3; ++c) {
    float t = cs.f[slot][c][lane];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) t += __shfl_xor_sync(0xffffffffu, t, o);
    v[c] = t;
  }
}
__device__ __forceinline__ void block_total3(int (&v)[3], CutSmem& cs, int slot) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int c = 0; c < 3; ++c) {
    v[c] = __reduce_add_sync(0xffffffffu, v[c]);
    if (lane == 0) cs.i[slot][c][warp] = v[c];
  }
  __syncthreads();
#pragma unroll
  for (int c = 0; c < 3; ++c) v[c] = __reduce_add_sync(0xffffffffu, cs.i[slot][c][lane]);
}

// The cut of one row and the mass it keeps.
// FAST: V <= CUT_ELEMS * SAMPLER_THREADS and ws holds the row's weights exp((l - m) / T) in shared memory
// (skewed layout, written and visible to the block).  Otherwise keys and weights are recomputed from the
// logits in every step (large vocabularies; slow but the same arithmetic).
template <bool FAST>
__device__ void row_cut_impl(const float* row, const float* ws, int V, float m, float invT, int top_k, float top_p,
                             CutSmem& cs, float* cut_out, float* mass_out) {
  const int tid = threadIdx.x;
  uint32_t kr[CUT_ELEMS];   // FAST: a thread's keys; 0 = no token here, or a token already cut away
  if (FAST) {
#pragma unroll
    for (int j = 0; j < CUT_ELEMS; ++j) {
      const int i = tid + j * SAMPLER_THREADS;
      kr[j] = i < V ? order_key(row[i]) : 0u;
    }
  }
  const int wbase = tid + (tid >> 5);                      // skew(tid + 1024 j) = wbase + 1056 j
  uint32_t floor_key = 0;                                   // slow path: tokens under it are cut away
  // visit every token of this thread: body(key, weight)
  auto each = [&](auto body) {
    if (FAST) {
#pragma unroll
      for (int j = 0; j < CUT_ELEMS; ++j)   // no token, no load: the buffer only covers V entries
        body(kr[j], kr[j] ? ws[wbase + j * (SAMPLER_THREADS + SAMPLER_WARPS)] : 0.f);
    } else {
      for (int i = tid; i < V; i += SAMPLER_THREADS) {
        const float l = row[i];
        const uint32_t k = order_key(l);
        body(k >= floor_key ? k : 0u, expf((l - m) * invT));
      }
    }
  };
  uint32_t key = 0;
  int slot = 0;
  if (top_k >= 1 && top_k < V) {
#pragma unroll 1
    for (int b = 30; b >= 0; b -= 2) {
      int cnt[3] = {0, 0, 0};
      const uint32_t c1 = key | (1u << b), c2 = key | (2u << b), c3 = key | (3u << b);
      each([&](uint32_t k, float) {
        cnt[0] += k >= c1;
        cnt[1] += k >= c2;
        cnt[2] += k >= c3;
      });
      block_total3(cnt, cs, slot);
      slot ^= 1;
      key = cnt[2] >= top_k ? c3 : (cnt[1] >= top_k ? c2 : (cnt[0] >= top_k ? c1 : key));
    }
    if (FAST) {
#pragma unroll
      for (int j = 0; j < CUT_ELEMS; ++j)
        if (kr[j] < key) kr[j] = 0u;
    }
    floor_key = key;
  }
  // mass of what is left
  float z[3] = {0.f, 0.f, 0.f};
  each([&](uint32_t k, float w) { if (k) z[0] += w; });
  block_total3(z, cs, slot);
  slot ^= 1;
  float Z = z[0];
  if (top_p < 1.0f) {
    const float target = top_p * Z;
    uint32_t kp = 0;
#pragma unroll 1
    for (int b = 30; b >= 0; b -= 2) {
      float sm3[3] = {0.f, 0.f, 0.f};
      const uint32_t c1 = kp | (1u << b), c2 = kp | (2u << b), c3 = kp | (3u << b);
      each([&](uint32_t k, float w) {
        if (k >= c1) sm3[0] += w;
        if (k >= c2) sm3[1] += w;
        if (k >= c3) sm3[2] += w;
      });
      block_total3(sm3, cs, slot);
      slot ^= 1;
      kp = sm3[2] >= target ? c3 : (sm3[1] >= target ? c2 : (sm3[0] >= target ? c1 : kp));
    }
    if (kp > key) {
      key = kp;
      float zz[3] = {0.f, 0.f, 0.f};
      each([&](uint32_t k, float w) { if (k >= key) zz[0] += w; });
      block_total3(zz, cs, slot);
      Z = zz[0];
    }
  }
  __syncthreads();   // the scratch may be reused at once by the caller's next cut
  *cut_out = key == 0u ? -INFINITY : order_key_inv(key);
  *mass_out = Z;
}

// Cuts row `row` (maximum m).  With have_ws the weights are staged in ws first (the caller's shared buffer).
__device__ void row_cut(const float* row, float* ws, bool have_ws, int V, float m, float invT, int top_k, float top_p,
                        CutSmem& cs, float* cut_out, float* mass_out) {
  if (have_ws && V <= CUT_ELEMS * SAMPLER_THREADS) {
    for (int i = threadIdx.x; i < V; i += SAMPLER_THREADS) ws[i + (i >> 5)] = expf((row[i] - m) * invT);
    __syncthreads();
    row_cut_impl<true>(row, ws, V, m, invT, top_k, top_p, cs, cut_out, mass_out);
  } else {
    row_cut_impl<false>(row, ws, V, m, invT, top_k, top_p, cs, cut_out, mass_out);
  }
}

// ------------------------------------------------------------------------------------------------
// x ~ softmax(logits / T) by inverse CDF with u_draft(b, s, t)  (the draft draws of Algorithm 2's first
// for-loop; with t = 0 and u_res it is Algorithm 1's sample).
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(SAMPLER_THREADS) sample_kernel(SampleArgs a) {
  __shared__ ScanSmem sm;
  __shared__ CutSmem cs;
  __shared__ float s_part[SAMPLER_WARPS];
  __shared__ float s_val;
  const int b = blockIdx.x;
  pdl_launch_dependents();
  pdl_wait();
  float T = a.temperature;
  uint64_t seed = a.seed;
  uint32_t step = a.step;
  int top_k = a.top_k;
  float top_p = a.top_p;
  uint32_t seq = (uint32_t)b;   // Philox sequence index
  if (a.st) { T = a.st->temperature; seed = a.st->seed; step = a.st->step; top_k = a.st->top_k; top_p = a.st->top_p; seq += a.st->seq0; }
  const float invT = 1.0f / T;
  const float* row = a.logits + (long long)b * a.ld;
  const Uniforms u = sps_uniforms(seed, seq, step, a.t);
  int tok;
  if ((top_k >= 1 && top_k < a.V) || top_p < 1.0f) {
    // filtered draw: tokens under the cut weigh nothing
    float m = -INFINITY;
    for (int i = threadIdx.x; i < a.V; i += blockDim.x) m = fmaxf(m, row[i]);
    m = block_max_f(m, s_part, &s_val);
    extern __shared__ float ws[];
    float cut, mass;
    row_cut(row, ws, a.smem_weights != 0, a.V, m, invT, top_k, top_p, cs, &cut, &mass);
    auto w = [&](int i) { const float l = row[i]; return l >= cut ? expf((l - m) * invT) : 0.f; };
    if (a.smem_weights) {
      for (int i = threadIdx.x; i < a.V; i += blockDim.x) ws[skew(i)] = w(i);
      __syncthreads();
      tok = block_invcdf_smem(ws, a.V, u.u_draft, sm, nullptr);
    } else {
      tok = block_invcdf(w, a.V, u.u_draft, sm, nullptr);
    }
  } else if (a.smem_weights && a.V <= 32 * SAMPLER_THREADS) {
    // the row is read once: a thread keeps its (at most 32) logits in registers between the max and the exp
    extern __shared__ float ws[];
    float l[32];
#pragma unroll
    for (int j = 0; j < 32; ++j) {
      const int i = threadIdx.x + j * SAMPLER_THREADS;
      l[j] = i < a.V ? row[i] : -INFINITY;
    }
    float m = -INFINITY;
#pragma unroll
    for (int j = 0; j < 32; ++j) m = fmaxf(m, l[j]);
    m = block_max_f(m, s_part, &s_val);
#pragma unroll
    for (int j = 0; j < 32; ++j) {
      const int i = threadIdx.x + j * SAMPLER_THREADS;
      if (i < a.V) ws[skew(i)] = expf((l[j] - m) * invT);
    }
    __syncthreads();
    float total;
    tok = block_invcdf_smem(ws, a.V, u.u_draft, sm, &total);
    // the row's statistics, for the accept kernel: the very numbers this draw was made with
    if (a.stats && threadIdx.x == 0) a.stats[(long long)b * a.stats_ld] = make_float2(m, total);
  } else {
    float m = -INFINITY;
    for (int i = threadIdx.x; i < a.V; i += blockDim.x) m = fmaxf(m, row[i]);
    m = block_max_f(m, s_part, &s_val);
    float total;
    if (a.smem_weights) {
      extern __shared__ float ws[];
      for (int i = threadIdx.x; i < a.V; i += blockDim.x) ws[skew(i)] = expf((row[i] - m) * invT);
      __syncthreads();
      tok = block_invcdf_smem(ws, a.V, u.u_draft, sm, &total);
    } else {
      auto w = [&](int i) { return expf((row[i] - m) * invT); };
      tok = block_invcdf(w, a.V, u.u_draft, sm, &total);
    }
    if (a.stats && threadIdx.x == 0) a.stats[(long long)b * a.stats_ld] = make_float2(m, total);
  }
  if (threadIdx.x == 0) a.out[(long long)b * a.out_ld] = tok;
}

// bytes of the shared weight buffer for a vocabulary, or 0 when it does not fit (weights are then recomputed)
static size_t weights_smem(int V) {
  const size_t bytes = sizeof(float) * ((size_t)V + (size_t)V / 32 + 32);
  return bytes <= 200 * 1024 ? bytes : 0;
}
template <class Kern>
static cudaError_t sampler_smem_attr(Kern k, size_t bytes, DevSmemCache& cached) { return sps_ensure_smem(k, bytes, cached); }

cudaError_t sample_launch(const SampleArgs& a_in, cudaStream_t st) {
  static DevSmemCache cached{};
  SampleArgs a = a_in;
  const size_t smem = weights_smem(a.V);
  a.smem_weights = smem ? 1 : 0;
  cudaError_t e = sampler_smem_attr(sample_kernel, smem, cached);
  if (e != cudaSuccess) return e;
  return launch_k(sample_kernel, dim3(a.B), dim3(SAMPLER_THREADS), smem, st, a);
}

// ------------------------------------------------------------------------------------------------
// Modified rejection sampling, fused (Algorithm 2, second for-loop and extra-token line).
// Phase 1: max and sum-exp of all 2K+1 rows.  Phase 2: thread 0 walks the accept chain.
// Phase 3: one vocabulary-wide prefix sum, over max(0, q_t - p_t) at the rejected position or over
// q_K when every draft was accepted.  When a DevState is given the loop is advanced in place.
// ------------------------------------------------------------------------------------------------
#define ACC_MAX_ROWS (2 * 15 + 1)

__global__ void __launch_bounds__(SAMPLER_THREADS) accept_kernel(AcceptArgs a) {
  __shared__ ScanSmem sm;
  __shared__ float s_red[SAMPLER_WARPS][ACC_MAX_ROWS + 1];
  __shared__ float s_max[ACC_MAX_ROWS], s_sum[ACC_MAX_ROWS], s_cut[ACC_MAX_ROWS];
  __shared__ int s_stop;
  __shared__ CutSmem cs;
  extern __shared__ float ws[];
  const int b = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int K = a.K, V = a.V, R = 2 * K + 1;
  pdl_launch_dependents();
  pdl_wait();
  float T = a.temperature;
  uint64_t seed = a.seed;
  uint32_t step = a.step;
  int top_k = a.top_k;
  float top_p = a.top_p;
  uint32_t seq = (uint32_t)b;   // Philox sequence index
  if (a.st) { T = a.st->temperature; seed = a.st->seed; step = a.st->step; top_k = a.st->top_k; top_p = a.st->top_p; seq += a.st->seq0; }
  const bool filt = (top_k >= 1 && top_k < V) || top_p < 1.0f;
  const float invT = 1.0f / T;
  const float* qrow = a.q_logits + (long long)b * (K + 1) * V;
  const float* prow = a.p_logits + (long long)b * K * V;
  auto rowptr = [&](int r) { return r <= K ? qrow + (long long)r * V : prow + (long long)(r - K - 1) * V; };

  // ---- phase 1a: maxima
  for (int r = 0; r < R; ++r) {
    const float* row = rowptr(r);
    float m = -INFINITY;
    for (int i = tid; i < V; i += SAMPLER_THREADS) m = fmaxf(m, row[i]);
    m = warp_max(m);
    if (lane == 0) s_red[warp][r] = m;
  }
  __syncthreads();
  if (tid < R) {
    float m = -INFINITY;
    for (int w = 0; w < SAMPLER_WARPS; ++w) m = fmaxf(m, s_red[w][tid]);
    s_max[tid] = m;
  }
  __syncthreads();
  // ---- phase 1b: sums of exp((l - max) / T)
  for (int r = 0; r < R; ++r) {
    const float* row = rowptr(r);
    const float m = s_max[r];
    float s = 0.f;
    for (int i = tid; i < V; i += SAMPLER_THREADS) s += expf((row[i] - m) * invT);
    s = warp_sum(s);
    if (lane == 0) s_red[warp][r] = s;
  }
  __syncthreads();
  if (tid < R) {
    float s = 0.f;
    for (int w = 0; w < SAMPLER_WARPS; ++w) s += s_red[w][tid];
    s_sum[tid] = s;
    s_cut[tid] = -INFINITY;
  }
  __syncthreads();
  // with top-k / nucleus filtering a row's cut and kept mass replace its plain sum; rows are cut when the
  // chain reaches them (block-wide work), so a loop that stops early does not pay for the later rows
  auto cut_row = [&](int r) {
    float cut, mass;
    row_cut(rowptr(r), ws, a.smem_weights != 0, V, s_max[r], invT, top_k, top_p, cs, &cut, &mass);
    if (tid == 0) { s_cut[r] = cut; s_sum[r] = mass; }
    __syncthreads();
  };

  // ---- phase 2: accept chain, left to right
  const int32_t* drafts = a.drafts + (long long)b * a.drafts_ld;
  const float forced = a.st ? __uint_as_float(a.st->pad0) : 0.f;
  auto accept_at = [&](int t) {   // thread 0: does draft t pass?
    int d = drafts[t];
    if (d < 0 || d >= V) { d = 0; if (a.st) atomicExch(a.st->err, 1); }
    const float lq = qrow[(long long)t * V + d], lp = prow[(long long)t * V + d];
    const float qd = lq >= s_cut[t] ? expf((lq - s_max[t]) * invT) / s_sum[t] : 0.f;
    const float pd = lp >= s_cut[K + 1 + t] ? expf((lp - s_max[K + 1 + t]) * invT) / s_sum[K + 1 + t] : 0.f;
    // accept with probability min(1, q(d)/p(d)); p == 0 with q > 0 accepts, 0/0 rejects
    const float ratio = (pd > 0.f) ? fminf(1.0f, qd / pd) : (qd > 0.f ? 1.0f : 0.0f);
    const Uniforms u = sps_uniforms(seed, seq, step, (uint32_t)t);
    // measurement mode only: accept with a fixed probability whatever the models say (tokens per loop as a function
    // of the acceptance rate alone); the emitted tokens then follow no particular law
    if (forced > 0.f) return u.u_acc < forced;
    return u.u_acc < ratio;
  };
  if (!filt) {
    if (tid == 0) {
      int stop = K;
      for (int t = 0; t < K; ++t)
        if (!accept_at(t)) { stop = t; break; }
      s_stop = stop;
    }
    __syncthreads();
  } else {
    if (tid == 0) s_stop = K;
    __syncthreads();
    for (int t = 0; t < K; ++t) {
      cut_row(t);
      cut_row(K + 1 + t);
      if (tid == 0 && !accept_at(t)) s_stop = t;
      __syncthreads();
      if (s_stop != K) break;
    }
    if (s_stop == K) cut_row(K);
  }
  const int stop = s_stop;
  uint32_t fl = 0;
  int tok;
  if (stop < K) {
    // ---- rejected at `stop`: x ~ max(0, q - p) / sum max(0, q - p)
    const float* ql = qrow + (long long)stop * V;
    const float* pl = prow + (long long)stop * V;
    const float mq = s_max[stop], mp = s_max[K + 1 + stop];
    const float iq = 1.0f / s_sum[stop], ip = 1.0f / s_sum[K + 1 + stop];
    const Uniforms u = sps_uniforms(seed, seq, step, (uint32_t)stop);
    const float cq = s_cut[stop], cp = s_cut[K + 1 + stop];
    auto wres = [&](int i) {
      const float lq = ql[i], lp = pl[i];
      const float qv = lq >= cq ? expf((lq - mq) * invT) * iq : 0.f;
      const float pv = lp >= cp ? expf((lp - mp) * invT) * ip : 0.f;
      return fmaxf(0.f, qv - pv);
    };
    auto wq = [&](int i) { const float lq = ql[i]; return lq >= cq ? expf((lq - mq) * invT) : 0.f; };
    float total;
    if (a.smem_weights) {
      for (int i = tid; i < V; i += SAMPLER_THREADS) ws[skew(i)] = wres(i);
      __syncthreads();
      tok = block_invcdf_smem(ws, V, u.u_res, sm, &total);
    } else {
      tok = block_invcdf(wres, V, u.u_res, sm, &total);
    }
    fl |= 1u;
    if (!(total > 0.f)) {
      tok = block_invcdf(wq, V, u.u_res, sm, nullptr);
      fl |= 4u;
    }
  } else {
    // ---- every draft accepted: extra token from the (K+1)-th target distribution
    const float* ql = qrow + (long long)K * V;
    const float mq = s_max[K], cq = s_cut[K];
    const Uniforms u = sps_uniforms(seed, seq, step, (uint32_t)K);
    auto wq = [&](int i) { const float lq = ql[i]; return lq >= cq ? expf((lq - mq) * invT) : 0.f; };
    if (a.smem_weights) {
      for (int i = tid; i < V; i += SAMPLER_THREADS) ws[skew(i)] = wq(i);
      __syncthreads();
      tok = block_invcdf_smem(ws, V, u.u_res, sm, nullptr);
    } else {
      tok = block_invcdf(wq, V, u.u_res, sm, nullptr);
    }
    fl |= 2u;
  }
  // ---- results
  int32_t* out = a.out_tok + (long long)b * a.out_ld;
  if (tid <= K) out[tid] = (tid < stop) ? drafts[tid] : (tid == stop ? tok : -1);
  if (tid == 0) {
    a.n_acc[b] = stop;
    a.flags[b] = fl;
  }
  if (a.st) {
    // advance the sequence in place: accepted drafts, then the resampled / extra token
    DevState* st = a.st;
    const int n = st->n[b];
    const bool live = n < st->limit[b];   // a finished sequence of a batch keeps its length
    __syncthreads();
    if (live && tid <= stop && n + tid < st->max_seq)
      st->tokens[(long long)b * st->max_seq + n + tid] = (tid < stop) ? drafts[tid] : tok;
    __syncthreads();
    if (tid == 0) {
      if (live) st->n[b] = n + stop + 1;
      __threadfence();
      // the last sequence to finish moves the loop counter
      const uint32_t done = atomicAdd(st->done_counter, 1u);
      if (done == (uint32_t)gridDim.x - 1) {
        *st->done_counter = 0u;
        st->step = step + 1u;
      }
    }
  }
}

// ------------------------------------------------------------------------------------------------
// The same sampler spread over a thread-block cluster: C CTAs per sequence, CTA c owning tokens
// [c * slice, (c + 1) * slice) of every row (unfiltered distributions; the filtered ones keep the kernel above).
//   1. every row whose softmax statistics are needed is read ONCE: its slice goes to shared memory with 16-byte
//      loads, the CTA takes the slice's maximum and the sum of exp((l - max) / T) from there; the C partial
//      (max, sum) pairs of a row meet in every CTA's shared memory (distributed shared memory) and are merged
//      in CTA order.  Draft rows whose statistics the draft sampler left at draft time (p_stats) are not read.
//   2. every CTA walks the accept chain for itself (same numbers, same decisions): the 2K logits it needs were
//      asked for at kernel start.
//   3. the weights of the one distribution that is drawn from -- max(0, q_t - p_t) at the rejected position, or
//      q_K -- are formed for the CTA's slice (from the rows kept in shared memory when they fit, else re-read),
//      scanned as in block_invcdf, the CTAs' totals meet as the statistics did, and each CTA looks for the
//      first running sum above u * total inside its slice; the smallest candidate wins.
// All sums run in a fixed order (thread chunk, warp scan, warp totals, CTA order): bit-reproducible.
// ------------------------------------------------------------------------------------------------
#include <cooperative_groups.h>
namespace cg = cooperative_groups;

#define ACCF_MAX_C 8
#define ACCF_MAX_STAGES 32
// exp((l - m) / T) as 2^((l - m) * c) with c = log2(e) / T: a subtraction, a multiplication and the hardware's
// base-2 exponential (relative error about 2^-22, plus |argument| * 2^-23 from the product's rounding: below 1e-6 for
// every weight that carries mass).  The passes over whole rows are bound by instruction issue, and the library
// exponential costs four times as many instructions.
__device__ __forceinline__ float exp2_scaled(float l, float m, float c) {
  float r;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"((l - m) * c));
  return r;
}
struct AccfShared {
  ScanSmem sm;
  float2 seg[ACC_MAX_ROWS][SAMPLER_WARPS];   // (max, sum) of the segments of each row of the batch in hand
  float2 part[ACC_MAX_ROWS][ACCF_MAX_C];     // (max, sum) of each row's slice, by CTA rank (filled by all CTAs of the cluster)
  float row_m[ACC_MAX_ROWS], row_s[ACC_MAX_ROWS];
  float lq[16], lp[16];                      // logits of the draft tokens in their target / draft rows
  int dtok[16], okt[16];
  float tot[ACCF_MAX_C];                     // the CTAs' weight totals
  int cand[ACCF_MAX_C], lastpos[ACCF_MAX_C];
  int wcand[SAMPLER_WARPS], wlast[SAMPLER_WARPS];
  int stop, timeout;
  unsigned long long bar[ACCF_MAX_STAGES];   // one mbarrier per unit buffer
};

__device__ __forceinline__ uint32_t s_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
// 16 bytes global -> shared without passing through registers; completion is waited for with cp_async_wait
__device__ __forceinline__ void cp_async16(float* dst, const float* src) {
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(s_smem_u32(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
// wait for a phase of an mbarrier, at most limit_ns of the global timer; false when the bound ran out
__device__ __forceinline__ bool s_mbar_wait(uint32_t bar, uint32_t parity, unsigned long long limit_ns) {
  unsigned long long t0 = 0;
  for (int spin = 0;; ++spin) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    if (ok) return true;
    if ((spin & 63) == 63) {
      unsigned long long t;
      asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
      if (t0 == 0) t0 = t;
      else if (t - t0 > limit_ns) return false;
    }
  }
}

__global__ void __launch_bounds__(SAMPLER_THREADS) accept_cluster_kernel(AcceptArgs a) {
  __shared__ AccfShared sh;
  extern __shared__ __align__(128) float dyn[];
  cg::cluster_group cluster = cg::this_cluster();
  const int C = a.csize, rank = (int)cluster.block_rank(), b = blockIdx.x / C;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int K = a.K, V = a.V;
  const int i0 = min(rank * a.slice, V), i1 = min(i0 + a.slice, V), ns = i1 - i0;   // ns is a multiple of 4 (launcher: V % 4 == 0)
  const bool have_p = a.p_stats != nullptr;
  const int R = have_p ? K + 1 : 2 * K + 1;       // rows whose statistics are worked out here: q_0..q_K, then p_0..p_{K-1}
  const int slice_pad = a.slice;                  // a multiple of 4
  // A row's slice travels in chunks of CH floats (one chunk when the slice is short): unit u = (row u / NCH, chunk u % NCH).
  // Either every unit has a buffer of its own (`resident`: the rows stay for step 3), or the units go through a ring.
  const int CH = a.chunk, NCH = (slice_pad + CH - 1) / CH, U = R * NCH, NSTG = a.resident ? U : a.stages;
  if (tid == 0) {
    for (int i = 0; i < NSTG; ++i) asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(s_smem_u32(&sh.bar[i])) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    sh.timeout = 0;
  }
  cluster.barrier_arrive();     // its wait stands before the first access to another CTA's shared memory: by then every CTA runs
  __syncthreads();
  pdl_launch_dependents();
  pdl_wait();
  float T = a.temperature;
  uint64_t seed = a.seed;
  uint32_t step = a.step;
  uint32_t seq = (uint32_t)b;
  if (a.st) { T = a.st->temperature; seed = a.st->seed; step = a.st->step; seq += a.st->seq0; }
  const float invT = 1.0f / T;
  const float c2 = invT * 1.4426950408889634f;    // log2(e) / T
  const float* qrow = a.sample_t >= 0 ? a.q_logits + (long long)b * a.q_ld : a.q_logits + (long long)b * (K + 1) * V;
  const float* prow = a.p_logits + (long long)b * K * V;
  const int32_t* drafts = a.drafts + (long long)b * a.drafts_ld;
  auto rowptr = [&](int r) { return r <= K ? qrow + (long long)r * V : prow + (long long)(r - K - 1) * V; };
  auto unit_floats = [&](int u) { const int ch = u % NCH; return max(0, min(CH, ns - ch * CH)); };
  // units [u0, u0 + nb) on their way into their buffers: one bulk copy each (the copy engine works while the warps
  // compute), completion counted on the buffer's mbarrier.  Issued by thread 0.
  auto issue_units = [&](int u0, int nb) {
    for (int j = 0; j < nb; ++j) {
      const int u = u0 + j, r = u / NCH, ch = u - r * NCH;
      const uint32_t bar = s_smem_u32(&sh.bar[u % NSTG]), bytes = (uint32_t)unit_floats(u) * 4u;
      if (bytes == 0) { asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory"); continue; }
      asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
      asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                   ::"r"(s_smem_u32(dyn + (size_t)(u % NSTG) * CH)), "l"(rowptr(r) + i0 + (size_t)ch * CH), "r"(bytes), "r"(bar) : "memory");
    }
  };
  // resident: all units in one batch.  Ring: half the ring at a time, the other half is in flight meanwhile.
  const int units_at_once = a.resident ? U : max(1, NSTG / 2);
  if (tid == 0) issue_units(0, min(U, a.resident ? U : NSTG));
  // the draft tokens' logits: asked for now, used by the chain
  if (tid >= 32 && tid < 32 + K) {
    const int t = tid - 32;
    int d = drafts[t];
    if (d < 0 || d >= V) { d = 0; if (a.st) atomicExch(a.st->err, 1); }
    sh.dtok[t] = d;
    sh.lq[t] = qrow[(long long)t * V + d];
    sh.lp[t] = prow[(long long)t * V + d];
  }
  // ---- 1. statistics.  A warp takes one segment of one unit: its maximum, then the sum of exp((l - max) / T); the
  // segments are merged by one thread per row, in unit and segment order.
  if (tid < R) { sh.row_m[tid] = -INFINITY; sh.row_s[tid] = 0.f; }
  const int NSEG = max(1, SAMPLER_WARPS / units_at_once);
  for (int u0 = 0; u0 < U; u0 += units_at_once) {
    const int nb = min(units_at_once, U - u0);
    for (int item = warp; item < nb * NSEG; item += SAMPLER_WARPS) {
      const int j = item / NSEG, sg = item - j * NSEG, u = u0 + j;
      // a warp waits for its own unit only: units that have landed are worked on while the others are in flight
      if (!s_mbar_wait(s_smem_u32(&sh.bar[u % NSTG]), (uint32_t)((u / NSTG) & 1), a.wait_ns)) sh.timeout = 1;
      const float4* src = reinterpret_cast<const float4*>(dyn + (size_t)(u % NSTG) * CH);
      const int n4 = unit_floats(u) >> 2, per = (n4 + NSEG - 1) / NSEG, q0 = min(sg * per, n4), q1 = min(q0 + per, n4);
      float m = -INFINITY;
      for (int q4 = q0 + lane; q4 < q1; q4 += 32) { const float4 v = src[q4]; m = fmaxf(fmaxf(m, fmaxf(v.x, v.y)), fmaxf(v.z, v.w)); }
      m = warp_max(m);
      float sum = 0.f;
      for (int q4 = q0 + lane; q4 < q1; q4 += 32) {
        const float4 v = src[q4];
        sum += (exp2_scaled(v.x, m, c2) + exp2_scaled(v.y, m, c2)) + (exp2_scaled(v.z, m, c2) + exp2_scaled(v.w, m, c2));
      }
      sum = warp_sum(sum);
      if (lane == 0) sh.seg[j][sg] = make_float2(q1 > q0 ? m : -INFINITY, q1 > q0 ? sum : 0.f);
    }
    __syncthreads();
    if (warp < nb) {
      // unit `warp` of the batch: its segments, one per lane, merged with shuffles (a fixed tree)
      const float2 v = lane < NSEG ? sh.seg[warp][lane] : make_float2(-INFINITY, 0.f);
      const float mu = warp_max(v.x);
      const float su = warp_sum(v.y > 0.f ? v.y * expf((v.x - mu) * invT) : 0.f);
      if (lane == 0) sh.seg[warp][0] = make_float2(mu, su);
    }
    __syncthreads();
    if (tid < R) {
      // row `tid` takes in its units of this batch, in unit order (this CTA's slice only, for now)
      float rm = sh.row_m[tid], rs = sh.row_s[tid];
      for (int j = 0; j < nb; ++j) {
        const float2 v = sh.seg[j][0];
        if ((u0 + j) / NCH != tid || !(v.y > 0.f)) continue;
        const float m = fmaxf(rm, v.x);
        rs = (rs > 0.f ? rs * expf((rm - m) * invT) : 0.f) + v.y * expf((v.x - m) * invT);
        rm = m;
      }
      sh.row_m[tid] = rm; sh.row_s[tid] = rs;
    }
    __syncthreads();              // this batch's buffers and the segment scratch are free again
    if (!a.resident && tid == 0 && u0 + NSTG < U) issue_units(u0 + NSTG, min(nb, U - u0 - NSTG));   // the units that take these buffers next
  }
  __syncthreads();
  // the C partial statistics of every row meet in every CTA
  cluster.barrier_wait();
  for (int idx = tid; idx < R * C; idx += SAMPLER_THREADS) {
    const int r = idx / C, c = idx - r * C;
    float2* remote = cluster.map_shared_rank(&sh.part[r][rank], c);
    *remote = make_float2(ns > 0 ? sh.row_m[r] : -INFINITY, ns > 0 ? sh.row_s[r] : 0.f);
  }
  cluster.sync();
  if (tid < 2 * K + 1) {
    const int r = tid;
    if (r < R) {
      float m = -INFINITY;
      for (int c = 0; c < C; ++c) m = fmaxf(m, sh.part[r][c].x);
      float sum = 0.f;
      for (int c = 0; c < C; ++c) { const float2 pc = sh.part[r][c]; if (pc.y > 0.f) sum += pc.y * expf((pc.x - m) * invT); }
      sh.row_m[r] = m; sh.row_s[r] = sum;
    } else {
      const float2 ps = a.p_stats[(long long)b * a.p_stats_ld + (r - K - 1)];
      sh.row_m[r] = ps.x; sh.row_s[r] = ps.y;
    }
  }
  __syncthreads();
  // ---- 2. the accept chain: every test on its own thread, the first failure stops the chain (every CTA, identically)
  if (tid < K) {
    const int t = tid;
    const float forced = a.st ? __uint_as_float(a.st->pad0) : 0.f;
    const float qd = expf((sh.lq[t] - sh.row_m[t]) * invT) / sh.row_s[t];
    const float pd = expf((sh.lp[t] - sh.row_m[K + 1 + t]) * invT) / sh.row_s[K + 1 + t];
    // accept with probability min(1, q(d)/p(d)); p == 0 with q > 0 accepts, 0/0 rejects
    const float ratio = (pd > 0.f) ? fminf(1.0f, qd / pd) : (qd > 0.f ? 1.0f : 0.0f);
    const Uniforms ut = sps_uniforms(seed, seq, step, (uint32_t)t);
    sh.okt[t] = forced > 0.f ? (ut.u_acc < forced) : (ut.u_acc < ratio);   // forced: measurement mode only
  }
  __syncthreads();
  int stop = K;
  for (int t = K - 1; t >= 0; --t) if (!sh.okt[t]) stop = t;
  const Uniforms u = sps_uniforms(seed, seq, step, (uint32_t)stop);
  uint32_t fl = stop < K ? 1u : 2u;
  // ---- 3. the draw: residual at `stop`, or q_K; if the residual sums to nothing, q_stop (flagged)
  // (resident: one chunk per row, so row r sits at dyn + r * CH)
  float* wbuf = a.resident ? dyn + (size_t)R * CH : dyn;     // skewed: element i of the slice at i + (i >> 5)
  const float* ql = (a.resident ? dyn + (size_t)stop * CH : qrow + (long long)stop * V + i0);
  const float* pl = stop < K ? ((a.resident && !have_p) ? dyn + (size_t)(K + 1 + stop) * CH : prow + (long long)stop * V + i0) : ql;
  const float mq = sh.row_m[stop], iq = 1.0f / sh.row_s[stop];
  const float mp = stop < K ? sh.row_m[K + 1 + stop] : 0.f, ip = stop < K ? 1.0f / sh.row_s[K + 1 + stop] : 0.f;
  int tok = -1;
  for (int attempt = 0; attempt < 2; ++attempt) {
    const bool residual = stop < K && attempt == 0;
    __syncthreads();
    {
      const float4* q4p = reinterpret_cast<const float4*>(ql);
      const float4* p4p = reinterpret_cast<const float4*>(pl);
      for (int q4 = tid; q4 < (ns >> 2); q4 += SAMPLER_THREADS) {
        const float4 lq4 = q4p[q4];
        float w[4] = {exp2_scaled(lq4.x, mq, c2), exp2_scaled(lq4.y, mq, c2), exp2_scaled(lq4.z, mq, c2), exp2_scaled(lq4.w, mq, c2)};
        if (residual) {
          const float4 lp4 = p4p[q4];
          w[0] = fmaxf(0.f, w[0] * iq - exp2_scaled(lp4.x, mp, c2) * ip);
          w[1] = fmaxf(0.f, w[1] * iq - exp2_scaled(lp4.y, mp, c2) * ip);
          w[2] = fmaxf(0.f, w[2] * iq - exp2_scaled(lp4.z, mp, c2) * ip);
          w[3] = fmaxf(0.f, w[3] * iq - exp2_scaled(lp4.w, mp, c2) * ip);
        }
        const int i = q4 << 2;                    // four consecutive elements never straddle a skew boundary
        float* dst = wbuf + skew(i);
        dst[0] = w[0]; dst[1] = w[1]; dst[2] = w[2]; dst[3] = w[3];
      }
    }
    __syncthreads();
    // scan of the slice: chunk sums, warp scan, scan of the warp totals (as block_invcdf)
    const int chunk = (ns + SAMPLER_THREADS - 1) / SAMPLER_THREADS;
    const int c0 = min(tid * chunk, ns), c1 = min(c0 + chunk, ns);
    float local = 0.f;
    for (int i = c0; i < c1; ++i) local += wbuf[skew(i)];
    float incl = local;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const float v = __shfl_up_sync(0xffffffffu, incl, o);
      if (lane >= o) incl += v;
    }
    if (lane == 31) sh.sm.warp_part[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      const float v = sh.sm.warp_part[lane];
      float iv = v;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const float x = __shfl_up_sync(0xffffffffu, iv, o);
        if (lane >= o) iv += x;
      }
      sh.sm.warp_part[lane] = iv - v;
      const float tot_cta = __shfl_sync(0xffffffffu, iv, 31);
      if (lane == 31) sh.sm.total = iv;
      if (lane < C) *cluster.map_shared_rank(&sh.tot[rank], lane) = tot_cta;
    }
    cluster.sync();               // also orders this CTA's warp_part / total
    const float pre_cta = sh.sm.warp_part[warp] + (incl - local);
    float offset = 0.f, grand = 0.f;
    for (int c = 0; c < C; ++c) { if (c == rank) offset = grand; grand += sh.tot[c]; }
    if (residual && !(grand > 0.f)) { fl |= 4u; cluster.sync(); continue; }   // nothing left of q - p: draw from q_stop (every CTA decides the same)
    const float target = (a.sample_t >= 0 ? sps_uniforms(seed, seq, step, (uint32_t)a.sample_t).u_draft : u.u_res) * grand;
    int cand = INT_MAX, last = -1;
    float cs = offset + pre_cta;
    for (int i = c0; i < c1; ++i) {
      const float w = wbuf[skew(i)];
      cs += w;
      if (w > 0.f) last = i0 + i;
      if (cs > target && cand == INT_MAX) cand = i0 + i;
    }
    cand = warp_min_int(cand);
    last = warp_max_int(last);
    if (lane == 0) { sh.wcand[warp] = cand; sh.wlast[warp] = last; }
    __syncthreads();
    if (warp == 0) {
      cand = warp_min_int(sh.wcand[lane]);
      last = warp_max_int(sh.wlast[lane]);
      if (lane == 0) {
        *cluster.map_shared_rank(&sh.cand[rank], 0) = cand;
        *cluster.map_shared_rank(&sh.lastpos[rank], 0) = last;
      }
    }
    cluster.sync();
    if (rank == 0) {
      int best = INT_MAX, lp = -1;
      for (int c = 0; c < C; ++c) { best = min(best, sh.cand[c]); lp = max(lp, sh.lastpos[c]); }
      tok = best != INT_MAX ? best : (lp >= 0 ? lp : V - 1);
    }
    break;
  }
  if (sh.timeout) {   // a copy never arrived within the bound: the outputs mean nothing; say so
    fl |= 8u;         // SPS_FLAG_TIMEOUT
    if (a.st && tid == 0) atomicExch(a.st->err, 3);
  }
  if (rank != 0) return;
  // ---- results (first CTA of the cluster)
  if (a.sample_t >= 0) {   // the draft sampler: the token, and the row's statistics for the accept kernel
    if (tid == 0) {
      a.out_tok[(long long)b * a.out_ld] = tok;
      if (a.stats_out) a.stats_out[(long long)b * a.stats_ld] = make_float2(sh.row_m[0], sh.row_s[0]);
    }
    return;
  }
  int32_t* out = a.out_tok + (long long)b * a.out_ld;
  if (tid <= K) out[tid] = (tid < stop) ? sh.dtok[tid] : (tid == stop ? tok : -1);
  if (tid == 0) {
    a.n_acc[b] = stop;
    a.flags[b] = fl;
  }
  if (a.st) {
    // advance the sequence in place: accepted drafts, then the resampled / extra token
    DevState* st = a.st;
    const int n = st->n[b];
    const bool live = n < st->limit[b];   // a finished sequence of a batch keeps its length
    __syncthreads();
    if (live && tid <= stop && n + tid < st->max_seq)
      st->tokens[(long long)b * st->max_seq + n + tid] = (tid < stop) ? sh.dtok[tid] : tok;
    __syncthreads();
    if (tid == 0) {
      if (live) st->n[b] = n + stop + 1;
      __threadfence();
      // the last sequence to finish moves the loop counter
      const uint32_t done = atomicAdd(st->done_counter, 1u);
      if (done == (uint32_t)(gridDim.x / C) - 1) {
        *st->done_counter = 0u;
        st->step = step + 1u;
      }
    }
  }
}

// how many CTAs share a sequence: enough to put every SM to work at small batches, one when the batch fills the GPU
static int accept_cluster_size(int B, int V) {
  static const int forced = [] { const char* e = getenv("SPS_ACCEPT_CLUSTER"); return e ? atoi(e) : -1; }();   // tuning: 0 = the one-CTA kernel
  if (forced >= 0) return forced;
  if (V < 8192) return 0;          // small vocabularies: the one-CTA kernel
  int num_sm = SPS_NUM_SM_FALLBACK, dev = 0;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&num_sm, cudaDevAttrMultiProcessorCount, dev);
  // the largest power of two, at most 8 (the portable cluster size), that keeps all the sequences' CTAs on the GPU at once
  int c = ACCF_MAX_C;
  while (c > 1 && (long long)B * c > num_sm) c >>= 1;
  return c;
}

cudaError_t accept_launch(const AcceptArgs& a_in, cudaStream_t st) {
  static DevSmemCache cached{};
  AcceptArgs a = a_in;
  const size_t smem = weights_smem(a.V);
  a.smem_weights = smem ? 1 : 0;
  cudaError_t e = sampler_smem_attr(accept_kernel, smem, cached);
  if (e != cudaSuccess) return e;
  return launch_k(accept_kernel, dim3(a.B), dim3(SAMPLER_THREADS), smem, st, a);
}

// the cluster form of the draft draw: the accept kernel with K = 0 and one row
cudaError_t sample_launch_fast(const SampleArgs& s, bool filtered, cudaStream_t st) {
  const int C = filtered ? 0 : accept_cluster_size(s.B, s.V);
  const bool aligned = (s.V % 4 == 0) && ((s.ld & 3) == 0) && ((((size_t)s.logits) & 15) == 0);
  if (C < 1 || !aligned) return sample_launch(s, st);
  AcceptArgs a{};
  a.st = const_cast<DevState*>(s.st); a.q_logits = s.logits; a.p_logits = s.logits; a.drafts = s.out; a.drafts_ld = 0;
  a.B = s.B; a.K = 0; a.V = s.V; a.out_tok = s.out; a.out_ld = s.out_ld;
  a.temperature = s.temperature; a.seed = s.seed; a.step = s.step;
  a.sample_t = (int)s.t; a.q_ld = s.ld; a.stats_out = s.stats; a.stats_ld = s.stats_ld;
  const cudaError_t e = accept_launch_fast(a, false, st);
  if (e != cudaErrorInvalidValue) return e;
  (void)cudaGetLastError();          // a shape the cluster kernel does not take: the one-CTA kernel
  return sample_launch(s, st);
}

// the cluster form; `filtered` says whether top-k / nucleus filtering is in force (then the kernel above runs)
cudaError_t accept_launch_fast(const AcceptArgs& a_in, bool filtered, cudaStream_t st) {
  const int C = filtered ? 0 : accept_cluster_size(a_in.B, a_in.V);
  // rows travel as bulk copies: 16-byte aligned row starts and slices
  const bool aligned = (a_in.V % 4 == 0) && ((((size_t)a_in.q_logits | (size_t)a_in.p_logits) & 15) == 0);
  if (C < 1 || a_in.K > 15 || !aligned) return a_in.sample_t >= 0 ? cudaErrorInvalidValue : accept_launch(a_in, st);
  static DevSmemCache cached{};
  AcceptArgs a = a_in;
  a.csize = C;
  a.slice = (((a.V + C - 1) / C) + 3) & ~3;
  a.wait_ns = sps_wait_knobs().limit_ns;
  const int R = a.p_stats ? a.K + 1 : 2 * a.K + 1;
  const size_t slice_pad = (size_t)a.slice;
  const size_t wbytes = sizeof(float) * (slice_pad + slice_pad / 32 + 32);
  const size_t budget = 196 * 1024;
  size_t smem;
  if (sizeof(float) * R * slice_pad + wbytes <= budget && R <= ACCF_MAX_STAGES) {
    a.resident = 1; a.chunk = a.slice; a.stages = R;             // every row's slice stays in shared memory
    smem = sizeof(float) * R * slice_pad + wbytes;
  } else {
    a.resident = 0;                                              // chunks of at most 32 KB through a ring; the weights reuse it afterwards
    a.chunk = a.slice < 8192 ? a.slice : 8192;
    if (wbytes > budget) return a_in.sample_t >= 0 ? cudaErrorInvalidValue : accept_launch(a_in, st);   // a slice whose weights do not fit: one-CTA kernel
    int stages = (int)(budget / (sizeof(float) * a.chunk));
    const int units = R * ((a.slice + a.chunk - 1) / a.chunk);
    if (stages > units) stages = units;
    if (stages > ACCF_MAX_STAGES) stages = ACCF_MAX_STAGES;
    if (stages < 2) stages = 2;
    stages &= ~1;                                                // two halves: one being read, one in flight
    a.stages = stages;
    smem = std::max(sizeof(float) * (size_t)stages * a.chunk, wbytes);
  }
  cudaError_t e = sampler_smem_attr(accept_cluster_kernel, smem, cached);
  if (e != cudaSuccess) return e;
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(a.B * C); cfg.blockDim = dim3(SAMPLER_THREADS); cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = C; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = sps_pdl_enabled() ? 2 : 1;
  return cudaLaunchKernelEx(&cfg, accept_cluster_kernel, a);
}

__global__ void philox_kernel(const uint32_t* ctr, const uint32_t* key, int n, uint32_t* out) {
  const int i = blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  uint32_t w[4];
  philox4x32_10(ctr[4 * i], ctr[4 * i + 1], ctr[4 * i + 2], ctr[4 * i + 3], key[2 * i], key[2 * i + 1], w);
  for (int j = 0; j < 4; ++j) out[4 * i + j] = w[j];
}
cudaError_t philox_launch(const uint32_t* ctr, const uint32_t* key, int n, uint32_t* out, cudaStream_t st) {
  philox_kernel<<<(n + 127) / 128, 128, 0, st>>>(ctr, key, n, out);
  return cudaGetLastError();
}
