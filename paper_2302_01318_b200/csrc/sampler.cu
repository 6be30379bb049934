// Sampling kernels: the inverse-CDF draw used for draft tokens, and the fused modified rejection
// sampler of Algorithm 2 (accept test, residual resample, extra token) -- one CTA per sequence,
// warp shuffles plus a block prefix sum over the vocabulary.
#include <limits.h>

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
// Top-k and nucleus filtering ("standard sampling methods such as nucleus, top-k sampling and adjusting
// temperature ... modify the probabilities accordingly before applying this rejection sampling scheme",
// section Modified Rejection Sampling).  A row keeps every token whose logit is at least a cut:
//   top-k   : the cut is the k-th largest logit (tokens tied with it stay);
//   nucleus : over what top-k kept, mass Z_k, the largest logit value v such that the tokens with logit
//             >= v hold at least top_p * Z_k.
// Both are "the largest key whose upper tail reaches a target": a radix descent over the order-preserving
// bit pattern of the logit, eight bits per pass, with a 256-bin histogram of the tail function (token
// counts for top-k, weights for the nucleus).  No sort.  Weights enter the histogram as 40-bit fixed
// point integers, so the sums do not depend on the order in which threads add them.
// ------------------------------------------------------------------------------------------------
struct CutSmem {
  unsigned long long bin[256];
  unsigned long long acc;
  unsigned int sel;
  unsigned int found;
};

__device__ __forceinline__ uint32_t order_key(float f) {   // unsigned order of keys == order of the floats
  const uint32_t b = __float_as_uint(f);
  return (b & 0x80000000u) ? ~b : (b | 0x80000000u);
}
__device__ __forceinline__ float order_key_inv(uint32_t k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}
__device__ __forceinline__ unsigned long long fixed40(float w) {   // w in [0, 1]
  return __float2ull_rn(w * 1099511627776.0f);
}

// The largest key K* (among tokens with key >= dom_key) with F(K*) = sum over tokens of key >= K* of f
// reaching `target`; f = 1 (SUM == false) or the token's fixed-point weight.  Returns F(K*) and whether
// such a key exists.  All threads of the block call it; all get the same answer.
template <bool SUM>
__device__ bool tail_descent(const float* row, int V, float m, float invT, uint32_t dom_key, unsigned long long target,
                             CutSmem& cs, uint32_t* key_out, unsigned long long* F_out) {
  const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31, warp = tid >> 5;
  uint32_t prefix = 0, mask = 0;
  unsigned long long acc = 0, at_key = 0;
  for (int pass = 0; pass < 4; ++pass) {
    const int shift = 24 - 8 * pass;
    for (int d = tid; d < 256; d += nthr) cs.bin[d] = 0;
    __syncthreads();
    // a thread adds runs of equal digits locally: in the first passes nearly all tokens share one digit
    int cur = -1;
    unsigned long long loc = 0;
    for (int i = tid; i < V; i += nthr) {
      const float l = row[i];
      const uint32_t k = order_key(l);
      if ((k & mask) != prefix || k < dom_key) continue;
      const int d = (int)((k >> shift) & 255u);
      const unsigned long long f = SUM ? fixed40(expf((l - m) * invT)) : 1ull;
      if (d != cur) {
        if (cur >= 0) atomicAdd(&cs.bin[cur], loc);
        cur = d;
        loc = 0;
      }
      loc += f;
    }
    if (cur >= 0) atomicAdd(&cs.bin[cur], loc);
    __syncthreads();
    if (warp == 0) {
      // lane l owns digits 255 - 8l .. 248 - 8l; the tail above them is a warp prefix sum
      unsigned long long t = 0;
#pragma unroll
      for (int j = 0; j < 8; ++j) t += cs.bin[255 - 8 * lane - j];
      unsigned long long incl = t;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const unsigned long long v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
      }
      const unsigned long long above = acc + (incl - t);
      const bool cross = above < target && above + t >= target;
      const unsigned int who = __ballot_sync(0xffffffffu, cross);
      if (lane == 0) cs.found = who != 0u;
      if (cross) {
        unsigned long long run = above;
        for (int j = 0; j < 8; ++j) {
          const int d = 255 - 8 * lane - j;
          if (run + cs.bin[d] >= target) { cs.sel = (unsigned int)d; cs.acc = run; break; }
          run += cs.bin[d];
        }
      }
    }
    __syncthreads();
    if (!cs.found) return false;   // the whole domain holds less than the target (callers make sure it does not)
    prefix |= cs.sel << shift;
    mask |= 255u << shift;
    acc = cs.acc;
    at_key = cs.bin[cs.sel];
    __syncthreads();
  }
  *key_out = prefix;
  *F_out = acc + at_key;
  return true;
}

// sum over tokens with key >= dom_key of the fixed-point weight
__device__ unsigned long long tail_mass(const float* row, int V, float m, float invT, uint32_t dom_key, CutSmem& cs) {
  const int tid = threadIdx.x, nthr = blockDim.x;
  if (tid == 0) cs.acc = 0;
  __syncthreads();
  unsigned long long loc = 0;
  for (int i = tid; i < V; i += nthr) {
    const float l = row[i];
    if (order_key(l) >= dom_key) loc += fixed40(expf((l - m) * invT));
  }
  loc += __shfl_xor_sync(0xffffffffu, loc, 16);
  loc += __shfl_xor_sync(0xffffffffu, loc, 8);
  loc += __shfl_xor_sync(0xffffffffu, loc, 4);
  loc += __shfl_xor_sync(0xffffffffu, loc, 2);
  loc += __shfl_xor_sync(0xffffffffu, loc, 1);
  if ((tid & 31) == 0) atomicAdd(&cs.acc, loc);
  __syncthreads();
  const unsigned long long z = cs.acc;
  __syncthreads();
  return z;
}

// The cut of one row and the mass it keeps (sum of exp((l - m) / T) over kept tokens).  m = the row's maximum.
__device__ void row_cut(const float* row, int V, float m, float invT, int top_k, float top_p, CutSmem& cs,
                        float* cut_out, float* mass_out) {
  uint32_t key = 0;   // keep everything
  unsigned long long F = 0;
  if (top_k >= 1 && top_k < V) {
    if (!tail_descent<false>(row, V, m, invT, 0u, (unsigned long long)top_k, cs, &key, &F)) key = 0;
  }
  unsigned long long Z = tail_mass(row, V, m, invT, key, cs);
  if (top_p < 1.0f) {
    unsigned long long target = (unsigned long long)((double)top_p * (double)Z);
    if (target < 1ull) target = 1ull;
    uint32_t kp;
    unsigned long long Fp;
    if (target <= Z && tail_descent<true>(row, V, m, invT, key, target, cs, &kp, &Fp)) { key = kp; Z = Fp; }
  }
  *cut_out = key == 0u ? -INFINITY : order_key_inv(key);
  *mass_out = (float)((double)Z * (1.0 / 1099511627776.0));
}

// ------------------------------------------------------------------------------------------------
// x ~ softmax(logits / T) by inverse CDF with u_draft(b, s, t)  (Algorithm 2: "sample draft
// auto-regressively"; with t = 0 and u_res it is Algorithm 1's sample).
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
  if (a.st) { T = a.st->temperature; seed = a.st->seed; step = a.st->step; top_k = a.st->top_k; top_p = a.st->top_p; }
  const float invT = 1.0f / T;
  const float* row = a.logits + (long long)b * a.ld;
  const Uniforms u = sps_uniforms(seed, (uint32_t)b, step, a.t);
  int tok;
  if ((top_k >= 1 && top_k < a.V) || top_p < 1.0f) {
    // filtered draw: tokens under the cut weigh nothing
    float m = -INFINITY;
    for (int i = threadIdx.x; i < a.V; i += blockDim.x) m = fmaxf(m, row[i]);
    m = block_max_f(m, s_part, &s_val);
    float cut, mass;
    row_cut(row, a.V, m, invT, top_k, top_p, cs, &cut, &mass);
    auto w = [&](int i) { const float l = row[i]; return l >= cut ? expf((l - m) * invT) : 0.f; };
    if (a.smem_weights) {
      extern __shared__ float ws[];
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
    tok = block_invcdf_smem(ws, a.V, u.u_draft, sm, nullptr);
  } else {
    float m = -INFINITY;
    for (int i = threadIdx.x; i < a.V; i += blockDim.x) m = fmaxf(m, row[i]);
    m = block_max_f(m, s_part, &s_val);
    if (a.smem_weights) {
      extern __shared__ float ws[];
      for (int i = threadIdx.x; i < a.V; i += blockDim.x) ws[skew(i)] = expf((row[i] - m) * invT);
      __syncthreads();
      tok = block_invcdf_smem(ws, a.V, u.u_draft, sm, nullptr);
    } else {
      auto w = [&](int i) { return expf((row[i] - m) * invT); };
      tok = block_invcdf(w, a.V, u.u_draft, sm, nullptr);
    }
  }
  if (threadIdx.x == 0) a.out[(long long)b * a.out_ld] = tok;
}

// bytes of the shared weight buffer for a vocabulary, or 0 when it does not fit (weights are then recomputed)
static size_t weights_smem(int V) {
  const size_t bytes = sizeof(float) * ((size_t)V + (size_t)V / 32 + 32);
  return bytes <= 200 * 1024 ? bytes : 0;
}
template <class Kern>
static cudaError_t sampler_smem_attr(Kern k, size_t bytes, size_t& cached) {
  if (bytes <= cached) return cudaSuccess;
  cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  if (e == cudaSuccess) cached = bytes;
  return e;
}

cudaError_t sample_launch(const SampleArgs& a_in, cudaStream_t st) {
  static size_t cached = 48 * 1024;
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
  if (a.st) { T = a.st->temperature; seed = a.st->seed; step = a.st->step; top_k = a.st->top_k; top_p = a.st->top_p; }
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
    row_cut(rowptr(r), V, s_max[r], invT, top_k, top_p, cs, &cut, &mass);
    if (tid == 0) { s_cut[r] = cut; s_sum[r] = mass; }
    __syncthreads();
  };

  // ---- phase 2: accept chain, left to right
  const int32_t* drafts = a.drafts + (long long)b * a.drafts_ld;
  auto accept_at = [&](int t) {   // thread 0: does draft t pass?
    int d = drafts[t];
    if (d < 0 || d >= V) { d = 0; if (a.st) atomicExch(a.st->err, 1); }
    const float lq = qrow[(long long)t * V + d], lp = prow[(long long)t * V + d];
    const float qd = lq >= s_cut[t] ? expf((lq - s_max[t]) * invT) / s_sum[t] : 0.f;
    const float pd = lp >= s_cut[K + 1 + t] ? expf((lp - s_max[K + 1 + t]) * invT) / s_sum[K + 1 + t] : 0.f;
    // accept with probability min(1, q(d)/p(d)); p == 0 with q > 0 accepts, 0/0 rejects
    const float ratio = (pd > 0.f) ? fminf(1.0f, qd / pd) : (qd > 0.f ? 1.0f : 0.0f);
    const Uniforms u = sps_uniforms(seed, (uint32_t)b, step, (uint32_t)t);
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
    const Uniforms u = sps_uniforms(seed, (uint32_t)b, step, (uint32_t)stop);
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
    const Uniforms u = sps_uniforms(seed, (uint32_t)b, step, (uint32_t)K);
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

cudaError_t accept_launch(const AcceptArgs& a_in, cudaStream_t st) {
  static size_t cached = 48 * 1024;
  AcceptArgs a = a_in;
  const size_t smem = weights_smem(a.V);
  a.smem_weights = smem ? 1 : 0;
  cudaError_t e = sampler_smem_attr(accept_kernel, smem, cached);
  if (e != cudaSuccess) return e;
  return launch_k(accept_kernel, dim3(a.B), dim3(SAMPLER_THREADS), smem, st, a);
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
