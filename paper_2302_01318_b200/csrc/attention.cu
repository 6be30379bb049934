// Row set-up + embedding, and decode attention over the KV cache for 1..16 query rows per sequence
// with rotary positions and the cache append fused in.
//
// Cache layout (per layer): [sequence][key / value head][position][d_head] in the model's storage type, so
// one (sequence, head) CTA streams two contiguous spans.  With fewer key / value heads than query heads
// (grouped-query / multi-query attention) the CTAs of a group read the same spans; each of them rotates
// this pass's keys for itself and the group's first head alone appends them to the cache.  Rejected drafts are never erased: a row only
// ever reads positions <= its own, and the next pass overwrites the stale ones ("rollback" is the
// sequence length moving back, nothing else).
#include <cooperative_groups.h>

#include <cstdlib>

#include "common.cuh"
namespace cg = cooperative_groups;

template <typename CT> struct CacheIO;
template <> struct CacheIO<float> {
  static __device__ __forceinline__ float ld(const float* p) { return *p; }
  static __device__ __forceinline__ void st(float* p, float v) { *p = v; }
};
template <> struct CacheIO<__nv_bfloat16> {
  static __device__ __forceinline__ float ld(const __nv_bfloat16* p) { return __bfloat162float(*p); }
  static __device__ __forceinline__ void st(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }
};

// ------------------------------------------------------------------------------------------------
// rows of a pass: which token sits at which position, x = E[token], and sum(x^2) for the first norm
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) embed_kernel(EmbedArgs a) {
  __shared__ float s_part[8];
  const int row = blockIdx.x, tid = threadIdx.x;
  const int rps = a.rows_per_seq;
  pdl_launch_dependents();
  pdl_wait();
  const int b = row / rps, i = row - b * rps;
  DevState* st = a.st;
  const int max_seq = st->max_seq;
  const int n = st->n[b];
  int tok, pos;
  switch (a.mode) {
    case PASS_PREFILL: pos = a.c0 + i; tok = st->tokens[(long long)b * max_seq + min(pos, max_seq - 1)]; break;
    case PASS_DRAFT0: pos = (i == 0) ? max(n - 2, 0) : n - 1; tok = st->tokens[(long long)b * max_seq + pos]; break;
    case PASS_DRAFT_T: pos = n - 1 + a.t; tok = st->drafts[b * st->max_K + a.t - 1]; break;
    case PASS_VERIFY:
      pos = n - 1 + i;
      tok = (i == 0) ? st->tokens[(long long)b * max_seq + n - 1] : st->drafts[b * st->max_K + i - 1];
      break;
    default: tok = st->row_tok[row]; pos = st->row_pos[row]; break;
  }
  // A sequence of a batch that has reached its length keeps its slot in every pass (the pass has a fixed shape) but
  // no longer matters: its rows are parked on a valid position and raise nothing, whatever its overshoot was.
  const bool dead = a.mode != PASS_PREFILL && a.mode != PASS_EXPLICIT && n >= st->limit[b];
  if (tok < 0 || tok >= a.V) { tok = 0; if (tid == 0 && !dead) atomicExch(st->err, 1); }
  if (pos < 0 || pos >= max_seq) { pos = max(0, min(pos, max_seq - 1)); if (tid == 0 && !dead) atomicExch(st->err, 2); }
  if (tid == 0) { st->row_tok[row] = tok; st->row_pos[row] = pos; }
  float local = 0.f;
  float* xr = a.x + (size_t)row * a.d;
  if (a.dtype == 0) {
    const float* e = reinterpret_cast<const float*>(a.tok_embed) + (size_t)tok * a.d;
    for (int k = tid; k < a.d; k += blockDim.x) { const float v = e[k]; xr[k] = v; local += v * v; }
  } else {
    const __nv_bfloat16* e = reinterpret_cast<const __nv_bfloat16*>(a.tok_embed) + (size_t)tok * a.d;
    for (int k = tid; k < a.d; k += blockDim.x) { const float v = __bfloat162float(e[k]); xr[k] = v; local += v * v; }
  }
  local = warp_sum(local);
  if ((tid & 31) == 0) s_part[tid >> 5] = local;
  __syncthreads();
  if (tid == 0) {
    float t = 0.f;
    for (int w = 0; w < 8; ++w) t += s_part[w];
    a.ssq[SSQ_IDX(0, row)] = t;
  }
}

cudaError_t embed_launch(const EmbedArgs& a, cudaStream_t st) {
  return launch_k(embed_kernel, dim3(a.B * a.rows_per_seq), dim3(256), 0, st, a);
}

// ------------------------------------------------------------------------------------------------
// attention: one CTA per (head, sequence), flash-decoding style.
//
// The cached keys / values of a (sequence, head) are one contiguous span, so a tile of TP positions is
// brought into shared memory by two bulk async copies (one for K, one for V) that are issued before the
// kernel waits for its predecessor: old cache rows do not depend on it.  The rows of this pass (rotary
// applied, rounded to the storage type, appended to the cache) are patched into the tile from shared
// memory, so the tile never depends on reading back what this CTA just wrote.  Per tile: scores with
// one warp per position (lanes split the dims), running max / sum per row (online softmax), then P.V
// with one thread per (pair of dims, position group).  Loops over rows are the only unrolled ones: the code stays small
// enough for the instruction cache, which is what a kernel that runs for microseconds lives or dies by.
// ------------------------------------------------------------------------------------------------
#define ATTN_THREADS 512
#define ATTN_WARPS 16
#define ATTN_TILE_BYTES 32768

__device__ __forceinline__ uint32_t a_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ bool a_mbar_wait(uint32_t bar, uint32_t parity, int* err) {
  unsigned long long t0 = 0;
  for (int spin = 0;; ++spin) {
    uint32_t ok;
    asm volatile(
        "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    if (ok) return true;
    if ((spin & 255) == 255) {
      unsigned long long t;
      asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
      if (t0 == 0) t0 = t;
      else if (t - t0 > 2000000000ull) { atomicExch(err, 3); return false; }
    }
  }
}

template <typename CT> __device__ __forceinline__ float ct_to_f(CT v);
template <> __device__ __forceinline__ float ct_to_f<float>(float v) { return v; }
template <> __device__ __forceinline__ float ct_to_f<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename CT> __device__ __forceinline__ CT f_to_ct(float v);
template <> __device__ __forceinline__ float f_to_ct<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 f_to_ct<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

// position of row i of sequence b in this pass (the same rule as embed_kernel)
__device__ __forceinline__ int row_position(const AttnArgs& a, int b, int i) {
  const DevState* st = a.st;
  const int n = st->n[b];
  int pos;
  switch (a.mode) {
    case PASS_PREFILL: pos = a.c0 + i; break;
    case PASS_DRAFT0: pos = (i == 0) ? max(n - 2, 0) : n - 1; break;
    case PASS_DRAFT_T: pos = n - 1 + a.t; break;
    case PASS_VERIFY: pos = n - 1 + i; break;
    default: pos = st->row_pos[b * a.rows_per_seq + i]; break;
  }
  return max(0, min(pos, a.max_seq - 1));
}

template <int DH, typename CT, int MR>
__global__ void __launch_bounds__(ATTN_THREADS) attn_kernel(AttnArgs a) {
  constexpr int TP = ATTN_TILE_BYTES / (DH * (int)sizeof(CT));   // positions per tile
  constexpr int DPL = DH / 32;                                   // dims per lane in the score phase (4 or 2)
  constexpr int PG = ATTN_THREADS / (DH / 2);                    // position groups in the P.V phase (8 or 16)
  constexpr int LOG_MR = MR == 2 ? 1 : (MR == 8 ? 3 : 4);
  extern __shared__ __align__(128) unsigned char asm_[];
  CT* Ks = reinterpret_cast<CT*>(asm_);                          // [TP][DH]
  CT* Vs = Ks + TP * DH;                                         // [TP][DH]
  CT* knew = Vs + TP * DH;                                       // [MR][DH]  this pass's keys (storage-rounded)
  CT* vnew = knew + MR * DH;                                     // [MR][DH]
  float* q_s = reinterpret_cast<float*>(vnew + MR * DH);         // [MR][DH]
  float* sc = q_s + MR * DH;                                     // [MR][TP]
  float* red = sc + MR * TP;                                     // [PG][MR][DH]
  float* row_m = red + PG * MR * DH;                             // [MR] running max
  float* row_l = row_m + MR;                                     // [MR] running sum
  float* row_a = row_l + MR;                                     // [MR] rescale of this tile
  int* pos_s = reinterpret_cast<int*>(row_a + MR);               // [MR]
  uint64_t* bar = reinterpret_cast<uint64_t*>(pos_s + MR);       // 8-byte aligned by construction
  // split context: the first CTA of the cluster receives every CTA's (max, sum, unnormalised output) here
  float* xo = reinterpret_cast<float*>(bar + 2);                 // [SPLIT][MR][DH]
  float* xm = xo + (size_t)a.split * MR * DH;                    // [SPLIT][MR]
  float* xl = xm + a.split * MR;                                 // [SPLIT][MR]

  // The context of a (head, sequence) may be split over the `split` CTAs of a thread-block cluster (grid z): CTA c
  // attends over positions [c * chunk, (c + 1) * chunk) and the partial results -- running maximum, sum and
  // unnormalised output per query row -- meet in the first CTA's shared memory, where they are merged in CTA order.
  const int SPLIT = a.split, crank = SPLIT > 1 ? (int)cg::this_cluster().block_rank() : 0;
  if (SPLIT > 1) cg::this_cluster().barrier_arrive();   // waited for before the first remote store: by then every CTA runs
  const int h = blockIdx.x, b = a.seq0 + blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int Mb = a.rows_per_seq, row0 = blockIdx.y * Mb, d = a.d, max_seq = a.max_seq;
  const int group = a.H / a.Hkv, hk = h / group;   // the key / value head this query head reads
  const bool appends = (h - hk * group) == 0 && crank == 0;   // one CTA of one head of a group writes the cache
  const int ldq = d + 2 * a.Hkv * DH;                // row stride of the q | k | v buffer
  CT* kc = reinterpret_cast<CT*>(a.kcache) + ((size_t)b * a.Hkv + hk) * (size_t)max_seq * DH;
  CT* vc = reinterpret_cast<CT*>(a.vcache) + ((size_t)b * a.Hkv + hk) * (size_t)max_seq * DH;
  const float scale = rsqrtf((float)DH);
  const uint32_t bar_addr = a_smem_u32(bar);

  if (tid < MR) {
    pos_s[tid] = tid < Mb ? row_position(a, b, tid) : -1;
    row_m[tid] = -INFINITY;
    row_l[tid] = 0.f;
  }
  if (tid == 0) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(bar_addr) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  int n_ctx = 0, n_old = max_seq;
  for (int i = 0; i < Mb; ++i) { n_ctx = max(n_ctx, pos_s[i] + 1); n_old = min(n_old, pos_s[i]); }
  // this CTA's share of the context: [p0, p1) (a multiple of 8 positions per CTA, at least 32)
  int p0 = 0, p1 = n_ctx;
  if (SPLIT > 1) {
    const int chunk = max(32, (((n_ctx + SPLIT - 1) / SPLIT) + 7) & ~7);
    p0 = min(crank * chunk, n_ctx);
    p1 = min(p0 + chunk, n_ctx);
  }
  // Rows [0, n_old) were cached by earlier passes; rows >= n_old of a tile come from knew / vnew.
  // Of the old rows, [0, n_safe) were written before the host last waited for the stream (the host
  // waits once per loop and after the prompt pass), so they may be fetched before this kernel waits
  // for its predecessor; rows written by earlier passes of the SAME loop may not: under programmatic
  // launch only the immediate predecessor is known to be complete, and only after the wait.
  int n_safe = 0;
  if (a.mode == PASS_VERIFY) n_safe = max(a.st->n[b] - 1, 0);
  else if (a.mode == PASS_DRAFT0 || a.mode == PASS_DRAFT_T) n_safe = max(a.st->n[b] - 2, 0);
  n_safe = min(n_safe, n_old);
  auto copy_rows = [&](int t0, int r0, int r1) {   // cache rows [r0, r1) into rows r0 - t0 .. of the tile buffers
    const uint32_t bytes = (uint32_t)(r1 - r0) * DH * (uint32_t)sizeof(CT);
    const int tr = r0 - t0;
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(a_smem_u32(Ks + tr * DH)), "l"(kc + (size_t)r0 * DH), "r"(bytes), "r"(bar_addr) : "memory");
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(a_smem_u32(Vs + tr * DH)), "l"(vc + (size_t)r0 * DH), "r"(bytes), "r"(bar_addr) : "memory");
    return 2 * bytes;
  };
  // the part of the tile that starts at t0 which is fetched after the wait; it also arrives on the tile's barrier
  auto issue_tile = [&](int t0, int from) {
    const int r1 = min(min(t0 + TP, n_old), p1);
    if (r1 > from) {
      const uint32_t bytes = 2u * (uint32_t)(r1 - from) * DH * (uint32_t)sizeof(CT);
      asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar_addr), "r"(bytes) : "memory");
      copy_rows(t0, from, r1);
    } else {
      asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar_addr) : "memory");
    }
  };
  const int pre_end = min(min(p0 + TP, n_safe), p1);   // rows [p0, pre_end) of the first tile are fetched right away
  const int pre = max(pre_end - p0, 0);
  if (tid == 0 && pre > 0) {
    const uint32_t bytes = 2u * (uint32_t)pre * DH * (uint32_t)sizeof(CT);
    asm volatile("mbarrier.expect_tx.relaxed.cta.shared::cta.b64 [%0], %1;" ::"r"(bar_addr), "r"(bytes) : "memory");
    copy_rows(p0, p0, p0 + pre);
  }
  pdl_launch_dependents();
  pdl_wait();
  if (tid == 0 && p1 > p0) issue_tile(p0, p0 + pre);

  // ---- rotary on q and k (adjacent pairs, angle = pos * base^(-2i/dh)); append k, v at the row's position
  for (int idx = tid; idx < Mb * (DH / 2); idx += ATTN_THREADS) {
    const int i = idx / (DH / 2), pr = idx - i * (DH / 2);
    const int pos = pos_s[i];
    const float2 cs = a.rope[(size_t)pos * (DH / 2) + pr];
    const float* src = a.qkv + (size_t)(row0 + i) * ldq;
    const float* ksrc = src + d + hk * DH + 2 * pr;
    const float* vsrc = ksrc + a.Hkv * DH;
    const float q0 = src[h * DH + 2 * pr], q1 = src[h * DH + 2 * pr + 1];
    const float k0 = ksrc[0], k1 = ksrc[1];
    const float v0 = vsrc[0], v1 = vsrc[1];
    q_s[i * DH + 2 * pr] = (q0 * cs.x - q1 * cs.y) * scale;
    q_s[i * DH + 2 * pr + 1] = (q0 * cs.y + q1 * cs.x) * scale;
    const CT ka = f_to_ct<CT>(k0 * cs.x - k1 * cs.y), kb = f_to_ct<CT>(k0 * cs.y + k1 * cs.x);
    const CT va = f_to_ct<CT>(v0), vb = f_to_ct<CT>(v1);
    knew[i * DH + 2 * pr] = ka; knew[i * DH + 2 * pr + 1] = kb;
    vnew[i * DH + 2 * pr] = va; vnew[i * DH + 2 * pr + 1] = vb;
    if (appends) {
      kc[(size_t)pos * DH + 2 * pr] = ka; kc[(size_t)pos * DH + 2 * pr + 1] = kb;
      vc[(size_t)pos * DH + 2 * pr] = va; vc[(size_t)pos * DH + 2 * pr + 1] = vb;
    }
  }
  for (int idx = tid; idx < (MR - Mb) * DH; idx += ATTN_THREADS) q_s[Mb * DH + idx] = 0.f;

  float o[MR][2];   // P.V accumulators: this thread's pair of dims, its position group
#pragma unroll
  for (int i = 0; i < MR; ++i) o[i][0] = o[i][1] = 0.f;
  const int dp = tid % (DH / 2), pg = tid / (DH / 2);
  float qreg[MR][DPL];   // this lane's dims of every query row (score phase)
  bool ok = true;
  int phase = 0;
  for (int t0 = p0; t0 < p1; t0 += TP, phase ^= 1) {
    const int tn = min(TP, p1 - t0);   // positions of this tile
    if (!a_mbar_wait(bar_addr, (uint32_t)phase, a.st->err)) ok = false;
    __syncthreads();   // also: phase A's shared writes are visible
    // patch in the rows of this pass that fall into the tile
    for (int idx = tid; idx < Mb * DH; idx += ATTN_THREADS) {
      const int i = idx / DH, e = idx - i * DH;
      const int j = pos_s[i] - t0;
      if (j >= 0 && j < TP) { Ks[j * DH + e] = knew[idx]; Vs[j * DH + e] = vnew[idx]; }
    }
    if (t0 == p0) {
#pragma unroll
      for (int i = 0; i < MR; ++i)
#pragma unroll
        for (int e = 0; e < DPL; ++e) qreg[i][e] = q_s[i * DH + lane * DPL + e];
    }
    __syncthreads();
    // ---- scores: a warp takes one position at a time, its lanes split the head's dims (the key row is
    // read as one contiguous 32-lane access); the MR partial dot products are summed across lanes with
    // a folding butterfly that halves the values a lane carries at every step.
    for (int j = warp; j < tn; j += ATTN_WARPS) {
      float kf[DPL];
      const CT* kr = Ks + j * DH + lane * DPL;
#pragma unroll
      for (int e = 0; e < DPL; ++e) kf[e] = ct_to_f<CT>(kr[e]);
      float v[MR];
#pragma unroll
      for (int i = 0; i < MR; ++i) {
        float t = 0.f;
#pragma unroll
        for (int e = 0; e < DPL; ++e) t += kf[e] * qreg[i][e];
        v[i] = t;
      }
      int off = 16;
#pragma unroll
      for (int w = MR / 2; w >= 1; w >>= 1, off >>= 1) {
        const bool upper = (lane & off) != 0;
#pragma unroll
        for (int k = 0; k < w; ++k) {
          const float send = upper ? v[k] : v[k + w];
          const float keep = upper ? v[k + w] : v[k];
          v[k] = keep + __shfl_xor_sync(0xffffffffu, send, off);
        }
      }
#pragma unroll
      for (int o2 = 16 >> LOG_MR; o2 >= 1; o2 >>= 1) v[0] += __shfl_xor_sync(0xffffffffu, v[0], o2);
      const int i = lane >> (5 - LOG_MR);   // the row whose sum this lane ended up with
      if ((lane & ((32 >> LOG_MR) - 1)) == 0 && i < Mb) sc[i * TP + j] = (t0 + j <= pos_s[i]) ? v[0] : -INFINITY;
    }
    __syncthreads();
    // ---- online softmax: warp per row
    for (int i = warp; i < Mb; i += ATTN_WARPS) {
      float* srow = sc + i * TP;
      float m = -INFINITY;
      for (int j = lane; j < tn; j += 32) m = fmaxf(m, srow[j]);
      m = warp_max(m);
      const float m_old = row_m[i];
      const float m_new = fmaxf(m_old, m);
      float sum = 0.f;
      for (int j = lane; j < tn; j += 32) {
        const float e = (m_new == -INFINITY) ? 0.f : expf(srow[j] - m_new);
        srow[j] = e;
        sum += e;
      }
      sum = warp_sum(sum);
      if (lane == 0) {
        const float alpha = (m_old == -INFINITY) ? 0.f : expf(m_old - m_new);
        row_a[i] = alpha;
        row_l[i] = row_l[i] * alpha + sum;
        row_m[i] = m_new;
      }
    }
    __syncthreads();
    // ---- o = alpha * o + sum_j p_j v_j: thread = (pair of dims, position group)
#pragma unroll
    for (int i = 0; i < MR; ++i) if (i < Mb) { o[i][0] *= row_a[i]; o[i][1] *= row_a[i]; }
#pragma unroll 4
    for (int j = pg; j < tn; j += PG) {
      const float v0 = ct_to_f<CT>(Vs[j * DH + 2 * dp]), v1 = ct_to_f<CT>(Vs[j * DH + 2 * dp + 1]);
#pragma unroll
      for (int i = 0; i < MR; ++i) {
        if (i < Mb) {
          const float p = sc[i * TP + j];
          o[i][0] += p * v0;
          o[i][1] += p * v1;
        }
      }
    }
    __syncthreads();   // the tile buffers and sc are free again
    if (tid == 0 && t0 + TP < p1) issue_tile(t0 + TP, t0 + TP);
  }
#pragma unroll
  for (int i = 0; i < MR; ++i)
    if (i < Mb) { red[(pg * MR + i) * DH + 2 * dp] = o[i][0]; red[(pg * MR + i) * DH + 2 * dp + 1] = o[i][1]; }
  __syncthreads();
  if (SPLIT > 1) {
    // every CTA's partial result goes to the first CTA of the cluster (distributed shared memory)
    cg::cluster_group cluster = cg::this_cluster();
    cluster.barrier_wait();
    float* rxo = cluster.map_shared_rank(xo, 0) + (size_t)crank * MR * DH;
    for (int idx = tid; idx < Mb * DH; idx += ATTN_THREADS) {
      const int i = idx / DH, e = idx - i * DH;
      float t = 0.f;
#pragma unroll
      for (int g = 0; g < PG; ++g) t += red[(g * MR + i) * DH + e];
      rxo[i * DH + e] = ok ? t : 0.f;
    }
    if (tid < Mb) {
      cluster.map_shared_rank(xm, 0)[crank * MR + tid] = (ok && p1 > p0) ? row_m[tid] : -INFINITY;
      cluster.map_shared_rank(xl, 0)[crank * MR + tid] = (ok && p1 > p0) ? row_l[tid] : 0.f;
    }
    cluster.sync();
    if (crank != 0) return;
    // merge in CTA order: o = sum_c e^(m_c - M) o_c / sum_c e^(m_c - M) l_c
    if (tid < Mb) {
      float M = -INFINITY;
      for (int c = 0; c < SPLIT; ++c) M = fmaxf(M, xm[c * MR + tid]);
      float den = 0.f;
      for (int c = 0; c < SPLIT; ++c) {
        const float mc = xm[c * MR + tid];
        const float w = (mc == -INFINITY) ? 0.f : expf(mc - M);
        xm[c * MR + tid] = w;             // from here on: the CTA's weight
        den += w * xl[c * MR + tid];
      }
      row_l[tid] = den;
    }
    __syncthreads();
  }
  for (int idx = tid; idx < Mb * DH; idx += ATTN_THREADS) {
    const int i = idx / DH, e = idx - i * DH;
    float t = 0.f;
    if (SPLIT > 1) {
      for (int c = 0; c < SPLIT; ++c) t += xm[c * MR + i] * xo[((size_t)c * MR + i) * DH + e];
    } else {
#pragma unroll
      for (int g = 0; g < PG; ++g) t += red[(g * MR + i) * DH + e];
    }
    const float val = (ok && row_l[i] > 0.f) ? t / row_l[i] : 0.f;
    const size_t oi = (size_t)(row0 + i) * d + h * DH + e;
    a.out[oi] = val;
    if (a.out_hi) {
      const __nv_bfloat16 vh = __float2bfloat16_rn(val);
      reinterpret_cast<__nv_bfloat16*>(a.out_hi)[oi] = vh;
      reinterpret_cast<__nv_bfloat16*>(a.out_lo)[oi] = __float2bfloat16_rn(val - __bfloat162float(vh));
    }
  }
}

template <int DH, typename CT, int MR>
static size_t attn_smem_t(int split) {
  constexpr int TP = ATTN_TILE_BYTES / (DH * (int)sizeof(CT));
  constexpr int PG = ATTN_THREADS / (DH / 2);
  return 2 * (size_t)ATTN_TILE_BYTES + 2 * (size_t)MR * DH * sizeof(CT) + sizeof(float) * ((size_t)MR * DH + (size_t)MR * TP + (size_t)PG * MR * DH + 3 * MR) +
         sizeof(int) * MR + 16 + sizeof(float) * (size_t)split * ((size_t)MR * DH + 2 * MR);
}

size_t attn_smem_bytes(int rows_per_seq, int max_seq, int dh) {
  (void)rows_per_seq; (void)max_seq; (void)dh;
  return attn_smem_t<128, float, 16>(1);   // the largest instantiation
}

// CTAs a (head, sequence) is split over: enough to put the SMs to work, as far as the exchange buffer (32 KB) allows
static int attn_split(int heads_x_seqs, int MR, int DH) {
  static const int forced = [] { const char* e = getenv("SPS_ATTN_SPLIT"); return e ? atoi(e) : 0; }();   // tuning: 1 = never split
  int num_sm = SPS_NUM_SM_FALLBACK, dev = 0;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&num_sm, cudaDevAttrMultiProcessorCount, dev);
  int s = num_sm / (heads_x_seqs > 0 ? heads_x_seqs : 1);
  const int cap = 8192 / (MR * DH);        // exchange buffer: split x MR x DH floats <= 32 KB
  if (s > cap) s = cap;
  if (s > 8) s = 8;
  if (forced > 0 && forced < s) s = forced;
  return s < 1 ? 1 : s;
}

template <int DH, typename CT, int MR>
static cudaError_t attn_go(const AttnArgs& a_in, cudaStream_t st) {
  static DevSmemCache cached{};   // per device, like the attribute itself
  AttnArgs a = a_in;
  a.split = attn_split(a.H * a.B, MR, DH);
  const size_t smem = attn_smem_t<DH, CT, MR>(a.split);
  cudaError_t e = sps_ensure_smem(attn_kernel<DH, CT, MR>, smem, cached);
  if (e != cudaSuccess) return e;
  if (a.split == 1) return launch_k(attn_kernel<DH, CT, MR>, dim3(a.H, a.B), dim3(ATTN_THREADS), smem, st, a);
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = dim3(a.H, a.B, a.split); cfg.blockDim = dim3(ATTN_THREADS); cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute at[2];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = 1; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = a.split;
  at[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = sps_pdl_enabled() ? 2 : 1;
  return cudaLaunchKernelEx(&cfg, attn_kernel<DH, CT, MR>, a);
}

template <int DH, typename CT>
static cudaError_t attn_rows(const AttnArgs& a, cudaStream_t st) {
  if (a.rows_per_seq <= 2) return attn_go<DH, CT, 2>(a, st);
  if (a.rows_per_seq <= 8) return attn_go<DH, CT, 8>(a, st);
  return attn_go<DH, CT, 16>(a, st);
}

cudaError_t attn_launch(const AttnArgs& a, cudaStream_t st) {
  if (a.Hkv < 1 || a.H % a.Hkv) return cudaErrorInvalidValue;
  if (a.dh == 64 && a.dtype == 0) return attn_rows<64, float>(a, st);
  if (a.dh == 128 && a.dtype == 0) return attn_rows<128, float>(a, st);
  if (a.dh == 64 && a.dtype == 1) return attn_rows<64, __nv_bfloat16>(a, st);
  if (a.dh == 128 && a.dtype == 1) return attn_rows<128, __nv_bfloat16>(a, st);
  return cudaErrorInvalidValue;
}
