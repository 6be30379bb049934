// Row set-up + embedding, and decode attention over the KV cache for 1..16 query rows per sequence
// with rotary positions and the cache append fused in.
//
// Cache layout (per layer): [sequence][head][position][d_head] in the model's storage type, so one
// (sequence, head) CTA streams two contiguous spans.  Rejected drafts are never erased: a row only
// ever reads positions <= its own, and the next pass overwrites the stale ones ("rollback" is the
// sequence length moving back, nothing else).
#include "common.cuh"

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
  if (tok < 0 || tok >= a.V) { tok = 0; if (tid == 0) atomicExch(st->err, 1); }
  if (pos < 0 || pos >= max_seq) { pos = max(0, min(pos, max_seq - 1)); if (tid == 0) atomicExch(st->err, 2); }
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
    a.ssq[row] = t;
  }
}

cudaError_t embed_launch(const EmbedArgs& a, cudaStream_t st) {
  embed_kernel<<<a.B * a.rows_per_seq, 256, 0, st>>>(a);
  return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// attention: one CTA per (head, sequence)
// ------------------------------------------------------------------------------------------------
#define ATTN_THREADS 256
#define ATTN_WARPS 8

template <int DH, typename CT>
__global__ void __launch_bounds__(ATTN_THREADS) attn_kernel(AttnArgs a) {
  extern __shared__ float sm[];
  const int h = blockIdx.x, b = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int Mb = a.rows_per_seq, row0 = b * Mb, d = a.d, max_seq = a.max_seq;
  float* q_s = sm;                                  // [Mb][DH]
  float* red = q_s + Mb * DH;                       // [ATTN_WARPS][Mb][DH]
  float* inv_sum = red + ATTN_WARPS * Mb * DH;      // [16]
  int* pos_s = reinterpret_cast<int*>(inv_sum + 16);  // [16]
  float* sc = inv_sum + 32;                         // [Mb][max_seq]
  CT* kc = reinterpret_cast<CT*>(a.kcache) + ((size_t)b * a.H + h) * (size_t)max_seq * DH;
  CT* vc = reinterpret_cast<CT*>(a.vcache) + ((size_t)b * a.H + h) * (size_t)max_seq * DH;
  const float scale = rsqrtf((float)DH);

  if (tid < Mb) pos_s[tid] = a.st->row_pos[row0 + tid];
  __syncthreads();
  // ---- rotary on q and k (adjacent pairs, angle = pos * base^(-2i/dh)); append k, v at the row's position
  for (int idx = tid; idx < Mb * (DH / 2); idx += ATTN_THREADS) {
    const int i = idx / (DH / 2), pr = idx - i * (DH / 2);
    const int pos = pos_s[i];
    const float2 cs = a.rope[(size_t)pos * (DH / 2) + pr];
    const float* src = a.qkv + (size_t)(row0 + i) * 3 * d + h * DH + 2 * pr;
    const float q0 = src[0], q1 = src[1];
    const float k0 = src[d], k1 = src[d + 1];
    const float v0 = src[2 * d], v1 = src[2 * d + 1];
    q_s[i * DH + 2 * pr] = (q0 * cs.x - q1 * cs.y) * scale;
    q_s[i * DH + 2 * pr + 1] = (q0 * cs.y + q1 * cs.x) * scale;
    CT* kd = kc + (size_t)pos * DH + 2 * pr;
    CT* vd = vc + (size_t)pos * DH + 2 * pr;
    CacheIO<CT>::st(kd, k0 * cs.x - k1 * cs.y);
    CacheIO<CT>::st(kd + 1, k0 * cs.y + k1 * cs.x);
    CacheIO<CT>::st(vd, v0);
    CacheIO<CT>::st(vd + 1, v1);
  }
  __syncthreads();
  int n_ctx = 0;
  for (int i = 0; i < Mb; ++i) n_ctx = max(n_ctx, pos_s[i] + 1);

  // ---- scores: one thread per cached position, all rows at once
  for (int j = tid; j < n_ctx; j += ATTN_THREADS) {
    float acc[SPS_MAX_ROWS];
#pragma unroll
    for (int i = 0; i < SPS_MAX_ROWS; ++i) acc[i] = 0.f;
    const CT* kr = kc + (size_t)j * DH;
#pragma unroll 2
    for (int c = 0; c < DH; c += 8) {
      float kv[8];
      if (sizeof(CT) == 2) {
        const uint4 raw = *reinterpret_cast<const uint4*>(kr + c);
        const uint32_t w[4] = {raw.x, raw.y, raw.z, raw.w};
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          kv[2 * e] = __uint_as_float(w[e] << 16);
          kv[2 * e + 1] = __uint_as_float(w[e] & 0xffff0000u);
        }
      } else {
        const float4 r0 = *reinterpret_cast<const float4*>(kr + c);
        const float4 r1 = *reinterpret_cast<const float4*>(kr + c + 4);
        kv[0] = r0.x; kv[1] = r0.y; kv[2] = r0.z; kv[3] = r0.w;
        kv[4] = r1.x; kv[5] = r1.y; kv[6] = r1.z; kv[7] = r1.w;
      }
#pragma unroll
      for (int i = 0; i < SPS_MAX_ROWS; ++i) {
        if (i < Mb) {
          const float4 qa = *reinterpret_cast<const float4*>(q_s + i * DH + c);
          const float4 qb = *reinterpret_cast<const float4*>(q_s + i * DH + c + 4);
          acc[i] += kv[0] * qa.x + kv[1] * qa.y + kv[2] * qa.z + kv[3] * qa.w + kv[4] * qb.x + kv[5] * qb.y +
                    kv[6] * qb.z + kv[7] * qb.w;
        }
      }
    }
#pragma unroll
    for (int i = 0; i < SPS_MAX_ROWS; ++i)
      if (i < Mb) sc[(size_t)i * max_seq + j] = (j <= pos_s[i]) ? acc[i] : -INFINITY;
  }
  __syncthreads();
  // ---- softmax over positions, one warp per row
  for (int i = warp; i < Mb; i += ATTN_WARPS) {
    float* s = sc + (size_t)i * max_seq;
    float m = -INFINITY;
    for (int j = lane; j < n_ctx; j += 32) m = fmaxf(m, s[j]);
    m = warp_max(m);
    float sum = 0.f;
    for (int j = lane; j < n_ctx; j += 32) { const float e = expf(s[j] - m); s[j] = e; sum += e; }
    sum = warp_sum(sum);
    if (lane == 0) inv_sum[i] = 1.0f / sum;
  }
  __syncthreads();
  // ---- o = sum_j p_j v_j: a lane owns DH/32 dims, warps split the positions
  constexpr int DPT = DH / 32;
  float o[SPS_MAX_ROWS][DPT];
#pragma unroll
  for (int i = 0; i < SPS_MAX_ROWS; ++i)
#pragma unroll
    for (int e = 0; e < DPT; ++e) o[i][e] = 0.f;
  for (int j = warp; j < n_ctx; j += ATTN_WARPS) {
    float vv[DPT];
    const CT* vr = vc + (size_t)j * DH + lane * DPT;
#pragma unroll
    for (int e = 0; e < DPT; ++e) vv[e] = CacheIO<CT>::ld(vr + e);
#pragma unroll
    for (int i = 0; i < SPS_MAX_ROWS; ++i) {
      if (i < Mb) {
        const float p = sc[(size_t)i * max_seq + j];
#pragma unroll
        for (int e = 0; e < DPT; ++e) o[i][e] += p * vv[e];
      }
    }
  }
#pragma unroll
  for (int i = 0; i < SPS_MAX_ROWS; ++i)
    if (i < Mb)
#pragma unroll
      for (int e = 0; e < DPT; ++e) red[((size_t)warp * Mb + i) * DH + lane * DPT + e] = o[i][e];
  __syncthreads();
  for (int idx = tid; idx < Mb * DH; idx += ATTN_THREADS) {
    const int i = idx / DH, dim = idx - i * DH;
    float t = 0.f;
#pragma unroll
    for (int w = 0; w < ATTN_WARPS; ++w) t += red[((size_t)w * Mb + i) * DH + dim];
    a.out[(size_t)(row0 + i) * d + h * DH + dim] = t * inv_sum[i];
  }
}

size_t attn_smem_bytes(int rows_per_seq, int max_seq, int dh) {
  return sizeof(float) * ((size_t)rows_per_seq * dh + (size_t)ATTN_WARPS * rows_per_seq * dh + 32 +
                          (size_t)rows_per_seq * max_seq);
}

template <int DH, typename CT>
static cudaError_t attn_go(const AttnArgs& a, cudaStream_t st, size_t& cached) {
  const size_t smem = attn_smem_bytes(a.rows_per_seq, a.max_seq, DH);
  if (smem > cached) {
    cudaError_t e = cudaFuncSetAttribute(attn_kernel<DH, CT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    cached = smem;
  }
  attn_kernel<DH, CT><<<dim3(a.H, a.B), ATTN_THREADS, smem, st>>>(a);
  return cudaGetLastError();
}

cudaError_t attn_launch(const AttnArgs& a, cudaStream_t st) {
  static size_t c0 = 48 * 1024, c1 = 48 * 1024, c2 = 48 * 1024, c3 = 48 * 1024;
  if (a.dh == 64 && a.dtype == 0) return attn_go<64, float>(a, st, c0);
  if (a.dh == 128 && a.dtype == 0) return attn_go<128, float>(a, st, c1);
  if (a.dh == 64 && a.dtype == 1) return attn_go<64, __nv_bfloat16>(a, st, c2);
  if (a.dh == 128 && a.dtype == 1) return attn_go<128, __nv_bfloat16>(a, st, c3);
  return cudaErrorInvalidValue;
}
