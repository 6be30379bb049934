// The memory-bound linear layer of the draft steps (M = 1..2) and of the scoring pass (M = K+1):
//   Y[M,N] = f(X)[M,D] W[N,D]^T,  W streamed once from HBM in its caller-owned row-major layout.
//
// bf16 path.  The weights are the 16-row "A" operand of mma.m16n8k16 and the (at most 16) activation
// rows are the narrow "B" side, so the tensor cores only keep the FMA work off the critical path.
// A warp owns a 128-wide slice of the reduction dimension for a whole range of output rows: its slice
// of X is split into bf16 hi + lo parts once (fp32-grade accuracy with bf16 MMAs) and stays in
// registers, while weight rows stream through registers with 128-bit loads, one 16-row tile of
// look-ahead.  A dot product does not care about the order of k, so each lane feeds the 8 consecutive
// bf16 it loaded straight into two MMAs and X uses the same permutation: no shared-memory staging
// or transposes of the weights at all.
// Partial sums meet in three fixed-order steps: the warps of a CTA through shared memory, the CTAs
// that split D through an L2-resident scratch buffer (the last CTA to arrive sums them in split
// order, not arrival order), and -- for the residual epilogue -- the per-range sums of squares that
// the next RMSNorm needs.  No floating-point atomics: results are bit-reproducible.
//
// fp32 path (token-exact parity configuration): one warp per output row, plain FMAs.
#include "common.cuh"

__device__ __forceinline__ uint4 ldg_stream(const void* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w)
               : "l"(p));
  return v;
}

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ void split_pack(float v0, float v1, uint32_t& hi, uint32_t& lo) {
  const __nv_bfloat16 h0 = __float2bfloat16_rn(v0), h1 = __float2bfloat16_rn(v1);
  const __nv_bfloat16 l0 = __float2bfloat16_rn(v0 - __bfloat162float(h0));
  const __nv_bfloat16 l1 = __float2bfloat16_rn(v1 - __bfloat162float(h1));
  hi = (uint32_t)__bfloat16_as_ushort(h0) | ((uint32_t)__bfloat16_as_ushort(h1) << 16);
  lo = (uint32_t)__bfloat16_as_ushort(l0) | ((uint32_t)__bfloat16_as_ushort(l1) << 16);
}

__device__ __forceinline__ float gelu_tanh(float v) {
  return 0.5f * v * (1.0f + tanhf(0.7978845608028654f * (v + 0.044715f * v * v * v)));
}

__device__ __forceinline__ const void* pick_mat(const LinArgs& a, int n, int& row_in_mat) {
  const int rpm = a.rows_per_mat;
  if (n < rpm) { row_in_mat = n; return a.W[0]; }
  if (n < 2 * rpm) { row_in_mat = n - rpm; return a.W[1]; }
  row_in_mat = n - 2 * rpm;
  return a.W[2];
}

// The epilogue, run by the last CTA to finish an output-row range: sum the split-K partials in split
// order and store, or add into the residual stream and accumulate its sum of squares.
__device__ void lin_epilogue(const LinArgs& a, int r, int row_begin, int nrows, float* s_red, int* s_flag) {
  const int tid = threadIdx.x, nthr = blockDim.x, lane = tid & 31, warp = tid >> 5, nwarp = nthr >> 5;
  const int S = a.S, N = a.N;
  for (int m = 0; m < a.M; ++m) {
    float local = 0.f;
    for (int i = tid; i < nrows; i += nthr) {
      const int n = row_begin + i;
      float y = 0.f;
      for (int s = 0; s < S; ++s) y += __ldcg(a.part + ((size_t)s * SPS_MAX_ROWS + m) * N + n);
      float* dst = a.Y + (long long)m * a.ldy + n;
      if (a.epi == EPI_RESIDUAL) {
        y += *dst;
        local += y * y;
      }
      *dst = y;
    }
    if (a.epi == EPI_RESIDUAL) {
      local = warp_sum(local);
      __syncthreads();
      if (lane == 0) s_red[warp] = local;
      __syncthreads();
      if (tid == 0) {
        float t = 0.f;
        for (int w = 0; w < nwarp; ++w) t += s_red[w];
        a.ssq_part[(size_t)r * SPS_MAX_ROWS + m] = t;
      }
    }
  }
  if (tid == 0) a.counters[r] = 0;
  if (a.epi == EPI_RESIDUAL) {
    // the last range to finish adds the per-range sums of squares in range order
    __threadfence();
    __syncthreads();
    if (tid == 0) *s_flag = (atomicAdd(&a.counters[a.R], 1) == a.R - 1);
    __syncthreads();
    if (*s_flag) {
      __threadfence();
      if (tid < a.M) {
        float t = 0.f;
        for (int rr = 0; rr < a.R; ++rr) t += __ldcg(a.ssq_part + (size_t)rr * SPS_MAX_ROWS + tid);
        a.ssq_out[tid] = t;
      }
      if (tid == 0) a.counters[a.R] = 0;
    }
  }
}

template <int NT>
__global__ void __launch_bounds__(NT == 1 ? 512 : 384, 1) lin_bf16_kernel(const LinArgs a) {
  extern __shared__ float red[];  // [WC][8*NT][PR+4]
  __shared__ int s_flag;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, g = lane >> 2, t = lane & 3;
  const int r = blockIdx.x, s = blockIdx.y, WC = a.WC;
  const int k0 = (s * WC + warp) * 128;
  const int row_begin = (int)(((long long)r * a.N) / a.R);
  const int row_end = (int)(((long long)(r + 1) * a.N) / a.R);
  const int nrows = row_end - row_begin;
  const int PR = a.PR, PRp = PR + 4, TP = PR >> 4;
  const int D = a.D;

  // ---- prologue: this warp's slice of X as MMA "B" fragments, bf16 hi and lo parts
  uint32_t xh[NT][4][4], xl[NT][4][4];
#pragma unroll
  for (int nt = 0; nt < NT; ++nt) {
    const int m = nt * 8 + g;
    if (m < a.M) {
      const int srow = a.x_row0 + m * a.x_rowstep;
      const float* src = a.X + (size_t)srow * a.ldx + k0 + 8 * t;
      float scale = 1.f;
      if (a.pro == PRO_RMSNORM) scale = rsqrtf(a.ssq_in[srow] / (float)D + a.eps);
#pragma unroll
      for (int j = 0; j < 4; ++j) {
        const float4 v0 = *reinterpret_cast<const float4*>(src + 32 * j);
        const float4 v1 = *reinterpret_cast<const float4*>(src + 32 * j + 4);
        float v[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
        if (a.pro == PRO_RMSNORM) {
          const float4 g0 = *reinterpret_cast<const float4*>(a.gain + k0 + 8 * t + 32 * j);
          const float4 g1 = *reinterpret_cast<const float4*>(a.gain + k0 + 8 * t + 32 * j + 4);
          const float gg[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
#pragma unroll
          for (int i = 0; i < 8; ++i) v[i] = gg[i] * v[i] * scale;
        } else if (a.pro == PRO_GELU) {
#pragma unroll
          for (int i = 0; i < 8; ++i) v[i] = gelu_tanh(v[i]);
        }
#pragma unroll
        for (int i = 0; i < 4; ++i) split_pack(v[2 * i], v[2 * i + 1], xh[nt][j][i], xl[nt][j][i]);
      }
    } else {
#pragma unroll
      for (int j = 0; j < 4; ++j)
#pragma unroll
        for (int i = 0; i < 4; ++i) { xh[nt][j][i] = 0u; xl[nt][j][i] = 0u; }
    }
  }

  const int ntiles = (nrows + 15) >> 4;
  uint4 A0[4], B0[4], A1[4], B1[4];
  float acc[NT][4];

  auto load_tile = [&](int tile, uint4(&A)[4], uint4(&B)[4]) {
    int ra = row_begin + tile * 16 + g, rb = ra + 8;
    ra = min(ra, row_end - 1);
    rb = min(rb, row_end - 1);
    int ia, ib;
    const __nv_bfloat16* pa = reinterpret_cast<const __nv_bfloat16*>(pick_mat(a, ra, ia));
    const __nv_bfloat16* pb = reinterpret_cast<const __nv_bfloat16*>(pick_mat(a, rb, ib));
    pa += (size_t)ia * D + k0 + 8 * t;
    pb += (size_t)ib * D + k0 + 8 * t;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      A[j] = ldg_stream(pa + 32 * j);
      B[j] = ldg_stream(pb + 32 * j);
    }
  };
  auto compute = [&](const uint4(&A)[4], const uint4(&B)[4]) {
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) { acc[nt][0] = acc[nt][1] = acc[nt][2] = acc[nt][3] = 0.f; }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
#pragma unroll
      for (int nt = 0; nt < NT; ++nt) {
        mma_bf16_16816(acc[nt], A[j].x, B[j].x, A[j].y, B[j].y, xh[nt][j][0], xh[nt][j][1]);
        mma_bf16_16816(acc[nt], A[j].x, B[j].x, A[j].y, B[j].y, xl[nt][j][0], xl[nt][j][1]);
        mma_bf16_16816(acc[nt], A[j].z, B[j].z, A[j].w, B[j].w, xh[nt][j][2], xh[nt][j][3]);
        mma_bf16_16816(acc[nt], A[j].z, B[j].z, A[j].w, B[j].w, xl[nt][j][2], xl[nt][j][3]);
      }
    }
  };
  // per-warp partial tile -> shared memory, transposed ([column][row], pitch PR+4: conflict-free)
  auto store = [&](int tile) {
    const int rl = (tile % TP) * 16 + g;
#pragma unroll
    for (int nt = 0; nt < NT; ++nt) {
      float* base = red + (size_t)(warp * 8 * NT + nt * 8 + 2 * t) * PRp + rl;
      base[0] = acc[nt][0];
      base[PRp] = acc[nt][1];
      base[8] = acc[nt][2];
      base[PRp + 8] = acc[nt][3];
    }
  };
  // end of a shared-memory pass: sum the warps' partials (warp order) into this split's scratch slab
  auto flush = [&](int tile) {
    const int pass_row0 = (tile / TP) * PR;
    const int rows_in_pass = min(PR, nrows - pass_row0);
    __syncthreads();
    const int total = a.M * rows_in_pass;
    for (int idx = tid; idx < total; idx += blockDim.x) {
      const int col = idx / rows_in_pass, rl = idx - col * rows_in_pass;
      float sum = 0.f;
      for (int w = 0; w < WC; ++w) sum += red[(size_t)(w * 8 * NT + col) * PRp + rl];
      a.part[((size_t)s * SPS_MAX_ROWS + col) * a.N + row_begin + pass_row0 + rl] = sum;
    }
    __syncthreads();
  };

  if (ntiles > 0) load_tile(0, A0, B0);
#pragma unroll 1
  for (int tile = 0; tile < ntiles; tile += 2) {
    if (tile + 1 < ntiles) load_tile(tile + 1, A1, B1);
    compute(A0, B0);
    store(tile);
    if ((tile % TP) == TP - 1 || tile == ntiles - 1) flush(tile);
    if (tile + 2 < ntiles) load_tile(tile + 2, A0, B0);
    if (tile + 1 < ntiles) {
      compute(A1, B1);
      store(tile + 1);
      if (((tile + 1) % TP) == TP - 1 || tile + 1 == ntiles - 1) flush(tile + 1);
    }
  }

  // ---- arrival: the last of the S CTAs that split D for this range runs the epilogue
  __threadfence();
  __syncthreads();
  if (tid == 0) s_flag = (atomicAdd(&a.counters[r], 1) == a.S - 1);
  __syncthreads();
  if (!s_flag) return;
  __threadfence();
  lin_epilogue(a, r, row_begin, nrows, red, &s_flag);
}

// ---- fp32 weights: one warp per output row, X (after the prologue) in shared memory ---------------
template <int NT>
__global__ void __launch_bounds__(256) lin_f32_kernel(const LinArgs a) {
  extern __shared__ float xs[];  // [M][D]
  __shared__ float s_ssq[8][SPS_MAX_ROWS];
  __shared__ int s_flag;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int r = blockIdx.x, D = a.D, M = a.M;
  const int row_begin = (int)(((long long)r * a.N) / a.R);
  const int row_end = (int)(((long long)(r + 1) * a.N) / a.R);
  for (int m = 0; m < M; ++m) {
    const int srow = a.x_row0 + m * a.x_rowstep;
    const float* src = a.X + (size_t)srow * a.ldx;
    float scale = 1.f;
    if (a.pro == PRO_RMSNORM) scale = rsqrtf(a.ssq_in[srow] / (float)D + a.eps);
    for (int k = tid; k < D; k += blockDim.x) {
      float v = src[k];
      if (a.pro == PRO_RMSNORM) v = a.gain[k] * v * scale;
      else if (a.pro == PRO_GELU) v = gelu_tanh(v);
      xs[(size_t)m * D + k] = v;
    }
  }
  __syncthreads();
  float ssq[8 * NT];
#pragma unroll
  for (int m = 0; m < 8 * NT; ++m) ssq[m] = 0.f;
  for (int n = row_begin + warp; n < row_end; n += 8) {
    int ri;
    const float* w = reinterpret_cast<const float*>(pick_mat(a, n, ri)) + (size_t)ri * D;
    float acc[8 * NT];
#pragma unroll
    for (int m = 0; m < 8 * NT; ++m) acc[m] = 0.f;
    for (int k = lane; k < D; k += 32) {
      const float wv = __ldg(w + k);
#pragma unroll
      for (int m = 0; m < 8 * NT; ++m)
        if (m < M) acc[m] = fmaf(wv, xs[(size_t)m * D + k], acc[m]);
    }
#pragma unroll
    for (int m = 0; m < 8 * NT; ++m) {
      if (m < M) {
        float y = warp_sum(acc[m]);
        if (lane == 0) {
          float* dst = a.Y + (long long)m * a.ldy + n;
          if (a.epi == EPI_RESIDUAL) { y += *dst; ssq[m] += y * y; }
          *dst = y;
        }
      }
    }
  }
  if (a.epi != EPI_RESIDUAL) return;
  if (lane == 0) {
#pragma unroll
    for (int m = 0; m < 8 * NT; ++m) s_ssq[warp][m] = ssq[m];
  }
  __syncthreads();
  if (tid < M) {
    float t = 0.f;
    for (int w = 0; w < 8; ++w) t += s_ssq[w][tid];
    a.ssq_part[(size_t)r * SPS_MAX_ROWS + tid] = t;
  }
  __threadfence();
  __syncthreads();
  if (tid == 0) s_flag = (atomicAdd(&a.counters[a.R], 1) == a.R - 1);
  __syncthreads();
  if (s_flag) {
    __threadfence();
    if (tid < M) {
      float t = 0.f;
      for (int rr = 0; rr < a.R; ++rr) t += __ldcg(a.ssq_part + (size_t)rr * SPS_MAX_ROWS + tid);
      a.ssq_out[tid] = t;
    }
    if (tid == 0) a.counters[a.R] = 0;
  }
}

// ------------------------------------------------------------------------------------------------
// host side: how a shape is cut into CTAs
// ------------------------------------------------------------------------------------------------
static const size_t kSmemBudget = 200 * 1024;

LinPlan lin_plan(int dtype, int M, int N, int D, int num_sm) {
  LinPlan p{};
  p.NT = (M + 7) / 8;
  if (num_sm <= 0) num_sm = SPS_NUM_SM_FALLBACK;
  if (dtype == 0) {
    p.S = 1; p.WC = 8; p.PR = 0;
    int R = (N + 7) / 8;
    if (R > 2 * num_sm) R = 2 * num_sm;
    if (R > LIN_MAX_R) R = LIN_MAX_R;
    if (R < 1) R = 1;
    p.R = R;
    p.smem = (size_t)M * D * sizeof(float);
    return p;
  }
  const int chunks = D / 128;
  const int wc_max = (p.NT == 1) ? 16 : 12;
  int WC = 1;
  for (int w = 1; w <= wc_max; ++w) if (chunks % w == 0) WC = w;
  p.WC = WC;
  p.S = chunks / WC;
  int R = num_sm / p.S;
  if (R < 1) R = 1;
  const int max_r = (N + 15) / 16;
  if (R > max_r) R = max_r;
  if (R > LIN_MAX_R) R = LIN_MAX_R;
  p.R = R;
  const int rows_max = (N + R - 1) / R + 1;
  int pr_fit = (int)(kSmemBudget / (sizeof(float) * WC * 8 * p.NT)) - 4;
  pr_fit = (pr_fit / 32) * 32;
  int pr_need = ((rows_max + 31) / 32) * 32;
  p.PR = pr_need < pr_fit ? pr_need : pr_fit;
  if (p.PR < 32) p.PR = 32;
  p.smem = sizeof(float) * (size_t)WC * 8 * p.NT * (p.PR + 4);
  return p;
}

size_t lin_part_floats(int N, int S) { return (size_t)S * SPS_MAX_ROWS * (size_t)N; }

template <class Kern>
static cudaError_t ensure_smem(Kern k, size_t bytes, size_t& cached) {
  if (bytes <= cached) return cudaSuccess;
  cudaError_t e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  if (e == cudaSuccess) cached = bytes;
  return e;
}

cudaError_t lin_launch(int dtype, const LinArgs& a_in, const LinPlan& p, cudaStream_t st) {
  LinArgs a = a_in;
  a.R = p.R; a.S = p.S; a.WC = p.WC; a.PR = p.PR;
  static size_t c_b1 = 48 * 1024, c_b2 = 48 * 1024, c_f1 = 48 * 1024, c_f2 = 48 * 1024;
  cudaError_t e;
  if (dtype == 0) {
    if (p.NT == 1) {
      if ((e = ensure_smem(lin_f32_kernel<1>, p.smem, c_f1)) != cudaSuccess) return e;
      lin_f32_kernel<1><<<p.R, 256, p.smem, st>>>(a);
    } else {
      if ((e = ensure_smem(lin_f32_kernel<2>, p.smem, c_f2)) != cudaSuccess) return e;
      lin_f32_kernel<2><<<p.R, 256, p.smem, st>>>(a);
    }
  } else {
    dim3 grid(p.R, p.S);
    if (p.NT == 1) {
      if ((e = ensure_smem(lin_bf16_kernel<1>, p.smem, c_b1)) != cudaSuccess) return e;
      lin_bf16_kernel<1><<<grid, p.WC * 32, p.smem, st>>>(a);
    } else {
      if ((e = ensure_smem(lin_bf16_kernel<2>, p.smem, c_b2)) != cudaSuccess) return e;
      lin_bf16_kernel<2><<<grid, p.WC * 32, p.smem, st>>>(a);
    }
  }
  return cudaGetLastError();
}
