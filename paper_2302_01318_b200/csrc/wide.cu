// Passes with many rows as a real GEMM: 9 .. 128 activation rows at once on the 5th-generation tensor cores.
//
// The decode kernels (linear.cu) stream every weight once per <= 16 rows, which is right for the loop's usual
// 1 .. K+1 rows and wrong for a prompt (127 prompt rows would cost eight full sweeps over the weights) or for
// a batch of sequences.  Here Y[M, N] = X[M, D] W[N, D]^T runs as tcgen05.mma (cta_group::1, M = 128 -- or 64
// when the pass has at most 64 rows --, N = 256, K = 16, bf16 operands, fp32 accumulators in tensor memory):
//
//   * grid = (tiles of 256 weight rows, over up to three stacked matrices q | k | v) x (S k-splits);
//   * warp 0 (one lane) is the copy producer: per 64-wide k-block one TMA box of W (256 rows x 128 B) and one
//     each of the activations' high and low bf16 halves (128 or 64 rows x 128 B), 128-byte swizzle, into a ring
//     of 3 (4) stages of 64 (48) KB guarded by full / empty mbarriers; the first ring-full of W boxes is
//     asked for before the kernel waits for its predecessor (weights are constants);
//   * warp 1 (one lane) issues the MMAs: 4 k-steps x (high, low) per k-block -- the two halves make the
//     activations exact to ~16 bits as in the decode kernels -- into two accumulators (all 512 columns of
//     tensor memory: high-half products and low-half products are summed apart and added once at the end),
//     and releases the stage with tcgen05.commit;
//   * warps 2..5 read the accumulators back with tcgen05.ld once the last commit has landed (warp w owns
//     tensor-memory lanes 32 (w % 4) ..).  With one k-split they finish the layer themselves (store / add
//     to the residual stream / GeLU + split into bf16 halves, int8 row scales); otherwise they write the
//     CTA's partial tile and wide_epilogue_kernel adds the k-splits in a fixed order and does the same.
//
// Per weight byte the activations cost one byte of L2 traffic (128 rows x 2 halves x 2 B per 256 weight
// rows), so the pass stays bound by the weight stream from HBM up to 64 rows and by the tensor pipe above.
// Every wait is bounded (2 s of %globaltimer): on expiry the CTA records error 3, lets its copies land, frees
// its tensor memory and returns.  No multicast, no clusters.
#include "common.cuh"

#include <cuda.h>
#include <cudaTypedefs.h>

#include <map>
#include <mutex>
#include <tuple>

namespace {

constexpr int WIDE_M = 128;        // activation rows of one pass (tensor-memory lanes)
constexpr int WIDE_BN = 256;       // weight rows per CTA (tensor-memory columns)
constexpr int WIDE_BK = 64;        // k per stage: 128 bytes of bf16 = one swizzle row
constexpr uint32_t WIDE_B_BYTES = WIDE_BN * WIDE_BK * 2;    // 32 KB
// MR = rows the MMA carries: 128, or 64 for passes of up to 64 rows (half the tensor work, a fourth stage in the ring)
template <int MR> struct WideCfg {
  static constexpr int STAGES = MR == 64 ? 4 : 3;
  static constexpr uint32_t A_BYTES = MR * WIDE_BK * 2;     // 16 KB (8 KB) per half
  static constexpr uint32_t STAGE_BYTES = 2 * A_BYTES + WIDE_B_BYTES;
  static constexpr size_t SMEM = 1024 + (size_t)STAGES * STAGE_BYTES + 1024;   // header + ring + alignment slack
  // kind::f16 instruction descriptor: fp32 accumulator, bf16 x bf16, both operands K-major, N = 256, M = MR
  static constexpr uint32_t IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(WIDE_BN >> 3) << 17) | ((uint32_t)(MR >> 4) << 24);
};

__device__ __forceinline__ uint32_t w_smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ unsigned long long w_timer() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void w_mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void w_mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint32_t w_mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}
// bounded wait: false (and error word 3) after limit_ns of the global timer (2 s unless a test shortened it)
__device__ __forceinline__ bool w_mbar_wait(uint32_t bar, uint32_t parity, int* err, unsigned long long limit_ns) {
  if (w_mbar_try(bar, parity)) return true;
  const unsigned long long t0 = w_timer();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 128; ++i)
      if (w_mbar_try(bar, parity)) return true;
    if (w_timer() - t0 > limit_ns) {
      atomicExch(err, 3);
      return false;
    }
  }
}
__device__ __forceinline__ void w_tma_2d(uint32_t dst, const CUtensorMap* tm, int c0, int c1, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(tm), "r"(c0), "r"(c1), "r"(bar)
      : "memory");
}

// Shared-memory operand descriptor for a K-major tile whose rows are 128 bytes (64 bf16) under the
// 128-byte swizzle: groups of 8 rows are 1024 bytes apart (stride offset), the leading offset is unused,
// descriptor version 1, layout type 2 (128-byte swizzle).  Stepping 16 elements along k inside the
// swizzle row adds 32 bytes to the start address.
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3ffffu) >> 4);
  d |= (uint64_t)1 << 16;                       // leading byte offset (ignored for swizzled K-major)
  d |= (uint64_t)(1024 >> 4) << 32;             // stride byte offset: 8 rows x 128 B
  d |= (uint64_t)1 << 46;                       // descriptor version
  d |= (uint64_t)2 << 61;                       // 128-byte swizzle
  return d;
}
__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
      " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// arrives on the barrier once every MMA issued so far by this thread has finished reading its operands
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]),
        "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]),
        "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

__device__ __forceinline__ float wide_gelu_dev(float v) {
  return 0.5f * v * (1.0f + tanhf(0.7978845608028654f * (v + 0.044715f * v * v * v)));
}
__device__ __forceinline__ uint2 wide_split4_dev(const float4& v, uint2& lo) {
  const float f[4] = {v.x, v.y, v.z, v.w};
  uint32_t h[4], l[4];
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const __nv_bfloat16 hb = __float2bfloat16_rn(f[i]);
    h[i] = __bfloat16_as_ushort(hb);
    l[i] = __bfloat16_as_ushort(__float2bfloat16_rn(f[i] - __bfloat162float(hb)));
  }
  lo = make_uint2(l[0] | (l[1] << 16), l[2] | (l[3] << 16));
  return make_uint2(h[0] | (h[1] << 16), h[2] | (h[3] << 16));
}

struct WideGemmArgs {
  CUtensorMap tm_hi, tm_lo, tm_w[3];   // up to three stacked weight matrices (q | k | v): output columns side by side
  int rows_mat[3], tiles_mat[3];       // rows of each matrix and its tiles of 256 rows (0 for unused slots)
  float* part;        // [S][128][N] partial products of the k-splits
  int M, N, D, S;     // live rows, weight rows of all matrices together, width, k-splits (D / 64 is a multiple of S)
  int w_is_output;    // the weights were written by the predecessor kernel (bf16 copy of int8 weights): no early fetch
  // one k-split: the epilogue warps finish the layer themselves (mode WIDE_EPI_*; scale: int8 row scales per matrix)
  int fused, mode, vec, ldp;
  float* y;
  long long ldy;
  __nv_bfloat16 *yhi, *ylo;
  const float* scale[3];
  int* err;
  unsigned long long wait_ns;   // bound of every wait inside the kernel
  int drop_stage;               // >= 0: CTA (0, 0)'s producer leaves out that k-block (test hook); -1 = none
};

template <int MR>
__global__ void __launch_bounds__(192, 1) wide_gemm_kernel(const __grid_constant__ WideGemmArgs a) {
  constexpr int WIDE_STAGES = WideCfg<MR>::STAGES;
  constexpr uint32_t WIDE_A_BYTES = WideCfg<MR>::A_BYTES, WIDE_STAGE_BYTES = WideCfg<MR>::STAGE_BYTES;
  extern __shared__ unsigned char wsm_raw[];
  // header: full[3], empty[3], accumulator-ready barrier, tensor-memory base, abort flag; ring 1024-aligned
  const uint32_t raw = w_smem_u32(wsm_raw);
  const uint32_t base = (raw + 1023u) & ~1023u;
  unsigned char* hdr = wsm_raw + (base - raw);
  const uint32_t bar_full = base, bar_empty = base + 64, bar_acc = base + 128;
  volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(hdr + 192);
  volatile int* s_abort = reinterpret_cast<volatile int*>(hdr + 200);
  const uint32_t ring = base + 1024;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int tile = blockIdx.x, s = blockIdx.y;
  const int kb_all = a.D / WIDE_BK, kb_n = kb_all / a.S, kb0 = s * kb_n;
  // which matrix this tile belongs to, its first row there, and its first column of the stacked output
  int mat = 0, ltile = tile, col0 = 0;
  while (mat < 2 && ltile >= a.tiles_mat[mat]) { ltile -= a.tiles_mat[mat]; col0 += a.rows_mat[mat]; ++mat; }
  const int wrow0 = ltile * WIDE_BN;
  const CUtensorMap* tm_w = &a.tm_w[mat];

  if (tid == 0) {
    for (int i = 0; i < WIDE_STAGES; ++i) { w_mbar_init(bar_full + 8 * i, 1); w_mbar_init(bar_empty + 8 * i, 1); }
    w_mbar_init(bar_acc, 1);
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    // all 512 columns of tensor memory: two 128 x 256 fp32 accumulators, one for the products of the activations'
    // high halves and one for the low halves' (one CTA per SM: always available).  Kept apart, the small low-half
    // products are not rounded against the large running sum at every step; the epilogue adds the two once.
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(base + 192), "r"(2 * WIDE_BN) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = *s_tmem;
  // Weights do not depend on the predecessor kernel: the first ring-full of W boxes is on its way before the wait;
  // the activations are the predecessor's output and follow after it.
  const int pre = a.w_is_output ? 0 : (kb_n < WIDE_STAGES ? kb_n : WIDE_STAGES);
  if (warp == 0 && lane == 0) {
    for (int kb = 0; kb < pre; ++kb) {
      w_mbar_expect_tx(bar_full + 8 * kb, WIDE_STAGE_BYTES);
      w_tma_2d(ring + kb * WIDE_STAGE_BYTES + 2 * WIDE_A_BYTES, tm_w, (kb0 + kb) * WIDE_BK, wrow0, bar_full + 8 * kb);
    }
  }
  pdl_launch_dependents();
  pdl_wait();

  if (warp == 0) {
    if (lane == 0) {
      bool ok = true;
      int issued = 0;
      for (int kb = 0; kb < kb_n && ok; ++kb, ++issued) {
        const int st = kb % WIDE_STAGES, use = kb / WIDE_STAGES;
        if (use > 0 && !w_mbar_wait(bar_empty + 8 * st, (uint32_t)(use - 1) & 1u, a.err, a.wait_ns)) { ok = false; break; }
        if (*s_abort) { ok = false; break; }
        if (tile == 0 && s == 0 && kb >= pre && kb == a.drop_stage) continue;   // test hook: nothing is asked for, the MMA warp's wait runs out
        const uint32_t dst = ring + st * WIDE_STAGE_BYTES;
        const int k = (kb0 + kb) * WIDE_BK;
        if (kb >= pre) w_mbar_expect_tx(bar_full + 8 * st, WIDE_STAGE_BYTES);
        w_tma_2d(dst, &a.tm_hi, k, 0, bar_full + 8 * st);
        w_tma_2d(dst + WIDE_A_BYTES, &a.tm_lo, k, 0, bar_full + 8 * st);
        if (kb >= pre) w_tma_2d(dst + 2 * WIDE_A_BYTES, tm_w, k, wrow0, bar_full + 8 * st);
      }
      if (!ok) {
        *s_abort = 1;
        // let the copies already issued land before this CTA's shared memory goes away
        for (int j = max(0, issued - WIDE_STAGES); j < issued; ++j)
          if (!(tile == 0 && s == 0 && j >= pre && j == a.drop_stage))
            w_mbar_wait(bar_full + 8 * (j % WIDE_STAGES), (uint32_t)(j / WIDE_STAGES) & 1u, a.err, a.wait_ns);
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {
      bool ok = true;
      for (int kb = 0; kb < kb_n && ok; ++kb) {
        const int st = kb % WIDE_STAGES, use = kb / WIDE_STAGES;
        if (!w_mbar_wait(bar_full + 8 * st, (uint32_t)use & 1u, a.err, a.wait_ns) || *s_abort) { ok = false; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t sa = ring + st * WIDE_STAGE_BYTES;
        const uint64_t d_hi = umma_desc(sa), d_lo = umma_desc(sa + WIDE_A_BYTES), d_w = umma_desc(sa + 2 * WIDE_A_BYTES);
#pragma unroll
        for (int k = 0; k < WIDE_BK / 16; ++k) {
          // 16 elements along k = 32 bytes = 2 units of the descriptor's address field
          umma_bf16(tmem, d_hi + 2 * k, d_w + 2 * k, WideCfg<MR>::IDESC, (kb > 0 || k > 0) ? 1u : 0u);
          umma_bf16(tmem + WIDE_BN, d_lo + 2 * k, d_w + 2 * k, WideCfg<MR>::IDESC, (kb > 0 || k > 0) ? 1u : 0u);
        }
        umma_commit(bar_empty + 8 * st);   // the stage is free once these MMAs have read it
      }
      if (ok) umma_commit(bar_acc);         // ... and the accumulator is complete once all of them are done
      else *s_abort = 1;
    }
  } else {
    // epilogue warps 2..5: tensor-memory lanes 32 q .. 32 q + 31 with q = warp % 4.  A 128-row accumulator keeps row i
    // in lane i; a 64-row one keeps 16 rows in the first 16 lanes of each of the four lane quarters.
    const int q = warp & 3, row = MR == 128 ? q * 32 + lane : (lane < 16 ? q * 16 + lane : WIDE_M);
    bool ok = w_mbar_wait(bar_acc, 0u, a.err, a.wait_ns) && !*s_abort;
    ok = __all_sync(0xffffffffu, ok);
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    if (ok) {
      float* dst = a.part + ((size_t)s * WIDE_M + row) * a.N + (size_t)(col0 + wrow0);
      const int ncols = min(WIDE_BN, a.rows_mat[mat] - wrow0);
#pragma unroll 1
      for (int c = 0; c < WIDE_BN; c += 32) {
        float v[32], vl[32];
        tmem_ld32(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)c, v);   // the whole warp takes part in the loads
        tmem_ld32(tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)(WIDE_BN + c), vl);
#pragma unroll
        for (int i = 0; i < 32; ++i) v[i] += vl[i];
        if (row < a.M && c < ncols && a.fused) {
          // no other k-split: store / add to the residual stream / GeLU + split right here
          const int lim = min(32, ncols - c), cn = col0 + wrow0 + c;
          if (a.scale[0]) {
            const float* sc = a.scale[mat] + wrow0 + c;
#pragma unroll
            for (int i = 0; i < 32; ++i) if (i < lim) v[i] *= __ldg(sc + i);
          }
          if (a.mode == 2) {
#pragma unroll
            for (int i = 0; i < 32; ++i) v[i] = wide_gelu_dev(v[i]);
          }
          const bool full = lim == 32 && a.vec;
          if (a.mode == 0) {
            float* yp = a.y + row * a.ldy + cn;
            if (full) {
#pragma unroll
              for (int i = 0; i < 32; i += 4) *reinterpret_cast<float4*>(yp + i) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
            } else {
              for (int i = 0; i < lim; ++i) yp[i] = v[i];
            }
          } else if (a.mode == 1) {
            float* yp = a.y + row * a.ldy + cn;
            for (int i = 0; i < lim; ++i) yp[i] += v[i];
          } else {
            __nv_bfloat16* hp = a.yhi + (size_t)row * a.ldp + cn;
            __nv_bfloat16* lp = a.ylo + (size_t)row * a.ldp + cn;
            if (full) {
#pragma unroll
              for (int i = 0; i < 32; i += 4) {
                uint2 l;
                const uint2 h = wide_split4_dev(make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]), l);
                *reinterpret_cast<uint2*>(hp + i) = h;
                *reinterpret_cast<uint2*>(lp + i) = l;
              }
            } else {
              for (int i = 0; i < lim; ++i) {
                const __nv_bfloat16 h = __float2bfloat16_rn(v[i]);
                hp[i] = h;
                lp[i] = __float2bfloat16_rn(v[i] - __bfloat162float(h));
              }
            }
          }
        } else if (row < a.M && c < ncols) {
          if (c + 32 <= ncols && ((a.N | col0) & 3) == 0) {
#pragma unroll
            for (int i = 0; i < 32; i += 4) *reinterpret_cast<float4*>(dst + c + i) = make_float4(v[i], v[i + 1], v[i + 2], v[i + 3]);
          } else {
            for (int i = 0; i < 32 && c + i < ncols; ++i) dst[c + i] = v[i];
          }
        }
      }
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(2 * WIDE_BN) : "memory");
  }
}

}  // namespace

// ------------------------------------------------------------------------------------------------
// Elementwise companions of the GEMM (all rows x features, memory-bound, a few microseconds each)
// ------------------------------------------------------------------------------------------------
namespace {

__device__ __forceinline__ void wide_split(float v, __nv_bfloat16& hi, __nv_bfloat16& lo) {
  hi = __float2bfloat16_rn(v);
  lo = __float2bfloat16_rn(v - __bfloat162float(hi));
}
__device__ __forceinline__ float wide_gelu(float v) {
  return 0.5f * v * (1.0f + tanhf(0.7978845608028654f * (v + 0.044715f * v * v * v)));
}

// x[row] = E[token at position c0 + row of sequence seq] for the rows of one prompt chunk
__global__ void __launch_bounds__(256) wide_embed_kernel(const DevState* st, const __nv_bfloat16* tok_embed, float* x, int d, int V, int seq,
                                                         int c0) {
  pdl_wait();
  pdl_launch_dependents();
  const int row = blockIdx.x;
  int tok = st->tokens[(long long)seq * st->max_seq + c0 + row];
  if (tok < 0 || tok >= V) { tok = 0; if (threadIdx.x == 0) atomicExch(st->err, 1); }
  const __nv_bfloat16* e = tok_embed + (size_t)tok * d;
  for (int k = threadIdx.x; k < d; k += blockDim.x) x[(size_t)row * d + k] = __bfloat162float(e[k]);
}

__device__ __forceinline__ uint2 wide_split4(const float4& v, uint2& lo) {
  __nv_bfloat16 h[4], l[4];
  wide_split(v.x, h[0], l[0]); wide_split(v.y, h[1], l[1]); wide_split(v.z, h[2], l[2]); wide_split(v.w, h[3], l[3]);
  uint2 hi;
  hi.x = (uint32_t)__bfloat16_as_ushort(h[0]) | ((uint32_t)__bfloat16_as_ushort(h[1]) << 16);
  hi.y = (uint32_t)__bfloat16_as_ushort(h[2]) | ((uint32_t)__bfloat16_as_ushort(h[3]) << 16);
  lo.x = (uint32_t)__bfloat16_as_ushort(l[0]) | ((uint32_t)__bfloat16_as_ushort(l[1]) << 16);
  lo.y = (uint32_t)__bfloat16_as_ushort(l[2]) | ((uint32_t)__bfloat16_as_ushort(l[3]) << 16);
  return hi;
}

// one CTA of 1024 threads per row: (optionally) RMS-normalise with the gain, then split into bf16 high and low halves;
// four features per thread and step when the widths allow (the second sweep over the row hits L1)
__global__ void __launch_bounds__(1024) wide_pack_kernel(const float* x, int ldx, const float* gain, float eps, int d,
                                                         __nv_bfloat16* hi, __nv_bfloat16* lo, int ldp) {
  __shared__ float s_part[32];
  __shared__ float s_inv;
  pdl_wait();
  pdl_launch_dependents();
  const int row = blockIdx.x, tid = threadIdx.x, nth = blockDim.x;
  const float* xr = x + (size_t)row * ldx;
  const bool vec = (((d | ldx | ldp) & 3) == 0) && ((((uintptr_t)x | (uintptr_t)hi | (uintptr_t)lo | (uintptr_t)gain) & 15) == 0);
  float inv = 1.f;
  if (gain) {
    float local = 0.f;
    if (vec) {
      for (int q = tid; q < (d >> 2); q += nth) {
        const float4 v = reinterpret_cast<const float4*>(xr)[q];
        local += (v.x * v.x + v.y * v.y) + (v.z * v.z + v.w * v.w);
      }
    } else {
      for (int k = tid; k < d; k += nth) { const float v = xr[k]; local += v * v; }
    }
    local = warp_sum(local);
    if ((tid & 31) == 0) s_part[tid >> 5] = local;
    __syncthreads();
    if (tid == 0) {
      float t = 0.f;
      for (int w = 0; w < (nth >> 5); ++w) t += s_part[w];
      s_inv = rsqrtf(t / (float)d + eps);
    }
    __syncthreads();
    inv = s_inv;
  }
  if (vec) {
    for (int q = tid; q < (d >> 2); q += nth) {
      float4 v = reinterpret_cast<const float4*>(xr)[q];
      if (gain) {
        const float4 g = __ldg(reinterpret_cast<const float4*>(gain) + q);
        v.x = g.x * (v.x * inv); v.y = g.y * (v.y * inv); v.z = g.z * (v.z * inv); v.w = g.w * (v.w * inv);
      }
      uint2 l;
      const uint2 h = wide_split4(v, l);
      reinterpret_cast<uint2*>(hi + (size_t)row * ldp)[q] = h;
      reinterpret_cast<uint2*>(lo + (size_t)row * ldp)[q] = l;
    }
  } else {
    for (int k = tid; k < d; k += nth) {
      const float v = gain ? gain[k] * (xr[k] * inv) : xr[k];
      __nv_bfloat16 h, l;
      wide_split(v, h, l);
      hi[(size_t)row * ldp + k] = h;
      lo[(size_t)row * ldp + k] = l;
    }
  }
}

enum { WIDE_EPI_STORE = 0, WIDE_EPI_RESIDUAL = 1, WIDE_EPI_GELU_PACK = 2 };

// int8 weights take this GEMM through a bf16 copy (signed bytes are exact in bf16); the rows' scales multiply the sums
__global__ void __launch_bounds__(256) wide_dequant_kernel(const int8_t* q, __nv_bfloat16* out, long long n16) {
  pdl_wait();
  pdl_launch_dependents();
  for (long long i = (long long)blockIdx.x * 256 + threadIdx.x; i < n16; i += (long long)gridDim.x * 256) {
    const int4 v = __ldg(reinterpret_cast<const int4*>(q) + i);
    const int w[4] = {v.x, v.y, v.z, v.w};
    __align__(16) __nv_bfloat16 o[16];
#pragma unroll
    for (int j = 0; j < 4; ++j)
#pragma unroll
      for (int b = 0; b < 4; ++b) o[4 * j + b] = __float2bfloat16_rn((float)(int8_t)((w[j] >> (8 * b)) & 0xff));
    reinterpret_cast<uint4*>(out)[2 * i] = reinterpret_cast<const uint4*>(o)[0];
    reinterpret_cast<uint4*>(out)[2 * i + 1] = reinterpret_cast<const uint4*>(o)[1];
  }
}

struct WideScales {          // fp32 scale per output column, matrix by matrix (s[0] == nullptr: none)
  const float* s[3];
  int rows[3];
};

// y = sum over the k-splits in order, then: store / add to the residual stream / GeLU and split for the next GEMM
__global__ void __launch_bounds__(256) wide_epilogue_kernel(const float* part, int S, int M, int N, int mode, float* y, long long ldy,
                                                            __nv_bfloat16* hi, __nv_bfloat16* lo, int ldp, WideScales sc, int vec) {
  pdl_wait();
  pdl_launch_dependents();
  if (vec) {
    // four columns per thread: they lie in one matrix (every matrix has a multiple of four rows)
    const int N4 = N >> 2;
    const long long total = (long long)M * N4;
    for (long long i = (long long)blockIdx.x * 256 + threadIdx.x; i < total; i += (long long)gridDim.x * 256) {
      const int row = (int)(i / N4), n = (int)(i - (long long)row * N4) << 2;
      float4 t = make_float4(0.f, 0.f, 0.f, 0.f);
      for (int s = 0; s < S; ++s) {
        const float4 p = *reinterpret_cast<const float4*>(part + ((size_t)s * WIDE_M + row) * N + n);
        t.x += p.x; t.y += p.y; t.z += p.z; t.w += p.w;
      }
      if (sc.s[0]) {
        int m = 0, r = n;
        while (m < 2 && r >= sc.rows[m]) { r -= sc.rows[m]; ++m; }
        const float4 g = __ldg(reinterpret_cast<const float4*>(sc.s[m] + r));
        t.x *= g.x; t.y *= g.y; t.z *= g.z; t.w *= g.w;
      }
      if (mode == WIDE_EPI_STORE) *reinterpret_cast<float4*>(y + row * ldy + n) = t;
      else if (mode == WIDE_EPI_RESIDUAL) {
        float4* yp = reinterpret_cast<float4*>(y + row * ldy + n);
        float4 o = *yp;
        o.x += t.x; o.y += t.y; o.z += t.z; o.w += t.w;
        *yp = o;
      } else {
        t.x = wide_gelu(t.x); t.y = wide_gelu(t.y); t.z = wide_gelu(t.z); t.w = wide_gelu(t.w);
        uint2 l;
        const uint2 h = wide_split4(t, l);
        *reinterpret_cast<uint2*>(hi + (size_t)row * ldp + n) = h;
        *reinterpret_cast<uint2*>(lo + (size_t)row * ldp + n) = l;
      }
    }
    return;
  }
  const long long total = (long long)M * N;
  for (long long i = (long long)blockIdx.x * 256 + threadIdx.x; i < total; i += (long long)gridDim.x * 256) {
    const int row = (int)(i / N), n = (int)(i - (long long)row * N);
    float t = 0.f;
    for (int s = 0; s < S; ++s) t += part[((size_t)s * WIDE_M + row) * N + n];
    if (sc.s[0]) {
      int m = 0, r = n;
      while (m < 2 && r >= sc.rows[m]) { r -= sc.rows[m]; ++m; }
      t *= __ldg(sc.s[m] + r);
    }
    if (mode == WIDE_EPI_STORE) y[row * ldy + n] = t;
    else if (mode == WIDE_EPI_RESIDUAL) y[row * ldy + n] += t;
    else {
      __nv_bfloat16 h, l;
      wide_split(wide_gelu(t), h, l);
      hi[(size_t)row * ldp + n] = h;
      lo[(size_t)row * ldp + n] = l;
    }
  }
}

PFN_cuTensorMapEncodeTiled_v12000 wide_encoder() {
  static PFN_cuTensorMapEncodeTiled_v12000 encode = nullptr;
  static std::mutex mu;
  std::lock_guard<std::mutex> lock(mu);
  if (!encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess) return nullptr;
    if (qres != cudaDriverEntryPointSuccess || !fn) return nullptr;
    encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(fn);
  }
  return encode;
}

// bf16 [rows][D] row-major, boxes of 64 elements x box_rows rows under the 128-byte swizzle; rows beyond the
// matrix read as zeros
cudaError_t wide_map(const void* p, int rows, int D, int box_rows, CUtensorMap* out) {
  static std::mutex mu;
  static std::map<std::tuple<const void*, int, int, int>, CUtensorMap> cache;
  PFN_cuTensorMapEncodeTiled_v12000 encode = wide_encoder();
  if (!encode) return cudaErrorNotSupported;
  std::lock_guard<std::mutex> lock(mu);
  const auto key = std::make_tuple(p, rows, D, box_rows);
  auto it = cache.find(key);
  if (it != cache.end()) { *out = it->second; return cudaSuccess; }
  const cuuint64_t gdim[2] = {(cuuint64_t)D, (cuuint64_t)rows};
  const cuuint64_t gstride[1] = {(cuuint64_t)D * 2};
  const cuuint32_t box[2] = {(cuuint32_t)WIDE_BK, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  CUtensorMap tm;
  const CUresult cr = encode(&tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(p), gdim, gstride, box, estr,
                             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (cr != CUDA_SUCCESS) return cudaErrorInvalidValue;
  if (cache.size() > 100000) cache.clear();
  cache[key] = tm;
  *out = tm;
  return cudaSuccess;
}

}  // namespace

static int wide_splits_tiles(int tiles, int D, int num_sm) {
  const int kb = D / WIDE_BK;
  int S = 1;
  for (int s = 1; s <= kb && s * tiles <= (num_sm > 0 ? num_sm : SPS_NUM_SM_FALLBACK); ++s)
    if (kb % s == 0) S = s;
  return S;
}
int wide_splits(int N, int D, int num_sm) {
  const int tiles = (N + WIDE_BN - 1) / WIDE_BN, kb = D / WIDE_BK;
  int S = 1;
  for (int s = 1; s <= kb && s * tiles <= (num_sm > 0 ? num_sm : SPS_NUM_SM_FALLBACK); ++s)
    if (kb % s == 0) S = s;
  return S;
}
// kernels one GEMM call launches: with a single k-split the epilogue is part of the GEMM kernel
int wide_gemm_launch_count(const int* rows, int nmat, int D, int num_sm) {
  int tiles = 0;
  for (int i = 0; i < nmat; ++i) tiles += (rows[i] + WIDE_BN - 1) / WIDE_BN;
  return wide_splits_tiles(tiles, D, num_sm) == 1 ? 1 : 2;
}
size_t wide_part_floats(int N, int D, int num_sm) { return (size_t)wide_splits(N, D, num_sm) * WIDE_M * (size_t)N; }
// enough for any (stacked) shape of N output columns: S * tiles <= SMs bounds S * N by 256 * SMs when S > 1
size_t wide_part_bound(int N, int num_sm) {
  const size_t cap = (size_t)WIDE_BN * (size_t)(num_sm > 0 ? num_sm : SPS_NUM_SM_FALLBACK);
  return (size_t)WIDE_M * ((size_t)N + WIDE_BN > cap ? (size_t)N + WIDE_BN : cap);
}

cudaError_t wide_embed_launch(const DevState* st, const void* tok_embed, float* x, int rows, int d, int V, int seq, int c0, cudaStream_t s) {
  return launch_k(wide_embed_kernel, dim3(rows), dim3(256), 0, s, st, reinterpret_cast<const __nv_bfloat16*>(tok_embed), x, d, V, seq, c0);
}
cudaError_t wide_pack_launch(const float* x, int ldx, const float* gain, float eps, int rows, int d, void* hi, void* lo, int ldp, cudaStream_t s) {
  return launch_k(wide_pack_kernel, dim3(rows), dim3(1024), 0, s, x, ldx, gain, eps, d, reinterpret_cast<__nv_bfloat16*>(hi),
                  reinterpret_cast<__nv_bfloat16*>(lo), ldp);
}

// Y = epilogue(sum_k-splits (hi + lo)[M, D] W[N, D]^T).  hi / lo: bf16 [128][D] (rows >= M are never read back);
// part: wide_part_floats(N, D) floats.  mode WIDE_EPI_*: y / ldy for store and residual, yhi / ylo / ldp for GeLU + split.
cudaError_t wide_gemm_launch(const void* W, const void* hi, const void* lo, int M, int N, int D, float* part, int mode, float* y,
                             long long ldy, void* yhi, void* ylo, int ldp, int* err, int num_sm, cudaStream_t st, const float* scale) {
  const void* Ws[3] = {W, nullptr, nullptr};
  const int rows[3] = {N, 0, 0};
  const float* scs[3] = {scale, nullptr, nullptr};
  return wide_gemm_launch_stacked(Ws, rows, 1, hi, lo, M, D, part, mode, y, ldy, yhi, ylo, ldp, err, num_sm, st, scale ? scs : nullptr);
}

// signed bytes -> bf16, n a multiple of 16, both pointers 16-byte aligned
cudaError_t wide_dequant_launch(const void* q, void* out, long long n, int num_sm, cudaStream_t st) {
  if (n % 16) return cudaErrorInvalidValue;
  long long blocks = (n / 16 + 255) / 256;
  const long long cap = 16LL * (num_sm > 0 ? num_sm : SPS_NUM_SM_FALLBACK);
  if (blocks > cap) blocks = cap;
  return launch_k(wide_dequant_kernel, dim3((unsigned)blocks), dim3(256), 0, st, reinterpret_cast<const int8_t*>(q),
                  reinterpret_cast<__nv_bfloat16*>(out), n / 16);
}

// the same over up to three matrices that share the activations (q | k | v): output columns are the matrices' rows side
// by side; part must hold 128 * max(N, 256 * SMs) floats
cudaError_t wide_gemm_launch_stacked(const void* const* Ws, const int* rows, int nmat, const void* hi, const void* lo, int M, int D,
                                     float* part, int mode, float* y, long long ldy, void* yhi, void* ylo, int ldp, int* err, int num_sm,
                                     cudaStream_t st, const float* const* scales) {
  if (M < 1 || M > WIDE_M || nmat < 1 || nmat > 3 || D < WIDE_BK || (D % WIDE_BK)) return cudaErrorInvalidValue;
  WideGemmArgs a;
  cudaError_t e;
  const int mr = M <= 64 ? 64 : WIDE_M;   // rows the MMA carries
  if ((e = wide_map(hi, WIDE_M, D, mr, &a.tm_hi)) != cudaSuccess) return e;
  if ((e = wide_map(lo, WIDE_M, D, mr, &a.tm_lo)) != cudaSuccess) return e;
  int N = 0, tiles = 0;
  for (int i = 0; i < 3; ++i) {
    const bool has = i < nmat;
    if (has && (rows[i] < 1 || !Ws[i])) return cudaErrorInvalidValue;
    a.rows_mat[i] = has ? rows[i] : 0;
    a.tiles_mat[i] = has ? (rows[i] + WIDE_BN - 1) / WIDE_BN : 0;
    if ((e = wide_map(Ws[has ? i : 0], rows[has ? i : 0], D, WIDE_BN, &a.tm_w[i])) != cudaSuccess) return e;
    N += a.rows_mat[i]; tiles += a.tiles_mat[i];
  }
  a.part = part; a.M = M; a.N = N; a.D = D; a.S = wide_splits_tiles(tiles, D, num_sm); a.err = err;
  a.w_is_output = scales ? 1 : 0;
  { const WaitKnobs wk = sps_wait_knobs(); a.wait_ns = wk.limit_ns; a.drop_stage = wk.drop_stage; }
  // four columns per access when every matrix, stride and pointer allows 16-byte (8-byte for bf16) accesses
  int vec = ((N | a.rows_mat[0] | a.rows_mat[1] | a.rows_mat[2] | ldp) & 3) == 0 && (ldy & 3) == 0 &&
            (((uintptr_t)part | (uintptr_t)y | (uintptr_t)yhi | (uintptr_t)ylo) & 15) == 0;
  for (int i = 0; i < 3; ++i) if (scales && i < nmat && ((uintptr_t)scales[i] & 15)) vec = 0;
  a.fused = a.S == 1 ? 1 : 0; a.mode = mode; a.vec = vec; a.ldp = ldp; a.y = y; a.ldy = ldy;
  a.yhi = reinterpret_cast<__nv_bfloat16*>(yhi); a.ylo = reinterpret_cast<__nv_bfloat16*>(ylo);
  for (int i = 0; i < 3; ++i) a.scale[i] = (scales && i < nmat) ? scales[i] : nullptr;
  static DevSmemCache c64{}, c128{};   // the attribute is per device
  if ((e = sps_ensure_smem(wide_gemm_kernel<64>, WideCfg<64>::SMEM, c64)) != cudaSuccess) return e;
  if ((e = sps_ensure_smem(wide_gemm_kernel<128>, WideCfg<128>::SMEM, c128)) != cudaSuccess) return e;
  if (mr == 64) e = launch_k(wide_gemm_kernel<64>, dim3(tiles, a.S), dim3(192), WideCfg<64>::SMEM, st, a);
  else e = launch_k(wide_gemm_kernel<128>, dim3(tiles, a.S), dim3(192), WideCfg<128>::SMEM, st, a);
  if (e != cudaSuccess || a.fused) return e;
  const long long total = (long long)M * (vec ? N / 4 : N);
  int blocks = (int)((total + 255) / 256);
  if (blocks > 8 * (num_sm > 0 ? num_sm : SPS_NUM_SM_FALLBACK)) blocks = 8 * (num_sm > 0 ? num_sm : SPS_NUM_SM_FALLBACK);
  WideScales sc{};
  for (int i = 0; i < 3; ++i) { sc.s[i] = (scales && i < nmat) ? scales[i] : nullptr; sc.rows[i] = a.rows_mat[i]; }
  return launch_k(wide_epilogue_kernel, dim3(blocks), dim3(256), 0, st, (const float*)part, a.S, M, N, mode, y, ldy,
                  reinterpret_cast<__nv_bfloat16*>(yhi), reinterpret_cast<__nv_bfloat16*>(ylo), ldp, sc, vec);
}
