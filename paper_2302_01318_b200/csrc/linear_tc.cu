// The memory-bound linear layer on the 5th-generation tensor cores: Y[M, N] = f(X)[M, D] W[N, D]^T for the 1 .. 16
// activation rows of a draft step or a scoring pass (K + 1 rows), bf16 weights streamed once from HBM.
//
// The weights are the 128-row A operand of tcgen05.mma (cta_group::1, M = 128, K = 16), read by the tensor core
// straight from the shared-memory ring the copy engine fills -- no warp ever loads a weight into registers.  The
// activations are the narrow B operand: their bf16 high halves and bf16 remainders (together ~16 bits, as in
// every layer of this library) sit side by side as columns of one MMA -- N = 16 for up to 8 rows (8 high + 8
// low), N = 32 for up to 16 -- so five rows cost what one row costs.  Accumulators live in tensor memory, two
// of them, so that one tile is read back while the next is being multiplied.
//
//   * grid = (R row ranges) x (S k-splits).  Within k-split s the T x SPT stages (T tiles of 128 weight rows, SPT
//     stages of KBX k-blocks of 64 k) are cut into R equal contiguous pieces: CTA r owns stages
//     [r tot / R, (r + 1) tot / R) -- balanced to one stage (16 or 32 KB), with no run-time queue.
//   * warp 0 (one lane): copy producer.  One 3-D TMA box {64 k, 128 rows, KBX} per stage, 128-byte swizzle, into a
//     ring guarded by full / empty mbarriers; the first ring-full is asked for before the kernel waits for its
//     predecessor (weights are constants).  Packed activations (left by the producing layer's epilogue) arrive as
//     TMA boxes of 8 rows too; otherwise warps 2..5 convert X (RMSNorm / GeLU prologue) and write the swizzled
//     layout themselves.
//   * warp 1 (one lane): issues 4 KBX MMAs per stage, releases the stage with tcgen05.commit, and commits the
//     accumulator when a tile's piece is complete.
//   * warps 2..5: tcgen05.ld the finished accumulator (lane = weight row), add the high and low columns of each
//     activation row, and write the piece's partial sums: a piece that starts a tile's k-range goes to
//     part[s][m][n]; a piece that starts in the MIDDLE of one (the tile was begun by CTA r - 1) goes to
//     carry[cta][m][row].  lin_epilogue_kernel adds, per output, the k-splits in order and the carry of the one
//     CTA boundary that may fall inside the tile, so the result does not depend on timing.
//
// Every wait is bounded; on expiry the CTA records error 3, lets its copies land, waits for the MMAs it issued,
// frees its tensor memory and returns.  No multicast, no clusters.
#include <cuda.h>
#include <cudaTypedefs.h>

#include <cstdlib>
#include <map>
#include <mutex>
#include <tuple>

#include "common.cuh"

namespace {

constexpr int TC_THREADS = 192;
constexpr uint32_t TC_TMEM_COLS = 64;   // two accumulators, 32 columns apart

__device__ __forceinline__ uint32_t t_smem(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ unsigned long long t_timer() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void t_mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void t_mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void t_mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
// one try: the thread sleeps in hardware until the phase completes or about a microsecond has passed (no busy polling:
// the kernel runs at the board's power cap, and what idle lanes burn comes off the clock)
__device__ __forceinline__ uint32_t t_mbar_try(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n selp.u32 %0, 1, 0, p;\n}\n"
      : "=r"(ok)
      : "r"(bar), "r"(parity), "r"(1000u)
      : "memory");
  return ok;
}
// bounded wait: false (and error word 3) after limit_ns of the global timer, or as soon as another thread of the CTA gave up
__device__ __forceinline__ bool t_mbar_wait(uint32_t bar, uint32_t parity, int* err, unsigned long long limit_ns, volatile int* abort_flag) {
  if (t_mbar_try(bar, parity)) return true;
  const unsigned long long t0 = t_timer();
  for (;;) {
#pragma unroll 1
    for (int i = 0; i < 128; ++i)
      if (t_mbar_try(bar, parity)) return true;
    if (*abort_flag) return false;
    if (t_timer() - t0 > limit_ns) {
      atomicExch(err, 3);
      *abort_flag = 1;
      return false;
    }
  }
}
__device__ __forceinline__ void t_tma_3d(uint32_t dst, const CUtensorMap* tm, int c0, int c1, int c2, uint32_t bar, uint64_t policy) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint"
      " [%0], [%1, {%2, %3, %4}], [%5], %6;"
      ::"r"(dst), "l"(tm), "r"(c0), "r"(c1), "r"(c2), "r"(bar), "l"(policy)
      : "memory");
}
__device__ __forceinline__ void t_tma_3d_plain(uint32_t dst, const CUtensorMap* tm, int c0, int c1, int c2, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
      ::"r"(dst), "l"(tm), "r"(c0), "r"(c1), "r"(c2), "r"(bar)
      : "memory");
}

// Shared-memory operand descriptor, K-major, rows of 128 bytes (64 bf16) under the 128-byte swizzle: the 8 rows of a
// group are 128 bytes apart, groups `sbo` bytes apart (1024 for a dense tile; the activations keep their groups in
// separate regions), descriptor version 1, layout type 2.  16 elements along k = +32 bytes on the start address.
__device__ __forceinline__ uint64_t t_desc(uint32_t smem_addr, uint32_t sbo) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3ffffu) >> 4);
  d |= (uint64_t)1 << 16;
  d |= (uint64_t)(sbo >> 4) << 32;
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}
__device__ __forceinline__ void t_mma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
  asm volatile(
      "{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n"
      " tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
__device__ __forceinline__ void t_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void t_ld16(uint32_t taddr, float (&v)[16]) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]),
        "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr)
      : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

__device__ __forceinline__ float t_gelu(float v) {   // v * sigmoid(2u), u = sqrt(2/pi) (v + 0.044715 v^3)
  const float u = 0.7978845608028654f * (v + 0.044715f * v * v * v);
  return __fdividef(v, 1.0f + __expf(-2.0f * u));
}
__device__ __forceinline__ void t_split(float v, uint32_t& hi, uint32_t& lo) {
  const __nv_bfloat16 h = __float2bfloat16_rn(v);
  hi = __bfloat16_as_ushort(h);
  lo = __bfloat16_as_ushort(__float2bfloat16_rn(v - __bfloat162float(h)));
}
__device__ __forceinline__ int t_mat_of(const LinArgs& a, int n, int& row_in_mat) {
  const int r0 = a.rows_per_mat, rt = a.rows_tail;
  if (n < r0) { row_in_mat = n; return 0; }
  if (n < r0 + rt) { row_in_mat = n - r0; return 1; }
  row_in_mat = n - r0 - rt;
  return 2;
}

struct LinTcArgs {
  LinArgs a;
  CUtensorMap tm_w[3];
  CUtensorMap tm_xh, tm_xl;
  int KBS;      // k-blocks (64 k) of a CTA's k-range
  int KBX;      // k-blocks per stage
  int NS;       // ring stages
  int NGRP;     // 8-row groups of the activations' operand: 2 (N = 16) or 4 (N = 32)
  int BR;       // weight rows per tile: 128 or 64 (the MMA's M)
};

__global__ void __launch_bounds__(TC_THREADS, 1) lin_tc_kernel(const __grid_constant__ LinTcArgs ta) {
  // activations' regions and the ring (both want 1024-byte alignment) first, a 512-byte header behind them
  extern __shared__ __align__(1024) unsigned char tc_raw[];
  const LinArgs& a = ta.a;
  const uint32_t xs = t_smem(tc_raw);
  unsigned char* xs_p = tc_raw;
  // header: full[16], empty[16], x, acc[2], free[2], done, tensor-memory base, abort flag, 1/rms of the rows
  unsigned char* hdr = tc_raw + (size_t)ta.NGRP * ta.KBS * 1024 + (size_t)ta.NS * ta.KBX * ta.BR * 128;
  const uint32_t base = t_smem(hdr);
  const uint32_t bar_full = base, bar_empty = base + 128, bar_x = base + 256, bar_acc = base + 264, bar_free = base + 280, bar_done = base + 296;
  volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(hdr + 320);
  volatile int* s_abort = reinterpret_cast<volatile int*>(hdr + 328);
  float* s_scale = reinterpret_cast<float*>(hdr + 384);
  const int KBS = ta.KBS, KBX = ta.KBX, NS = ta.NS, NGRP = ta.NGRP, BR = ta.BR;
  const uint32_t BLOCK = (uint32_t)BR * 128u;   // one k-block of a weight tile: BR rows x 64 bf16
  const uint32_t REGION = (uint32_t)KBS * 1024u, STAGE = (uint32_t)KBX * BLOCK;
  const uint32_t ring = xs + (uint32_t)NGRP * REGION;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int r = blockIdx.x, s = blockIdx.y, R = gridDim.x, cta = r * a.S + s;
  const int T = (a.N + BR - 1) / BR, SPT = KBS / KBX;
  const long long tot = (long long)T * SPT;
  const int x0 = (int)((r * tot) / R), x1 = (int)(((r + 1) * tot) / R);
  const bool packed = a.xp_hi != nullptr;

  if (tid == 0) {
    for (int i = 0; i < NS; ++i) { t_mbar_init(bar_full + 8 * i, 1); t_mbar_init(bar_empty + 8 * i, 1); }
    t_mbar_init(bar_x, packed ? 1u : 128u);
    t_mbar_init(bar_done, 1);
    for (int i = 0; i < 2; ++i) { t_mbar_init(bar_acc + 8 * i, 1); t_mbar_init(bar_free + 8 * i, 4); }
    *s_abort = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(base + 320), "n"(TC_TMEM_COLS) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem = *s_tmem;
  pdl_launch_dependents();

  if (warp == 0) {
    // ------------------------------------------------------------------ copy producer
    if (lane == 0) {
      uint64_t policy;
      asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(policy));
      bool ok = true;
      int it = 0;
      auto issue = [&](int x) {
        const int slot = it % NS, use = it / NS;
        if (use > 0 && !t_mbar_wait(bar_empty + 8 * slot, (uint32_t)(use - 1) & 1u, a.err, a.wait_ns, s_abort)) { ok = false; return; }
        if (!(cta == 0 && it == a.drop_stage)) {   // test hook: that stage is never asked for, the MMA lane's wait runs out
          const int tile = x / SPT, j = x - tile * SPT;
          int rin;
          const int mat = t_mat_of(a, tile * BR, rin);
          t_mbar_expect_tx(bar_full + 8 * slot, STAGE);
          t_tma_3d(ring + slot * STAGE, &ta.tm_w[mat], 0, rin, s * KBS + j * KBX, bar_full + 8 * slot, policy);
        }
        ++it;
      };
      const int pre = min(NS, x1 - x0);
      for (int i = 0; i < pre && ok; ++i) issue(x0 + i);
      pdl_wait();
      if (packed) {
        // the activations' halves: region g holds rows 8 g' .. 8 g' + 7 (g' = g mod NGRP / 2) of the high (g < NGRP / 2) or low halves
        t_mbar_expect_tx(bar_x, (uint32_t)NGRP * REGION);
        for (int g = 0; g < NGRP; ++g) {
          const int half = NGRP >> 1, lo = g >= half ? 1 : 0, g8 = (g - lo * half) * 8;
          t_tma_3d_plain(xs + g * REGION, lo ? &ta.tm_xl : &ta.tm_xh, 0, g8, s * KBS, bar_x);
        }
      }
      for (int x = x0 + pre; x < x1 && ok; ++x) issue(x);
      if (!ok || *s_abort) {
        // a wait ran out somewhere: let the copies already issued land before this CTA's shared memory goes away
        *s_abort = 1;
        for (int j = max(0, it - NS); j < it; ++j)
          if (!(cta == 0 && j == a.drop_stage)) {
            const uint32_t bar = bar_full + 8 * (j % NS), par = (uint32_t)(j / NS) & 1u;
            const unsigned long long t0 = t_timer();
            while (!t_mbar_try(bar, par) && t_timer() - t0 <= a.wait_ns) {}
          }
        if (packed) {
          const unsigned long long t0 = t_timer();
          while (!t_mbar_try(bar_x, 0u) && t_timer() - t0 <= a.wait_ns) {}
        }
      }
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issue
    if (lane == 0) {
      // kind::f16: fp32 accumulator, bf16 x bf16, both operands K-major, N = 8 NGRP, M = BR
      const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)NGRP << 17) | ((uint32_t)(BR >> 4) << 24);
      bool ok = t_mbar_wait(bar_x, 0u, a.err, a.wait_ns, s_abort);
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      int buf = 0, seg = 0, it = 0;
      uint32_t acc = 0;
      for (int x = x0; x < x1 && ok; ++x, ++it) {
        const int tile = x / SPT, j = x - tile * SPT;
        if (x == x0 || j == 0) {
          // a new piece: its accumulator must have been read back (two pieces ago)
          if (seg >= 2 && !t_mbar_wait(bar_free + 8 * buf, (uint32_t)((seg >> 1) - 1) & 1u, a.err, a.wait_ns, s_abort)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          acc = 0;
        }
        const int slot = it % NS, use = it / NS;
        if (!t_mbar_wait(bar_full + 8 * slot, (uint32_t)use & 1u, a.err, a.wait_ns, s_abort)) { ok = false; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t wa = ring + slot * STAGE;
        for (int kb = 0; kb < KBX; ++kb) {
          const uint64_t da = t_desc(wa + kb * BLOCK, 1024u), db = t_desc(xs + (uint32_t)(j * KBX + kb) * 1024u, REGION);
#pragma unroll
          for (int k = 0; k < 4; ++k) {
            t_mma(tmem + (uint32_t)buf * 32u, da + 2 * k, db + 2 * k, idesc, acc);
            acc = 1;
          }
        }
        t_commit(bar_empty + 8 * slot);            // the stage is free once these MMAs have read it
        if (x == x1 - 1 || j == SPT - 1) {
          t_commit(bar_acc + 8 * buf);             // ... and the piece's accumulator is complete once all of them are done
          buf ^= 1;
          ++seg;
        }
      }
      if (!ok) {
        // gave up: every MMA issued so far must have finished before the tensor memory and the ring go away
        *s_abort = 1;
        t_commit(bar_done);
        const unsigned long long t0 = t_timer();
        while (!t_mbar_try(bar_done, 0u) && t_timer() - t0 <= a.wait_ns) {}
      }
    }
  } else {
    // ------------------------------------------------------------------ warps 2..5: activations in, partial sums out
    const int q = warp & 3, et = tid - 64;   // tensor-memory lanes 32 q .. 32 q + 31; et = 0 .. 127
    const int MH = NGRP * 4;                 // activation rows the operand carries (8 or 16)
    pdl_wait();
    bool ok = true;
    if (a.pro == PRO_RMSNORM && (!packed || cta == 0)) {
      // 1/rms of each row from the partial sums of squares its producer left (lanes stride, then a shuffle tree)
      for (int m = warp - 2; m < a.M; m += 4) {
        const int srow = a.x_row0 + m * a.x_rowstep;
        float tt = 0.f;
        for (int i = lane; i < a.ssq_in_n; i += 32) tt += a.ssq_in[SSQ_IDX(i, srow)];
        tt = warp_sum(tt);
        if (lane == 0) {
          const float sc = rsqrtf(tt / (float)a.D + a.eps);
          s_scale[m] = sc;
          // packed input: the gain is in it already and the epilogue kernel multiplies the sums by 1/rms
          if (packed) reinterpret_cast<float*>(a.counters + LIN_SCALE_SLOT)[m] = sc;
        }
      }
    }
    if (!packed) {
      asm volatile("bar.sync 1, 128;" ::: "memory");
      // X -> bf16 high halves and remainders in the operand's swizzled layout: row m of group g = m / 8 is 128 bytes
      // per k-block, its 16-byte chunk c stored at chunk c ^ (m & 7); rows beyond M are zero
      const int chunks = KBS * 8, KS = KBS * 64, half = NGRP >> 1;
      for (int c = et; c < MH * chunks; c += 128) {
        const int m = c / chunks, qq = c - m * chunks, kb = qq >> 3, ch = qq & 7;
        uint4 hi = make_uint4(0u, 0u, 0u, 0u), lo = hi;
        if (m < a.M) {
          const int k = s * KS + qq * 8;
          const float* src = a.X + (size_t)(a.x_row0 + m * a.x_rowstep) * a.ldx + k;
          const float4 v0 = *reinterpret_cast<const float4*>(src), v1 = *reinterpret_cast<const float4*>(src + 4);
          float f[8] = {v0.x, v0.y, v0.z, v0.w, v1.x, v1.y, v1.z, v1.w};
          if (a.pro == PRO_RMSNORM) {
            const float4 g0 = __ldg(reinterpret_cast<const float4*>(a.gain + k)), g1 = __ldg(reinterpret_cast<const float4*>(a.gain + k + 4));
            const float gg[8] = {g0.x, g0.y, g0.z, g0.w, g1.x, g1.y, g1.z, g1.w};
            const float sc = s_scale[m];
#pragma unroll
            for (int i = 0; i < 8; ++i) f[i] = gg[i] * f[i] * sc;
          } else if (a.pro == PRO_GELU) {
#pragma unroll
            for (int i = 0; i < 8; ++i) f[i] = t_gelu(f[i]);
          }
          uint32_t h[8], l[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) t_split(f[i], h[i], l[i]);
          hi = make_uint4(h[0] | (h[1] << 16), h[2] | (h[3] << 16), h[4] | (h[5] << 16), h[6] | (h[7] << 16));
          lo = make_uint4(l[0] | (l[1] << 16), l[2] | (l[3] << 16), l[4] | (l[5] << 16), l[6] | (l[7] << 16));
        }
        const uint32_t off = (uint32_t)kb * 1024u + (uint32_t)(m & 7) * 128u + (uint32_t)((ch ^ (m & 7)) << 4);
        *reinterpret_cast<uint4*>(xs_p + (size_t)(m >> 3) * REGION + off) = hi;
        *reinterpret_cast<uint4*>(xs_p + (size_t)(half + (m >> 3)) * REGION + off) = lo;
      }
      asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the tensor core reads these through the async proxy
      t_mbar_arrive(bar_x);
    }
    int buf = 0, seg = 0;
    for (int xa = x0; xa < x1 && ok; ++seg, buf ^= 1) {
      const int tile = xa / SPT, xe = min(x1, (tile + 1) * SPT);
      const bool mid = xa != tile * SPT;      // the tile was begun by the CTA before this one
      ok = lane != 0 || t_mbar_wait(bar_acc + 8 * buf, (uint32_t)(seg >> 1) & 1u, a.err, a.wait_ns, s_abort);   // one lane waits, the warp follows
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      // columns: [high halves of the rows | low halves]
      float v[32];
      {
        const uint32_t tb = tmem + ((uint32_t)(q * 32) << 16) + (uint32_t)buf * 32u;
        float v16[16];
        t_ld16(tb, v16);
#pragma unroll
        for (int i = 0; i < 16; ++i) v[i] = v16[i];
        if (NGRP == 4) {
          t_ld16(tb + 16u, v16);
#pragma unroll
          for (int i = 0; i < 16; ++i) v[16 + i] = v16[i];
        }
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) t_mbar_arrive(bar_free + 8 * buf);   // the accumulator may be overwritten
      // a 128-row accumulator keeps row i in lane i; a 64-row one keeps 16 rows in the first 16 lanes of each lane quarter
      const int row = BR == 128 ? q * 32 + lane : q * 16 + lane, n = tile * BR + row;
      if (n < a.N && (BR == 128 || lane < 16)) {
        float* dst = mid ? a.carry + (size_t)cta * SPS_MAX_ROWS * 128 + row : a.part + (size_t)s * SPS_MAX_ROWS * a.N + n;
        const size_t ld = mid ? 128 : (size_t)a.N;
        if (NGRP == 2) {
#pragma unroll
          for (int m = 0; m < 8; ++m) if (m < a.M) dst[m * ld] = v[m] + v[8 + m];
        } else {
#pragma unroll
          for (int m = 0; m < 16; ++m) if (m < a.M) dst[m * ld] = v[m] + v[16 + m];
        }
      }
      xa = xe;
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "n"(TC_TMEM_COLS) : "memory");
  }
}

PFN_cuTensorMapEncodeTiled_v12000 tc_encoder() {
  static PFN_cuTensorMapEncodeTiled_v12000 encode = nullptr;
  if (!encode) {
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres) != cudaSuccess) return nullptr;
    if (qres != cudaDriverEntryPointSuccess || !fn) return nullptr;
    encode = reinterpret_cast<PFN_cuTensorMapEncodeTiled_v12000>(fn);
  }
  return encode;
}

// [rows][ld] bf16 as {64 k, rows, D / 64} with byte strides {row_stride, 128}, box {64, box_rows, box_blocks}, 128-byte swizzle;
// descriptors are cached per (pointer, shape)
cudaError_t tc_tensor_map(const void* base, int rows, long long row_stride_bytes, int D, int box_rows, int box_blocks, bool weights,
                          CUtensorMap* out) {
  static std::mutex mu;
  static std::map<std::tuple<const void*, int, long long, int, int, int>, CUtensorMap> cache;
  std::lock_guard<std::mutex> lock(mu);
  PFN_cuTensorMapEncodeTiled_v12000 encode = tc_encoder();
  if (!encode) return cudaErrorNotSupported;
  const auto key = std::make_tuple(base, rows, row_stride_bytes, D, box_rows, box_blocks);
  auto it = cache.find(key);
  if (it != cache.end()) { *out = it->second; return cudaSuccess; }
  const cuuint64_t gdim[3] = {64, (cuuint64_t)rows, (cuuint64_t)(D / 64)};
  const cuuint64_t gstride[2] = {(cuuint64_t)row_stride_bytes, 128};
  const cuuint32_t box[3] = {64, (cuuint32_t)box_rows, (cuuint32_t)box_blocks};
  const cuuint32_t estr[3] = {1, 1, 1};
  CUtensorMap tm;
  const CUresult cr = encode(&tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), gdim, gstride, box, estr,
                             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                             weights ? CU_TENSOR_MAP_L2_PROMOTION_L2_256B : CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (cr != CUDA_SUCCESS) return cudaErrorInvalidValue;
  if (cache.size() > 100000) cache.clear();
  cache[key] = tm;
  *out = tm;
  return cudaSuccess;
}

// What a CTA may take so that one CTA of the epilogue kernel (about 100 bytes of shared memory, plus the 1 KB the
// hardware reserves per CTA) still fits on the same SM's 228 KB: the epilogue CTAs wait beside the layer's and must not
// keep the next layer's CTAs off the SMs.
const size_t kTcSmem = 224 * 1024 + 512;

}  // namespace

// Whether a layer can run on lin_tc_kernel, and how: bf16 weights, several k-splits of the plan's KS (a multiple of 64),
// stacked matrices cut on multiples of 128 rows, at least as many 128-row tiles as row ranges, 16-byte aligned rows.
bool lin_tc_plan(const LinArgs& a, const LinPlan& p, LinTcPlan* out) {
  static const int on = [] { const char* e = getenv("SPS_LIN_TC"); return e ? atoi(e) : 1; }();   // tuning: 0 = the mma.sync kernel everywhere
  if (!on || !a.carry || p.variant != 2 || p.KS < 64 || p.KS % 64 || a.D % 64 || p.S < 2) return false;
  static const int br_env = [] { const char* e = getenv("SPS_LIN_TC_BR"); return e ? atoi(e) : 128; }();   // tuning: weight rows per tile
  const int BR = br_env == 64 ? 64 : 128;
  const int T = (a.N + BR - 1) / BR;
  if (a.N > a.rows_per_mat && ((a.rows_per_mat % BR) || ((a.rows_tail > 0 ? a.rows_tail : a.rows_per_mat) % BR))) return false;
  static const int min_m = [] { const char* e = getenv("SPS_LIN_TC_MIN_M"); return e ? atoi(e) : 5; }();   // tuning: fewer rows go to the mma.sync kernel
  if (a.M < min_m || a.M > SPS_MAX_ROWS) return false;
  for (int i = 0; i < 3; ++i) if (a.W[i] && (((size_t)a.W[i]) & 15)) return false;
  if (a.xp_hi) {
    if ((a.ldx % 8) || ((((size_t)a.xp_hi | (size_t)a.xp_lo)) & 15)) return false;
  } else {
    if ((a.ldx % 4) || (((size_t)a.X) & 15) || (a.pro == PRO_RMSNORM && (((size_t)a.gain) & 15))) return false;
  }
  LinTcPlan t{};
  t.NGRP = a.M <= 8 ? 2 : 4;
  t.KBS = p.KS / 64;
  t.BR = BR;
  // k-blocks per stage: 32 KB stages unless told otherwise (a row of the tile then contributes KBX * 128 contiguous bytes)
  static const int kbx_env = [] { const char* e = getenv("SPS_LIN_TC_KBX"); return e ? atoi(e) : 0; }();   // tuning
  int kbx = kbx_env > 0 ? kbx_env : 32768 / (BR * 128);
  while (kbx > 1 && t.KBS % kbx) kbx >>= 1;
  t.KBX = kbx;
  const size_t xbytes = (size_t)t.NGRP * t.KBS * 1024, stage = (size_t)t.KBX * BR * 128;
  if (512 + xbytes + 2 * stage > kTcSmem) return false;
  int NS = (int)((kTcSmem - 512 - xbytes) / stage);
  if (NS > 16) NS = 16;
  t.NS = NS;
  t.smem = 512 + xbytes + (size_t)NS * stage;
  t.R = p.R < T ? p.R : T;
  if (t.R * 10 < p.R * 9) return false;   // a layer of few 128-row tiles would leave SMs idle: the 16-row tiles of the mma.sync kernel
  if (t.R < 1 || (long long)t.R * p.S > LIN_TC_MAX_CTAS) return false;
  t.SPT = t.KBS / t.KBX;
  t.tot = T * t.SPT;
  if ((long long)t.tot * t.R >= (1LL << 30)) return false;   // the epilogue's 32-bit arithmetic
  *out = t;
  return true;
}

cudaError_t lin_tc_launch(const LinArgs& a, const LinTcPlan& t, cudaStream_t st) {
  LinTcArgs ta;
  ta.a = a;
  ta.KBS = t.KBS; ta.KBX = t.KBX; ta.NS = t.NS; ta.NGRP = t.NGRP; ta.BR = t.BR;
  cudaError_t e;
  const int rows_tail = a.rows_tail > 0 ? a.rows_tail : a.rows_per_mat;
  const int nmat = a.N > a.rows_per_mat ? 1 + (a.N - a.rows_per_mat + rows_tail - 1) / rows_tail : 1;
  for (int i = 0; i < 3; ++i) {
    const bool has = i < nmat;   // unused slots repeat the first matrix
    const int rows = has && i > 0 ? rows_tail : (a.N < a.rows_per_mat ? a.N : a.rows_per_mat);
    if ((e = tc_tensor_map(a.W[has ? i : 0], rows, (long long)a.D * 2, a.D, t.BR, t.KBX, true, &ta.tm_w[i])) != cudaSuccess) return e;
  }
  if (a.xp_hi) {
    const long long stride = (long long)a.x_rowstep * a.ldx * 2;
    const __nv_bfloat16* h = a.xp_hi + (size_t)a.x_row0 * a.ldx;
    const __nv_bfloat16* l = a.xp_lo + (size_t)a.x_row0 * a.ldx;
    // a single row has no stride to speak of; the encoder still wants a multiple of 16 bytes
    const long long sb = a.M > 1 ? stride : (long long)a.ldx * 2;
    if (sb <= 0 || sb % 16) return cudaErrorInvalidValue;
    if ((e = tc_tensor_map(h, a.M, sb, a.D, 8, t.KBS, false, &ta.tm_xh)) != cudaSuccess) return e;
    if ((e = tc_tensor_map(l, a.M, sb, a.D, 8, t.KBS, false, &ta.tm_xl)) != cudaSuccess) return e;
  } else {
    ta.tm_xh = ta.tm_w[0];
    ta.tm_xl = ta.tm_w[0];
  }
  static DevSmemCache cached{};
  if ((e = sps_ensure_smem(lin_tc_kernel, t.smem, cached)) != cudaSuccess) return e;
  return launch_k(lin_tc_kernel, dim3(t.R, a.S), dim3(TC_THREADS), t.smem, st, ta);
}

