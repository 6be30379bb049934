// Tensor-parallel passes: the exchange that follows the attention block and the feed-forward block of every layer.
//
// The paper serves its models Megatron-style over several chips (section Conditional Scoring: the attention and
// feed-forward blocks are sharded, and each is followed by an all-reduce whose message is (K + 1) x d_model numbers:
// latency-bound, and about as costly for K + 1 rows as for one).  Here rank r of `world` holds the query / key / value
// heads and the feed-forward features of its shard (wq, wk, wv, w_up by output rows; wo, w_down by input columns), so
// its output projection yields a PARTIAL [rows, d_model] update of the residual stream.  The all-reduce is two small
// kernels per block, written for one process per GPU:
//
//   tp_push_kernel    copies the rank's partial into slot [parity][rank] of every rank's inbox (plain stores into
//                     peer memory; its own inbox included), makes them visible system-wide and then writes the
//                     exchange's number into its flag in every rank's flag array;
//   tp_reduce_kernel  waits -- bounded -- until every rank's flag shows this exchange, then sums the `world` slots of
//                     its OWN inbox in rank order (remote partials are only ever read from local memory, and every
//                     rank adds in the same order, so all ranks hold bit-identical residual streams), adds the
//                     residual, leaves the per-CTA sums of squares for the next RMSNorm and the next layer's packed
//                     input, exactly as the epilogue of an unsharded layer does.
//
// Slots alternate with the exchange's parity: a rank can be at most one exchange ahead of a peer that is still
// reading (it cannot finish exchange e + 1 before that peer has pushed e + 1, which the peer does after reading e).
// No multicast, no cluster, no library collective; loads from peer memory never happen.
#include <cuda_fp16.h>

#include "common.cuh"

namespace {

__device__ __forceinline__ unsigned long long tp_timer() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}

__global__ void __launch_bounds__(1024) tp_push_kernel(TpArgs a) {
  pdl_launch_dependents();
  pdl_wait();
  const int tid = threadIdx.x;
  const uint32_t epoch = *a.epoch_ctr + 1u;    // the exchange this push opens
  const long long n4 = (long long)a.rows * a.d / 4;
  const float4* src = reinterpret_cast<const float4*>(a.send);
  const size_t slot = ((size_t)(epoch & 1u) * a.world + a.rank) * a.slot_floats;
  for (int w = 0; w < a.world; ++w) {
    float4* dst = reinterpret_cast<float4*>(a.peer_inbox[w] + slot);
    for (long long i = tid; i < n4; i += blockDim.x) dst[i] = src[i];
  }
  __threadfence_system();     // the partial is visible to every device before the flag is
  __syncthreads();
  if (tid < a.world) {
    volatile uint32_t* f = a.peer_flags[tid] + a.rank;
    *f = epoch;
  }
  if (tid == 0) *a.epoch_ctr_w = epoch;        // the reduce kernel that follows on this stream reads it
}

// p_inv etc. as in the linear layers' epilogue: y = x + sum_r part_r; ssq; packed copy of gain * y
__global__ void __launch_bounds__(256) tp_reduce_kernel(TpArgs a) {
  __shared__ int s_ok;
  __shared__ float s_red[8][SPS_MAX_ROWS];
  pdl_launch_dependents();
  pdl_wait();
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t epoch = *a.epoch_ctr;         // opened by this rank's push, just before on this stream
  if (tid == 0) {
    // every rank's flag must show this exchange (flags only grow; the comparison is wrap-safe)
    int ok = 1;
    const unsigned long long t0 = tp_timer();
    for (int r = 0; r < a.world && ok; ++r) {
      volatile uint32_t* f = a.my_flags + r;
      while ((int32_t)(*f - epoch) < 0) {
        __nanosleep(100);
        if (tp_timer() - t0 > a.wait_ns) { atomicExch(a.err, 3); ok = 0; break; }
      }
    }
    __threadfence_system();   // the partials the flags announce are read after this
    s_ok = ok;
  }
  __syncthreads();
  if (!s_ok) return;
  const int C = gridDim.x, cta = blockIdx.x, d = a.d;
  const int quads = d >> 2;
  const int q0 = (int)(((long long)cta * quads) / C), q1 = (int)(((long long)(cta + 1) * quads) / C);
  const float* inbox = a.my_inbox + (size_t)(epoch & 1u) * a.world * a.slot_floats;
  float loc[SPS_MAX_ROWS];
#pragma unroll
  for (int m = 0; m < SPS_MAX_ROWS; ++m) loc[m] = 0.f;
  const int per = q1 - q0;
  for (int e = tid; e < per * a.rows; e += blockDim.x) {
    const int m = e / per, n = (q0 + (e - m * per)) << 2;
    float4 y = *reinterpret_cast<const float4*>(a.x + (size_t)m * d + n);
    for (int r = 0; r < a.world; ++r) {
      const float4 v = __ldcg(reinterpret_cast<const float4*>(inbox + (size_t)r * a.slot_floats + (size_t)m * d + n));
      y.x += v.x; y.y += v.y; y.z += v.z; y.w += v.w;
    }
    *reinterpret_cast<float4*>(a.x + (size_t)m * d + n) = y;
    const float sq = ((y.x * y.x + y.y * y.y) + y.z * y.z) + y.w * y.w;
#pragma unroll
    for (int mm = 0; mm < SPS_MAX_ROWS; ++mm) if (mm == m) loc[mm] += sq;
    if (a.yp_hi) {
      float4 z = y;
      if (a.yp_gain) {
        const float4 g = __ldg(reinterpret_cast<const float4*>(a.yp_gain + n));
        z.x *= g.x; z.y *= g.y; z.z *= g.z; z.w *= g.w;
      }
      uint2 hi, lo;
      const float zz[4] = {z.x, z.y, z.z, z.w};
      uint32_t hw[4], lw[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) {
        if (a.half_is_fp16) {
          const __half hh = __float2half_rn(zz[i]);
          hw[i] = __half_as_ushort(hh);
          lw[i] = __half_as_ushort(__float2half_rn(zz[i] - __half2float(hh)));
        } else {
          const __nv_bfloat16 hb = __float2bfloat16_rn(zz[i]);
          hw[i] = __bfloat16_as_ushort(hb);
          lw[i] = __bfloat16_as_ushort(__float2bfloat16_rn(zz[i] - __bfloat162float(hb)));
        }
      }
      hi = make_uint2(hw[0] | (hw[1] << 16), hw[2] | (hw[3] << 16));
      lo = make_uint2(lw[0] | (lw[1] << 16), lw[2] | (lw[3] << 16));
      *reinterpret_cast<uint2*>(a.yp_hi + (size_t)m * d + n) = hi;
      *reinterpret_cast<uint2*>(a.yp_lo + (size_t)m * d + n) = lo;
    }
  }
  // this CTA's share of every row's sum of squares (fixed order: lanes, then warps)
#pragma unroll
  for (int m = 0; m < SPS_MAX_ROWS; ++m) {
    if (m < a.rows) {
      const float v = warp_sum(loc[m]);
      if (lane == 0) s_red[warp][m] = v;
    }
  }
  __syncthreads();
  if (tid < a.rows) {
    float t = 0.f;
    for (int w = 0; w < 8; ++w) t += s_red[w][tid];
    a.ssq_out[SSQ_IDX(cta, tid)] = t;
  }
}

}  // namespace

int tp_reduce_ctas(int d, int num_sm) {
  int c = (d / 4 + 255) / 256;      // about one quad per thread and row
  if (c > num_sm) c = num_sm;
  if (c > LIN_MAX_R) c = LIN_MAX_R;
  return c < 1 ? 1 : c;
}

cudaError_t tp_push_launch(const TpArgs& a, cudaStream_t st) { return launch_k(tp_push_kernel, dim3(1), dim3(1024), 0, st, a); }

cudaError_t tp_reduce_launch(const TpArgs& a, int ctas, cudaStream_t st) { return launch_k(tp_reduce_kernel, dim3(ctas), dim3(256), 0, st, a); }
