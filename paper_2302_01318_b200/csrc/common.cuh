// Shared declarations of the CUDA library: argument blocks of the kernels, their host launchers,
// and small device helpers (counter-based random numbers, warp/block reductions, bf16 packing).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#define SPS_MAX_ROWS 16   // activation rows one pass may carry (two 8-column MMA tiles)
#define SPS_NUM_SM_FALLBACK 148

// ------------------------------------------------------------------------------------------------
// Random numbers (see include/sps.h): Philox4x32-10, counter (t, s, b, 0), key (seed lo, seed hi).
// ------------------------------------------------------------------------------------------------
__host__ __device__ inline void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0,
                                              uint32_t k1, uint32_t out[4]) {
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    const uint64_t a = (uint64_t)0xD2511F53u * c0;
    const uint64_t b = (uint64_t)0xCD9E8D57u * c2;
    const uint32_t n0 = (uint32_t)(b >> 32) ^ c1 ^ k0;
    const uint32_t n1 = (uint32_t)b;
    const uint32_t n2 = (uint32_t)(a >> 32) ^ c3 ^ k1;
    const uint32_t n3 = (uint32_t)a;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    k0 += 0x9E3779B9u;
    k1 += 0xBB67AE85u;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// 24-bit grid in [0,1): exact in fp32
__host__ __device__ inline float u01_from_word(uint32_t w) { return (float)(w >> 8) * (1.0f / 16777216.0f); }

struct Uniforms { float u_draft, u_acc, u_res; };
__device__ inline Uniforms sps_uniforms(uint64_t seed, uint32_t b, uint32_t s, uint32_t t) {
  uint32_t w[4];
  philox4x32_10(t, s, b, 0u, (uint32_t)seed, (uint32_t)(seed >> 32), w);
  Uniforms u;
  u.u_draft = u01_from_word(w[0]);
  u.u_acc = u01_from_word(w[1]);
  u.u_res = u01_from_word(w[2]);
  return u;
}

// ------------------------------------------------------------------------------------------------
// Programmatic dependent launch: every kernel lets its successor start early (its CTAs may become
// resident and prefetch constant data) and waits for its predecessor before touching anything the
// predecessor wrote.  Without the launch attribute both instructions are no-ops.
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ void pdl_launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

bool sps_pdl_enabled();
template <class... KArgs, class... Args>
inline cudaError_t launch_k(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at;
  cfg.numAttrs = sps_pdl_enabled() ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kern, args...);
}

// ------------------------------------------------------------------------------------------------
// cudaFuncSetAttribute is per device: what a launcher remembers about it is kept per device too, so that
// handles on several GPUs of one process each set the attribute on their own device.
// ------------------------------------------------------------------------------------------------
#define SPS_MAX_DEVICES 64
struct DevSmemCache {
  size_t bytes[SPS_MAX_DEVICES];
  bool init;
};
template <class Kern>
inline cudaError_t sps_ensure_smem(Kern k, size_t bytes, DevSmemCache& c) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= SPS_MAX_DEVICES) return cudaErrorInvalidDevice;
  // 48 KB is the limit for static and dynamic shared memory TOGETHER unless the attribute says more: set it from 32 KB on
  if (!c.init) { for (size_t& b : c.bytes) b = 32 * 1024; c.init = true; }
  if (bytes <= c.bytes[dev]) return cudaSuccess;
  e = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)bytes);
  if (e == cudaSuccess) c.bytes[dev] = bytes;
  return e;
}
// one-time (per device) attribute calls: true the first time on the current device
struct DevOnce { bool done[SPS_MAX_DEVICES]; };
inline bool sps_first_on_device(DevOnce& o) {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= SPS_MAX_DEVICES) return true;
  if (o.done[dev]) return false;
  o.done[dev] = true;
  return true;
}

// Bound of every device-side wait, in nanoseconds of %globaltimer (2 s), and the test hook that shortens it and
// makes one copy producer leave out one stage, so that the give-up path of the kernels can be run on purpose
// (sps_debug_set_wait in the header).  drop_stage < 0: nothing is left out.
struct WaitKnobs { unsigned long long limit_ns; int drop_stage; };
WaitKnobs sps_wait_knobs();

// ------------------------------------------------------------------------------------------------
// Reductions with a fixed tree (results are bit-reproducible run to run).
// ------------------------------------------------------------------------------------------------
__device__ inline float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ inline float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ inline int warp_min_int(int v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = min(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}
__device__ inline int warp_max_int(int v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = max(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// ------------------------------------------------------------------------------------------------
// Device-resident state of a handle: everything a loop iteration reads or advances, so that a
// captured graph can be replayed with no host patching.
// ------------------------------------------------------------------------------------------------
struct DevState {
  // per-call parameters, written by the host before a loop / generation
  float temperature;
  float inv_temperature;
  uint32_t step;      // loop index s, advanced on the device after each loop
  uint32_t pad0;      // bits of the forced acceptance probability (0 = off): measurement mode, see sps_set_forced_acceptance
  uint64_t seed;
  float top_p;        // nucleus mass kept (1 = off), both models
  int32_t top_k;      // tokens kept (0 = off), both models
  int32_t B;          // live sequences
  int32_t max_seq;
  // per sequence
  int32_t* n;         // [B] tokens known so far
  int32_t* limit;     // [B] a sequence that has reached this many tokens stops advancing
  int32_t* tokens;    // [B][max_seq]
  int32_t* drafts;    // [B][max_K]
  // rows of the pass in flight
  int32_t* row_tok;   // [SPS_MAX_ROWS]
  int32_t* row_pos;   // [SPS_MAX_ROWS]
  // loop results
  int32_t* n_acc;     // [B]
  int32_t* out_tok;   // [B][max_K+1]
  uint32_t* flags;    // [B]
  int32_t* err;       // [1] sticky device-side error word (token out of range ...)
  int32_t max_K;
  uint32_t seq0;      // sequence b draws its random numbers as Philox sequence seq0 + b (sps_set_sequence_index0)
  uint32_t* done_counter;  // [1] CTAs of the accept kernel that finished (for the step advance)
};

// which rows a pass feeds (per sequence)
enum PassMode : int {
  PASS_PREFILL = 0,   // rows = tokens[c0 .. c0+m) of the sequence, positions the same
  PASS_DRAFT0 = 1,    // 2 rows: positions max(n-2,0), n-1          (catches the draft cache up)
  PASS_DRAFT_T = 2,   // 1 row : draft t-1 at position n-1+t
  PASS_VERIFY = 3,    // K+1 rows: x[n-1], d_0..d_{K-1} at positions n-1..n-1+K
  PASS_EXPLICIT = 4   // rows already written to row_tok / row_pos by the host
};

// ------------------------------------------------------------------------------------------------
// Linear layer  Y[M,N] = f(X)[M,D] W[N,D]^T  with fused prologue f and epilogue.
// ------------------------------------------------------------------------------------------------
enum { PRO_NONE = 0, PRO_RMSNORM = 1, PRO_GELU = 2 };
enum { EPI_STORE = 0, EPI_RESIDUAL = 1 };

struct LinArgs {
  const void* W[3];       // up to three stacked matrices (fused Q,K,V): W[0] is [rows_per_mat][D], W[1], W[2] are [rows_tail][D]
  int rows_per_mat;
  int rows_tail;          // rows of the second and third matrix (0 = rows_per_mat; fewer for grouped key / value heads)
  int N;                  // total output features = rows_per_mat + (n_mats - 1) * rows_tail
  int D;                  // input features
  int M;                  // activation rows, 1..16
  const float* X;         // [*, ldx] fp32; row of activation m is x_row0 + m * x_rowstep
  int ldx, x_row0, x_rowstep;
  int pro;                // PRO_*
  const float* gain;      // [D] fp32 (PRO_RMSNORM)
  const float* ssq_in;    // partial sums of squares of each X row (PRO_RMSNORM): SSQ_IDX(part, row), part < ssq_in_n
  int ssq_in_n;
  float eps;
  int epi;                // EPI_*
  float* Y;               // EPI_STORE: Y[m*ldy + n] = y.  EPI_RESIDUAL: Y[m*ldy + n] += y
  long long ldy;
  float* ssq_out;         // EPI_RESIDUAL: SSQ_IDX(part, m) = one CTA's share of the sum over n of the updated Y[m][n]^2
  // scratch (owned by the handle / caller): split-K partials and arrival counters
  float* part;            // [S][SPS_MAX_ROWS][N]
  int* counters;          // [2 * LIN_MAX_R + 2], zero between launches (the kernel re-zeroes what it used)
  int R, S, WC;           // row ranges, K splits, warps per CTA
  int PR;                 // rows per shared-memory pass (multiple of 32)      [register-streaming variant]
  int KS, KST, NS, G;     // k-range per CTA, k-range per stage, ring stages, warps per tile [TMA variant]
  int* err;               // sticky error word: set to 3 if a bounded wait ran out
  unsigned long long wait_ns;   // set by the launcher: bound of every wait inside the kernel
  int drop_stage;         // set by the launcher: >= 0 makes CTA 0's producer leave out that stage (test hook), -1 = none
  // Packed activations (bf16 TMA kernel only).  A layer may leave, beside Y, the next layer's input ready
  // for the tensor cores: act(y) * gain split into a bf16 high part and a bf16 remainder.  A layer given
  // such an input copies it into shared memory instead of converting X; with PRO_RMSNORM the gain is
  // already in it and the row's 1/rms (from ssq_in) multiplies the output instead of the input.
  const __nv_bfloat16* xp_hi;   // [*][ldx] packed input (row = x_row0 + m * x_rowstep), null = convert X
  const __nv_bfloat16* xp_lo;
  __nv_bfloat16* yp_hi;         // [M][ldyp] packed copy of the output, null = none
  __nv_bfloat16* yp_lo;
  long long ldyp;
  const float* yp_gain;         // [N] multiplied in before packing, null = ones
  int yp_act;                   // PRO_GELU: gelu before packing; PRO_NONE: none
  int split_epi;                // set by the launcher: the split-K epilogue runs as a kernel of its own
  // Per-tile epilogue (set by the launcher).  Each 16-row output tile is finished as soon as the last of the
  // warps that hold a share of it (k-splits x warps of a group) has written its partial sums: that warp adds the
  // k-splits in split order and stores / adds to the residual stream / packs -- no epilogue kernel, no grid-wide
  // meeting.  tile_ctr counts the arrivals per tile and is left at zero; the sums of squares of a residual
  // update are then kept per tile: ssq_out[SSQ_IDX(tile, m)].
  int tile_epi;
  int* tile_ctr;                // [ceil(N / 16)] arrival counters, zero between launches
  // int8 weights (dtype 2): W holds signed bytes, row n of matrix i is scaled by wscale[i][n] (fp32, applied to
  // the output); the activations' halves are then fp16, not bf16 -- in the slab and in the packed arrays.
  const float* wscale[3];
  int q8;                       // set by the launcher
  // Tensor-core kernel (lin_tc_kernel; set by the launcher, sk_R = 0 otherwise).  Within a k-split the sk_tot stages of
  // the layer (sk_SPT per 128-row tile) are cut into sk_R equal pieces, one per CTA; a piece that starts inside a
  // tile leaves its partial sums in carry[cta][m][row of the tile] instead of part, and the epilogue adds them in.
  float* carry;                 // [LIN_TC_MAX_CTAS][SPS_MAX_ROWS][128], null = the kernel is not used
  int sk_R, sk_SPT, sk_tot, sk_BR;   // sk_BR: weight rows per tile (64 or 128)
};

struct LinPlan { int R, S, WC, PR, NT, variant, KS, KST, NS, G, ssq_parts, tile_epi; size_t smem; };
size_t lin_tile_ctr_ints(int N);           // arrival counters a layer of N output features needs
LinPlan lin_plan(int dtype, int M, int N, int D, int num_sm);
int lin_launch_count(const LinPlan& p);   // kernels one lin_launch enqueues
cudaError_t lin_launch(int dtype, const LinArgs& a, const LinPlan& p, cudaStream_t st);
size_t lin_part_floats(int N, int S_max);
#define LIN_TC_MAX_CTAS 160
inline size_t lin_carry_floats() { return (size_t)LIN_TC_MAX_CTAS * SPS_MAX_ROWS * 128; }
struct LinTcPlan { int KBS, KBX, NS, NGRP, BR, R, SPT, tot; size_t smem; };
bool lin_tc_plan(const LinArgs& a, const LinPlan& p, LinTcPlan* out);     // can the layer run on the tcgen05 kernel, and how
cudaError_t lin_tc_launch(const LinArgs& a, const LinTcPlan& t, cudaStream_t st);
void sps_set_global_error(const char* msg);   // text returned by sps_last_error(NULL)
#define LIN_MAX_R 512
// partial sums of squares: the partials of one row are neighbours, so a warp fetches them with a few coalesced loads
#define SSQ_IDX(part, row) ((size_t)(row) * LIN_MAX_R + (size_t)(part))
#define LIN_CONSUMER_WARPS 8
#define LIN_MAX_S 64
#define LIN_SCALE_SLOT 768   // counters[768..783] as floats: the rows' 1/rms handed from the layer kernel to its epilogue kernel

// ------------------------------------------------------------------------------------------------
// Rows / embedding, attention, samplers
// ------------------------------------------------------------------------------------------------
struct EmbedArgs {
  DevState* st;
  const void* tok_embed;  // [V][d]
  int dtype, d, V;
  int mode, t, K, c0, rows_per_seq, B;
  float* x;               // [rows][d] fp32 residual stream
  float* ssq;             // SSQ_IDX(0, row): one partial per row
};
cudaError_t embed_launch(const EmbedArgs& a, cudaStream_t st);

struct AttnArgs {
  const DevState* st;
  const float* qkv;       // [rows][d + 2 * Hkv * dh]: queries, then keys, then values
  float* out;             // [rows][d]
  void* out_hi;           // when non-null: the same values split into bf16 high and low halves, [rows][d] each
  void* out_lo;           //   (the operand of a tensor-core GEMM that follows)
  void* kcache;           // this layer: [B][Hkv][max_seq][dh]
  void* vcache;
  const float2* rope;     // [max_seq][dh/2] (cos, sin)
  int dtype, H, dh, d, max_seq, rows_per_seq, B;
  int Hkv;                // key / value heads: query head h uses head h / (H / Hkv)
  int seq0;               // grid row y works on sequence seq0 + y (its cache and state) and on rows y * rows_per_seq .. of qkv / out
  int mode, t, c0;        // which rows the pass feeds (PassMode), as in EmbedArgs
  int split;              // set by the launcher: CTAs (one thread-block cluster) that share a (head, sequence)'s context
};
cudaError_t attn_launch(const AttnArgs& a, cudaStream_t st);

// ------------------------------------------------------------------------------------------------
// The prompt pass as a GEMM over up to 128 rows on tcgen05 tensor cores (wide.cu), bf16 models.
// ------------------------------------------------------------------------------------------------
#define WIDE_ROWS 128
enum { WIDE_STORE = 0, WIDE_RESIDUAL = 1, WIDE_GELU_PACK = 2 };
int wide_splits(int N, int D, int num_sm);
size_t wide_part_floats(int N, int D, int num_sm);
size_t wide_part_bound(int N, int num_sm);
int wide_gemm_launch_count(const int* rows, int nmat, int D, int num_sm);
cudaError_t wide_gemm_launch_stacked(const void* const* Ws, const int* rows, int nmat, const void* hi, const void* lo, int M, int D,
                                     float* part, int mode, float* y, long long ldy, void* yhi, void* ylo, int ldp, int* err, int num_sm,
                                     cudaStream_t st, const float* const* scales = nullptr);
cudaError_t wide_embed_launch(const DevState* st, const void* tok_embed, float* x, int rows, int d, int V, int seq, int c0, cudaStream_t s);
cudaError_t wide_pack_launch(const float* x, int ldx, const float* gain, float eps, int rows, int d, void* hi, void* lo, int ldp, cudaStream_t s);
cudaError_t wide_gemm_launch(const void* W, const void* hi, const void* lo, int M, int N, int D, float* part, int mode, float* y,
                             long long ldy, void* yhi, void* ylo, int ldp, int* err, int num_sm, cudaStream_t st,
                             const float* scale = nullptr);
cudaError_t wide_dequant_launch(const void* q, void* out, long long n, int num_sm, cudaStream_t st);
size_t attn_smem_bytes(int rows_per_seq, int max_seq, int dh);

// ------------------------------------------------------------------------------------------------
// Tensor-parallel exchange (tp.cu): the all-reduce of the partial residual updates as peer stores + a local sum
// ------------------------------------------------------------------------------------------------
#define SPS_TP_MAX_WORLD 8
struct TpArgs {
  int rank, world, rows, d;         // this rank, ranks, activation rows of the pass, d_model
  const uint32_t* epoch_ctr;        // device counter of finished exchanges (push works on *ctr + 1 and stores it; reduce reads it)
  uint32_t* epoch_ctr_w;
  size_t slot_floats;               // floats of one (parity, rank) slot of an inbox
  const float* send;                // [rows][d] this rank's partial update
  float* peer_inbox[SPS_TP_MAX_WORLD];     // every rank's inbox [2][world][slot_floats] as this device addresses it (own included)
  uint32_t* peer_flags[SPS_TP_MAX_WORLD];  // every rank's flags [world]: flags[r] = last exchange rank r has pushed
  const float* my_inbox;
  uint32_t* my_flags;
  float* x;                         // [rows][d] residual stream, updated in place
  float* ssq_out;                   // SSQ_IDX(cta, row): per-CTA sums of squares of the updated rows
  unsigned short* yp_hi;            // packed copy of gain * x for the next layer (null = none): bf16, or fp16 for int8-weight models
  unsigned short* yp_lo;
  const float* yp_gain;
  int half_is_fp16;
  int* err;
  unsigned long long wait_ns;
};
int tp_reduce_ctas(int d, int num_sm);
cudaError_t tp_push_launch(const TpArgs& a, cudaStream_t st);
cudaError_t tp_reduce_launch(const TpArgs& a, int ctas, cudaStream_t st);

struct SampleArgs {        // one inverse-CDF draw per sequence from softmax(logits/T)
  const DevState* st;      // T, seed, step come from here when st != nullptr
  const float* logits;     // row b at logits + b*ld
  long long ld;
  int V, B;
  uint32_t t;              // Philox position
  int32_t* out;            // out[b*out_ld]
  int out_ld;
  float temperature; uint64_t seed; uint32_t step;  // used when st == nullptr
  int top_k; float top_p;  // used when st == nullptr (0 / 1 = no filtering)
  int smem_weights;        // set by the launcher: weights are staged in shared memory
  float2* stats;           // when non-null: stats[b * stats_ld] = (row maximum, sum of exp((l - max) / T)) of the row drawn from
  int stats_ld;
};
cudaError_t sample_launch(const SampleArgs& a, cudaStream_t st);
// the draw spread over a thread-block cluster (unfiltered distributions, large vocabularies); else the kernel above
cudaError_t sample_launch_fast(const SampleArgs& a, bool filtered, cudaStream_t st);

struct AcceptArgs {
  DevState* st;            // when non-null: T/seed/step from the state, and the loop is advanced
  const float* q_logits;   // [B][K+1][V]
  const float* p_logits;   // [B][K][V]
  const int32_t* drafts;   // [B][drafts_ld]
  int drafts_ld;
  int B, K, V;
  int32_t* n_acc;          // [B]
  int32_t* out_tok;        // [B][out_ld]
  int out_ld;
  uint32_t* flags;         // [B]
  float temperature; uint64_t seed; uint32_t step;  // used when st == nullptr
  int top_k; float top_p;  // used when st == nullptr (0 / 1 = no filtering)
  int smem_weights;        // set by the launcher: weights are staged in shared memory
  // (row maximum, sum of exp((l - max) / T)) of each draft row, as the kernel that drew the draft tokens left them:
  // p_stats[b * p_stats_ld + t].  Null: the accept kernel works them out from p_logits itself.
  const float2* p_stats;
  int p_stats_ld;
  // set by the launcher (cluster form of the kernel): CTAs per sequence, tokens per CTA, rows resident in shared memory
  int csize, slice, resident, chunk, stages;
  unsigned long long wait_ns;   // bound of the waits on the row copies
  // The cluster kernel as the draft sampler: K = 0, one row per sequence (q_logits, row stride q_ld), the draw uses
  // u_draft of position sample_t, the token goes to out_tok[b * out_ld] and the row's (max, sum) to stats_out.
  int sample_t;                 // < 0: accept mode
  long long q_ld;               // sample mode: floats between consecutive sequences' rows
  float2* stats_out;
  int stats_ld;
};
cudaError_t accept_launch(const AcceptArgs& a, cudaStream_t st);
// the thread-block-cluster form of the same sampler (unfiltered distributions); falls back to the kernel above when
// `filtered`, for small vocabularies and for shapes it does not take
cudaError_t accept_launch_fast(const AcceptArgs& a, bool filtered, cudaStream_t st);
cudaError_t philox_launch(const uint32_t* ctr, const uint32_t* key, int n, uint32_t* out, cudaStream_t st);
