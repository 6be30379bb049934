// The C ABI of include/sps.h: handle, passes over a model, the speculative loop and its pieces.
// Host code only enqueues kernels (or replays graphs of them) and reads back a few integers per loop;
// every step of the path runs in the kernels of linear.cu, attention.cu and sampler.cu.
#include <cmath>
#include <cstdlib>
#include <cstdio>
#include <cstring>
#include <map>
#include <string>
#include <vector>

#include "../../include/sps.h"
#include "common.cuh"

namespace {

std::string g_err;  // last error of the handle-less entry points

struct ModelDev {
  sps_model_cfg cfg{};
  bool present = false;
  const void *tok_embed = nullptr, *unembed = nullptr, *final_norm = nullptr;
  std::vector<const void*> attn_norm, ffn_norm, wq, wk, wv, wo, w_up, w_down;
  char* kcache = nullptr;  // [L][B][key / value heads][max_seq][dh] in the storage type
  char* vcache = nullptr;
  size_t layer_bytes = 0;
  float2* rope = nullptr;  // [max_seq][dh/2]
  const float* unembed_scale = nullptr;   // int8 weights: row scales
  std::vector<const float*> wq_s, wk_s, wv_s, wo_s, w_up_s, w_down_s;
  bool packed = false;     // every linear layer of this model runs on the bf16 TMA kernel: activations travel packed
};

struct HostParams { float temperature, inv_temperature; uint32_t step, pad0; uint64_t seed; float top_p; int32_t top_k; };   // head of DevState

}  // namespace

void sps_set_global_error(const char* msg) { g_err = msg ? msg : ""; }

// bound of the kernels' waits and the stage a producer leaves out (test hook, sps_debug_set_wait); process-wide
static WaitKnobs g_wait_knobs = {2000000000ull, -1};
WaitKnobs sps_wait_knobs() { return g_wait_knobs; }

struct sps_handle {
  sps_cfg cfg{};
  cudaStream_t stream = nullptr;
  bool own_stream = false;
  int num_sm = SPS_NUM_SM_FALLBACK;
  ModelDev tgt, drf;
  DevState hst{};          // host image of the device state block
  DevState* dst = nullptr;
  float *x = nullptr, *qkv = nullptr, *attn = nullptr, *up = nullptr, *ssqA = nullptr, *ssqB = nullptr;
  // the prompt pass over up to 128 rows at once (bf16 models, one sequence): residual stream, q|k|v, attention output,
  // the GEMM operands' bf16 halves (normalised rows / GeLU outputs) and the k-splits' partial products
  bool wide = false;
  int max_rows = SPS_MAX_ROWS;   // rows one pass may carry: 16, or up to 128 when the target is bf16 (wide passes)
  float *wx = nullptr, *wqkv = nullptr, *watt = nullptr, *wpart = nullptr;
  void *wa_hi = nullptr, *wa_lo = nullptr, *wu_hi = nullptr, *wu_lo = nullptr;
  void* wdq = nullptr;   // bf16 copy of the int8 matrix (or q | k | v) the prompt-pass GEMM is reading
  __nv_bfloat16 *xp_hi = nullptr, *xp_lo = nullptr, *up_hi = nullptr, *up_lo = nullptr;   // packed activations (bf16 models)
  __nv_bfloat16 *ap_hi = nullptr, *ap_lo = nullptr;   // the attention output, packed by the attention kernel for the output projection
  float *q_logits = nullptr, *p_logits = nullptr, *part = nullptr;
  size_t part_floats = 0;   // floats of `part` ahead of the carry tiles
  int* counters = nullptr;
  // tensor parallelism (SPS_CFG_TENSOR_PARALLEL): this handle holds one rank's shard of both models
  bool tp = false;           // the models are shards: n_heads * d_head may be less than d_model
  bool tp_attached = false;  // sps_tp_attach has given the peers' buffers
  int tp_rank = 0, tp_world = 1;
  float* tp_send = nullptr;  // [16][d_model] this rank's partial update of the residual stream
  float* tp_inbox = nullptr; // [2][SPS_TP_MAX_WORLD][16 * d_model] partial updates received, by exchange parity and rank
  uint32_t* tp_flags = nullptr;   // [SPS_TP_MAX_WORLD] last exchange each rank has pushed here
  uint32_t* tp_epoch = nullptr;   // [1] exchanges this rank has opened
  float* tp_peer_inbox[SPS_TP_MAX_WORLD] = {nullptr};
  uint32_t* tp_peer_flags[SPS_TP_MAX_WORLD] = {nullptr};
  size_t tp_slot_floats = 0;
  int pass_nA = 1, pass_nB = 1;   // partial sums of squares in ssqA / ssqB (carried between the phases of a pass)
  float2* p_stats = nullptr; // [max_batch][max_K] (row maximum, sum of exponentials) of each draft row, left by the draft sampler
  bool filtered = false;     // top-k / nucleus / greedy in force for the calls being made (write_params)
  int* tile_ctr = nullptr;   // per-tile arrival counters of the linear layers' epilogue (zero between launches)
  size_t tile_ctr_ints = 0;
  int32_t* res = nullptr;    // device: [n_acc B][flags B][out_tok B*(maxK+1)][err 1]
  int32_t* h_res = nullptr;  // pinned mirror
  HostParams* h_par = nullptr;  // pinned
  int top_k = 0;                // sps_set_sampling: tokens kept (0 = off)
  float top_p = 1.f;            //                   nucleus mass kept (1 = off)
  float forced_accept = 0.f;    // sps_set_forced_acceptance: fixed acceptance probability (0 = off; measurement only)
  int32_t* h_rows = nullptr;    // pinned [2][16]
  size_t res_words = 0;
  int B = 0;
  int seq_len[SPS_MAX_ROWS] = {0};   // host view of n per sequence
  bool ready = false;
  std::map<int, cudaGraphExec_t> g_draft, g_verify;  // key = K * 32 + B
  std::map<int, int> warm;                          // key -> eager runs done
  cudaEvent_t ev[7]{};
  long long launches = 0;                 // kernels enqueued (graph nodes counted per replay)
  std::map<const void*, long long> graph_launches;
  std::string err;
  int last_K = -1;
  std::vector<float> trace_ms;            // per-loop record of the last generation (sps_last_loop_trace)
  std::vector<int32_t> trace_emit, trace_K;
  bool traced = false;
};

namespace {

int fail(sps_handle* h, int code, const std::string& msg) {
  if (h) h->err = msg; else g_err = msg;
  return code;
}
#define CU(h, call)                                                                         \
  do {                                                                                      \
    cudaError_t e__ = (call);                                                               \
    if (e__ != cudaSuccess)                                                                 \
      return fail(h, SPS_ECUDA, std::string(#call) + ": " + cudaGetErrorString(e__));       \
  } while (0)

size_t esize(int dtype) { return dtype == 0 ? 4 : 2; }   // embeddings and KV cache: fp32, or bf16 (also for int8-weight models)
inline int act_dtype(int dtype) { return dtype == 0 ? 0 : 1; }   // what the embedding / attention kernels see
inline int kv_heads(const sps_model_cfg& c) { return c.n_kv_heads > 0 ? c.n_kv_heads : c.n_heads; }
inline int kv_width(const sps_model_cfg& c) { return kv_heads(c) * c.d_head; }   // rows of wk / wv, numbers cached per position

inline int attn_width(const sps_model_cfg& c) { return c.n_heads * c.d_head; }   // rows of wq, columns of wo (= d_model unless the model is a tensor-parallel shard)

int check_model_cfg(const sps_model_cfg& c, std::string& why, bool shard) {
  if (c.n_layers < 0 || c.d_model <= 0 || c.n_heads <= 0 || c.d_ff <= 0 || c.vocab <= 0) { why = "non-positive model dimension"; return 0; }
  if (!shard && c.n_heads * c.d_head != c.d_model) { why = "n_heads * d_head must equal d_model"; return 0; }
  if (shard && (c.n_heads * c.d_head > c.d_model || (c.dtype >= 1 && (c.n_heads * c.d_head) % 128))) { why = "a shard's n_heads * d_head must not exceed d_model (bf16 / int8: a multiple of 128)"; return 0; }
  if (c.d_head != 64 && c.d_head != 128) { why = "d_head must be 64 or 128"; return 0; }
  if (c.n_kv_heads < 0 || c.n_heads % kv_heads(c)) { why = "n_kv_heads must be 0 or a divisor of n_heads"; return 0; }
  if (c.dtype < 0 || c.dtype > 2) { why = "dtype must be 0 (fp32), 1 (bf16) or 2 (int8 weights)"; return 0; }
  if (c.dtype >= 1 && (c.d_model % 128 || c.d_ff % 128)) { why = "bf16 / int8 models need d_model and d_ff multiples of 128"; return 0; }
  if (c.dtype == 0 && ((size_t)SPS_MAX_ROWS * (size_t)(c.d_ff > c.d_model ? c.d_ff : c.d_model) * 4 > 200 * 1024)) { why = "fp32 model too wide for the fp32 kernel"; return 0; }
  if (c.d_model % 4 || c.d_ff % 4) { why = "d_model and d_ff must be multiples of 4"; return 0; }
  return 1;
}

int load_model(sps_handle* h, ModelDev& m, const sps_model_cfg& c, const sps_weights* w, int max_seq, int max_batch) {
  m.cfg = c;
  m.present = true;
  m.tok_embed = w->tok_embed; m.unembed = w->unembed; m.final_norm = w->final_norm;
  if (!m.tok_embed || !m.unembed || !m.final_norm) return fail(h, SPS_EINVAL, "null embedding / unembedding / final_norm");
  const void* const* srcs[8] = {w->attn_norm, w->ffn_norm, w->wq, w->wk, w->wv, w->wo, w->w_up, w->w_down};
  std::vector<const void*>* dsts[8] = {&m.attn_norm, &m.ffn_norm, &m.wq, &m.wk, &m.wv, &m.wo, &m.w_up, &m.w_down};
  for (int i = 0; i < 8; ++i) {
    if (c.n_layers > 0 && !srcs[i]) return fail(h, SPS_EINVAL, "null per-layer pointer array");
    dsts[i]->assign(c.n_layers, nullptr);
    for (int l = 0; l < c.n_layers; ++l) {
      if (!srcs[i][l]) return fail(h, SPS_EINVAL, "null layer weight pointer");
      if (((uintptr_t)srcs[i][l]) & 15) return fail(h, SPS_EINVAL, "weight pointers must be 16-byte aligned");
      (*dsts[i])[l] = srcs[i][l];
    }
  }
  if (c.dtype == 2) {
    const int shapes[5][2] = {{attn_width(c) + 2 * kv_width(c), c.d_model}, {c.d_model, attn_width(c)}, {c.d_ff, c.d_model}, {c.d_model, c.d_ff}, {c.vocab, c.d_model}};
    for (int M : {1, SPS_MAX_ROWS})
      for (auto& sh : shapes)
        if (lin_plan(2, M, sh[0], sh[1], h->num_sm).variant != 2) return fail(h, SPS_EINVAL, "int8 weights: a layer width splits into more k-ranges than the kernel supports");
    m.unembed_scale = w->unembed_scale;
    if (!m.unembed_scale || ((uintptr_t)m.unembed_scale & 15)) return fail(h, SPS_EINVAL, "int8 weights need 16-byte aligned row scales");
    const float* const* ssrc[6] = {w->wq_scale, w->wk_scale, w->wv_scale, w->wo_scale, w->w_up_scale, w->w_down_scale};
    std::vector<const float*>* sdst[6] = {&m.wq_s, &m.wk_s, &m.wv_s, &m.wo_s, &m.w_up_s, &m.w_down_s};
    for (int i = 0; i < 6; ++i) {
      if (c.n_layers > 0 && !ssrc[i]) return fail(h, SPS_EINVAL, "int8 weights need row scales for every matrix");
      sdst[i]->assign(c.n_layers, nullptr);
      for (int l = 0; l < c.n_layers; ++l) {
        if (!ssrc[i][l] || ((uintptr_t)ssrc[i][l] & 15)) return fail(h, SPS_EINVAL, "int8 weights need 16-byte aligned row scales");
        (*sdst[i])[l] = ssrc[i][l];
      }
    }
  }
  m.layer_bytes = (size_t)max_batch * kv_heads(c) * (size_t)max_seq * c.d_head * esize(c.dtype);
  const size_t total = m.layer_bytes * (size_t)(c.n_layers > 0 ? c.n_layers : 1);
  if (cudaMalloc(&m.kcache, total) != cudaSuccess || cudaMalloc(&m.vcache, total) != cudaSuccess)
    return fail(h, SPS_ENOMEM, "KV cache allocation failed");
  CU(h, cudaMemsetAsync(m.kcache, 0, total, h->stream));
  CU(h, cudaMemsetAsync(m.vcache, 0, total, h->stream));
  // rotary table: angle = pos * base^(-2i/dh), computed in double, stored as fp32 (cos, sin)
  const int half = c.d_head / 2;
  std::vector<float2> tab((size_t)max_seq * half);
  for (int p = 0; p < max_seq; ++p)
    for (int i = 0; i < half; ++i) {
      const double ang = (double)p * std::pow((double)c.rope_base, -2.0 * i / c.d_head);
      tab[(size_t)p * half + i] = make_float2((float)std::cos(ang), (float)std::sin(ang));
    }
  if (cudaMalloc(&m.rope, tab.size() * sizeof(float2)) != cudaSuccess) return fail(h, SPS_ENOMEM, "rope table allocation failed");
  CU(h, cudaMemcpy(m.rope, tab.data(), tab.size() * sizeof(float2), cudaMemcpyHostToDevice));
  return SPS_OK;
}

void free_model(ModelDev& m) {
  if (m.kcache) cudaFree(m.kcache);
  if (m.vcache) cudaFree(m.vcache);
  if (m.rope) cudaFree(m.rope);
  m.kcache = m.vcache = nullptr; m.rope = nullptr;
}

// scratch need of one model's linear layers, over every row count the handle may use
size_t model_part_floats(const ModelDev& m, int num_sm) {
  if (!m.present) return 0;
  const sps_model_cfg& c = m.cfg;
  size_t need = 0;
  const int shapes[5][2] = {{attn_width(c) + 2 * kv_width(c), c.d_model}, {c.d_model, attn_width(c)}, {c.d_ff, c.d_model}, {c.d_model, c.d_ff}, {c.vocab, c.d_model}};
  for (int M : {1, SPS_MAX_ROWS})
    for (auto& s : shapes) {
      const LinPlan p = lin_plan(c.dtype, M, s[0], s[1], num_sm);
      const size_t f = lin_part_floats(s[0], p.S);
      if (f > need) need = f;
    }
  return need;
}

// packed activations need every shape of the model, at every row count, on the TMA kernel
bool model_can_pack(const ModelDev& m, int num_sm) {
  const sps_model_cfg& c = m.cfg;
  if (!m.present || c.dtype < 1) return false;
  const int shapes[5][2] = {{attn_width(c) + 2 * kv_width(c), c.d_model}, {c.d_model, attn_width(c)}, {c.d_ff, c.d_model}, {c.d_model, c.d_ff}, {c.vocab, c.d_model}};
  for (int M : {1, SPS_MAX_ROWS})
    for (auto& s : shapes)
      if (lin_plan(c.dtype, M, s[0], s[1], num_sm).variant != 2) return false;
  static const bool off = [] { const char* e = getenv("SPS_LIN_PACKED"); return e && atoi(e) == 0; }();   // tuning: 0 = convert in every layer
  return !off;
}

struct PassSpec {
  int mode, t, K, c0, rows_per_seq;
  float* logits;        // null: skip the unembedding
  long long logits_ld;  // stride between logits rows
  int lrow0, lrowstep, lrows;  // which residual rows get logits
};

// one forward pass of a model over the rows `ps` describes, for the handle's B live sequences
int run_pass_wide(sps_handle* h, ModelDev& m, const PassSpec& ps);

// The pass is a list of phases so that the ranks of a tensor-parallel group emulated on one GPU can be stepped
// through it together: phase 0 = rows + embedding; per layer l, 1 + 4 l = attention block (q | k | v, attention,
// output projection), + 1 = its exchange's reduction (sharded models only), + 2 = feed-forward block, + 3 = its
// reduction; the last phase = logits.  An unsharded model's blocks add to the residual stream themselves and its
// reduction phases are empty.
int pass_phases(const ModelDev& m) { return 2 + 4 * m.cfg.n_layers; }

TpArgs tp_args(sps_handle* h, const sps_model_cfg& c, int rows) {
  TpArgs t{};
  t.rank = h->tp_rank; t.world = h->tp_world; t.rows = rows; t.d = c.d_model;
  t.epoch_ctr = h->tp_epoch; t.epoch_ctr_w = h->tp_epoch; t.slot_floats = h->tp_slot_floats;
  t.send = h->tp_send;
  for (int w = 0; w < h->tp_world; ++w) { t.peer_inbox[w] = h->tp_peer_inbox[w]; t.peer_flags[w] = h->tp_peer_flags[w]; }
  t.my_inbox = h->tp_inbox; t.my_flags = h->tp_flags;
  t.x = h->x; t.err = h->hst.err; t.wait_ns = sps_wait_knobs().limit_ns;
  t.half_is_fp16 = c.dtype == 2 ? 1 : 0;
  return t;
}

int run_pass_range(sps_handle* h, ModelDev& m, const PassSpec& ps, int ph0, int ph1) {
  const sps_model_cfg& c = m.cfg;
  const int B = h->B, rows = B * ps.rows_per_seq, d = c.d_model, dff = c.d_ff, da = attn_width(c), dkv = kv_width(c);
  const bool tp = h->tp && h->tp_world > 1;
  if (h->tp && !h->tp_attached) return fail(h, SPS_ESTATE, "tensor-parallel handle: sps_tp_attach has not been called");
  cudaStream_t st = h->stream;
  LinArgs base{};
  base.part = h->part; base.carry = h->part + h->part_floats; base.counters = h->counters; base.tile_ctr = h->tile_ctr; base.eps = c.rms_eps;
  base.err = h->hst.err;
  const int last = pass_phases(m) - 1;
  for (int ph = ph0; ph < ph1; ++ph) {
    if (ph == 0) {
      EmbedArgs ea{};
      ea.st = h->dst; ea.tok_embed = m.tok_embed; ea.dtype = act_dtype(c.dtype); ea.d = d; ea.V = c.vocab;
      ea.mode = ps.mode; ea.t = ps.t; ea.K = ps.K; ea.c0 = ps.c0; ea.rows_per_seq = ps.rows_per_seq; ea.B = B;
      ea.x = h->x; ea.ssq = h->ssqA;
      CU(h, embed_launch(ea, st)); h->launches++;
      h->pass_nA = 1; h->pass_nB = 1;   // how many partial sums of squares sit in ssqA / ssqB
      continue;
    }
    if (ph == last) {
      if (!ps.logits) continue;
      LinArgs a = base;
      a.W[0] = m.unembed; a.rows_per_mat = c.vocab; a.N = c.vocab; a.D = d; a.M = ps.lrows;
      if (c.dtype == 2) a.wscale[0] = m.unembed_scale;
      a.X = h->x; a.ldx = d; a.x_row0 = ps.lrow0; a.x_rowstep = ps.lrowstep;
      a.pro = PRO_RMSNORM; a.gain = (const float*)m.final_norm; a.ssq_in = h->ssqA; a.ssq_in_n = h->pass_nA;
      if (m.packed) { a.xp_hi = h->xp_hi; a.xp_lo = h->xp_lo; }
      a.epi = EPI_STORE; a.Y = ps.logits; a.ldy = ps.logits_ld;
      const LinPlan pl = lin_plan(c.dtype, ps.lrows, a.N, a.D, h->num_sm);
      CU(h, lin_launch(c.dtype, a, pl, st)); h->launches += lin_launch_count(pl);
      continue;
    }
    const int l = (ph - 1) / 4, sub = (ph - 1) % 4;
    if (sub == 0) {
      {  // q, k, v = Wq h, Wk h, Wv h with h = rmsnorm(x, g_attn), one launch over the three matrices
        LinArgs a = base;
        a.W[0] = m.wq[l]; a.W[1] = m.wk[l]; a.W[2] = m.wv[l];
        if (c.dtype == 2) { a.wscale[0] = m.wq_s[l]; a.wscale[1] = m.wk_s[l]; a.wscale[2] = m.wv_s[l]; }
        a.rows_per_mat = da; a.rows_tail = dkv; a.N = da + 2 * dkv; a.D = d; a.M = rows;
        a.X = h->x; a.ldx = d; a.x_row0 = 0; a.x_rowstep = 1;
        a.pro = PRO_RMSNORM; a.gain = (const float*)m.attn_norm[l]; a.ssq_in = h->ssqA; a.ssq_in_n = h->pass_nA;
        if (m.packed && l > 0) { a.xp_hi = h->xp_hi; a.xp_lo = h->xp_lo; }   // left there by the layer below
        a.epi = EPI_STORE; a.Y = h->qkv; a.ldy = a.N;
        const LinPlan pl = lin_plan(c.dtype, rows, a.N, a.D, h->num_sm);
        CU(h, lin_launch(c.dtype, a, pl, st)); h->launches += lin_launch_count(pl);
      }
      {
        AttnArgs aa{};
        aa.st = h->dst; aa.qkv = h->qkv; aa.out = h->attn;
        aa.kcache = m.kcache + (size_t)l * m.layer_bytes; aa.vcache = m.vcache + (size_t)l * m.layer_bytes;
        aa.rope = m.rope; aa.dtype = act_dtype(c.dtype); aa.H = c.n_heads; aa.Hkv = kv_heads(c); aa.dh = c.d_head; aa.d = da;
        aa.max_seq = h->cfg.max_seq; aa.rows_per_seq = ps.rows_per_seq; aa.B = B;
        aa.mode = ps.mode; aa.t = ps.t; aa.c0 = ps.c0;
        // bf16 models: the output also as bf16 halves, ready for the output projection's tensor-core operand
        if (m.packed && c.dtype == 1) { aa.out_hi = h->ap_hi; aa.out_lo = h->ap_lo; }
        CU(h, attn_launch(aa, st)); h->launches++;
      }
      {  // x += Wo o ; also sum(x^2) for the FFN norm.  A shard's Wo (its columns) gives a partial update instead.
        LinArgs a = base;
        a.W[0] = m.wo[l]; a.rows_per_mat = d; a.N = d; a.D = da; a.M = rows;
        if (c.dtype == 2) a.wscale[0] = m.wo_s[l];
        a.X = h->attn; a.ldx = da; a.x_row0 = 0; a.x_rowstep = 1; a.pro = PRO_NONE;
        if (m.packed && c.dtype == 1) { a.xp_hi = h->ap_hi; a.xp_lo = h->ap_lo; }
        const LinPlan pl = lin_plan(c.dtype, rows, a.N, a.D, h->num_sm);
        if (tp) { a.epi = EPI_STORE; a.Y = h->tp_send; a.ldy = d; }
        else {
          a.epi = EPI_RESIDUAL; a.Y = h->x; a.ldy = d; a.ssq_out = h->ssqB;
          if (m.packed) { a.yp_hi = h->xp_hi; a.yp_lo = h->xp_lo; a.ldyp = d; a.yp_gain = (const float*)m.ffn_norm[l]; a.yp_act = PRO_NONE; }
          h->pass_nB = pl.ssq_parts;
        }
        CU(h, lin_launch(c.dtype, a, pl, st)); h->launches += lin_launch_count(pl);
        if (tp) { CU(h, tp_push_launch(tp_args(h, c, rows), st)); h->launches++; }
      }
    } else if (sub == 1 || sub == 3) {
      if (!tp) continue;
      // the exchange's second half: x += the ranks' partial updates, sums of squares and packed copy for what follows
      TpArgs t = tp_args(h, c, rows);
      const int ctas = tp_reduce_ctas(d, h->num_sm);
      const void* gain = sub == 1 ? m.ffn_norm[l] : (l + 1 < c.n_layers ? m.attn_norm[l + 1] : m.final_norm);
      t.ssq_out = sub == 1 ? h->ssqB : h->ssqA;
      if (m.packed) { t.yp_hi = (unsigned short*)h->xp_hi; t.yp_lo = (unsigned short*)h->xp_lo; t.yp_gain = (const float*)gain; }
      CU(h, tp_reduce_launch(t, ctas, st)); h->launches++;
      if (sub == 1) h->pass_nB = ctas; else h->pass_nA = ctas;
    } else {
      {  // up = Wup rmsnorm(x, g_ffn)
        LinArgs a = base;
        a.W[0] = m.w_up[l]; a.rows_per_mat = dff; a.N = dff; a.D = d; a.M = rows;
        if (c.dtype == 2) a.wscale[0] = m.w_up_s[l];
        a.X = h->x; a.ldx = d; a.x_row0 = 0; a.x_rowstep = 1;
        a.pro = PRO_RMSNORM; a.gain = (const float*)m.ffn_norm[l]; a.ssq_in = h->ssqB; a.ssq_in_n = h->pass_nB;
        a.epi = EPI_STORE; a.Y = h->up; a.ldy = dff;
        if (m.packed) {
          a.xp_hi = h->xp_hi; a.xp_lo = h->xp_lo;
          a.yp_hi = h->up_hi; a.yp_lo = h->up_lo; a.ldyp = dff; a.yp_gain = nullptr; a.yp_act = PRO_GELU;
        }
        const LinPlan pl = lin_plan(c.dtype, rows, a.N, a.D, h->num_sm);
        CU(h, lin_launch(c.dtype, a, pl, st)); h->launches += lin_launch_count(pl);
      }
      {  // x += Wdown gelu(up) ; also sum(x^2) for the next norm (a shard: a partial update)
        LinArgs a = base;
        a.W[0] = m.w_down[l]; a.rows_per_mat = d; a.N = d; a.D = dff; a.M = rows;
        if (c.dtype == 2) a.wscale[0] = m.w_down_s[l];
        a.X = h->up; a.ldx = dff; a.x_row0 = 0; a.x_rowstep = 1; a.pro = PRO_GELU;
        if (m.packed) { a.xp_hi = h->up_hi; a.xp_lo = h->up_lo; }
        const LinPlan pl = lin_plan(c.dtype, rows, a.N, a.D, h->num_sm);
        if (tp) { a.epi = EPI_STORE; a.Y = h->tp_send; a.ldy = d; }
        else {
          a.epi = EPI_RESIDUAL; a.Y = h->x; a.ldy = d; a.ssq_out = h->ssqA;
          if (m.packed) {
            a.yp_hi = h->xp_hi; a.yp_lo = h->xp_lo; a.ldyp = d; a.yp_act = PRO_NONE;
            a.yp_gain = (const float*)(l + 1 < c.n_layers ? m.attn_norm[l + 1] : m.final_norm);
          }
          h->pass_nA = pl.ssq_parts;
        }
        CU(h, lin_launch(c.dtype, a, pl, st)); h->launches += lin_launch_count(pl);
        if (tp) { CU(h, tp_push_launch(tp_args(h, c, rows), st)); h->launches++; }
      }
    }
  }
  return SPS_OK;
}

int run_pass(sps_handle* h, ModelDev& m, const PassSpec& ps) {
  const sps_model_cfg& c = m.cfg;
  const int rows = h->B * ps.rows_per_seq;
  // Up to 16 rows stream the weights once (for bf16 models through the tcgen05 weight-streaming kernel, which carries 16 rows
  // at the cost of one); the GEMM path takes over above that.  SPS_WIDE_MIN_ROWS moves the switch (tuning only).
  static const int wide_min = [] { const char* e = getenv("SPS_WIDE_MIN_ROWS"); return e ? atoi(e) : 17; }();
  if (rows > SPS_MAX_ROWS || (rows >= wide_min && h->wide && c.dtype == 1 && (!ps.logits || (ps.lrow0 == 0 && ps.lrowstep == 1 && ps.lrows == rows))))
    return run_pass_wide(h, m, ps);
  return run_pass_range(h, m, ps, 0, pass_phases(m));
}

// A pass over 17..128 rows (several sequences' K + 1 rows): the same layers, every linear layer as one GEMM on the
// tcgen05 tensor cores (wide.cu) instead of the 16-row weight-streaming kernel; attention as in run_pass, one CTA per
// (head, sequence) over that sequence's rows.  bf16 models only.
int run_pass_wide(sps_handle* h, ModelDev& m, const PassSpec& ps) {
  const sps_model_cfg& c = m.cfg;
  const int B = h->B, rows = B * ps.rows_per_seq, d = c.d_model, dff = c.d_ff, dkv = kv_width(c), ldq = d + 2 * dkv;
  if (!h->wide || c.dtype != 1 || rows > WIDE_ROWS) return fail(h, SPS_EINVAL, "more than 16 rows per pass need a bf16 model and at most 128 rows");
  if (ps.logits && (ps.lrow0 != 0 || ps.lrowstep != 1 || ps.lrows != rows)) return fail(h, SPS_EINVAL, "a wide pass computes logits for all of its rows");
  cudaStream_t st = h->stream;
  int* err = h->hst.err;
  EmbedArgs ea{};
  ea.st = h->dst; ea.tok_embed = m.tok_embed; ea.dtype = act_dtype(c.dtype); ea.d = d; ea.V = c.vocab;
  ea.mode = ps.mode; ea.t = ps.t; ea.K = ps.K; ea.c0 = ps.c0; ea.rows_per_seq = ps.rows_per_seq; ea.B = B;
  ea.x = h->wx; ea.ssq = h->ssqA;
  CU(h, embed_launch(ea, st)); h->launches++;
  for (int l = 0; l < c.n_layers; ++l) {
    CU(h, wide_pack_launch(h->wx, d, (const float*)m.attn_norm[l], c.rms_eps, rows, d, h->wa_hi, h->wa_lo, d, st));
    {
      const void* qkv_w[3] = {m.wq[l], m.wk[l], m.wv[l]};
      const int qkv_rows[3] = {d, dkv, dkv};
      CU(h, wide_gemm_launch_stacked(qkv_w, qkv_rows, 3, h->wa_hi, h->wa_lo, rows, d, h->wpart, WIDE_STORE, h->wqkv, ldq, nullptr, nullptr, 0, err, h->num_sm, st));
    }
    AttnArgs aa{};
    aa.st = h->dst; aa.qkv = h->wqkv; aa.out = h->watt;
    aa.kcache = m.kcache + (size_t)l * m.layer_bytes; aa.vcache = m.vcache + (size_t)l * m.layer_bytes;
    aa.rope = m.rope; aa.dtype = act_dtype(c.dtype); aa.H = c.n_heads; aa.Hkv = kv_heads(c); aa.dh = c.d_head; aa.d = d;
    aa.max_seq = h->cfg.max_seq; aa.rows_per_seq = ps.rows_per_seq; aa.B = B;
    aa.mode = ps.mode; aa.t = ps.t; aa.c0 = ps.c0;
    aa.out_hi = h->wa_hi; aa.out_lo = h->wa_lo;   // the next GEMM's operand, split into bf16 halves by the attention kernel
    CU(h, attn_launch(aa, st));
    CU(h, wide_gemm_launch(m.wo[l], h->wa_hi, h->wa_lo, rows, d, d, h->wpart, WIDE_RESIDUAL, h->wx, d, nullptr, nullptr, 0, err, h->num_sm, st));
    CU(h, wide_pack_launch(h->wx, d, (const float*)m.ffn_norm[l], c.rms_eps, rows, d, h->wa_hi, h->wa_lo, d, st));
    CU(h, wide_gemm_launch(m.w_up[l], h->wa_hi, h->wa_lo, rows, dff, d, h->wpart, WIDE_GELU_PACK, nullptr, 0, h->wu_hi, h->wu_lo, dff, err, h->num_sm, st));
    CU(h, wide_gemm_launch(m.w_down[l], h->wu_hi, h->wu_lo, rows, d, dff, h->wpart, WIDE_RESIDUAL, h->wx, d, nullptr, nullptr, 0, err, h->num_sm, st));
    {
      const int qr[3] = {d, dkv, dkv}, r1[1] = {d}, r2[1] = {dff};
      h->launches += 3 + wide_gemm_launch_count(qr, 3, d, h->num_sm) + wide_gemm_launch_count(r2, 1, d, h->num_sm) + wide_gemm_launch_count(r1, 1, d, h->num_sm) +
                     wide_gemm_launch_count(r1, 1, dff, h->num_sm);
    }
  }
  if (ps.logits) {
    CU(h, wide_pack_launch(h->wx, d, (const float*)m.final_norm, c.rms_eps, rows, d, h->wa_hi, h->wa_lo, d, st));
    CU(h, wide_gemm_launch(m.unembed, h->wa_hi, h->wa_lo, rows, c.vocab, d, h->wpart, WIDE_STORE, ps.logits, ps.logits_ld, nullptr, nullptr, 0, err, h->num_sm, st));
    const int rv[1] = {c.vocab};
    h->launches += 1 + wide_gemm_launch_count(rv, 1, d, h->num_sm);
  }
  return SPS_OK;
}

// K draft steps: step 0 feeds two rows per sequence (positions n-2, n-1) so that a draft cache left
// one token behind by a fully accepted loop catches up in the same fixed-shape pass
PassSpec draft_spec(sps_handle* h, int K, int t) {
  const int V = h->tgt.cfg.vocab;
  PassSpec ps{};
  ps.mode = t == 0 ? PASS_DRAFT0 : PASS_DRAFT_T; ps.t = t; ps.K = K; ps.rows_per_seq = t == 0 ? 2 : 1;
  ps.logits = h->p_logits + (size_t)t * V; ps.logits_ld = (long long)K * V;
  ps.lrow0 = t == 0 ? 1 : 0; ps.lrowstep = t == 0 ? 2 : 1; ps.lrows = h->B;
  return ps;
}

int enqueue_sample(sps_handle* h, int K, int t) {
  const PassSpec ps = draft_spec(h, K, t);
  SampleArgs sa{};
  sa.st = h->dst; sa.logits = ps.logits; sa.ld = ps.logits_ld; sa.V = h->tgt.cfg.vocab; sa.B = h->B; sa.t = (uint32_t)t;
  sa.out = h->hst.drafts + t; sa.out_ld = h->hst.max_K;
  sa.stats = h->p_stats + t; sa.stats_ld = h->hst.max_K;
  CU(h, sample_launch_fast(sa, h->filtered, h->stream)); h->launches++;
  return SPS_OK;
}

int enqueue_draft(sps_handle* h, int K) {
  for (int t = 0; t < K; ++t) {
    int rc = run_pass(h, h->drf, draft_spec(h, K, t));
    if (rc) return rc;
    if ((rc = enqueue_sample(h, K, t))) return rc;
  }
  return SPS_OK;
}

PassSpec verify_spec(sps_handle* h, int K) {
  PassSpec ps{};
  ps.mode = PASS_VERIFY; ps.K = K; ps.rows_per_seq = K + 1;
  ps.logits = h->q_logits; ps.logits_ld = h->tgt.cfg.vocab; ps.lrow0 = 0; ps.lrowstep = 1; ps.lrows = h->B * (K + 1);
  return ps;
}

int enqueue_verify(sps_handle* h, int K) { return run_pass(h, h->tgt, verify_spec(h, K)); }

int enqueue_accept(sps_handle* h, int K) {
  AcceptArgs aa{};
  aa.st = h->dst; aa.q_logits = h->q_logits; aa.p_logits = h->p_logits; aa.drafts = h->hst.drafts;
  aa.drafts_ld = h->hst.max_K; aa.B = h->B; aa.K = K; aa.V = h->tgt.cfg.vocab;
  aa.n_acc = h->hst.n_acc; aa.out_tok = h->hst.out_tok; aa.out_ld = h->hst.max_K + 1; aa.flags = h->hst.flags;
  // the draft rows' softmax statistics come from the kernel that drew the drafts (the same numbers the draws used)
  aa.p_stats = K > 0 ? h->p_stats : nullptr; aa.p_stats_ld = h->hst.max_K; aa.sample_t = -1;
  CU(h, accept_launch_fast(aa, h->filtered, h->stream)); h->launches++;
  return SPS_OK;
}

// replay (or, the first two times, run eagerly and then capture) one phase
int launch_phase(sps_handle* h, std::map<int, cudaGraphExec_t>& cache, int K, int (*enq)(sps_handle*, int), int tag) {
  if (h->cfg.flags & SPS_CFG_NO_GRAPH) return enq(h, K);
  const int key = K * 32 + h->B;
  auto it = cache.find(key);
  if (it != cache.end()) {
    CU(h, cudaGraphLaunch(it->second, h->stream));
    h->launches += h->graph_launches[(const void*)it->second];
    return SPS_OK;
  }
  int& w = h->warm[key * 2 + tag];
  if (w == 0) { ++w; return enq(h, K); }   // first use runs eagerly (it also sets kernel attributes)
  cudaGraph_t g = nullptr;
  CU(h, cudaStreamBeginCapture(h->stream, cudaStreamCaptureModeThreadLocal));
  const long long before = h->launches;
  int rc = enq(h, K);
  const long long in_graph = h->launches - before;
  cudaError_t e = cudaStreamEndCapture(h->stream, &g);
  if (rc) { if (g) cudaGraphDestroy(g); return rc; }
  if (e != cudaSuccess) return fail(h, SPS_ECUDA, std::string("graph capture: ") + cudaGetErrorString(e));
  cudaGraphExec_t ge = nullptr;
  e = cudaGraphInstantiate(&ge, g, 0);
  cudaGraphDestroy(g);
  if (e != cudaSuccess) return fail(h, SPS_ECUDA, std::string("graph instantiate: ") + cudaGetErrorString(e));
  cache[key] = ge;
  h->graph_launches[(const void*)ge] = in_graph;
  CU(h, cudaGraphLaunch(ge, h->stream));
  return SPS_OK;
}

// the device's sticky status word after a pass the host has waited for: 0, 3 (a bounded wait ran out), else a range error
int check_device_status(sps_handle* h) {
  int32_t errw = 0;
  CU(h, cudaMemcpy(&errw, h->hst.err, 4, cudaMemcpyDeviceToHost));
  if (errw == 0) return SPS_OK;
  if (errw == 3) {
    // a kernel that gave up may have left arrival counters and tile queues half-way: clear them for the next call
    cudaMemsetAsync(h->counters, 0, sizeof(int) * (2 * LIN_MAX_R + 2), h->stream);
    cudaMemsetAsync(h->tile_ctr, 0, sizeof(int) * h->tile_ctr_ints, h->stream);
    cudaMemsetAsync(h->res + (h->res_words - 1), 0, 4, h->stream);
    cudaStreamSynchronize(h->stream);
    return fail(h, SPS_ETIMEOUT, "a bounded device-side wait ran out");
  }
  return fail(h, SPS_ERANGE, "device flagged a token id or position out of range");
}

int write_params(sps_handle* h, float T, uint64_t seed, uint32_t step) {
  // temperature 0 = greedy decoding: the one-token limit of top-k, applied to both models
  const bool greedy = T == 0.f;
  if (greedy) T = 1.f;
  h->h_par->temperature = T; h->h_par->inv_temperature = 1.0f / T; h->h_par->step = step;
  std::memcpy(&h->h_par->pad0, &h->forced_accept, 4);
  h->h_par->seed = seed;
  h->h_par->top_k = greedy ? 1 : h->top_k;
  h->h_par->top_p = greedy ? 1.f : h->top_p;
  h->filtered = greedy || h->top_k >= 1 || h->top_p < 1.f;
  CU(h, cudaMemcpyAsync(h->dst, h->h_par, sizeof(HostParams), cudaMemcpyHostToDevice, h->stream));
  return SPS_OK;
}

// one loop iteration for all live sequences; results land in h->h_res after the sync
int loop_once(sps_handle* h, int K, bool timed) {
  int rc;
  if (timed) CU(h, cudaEventRecord(h->ev[0], h->stream));
  if (K > 0 && (rc = launch_phase(h, h->g_draft, K, enqueue_draft, 0))) return rc;
  if (timed) CU(h, cudaEventRecord(h->ev[1], h->stream));
  if ((rc = launch_phase(h, h->g_verify, K, enqueue_verify, 1))) return rc;
  if (timed) CU(h, cudaEventRecord(h->ev[2], h->stream));
  if ((rc = enqueue_accept(h, K))) return rc;
  if (timed) CU(h, cudaEventRecord(h->ev[3], h->stream));
  CU(h, cudaMemcpyAsync(h->h_res, h->res, h->res_words * 4, cudaMemcpyDeviceToHost, h->stream));
  CU(h, cudaStreamSynchronize(h->stream));
  h->last_K = K;
  if (h->h_res[h->res_words - 1] == 3) {
    // a kernel that gave up may have left arrival counters and tile queues half-way: clear them for the next call
    cudaMemsetAsync(h->counters, 0, sizeof(int) * (2 * LIN_MAX_R + 2), h->stream);
    cudaMemsetAsync(h->tile_ctr, 0, sizeof(int) * h->tile_ctr_ints, h->stream);
    cudaMemsetAsync(h->res + (h->res_words - 1), 0, 4, h->stream);
    cudaStreamSynchronize(h->stream);
    return fail(h, SPS_ETIMEOUT, "a bounded device-side wait ran out");
  }
  if (h->h_res[h->res_words - 1] != 0) return fail(h, SPS_ERANGE, "device flagged a token id or position out of range");
  return SPS_OK;
}

// toks: host [B][ld]; sequence b is toks[b][0 .. lens[b]) (lens == nullptr: every sequence has n tokens)
int set_sequences(sps_handle* h, const int32_t* toks, int B, int n, const int32_t* lens = nullptr, int ld = 0) {
  const int max_seq = h->cfg.max_seq;
  if (B < 1 || B > h->cfg.max_batch) return fail(h, SPS_EINVAL, "batch outside 1..max_batch");
  if (ld <= 0) ld = n;
  const int V = h->tgt.cfg.vocab;
  std::vector<int32_t> nn(B, n);
  int n_max = 0;
  for (int b = 0; b < B; ++b) {
    if (lens) nn[b] = lens[b];
    if (nn[b] < 1) return fail(h, SPS_EINVAL, "a sequence needs at least one token");
    if (nn[b] > max_seq || nn[b] > ld) return fail(h, SPS_ERANGE, "sequence longer than max_seq (or than its row of the input)");
    if (nn[b] > n_max) n_max = nn[b];
  }
  // what lies beyond a sequence's length is never meaningful: it travels as token 0
  std::vector<int32_t> stage((size_t)B * n_max, 0);
  for (int b = 0; b < B; ++b)
    for (int i = 0; i < nn[b]; ++i) {
      const int32_t t = toks[(size_t)b * ld + i];
      if (t < 0 || t >= V) return fail(h, SPS_ERANGE, "token id outside the vocabulary");
      stage[(size_t)b * n_max + i] = t;
    }
  h->B = B;
  CU(h, cudaMemcpy2DAsync(h->hst.tokens, (size_t)max_seq * 4, stage.data(), (size_t)n_max * 4, (size_t)n_max * 4, B, cudaMemcpyHostToDevice, h->stream));
  CU(h, cudaMemcpyAsync(h->hst.n, nn.data(), B * 4, cudaMemcpyHostToDevice, h->stream));
  int32_t Bv = B;
  CU(h, cudaMemcpyAsync(&h->dst->B, &Bv, 4, cudaMemcpyHostToDevice, h->stream));
  std::vector<int32_t> lim(B, 0x7fffffff);
  CU(h, cudaMemcpyAsync(h->hst.limit, lim.data(), B * 4, cudaMemcpyHostToDevice, h->stream));
  CU(h, cudaStreamSynchronize(h->stream));  // stage / nn / lim are stack-lifetime host buffers
  for (int b = 0; b < B; ++b) h->seq_len[b] = nn[b];
  return SPS_OK;
}

// both caches ingest positions 0..n-2 of every live sequence
// The prompt pass of a bf16 model for one sequence of the batch, in chunks of up to 128 rows: every linear layer is one GEMM on the
// tcgen05 tensor cores (wide.cu), so a chunk reads the weights once; attention runs the decode kernel over 16 of the
// chunk's rows at a time (earlier rows' keys come from the cache, which the chunk's earlier launches have filled).
// No logits: the prompt's last token is fed by the first loop.
int prefill_wide(sps_handle* h, ModelDev& m, int n, int seq) {
  const sps_model_cfg& c = m.cfg;
  const int d = c.d_model, dff = c.d_ff, dkv = kv_width(c), ldq = d + 2 * dkv;
  cudaStream_t st = h->stream;
  int* err = h->hst.err;
  const bool q8 = c.dtype == 2;
  // int8 weights: the GEMM reads a bf16 copy made just before it (bytes are exact in bf16); the row scales multiply the sums
  cudaError_t dq_err = cudaSuccess;
  auto Wb = [&](const void* w, size_t elems, size_t at) -> const void* {
    if (!q8) return w;
    __nv_bfloat16* dst = reinterpret_cast<__nv_bfloat16*>(h->wdq) + at;
    const cudaError_t e = wide_dequant_launch(w, dst, (long long)elems, h->num_sm, st);
    if (e != cudaSuccess) dq_err = e;
    h->launches++;
    return dst;
  };
  for (int c0 = 0; c0 < n - 1; c0 += WIDE_ROWS) {
    const int rows = (n - 1 - c0) < WIDE_ROWS ? (n - 1 - c0) : WIDE_ROWS;
    CU(h, wide_embed_launch(h->dst, m.tok_embed, h->wx, rows, d, c.vocab, seq, c0, st)); h->launches++;
    for (int l = 0; l < c.n_layers; ++l) {
      CU(h, wide_pack_launch(h->wx, d, (const float*)m.attn_norm[l], c.rms_eps, rows, d, h->wa_hi, h->wa_lo, d, st));
      {
        const void* qkv_w[3] = {Wb(m.wq[l], (size_t)d * d, 0), Wb(m.wk[l], (size_t)dkv * d, (size_t)d * d),
                                Wb(m.wv[l], (size_t)dkv * d, (size_t)d * d + (size_t)dkv * d)};
        const int qkv_rows[3] = {d, dkv, dkv};
        const float* qkv_s[3] = {q8 ? m.wq_s[l] : nullptr, q8 ? m.wk_s[l] : nullptr, q8 ? m.wv_s[l] : nullptr};
        CU(h, wide_gemm_launch_stacked(qkv_w, qkv_rows, 3, h->wa_hi, h->wa_lo, rows, d, h->wpart, WIDE_STORE, h->wqkv, ldq, nullptr, nullptr, 0, err, h->num_sm, st,
                                       q8 ? qkv_s : nullptr));
      }
      {
        const int qr[3] = {d, dkv, dkv}, r1[1] = {d}, r2[1] = {dff};
        // pack, q|k|v GEMM; pack, up GEMM; wo and down GEMMs (attention launches are counted where they are made)
        h->launches += 2 + wide_gemm_launch_count(qr, 3, d, h->num_sm) + wide_gemm_launch_count(r2, 1, d, h->num_sm) + wide_gemm_launch_count(r1, 1, d, h->num_sm) +
                       wide_gemm_launch_count(r1, 1, dff, h->num_sm);
      }
      for (int r0 = 0; r0 < rows; r0 += SPS_MAX_ROWS) {
        AttnArgs aa{};
        aa.st = h->dst; aa.qkv = h->wqkv + (size_t)r0 * ldq; aa.out = h->watt + (size_t)r0 * d;
        aa.kcache = m.kcache + (size_t)l * m.layer_bytes; aa.vcache = m.vcache + (size_t)l * m.layer_bytes;
        aa.rope = m.rope; aa.dtype = act_dtype(c.dtype); aa.H = c.n_heads; aa.Hkv = kv_heads(c); aa.dh = c.d_head; aa.d = d;
        aa.max_seq = h->cfg.max_seq; aa.rows_per_seq = (rows - r0) < SPS_MAX_ROWS ? (rows - r0) : SPS_MAX_ROWS; aa.B = 1;
        aa.mode = PASS_PREFILL; aa.t = 0; aa.c0 = c0 + r0; aa.seq0 = seq;
        // the attention output is the next GEMM's operand: the kernel leaves it split into bf16 halves as well
        aa.out_hi = reinterpret_cast<__nv_bfloat16*>(h->wa_hi) + (size_t)r0 * d;
        aa.out_lo = reinterpret_cast<__nv_bfloat16*>(h->wa_lo) + (size_t)r0 * d;
        CU(h, attn_launch(aa, st)); h->launches++;
      }
      CU(h, wide_gemm_launch(Wb(m.wo[l], (size_t)d * d, 0), h->wa_hi, h->wa_lo, rows, d, d, h->wpart, WIDE_RESIDUAL, h->wx, d, nullptr, nullptr, 0, err, h->num_sm, st,
                             q8 ? m.wo_s[l] : nullptr));
      CU(h, wide_pack_launch(h->wx, d, (const float*)m.ffn_norm[l], c.rms_eps, rows, d, h->wa_hi, h->wa_lo, d, st));
      CU(h, wide_gemm_launch(Wb(m.w_up[l], (size_t)dff * d, 0), h->wa_hi, h->wa_lo, rows, dff, d, h->wpart, WIDE_GELU_PACK, nullptr, 0, h->wu_hi, h->wu_lo, dff, err, h->num_sm, st,
                             q8 ? m.w_up_s[l] : nullptr));
      CU(h, wide_gemm_launch(Wb(m.w_down[l], (size_t)dff * d, 0), h->wu_hi, h->wu_lo, rows, d, dff, h->wpart, WIDE_RESIDUAL, h->wx, d, nullptr, nullptr, 0, err, h->num_sm, st,
                             q8 ? m.w_down_s[l] : nullptr));
      CU(h, dq_err);
    }
  }
  return SPS_OK;
}

// (positions 0 .. seq_len[b] - 2 of sequence b; with ragged lengths the 16-row pass runs every sequence up to the
// longest one -- the rows beyond a sequence's own length write cache positions that its first loop overwrites
// before anything reads them)
int prefill_all(sps_handle* h) {
  const int per = SPS_MAX_ROWS / h->B;
  int n = 0;
  for (int b = 0; b < h->B; ++b) n = h->seq_len[b] > n ? h->seq_len[b] : n;
  for (int which = 0; which < 2; ++which) {
    ModelDev& m = which == 0 ? h->tgt : h->drf;
    if (!m.present) continue;
    if (h->wide && m.cfg.dtype >= 1 && n - 1 > SPS_MAX_ROWS / h->B) {
      // one sequence after the other, each in chunks of 128 rows
      for (int b = 0; b < h->B; ++b) {
        int rc = prefill_wide(h, m, h->seq_len[b], b);
        if (rc) return rc;
      }
      continue;
    }
    for (int c0 = 0; c0 < n - 1; c0 += per) {
      PassSpec ps{};
      ps.mode = PASS_PREFILL; ps.c0 = c0; ps.rows_per_seq = (n - 1 - c0) < per ? (n - 1 - c0) : per;
      int rc = run_pass(h, m, ps);
      if (rc) return rc;
    }
  }
  h->ready = true;
  return SPS_OK;
}

void add_loop_stats(sps_stats* s, int K, int a, uint32_t fl) {
  s->loops += 1;
  s->draft_calls += K;
  s->emitted += a + 1;
  s->accepted += a;
  if (fl & SPS_FLAG_RESAMPLED) s->resampled += 1;
  if (fl & SPS_FLAG_BONUS) s->bonus += 1;
  if (fl & SPS_FLAG_FALLBACK) s->fallback += 1;
  s->hist_emitted[a + 1] += 1;
}

int check_K(sps_handle* h, int K) {
  if (K < 0 || K > h->cfg.max_K) return fail(h, SPS_EINVAL, "K outside 0..max_K");
  if (K > 0 && !h->drf.present) return fail(h, SPS_EINVAL, "K > 0 needs a draft model");
  if (h->B * (K + 1) > h->max_rows) return fail(h, SPS_EINVAL, "batch * (K + 1) exceeds the rows one pass may carry (16; 128 with a bf16 target)");
  if (h->B * (K + 1) > SPS_MAX_ROWS && !(h->wide && h->tgt.cfg.dtype == 1)) return fail(h, SPS_EINVAL, "more than 16 rows per pass need a bf16 target");
  return SPS_OK;
}

}  // namespace

// ================================================================================================
extern "C" {

const char* sps_last_error(sps_handle* h) { return h ? h->err.c_str() : g_err.c_str(); }

int sps_create(const sps_weights* target_w, const sps_weights* draft_w, const sps_cfg* cfg, sps_handle** out) {
  if (!target_w || !cfg || !out) return fail(nullptr, SPS_EINVAL, "null argument");
  *out = nullptr;
  std::string why;
  const bool shard = (cfg->flags & SPS_CFG_TENSOR_PARALLEL) != 0;
  if (!check_model_cfg(cfg->target, why, shard)) return fail(nullptr, SPS_EINVAL, "target: " + why);
  if (draft_w) {
    if (!check_model_cfg(cfg->draft, why, shard)) return fail(nullptr, SPS_EINVAL, "draft: " + why);
    if (cfg->draft.vocab != cfg->target.vocab) return fail(nullptr, SPS_EINVAL, "draft and target vocabularies differ");
  }
  if (cfg->max_K < 0 || cfg->max_K > SPS_MAX_K) return fail(nullptr, SPS_EINVAL, "max_K outside 0..15");
  const int want_rows = cfg->max_batch * (cfg->max_K + 1);
  if (cfg->max_batch < 1 || cfg->max_batch * 2 > SPS_MAX_ROWS || want_rows > WIDE_ROWS || (want_rows > SPS_MAX_ROWS && cfg->target.dtype != 1))
    return fail(nullptr, SPS_EINVAL, "max_batch * (max_K + 1) must be <= 16 (<= 128 with a bf16 target), max_batch <= 8");
  if (cfg->max_seq < 2) return fail(nullptr, SPS_EINVAL, "max_seq too small");
  {
    const int dh_max = (draft_w && cfg->draft.d_head > cfg->target.d_head) ? cfg->draft.d_head : cfg->target.d_head;
    if (attn_smem_bytes(SPS_MAX_ROWS / cfg->max_batch, cfg->max_seq, dh_max) > 220 * 1024)
      return fail(nullptr, SPS_EINVAL, "max_seq too large for the attention kernel's score buffer");
  }
  cudaError_t e = cudaSetDevice(cfg->device);
  if (e != cudaSuccess) return fail(nullptr, SPS_ECUDA, std::string("cudaSetDevice: ") + cudaGetErrorString(e));
  sps_handle* h = new sps_handle();
  h->cfg = *cfg;
  int rc = SPS_OK;
  auto bail = [&](int code) { g_err = h->err; sps_destroy(h); return code; };
  cudaDeviceGetAttribute(&h->num_sm, cudaDevAttrMultiProcessorCount, cfg->device);
  if (cfg->stream) h->stream = (cudaStream_t)cfg->stream;
  else {
    if (cudaStreamCreateWithFlags(&h->stream, cudaStreamNonBlocking) != cudaSuccess) return bail(fail(h, SPS_ECUDA, "stream creation failed"));
    h->own_stream = true;
  }
  for (auto& ev : h->ev) if (cudaEventCreate(&ev) != cudaSuccess) return bail(fail(h, SPS_ECUDA, "event creation failed"));
  if ((rc = load_model(h, h->tgt, cfg->target, target_w, cfg->max_seq, cfg->max_batch))) return bail(rc);
  if (draft_w && (rc = load_model(h, h->drf, cfg->draft, draft_w, cfg->max_seq, cfg->max_batch))) return bail(rc);
  h->tgt.packed = model_can_pack(h->tgt, h->num_sm);
  h->drf.packed = model_can_pack(h->drf, h->num_sm);

  const int V = cfg->target.vocab, maxK = cfg->max_K > 0 ? cfg->max_K : 1, MB = cfg->max_batch;
  int dmax = cfg->target.d_model, fmax = cfg->target.d_ff;
  if (draft_w) { if (cfg->draft.d_model > dmax) dmax = cfg->draft.d_model; if (cfg->draft.d_ff > fmax) fmax = cfg->draft.d_ff; }
  size_t part_floats = model_part_floats(h->tgt, h->num_sm);
  const size_t pf2 = model_part_floats(h->drf, h->num_sm);
  if (pf2 > part_floats) part_floats = pf2;
  if (part_floats == 0) part_floats = 1;
  part_floats = (part_floats + 63) / 64 * 64;
  h->part_floats = part_floats;
  h->res_words = (size_t)MB * 2 + (size_t)MB * (maxK + 1) + 1;
  {
    int n_max = V;
    for (const ModelDev* m : {&h->tgt, &h->drf})
      if (m->present) n_max = std::max(n_max, std::max(m->cfg.d_ff, m->cfg.d_model + 2 * kv_width(m->cfg)));
    h->tile_ctr_ints = lin_tile_ctr_ints(n_max);
  }
  {
    // buffers of the 128-row prompt pass, when a bf16 model is there to use it (SPS_WIDE_PREFILL=0 keeps the 16-row pass)
    static const bool off = [] { const char* e = getenv("SPS_WIDE_PREFILL"); return e && atoi(e) == 0; }();
    size_t wd = 0, wf = 0, wpart = 0, wdq = 0;
    for (const ModelDev* m : {&h->tgt, &h->drf}) {
      if (!m->present || m->cfg.dtype < 1) continue;
      const sps_model_cfg& c = m->cfg;
      if (c.dtype == 2) wdq = std::max(wdq, std::max((size_t)c.d_ff * c.d_model, (size_t)(c.d_model + 2 * kv_width(c)) * c.d_model));
      wd = std::max(wd, (size_t)c.d_model); wf = std::max(wf, (size_t)c.d_ff);
      for (int n_out : {c.d_model + 2 * kv_width(c), c.d_ff, c.vocab}) wpart = std::max(wpart, wide_part_bound(n_out, h->num_sm));
    }
    if (wd > 0 && !off && !shard) {     // (a tensor-parallel shard keeps the 16-row passes)
      struct WW { void** p; size_t bytes; };
      const WW ww[] = {{(void**)&h->wx, sizeof(float) * WIDE_ROWS * wd},       {(void**)&h->wqkv, sizeof(float) * WIDE_ROWS * 3 * wd},
                       {(void**)&h->watt, sizeof(float) * WIDE_ROWS * wd},     {(void**)&h->wpart, sizeof(float) * wpart},
                       {&h->wa_hi, 2 * (size_t)WIDE_ROWS * wd},                {&h->wa_lo, 2 * (size_t)WIDE_ROWS * wd},
                       {&h->wu_hi, 2 * (size_t)WIDE_ROWS * wf},                {&h->wu_lo, 2 * (size_t)WIDE_ROWS * wf},
                       {&h->wdq, 2 * (wdq > 0 ? wdq : 8)}};
      for (const WW& w : ww) {
        if (cudaMalloc(w.p, w.bytes) != cudaSuccess) return bail(fail(h, SPS_ENOMEM, "device allocation failed"));
        if (cudaMemsetAsync(*w.p, 0, w.bytes, h->stream) != cudaSuccess) return bail(fail(h, SPS_ECUDA, "memset failed"));
      }
      h->wide = true;
    }
    if (want_rows > SPS_MAX_ROWS) {
      if (!h->wide) return bail(fail(h, SPS_EINVAL, "more than 16 rows per pass need the wide passes (SPS_WIDE_PREFILL=0 turns them off)"));
      h->max_rows = want_rows;
    }
  }
  const size_t MR = (size_t)h->max_rows, PR = std::max((size_t)SPS_MAX_ROWS, (size_t)cfg->max_batch * (size_t)(cfg->max_K > 0 ? cfg->max_K : 1));
  struct Want { void** p; size_t bytes; };
  DevState& s = h->hst;
  const Want wants[] = {
      {(void**)&h->x, sizeof(float) * SPS_MAX_ROWS * (size_t)dmax},
      {(void**)&h->qkv, sizeof(float) * SPS_MAX_ROWS * 3 * (size_t)dmax},
      {(void**)&h->attn, sizeof(float) * SPS_MAX_ROWS * (size_t)dmax},
      {(void**)&h->up, sizeof(float) * SPS_MAX_ROWS * (size_t)fmax},
      {(void**)&h->xp_hi, sizeof(__nv_bfloat16) * SPS_MAX_ROWS * (size_t)dmax},
      {(void**)&h->xp_lo, sizeof(__nv_bfloat16) * SPS_MAX_ROWS * (size_t)dmax},
      {(void**)&h->ap_hi, sizeof(__nv_bfloat16) * SPS_MAX_ROWS * (size_t)dmax},
      {(void**)&h->ap_lo, sizeof(__nv_bfloat16) * SPS_MAX_ROWS * (size_t)dmax},
      {(void**)&h->up_hi, sizeof(__nv_bfloat16) * SPS_MAX_ROWS * (size_t)fmax},
      {(void**)&h->up_lo, sizeof(__nv_bfloat16) * SPS_MAX_ROWS * (size_t)fmax},
      {(void**)&h->ssqA, sizeof(float) * LIN_MAX_R * MR},
      {(void**)&h->ssqB, sizeof(float) * LIN_MAX_R * SPS_MAX_ROWS},
      {(void**)&h->q_logits, sizeof(float) * MR * (size_t)V},
      {(void**)&h->p_logits, sizeof(float) * PR * (size_t)V},
      {(void**)&h->part, sizeof(float) * (part_floats + lin_carry_floats())},   // split-K partial sums, then the tensor-core kernel's carry tiles
      {(void**)&h->counters, sizeof(int) * (2 * LIN_MAX_R + 2)},
      {(void**)&h->tile_ctr, sizeof(int) * h->tile_ctr_ints},
      {(void**)&h->p_stats, sizeof(float2) * (size_t)MB * maxK},
      {(void**)&h->tp_send, shard ? sizeof(float) * SPS_MAX_ROWS * (size_t)dmax : 16},
      {(void**)&h->tp_inbox, shard ? sizeof(float) * 2 * SPS_TP_MAX_WORLD * SPS_MAX_ROWS * (size_t)dmax : 16},
      {(void**)&h->tp_flags, sizeof(uint32_t) * SPS_TP_MAX_WORLD},
      {(void**)&h->tp_epoch, sizeof(uint32_t) * 4},
      {(void**)&h->res, 4 * h->res_words},
      {(void**)&h->dst, sizeof(DevState)},
      {(void**)&s.n, 4 * (size_t)MB},
      {(void**)&s.limit, 4 * (size_t)MB},
      {(void**)&s.tokens, 4 * (size_t)MB * cfg->max_seq},
      {(void**)&s.drafts, 4 * (size_t)MB * maxK},
      {(void**)&s.row_tok, 4 * MR},
      {(void**)&s.row_pos, 4 * MR},
      {(void**)&s.done_counter, 4},
  };
  for (const Want& w : wants) {
    if (cudaMalloc(w.p, w.bytes) != cudaSuccess) return bail(fail(h, SPS_ENOMEM, "device allocation failed"));
    if (cudaMemsetAsync(*w.p, 0, w.bytes, h->stream) != cudaSuccess) return bail(fail(h, SPS_ECUDA, "memset failed"));
  }
  if (cudaMallocHost(&h->h_res, 4 * h->res_words) != cudaSuccess || cudaMallocHost(&h->h_par, sizeof(HostParams)) != cudaSuccess ||
      cudaMallocHost(&h->h_rows, 4 * 2 * SPS_MAX_ROWS) != cudaSuccess)
    return bail(fail(h, SPS_ENOMEM, "pinned host allocation failed"));
  s.temperature = 1.f; s.inv_temperature = 1.f; s.step = 0; s.seed = 0; s.top_p = 1.f; s.top_k = 0; s.B = 1; s.max_seq = cfg->max_seq; s.max_K = maxK; s.seq0 = 0;
  s.n_acc = h->res;
  s.flags = (uint32_t*)(h->res + MB);
  s.out_tok = h->res + 2 * MB;
  s.err = h->res + (h->res_words - 1);
  if (cudaMemcpyAsync(h->dst, &h->hst, sizeof(DevState), cudaMemcpyHostToDevice, h->stream) != cudaSuccess ||
      cudaStreamSynchronize(h->stream) != cudaSuccess)
    return bail(fail(h, SPS_ECUDA, "state upload failed"));
  h->B = 1;
  h->tp = shard;
  h->tp_slot_floats = (size_t)SPS_MAX_ROWS * dmax;
  *out = h;
  return SPS_OK;
}

int sps_destroy(sps_handle* h) {
  if (!h) return SPS_OK;
  cudaSetDevice(h->cfg.device);
  if (h->stream) cudaStreamSynchronize(h->stream);
  for (auto& kv : h->g_draft) cudaGraphExecDestroy(kv.second);
  for (auto& kv : h->g_verify) cudaGraphExecDestroy(kv.second);
  free_model(h->tgt);
  free_model(h->drf);
  void* bufs[] = {h->wdq, h->wx, h->wqkv, h->watt, h->wpart, h->wa_hi, h->wa_lo, h->wu_hi, h->wu_lo, h->xp_hi, h->xp_lo, h->ap_hi, h->ap_lo, h->up_hi, h->up_lo, h->x, h->qkv, h->attn, h->up, h->ssqA, h->ssqB, h->q_logits, h->p_logits, h->part,
                  h->counters, h->tile_ctr, h->p_stats, h->tp_send, h->tp_inbox, h->tp_flags, h->tp_epoch, h->res, h->dst, h->hst.n, h->hst.limit, h->hst.tokens, h->hst.drafts, h->hst.row_tok,
                  h->hst.row_pos, h->hst.done_counter};
  for (void* p : bufs) if (p) cudaFree(p);
  if (h->h_res) cudaFreeHost(h->h_res);
  if (h->h_par) cudaFreeHost(h->h_par);
  if (h->h_rows) cudaFreeHost(h->h_rows);
  for (auto& ev : h->ev) if (ev) cudaEventDestroy(ev);
  if (h->own_stream && h->stream) cudaStreamDestroy(h->stream);
  delete h;
  return SPS_OK;
}

int sps_reset(sps_handle* h) {
  if (!h) return fail(nullptr, SPS_EINVAL, "null handle");
  CU(h, cudaSetDevice(h->cfg.device));
  h->ready = false;
  h->B = 1;
  for (int& v : h->seq_len) v = 0;
  CU(h, cudaMemsetAsync(h->hst.n, 0, 4 * (size_t)h->cfg.max_batch, h->stream));
  CU(h, cudaMemsetAsync(h->res, 0, 4 * h->res_words, h->stream));
  CU(h, cudaMemsetAsync(h->hst.done_counter, 0, 4, h->stream));
  CU(h, cudaStreamSynchronize(h->stream));
  return SPS_OK;
}

int sps_prefill(sps_handle* h, const int32_t* toks, int32_t n) {
  if (!h || !toks) return fail(h, SPS_EINVAL, "null argument");
  CU(h, cudaSetDevice(h->cfg.device));
  int rc = set_sequences(h, toks, 1, n);
  if (rc) return rc;
  if ((rc = prefill_all(h))) return rc;
  CU(h, cudaStreamSynchronize(h->stream));
  return check_device_status(h);
}

int sps_prefill_batch(sps_handle* h, const int32_t* toks, const int32_t* lens, int32_t B, int32_t ld) {
  if (!h || !toks || !lens) return fail(h, SPS_EINVAL, "null argument");
  CU(h, cudaSetDevice(h->cfg.device));
  int rc = set_sequences(h, toks, B, 0, lens, ld);
  if (rc) return rc;
  if ((rc = prefill_all(h))) return rc;
  CU(h, cudaStreamSynchronize(h->stream));
  return check_device_status(h);
}

int sps_set_sequence_index0(sps_handle* h, uint32_t index0) {
  if (!h) return fail(nullptr, SPS_EINVAL, "null handle");
  CU(h, cudaSetDevice(h->cfg.device));
  h->hst.seq0 = index0;
  CU(h, cudaMemcpyAsync(&h->dst->seq0, &h->hst.seq0, 4, cudaMemcpyHostToDevice, h->stream));
  CU(h, cudaStreamSynchronize(h->stream));
  return SPS_OK;
}

int sps_debug_set_wait(int64_t limit_us, int32_t drop_stage) {
  if (limit_us < 0 || limit_us > 2000000) return fail(nullptr, SPS_EINVAL, "limit_us outside 0..2000000 (0 = the default of 2 s)");
  g_wait_knobs.limit_ns = limit_us == 0 ? 2000000000ull : (unsigned long long)limit_us * 1000ull;
  g_wait_knobs.drop_stage = drop_stage < 0 ? -1 : drop_stage;
  return SPS_OK;
}

int sps_step(sps_handle* h, int32_t K, float temperature, uint64_t seed, uint32_t step, int32_t* out_tokens,
             int32_t* out_n_emitted, uint32_t* out_flags) {
  if (!h || !out_tokens || !out_n_emitted) return fail(h, SPS_EINVAL, "null argument");
  if (!h->ready) return fail(h, SPS_ESTATE, "sps_step before sps_prefill");
  if (!(temperature >= 0.f)) return fail(h, SPS_EINVAL, "temperature must be >= 0 (0 = greedy)");
  CU(h, cudaSetDevice(h->cfg.device));
  int rc = check_K(h, K);
  if (rc) return rc;
  for (int b = 0; b < h->B; ++b)
    if (h->seq_len[b] + K + 1 > h->cfg.max_seq) return fail(h, SPS_ERANGE, "sequence would exceed max_seq");
  if ((rc = write_params(h, temperature, seed, step))) return rc;
  if ((rc = loop_once(h, K, false))) return rc;
  const int MB = h->cfg.max_batch, ld = h->hst.max_K + 1;
  for (int b = 0; b < h->B; ++b) {
    const int a = h->h_res[b];
    out_n_emitted[b] = a + 1;
    if (out_flags) out_flags[b] = (uint32_t)h->h_res[MB + b];
    for (int i = 0; i <= K; ++i) out_tokens[b * (K + 1) + i] = h->h_res[2 * MB + b * ld + i];
    h->seq_len[b] += a + 1;
  }
  return SPS_OK;
}

int sps_last_logits(sps_handle* h, int32_t K, float* q_logits, float* p_logits, int32_t* drafts) {
  if (!h) return fail(nullptr, SPS_EINVAL, "null handle");
  if (K != h->last_K) return fail(h, SPS_ESTATE, "K differs from the last step's");
  CU(h, cudaSetDevice(h->cfg.device));
  const size_t V = h->tgt.cfg.vocab;
  if (q_logits) CU(h, cudaMemcpyAsync(q_logits, h->q_logits, 4 * V * h->B * (K + 1), cudaMemcpyDeviceToHost, h->stream));
  if (p_logits && K > 0) CU(h, cudaMemcpyAsync(p_logits, h->p_logits, 4 * V * h->B * K, cudaMemcpyDeviceToHost, h->stream));
  if (drafts && K > 0)
    CU(h, cudaMemcpy2DAsync(drafts, (size_t)K * 4, h->hst.drafts, (size_t)h->hst.max_K * 4, (size_t)K * 4, h->B, cudaMemcpyDeviceToHost, h->stream));
  CU(h, cudaStreamSynchronize(h->stream));
  return SPS_OK;
}

int sps_last_loop_trace(sps_handle* h, float* loop_ms, int32_t* loop_emitted, int32_t* loop_K, int32_t cap, int32_t* out_loops) {
  if (!h || !out_loops || cap < 0) return fail(h, SPS_EINVAL, "null argument");
  if (!h->traced) return fail(h, SPS_ESTATE, "no generation has run on this handle");
  const size_t n = h->trace_ms.size(), m = n < (size_t)cap ? n : (size_t)cap;
  for (size_t i = 0; i < m; ++i) {
    if (loop_ms) loop_ms[i] = h->trace_ms[i];
    if (loop_emitted) loop_emitted[i] = h->trace_emit[i];
    if (loop_K) loop_K[i] = h->trace_K[i];
  }
  *out_loops = (int32_t)n;
  return SPS_OK;
}

// K_min == K: fixed lookahead.  K_min < K: the lookahead moves between K_min and K from loop to loop (see
// sps_generate_adaptive in the header); one sequence only.
static int generate_impl(sps_handle* h, const int32_t* prompts, int B, int P, int n_new, int K_min, int K, float T, uint64_t seed,
                         int32_t* out_tokens, sps_stats* out_stats) {
  if (!h || !prompts || !out_tokens) return fail(h, SPS_EINVAL, "null argument");
  if (n_new < 1) return fail(h, SPS_EINVAL, "n_new must be >= 1");
  if (!(T >= 0.f)) return fail(h, SPS_EINVAL, "temperature must be >= 0 (0 = greedy)");
  CU(h, cudaSetDevice(h->cfg.device));
  if (P < 1) return fail(h, SPS_EINVAL, "prompt_len must be >= 1");
  if ((long long)P + n_new + K > h->cfg.max_seq) return fail(h, SPS_ERANGE, "prompt_len + n_new + K exceeds max_seq");
  int rc = sps_reset(h);
  if (rc) return rc;
  h->B = B;
  if ((rc = check_K(h, K))) return rc;
  const int K_max = K;
  if (K_min != K) {
    if (B != 1) return fail(h, SPS_EINVAL, "adaptive lookahead runs one sequence");
    if (K_min < 1 || K_min > K) return fail(h, SPS_EINVAL, "K_min outside 1..K_max");
    K = (K_min + K_max) / 2;
  }
  CU(h, cudaEventRecord(h->ev[4], h->stream));
  if ((rc = set_sequences(h, prompts, B, P))) return rc;
  {
    std::vector<int32_t> lim(B, P + n_new);
    CU(h, cudaMemcpy(h->hst.limit, lim.data(), B * 4, cudaMemcpyHostToDevice));
  }
  cudaEvent_t e_pre0 = h->ev[4];
  CU(h, cudaEventRecord(e_pre0, h->stream));
  if ((rc = prefill_all(h))) return rc;
  // the attention kernel may fetch cache rows of earlier loops before it waits for its predecessor;
  // that is only sound if the host has waited for the stream since those rows were written
  CU(h, cudaStreamSynchronize(h->stream));
  if ((rc = write_params(h, T, seed, 0u))) return rc;
  std::vector<sps_stats> st(B);
  for (auto& s : st) std::memset(&s, 0, sizeof(s));
  std::vector<int> made(B, 0);
  const int MB = h->cfg.max_batch, ld = h->hst.max_K + 1;
  float ms_draft = 0.f, ms_verify = 0.f, ms_accept = 0.f, ms_prefill = 0.f, ms_decode = 0.f;
  bool first = true;
  const long long launches0 = h->launches;
  h->trace_ms.clear(); h->trace_emit.clear(); h->trace_K.clear();
  h->traced = true;
  CU(h, cudaEventRecord(h->ev[5], h->stream));
  for (;;) {
    bool all = true;
    for (int b = 0; b < B; ++b) all = all && made[b] >= n_new;
    if (all) break;
    if ((rc = loop_once(h, K, true))) return rc;
    float a01 = 0, a12 = 0, a23 = 0;
    if (first) { cudaEventElapsedTime(&ms_prefill, e_pre0, h->ev[5]); first = false; }
    cudaEventElapsedTime(&a01, h->ev[0], h->ev[1]);
    cudaEventElapsedTime(&a12, h->ev[1], h->ev[2]);
    cudaEventElapsedTime(&a23, h->ev[2], h->ev[3]);
    ms_draft += a01; ms_verify += a12; ms_accept += a23;
    h->trace_ms.push_back(a01 + a12 + a23);
    h->trace_emit.push_back(h->h_res[0] + 1);
    h->trace_K.push_back(K);
    for (int b = 0; b < B; ++b) {
      if (made[b] >= n_new) continue;
      const int a = h->h_res[b];
      const uint32_t fl = (uint32_t)h->h_res[MB + b];
      add_loop_stats(&st[b], K, a, fl);
      for (int i = 0; i <= a; ++i) {
        const int32_t tok = h->h_res[2 * MB + b * ld + i];
        if (made[b] < n_new) out_tokens[(size_t)b * n_new + made[b]++] = tok;
        else st[b].overshoot += 1;
      }
      h->seq_len[b] += a + 1;
    }
    if (K_min != K_max) {
      // grow after a loop that accepted every draft, shrink after one that rejected the first
      const int a = h->h_res[0];
      if (a == K) K = K + 1 < K_max ? K + 1 : K_max;
      else if (a == 0) K = K - 1 > K_min ? K - 1 : K_min;
    }
  }
  CU(h, cudaEventRecord(h->ev[6], h->stream));
  CU(h, cudaEventSynchronize(h->ev[6]));
  CU(h, cudaEventElapsedTime(&ms_decode, h->ev[5], h->ev[6]));
  if (out_stats)
    for (int b = 0; b < B; ++b) {
      st[b].ms_prefill = ms_prefill; st[b].ms_draft = ms_draft; st[b].ms_verify = ms_verify; st[b].ms_accept = ms_accept;
      st[b].ms_decode = ms_decode;
      st[b].kernel_launches = (int32_t)(h->launches - launches0);
      out_stats[b] = st[b];
    }
  return SPS_OK;
}

int sps_generate(sps_handle* h, const int32_t* prompt, int32_t prompt_len, int32_t n_new, int32_t K, float temperature,
                 uint64_t seed, int32_t* out_tokens, sps_stats* out_stats) {
  return generate_impl(h, prompt, 1, prompt_len, n_new, K, K, temperature, seed, out_tokens, out_stats);
}

int sps_generate_adaptive(sps_handle* h, const int32_t* prompt, int32_t prompt_len, int32_t n_new, int32_t K_min, int32_t K_max,
                          float temperature, uint64_t seed, int32_t* out_tokens, sps_stats* out_stats) {
  if (h && (K_min < 1 || K_min > K_max)) return fail(h, SPS_EINVAL, "K_min outside 1..K_max");
  return generate_impl(h, prompt, 1, prompt_len, n_new, K_min, K_max, temperature, seed, out_tokens, out_stats);
}

int sps_generate_batch(sps_handle* h, const int32_t* prompts, int32_t B, int32_t prompt_len, int32_t n_new, int32_t K,
                       float temperature, uint64_t seed, int32_t* out_tokens, sps_stats* out_stats) {
  if (h && (B < 1 || B > h->cfg.max_batch)) return fail(h, SPS_EINVAL, "batch outside 1..max_batch");
  return generate_impl(h, prompts, B, prompt_len, n_new, K, K, temperature, seed, out_tokens, out_stats);
}

int sps_score(sps_handle* h, int32_t which, const int32_t* rows, int32_t n_rows, float* out_logits, float* out_ms) {
  if (!h || !rows || !out_logits) return fail(h, SPS_EINVAL, "null argument");
  if (!h->ready) return fail(h, SPS_ESTATE, "sps_score before sps_prefill");
  if (h->B != 1) return fail(h, SPS_ESTATE, "sps_score works on a batch-1 handle");
  if (n_rows < 1 || n_rows > SPS_MAX_ROWS) return fail(h, SPS_EINVAL, "n_rows outside 1..16");
  ModelDev& m = which == 0 ? h->tgt : h->drf;
  if (!m.present) return fail(h, SPS_EINVAL, "model not loaded");
  CU(h, cudaSetDevice(h->cfg.device));
  const int len = h->seq_len[0] - 1;
  if (len + n_rows > h->cfg.max_seq) return fail(h, SPS_ERANGE, "rows would exceed max_seq");
  for (int i = 0; i < n_rows; ++i) {
    if (rows[i] < 0 || rows[i] >= m.cfg.vocab) return fail(h, SPS_ERANGE, "token id outside the vocabulary");
    h->h_rows[i] = rows[i];
    h->h_rows[SPS_MAX_ROWS + i] = len + i;
  }
  CU(h, cudaMemcpyAsync(h->hst.row_tok, h->h_rows, 4 * n_rows, cudaMemcpyHostToDevice, h->stream));
  CU(h, cudaMemcpyAsync(h->hst.row_pos, h->h_rows + SPS_MAX_ROWS, 4 * n_rows, cudaMemcpyHostToDevice, h->stream));
  PassSpec ps{};
  ps.mode = PASS_EXPLICIT; ps.rows_per_seq = n_rows; ps.logits = out_logits; ps.logits_ld = m.cfg.vocab;
  ps.lrow0 = 0; ps.lrowstep = 1; ps.lrows = n_rows;
  CU(h, cudaEventRecord(h->ev[0], h->stream));
  int rc = run_pass(h, m, ps);
  if (rc) return rc;
  CU(h, cudaEventRecord(h->ev[1], h->stream));
  CU(h, cudaStreamSynchronize(h->stream));
  if (out_ms) CU(h, cudaEventElapsedTime(out_ms, h->ev[0], h->ev[1]));
  return check_device_status(h);
}

int sps_verify(sps_handle* h, const int32_t* rows, int32_t K, float* out_logits, float* out_ms) {
  if (K < 0 || K > SPS_MAX_K) return fail(h, SPS_EINVAL, "K outside 0..15");
  return sps_score(h, 0, rows, K + 1, out_logits, out_ms);
}

int sps_set_sampling(sps_handle* h, int32_t top_k, float top_p) {
  if (!h) return fail(nullptr, SPS_EINVAL, "null handle");
  if (top_k < 0) return fail(h, SPS_EINVAL, "top_k must be >= 0 (0 = off)");
  if (!(top_p > 0.f && top_p <= 1.f)) return fail(h, SPS_EINVAL, "top_p must be in (0, 1] (1 = off)");
  h->top_k = top_k;
  h->top_p = top_p;
  return SPS_OK;
}

int sps_set_forced_acceptance(sps_handle* h, float alpha) {
  if (!h) return fail(nullptr, SPS_EINVAL, "null handle");
  if (!(alpha >= 0.f && alpha <= 1.f)) return fail(h, SPS_EINVAL, "alpha must be in [0, 1] (0 = off)");
  h->forced_accept = alpha;
  return SPS_OK;
}

int sps_accept(const float* q_logits, const float* p_logits, const int32_t* draft_tokens, int32_t B, int32_t K, int32_t V,
               float temperature, uint64_t seed, uint32_t step, void* stream, int32_t* out_n_accepted,
               int32_t* out_tokens, uint32_t* out_flags) {
  if (!(temperature > 0.f)) return fail(nullptr, SPS_EINVAL, "temperature must be > 0");
  return sps_accept_filtered(q_logits, p_logits, draft_tokens, B, K, V, temperature, 0, 1.f, seed, step, stream, out_n_accepted,
                             out_tokens, out_flags);
}

int sps_accept_filtered(const float* q_logits, const float* p_logits, const int32_t* draft_tokens, int32_t B, int32_t K,
                        int32_t V, float temperature, int32_t top_k, float top_p, uint64_t seed, uint32_t step, void* stream,
                        int32_t* out_n_accepted, int32_t* out_tokens, uint32_t* out_flags) {
  if (!q_logits || !out_n_accepted || !out_tokens || !out_flags) return fail(nullptr, SPS_EINVAL, "null argument");
  if (K > 0 && (!p_logits || !draft_tokens)) return fail(nullptr, SPS_EINVAL, "K > 0 needs p_logits and draft_tokens");
  if (B < 1 || K < 0 || K > SPS_MAX_K || V < 1) return fail(nullptr, SPS_EINVAL, "B, K or V out of range");
  if (!(temperature >= 0.f)) return fail(nullptr, SPS_EINVAL, "temperature must be >= 0 (0 = greedy)");
  if (top_k < 0 || !(top_p > 0.f && top_p <= 1.f)) return fail(nullptr, SPS_EINVAL, "top_k must be >= 0 and top_p in (0, 1]");
  if (temperature == 0.f) { temperature = 1.f; top_k = 1; top_p = 1.f; }
  AcceptArgs a{};
  a.st = nullptr; a.q_logits = q_logits; a.p_logits = p_logits ? p_logits : q_logits;
  a.drafts = draft_tokens ? draft_tokens : out_tokens; a.drafts_ld = K;
  a.B = B; a.K = K; a.V = V; a.n_acc = out_n_accepted; a.out_tok = out_tokens; a.out_ld = K + 1; a.flags = out_flags;
  a.temperature = temperature; a.seed = seed; a.step = step; a.top_k = top_k; a.top_p = top_p; a.sample_t = -1;
  cudaError_t e = accept_launch_fast(a, (top_k >= 1 && top_k < V) || top_p < 1.f, (cudaStream_t)stream);
  if (e != cudaSuccess) return fail(nullptr, SPS_ECUDA, std::string("accept launch: ") + cudaGetErrorString(e));
  return SPS_OK;
}

int sps_sample(const float* logits, int32_t B, int32_t V, float temperature, uint64_t seed, uint32_t step, uint32_t t,
               void* stream, int32_t* out_tokens) {
  if (!(temperature > 0.f)) return fail(nullptr, SPS_EINVAL, "B, V or temperature out of range");
  return sps_sample_filtered(logits, B, V, temperature, 0, 1.f, seed, step, t, stream, out_tokens);
}

int sps_sample_filtered(const float* logits, int32_t B, int32_t V, float temperature, int32_t top_k, float top_p, uint64_t seed,
                        uint32_t step, uint32_t t, void* stream, int32_t* out_tokens) {
  if (!logits || !out_tokens) return fail(nullptr, SPS_EINVAL, "null argument");
  if (B < 1 || V < 1 || !(temperature >= 0.f)) return fail(nullptr, SPS_EINVAL, "B, V or temperature out of range");
  if (top_k < 0 || !(top_p > 0.f && top_p <= 1.f)) return fail(nullptr, SPS_EINVAL, "top_k must be >= 0 and top_p in (0, 1]");
  if (temperature == 0.f) { temperature = 1.f; top_k = 1; top_p = 1.f; }
  SampleArgs a{};
  a.st = nullptr; a.logits = logits; a.ld = V; a.V = V; a.B = B; a.t = t; a.out = out_tokens; a.out_ld = 1;
  a.temperature = temperature; a.seed = seed; a.step = step; a.top_k = top_k; a.top_p = top_p;
  cudaError_t e = sample_launch_fast(a, (top_k >= 1 && top_k < V) || top_p < 1.f, (cudaStream_t)stream);
  if (e != cudaSuccess) return fail(nullptr, SPS_ECUDA, std::string("sample launch: ") + cudaGetErrorString(e));
  return SPS_OK;
}

static int cur_num_sm() {
  int dev = 0, n = SPS_NUM_SM_FALLBACK;
  if (cudaGetDevice(&dev) == cudaSuccess) cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
  return n;
}

int64_t sps_linear_workspace_bytes(int32_t dtype, int32_t M, int32_t N, int32_t D) {
  if (M < 1 || M > SPS_MAX_ROWS || N < 1 || D < 1 || dtype < 0 || dtype > 2) return -1;
  const LinPlan p = lin_plan(dtype, M, N, D, cur_num_sm());
  return (int64_t)(sizeof(float) * ((lin_part_floats(N, p.S) + 63) / 64 * 64 + lin_carry_floats() + (size_t)LIN_MAX_R * SPS_MAX_ROWS) +
                   sizeof(int) * (2 * LIN_MAX_R + 2) + 256 + ((sizeof(int) * lin_tile_ctr_ints(N) + 255) / 256) * 256);
}

int64_t sps_linear_wide_workspace_bytes(int32_t N, int32_t D) {
  if (N < 1 || D < 64 || D % 64) return -1;
  // error word + the activations' two bf16 halves (128 rows each) + the k-splits' partial products
  return (int64_t)(256 + 2 * (size_t)WIDE_ROWS * D * 2 + sizeof(float) * wide_part_floats(N, D, cur_num_sm()));
}

int sps_linear_wide(const void* W, const float* X, int32_t M, int32_t N, int32_t D, float* Y, void* workspace, void* stream,
                    float* out_ms) {
  if (!W || !X || !Y || !workspace) return fail(nullptr, SPS_EINVAL, "null argument");
  if (M < 1 || M > WIDE_ROWS || N < 1 || D < 64 || D % 64) return fail(nullptr, SPS_EINVAL, "M must be 1..128, D a multiple of 64");
  if (((uintptr_t)W | (uintptr_t)workspace) & 15) return fail(nullptr, SPS_EINVAL, "W and workspace must be 16-byte aligned");
  char* ws = (char*)workspace;
  int* err = (int*)ws;
  void* hi = ws + 256;
  void* lo = ws + 256 + (size_t)WIDE_ROWS * D * 2;
  float* part = (float*)(ws + 256 + 2 * (size_t)WIDE_ROWS * D * 2);
  cudaStream_t st = (cudaStream_t)stream;
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  cudaError_t e = cudaMemsetAsync(err, 0, 4, st);
  if (out_ms) { cudaEventCreate(&e0); cudaEventCreate(&e1); cudaEventRecord(e0, st); }
  if (e == cudaSuccess) e = wide_pack_launch(X, D, nullptr, 0.f, M, D, hi, lo, D, st);
  if (e == cudaSuccess) e = wide_gemm_launch(W, hi, lo, M, N, D, part, WIDE_STORE, Y, N, nullptr, nullptr, 0, err, cur_num_sm(), st);
  if (out_ms) {
    cudaEventRecord(e1, st);
    cudaEventSynchronize(e1);
    cudaEventElapsedTime(out_ms, e0, e1);
    cudaEventDestroy(e0); cudaEventDestroy(e1);
  }
  if (e != cudaSuccess) return fail(nullptr, SPS_ECUDA, std::string("wide linear launch: ") + cudaGetErrorString(e));
  int errw = 0;
  if (cudaMemcpyAsync(&errw, err, 4, cudaMemcpyDeviceToHost, st) != cudaSuccess || cudaStreamSynchronize(st) != cudaSuccess)
    return fail(nullptr, SPS_ECUDA, std::string("wide linear: ") + cudaGetErrorString(cudaGetLastError()));
  if (errw == 3) return fail(nullptr, SPS_ETIMEOUT, "a bounded device-side wait ran out in the wide linear kernel");
  return SPS_OK;
}

int sps_linear(const void* W, int32_t dtype, const float* X, int32_t M, int32_t N, int32_t D, float* Y, void* workspace,
               void* stream, float* out_ms) {
  if (dtype != 0 && dtype != 1) return fail(nullptr, SPS_EINVAL, "dtype must be 0 or 1");
  return sps_linear_scaled(W, dtype, nullptr, X, M, N, D, Y, workspace, stream, out_ms);
}

int sps_linear_scaled(const void* W, int32_t dtype, const float* row_scale, const float* X, int32_t M, int32_t N, int32_t D,
                      float* Y, void* workspace, void* stream, float* out_ms) {
  if (!W || !X || !Y || !workspace) return fail(nullptr, SPS_EINVAL, "null argument");
  if (M < 1 || M > SPS_MAX_ROWS || N < 1 || D < 1) return fail(nullptr, SPS_EINVAL, "M, N or D out of range");
  if (dtype >= 1 && D % 128) return fail(nullptr, SPS_EINVAL, "bf16 / int8 need D to be a multiple of 128");
  if (dtype == 0 && (size_t)M * D * 4 > 200 * 1024) return fail(nullptr, SPS_EINVAL, "fp32: M * D too large");
  if (dtype < 0 || dtype > 2) return fail(nullptr, SPS_EINVAL, "dtype must be 0, 1 or 2");
  if ((dtype == 2) != (row_scale != nullptr)) return fail(nullptr, SPS_EINVAL, "row scales go with int8 weights (dtype 2) and only with them");
  const LinPlan p = lin_plan(dtype, M, N, D, cur_num_sm());
  if (p.variant < 0) return fail(nullptr, SPS_EINVAL, "int8: D splits into more ranges than the kernel has queues");
  LinArgs a{};
  a.wscale[0] = row_scale;
  a.W[0] = W; a.rows_per_mat = N; a.N = N; a.D = D; a.M = M; a.X = X; a.ldx = D; a.x_row0 = 0; a.x_rowstep = 1;
  a.pro = PRO_NONE; a.epi = EPI_STORE; a.Y = Y; a.ldy = N;
  char* ws = (char*)workspace;
  a.counters = (int*)ws;
  size_t off = ((sizeof(int) * (2 * LIN_MAX_R + 2) + 255) / 256) * 256;
  a.tile_ctr = (int*)(ws + off);
  off += ((sizeof(int) * lin_tile_ctr_ints(N) + 255) / 256) * 256;
  off += sizeof(float) * (size_t)LIN_MAX_R * SPS_MAX_ROWS;
  a.part = (float*)(ws + off);
  a.carry = a.part + (lin_part_floats(N, p.S) + 63) / 64 * 64;
  cudaStream_t st = (cudaStream_t)stream;
  cudaEvent_t e0 = nullptr, e1 = nullptr;
  cudaError_t e = cudaMemsetAsync(a.counters + 2 * LIN_MAX_R + 1, 0, sizeof(int), st);   // the sticky error word starts clear
  if (out_ms) { cudaEventCreate(&e0); cudaEventCreate(&e1); cudaEventRecord(e0, st); }
  if (e == cudaSuccess) e = lin_launch(dtype, a, p, st);
  if (out_ms) {
    cudaEventRecord(e1, st);
    cudaEventSynchronize(e1);
    cudaEventElapsedTime(out_ms, e0, e1);
    cudaEventDestroy(e0); cudaEventDestroy(e1);
    int errw = 0;
    if (e == cudaSuccess && cudaMemcpy(&errw, a.counters + 2 * LIN_MAX_R + 1, 4, cudaMemcpyDeviceToHost) == cudaSuccess && errw == 3)
      return fail(nullptr, SPS_ETIMEOUT, "a bounded device-side wait ran out in the linear kernel");
  }
  if (e != cudaSuccess) return fail(nullptr, SPS_ECUDA, std::string("linear launch: ") + cudaGetErrorString(e));
  return SPS_OK;
}

int sps_tp_buffers(sps_handle* h, void** inbox, void** flags, int64_t* inbox_bytes, int64_t* flags_bytes) {
  if (!h || !inbox || !flags) return fail(h, SPS_EINVAL, "null argument");
  if (!h->tp) return fail(h, SPS_ESTATE, "the handle was not created with SPS_CFG_TENSOR_PARALLEL");
  *inbox = h->tp_inbox; *flags = h->tp_flags;
  if (inbox_bytes) *inbox_bytes = (int64_t)(sizeof(float) * 2 * SPS_TP_MAX_WORLD * h->tp_slot_floats);
  if (flags_bytes) *flags_bytes = (int64_t)(sizeof(uint32_t) * SPS_TP_MAX_WORLD);
  return SPS_OK;
}

int sps_tp_attach(sps_handle* h, int32_t rank, int32_t world, void* const* peer_inbox, void* const* peer_flags) {
  if (!h || !peer_inbox || !peer_flags) return fail(h, SPS_EINVAL, "null argument");
  if (!h->tp) return fail(h, SPS_ESTATE, "the handle was not created with SPS_CFG_TENSOR_PARALLEL");
  if (world < 1 || world > SPS_TP_MAX_WORLD || rank < 0 || rank >= world) return fail(h, SPS_EINVAL, "rank / world out of range (world <= 8)");
  for (int w = 0; w < world; ++w) {
    if (!peer_inbox[w] || !peer_flags[w]) return fail(h, SPS_EINVAL, "null peer buffer");
    h->tp_peer_inbox[w] = (float*)peer_inbox[w];
    h->tp_peer_flags[w] = (uint32_t*)peer_flags[w];
  }
  if (peer_inbox[rank] != (void*)h->tp_inbox || peer_flags[rank] != (void*)h->tp_flags)
    return fail(h, SPS_EINVAL, "entry `rank` of the peer tables must be this handle's own buffers (sps_tp_buffers)");
  CU(h, cudaSetDevice(h->cfg.device));
  // exchanges are numbered from zero on every rank: attach all ranks before any of them runs a pass
  CU(h, cudaMemsetAsync(h->tp_flags, 0, sizeof(uint32_t) * SPS_TP_MAX_WORLD, h->stream));
  CU(h, cudaMemsetAsync(h->tp_epoch, 0, sizeof(uint32_t) * 4, h->stream));
  CU(h, cudaStreamSynchronize(h->stream));
  h->tp_rank = rank; h->tp_world = world; h->tp_attached = true;
  return SPS_OK;
}

// what the group calls check: `world` attached ranks of one group, in rank order, on one device and one stream
static int tp_group_check(sps_handle* const* ranks, int world) {
  if (!ranks || world < 1 || world > SPS_TP_MAX_WORLD) return fail(nullptr, SPS_EINVAL, "bad group");
  for (int r = 0; r < world; ++r) {
    sps_handle* h = ranks[r];
    if (!h || !h->tp || !h->tp_attached || h->tp_world != world || h->tp_rank != r) return fail(h, SPS_EINVAL, "group member is not rank r of `world` attached ranks");
    if (h->stream != ranks[0]->stream || h->cfg.device != ranks[0]->cfg.device)
      return fail(h, SPS_EINVAL, "the ranks of an emulated group share one device and one stream");
  }
  return SPS_OK;
}

int sps_tp_group_prefill(sps_handle* const* ranks, int32_t world, const int32_t* toks, int32_t n) {
  int rc = tp_group_check(ranks, world);
  if (rc) return rc;
  if (!toks) return fail(ranks[0], SPS_EINVAL, "null argument");
  CU(ranks[0], cudaSetDevice(ranks[0]->cfg.device));
  for (int r = 0; r < world; ++r)
    if ((rc = set_sequences(ranks[r], toks, 1, n))) return rc;
  for (int which = 0; which < 2; ++which) {
    if (!(which == 0 ? ranks[0]->tgt : ranks[0]->drf).present) continue;
    for (int c0 = 0; c0 < n - 1; c0 += SPS_MAX_ROWS) {
      PassSpec ps{};
      ps.mode = PASS_PREFILL; ps.c0 = c0; ps.rows_per_seq = (n - 1 - c0) < SPS_MAX_ROWS ? (n - 1 - c0) : SPS_MAX_ROWS;
      const int phases = pass_phases(which == 0 ? ranks[0]->tgt : ranks[0]->drf);
      // what `world` processes would each enqueue on their own GPU, here phase by phase on one stream: every rank's
      // push of an exchange is enqueued before any rank's reduction of it, so no kernel ever waits on a later one
      for (int ph = 0; ph < phases; ++ph)
        for (int r = 0; r < world; ++r)
          if ((rc = run_pass_range(ranks[r], which == 0 ? ranks[r]->tgt : ranks[r]->drf, ps, ph, ph + 1))) return rc;
    }
  }
  CU(ranks[0], cudaStreamSynchronize(ranks[0]->stream));
  for (int r = 0; r < world; ++r) ranks[r]->ready = true;
  return SPS_OK;
}

// one pass of every rank, phase by phase
static int tp_group_pass(sps_handle* const* ranks, int world, int which, PassSpec (*spec)(sps_handle*, int, int), int K, int t) {
  const int phases = pass_phases(which == 0 ? ranks[0]->tgt : ranks[0]->drf);
  for (int ph = 0; ph < phases; ++ph)
    for (int r = 0; r < world; ++r) {
      const int rc = run_pass_range(ranks[r], which == 0 ? ranks[r]->tgt : ranks[r]->drf, spec(ranks[r], K, t), ph, ph + 1);
      if (rc) return rc;
    }
  return SPS_OK;
}
static PassSpec verify_spec_t(sps_handle* h, int K, int) { return verify_spec(h, K); }

int sps_tp_group_generate(sps_handle* const* ranks, int32_t world, const int32_t* prompt, int32_t P, int32_t n_new, int32_t K,
                          float T, uint64_t seed, int32_t* out_tokens, sps_stats* out_stats) {
  int rc = tp_group_check(ranks, world);
  if (rc) return rc;
  sps_handle* h0 = ranks[0];
  if (!prompt || !out_tokens || n_new < 1 || P < 1 || !(T >= 0.f)) return fail(h0, SPS_EINVAL, "bad argument");
  if ((long long)P + n_new + K > h0->cfg.max_seq) return fail(h0, SPS_ERANGE, "prompt_len + n_new + K exceeds max_seq");
  CU(h0, cudaSetDevice(h0->cfg.device));
  for (int r = 0; r < world; ++r) {
    if ((rc = sps_reset(ranks[r]))) return rc;
    if ((rc = check_K(ranks[r], K))) return rc;
  }
  if ((rc = sps_tp_group_prefill(ranks, world, prompt, P))) return rc;
  for (int r = 0; r < world; ++r) {
    int32_t lim = P + n_new;
    CU(ranks[r], cudaMemcpy(ranks[r]->hst.limit, &lim, 4, cudaMemcpyHostToDevice));
    if ((rc = write_params(ranks[r], T, seed, 0u))) return rc;
  }
  sps_stats st;
  std::memset(&st, 0, sizeof(st));
  const int MB = h0->cfg.max_batch, ld = h0->hst.max_K + 1;
  int made = 0;
  CU(h0, cudaEventRecord(h0->ev[5], h0->stream));
  while (made < n_new) {
    // what each rank's process would enqueue for one loop, interleaved phase by phase
    for (int t = 0; t < K; ++t) {
      if ((rc = tp_group_pass(ranks, world, 1, draft_spec, K, t))) return rc;
      for (int r = 0; r < world; ++r) if ((rc = enqueue_sample(ranks[r], K, t))) return rc;
    }
    if ((rc = tp_group_pass(ranks, world, 0, verify_spec_t, K, 0))) return rc;
    for (int r = 0; r < world; ++r) {
      sps_handle* h = ranks[r];
      if ((rc = enqueue_accept(h, K))) return rc;
      CU(h, cudaMemcpyAsync(h->h_res, h->res, h->res_words * 4, cudaMemcpyDeviceToHost, h->stream));
    }
    CU(h0, cudaStreamSynchronize(h0->stream));
    for (int r = 0; r < world; ++r) {
      sps_handle* h = ranks[r];
      h->last_K = K;
      if (h->h_res[h->res_words - 1] == 3) return fail(h, SPS_ETIMEOUT, "a bounded device-side wait ran out");
      if (h->h_res[h->res_words - 1] != 0) return fail(h, SPS_ERANGE, "device flagged a token id or position out of range");
      // every rank holds the same residual stream bit for bit, hence the same logits, hence the same decisions
      if (std::memcmp(h->h_res, h0->h_res, 4 * (h->res_words - 1)) != 0) return fail(h, SPS_ESTATE, "the ranks of the group decided differently");
    }
    const int a = h0->h_res[0];
    add_loop_stats(&st, K, a, (uint32_t)h0->h_res[MB]);
    for (int i = 0; i <= a; ++i) {
      if (made < n_new) out_tokens[made++] = h0->h_res[2 * MB + i];
      else st.overshoot += 1;
    }
    for (int r = 0; r < world; ++r) ranks[r]->seq_len[0] += a + 1;
  }
  CU(h0, cudaEventRecord(h0->ev[6], h0->stream));
  CU(h0, cudaEventSynchronize(h0->ev[6]));
  CU(h0, cudaEventElapsedTime(&st.ms_decode, h0->ev[5], h0->ev[6]));
  if (out_stats) *out_stats = st;
  (void)ld;
  return SPS_OK;
}

int sps_tp_group_score(sps_handle* const* ranks, int32_t world, int32_t which, const int32_t* rows, int32_t n_rows,
                       float* const* out_logits, float* out_ms) {
  int rc = tp_group_check(ranks, world);
  if (rc) return rc;
  sps_handle* h0 = ranks[0];
  if (!rows || !out_logits) return fail(h0, SPS_EINVAL, "null argument");
  if (n_rows < 1 || n_rows > SPS_MAX_ROWS) return fail(h0, SPS_EINVAL, "n_rows outside 1..16");
  CU(h0, cudaSetDevice(h0->cfg.device));
  for (int r = 0; r < world; ++r) {
    sps_handle* h = ranks[r];
    ModelDev& m = which == 0 ? h->tgt : h->drf;
    if (!h->ready || h->B != 1 || !m.present || !out_logits[r]) return fail(h, SPS_ESTATE, "group score needs a batch-1 prefill on every rank and a logits buffer per rank");
    const int len = h->seq_len[0] - 1;
    if (len + n_rows > h->cfg.max_seq) return fail(h, SPS_ERANGE, "rows would exceed max_seq");
    for (int i = 0; i < n_rows; ++i) {
      if (rows[i] < 0 || rows[i] >= m.cfg.vocab) return fail(h, SPS_ERANGE, "token id outside the vocabulary");
      h->h_rows[i] = rows[i];
      h->h_rows[SPS_MAX_ROWS + i] = len + i;
    }
    CU(h, cudaMemcpyAsync(h->hst.row_tok, h->h_rows, 4 * n_rows, cudaMemcpyHostToDevice, h->stream));
    CU(h, cudaMemcpyAsync(h->hst.row_pos, h->h_rows + SPS_MAX_ROWS, 4 * n_rows, cudaMemcpyHostToDevice, h->stream));
  }
  CU(h0, cudaEventRecord(h0->ev[0], h0->stream));
  const int phases = pass_phases(which == 0 ? h0->tgt : h0->drf);
  for (int ph = 0; ph < phases; ++ph)
    for (int r = 0; r < world; ++r) {
      sps_handle* h = ranks[r];
      ModelDev& m = which == 0 ? h->tgt : h->drf;
      PassSpec ps{};
      ps.mode = PASS_EXPLICIT; ps.rows_per_seq = n_rows; ps.logits = out_logits[r]; ps.logits_ld = m.cfg.vocab;
      ps.lrow0 = 0; ps.lrowstep = 1; ps.lrows = n_rows;
      if ((rc = run_pass_range(h, m, ps, ph, ph + 1))) return rc;
    }
  CU(h0, cudaEventRecord(h0->ev[1], h0->stream));
  CU(h0, cudaStreamSynchronize(h0->stream));
  if (out_ms) CU(h0, cudaEventElapsedTime(out_ms, h0->ev[0], h0->ev[1]));
  for (int r = 0; r < world; ++r) {
    int32_t errw = 0;
    CU(ranks[r], cudaMemcpy(&errw, ranks[r]->hst.err, 4, cudaMemcpyDeviceToHost));
    if (errw == 3) return fail(ranks[r], SPS_ETIMEOUT, "a bounded device-side wait ran out");
    if (errw != 0) return fail(ranks[r], SPS_ERANGE, "device flagged a token id or position out of range");
  }
  return SPS_OK;
}

int sps_philox(const uint32_t* ctr, const uint32_t* key, int32_t n, void* stream, uint32_t* out) {
  if (!ctr || !key || !out || n < 1) return fail(nullptr, SPS_EINVAL, "bad argument");
  cudaError_t e = philox_launch(ctr, key, n, out, (cudaStream_t)stream);
  if (e != cudaSuccess) return fail(nullptr, SPS_ECUDA, std::string("philox launch: ") + cudaGetErrorString(e));
  return SPS_OK;
}

}  // extern "C"
