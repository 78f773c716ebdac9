// C ABI of the RSD step-loop library: context, workspace layout, and the orchestration of one
// prefill / one step (Algorithm 1 batched over rows) as kernel launches on the caller's stream.
#include "../../include/rsd.h"

#include <cmath>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "common.cuh"
#include "kernels.cuh"

using namespace rsd;

namespace {

std::string g_create_error;

struct ModelHost {
  rsd_model m{};
  std::vector<const void*> wqkv, wo, wgu, wdown, norm1, norm2;
  size_t elem = 4;
  int kv_dtype = 0;      // element type of this model's KV cache: 0 fp32, 2 fp16 (for bf16 weights)
  bool split = false;    // bf16 GEMM inputs are kept as hi + lo pairs
  // Dense passes (more than 128 tokens) of a split model run on fp16 copies of its layer matrices with ONE fp16
  // activation operand instead of the bf16 pair: half the tensor-core work at an 11-bit significand.
  bool f16_dense = false;
  char* w16 = nullptr;                  // the copies: per layer wqkv, wo, wgu, wdown back to back
  size_t w16_layer = 0;                 // elements of one layer's four matrices
  // fp16 copy of matrix `which` (0 wqkv, 1 wo, 2 wgu, 3 wdown) of layer l
  const void* w16_of(int l, int which) const {
    const size_t d = m.d_model, hq = (size_t)m.n_heads * m.head_dim, qkv = (size_t)(m.n_heads + 2 * m.n_kv_heads) * m.head_dim;
    const size_t off[4] = {0, qkv * d, qkv * d + d * hq, qkv * d + d * hq + 2 * (size_t)m.d_ffn * d};
    return w16 + ((size_t)l * w16_layer + off[which]) * 2;
  }
  size_t w16_elems(int which) const {
    const size_t d = m.d_model, hq = (size_t)m.n_heads * m.head_dim, qkv = (size_t)(m.n_heads + 2 * m.n_kv_heads) * m.head_dim;
    const size_t n[4] = {qkv * d, d * hq, 2 * (size_t)m.d_ffn * d, d * (size_t)m.d_ffn};
    return n[which];
  }
  float2* rope = nullptr;
  char* kv_pool = nullptr;
  size_t layer_stride = 0;  // bytes of one layer's slab
  int pool_pages = 0;
  double n_params = 0;
};

// Host-visible scalars mirrored from the device after each phase boundary.
struct Scalars {
  int32_t n_tok, n_rej, err, n_active, n_slots, next_page[3], iter, n_live;
  int32_t sd_rounds, sd_proposed, sd_matched, sd_round, sd_j, pad;   // speculative decoding of rejected steps
};

struct Layout {
  size_t bytes = 0;
  size_t take(size_t n) {
    size_t off = bytes;
    bytes += (n + 255) & ~(size_t)255;
    return off;
  }
};

}  // namespace

struct rsd_ctx {
  rsd_config cfg{};
  ModelHost mdl[3];
  bool loaded = false, prefilled = false, poisoned = false;
  RowState st{};
  LoopParams lp{};
  int B_max = 0, S = 0, C = 0, max_pages = 0, chunk = 0, v_limit = 0, T_max = 0;
  // activations (workspace)
  float *x = nullptr, *qkv = nullptr, *q = nullptr, *gu = nullptr, *logits = nullptr;
  void *h = nullptr, *attn = nullptr, *act = nullptr;
  void *h_lo = nullptr, *attn_lo = nullptr, *act_lo = nullptr;   // low halves (bf16 models)
  unsigned long long* sample_best = nullptr;   // packed sampling winners, one per slot
  float* dbg_logits[2] = {nullptr, nullptr};
  int32_t* d_scalars = nullptr;  // device block holding n_tok, n_rej, err, n_active, n_slots, next_page[3]
  // staging of step outputs (device) and their pinned host mirrors
  int32_t *o_tokens = nullptr, *o_len = nullptr;
  float* o_rewards = nullptr;
  uint8_t *o_accept = nullptr, *o_live = nullptr, *o_role = nullptr, *o_waiting = nullptr;
  int32_t* o_gen = nullptr;
  size_t o_block_bytes = 0;
  float* norm_ssq = nullptr;   // [B][chunks] sums of squares of the residual stream (decode path)
  // persistent decode kernel: parameter block per model (draft, target), built for the batch size mega_B
  void* mega_block[3] = {nullptr, nullptr, nullptr};
  int mega_B[3] = {0, 0, 0};
  int32_t* mega_sync = nullptr;
  unsigned long long* mega_prof[3] = {nullptr, nullptr, nullptr};   // RSD_DEBUG_MEGA_PROFILE
  char* pinned = nullptr;
  size_t pinned_bytes = 0;
  void* gemm_scratch = nullptr;
  size_t gemm_scratch_bytes = 0;
  void* attn_scratch = nullptr;
  size_t attn_scratch_bytes = 0;
  rsd_counters ctr{};
  int last_n_rej = 0;
  // one CUDA graph per decode phase (draft, target): a whole decode iteration, replayed per token
  cudaStream_t cap_stream = nullptr;
  // slot = phase * 4 + bucket of the number of rows that take part (all, a half, a quarter, an eighth or fewer);
  // 8 + bucket: a proposal iteration of the draft, 12 + bucket: the target's pass over a round's proposals
  // (speculative decoding of rejected steps)
  cudaGraphExec_t dec_graph[16] = {};
  int dec_graph_B[16] = {};
  uint64_t dec_graph_kernels[16] = {};
  int sd_k = 0, slots_max = 0;

  int attn_rows_hint = 0;      // rows expected to be active in the running decode phase (0: all slots)
  bool time_this_iter = false, in_decode = false;
  // per-phase timing of rsd_step (rsd_debug_phase_ms)
  bool time_phases = false;
  cudaEvent_t ph_ev[8] = {};
  double ph_ms[7] = {};
  // sampled GEMM timing (rsd_debug_gemm_timing)
  int time_stride = 0;
  uint64_t gemm_calls = 0;
  std::vector<cudaEvent_t> ev;          // pairs: start, stop
  std::vector<double> ev_bytes;
  std::vector<double> ev_flops;         // != 0: a dense launch (more than 128 rows), its algorithmic flops 2 M N K;
                                        // negative when the operand is a hi + lo pair (twice the tensor-core work)
  size_t ev_used = 0;
  double timed_ms = 0, timed_bytes = 0;
  uint64_t timed_launches = 0;
  double dense_ms[2] = {0, 0}, dense_flops[2] = {0, 0};  // the dense launches among them: [0] plain operand, [1] hi + lo
  uint64_t dense_launches[2] = {0, 0};
  std::string err;
};

namespace {

int fail(rsd_ctx* c, int code, const char* fmt, const char* detail = "") {
  char buf[512];
  snprintf(buf, sizeof(buf), fmt, detail);
  if (c) c->err = buf; else g_create_error = buf;
  return code;
}

#define CU(call)                                                                        \
  do {                                                                                  \
    cudaError_t e_ = (call);                                                            \
    if (e_ != cudaSuccess) {                                                            \
      c->poisoned = true;                                                               \
      return fail(c, RSD_ERR_CUDA, "CUDA error: %s", cudaGetErrorString(e_));           \
    }                                                                                   \
  } while (0)

int check_model(const rsd_model* m, const char** why) {
  *why = "";
  if (!m) { *why = "null model"; return RSD_ERR_ARG; }
  if (m->n_layers < 1 || m->d_model < 8 || m->n_heads < 1 || m->n_kv_heads < 1 || m->d_ffn < 8 || m->vocab < 1) {
    *why = "non-positive dimension"; return RSD_ERR_ARG;
  }
  if (m->n_heads % m->n_kv_heads != 0) { *why = "n_heads not a multiple of n_kv_heads"; return RSD_ERR_ARG; }
  if (m->dtype != RSD_F32 && m->dtype != RSD_BF16) { *why = "dtype"; return RSD_ERR_ARG; }
  if (m->head_dim != 64 && m->head_dim != 128) { *why = "head_dim must be 64 or 128"; return RSD_ERR_UNSUPPORTED; }
  const int vec = m->dtype == RSD_BF16 ? 8 : 4;
  if (m->d_model % vec || m->d_ffn % vec || (m->n_heads * m->head_dim) % vec) {
    *why = "inner dimensions must be multiples of a 16-byte vector"; return RSD_ERR_UNSUPPORTED;
  }
  if (m->head_kind < 0 || m->head_kind > 2) { *why = "head_kind"; return RSD_ERR_ARG; }
  return RSD_OK;
}

double count_params(const rsd_model& m) {
  const double d = m.d_model, hd = m.head_dim;
  const double per_layer = d * m.n_heads * hd + 2 * d * m.n_kv_heads * hd + m.n_heads * hd * d + 3 * d * m.d_ffn + 2 * d;
  const double head = m.head_kind == RSD_HEAD_LM ? (double)m.vocab * d : d;
  return (double)m.vocab * d + m.n_layers * per_layer + d + head;
}

// Whether model m caches keys and values as fp16 hi + lo pairs.  Setting 0 decides by depth: the rounding of
// 16-bit keys and values grows with the number of layers, and beyond 48 layers the logits of a bf16 model
// leave the 3e-2 band around an exact reference (80 layers: 5e-2 to 7e-2), so deep models get the pairs.
bool kv_extended_for(const rsd_model& m, int setting) {
  if (m.dtype != RSD_BF16) return false;
  return setting == 1 || (setting == 0 && m.n_layers > 48);
}

size_t kv_pool_bytes(const rsd_model& m, int pages, int kv_extended) {
  const size_t elem = m.dtype == RSD_BF16 ? 2 : 4;
  const size_t blocks = kv_extended_for(m, kv_extended) ? 4 : 2;   // keys, values (, their low halves)
  return (size_t)pages * m.n_layers * blocks * m.n_kv_heads * kPageTokens * m.head_dim * elem;
}

struct Dims {
  int d = 0, qkv = 0, hq = 0, f = 0, v = 0, hd = 0;
};

Dims max_dims(const rsd_model* const ms[3]) {
  Dims r;
  for (int i = 0; i < 3; ++i) {
    const rsd_model& m = *ms[i];
    r.d = std::max(r.d, m.d_model);
    r.qkv = std::max(r.qkv, (m.n_heads + 2 * m.n_kv_heads) * m.head_dim);
    r.hq = std::max(r.hq, m.n_heads * m.head_dim);
    r.f = std::max(r.f, m.d_ffn);
    if (m.head_kind == RSD_HEAD_LM) r.v = std::max(r.v, m.vocab);
    r.hd = std::max(r.hd, m.head_dim);
  }
  return r;
}

// Elements of one layer's four weight matrices.
size_t layer_weight_elems(const rsd_model& m) {
  const size_t d = m.d_model, hq = (size_t)m.n_heads * m.head_dim, qkv = (size_t)(m.n_heads + 2 * m.n_kv_heads) * m.head_dim;
  return qkv * d + d * hq + 2 * (size_t)m.d_ffn * d + d * (size_t)m.d_ffn;
}

// Which models get fp16 copies of their layer matrices for the dense passes: bf16 models that keep hi + lo operands
// (so not the narrow PRMs, which already run plain bf16), whose chunk attention is the kernel that can write a single
// fp16 operand (fp16 cache without the low halves, head_dim 128, groups of up to 8 heads), and whose copies stay
// within 20 GB (a 72B-shape model's would not fit beside the model itself).
bool wants_f16_dense(const rsd_config& cfg, const rsd_model& m, int which) {
  if (cfg.debug_flags & RSD_DEBUG_NO_F16_DENSE) return false;
  if (m.dtype != RSD_BF16) return false;
  if (which == RSD_PRM && (cfg.prm_shares_draft || m.d_model <= 2048)) return false;
  if (kv_extended_for(m, cfg.kv_extended)) return false;
  if (m.head_dim != 128 || m.n_heads % m.n_kv_heads != 0 || m.n_heads / m.n_kv_heads > 8) return false;
  return layer_weight_elems(m) * 2 * (size_t)m.n_layers <= ((size_t)20 << 30);
}

// Lays out the workspace; with c == nullptr only the size is computed.
size_t layout_workspace(const rsd_config& cfg, const rsd_model* const ms[3], rsd_ctx* c) {
  Layout L;
  const int B = cfg.max_batch, S = cfg.max_seq_tokens, C = cfg.max_step_tokens;
  const int max_pages = (S + kPageTokens - 1) / kPageTokens;
  const int chunk = cfg.max_chunk_tokens > 0 ? cfg.max_chunk_tokens : 4096;
  const int sd_k = cfg.sd_tokens > 0 ? cfg.sd_tokens : 0;
  const int slots = B * std::max(1, sd_k);      // token slots of one pass of a decode phase (a round's proposals)
  const int T = std::max(slots, chunk);
  const Dims dm = max_dims(ms);
  char* base = c ? (char*)cfg.workspace : nullptr;
  auto P = [&](size_t off) -> char* { return base ? base + off : nullptr; };
#define TAKE(type, n) (type*)P(L.take(sizeof(type) * (size_t)(n)))
  // row state
  RowState st{};
  st.B = 0; st.S = S; st.C = C; st.max_pages = max_pages; st.prm_shared = cfg.prm_shares_draft ? 1 : 0;
  st.z_len = TAKE(int32_t, B); st.live = TAKE(int32_t, B); st.n_steps = TAKE(int32_t, B);
  st.tok = TAKE(int32_t, (size_t)B * S);
  for (int w = 0; w < 3; ++w) {
    st.kv_len[w] = TAKE(int32_t, B);
    st.n_pages[w] = TAKE(int32_t, B);
    st.page_table[w] = TAKE(int32_t, (size_t)B * max_pages);
  }
  for (int p = 0; p < 2; ++p) {
    st.gen_len[p] = TAKE(int32_t, B);
    st.gen_tok[p] = TAKE(int32_t, (size_t)B * C);
    st.sampled[p] = TAKE(int32_t, (size_t)B * C);
    st.forced_tok[p] = TAKE(int32_t, (size_t)B * C);
    st.forced_len[p] = TAKE(int32_t, B);
  }
  st.forced_accept = TAKE(uint8_t, B);
  st.gen_active = TAKE(int32_t, B);
  st.rewards = TAKE(float, B);
  st.accept = TAKE(uint8_t, B);
  st.waiting = TAKE(uint8_t, B);
  st.rej_idx = TAKE(int32_t, B);
  st.slot_row = TAKE(int32_t, B);
  st.last_idx = TAKE(int32_t, B);
  st.prev_idx = TAKE(int32_t, B);
  st.target_rewards = TAKE(float, B);
  int32_t* scal = TAKE(int32_t, 16);
  st.n_tok = scal + 0; st.n_rej = scal + 1; st.err = scal + 2; st.n_active = scal + 3; st.n_slots = scal + 4; st.iter = scal + 8;
  st.next_page = scal + 5; st.n_live = scal + 9;
  st.sd_k = sd_k; st.sd_stats = scal + 10;
  st.sd_out_idx = TAKE(int32_t, slots);
  st.sd_forced_on = TAKE(uint8_t, B);
  st.sd_forced_props = (sd_k > 0 && (cfg.debug_flags & RSD_DEBUG_KEEP_LOGITS)) ? TAKE(int32_t, (size_t)B * C * sd_k) : nullptr;
  st.pass_capacity = B * S;
  st.pass_tok_id = TAKE(int32_t, (size_t)B * S);
  st.pass_tok_row = TAKE(int32_t, (size_t)B * S);
  st.pass_tok_pos = TAKE(int32_t, (size_t)B * S);
  // activations
  float* x = TAKE(float, (size_t)T * dm.d);
  void* h = TAKE(float, (size_t)T * dm.d);
  float* qkv = TAKE(float, (size_t)T * dm.qkv);
  float* q = TAKE(float, (size_t)T * dm.hq);
  void* attn = TAKE(float, (size_t)T * dm.hq);
  float* gu = TAKE(float, (size_t)T * 2 * dm.f);
  void* act = TAKE(float, (size_t)T * dm.f);
  float* logits = TAKE(float, (size_t)slots * dm.v);
  unsigned long long* sample_best = TAKE(unsigned long long, slots);
  float* norm_ssq = TAKE(float, (size_t)slots * 2 * norm_chunks(dm.d));   // room for 128-column chunks
  void* mega_block[3] = {nullptr, nullptr, nullptr};
  for (int w = 0; w < 3; w += 2) mega_block[w] = TAKE(char, mega_block_bytes(ms[w]->n_layers));
  int32_t* mega_sync = TAKE(int32_t, 1024);
  unsigned long long* mega_prof[3] = {nullptr, nullptr, nullptr};
  if (cfg.debug_flags & RSD_DEBUG_MEGA_PROFILE)
    for (int w = 0; w < 3; w += 2) mega_prof[w] = TAKE(unsigned long long, 1024);
  float2* rope[3];
  for (int w = 0; w < 3; ++w) rope[w] = TAKE(float2, (size_t)S * (ms[w]->head_dim / 2));
  char* w16[3] = {nullptr, nullptr, nullptr};
  for (int w = 0; w < 3; ++w)
    if (wants_f16_dense(cfg, *ms[w], w)) w16[w] = TAKE(char, layer_weight_elems(*ms[w]) * 2 * (size_t)ms[w]->n_layers);
  float* dbg[2] = {nullptr, nullptr};
  if (cfg.debug_flags & RSD_DEBUG_KEEP_LOGITS) {
    dbg[0] = TAKE(float, (size_t)B * C * ms[RSD_DRAFT]->vocab);
    dbg[1] = TAKE(float, (size_t)B * C * ms[RSD_TARGET]->vocab);
  }
  int32_t* o_tokens = TAKE(int32_t, (size_t)B * C);
  int32_t* o_len = TAKE(int32_t, B);
  float* o_rewards = TAKE(float, B);
  uint8_t* o_accept = TAKE(uint8_t, B);
  uint8_t* o_live = TAKE(uint8_t, B);
  uint8_t* o_role = TAKE(uint8_t, B);
  uint8_t* o_waiting = TAKE(uint8_t, B);
  int32_t* o_gen = TAKE(int32_t, 2 * (size_t)B);   // tokens each row generated in the draft / target phase of the call
  const size_t o_end = L.bytes;                    // the step's outputs form one block [o_tokens, o_end): one copy
  const size_t gs = gemm_scratch_bytes_any();
  void* gscr = TAKE(char, gs);
  int h_max = 0;
  for (int w = 0; w < 3; ++w) h_max = std::max(h_max, ms[w]->n_heads);
  const size_t as = attn_decode_scratch_bytes(slots, h_max, dm.hd, S);
  void* ascr = TAKE(char, as);
#undef TAKE
  if (c) {
    c->st = st; c->B_max = B; c->S = S; c->C = C; c->max_pages = max_pages; c->chunk = chunk; c->T_max = T;
    c->sd_k = sd_k; c->slots_max = slots;
    c->x = x; c->h = h; c->qkv = qkv; c->q = q; c->attn = attn; c->gu = gu; c->act = act; c->logits = logits;
    // each operand buffer was sized at 4 bytes per element: a bf16 hi array followed by its lo array
    c->h_lo = (char*)h + (size_t)T * dm.d * 2;
    c->attn_lo = (char*)attn + (size_t)T * dm.hq * 2;
    c->act_lo = (char*)act + (size_t)T * dm.f * 2;
    c->sample_best = sample_best;
    c->norm_ssq = norm_ssq;
    for (int w = 0; w < 3; ++w) { c->mega_block[w] = mega_block[w]; c->mega_B[w] = 0; }
    c->mega_sync = mega_sync;
    for (int w = 0; w < 3; ++w) c->mega_prof[w] = mega_prof[w];
    for (int w = 0; w < 3; ++w) c->mdl[w].rope = rope[w];
    for (int w = 0; w < 3; ++w) c->mdl[w].w16 = w16[w];
    c->dbg_logits[0] = dbg[0]; c->dbg_logits[1] = dbg[1];
    c->d_scalars = scal;
    c->o_tokens = o_tokens; c->o_len = o_len; c->o_rewards = o_rewards; c->o_accept = o_accept; c->o_live = o_live;
    c->o_role = o_role; c->o_waiting = o_waiting; c->o_gen = o_gen;
    c->o_block_bytes = o_end - (size_t)((char*)o_tokens - base);
    c->gemm_scratch = gscr; c->gemm_scratch_bytes = gs;
    c->attn_scratch = ascr; c->attn_scratch_bytes = as;
  }
  return L.bytes;
}

int check_config(const rsd_config* cfg, const char** why) {
  *why = "";
  if (!cfg) { *why = "null config"; return RSD_ERR_ARG; }
  if (cfg->max_batch < 1 || cfg->max_batch > kMaxBatch) { *why = "max_batch out of 1..1024"; return RSD_ERR_ARG; }
  if (cfg->page_tokens != kPageTokens) { *why = "page_tokens must be 16"; return RSD_ERR_UNSUPPORTED; }
  if (cfg->max_step_tokens < 1 || cfg->max_steps < 1 || cfg->max_seq_tokens < 2) { *why = "step/sequence limits"; return RSD_ERR_ARG; }
  if (cfg->temperature < 0.f) { *why = "temperature"; return RSD_ERR_ARG; }
  if (cfg->omega_kind < 0 || cfg->omega_kind > 4) { *why = "omega_kind"; return RSD_ERR_ARG; }
  if (cfg->step_end_mod < 0) { *why = "step_end_mod"; return RSD_ERR_ARG; }
  if (cfg->kv_extended < 0 || cfg->kv_extended > 2) { *why = "kv_extended out of 0..2"; return RSD_ERR_ARG; }
  if (cfg->sd_tokens < 0 || cfg->sd_tokens > 16) { *why = "sd_tokens out of 0..16"; return RSD_ERR_ARG; }
  return RSD_OK;
}

int drain_gemm_events(rsd_ctx* c);

// ---- device scalars <-> host ---------------------------------------------------------------
int read_scalars(rsd_ctx* c, cudaStream_t s, Scalars* out) {
  CU(cudaMemcpyAsync(c->pinned, c->d_scalars, sizeof(Scalars), cudaMemcpyDeviceToHost, s));
  // the tensor-core GEMM raises its own flag (bounded waits) at byte 4096 of its scratch
  CU(cudaMemcpyAsync(c->pinned + 128, (char*)c->gemm_scratch + 4096, sizeof(int32_t), cudaMemcpyDeviceToHost, s));
  CU(cudaStreamSynchronize(s));
  if (*(int32_t*)(c->pinned + 128) != 0) {
    c->poisoned = true;
    return fail(c, RSD_ERR_TIMEOUT, "a bounded wait inside the tensor-core GEMM expired%s");
  }
  if (c->ev_used) { int rc_ = drain_gemm_events(c); if (rc_) return rc_; }
  memcpy(out, c->pinned, sizeof(Scalars));
  if (out->err == RSD_ERR_OOM_PAGES) return fail(c, RSD_ERR_OOM_PAGES, "KV page pool or pass list exhausted%s");
  if (out->err != 0) { c->poisoned = true; return fail(c, RSD_ERR_TIMEOUT, "device-side error flag raised%s"); }
  return RSD_OK;
}

// ---- one model pass over T token slots ------------------------------------------------------
// Folds the finished event pairs into the running totals.  The stream must be idle.
int drain_gemm_events(rsd_ctx* c) {
  for (size_t i = 0; i < c->ev_used; ++i) {
    float ms = 0.f;
    CU(cudaEventElapsedTime(&ms, c->ev[2 * i], c->ev[2 * i + 1]));
    c->timed_ms += ms;
    c->timed_bytes += c->ev_bytes[i];
    ++c->timed_launches;
    if (c->ev_flops[i] != 0) {
      const int k = c->ev_flops[i] < 0 ? 1 : 0;
      c->dense_ms[k] += ms; c->dense_flops[k] += std::abs(c->ev_flops[i]); ++c->dense_launches[k];
    }
  }
  c->ev_used = 0;
  return RSD_OK;
}

// `pending` (nullable): the caller's next kernel adds up K-split partial sums itself, so the GEMM may
// leave them in the scratch; *pending then describes them (splits == 1: y is complete).
int gemm(rsd_ctx* c, const ModelHost& M, const void* W, const void* xin, const void* xin_lo, float* y, int Mrows, int N,
         int K, int accumulate, const int32_t* n_active, SplitSum* pending, cudaStream_t s, RowScale rs = RowScale()) {
  // ragged passes: every stride-th GEMM; decode: every GEMM of the iterations chosen by decode_phase
  const bool pick = c->in_decode ? c->time_this_iter
                                 : (c->time_stride > 0 && (c->gemm_calls++ % (uint64_t)c->time_stride) == 0);
  const bool timed = pick && c->ev_used < c->ev_bytes.size();
  if (timed) CU(cudaEventRecord(c->ev[2 * c->ev_used], s));
  int splits = 1;
  CU(launch_gemm(M.m.dtype, W, xin, M.split ? xin_lo : nullptr, y, Mrows, N, K, accumulate, 0, c->gemm_scratch,
                 c->gemm_scratch_bytes, n_active, pending ? &splits : nullptr, s, rs));
  if (pending) { pending->splits = splits; pending->partials = gemm_partials(c->gemm_scratch); }
  if (timed) {
    CU(cudaEventRecord(c->ev[2 * c->ev_used + 1], s));
    // algorithmic bytes: the weight matrix and the input once, the output once (twice when added to)
    c->ev_bytes[c->ev_used] = (double)N * K * M.elem + (double)Mrows * K * M.elem +
                              (double)Mrows * N * 4.0 * (accumulate ? 2.0 : 1.0);
    c->ev_flops[c->ev_used] = Mrows > 128 ? (M.split ? -1.0 : 1.0) * 2.0 * Mrows * (double)N * K : 0.0;
    ++c->ev_used;
  }
  return RSD_OK;
}

// Gate/up projection + SwiGLU in one kernel (bf16 models); timed like gemm().
int gemm_gu(rsd_ctx* c, const ModelHost& M, const void* Wgu, const void* xin, const void* xin_lo, void* act, void* act_lo,
            int Mrows, int F, int K, const int32_t* n_active, cudaStream_t s, RowScale rs = RowScale()) {
  const bool pick = c->in_decode ? c->time_this_iter
                                 : (c->time_stride > 0 && (c->gemm_calls++ % (uint64_t)c->time_stride) == 0);
  const bool timed = pick && c->ev_used < c->ev_bytes.size();
  if (timed) CU(cudaEventRecord(c->ev[2 * c->ev_used], s));
  CU(launch_gemm_gu(Wgu, xin, xin_lo, act, act_lo, Mrows, F, K, c->gemm_scratch, c->gemm_scratch_bytes, n_active, s, rs));
  if (timed) {
    CU(cudaEventRecord(c->ev[2 * c->ev_used + 1], s));
    // algorithmic bytes: the stacked weight matrix and the input pair once, the output pair once
    c->ev_bytes[c->ev_used] = 2.0 * F * K * M.elem + 2.0 * Mrows * K * M.elem + 2.0 * Mrows * F * M.elem;
    c->ev_flops[c->ev_used] = Mrows > 128 ? (M.split ? -1.0 : 1.0) * 2.0 * Mrows * 2.0 * F * K : 0.0;
    ++c->ev_used;
  }
  return RSD_OK;
}

// Up to 128 rows the one-tile-per-CTA fused kernel wins (one kernel and the fp32 gate/up array less); with more rows
// a CTA of that kernel cannot hide the heavier epilogue (measured at 4096 rows: 586 us against 367 + 64 us): there
// the caller takes the persistent kernel when it can (no idle flag), else the plain GEMM + SwiGLU kernel.
bool gu_fused_ok(const ModelHost& M, int rows) {
  return rows <= 128 && M.m.dtype == RSD_BF16 && M.split && gemm_gu_supported(1, rows, M.m.d_ffn, M.m.d_model);
}

// One dense GEMM of the fp16 pass, timed like gemm() (class "plain": its tensor-core work is the algorithm's).
int gemm_f16(rsd_ctx* c, const void* W16, const void* x16, float* y, int Mrows, int N, int K, int accumulate, cudaStream_t s) {
  const bool pick = c->time_stride > 0 && (c->gemm_calls++ % (uint64_t)c->time_stride) == 0;
  const bool timed = pick && c->ev_used < c->ev_bytes.size();
  if (timed) CU(cudaEventRecord(c->ev[2 * c->ev_used], s));
  CU(launch_gemm_f16_dense(W16, x16, y, Mrows, N, K, accumulate, c->gemm_scratch, c->gemm_scratch_bytes, s));
  if (timed) {
    CU(cudaEventRecord(c->ev[2 * c->ev_used + 1], s));
    c->ev_bytes[c->ev_used] = (double)N * K * 2 + (double)Mrows * K * 2 + (double)Mrows * N * 4.0 * (accumulate ? 2.0 : 1.0);
    c->ev_flops[c->ev_used] = 2.0 * Mrows * (double)N * K;
    ++c->ev_used;
  }
  return RSD_OK;
}

// The layer stack of a pass of more than 128 tokens on the fp16 copies of the weights: every GEMM operand (normed
// residual, attention output, SwiGLU output) is written once, as fp16, by the kernel that produces it.  x holds the
// embedded tokens on entry and the last layer's residual stream on exit, as in forward_pass.
int forward_pass_f16(rsd_ctx* c, int which, PassView p, cudaStream_t s) {
  const ModelHost& M = c->mdl[which];
  const rsd_model& m = M.m;
  const int d = m.d_model, H = m.n_heads, KV = m.n_kv_heads, hd = m.head_dim, F = m.d_ffn;
  const int T = p.T;
  for (int l = 0; l < m.n_layers; ++l) {
    KvView kv{M.kv_pool + (size_t)l * M.layer_stride, c->st.page_table[which], c->max_pages, 0};
    CU(launch_rmsnorm(m.dtype, c->x, M.norm1[l], c->h, nullptr, T, d, m.rms_eps, nullptr, nullptr, SplitSum(), s, true));
    int rc = gemm_f16(c, M.w16_of(l, 0), c->h, c->qkv, T, (H + 2 * KV) * hd, d, 0, s);
    if (rc) return rc;
    CU(launch_rope_kv(M.kv_dtype, c->qkv, SplitSum(), p, c->q, kv, M.rope, H, KV, hd, s));
    CU(launch_attn_chunk(M.kv_dtype, c->q, p, kv, c->attn, nullptr, 2, H, KV, hd, s, (int*)((char*)c->gemm_scratch + 4096)));
    rc = gemm_f16(c, M.w16_of(l, 1), c->attn, c->x, T, d, H * hd, 1, s);
    if (rc) return rc;
    CU(launch_rmsnorm(m.dtype, c->x, M.norm2[l], c->h, nullptr, T, d, m.rms_eps, nullptr, nullptr, SplitSum(), s, true));
    {
      const bool pick = c->time_stride > 0 && (c->gemm_calls++ % (uint64_t)c->time_stride) == 0;
      const bool timed = pick && c->ev_used < c->ev_bytes.size();
      if (timed) CU(cudaEventRecord(c->ev[2 * c->ev_used], s));
      CU(launch_gemm_gu_f16_dense(M.w16_of(l, 2), c->h, c->act, T, F, d, c->gemm_scratch, c->gemm_scratch_bytes, s));
      if (timed) {
        CU(cudaEventRecord(c->ev[2 * c->ev_used + 1], s));
        c->ev_bytes[c->ev_used] = 2.0 * F * d * 2 + (double)T * d * 2 + (double)T * F * 2;
        c->ev_flops[c->ev_used] = 2.0 * T * 2.0 * F * d;
        ++c->ev_used;
      }
    }
    rc = gemm_f16(c, M.w16_of(l, 3), c->act, c->x, T, d, F, 1, s);
    if (rc) return rc;
  }
  return RSD_OK;
}

int forward_pass(rsd_ctx* c, int which, PassView p, cudaStream_t s) {
  const ModelHost& M = c->mdl[which];
  const rsd_model& m = M.m;
  const int d = m.d_model, H = m.n_heads, KV = m.n_kv_heads, hd = m.head_dim, F = m.d_ffn;
  const int T = p.T;
  if (T <= 0) return RSD_OK;
  CU(launch_embed(m.dtype, m.tok_embed, p, c->x, d, s));
  // dense pass of a model with fp16 weight copies: one fp16 activation operand, no low halves
  const bool f16 = M.f16_dense && p.n_active == nullptr && T > 128 && gemm_gu_supported(1, T, F, d);
  if (f16) return forward_pass_f16(c, which, p, s);
  void* h_lo = M.split ? c->h_lo : nullptr;
  void* attn_lo = M.split ? c->attn_lo : nullptr;
  void* act_lo = M.split ? c->act_lo : nullptr;
  // K-split partial sums can be left for the consumer kernel to add up.  That pays where the
  // consumer runs many blocks (SwiGLU); RMSNorm and RoPE run one block per token, too few to pull
  // the partials in quickly, so those GEMMs reduce with their own kernel.
  const bool defer_small = false;
  SplitSum x_pending;   // partial sums of the last GEMM that adds into the residual stream
  for (int l = 0; l < m.n_layers; ++l) {
    KvView kv{M.kv_pool + (size_t)l * M.layer_stride, c->st.page_table[which], c->max_pages, M.kv_dtype == 3 ? 1 : 0};
    CU(launch_rmsnorm(m.dtype, c->x, M.norm1[l], c->h, h_lo, T, d, m.rms_eps, nullptr, p.n_active, x_pending, s));
    SplitSum qkv_pending;
    int rc = gemm(c, M, M.wqkv[l], c->h, h_lo, c->qkv, T, (H + 2 * KV) * hd, d, 0, p.n_active, defer_small ? &qkv_pending : nullptr, s);
    if (rc) return rc;
    CU(launch_rope_kv(M.kv_dtype, c->qkv, qkv_pending, p, c->q, kv, M.rope, H, KV, hd, s));
    if (p.n_active != nullptr) {
      // decode pass: one query per row slot
      CU(launch_attn_decode(M.kv_dtype, c->q, kv.pool_layer, kv.page_table, kv.max_pages, p.tok_row, p.tok_pos, 1,
                            c->attn, attn_lo, m.dtype, T, H, KV, hd, c->S, c->attn_scratch, c->attn_scratch_bytes,
                            p.n_active, s, c->attn_rows_hint));
    } else {
      CU(launch_attn_chunk(M.kv_dtype, c->q, p, kv, c->attn, attn_lo, m.dtype, H, KV, hd, s,
                           (int*)((char*)c->gemm_scratch + 4096)));
    }
    rc = gemm(c, M, M.wo[l], c->attn, attn_lo, c->x, T, d, H * hd, 1, p.n_active, defer_small ? &x_pending : nullptr, s);
    if (rc) return rc;
    CU(launch_rmsnorm(m.dtype, c->x, M.norm2[l], c->h, h_lo, T, d, m.rms_eps, nullptr, p.n_active, x_pending, s));
    // up to 128 rows: fused kernel; dense passes (no idle flag): the persistent kernel hides the SwiGLU epilogue
    // under the next tile's MMAs
    if (gu_fused_ok(M, T) || (T > 128 && p.n_active == nullptr && m.dtype == RSD_BF16 && gemm_gu_supported(1, T, F, d))) {
      rc = gemm_gu(c, M, M.wgu[l], c->h, h_lo, c->act, act_lo, T, F, d, p.n_active, s);
      if (rc) return rc;
    } else {
      SplitSum gu_pending;
      rc = gemm(c, M, M.wgu[l], c->h, h_lo, c->gu, T, 2 * F, d, 0, p.n_active, &gu_pending, s);
      if (rc) return rc;
      CU(launch_swiglu(m.dtype, c->gu, gu_pending, c->act, act_lo, T, F, p.n_active, s));
    }
    // the last layer's result must be complete in x when the pass ends
    const bool last = l + 1 == m.n_layers;
    x_pending = SplitSum();
    rc = gemm(c, M, M.wdown[l], c->act, act_lo, c->x, T, d, F, 1, p.n_active, (last || !defer_small) ? nullptr : &x_pending, s);
    if (rc) return rc;
  }
  return RSD_OK;
}

// Decode pass of a bf16 model with RMSNorm folded into its neighbours: the kernel that completes the
// residual stream (reduce_norm) also writes the next GEMM's operand x * gain and the sums of squares, and
// that GEMM scales its result rows by the RMSNorm denominator; the K-split sums of the qkv product are
// added up by the RoPE kernel.  Ten kernels per layer instead of thirteen.  On return h / h_lo hold
// x * final_gain and norm_ssq the sums of squares of the final residual stream.
bool fused_decode_ok(const ModelHost& M) { return M.m.dtype == RSD_BF16 && M.split && M.m.d_model % 4 == 0; }

int forward_decode_fused(rsd_ctx* c, int which, PassView p, const void* final_gain, cudaStream_t s) {
  const ModelHost& M = c->mdl[which];
  const rsd_model& m = M.m;
  const int d = m.d_model, H = m.n_heads, KV = m.n_kv_heads, hd = m.head_dim, F = m.d_ffn;
  const int T = p.T;
  if (T <= 0) return RSD_OK;
  const RowScale rs{c->norm_ssq, norm_chunks(d), 1.f / (float)d, m.rms_eps};
  CU(launch_embed(m.dtype, m.tok_embed, p, c->x, d, s));
  CU(launch_reduce_norm(nullptr, 1, c->x, M.norm1[0], c->h, c->h_lo, c->norm_ssq, T, d, p.n_active, s));
  for (int l = 0; l < m.n_layers; ++l) {
    KvView kv{M.kv_pool + (size_t)l * M.layer_stride, c->st.page_table[which], c->max_pages, M.kv_dtype == 3 ? 1 : 0};
    SplitSum qkv_pending, gu_pending, x_pending;
    int rc = gemm(c, M, M.wqkv[l], c->h, c->h_lo, c->qkv, T, (H + 2 * KV) * hd, d, 0, p.n_active, &qkv_pending, s, rs);
    if (rc) return rc;
    CU(launch_rope_kv(M.kv_dtype, c->qkv, qkv_pending, p, c->q, kv, M.rope, H, KV, hd, s));
    CU(launch_attn_decode(M.kv_dtype, c->q, kv.pool_layer, kv.page_table, kv.max_pages, p.tok_row, p.tok_pos, 1,
                          c->attn, c->attn_lo, m.dtype, T, H, KV, hd, c->S, c->attn_scratch, c->attn_scratch_bytes,
                          p.n_active, s, c->attn_rows_hint));
    rc = gemm(c, M, M.wo[l], c->attn, c->attn_lo, c->x, T, d, H * hd, 1, p.n_active, &x_pending, s);
    if (rc) return rc;
    CU(launch_reduce_norm(x_pending.partials, x_pending.splits, c->x, M.norm2[l], c->h, c->h_lo, c->norm_ssq, T, d,
                          p.n_active, s));
    if (gu_fused_ok(M, T)) {
      rc = gemm_gu(c, M, M.wgu[l], c->h, c->h_lo, c->act, c->act_lo, T, F, d, p.n_active, s, rs);
      if (rc) return rc;
    } else {
      rc = gemm(c, M, M.wgu[l], c->h, c->h_lo, c->gu, T, 2 * F, d, 0, p.n_active, &gu_pending, s, rs);
      if (rc) return rc;
      CU(launch_swiglu(m.dtype, c->gu, gu_pending, c->act, c->act_lo, T, F, p.n_active, s));
    }
    x_pending = SplitSum();
    rc = gemm(c, M, M.wdown[l], c->act, c->act_lo, c->x, T, d, F, 1, p.n_active, &x_pending, s);
    if (rc) return rc;
    const void* next_gain = l + 1 < m.n_layers ? M.norm1[l + 1] : final_gain;
    CU(launch_reduce_norm(x_pending.partials, x_pending.splits, c->x, next_gain, c->h, c->h_lo, c->norm_ssq, T, d,
                          p.n_active, s));
  }
  return RSD_OK;
}

// Multi-token pass over the flat list built by launch_build_pass, `chunk` tokens at a time.
int run_ingest(rsd_ctx* c, int which, int n_total, bool want_reward, cudaStream_t s) {
  for (int c0 = 0; c0 < n_total; c0 += c->chunk) {
    const int Tc = std::min(c->chunk, n_total - c0);
    PassView p{c->st.pass_tok_id + c0, c->st.pass_tok_row + c0, c->st.pass_tok_pos + c0, Tc, nullptr};
    int rc = forward_pass(c, which, p, s);
    if (rc) return rc;
    if (want_reward) {
      const rsd_model& m = c->mdl[which].m;
      CU(launch_reward(m.dtype, c->x, m.final_norm, m.head, m.head_kind, c->st.last_idx, c0, Tc, m.d_model, m.rms_eps,
                       c->st.rewards, c->st.B, s));
      // rows whose previous step came from the target: that step's reward, read at its last token on the way
      CU(launch_reward(m.dtype, c->x, m.final_norm, m.head, m.head_kind, c->st.prev_idx, c0, Tc, m.d_model, m.rms_eps,
                       c->st.target_rewards, c->st.B, s));
    }
  }
  return RSD_OK;
}

__global__ void scatter_logits_kernel(const float* logits, const int32_t* slot_row, float* dbg, int V, int C,
                                      const int32_t* iter, const int32_t* n_active) {
  RSD_PDL_SYNC();
  if (*n_active == 0) return;
  const int row = slot_row[blockIdx.x];
  if (row < 0) return;
  const float* src = logits + (size_t)blockIdx.x * V;
  float* dst = dbg + ((size_t)row * C + *iter) * V;
  for (int i = threadIdx.x; i < V; i += blockDim.x) dst[i] = src[i];
}

MegaShape mega_shape(const ModelHost& M) {
  const rsd_model& m = M.m;
  return MegaShape{m.n_layers, m.d_model, m.n_heads, m.n_kv_heads, m.head_dim, m.d_ffn, m.dtype == RSD_BF16 && M.split, m.rms_eps};
}

// The persistent decode kernel (opt-in) serves bf16 models with 16-bit caches at up to 64 rows.
bool mega_wanted(const rsd_ctx* c, int which) {
  const ModelHost& M = c->mdl[which];
  if (!(c->cfg.debug_flags & RSD_DEBUG_PERSISTENT_DECODE)) return false;
  if (which == RSD_PRM || !fused_decode_ok(M) || (M.kv_dtype != 2 && M.kv_dtype != 3)) return false;
  if (!mega_supported(mega_shape(M), c->st.B)) return false;
  const MegaShape sh = mega_shape(M);
  return mega_partials_floats(sh, c->st.B) * sizeof(float) + 4096 + 256 <= c->gemm_scratch_bytes && c->st.B * sh.KV <= 1000;
}

// (Re)builds the kernel's parameter block of model `which` for the current batch size.
int ensure_mega(rsd_ctx* c, int which, cudaStream_t s) {
  if (!mega_wanted(c, which)) { c->mega_B[which] = 0; return RSD_OK; }
  if (c->mega_B[which] == c->st.B) return RSD_OK;
  const ModelHost& M = c->mdl[which];
  const int B = c->st.B;
  MegaBuild a{};
  a.shape = mega_shape(M);
  a.B = B; a.max_pages = c->max_pages;
  a.embed = M.m.tok_embed;
  a.wqkv = M.m.wqkv; a.wo = M.m.wo; a.wgu = M.m.wgu; a.wdown = M.m.wdown; a.norm1 = M.m.norm1; a.norm2 = M.m.norm2;
  a.kv_pool = M.kv_pool; a.layer_stride = M.layer_stride;
  a.x = c->x; a.h = c->h; a.h_lo = c->h_lo; a.attn = c->attn; a.attn_lo = c->attn_lo; a.act = c->act; a.act_lo = c->act_lo;
  a.partials = const_cast<float*>(gemm_partials(c->gemm_scratch));
  a.ssq = c->norm_ssq;
  // the decode-attention scratch holds the context-split partials: (max, sum) pairs first, outputs after them
  const size_t head = ((sizeof(int32_t) * 2 * (size_t)c->B_max + 255) / 256) * 256;
  int h_max = 0;
  for (int w = 0; w < 3; ++w) h_max = std::max(h_max, c->mdl[w].m.n_heads);
  a.part_ml = (float*)((char*)c->attn_scratch + head);
  a.part_o = a.part_ml + (size_t)c->B_max * h_max * 32 * 2;
  a.sync_words = c->mega_sync;
  a.err = (int*)((char*)c->gemm_scratch + 4096);
  a.rope = M.rope;
  a.page_table = c->st.page_table[which];
  a.prof = c->mega_prof[which];
  cudaError_t e = mega_build(c->mega_block[which], a, s);
  if (e == cudaErrorNotSupported) { c->mega_B[which] = 0; return RSD_OK; }
  CU(e);
  c->mega_B[which] = B;
  return RSD_OK;
}

__global__ void scatter_logits_sd_kernel(const float* logits, const int32_t* tok_row, const int32_t* out_idx, float* dbg,
                                         int V, int C, const int32_t* n_active) {
  RSD_PDL_SYNC();
  if (*n_active == 0) return;
  const int row = tok_row[blockIdx.x];
  if (row < 0) return;
  const float* src = logits + (size_t)blockIdx.x * V;
  float* dst = dbg + ((size_t)row * C + out_idx[blockIdx.x]) * V;
  for (int i = threadIdx.x; i < V; i += blockDim.x) dst[i] = src[i];
}

// Model pass + final norm + lm head over the T token slots of p: logits [T, vocab] in c->logits.
int model_logits(rsd_ctx* c, int which, PassView p, bool allow_mega, cudaStream_t s) {
  const ModelHost& M = c->mdl[which];
  const rsd_model& m = M.m;
  const int T = p.T;
  int rc;
  if (allow_mega && c->mega_B[which] > 0 && c->mega_B[which] == c->st.B && T == c->st.B) {
    // the whole layer stack in one persistent kernel
    CU(launch_decode_mega(c->mega_block[which], c->st.B, M.kv_dtype == 3, p, m.final_norm, s));
    const RowScale rs{c->norm_ssq, m.d_model / 128, 1.f / (float)m.d_model, m.rms_eps};
    rc = gemm(c, M, m.head, c->h, c->h_lo, c->logits, T, m.vocab, m.d_model, 0, p.n_active, nullptr, s, rs);
  } else if (fused_decode_ok(M)) {
    if ((rc = forward_decode_fused(c, which, p, m.final_norm, s))) return rc;
    const RowScale rs{c->norm_ssq, norm_chunks(m.d_model), 1.f / (float)m.d_model, m.rms_eps};
    rc = gemm(c, M, m.head, c->h, c->h_lo, c->logits, T, m.vocab, m.d_model, 0, p.n_active, nullptr, s, rs);
  } else {
    if ((rc = forward_pass(c, which, p, s))) return rc;
    CU(launch_rmsnorm(m.dtype, c->x, m.final_norm, c->h, M.split ? c->h_lo : nullptr, T, m.d_model, m.rms_eps,
                      nullptr, p.n_active, SplitSum(), s));
    rc = gemm(c, M, m.head, c->h, c->h_lo, c->logits, T, m.vocab, m.d_model, 0, p.n_active, nullptr, s);
  }
  return rc;
}

// Enqueues one decode iteration: (prepare, model pass, final norm, lm_head, sample, append).
int decode_iteration(rsd_ctx* c, int which, int phase, int n_slots, cudaStream_t s) {
  const rsd_model& m = c->mdl[which].m;
  CU(launch_decode_prepare(c->st, which, n_slots, s));
  PassView p{c->st.pass_tok_id, c->st.pass_tok_row, c->st.pass_tok_pos, n_slots, c->st.n_active};
  int rc = model_logits(c, which, p, true, s);
  if (rc) return rc;
  if (c->dbg_logits[phase]) {
    RSD_LAUNCH((scatter_logits_kernel), n_slots, 256, 0, s, c->logits, c->st.pass_tok_row, c->dbg_logits[phase], m.vocab, c->C,
                                                  c->st.iter, c->st.n_active);
    CU(launched(1));
  }
  SampleArgs a{c->logits, n_slots, m.vocab, c->v_limit, c->cfg.temperature, c->cfg.seed, which,
               c->st.pass_tok_row, c->st.pass_tok_pos, nullptr, c->st.n_active, c->sample_best};
  CU(launch_sample(a, s));
  CU(launch_decode_update(c->st, which, phase, c->sample_best, n_slots, c->lp, s));
  return RSD_OK;
}

// Speculative decoding of rejected steps, one proposal iteration of the draft over the waiting rows' slots: the
// token at the draft's cursor goes through the draft, the sampled token becomes the round's next proposal.
int sd_propose_iteration(rsd_ctx* c, int n_slots, cudaStream_t s) {
  const rsd_model& m = c->mdl[RSD_DRAFT].m;
  CU(launch_sd_propose_prepare(c->st, n_slots, s));
  PassView p{c->st.pass_tok_id, c->st.pass_tok_row, c->st.pass_tok_pos, n_slots, c->st.n_active};
  int rc = model_logits(c, RSD_DRAFT, p, false, s);
  if (rc) return rc;
  SampleArgs a{c->logits, n_slots, m.vocab, c->v_limit, c->cfg.temperature, c->cfg.seed, RSD_DRAFT,
               c->st.pass_tok_row, c->st.pass_tok_pos, nullptr, c->st.n_active, c->sample_best};
  CU(launch_sample(a, s));
  CU(launch_sd_propose_update(c->st, c->sample_best, n_slots, s));
  return RSD_OK;
}

// ... and the target's pass over a round: sd_k token slots per row slot (the last written token and all proposals
// but the last), the target's choice at every one of them, then the prefix rule.
int sd_verify_pass(rsd_ctx* c, int n_slots, cudaStream_t s) {
  const rsd_model& m = c->mdl[RSD_TARGET].m;
  CU(launch_sd_verify_prepare(c->st, n_slots, s));
  const int T = n_slots * c->sd_k;
  PassView p{c->st.pass_tok_id, c->st.pass_tok_row, c->st.pass_tok_pos, T, c->st.n_active};
  int rc = model_logits(c, RSD_TARGET, p, false, s);
  if (rc) return rc;
  if (c->dbg_logits[1]) {
    RSD_LAUNCH((scatter_logits_sd_kernel), T, 256, 0, s, c->logits, c->st.pass_tok_row, c->st.sd_out_idx, c->dbg_logits[1],
               m.vocab, c->C, c->st.n_active);
    CU(launched(1));
  }
  SampleArgs a{c->logits, T, m.vocab, c->v_limit, c->cfg.temperature, c->cfg.seed, RSD_TARGET,
               c->st.pass_tok_row, c->st.pass_tok_pos, nullptr, c->st.n_active, c->sample_best};
  CU(launch_sample(a, s));
  CU(launch_sd_accept(c->st, c->sample_best, n_slots, c->lp, s));
  return RSD_OK;
}

enum IterKind { kIterDecode = 0, kIterSdPropose = 1, kIterSdVerify = 2 };

int enqueue_iteration(rsd_ctx* c, IterKind kind, int which, int phase, int n_slots, cudaStream_t s) {
  switch (kind) {
    case kIterSdPropose: return sd_propose_iteration(c, n_slots, s);
    case kIterSdVerify: return sd_verify_pass(c, n_slots, s);
    default: return decode_iteration(c, which, phase, n_slots, s);
  }
}

// Captures one iteration of `kind` over n_slots slots into a graph (idle slots are skipped inside the
// kernels), so that a token costs one graph launch instead of some 300 kernel launches.
int ensure_decode_graph(rsd_ctx* c, IterKind kind, int which, int phase, int g, int n_slots) {
  const int B = c->st.B;
  if (c->dec_graph[g] && c->dec_graph_B[g] == B) return RSD_OK;
  if (c->dec_graph[g]) { cudaGraphExecDestroy(c->dec_graph[g]); c->dec_graph[g] = nullptr; }
  if (!c->cap_stream) CU(cudaStreamCreateWithFlags(&c->cap_stream, cudaStreamNonBlocking));
  const uint64_t before = launches_total();
  CU(cudaStreamBeginCapture(c->cap_stream, cudaStreamCaptureModeThreadLocal));
  const bool was_in_decode = c->in_decode, was_timed = c->time_this_iter;
  c->in_decode = true; c->time_this_iter = false;          // no event records inside the capture
  const int rc = enqueue_iteration(c, kind, which, phase, n_slots, c->cap_stream);
  c->in_decode = was_in_decode; c->time_this_iter = was_timed;
  cudaGraph_t graph = nullptr;
  cudaError_t e = cudaStreamEndCapture(c->cap_stream, &graph);
  if (rc) { if (graph) cudaGraphDestroy(graph); return rc; }
  CU(e);
  c->dec_graph_kernels[g] = launches_total() - before;
  e = cudaGraphInstantiate(&c->dec_graph[g], graph, 0);
  cudaGraphDestroy(graph);
  CU(e);
  c->dec_graph_B[g] = B;
  return RSD_OK;
}

// One decode phase: up to C iterations; every 16 iterations the host looks at the number of rows
// still decoding and stops early when none is left.
int decode_phase(rsd_ctx* c, int which, int phase, int n_slots, cudaStream_t s) {
  CU(launch_decode_begin(c->st, phase, s));
  if (n_slots <= 0) return RSD_OK;
  const bool graphs = !(c->cfg.debug_flags & RSD_DEBUG_NO_GRAPHS);
  // The attention kernel splits every row's context over so many CTAs that the ACTIVE rows fill the machine; the
  // rows of the phase are known here, so the iteration is captured once per power-of-two bucket of that number.
  int bucket = 0, rows_eff = c->st.B;
  while (bucket < 3 && n_slots * 2 <= rows_eff) { rows_eff = (rows_eff + 1) / 2; ++bucket; }
  c->attn_rows_hint = rows_eff;
  const int g = phase * 4 + bucket;
  // fixed shape per bucket: the rows of the phase sit in the first slots, so the iteration runs over the bucket's
  // slot count (the persistent kernel is built for all B slots); slots beyond the phase's rows are idle
  if (c->mega_B[which] == c->st.B) n_slots = c->st.B;
  else if (graphs) n_slots = rows_eff;
  c->in_decode = true;
  int rc = RSD_OK;
  for (int j = 0; j < c->C && rc == RSD_OK; ++j) {
    const bool timed_iter = c->time_stride > 0 && (j % 16) == 5;
    // the first iteration ever runs kernel by kernel (it also sets every kernel's attributes), then
    // the iteration is captured once and replayed
    const bool have_graph = graphs && c->dec_graph[g] && c->dec_graph_B[g] == c->st.B;
    if (graphs && !have_graph && j > 0) {
      rc = ensure_decode_graph(c, kIterDecode, which, phase, g, n_slots);
      if (rc) break;
    }
    if (graphs && !timed_iter && c->dec_graph[g] && c->dec_graph_B[g] == c->st.B) {
      cudaError_t e = cudaGraphLaunch(c->dec_graph[g], s);
      if (e != cudaSuccess) { c->in_decode = false; CU(e); }
      note_replayed_launches(c->dec_graph_kernels[g]);
    } else {
      c->time_this_iter = timed_iter;
      rc = decode_iteration(c, which, phase, n_slots, s);
      c->time_this_iter = false;
    }
    if (rc == RSD_OK && (j & 15) == 15 && j + 1 < c->C) {
      Scalars sc;
      rc = read_scalars(c, s, &sc);
      if (rc == RSD_OK && sc.n_active == 0) break;
    }
  }
  c->in_decode = false;
  c->attn_rows_hint = 0;
  return rc;
}

// The target phase with speculative decoding: rounds of sd_k proposal iterations of the draft and one pass of the
// target over all of them, until every waiting row's step has ended.  A round writes at least one token per row, so
// there are at most C rounds; the host looks at the number of unfinished rows after each.  The first round runs
// kernel by kernel, the following ones replay two captured graphs (proposal iteration, target pass) per bucket.
int decode_phase_sd(rsd_ctx* c, int n_slots, cudaStream_t s) {
  CU(launch_decode_begin(c->st, 1, s));
  if (n_slots <= 0) return RSD_OK;
  const bool graphs = !(c->cfg.debug_flags & RSD_DEBUG_NO_GRAPHS);
  int bucket = 0, rows_eff = c->st.B;
  while (bucket < 3 && n_slots * 2 <= rows_eff) { rows_eff = (rows_eff + 1) / 2; ++bucket; }
  if (graphs) n_slots = rows_eff;
  c->in_decode = true;
  int rc = RSD_OK;
  auto run = [&](IterKind kind, int g, bool direct) -> int {
    c->attn_rows_hint = kind == kIterSdVerify ? rows_eff * c->sd_k : rows_eff;
    if (graphs && !direct) {
      int r = ensure_decode_graph(c, kind, kind == kIterSdVerify ? RSD_TARGET : RSD_DRAFT, 1, g, n_slots);
      if (r) return r;
      cudaError_t e = cudaGraphLaunch(c->dec_graph[g], s);
      if (e != cudaSuccess) { c->in_decode = false; CU(e); }
      note_replayed_launches(c->dec_graph_kernels[g]);
      return RSD_OK;
    }
    return enqueue_iteration(c, kind, 0, 1, n_slots, s);
  };
  for (int round = 0; round < c->C && rc == RSD_OK; ++round) {
    const bool direct = round == 0;
    for (int j = 0; j < c->sd_k && rc == RSD_OK; ++j) rc = run(kIterSdPropose, 8 + bucket, direct);
    if (rc == RSD_OK) rc = run(kIterSdVerify, 12 + bucket, direct);
    if (rc != RSD_OK) break;
    Scalars sc;
    rc = read_scalars(c, s, &sc);
    if (rc == RSD_OK && sc.n_active == 0) break;
  }
  c->in_decode = false;
  c->attn_rows_hint = 0;
  return rc;
}

__global__ void init_rows_kernel(RowState st, const int32_t* flat, const int32_t* offsets, int B) {
  RSD_PDL_SYNC();
  const int b = blockIdx.x;
  const int o = offsets[b], n = offsets[b + 1] - o;
  for (int i = threadIdx.x; i < n; i += blockDim.x) st.tok[(size_t)b * st.S + i] = flat[o + i];
  if (threadIdx.x == 0) {
    st.z_len[b] = n;
    st.live[b] = (n >= 1 && n + st.C <= st.S) ? 1 : 0;
    st.n_steps[b] = 0;
    for (int w = 0; w < 3; ++w) { st.kv_len[w][b] = 0; st.n_pages[w][b] = 0; }
    for (int p = 0; p < 2; ++p) { st.gen_len[p][b] = 0; st.forced_len[p][b] = 0; }
    st.forced_accept[b] = 255;
    st.rewards[b] = 0.f;
    st.target_rewards[b] = __int_as_float(0x7FC00000);   // NaN: no target-written step has been scored yet
    st.prev_idx[b] = -1;
    st.accept[b] = 0;
    st.waiting[b] = 0;
  }
}

int clear_forcing(rsd_ctx* c, cudaStream_t s) {
  CU(cudaMemsetAsync(c->st.forced_len[0], 0, sizeof(int32_t) * c->B_max, s));
  CU(cudaMemsetAsync(c->st.forced_len[1], 0, sizeof(int32_t) * c->B_max, s));
  CU(cudaMemsetAsync(c->st.forced_accept, 255, c->B_max, s));
  CU(cudaMemsetAsync(c->st.sd_forced_on, 0, c->B_max, s));
  return RSD_OK;
}

}  // namespace

// =================================================================================================
// C ABI
// =================================================================================================
extern "C" {

int rsd_query_sizes(const rsd_model* draft, const rsd_model* prm, const rsd_model* target, rsd_config* cfg) {
  const char* why;
  int rc = check_config(cfg, &why);
  if (rc) return fail(nullptr, rc, "config: %s", why);
  const rsd_model* ms[3] = {draft, prm, target};
  for (int i = 0; i < 3; ++i) {
    rc = check_model(ms[i], &why);
    if (rc) return fail(nullptr, rc, "model: %s", why);
  }
  const int max_pages = (cfg->max_seq_tokens + kPageTokens - 1) / kPageTokens;
  for (int i = 0; i < 3; ++i) cfg->kv_bytes[i] = kv_pool_bytes(*ms[i], cfg->max_batch * max_pages, cfg->kv_extended);
  if (cfg->prm_shares_draft) cfg->kv_bytes[RSD_PRM] = 0;   // the PRM reads the draft's cache
  cfg->workspace_bytes = layout_workspace(*cfg, ms, nullptr);
  return RSD_OK;
}

int rsd_create(const rsd_config* cfg, rsd_ctx** out) {
  const char* why;
  if (!out) return fail(nullptr, RSD_ERR_ARG, "null output pointer%s");
  *out = nullptr;
  int rc = check_config(cfg, &why);
  if (rc) return fail(nullptr, rc, "config: %s", why);
  if (!cfg->workspace || !cfg->kv_pool[0] || (!cfg->kv_pool[1] && !cfg->prm_shares_draft) || !cfg->kv_pool[2])
    return fail(nullptr, RSD_ERR_ARG, "workspace and KV pools must be provided by the caller%s");
  int dev_count = 0;
  if (cudaGetDeviceCount(&dev_count) != cudaSuccess || dev_count == 0)
    return fail(nullptr, RSD_ERR_CUDA, "no CUDA device: this library has no CPU fallback%s");
  rsd_ctx* c = new (std::nothrow) rsd_ctx();
  if (!c) return fail(nullptr, RSD_ERR_ARG, "out of host memory%s");
  c->cfg = *cfg;
  // scalars, then a mirror of the step's output block (every array of it rounded up to 256 bytes)
  c->pinned_bytes = 4096 + (size_t)cfg->max_batch * (cfg->max_step_tokens * 4 + 64) + 16 * 256;
  if (cudaHostAlloc((void**)&c->pinned, c->pinned_bytes, cudaHostAllocDefault) != cudaSuccess) {
    delete c;
    return fail(nullptr, RSD_ERR_CUDA, "pinned host allocation failed%s");
  }
  c->lp.step_end_id = cfg->step_end_id; c->lp.eos_id = cfg->eos_id; c->lp.step_end_mod = cfg->step_end_mod;
  c->lp.max_steps = cfg->max_steps; c->lp.omega_kind = cfg->omega_kind; c->lp.omega_alpha = cfg->omega_alpha;
  c->lp.seed = cfg->seed;
  *out = c;
  return RSD_OK;
}

int rsd_load_models(rsd_ctx* c, const rsd_model* draft, const rsd_model* prm, const rsd_model* target) {
  if (!c) return RSD_ERR_ARG;
  if (c->poisoned) return fail(c, RSD_ERR_STATE, "context unusable after a CUDA error%s");
  // captured decode graphs, parameter blocks and tensor maps hold the first models' pointers and shapes
  if (c->loaded) return fail(c, RSD_ERR_STATE, "models are loaded once per context: create a new context for other models%s");
  const rsd_model* ms[3] = {draft, prm, target};
  const char* why;
  for (int i = 0; i < 3; ++i) {
    int rc = check_model(ms[i], &why);
    if (rc) return fail(c, rc, "model: %s", why);
    const bool head_only = i == RSD_PRM && c->cfg.prm_shares_draft;
    if (!ms[i]->tok_embed || !ms[i]->final_norm || !ms[i]->head ||
        (!head_only && (!ms[i]->wqkv || !ms[i]->wo || !ms[i]->wgu || !ms[i]->wdown || !ms[i]->norm1 || !ms[i]->norm2)))
      return fail(c, RSD_ERR_ARG, "model: null weight pointer%s");
  }
  if (c->cfg.prm_shares_draft && (prm->d_model != draft->d_model || prm->dtype != draft->dtype))
    return fail(c, RSD_ERR_ARG, "prm_shares_draft: the PRM head must have the draft's width and dtype%s");
  if (draft->head_kind != RSD_HEAD_LM || target->head_kind != RSD_HEAD_LM || prm->head_kind == RSD_HEAD_LM)
    return fail(c, RSD_ERR_ARG, "draft and target need lm heads, the PRM a scalar head%s");
  const size_t need = layout_workspace(c->cfg, ms, nullptr);
  if (need > c->cfg.workspace_bytes) return fail(c, RSD_ERR_OOM_PAGES, "workspace smaller than rsd_query_sizes reports%s");
  layout_workspace(c->cfg, ms, c);
  const int max_pages = c->max_pages;
  for (int w = 0; w < 3; ++w) {
    ModelHost& M = c->mdl[w];
    M.m = *ms[w];
    if (w == RSD_PRM && c->cfg.prm_shares_draft) {
      // head on the draft's trunk: no layers, no cache of its own
      M.m.wqkv = M.m.wo = M.m.wgu = M.m.wdown = M.m.norm1 = M.m.norm2 = nullptr;
      M.elem = M.m.dtype == RSD_BF16 ? 2 : 4;
      M.split = M.m.dtype == RSD_BF16;
      M.n_params = count_params(M.m);
      M.pool_pages = 0;
      c->st.pool_pages[w] = 0;
      continue;
    }
    const int L = M.m.n_layers;
    M.wqkv.assign(ms[w]->wqkv, ms[w]->wqkv + L); M.wo.assign(ms[w]->wo, ms[w]->wo + L);
    M.wgu.assign(ms[w]->wgu, ms[w]->wgu + L); M.wdown.assign(ms[w]->wdown, ms[w]->wdown + L);
    M.norm1.assign(ms[w]->norm1, ms[w]->norm1 + L); M.norm2.assign(ms[w]->norm2, ms[w]->norm2 + L);
    M.m.wqkv = M.wqkv.data(); M.m.wo = M.wo.data(); M.m.wgu = M.wgu.data(); M.m.wdown = M.wdown.data();
    M.m.norm1 = M.norm1.data(); M.m.norm2 = M.norm2.data();
    M.elem = M.m.dtype == RSD_BF16 ? 2 : 4;
    M.kv_dtype = M.m.dtype == RSD_BF16 ? (kv_extended_for(M.m, c->cfg.kv_extended) ? 3 : 2) : 0;
    // hi + lo operands for the bf16 policies (logits within 3e-2 need them: plain bf16 GEMM inputs alone cost
    // 5.7e-2 at the 1.5B shape).  The PRM's one scalar is far less sensitive: with plain bf16 operands a
    // 1.5B-shape PRM errs by 1.5e-3 against the 1e-2 asked, a 7B-shape one by 1.1e-2; the error grows with the
    // width, so PRMs of up to 2048 columns take plain operands (half the tensor-core work of a scoring pass),
    // wider ones the pairs.
    M.split = M.m.dtype == RSD_BF16 && !(w == RSD_PRM && M.m.d_model <= 2048);
    M.f16_dense = M.split && M.w16 != nullptr && wants_f16_dense(c->cfg, M.m, w);
    M.w16_layer = layer_weight_elems(M.m);
    M.n_params = count_params(M.m);
    M.kv_pool = (char*)c->cfg.kv_pool[w];
    const size_t page_bytes = (size_t)(M.kv_dtype == 3 ? 4 : 2) * M.m.n_kv_heads * kPageTokens * M.m.head_dim * M.elem;
    int pages = (int)std::min<size_t>(c->cfg.kv_bytes[w] / (page_bytes * L), (size_t)c->B_max * max_pages);
    if (pages < 1) return fail(c, RSD_ERR_OOM_PAGES, "KV pool too small for a single page%s");
    M.pool_pages = pages;
    M.layer_stride = (size_t)pages * page_bytes;
    c->st.pool_pages[w] = pages;
  }
  c->v_limit = std::min(std::min(draft->vocab, prm->vocab), target->vocab);
  cudaStream_t s = 0;
  for (int w = 0; w < 3; ++w)
    CU(launch_rope_table(c->mdl[w].rope, c->S, c->mdl[w].m.head_dim, c->mdl[w].m.rope_theta, s));
  // fp16 copies of the layer matrices for the dense passes (exact for |w| >= 2^-14, to 2^-25 absolute below)
  for (int w = 0; w < 3; ++w) {
    const ModelHost& M = c->mdl[w];
    if (!M.f16_dense) continue;
    for (int l = 0; l < M.m.n_layers; ++l) {
      const void* src[4] = {M.wqkv[l], M.wo[l], M.wgu[l], M.wdown[l]};
      for (int k = 0; k < 4; ++k)
        CU(launch_bf16_to_f16(src[k], const_cast<void*>(M.w16_of(l, k)), M.w16_elems(k), s));
    }
  }
  CU(cudaMemsetAsync(c->d_scalars, 0, 16 * sizeof(int32_t), s));
  CU(cudaMemsetAsync(c->gemm_scratch, 0, c->gemm_scratch_bytes, s));
  CU(cudaMemsetAsync(c->sample_best, 0, sizeof(unsigned long long) * c->slots_max, s));
  CU(cudaMemsetAsync(c->mega_sync, 0, sizeof(int32_t) * 1024, s));
  int rc = clear_forcing(c, s);
  if (rc) return rc;
  CU(cudaStreamSynchronize(s));
  c->loaded = true;
  c->prefilled = false;
  return RSD_OK;
}

int rsd_reset(rsd_ctx* c) {
  if (!c) return RSD_ERR_ARG;
  if (c->poisoned) return fail(c, RSD_ERR_STATE, "context unusable after a CUDA error%s");
  if (!c->loaded) return fail(c, RSD_ERR_STATE, "no models loaded%s");
  CU(cudaDeviceSynchronize());
  CU(cudaMemset(c->d_scalars, 0, 16 * sizeof(int32_t)));
  c->st.B = 0;
  c->prefilled = false;
  memset(&c->ctr, 0, sizeof(c->ctr));
  return RSD_OK;
}

int rsd_prefill(rsd_ctx* c, const int32_t* tokens, const int32_t* offsets, int32_t B, void* cuda_stream) {
  if (!c) return RSD_ERR_ARG;
  if (c->poisoned) return fail(c, RSD_ERR_STATE, "context unusable after a CUDA error%s");
  if (!c->loaded) return fail(c, RSD_ERR_STATE, "rsd_prefill before rsd_load_models%s");
  if (!tokens || !offsets || B < 1 || B > c->B_max) return fail(c, RSD_ERR_ARG, "prefill: bad batch%s");
  if (offsets[0] != 0) return fail(c, RSD_ERR_ARG, "prefill: offsets[0] must be 0%s");
  for (int b = 0; b < B; ++b) {
    const int n = offsets[b + 1] - offsets[b];
    if (n < 1 || n > c->S) return fail(c, RSD_ERR_ARG, "prefill: prompt length out of 1..max_seq_tokens%s");
  }
  const int total = offsets[B];
  for (int i = 0; i < total; ++i)
    if (tokens[i] < 0 || tokens[i] >= c->v_limit) return fail(c, RSD_ERR_ARG, "prefill: token id out of range%s");
  cudaStream_t s = (cudaStream_t)cuda_stream;
  int rc = rsd_reset(c);
  if (rc) return rc;
  c->st.B = B;
  // stage the ragged prompt in the pass-list buffers, then scatter it into the row buffers
  CU(cudaMemcpyAsync(c->st.pass_tok_id, tokens, sizeof(int32_t) * total, cudaMemcpyHostToDevice, s));
  CU(cudaMemcpyAsync(c->st.pass_tok_row, offsets, sizeof(int32_t) * (B + 1), cudaMemcpyHostToDevice, s));
  RSD_LAUNCH((init_rows_kernel), B, 128, 0, s, c->st, c->st.pass_tok_id, c->st.pass_tok_row, B);
  CU(launched(1));
  CU(cudaStreamSynchronize(s));  // the staging buffers are reused below
  const bool merged = c->cfg.prm_shares_draft != 0;
  if ((rc = ensure_mega(c, RSD_DRAFT, s)) || (rc = ensure_mega(c, RSD_TARGET, s))) return rc;
  CU(launch_reserve_pages(c->st, RSD_DRAFT, kReservePrefillDraft, 1, s));
  if (!merged) CU(launch_reserve_pages(c->st, RSD_PRM, kReservePrefillPrm, 1, s));
  Scalars sc;
  CU(launch_build_pass(c->st, RSD_DRAFT, kPassIngestDraft, 1, s));
  rc = read_scalars(c, s, &sc);
  if (rc) return rc;
  rc = run_ingest(c, RSD_DRAFT, sc.n_tok, false, s);
  if (rc) return rc;
  c->ctr.ingest_tokens[RSD_DRAFT] += sc.n_tok;
  if (!merged) {
    CU(launch_build_pass(c->st, RSD_PRM, kPassScorePrm, 1, s));
    rc = read_scalars(c, s, &sc);
    if (rc) return rc;
    rc = run_ingest(c, RSD_PRM, sc.n_tok, false, s);
    if (rc) return rc;
    c->ctr.ingest_tokens[RSD_PRM] += sc.n_tok;
  }
  CU(cudaStreamSynchronize(s));
  c->prefilled = true;
  return RSD_OK;
}

// Merged PRM: r_i from the draft's trunk.  The draft's cache holds z_i and y^_i up to the step's last
// token; that token goes through the draft once more (its keys and values land beyond the cursor,
// which does not move) and the PRM's final norm and head read the hidden state.
static int score_with_draft_trunk(rsd_ctx* c, cudaStream_t s) {
  const ModelHost& D = c->mdl[RSD_DRAFT];
  const rsd_model& prm = c->mdl[RSD_PRM].m;
  const int B = c->st.B;
  CU(launch_score_prepare(c->st, s));
  PassView p{c->st.pass_tok_id, c->st.pass_tok_row, c->st.pass_tok_pos, B, c->st.n_active};
  int rc;
  const bool was_in_decode = c->in_decode;
  c->in_decode = true;             // GEMM timing: treated like a decode iteration that is not sampled
  if (fused_decode_ok(D)) rc = forward_decode_fused(c, RSD_DRAFT, p, prm.final_norm, s);
  else rc = forward_pass(c, RSD_DRAFT, p, s);
  c->in_decode = was_in_decode;
  if (rc) return rc;
  CU(launch_reward(prm.dtype, c->x, prm.final_norm, prm.head, prm.head_kind, c->st.last_idx, 0, B, prm.d_model,
                   prm.rms_eps, c->st.rewards, B, s));
  return RSD_OK;
}

static int step_impl(rsd_ctx* c, float delta, int min_target_rows, void* cuda_stream, int32_t* step_tokens,
                     int32_t* step_len, float* rewards, uint8_t* accept, uint8_t* live, uint8_t* waiting,
                     bool device_outputs = false) {
  if (!c) return RSD_ERR_ARG;
  if (c->poisoned) return fail(c, RSD_ERR_STATE, "context unusable after a CUDA error%s");
  if (!c->prefilled) return fail(c, RSD_ERR_STATE, "rsd_step before rsd_prefill%s");
  if (min_target_rows < 1) return fail(c, RSD_ERR_ARG, "min_target_rows must be at least 1%s");
  cudaStream_t s = (cudaStream_t)cuda_stream;
  const int B = c->st.B;
  Scalars sc;
  int rc;
#define PHASE(i) do { if (c->time_phases) CU(cudaEventRecord(c->ph_ev[i], s)); } while (0)
  PHASE(0);
  // draft: catch up on a step the target wrote last time, then decode y^_i (rows that wait for the
  // target take no part)
  CU(launch_reserve_pages(c->st, RSD_DRAFT, kReserveStepDraft, 1, s));
  CU(launch_build_pass(c->st, RSD_DRAFT, kPassIngestDraft, 1, s));
  if ((rc = read_scalars(c, s, &sc))) return rc;
  const int n_sync = sc.n_tok;
  if ((rc = run_ingest(c, RSD_DRAFT, n_sync, false, s))) return rc;
  PHASE(1);
  if ((rc = decode_phase(c, RSD_DRAFT, 0, B, s))) return rc;
  PHASE(2);
  // PRM: score y^_i at its last token
  const bool merged = c->cfg.prm_shares_draft != 0;
  int n_prm = 0;
  if (merged) {
    if ((rc = score_with_draft_trunk(c, s))) return rc;
  } else {
    CU(launch_reserve_pages(c->st, RSD_PRM, kReserveScorePrm, 1, s));
    CU(launch_build_pass(c->st, RSD_PRM, kPassScorePrm, 1, s));
    if ((rc = read_scalars(c, s, &sc))) return rc;
    n_prm = sc.n_tok;
    if ((rc = run_ingest(c, RSD_PRM, n_prm, true, s))) return rc;
  }
  PHASE(3);
  // gate, compaction of the waiting rows; once enough of them wait: target catch-up and decode
  CU(launch_gate(c->st, delta, c->lp, s));
  CU(launch_reserve_pages(c->st, RSD_TARGET, kReserveTarget, min_target_rows, s));
  CU(launch_build_pass(c->st, RSD_TARGET, kPassCatchupTarget, min_target_rows, s));
  if ((rc = read_scalars(c, s, &sc))) return rc;
  const int n_catch = sc.n_tok, n_rej = sc.n_rej;
  const bool target_runs = target_pass_due(n_rej, sc.n_live, min_target_rows);
  c->last_n_rej = n_rej;
  PHASE(4);
  if (target_runs && (rc = run_ingest(c, RSD_TARGET, n_catch, false, s))) return rc;
  PHASE(5);
  if (target_runs && (rc = c->sd_k > 0 ? decode_phase_sd(c, n_rej, s) : decode_phase(c, RSD_TARGET, 1, n_rej, s))) return rc;
  PHASE(6);
  // commit and read the results back
  CU(launch_commit(c->st, c->lp, target_runs ? 1 : 0, c->o_tokens, c->o_len, c->o_rewards, c->o_accept, c->o_live,
                   c->o_role, c->o_waiting, c->o_gen, s));
  // one device-to-host copy brings the whole output block; the arrays sit in it at their workspace offsets
  char* hp = c->pinned + 256;
  if (256 + c->o_block_bytes > c->pinned_bytes) return fail(c, RSD_ERR_STATE, "output mirror too small%s");
  CU(cudaMemcpyAsync(hp, c->o_tokens, c->o_block_bytes, cudaMemcpyDeviceToHost, s));
  auto mirror = [&](const void* dev) { return hp + ((const char*)dev - (const char*)c->o_tokens); };
  const int32_t* h_tokens = (const int32_t*)mirror(c->o_tokens);
  const int32_t* h_len = (const int32_t*)mirror(c->o_len);
  const int32_t* h_gen0 = (const int32_t*)mirror(c->o_gen);
  const int32_t* h_gen1 = h_gen0 + B;
  const float* h_rew = (const float*)mirror(c->o_rewards);
  const uint8_t* h_acc = (const uint8_t*)mirror(c->o_accept);
  const uint8_t* h_live = (const uint8_t*)mirror(c->o_live);
  const uint8_t* h_role = (const uint8_t*)mirror(c->o_role);
  const uint8_t* h_wait = (const uint8_t*)mirror(c->o_waiting);
  if (device_outputs) {
    // the caller's arrays are device memory: filled on the stream, in stream order with the call's kernels
    if (step_tokens) CU(cudaMemcpyAsync(step_tokens, c->o_tokens, sizeof(int32_t) * (size_t)B * c->C, cudaMemcpyDeviceToDevice, s));
    if (step_len) CU(cudaMemcpyAsync(step_len, c->o_len, sizeof(int32_t) * B, cudaMemcpyDeviceToDevice, s));
    if (rewards) CU(cudaMemcpyAsync(rewards, c->o_rewards, sizeof(float) * B, cudaMemcpyDeviceToDevice, s));
    if (accept) CU(cudaMemcpyAsync(accept, c->o_accept, B, cudaMemcpyDeviceToDevice, s));
    if (live) CU(cudaMemcpyAsync(live, c->o_live, B, cudaMemcpyDeviceToDevice, s));
    if (waiting) CU(cudaMemcpyAsync(waiting, c->o_waiting, B, cudaMemcpyDeviceToDevice, s));
  }
  if ((rc = clear_forcing(c, s))) return rc;
  PHASE(7);
#undef PHASE
  if ((rc = read_scalars(c, s, &sc))) return rc;
  if (c->time_phases) {
    for (int i = 0; i < 7; ++i) {
      float ms = 0.f;
      CU(cudaEventElapsedTime(&ms, c->ph_ev[i], c->ph_ev[i + 1]));
      c->ph_ms[i] += ms;
    }
  }
  // counters (Section 3.3 accounting): draft tokens when they are generated, steps when they are committed
  uint64_t gen_d = 0, gen_t = 0, n_acc = 0, n_tgt = 0, discarded = 0, n_scored = 0;
  for (int b = 0; b < B; ++b) {
    const int code = h_role[b] & 3;
    if (code) { gen_d += h_gen0[b]; ++n_scored; }
    if (code == 1) ++n_acc;
    if (code == 2) discarded += h_gen0[b];
    if (h_role[b] & 4) { gen_t += h_gen1[b]; ++n_tgt; }
  }
  c->ctr.gen_tokens[RSD_DRAFT] += gen_d;
  c->ctr.gen_tokens[RSD_TARGET] += gen_t;
  c->ctr.ingest_tokens[RSD_DRAFT] += n_sync;
  c->ctr.ingest_tokens[RSD_PRM] += merged ? 0 : (uint64_t)n_prm - gen_d;
  c->ctr.ingest_tokens[RSD_TARGET] += target_runs ? n_catch : 0;
  c->ctr.score_tokens += merged ? n_scored : gen_d;   // merged PRM: one token per scored step
  c->ctr.steps += n_acc + n_tgt; c->ctr.accepted_steps += n_acc; c->ctr.rejected_steps += n_tgt;
  c->ctr.discarded_draft_tokens += discarded;
  // speculative decoding of rejected steps: the device keeps running totals since the last reset
  c->ctr.sd_rounds = (uint64_t)sc.sd_rounds; c->ctr.sd_proposed = (uint64_t)sc.sd_proposed;
  c->ctr.sd_matched = (uint64_t)sc.sd_matched; c->ctr.sd_verified = (uint64_t)sc.sd_proposed;
  if (device_outputs) return RSD_OK;
  if (step_tokens) memcpy(step_tokens, h_tokens, sizeof(int32_t) * (size_t)B * c->C);
  if (step_len) memcpy(step_len, h_len, sizeof(int32_t) * B);
  if (rewards) memcpy(rewards, h_rew, sizeof(float) * B);
  if (accept) memcpy(accept, h_acc, B);
  if (live) memcpy(live, h_live, B);
  if (waiting) memcpy(waiting, h_wait, B);
  return RSD_OK;
}

int rsd_step(rsd_ctx* c, float delta, void* cuda_stream, int32_t* step_tokens, int32_t* step_len, float* rewards,
             uint8_t* accept, uint8_t* live) {
  return step_impl(c, delta, 1, cuda_stream, step_tokens, step_len, rewards, accept, live, nullptr);
}

int rsd_step_queued(rsd_ctx* c, float delta, int32_t min_target_rows, void* cuda_stream, int32_t* step_tokens,
                    int32_t* step_len, float* rewards, uint8_t* accept, uint8_t* live, uint8_t* waiting) {
  return step_impl(c, delta, min_target_rows, cuda_stream, step_tokens, step_len, rewards, accept, live, waiting);
}

int rsd_step_device(rsd_ctx* c, float delta, int32_t min_target_rows, void* cuda_stream, int32_t* step_tokens,
                    int32_t* step_len, float* rewards, uint8_t* accept, uint8_t* live, uint8_t* waiting) {
  return step_impl(c, delta, min_target_rows, cuda_stream, step_tokens, step_len, rewards, accept, live, waiting, true);
}

int rsd_flops_counters(rsd_ctx* c, rsd_counters* out) {
  if (!c || !out) return RSD_ERR_ARG;
  if (!c->loaded) return fail(c, RSD_ERR_STATE, "no models loaded%s");
  rsd_counters r = c->ctr;
  const double nd = c->mdl[RSD_DRAFT].n_params, np = c->mdl[RSD_PRM].n_params, nt = c->mdl[RSD_TARGET].n_params;
  // with speculative decoding the draft is billed its proposals too and the target every position it evaluated
  const double target_tokens = c->sd_k > 0 ? (double)r.sd_verified : (double)r.gen_tokens[RSD_TARGET];
  r.flops_paper = 2.0 * nd * (double)(r.gen_tokens[RSD_DRAFT] + r.sd_proposed) + 2.0 * nt * target_tokens +
                  2.0 * np * (double)(r.score_tokens + r.ingest_tokens[RSD_PRM]);
  r.flops_all_tokens = 2.0 * nd * (double)(r.gen_tokens[RSD_DRAFT] + r.sd_proposed + r.ingest_tokens[RSD_DRAFT]) +
                       2.0 * nt * (target_tokens + (double)r.ingest_tokens[RSD_TARGET]) +
                       2.0 * np * (double)(r.score_tokens + r.ingest_tokens[RSD_PRM]);
  *out = r;
  return RSD_OK;
}

int rsd_destroy(rsd_ctx* c) {
  if (!c) return RSD_OK;
  cudaDeviceSynchronize();
  for (cudaEvent_t e : c->ev) cudaEventDestroy(e);
  for (cudaEvent_t e : c->ph_ev) if (e) cudaEventDestroy(e);
  for (auto& g : c->dec_graph) if (g) cudaGraphExecDestroy(g);
  if (c->cap_stream) cudaStreamDestroy(c->cap_stream);

  if (c->pinned) cudaFreeHost(c->pinned);
  delete c;
  return RSD_OK;
}

const char* rsd_last_error(const rsd_ctx* c) { return c ? c->err.c_str() : g_create_error.c_str(); }

// ---- parity hooks ---------------------------------------------------------------------------
int rsd_debug_force(rsd_ctx* c, int which, const int32_t* tokens, const int32_t* len, const uint8_t* accept) {
  if (!c) return RSD_ERR_ARG;
  if (!c->prefilled) return fail(c, RSD_ERR_STATE, "forcing needs rows%s");
  const int B = c->st.B;
  if (which == RSD_PRM) {
    if (!accept) return fail(c, RSD_ERR_ARG, "null accept mask%s");
    CU(cudaMemcpy(c->st.forced_accept, accept, B, cudaMemcpyHostToDevice));
    return RSD_OK;
  }
  if (which != RSD_DRAFT && which != RSD_TARGET) return fail(c, RSD_ERR_ARG, "which%s");
  if (!tokens || !len) return fail(c, RSD_ERR_ARG, "null forcing arrays%s");
  for (int b = 0; b < B; ++b)
    if (len[b] < 0 || len[b] > c->C) return fail(c, RSD_ERR_ARG, "forced length out of range%s");
  const int p = which == RSD_DRAFT ? 0 : 1;
  CU(cudaMemcpy(c->st.forced_tok[p], tokens, sizeof(int32_t) * (size_t)B * c->C, cudaMemcpyHostToDevice));
  CU(cudaMemcpy(c->st.forced_len[p], len, sizeof(int32_t) * B, cudaMemcpyHostToDevice));
  return RSD_OK;
}

int rsd_debug_force_sd(rsd_ctx* c, const int32_t* props, const uint8_t* on) {
  if (!c || !props || !on) return RSD_ERR_ARG;
  if (!c->prefilled) return fail(c, RSD_ERR_STATE, "forcing needs rows%s");
  if (!c->st.sd_forced_props) return fail(c, RSD_ERR_STATE, "needs sd_tokens > 0 and RSD_DEBUG_KEEP_LOGITS%s");
  const int B = c->st.B;
  CU(cudaMemcpy(c->st.sd_forced_props, props, sizeof(int32_t) * (size_t)B * c->C * c->sd_k, cudaMemcpyHostToDevice));
  CU(cudaMemcpy(c->st.sd_forced_on, on, B, cudaMemcpyHostToDevice));
  return RSD_OK;
}

int rsd_debug_get_logits(rsd_ctx* c, int which, float* out) {
  if (!c || !out) return RSD_ERR_ARG;
  const int p = which == RSD_DRAFT ? 0 : (which == RSD_TARGET ? 1 : -1);
  if (p < 0 || !c->dbg_logits[p]) return fail(c, RSD_ERR_STATE, "logits were not kept%s");
  CU(cudaMemcpy(out, c->dbg_logits[p], sizeof(float) * (size_t)c->st.B * c->C * c->mdl[which].m.vocab, cudaMemcpyDeviceToHost));
  return RSD_OK;
}

int rsd_get_target_step_rewards(rsd_ctx* c, float* out) {
  if (!c || !out) return RSD_ERR_ARG;
  if (!c->prefilled) return fail(c, RSD_ERR_STATE, "no rows%s");
  CU(cudaDeviceSynchronize());
  CU(cudaMemcpy(out, c->st.target_rewards, sizeof(float) * c->st.B, cudaMemcpyDeviceToHost));
  return RSD_OK;
}

int rsd_debug_get_sampled(rsd_ctx* c, int which, int32_t* out) {
  if (!c || !out) return RSD_ERR_ARG;
  const int p = which == RSD_DRAFT ? 0 : (which == RSD_TARGET ? 1 : -1);
  if (p < 0 || !c->prefilled) return fail(c, RSD_ERR_ARG, "which%s");
  CU(cudaMemcpy(out, c->st.sampled[p], sizeof(int32_t) * (size_t)c->st.B * c->C, cudaMemcpyDeviceToHost));
  return RSD_OK;
}

int rsd_debug_get_state(rsd_ctx* c, int32_t* z_len, int32_t* kv_len, int32_t* n_pages, int32_t* page_table,
                        int32_t* next_page, int32_t* rej_idx, int32_t* n_rej) {
  if (!c) return RSD_ERR_ARG;
  if (!c->prefilled) return fail(c, RSD_ERR_STATE, "no rows%s");
  const int B = c->st.B;
  CU(cudaDeviceSynchronize());
  if (z_len) CU(cudaMemcpy(z_len, c->st.z_len, sizeof(int32_t) * B, cudaMemcpyDeviceToHost));
  for (int w = 0; w < 3; ++w) {
    if (kv_len) CU(cudaMemcpy(kv_len + (size_t)w * B, c->st.kv_len[w], sizeof(int32_t) * B, cudaMemcpyDeviceToHost));
    if (n_pages) CU(cudaMemcpy(n_pages + (size_t)w * B, c->st.n_pages[w], sizeof(int32_t) * B, cudaMemcpyDeviceToHost));
    if (page_table)
      CU(cudaMemcpy(page_table + (size_t)w * B * c->max_pages, c->st.page_table[w], sizeof(int32_t) * (size_t)B * c->max_pages, cudaMemcpyDeviceToHost));
  }
  if (next_page) CU(cudaMemcpy(next_page, c->st.next_page, sizeof(int32_t) * 3, cudaMemcpyDeviceToHost));
  if (rej_idx) CU(cudaMemcpy(rej_idx, c->st.rej_idx, sizeof(int32_t) * B, cudaMemcpyDeviceToHost));
  if (n_rej) *n_rej = c->last_n_rej;
  return RSD_OK;
}

int rsd_debug_gemm_timing_dense(rsd_ctx* c, double* ms, double* flops, uint64_t* launches) {
  if (!c) return RSD_ERR_ARG;
  CU(cudaDeviceSynchronize());
  int rc = drain_gemm_events(c);
  if (rc) return rc;
  for (int k = 0; k < 2; ++k) {
    if (ms) ms[k] = c->dense_ms[k];
    if (flops) flops[k] = c->dense_flops[k];
    if (launches) launches[k] = c->dense_launches[k];
    c->dense_ms[k] = 0; c->dense_flops[k] = 0; c->dense_launches[k] = 0;
  }
  return RSD_OK;
}

int rsd_debug_gemm_timing(rsd_ctx* c, int32_t stride, double* ms, double* bytes, uint64_t* launches) {
  if (!c || stride < 0) return RSD_ERR_ARG;
  CU(cudaDeviceSynchronize());
  int rc = drain_gemm_events(c);
  if (rc) return rc;
  if (ms) *ms = c->timed_ms;
  if (bytes) *bytes = c->timed_bytes;
  if (launches) *launches = c->timed_launches;
  c->timed_ms = 0; c->timed_bytes = 0; c->timed_launches = 0;
  c->gemm_calls = 0;
  if (stride > 0 && c->ev.empty()) {
    const size_t pairs = 8192;
    c->ev.resize(2 * pairs);
    for (auto& e : c->ev) CU(cudaEventCreate(&e));
    c->ev_bytes.assign(pairs, 0.0);
    c->ev_flops.assign(pairs, 0.0);
  }
  c->time_stride = stride;
  return RSD_OK;
}

uint64_t rsd_debug_launch_count(void) { return launches_total(); }

int rsd_debug_mega_profile(rsd_ctx* c, int which, uint64_t* stamps, int32_t capacity, int32_t* n_out) {
  if (!c || !stamps || !n_out || capacity < 1 || which < 0 || which > 2) return RSD_ERR_ARG;
  if (!c->mega_prof[which]) return fail(c, RSD_ERR_STATE, "RSD_DEBUG_MEGA_PROFILE was not set%s");
  CU(cudaDeviceSynchronize());
  unsigned long long n = 0;
  CU(cudaMemcpy(&n, c->mega_prof[which] + 1023, sizeof(n), cudaMemcpyDeviceToHost));
  const int take = (int)std::min<unsigned long long>(std::min<unsigned long long>(n, 1022), (unsigned long long)capacity);
  CU(cudaMemcpy(stamps, c->mega_prof[which], sizeof(uint64_t) * take, cudaMemcpyDeviceToHost));
  *n_out = take;
  return RSD_OK;
}

int rsd_debug_phase_ms(rsd_ctx* c, int32_t enable, double* out) {
  if (!c) return RSD_ERR_ARG;
  if (out) memcpy(out, c->ph_ms, sizeof(c->ph_ms));
  memset(c->ph_ms, 0, sizeof(c->ph_ms));
  if (enable && !c->ph_ev[0])
    for (auto& e : c->ph_ev) CU(cudaEventCreate(&e));
  c->time_phases = enable != 0;
  return RSD_OK;
}

// ---- single kernels -------------------------------------------------------------------------
#define KCU(call)                                     \
  do {                                                \
    cudaError_t e_ = (call);                          \
    if (e_ != cudaSuccess) {                          \
      g_create_error = cudaGetErrorString(e_);        \
      return RSD_ERR_CUDA;                            \
    }                                                 \
  } while (0)

size_t rsd_k_gemm_scratch_bytes(int32_t M, int32_t N, int32_t K) {
  (void)N; (void)K;
  return gemm_scratch_bytes(M);
}

int rsd_k_gemm(const void* W, const void* x, const void* x_lo, float* y, int32_t M, int32_t N, int32_t K, int32_t dtype,
               int32_t accumulate, int32_t impl, void* scratch, size_t scratch_bytes, void* cuda_stream) {
  if (!W || !x || !y || M < 0 || N < 1 || K < 1 || (dtype != RSD_F32 && dtype != RSD_BF16) || impl < 0 || impl > 4)
    return RSD_ERR_ARG;
  if (impl == 4) {
    // the dense form of the long passes: W and x hold fp16, one operand per activation, more than 128 rows
    if (x_lo || dtype != RSD_BF16) return RSD_ERR_ARG;
    if (M <= 128 || K % 8 || !gemm_tc_supported(dtype, M, N, K)) return RSD_ERR_UNSUPPORTED;
    if (!scratch || scratch_bytes < gemm_scratch_bytes(M)) return RSD_ERR_ARG;
    KCU(launch_gemm_f16_dense(W, x, y, M, N, K, accumulate, scratch, scratch_bytes, (cudaStream_t)cuda_stream));
    return RSD_OK;
  }
  if (K % (dtype == RSD_BF16 ? 8 : 4)) return RSD_ERR_UNSUPPORTED;
  if (impl >= 2 && !gemm_tc_supported(dtype, M, N, K)) return RSD_ERR_UNSUPPORTED;
  if (impl != 1 && (!scratch || scratch_bytes < gemm_scratch_bytes(M))) return RSD_ERR_ARG;
  if (x_lo && dtype != RSD_BF16) return RSD_ERR_ARG;
  KCU(launch_gemm(dtype, W, x, x_lo, y, M, N, K, accumulate, impl, scratch, scratch_bytes, nullptr, nullptr, (cudaStream_t)cuda_stream));
  return RSD_OK;
}

int rsd_debug_gemm_wait_probe(const void* W, const void* x, float* y, void* scratch, size_t scratch_bytes, void* cuda_stream) {
  if (!W || !x || !y || !scratch || scratch_bytes < gemm_scratch_bytes(16)) return RSD_ERR_ARG;
  cudaStream_t s = (cudaStream_t)cuda_stream;
  KCU(launch_gemm_wait_probe(W, x, y, scratch, scratch_bytes, s));
  int32_t flag = 0;
  KCU(cudaMemcpyAsync(&flag, (char*)scratch + 4096, sizeof(flag), cudaMemcpyDeviceToHost, s));
  KCU(cudaStreamSynchronize(s));
  if (flag == 0) return RSD_OK;                       // the wait did not run out: not what the probe is for
  KCU(cudaMemsetAsync((char*)scratch + 4096, 0, sizeof(flag), s));   // the scratch is usable again
  g_create_error = "a bounded wait inside the tensor-core GEMM expired";
  return RSD_ERR_TIMEOUT;
}

size_t rsd_k_attn_decode_scratch_bytes(int32_t B, int32_t H, int32_t hd, int32_t max_ctx) {
  return attn_decode_scratch_bytes(B, H, hd, max_ctx);
}

int rsd_k_attn_decode(const float* q, const void* kv_pool, const int32_t* page_table, const int32_t* ctx_len,
                      float* out, int32_t B, int32_t H, int32_t KV, int32_t hd, int32_t max_pages, int32_t dtype,
                      void* scratch, size_t scratch_bytes, void* cuda_stream) {
  if (!q || !kv_pool || !page_table || !ctx_len || !out || B < 1 || H < 1 || KV < 1 || H % KV || max_pages < 1)
    return RSD_ERR_ARG;
  if (hd != 64 && hd != 128) return RSD_ERR_UNSUPPORTED;
  if (scratch_bytes < attn_decode_scratch_bytes(B, H, hd, max_pages * kPageTokens) || !scratch) return RSD_ERR_ARG;
  if (dtype < 0 || dtype > 3) return RSD_ERR_ARG;
  KCU(launch_attn_decode(dtype, q, kv_pool, page_table, max_pages, nullptr, ctx_len, 0, out, nullptr, RSD_F32, B, H, KV, hd,
                         max_pages * kPageTokens, scratch, scratch_bytes, nullptr, (cudaStream_t)cuda_stream));
  return RSD_OK;
}

int rsd_k_attn_chunk(const float* q, const void* kv_pool, const int32_t* page_table, const int32_t* tok_row,
                     const int32_t* tok_pos, float* out, int32_t T, int32_t H, int32_t KV, int32_t hd, int32_t max_pages,
                     int32_t dtype, void* cuda_stream) {
  if (!q || !kv_pool || !page_table || !tok_row || !tok_pos || !out || T < 1 || H < 1 || KV < 1 || H % KV || max_pages < 1)
    return RSD_ERR_ARG;
  if (hd != 64 && hd != 128) return RSD_ERR_UNSUPPORTED;
  if (dtype < 0 || dtype > 3) return RSD_ERR_ARG;
  PassView p{nullptr, tok_row, tok_pos, T, nullptr};
  KvView kv{const_cast<void*>(kv_pool), page_table, max_pages};
  KCU(launch_attn_chunk(dtype, q, p, kv, out, nullptr, RSD_F32, H, KV, hd, (cudaStream_t)cuda_stream));
  return RSD_OK;
}

int rsd_k_gate_compact(const float* rewards, const uint8_t* live, float delta, uint8_t* accept, int32_t* rej_idx,
                       int32_t* n_rej, int32_t B, void* scratch, size_t scratch_bytes, void* cuda_stream) {
  if (!rewards || !live || !accept || !rej_idx || !n_rej || B < 1 || B > (1 << 24)) return RSD_ERR_ARG;
  if (!scratch || scratch_bytes < sizeof(int32_t) * (size_t)((B + 1023) / 1024)) return RSD_ERR_ARG;
  KCU(launch_gate_compact_large(rewards, live, delta, accept, rej_idx, n_rej, (int32_t*)scratch, B, (cudaStream_t)cuda_stream));
  return RSD_OK;
}

int rsd_k_rmsnorm(const float* x, const void* gain, void* out, int32_t T, int32_t d, float eps, int32_t dtype,
                  void* cuda_stream) {
  if (!x || !gain || !out || T < 0 || d < 4 || d % 4) return RSD_ERR_ARG;
  KCU(launch_rmsnorm(dtype, const_cast<float*>(x), gain, out, nullptr, T, d, eps, nullptr, nullptr, SplitSum(), (cudaStream_t)cuda_stream));
  return RSD_OK;
}

int rsd_k_rope(float* v, const int32_t* pos, int32_t T, int32_t n_heads, int32_t hd, float theta, void* cuda_stream) {
  if (!v || !pos || T < 0 || n_heads < 1 || hd < 2 || hd % 2) return RSD_ERR_ARG;
  KCU(launch_rope_only(v, pos, T, n_heads, hd, theta, (cudaStream_t)cuda_stream));
  return RSD_OK;
}

int rsd_k_swiglu(const float* gu, void* out, int32_t T, int32_t F, int32_t dtype, void* cuda_stream) {
  if (!gu || !out || T < 0 || F < 1) return RSD_ERR_ARG;
  KCU(launch_swiglu(dtype, gu, SplitSum(), out, nullptr, T, F, nullptr, (cudaStream_t)cuda_stream));
  return RSD_OK;
}

int rsd_k_gemm_gu(const void* Wgu, const void* x, const void* x_lo, void* act_hi, void* act_lo, int32_t M, int32_t F,
                  int32_t K, void* scratch, size_t scratch_bytes, void* cuda_stream) {
  if (!Wgu || !x || !act_hi || M < 0 || F < 1 || K < 1) return RSD_ERR_ARG;
  if ((x_lo == nullptr) != (act_lo == nullptr)) return RSD_ERR_ARG;      // plain operand in, plain operand out
  if (!gemm_gu_supported(RSD_BF16, M > 0 ? M : 1, F, K)) return RSD_ERR_UNSUPPORTED;
  if (x_lo == nullptr && M <= 128) return RSD_ERR_UNSUPPORTED;
  if (!scratch || scratch_bytes < gemm_scratch_bytes(M)) return RSD_ERR_ARG;
  KCU(launch_gemm_gu(Wgu, x, x_lo, act_hi, act_lo, M, F, K, scratch, scratch_bytes, nullptr, (cudaStream_t)cuda_stream));
  return RSD_OK;
}

int rsd_k_sample(const float* logits, int32_t B, int32_t V, int32_t v_limit, float temperature, uint64_t seed,
                 int32_t model_id, const int32_t* row, const int32_t* pos, int32_t* token, void* scratch,
                 size_t scratch_bytes, void* cuda_stream) {
  if (!logits || !row || !pos || !token || B < 1 || V < 1 || v_limit < 1 || v_limit > V || temperature < 0.f) return RSD_ERR_ARG;
  if (!scratch || scratch_bytes < sizeof(unsigned long long) * (size_t)B || ((uintptr_t)scratch & 7)) return RSD_ERR_ARG;
  KCU(cudaMemsetAsync(scratch, 0, sizeof(unsigned long long) * (size_t)B, (cudaStream_t)cuda_stream));
  SampleArgs a{logits, B, V, v_limit, temperature, seed, model_id, row, pos, token, nullptr, (unsigned long long*)scratch};
  KCU(launch_sample(a, (cudaStream_t)cuda_stream));
  return RSD_OK;
}

int rsd_k_philox(const uint32_t* ctr, const uint32_t* key, uint32_t* out, int32_t n, void* cuda_stream) {
  if (!ctr || !key || !out || n < 0) return RSD_ERR_ARG;
  KCU(launch_philox(ctr, key, out, n, (cudaStream_t)cuda_stream));
  return RSD_OK;
}

}  // extern "C"
