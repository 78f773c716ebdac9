// Host-side launchers of the RSD step-loop kernels.  Every launcher enqueues on `s` and returns the
// launch status; none synchronises or allocates.
#pragma once

#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

namespace rsd {

// Every launcher reports the kernels it enqueued; the total is what a caller can claim as its own
// GPU launches.
cudaError_t launched(int n_kernels);   // adds to the count and returns cudaGetLastError()
uint64_t launches_total();
void note_replayed_launches(uint64_t n);   // kernels run by replaying a captured graph

constexpr int kPageTokens = 16;   // tokens per KV page
constexpr int kMaxBatch = 1024;   // rows per context (one thread per row in the state kernels)

// A GEMM result that may still be spread over K-split partial sums: value = y (+) sum_s partials[s].
struct SplitSum {
  const float* partials = nullptr;
  int splits = 1;
};

// Per-row scale of a GEMM whose input rows were left un-normalised: row m of the result is multiplied by
// rsqrt(sum_c ssq[m * n_chunks + c] * inv_d + eps), i.e. the RMSNorm denominator of input row m whose
// squares were summed chunk by chunk by the producer of the input (reduce_norm).  ssq == nullptr: no scale.
struct RowScale {
  const float* ssq = nullptr;
  int n_chunks = 0;
  float inv_d = 0.f, eps = 0.f;
};

// A pass pushes T token slots through one model.  Slot t carries token tok_id[t] of row tok_row[t]
// at position tok_pos[t]; tok_row[t] < 0 marks an idle slot.  When n_active is non-null and reads
// 0 on the device the whole pass is skipped (every row of the decode phase has finished).
struct PassView {
  const int32_t* tok_id;
  const int32_t* tok_row;
  const int32_t* tok_pos;
  int T;
  const int32_t* n_active;
};

// Where one model keeps keys and values: per layer a slab of pages, each page holding the keys
// [KV][16 tokens][hd] followed by the values transposed [KV][hd][16 tokens].
struct KvView {
  void* pool_layer;            // slab of the current layer
  const int32_t* page_table;   // [rows, max_pages]
  int max_pages;
  int v_extra = 0;             // 1: every page carries two more blocks, the low halves of the keys and of
                               // the values (x = hi + lo, both fp16), laid out like the first two
};

cudaError_t launch_bf16_to_f16(const void* src, void* dst, size_t n, cudaStream_t s);
cudaError_t launch_embed(int dtype, const void* embed, PassView p, float* x, int d, cudaStream_t s);
// out[t] = rmsnorm(x[src ? src[t] : t]); rows with src[t] < 0 are skipped.
// out (and out_lo when given, bf16 only: the low half of a split-precision operand)
// pending (splits > 1): x[t] += sum of the partial sums [splits][T][d] first (x is written back).
cudaError_t launch_rmsnorm(int dtype, float* x, const void* gain, void* out, void* out_lo, int T, int d, float eps,
                           const int32_t* src, const int32_t* n_active, SplitSum pending, cudaStream_t s, bool out_f16 = false);
// x_lo (nullable, bf16 only): second operand matrix added to x (split-precision activations).
cudaError_t launch_gemm_simt(int dtype, const void* W, const void* x, const void* x_lo, float* y, int M, int N, int K,
                             int accumulate, const int32_t* n_active, cudaStream_t s);
// tcgen05 / TMEM / TMA GEMM (bf16): same contract as launch_gemm_simt; `scratch` holds split-K
// partial tiles and tile counters (the counters must be zero on entry and are left zero).
bool gemm_tc_supported(int dtype, int M, int N, int K);
size_t gemm_scratch_bytes(int M);
size_t gemm_scratch_bytes_any();
// deferred_splits (nullable): when given, a K-split launch leaves its partial sums in the scratch as
// [splits][M][N] (gemm_partials) for the consumer kernel to add up, and reports the split count;
// 1 means y holds the finished result.
cudaError_t launch_gemm_tc(const void* W, const void* x, const void* x_lo, float* y, int M, int N, int K, int accumulate,
                           void* scratch, size_t scratch_bytes, const int32_t* n_active, int* deferred_splits,
                           cudaStream_t s, RowScale rs = RowScale(), bool no_k_split = false);
const float* gemm_partials(const void* scratch);
// Failure-path probe of the tensor-core GEMM: one CTA whose copies are never issued; its bounded wait runs out and
// the error flag at byte 4096 of the scratch becomes -5.  W [128, 64] and x [16, 64] bf16, y [16, 128] fp32 (untouched).
cudaError_t launch_gemm_wait_probe(const void* W, const void* x, float* y, void* scratch, size_t scratch_bytes, cudaStream_t s);
// Gate/up projection with SwiGLU in the epilogue (bf16, split-precision operand): act_hi + act_lo [M, F] =
// silu(g) * u with [g | u] = rowscale * (x + x_lo)[M, K] * Wgu[2F, K]^T, Wgu rows = Wgate | Wup.  No K split and no
// fp32 gate/up array: the tile of a CTA is 64 gate rows and the 64 matching up rows.  F % 64 == 0.
bool gemm_gu_supported(int dtype, int M, int F, int K);
// Dense passes (more than 128 rows) on fp16 copies of the weights with one fp16 activation operand.
cudaError_t launch_gemm_f16_dense(const void* W16, const void* x16, float* y, int M, int N, int K, int accumulate,
                                  void* scratch, size_t scratch_bytes, cudaStream_t s);
cudaError_t launch_gemm_gu_f16_dense(const void* Wgu16, const void* x16, void* act16, int M, int F, int K, void* scratch,
                                     size_t scratch_bytes, cudaStream_t s);
cudaError_t launch_gemm_gu(const void* Wgu, const void* x, const void* x_lo, void* act_hi, void* act_lo, int M, int F, int K,
                           void* scratch, size_t scratch_bytes, const int32_t* n_active, cudaStream_t s, RowScale rs = RowScale());

// impl: 0 = by shape, 1 = SIMT split-K GEMV, 2 = tcgen05, 3 = tcgen05 without a K split.
cudaError_t launch_gemm(int dtype, const void* W, const void* x, const void* x_lo, float* y, int M, int N, int K,
                        int accumulate, int impl, void* scratch, size_t scratch_bytes, const int32_t* n_active,
                        int* deferred_splits, cudaStream_t s, RowScale rs = RowScale());
// x (+)= sum of the K-split partial sums [splits][M][d] (splits == 1: x is complete already); then the
// un-normalised RMSNorm operand of the next GEMM: hi + lo = x * gain as two bf16 arrays, and the sums of
// squares of x per 256-column chunk, ssq [M][ceil(d / 256)], for that GEMM's RowScale.
cudaError_t launch_reduce_norm(const float* partials, int splits, float* x, const void* gain, void* hi, void* lo,
                               float* ssq, int M, int d, const int32_t* n_active, cudaStream_t s);
inline int norm_chunks(int d) { return (d + 255) / 256; }
cudaError_t launch_rope_table(float2* table, int n_pos, int hd, float theta, cudaStream_t s);
// Splits qkv [T, (H+2KV)*hd] (fp32): rotated q -> q_out [T, H*hd] fp32; rotated k and v -> KV pages.
// kv_dtype: element type of the cache: 0 fp32, 1 bf16, 2 fp16.
// pending (splits > 1): qkv is the sum of the partial sums instead of the qkv array.
cudaError_t launch_rope_kv(int kv_dtype, const float* qkv, SplitSum pending, PassView p, float* q_out, KvView kv, const float2* rope,
                           int H, int KV, int hd, cudaStream_t s);
cudaError_t launch_rope_only(float* v, const int32_t* pos, int T, int n_heads, int hd, float theta, cudaStream_t s);
// Causal attention of every slot over positions [0, tok_pos] of its row, read from the pages.
cudaError_t launch_attn_generic(int kv_dtype, const float* q, PassView p, KvView kv, void* out, void* out_lo,
                                int out_dtype, int H, int KV, int hd, cudaStream_t s);
// Tensor-core versions of the above for 16-bit caches with H / KV <= 8 (falls back otherwise): the tcgen05 kernel for
// fp16 caches with head_dim 128 and at least 64 list entries (attn_chunk_tc.cu), else the mma.sync kernel.
// err (nullable): raised to -5 when a bounded wait of the tcgen05 kernel expires.
cudaError_t launch_attn_chunk(int kv_dtype, const float* q, PassView p, KvView kv, void* out, void* out_lo,
                              int out_dtype, int H, int KV, int hd, cudaStream_t s, int* err = nullptr);
bool attn_chunk_tc_supported(int kv_dtype, int H, int KV, int hd, int T);
cudaError_t launch_attn_chunk_tc(const float* q, PassView p, KvView kv, void* out, void* out_lo, int out_dtype, int H, int KV,
                                 int* err, cudaStream_t s);
cudaError_t launch_swiglu(int dtype, const float* gu, SplitSum pending, void* out, void* out_lo, int T, int F,
                          const int32_t* n_active, cudaStream_t s);

// Decode attention (one query per row) with split-KV partial results merged in a second pass.
size_t attn_decode_scratch_bytes(int B, int H, int hd, int max_ctx);
// Slot i attends positions [0, len_or_pos[i] + len_offset) of row slot_row[i] (slot i itself when
// slot_row is null); slot_row[i] < 0 skips the slot.  active_rows (0 = B): how many of the B slots are expected to
// carry a row; the context splits are chosen so that those fill the machine (idle slots cost nothing).
cudaError_t launch_attn_decode(int kv_dtype, const float* q, const void* pool_layer, const int32_t* page_table,
                               int max_pages, const int32_t* slot_row, const int32_t* len_or_pos, int len_offset,
                               void* out, void* out_lo, int out_dtype, int B, int H, int KV, int hd, int max_ctx, void* scratch,
                               size_t scratch_bytes, const int32_t* n_active, cudaStream_t s, int active_rows = 0);

// ---- persistent decode kernel: the whole layer stack of one decode iteration in one launch -------------
struct MegaShape {
  int n_layers, d, H, KV, hd, F;
  bool bf16;
  float eps;
};
// Everything the kernel needs for one model and one batch size; the arrays and buffers stay the caller's.
struct MegaBuild {
  MegaShape shape;
  int B, max_pages;
  const void* embed;
  const void* const *wqkv, *const *wo, *const *wgu, *const *wdown, *const *norm1, *const *norm2;
  char* kv_pool;
  size_t layer_stride;
  float* x;                                        // [B, d] residual stream
  void *h, *h_lo, *attn, *attn_lo, *act, *act_lo;  // bf16 operand pairs [B, d], [B, H*hd], [B, F]
  float* partials;                                 // K-split partial sums (mega_partials_floats)
  float* ssq;                                      // [B, d / 128] sums of squares of the residual stream
  float *part_o, *part_ml;                         // attention context-split partials [B, H, 16, hd] and [B, H, 16, 2]
  int32_t* sync_words;                             // 1024 ints, zero: grid barrier and split arrival counters
  int* err;                                        // raised to -5 when a bounded wait expires
  const float2* rope;
  const int32_t* page_table;
  unsigned long long* prof;                        // null, or 1024 words: CTA 0's global-timer stamps around every grid
                                                   // barrier of the last launch ([1023] = number of stamps)
};
bool mega_supported(const MegaShape& m, int B);
size_t mega_block_bytes(int n_layers);
size_t mega_partials_floats(const MegaShape& m, int B);
// Writes the kernel's parameter block (tensor maps, work plan, pointers) to dev_block (256-byte aligned).
cudaError_t mega_build(void* dev_block, const MegaBuild& a, cudaStream_t s);
// Runs embedding + all layers for the B slots of p (p.T == B).  On return x is the final residual stream,
// h / h_lo hold x * final_gain and ssq the sums of squares per 128-column chunk.
cudaError_t launch_decode_mega(const void* dev_block, int B, int kv_extended, PassView p, const void* final_gain,
                               cudaStream_t s);

struct SampleArgs {
  const float* logits;         // [n_slots, V]
  int n_slots, V, v_limit;
  float temperature;
  uint64_t seed;
  int model_id;
  const int32_t* slot_row;     // row id per slot (noise key); < 0 = idle slot
  const int32_t* slot_pos;     // position of the slot's input token; the new token sits at +1
  int32_t* token;              // [n_slots] out; null = leave the packed winners in `best`
  const int32_t* n_active;
  unsigned long long* best;    // [n_slots] scratch, zero on entry: packed (score, id) maxima
};
cudaError_t launch_sample(const SampleArgs& a, cudaStream_t s);
cudaError_t launch_philox(const uint32_t* ctr, const uint32_t* key, uint32_t* out, int n, cudaStream_t s);

// reward[row] = head(rmsnorm(x[last_idx[row] - t0])) for rows whose last token lies in [t0, t0+T).
cudaError_t launch_reward(int dtype, const float* x, const void* final_norm, const void* w_r, int head_kind,
                          const int32_t* last_idx, int t0, int T, int d, float eps, float* reward, int n_rows,
                          cudaStream_t s);

// block_cnt: scratch of ceil(B / 1024) ints.
cudaError_t launch_gate_compact_large(const float* rewards, const uint8_t* live, float delta, uint8_t* accept,
                                      int32_t* rej_idx, int32_t* n_rej, int32_t* block_cnt, int B, cudaStream_t s);

// ---- row state ------------------------------------------------------------------------------
struct RowState {
  int B, S, C, max_pages;      // rows in use, tokens per row, step cap, pages per row
  int prm_shared;              // 1: the PRM is a head on the draft's trunk and keeps no cache
  int32_t *z_len, *live, *n_steps, *tok;
  int32_t *kv_len[3], *n_pages[3], *page_table[3];
  int32_t* next_page;          // [3]
  int32_t pool_pages[3];
  int32_t *gen_len[2], *gen_tok[2], *sampled[2];   // 0 = draft phase, 1 = target phase
  int32_t *forced_tok[2], *forced_len[2];
  uint8_t* forced_accept;      // [B], 0/1 force, 255 free
  int32_t *gen_active, *n_active;
  float* rewards;
  uint8_t* accept;             // [B] this call: 0 took no draft step, 1 accepted, 2 rejected
  uint8_t* waiting;            // [B] 1: the row's draft step was rejected and the target has not written y_i yet
  int32_t *rej_idx, *n_rej;    // ascending list of the waiting rows and its length
  int32_t *n_live;             // live rows, counted by the gate
  int32_t *slot_row, *n_slots; // decode slots of the current phase
  int32_t *iter;               // iteration counter of the current decode phase
  int32_t *last_idx;           // [B] flat index of each row's last token in the current pass
  int32_t *prev_idx;           // [B] PRM scoring pass: flat index of the row's last COMMITTED token when the pass
                               // caches it (the row's previous step came from the target), else -1
  float* target_rewards;       // [B] reward of the row's latest target-written step (NaN until one was scored)
  int32_t *n_tok;              // tokens of the current pass
  int32_t *err;                // first error raised on the device
  int32_t *pass_tok_id, *pass_tok_row, *pass_tok_pos;  // flat pass lists
  int pass_capacity;
  // speculative decoding of rejected steps (sd_k proposals per round; 0 = off)
  int sd_k;
  int32_t* sd_stats;           // [5] rounds, proposed tokens, matched tokens (summed over rows since the last reset),
                               // index of the running round, index of the next proposal within it
  int32_t* sd_out_idx;         // [slots * sd_k] per verify slot: index of its token within the row's step, or -1
  int32_t* sd_forced_props;    // null, or [B][C][sd_k]: proposals imposed on the draft (parity hook), by row, round, index
  uint8_t* sd_forced_on;       // [B] 1: row b takes its proposals from sd_forced_props
};

enum ReserveMode { kReservePrefillDraft, kReservePrefillPrm, kReserveStepDraft, kReserveScorePrm, kReserveTarget };
enum PassMode { kPassIngestDraft, kPassScorePrm, kPassCatchupTarget };

struct LoopParams {
  int step_end_id, eos_id, step_end_mod, max_steps;
  int omega_kind;
  float omega_alpha;
  uint64_t seed;
};

// min_target_rows: the target serves the waiting rows only once that many wait, or every live row does
// (target_pass_due); it matters to the target modes alone.
cudaError_t launch_reserve_pages(const RowState& st, int which, ReserveMode mode, int min_target_rows, cudaStream_t s);
cudaError_t launch_build_pass(const RowState& st, int which, PassMode mode, int min_target_rows, cudaStream_t s);
inline __host__ __device__ bool target_pass_due(int n_waiting, int n_live, int min_target_rows) {
  const int want = min_target_rows < 1 ? 1 : min_target_rows;
  return n_waiting > 0 && n_waiting >= (want < n_live ? want : n_live);
}
cudaError_t launch_decode_begin(const RowState& st, int phase, cudaStream_t s);
// Merged PRM: one slot per row that took a draft step, carrying the step's last token at the draft's
// cursor (which stays where it is); n_active = number of such rows, last_idx[b] = b for them.
cudaError_t launch_score_prepare(const RowState& st, cudaStream_t s);
cudaError_t launch_decode_prepare(const RowState& st, int which, int n_slots, cudaStream_t s);
// best: packed winners left by launch_sample (cleared here).
cudaError_t launch_decode_update(const RowState& st, int which, int phase, unsigned long long* best,
                                 int n_slots, const LoopParams& lp, cudaStream_t s);
cudaError_t launch_gate(const RowState& st, float delta, const LoopParams& lp, cudaStream_t s);
// Speculative decoding of the waiting rows' steps (slot i <-> row slot_row[i], as in the target's decode phase).
// A round: sd_k draft iterations, each bracketed by propose_prepare (slot i feeds the token at the draft's cursor,
// while the round still has proposals to make for its row) and propose_update (the sampled token becomes proposal j:
// written after the fed token in the row's buffer, the draft's cursor moves on); then ONE target pass over
// n_slots * sd_k token slots laid out by verify_prepare (slot i * sd_k + j feeds the j-th token from the target's
// cursor on; unused slots idle), sampling at every slot, and accept: the target's choices are written one by one
// while the ones before equalled the proposals; both cursors end at the last written token.
cudaError_t launch_sd_propose_prepare(const RowState& st, int n_slots, cudaStream_t s);
cudaError_t launch_sd_propose_update(const RowState& st, unsigned long long* best, int n_slots, cudaStream_t s);
cudaError_t launch_sd_verify_prepare(const RowState& st, int n_slots, cudaStream_t s);
cudaError_t launch_sd_accept(const RowState& st, unsigned long long* best, int n_slots, const LoopParams& lp, cudaStream_t s);
// target_ran: the waiting rows' steps were written by the target in this call.  out_role[b]: bits 0-1 =
// accept code of this call, bit 2 = the row committed a target step; out_waiting[b]: still waiting;
// out_gen [2, B]: tokens the draft / the target generated for the row in this call.
cudaError_t launch_commit(const RowState& st, const LoopParams& lp, int target_ran, int32_t* out_tokens,
                          int32_t* out_len, float* out_rewards, uint8_t* out_accept, uint8_t* out_live,
                          uint8_t* out_role, uint8_t* out_waiting, int32_t* out_gen, cudaStream_t s);

}  // namespace rsd
