/* rsd.h -- C ABI of the B200 (sm_100a) library for the batched step loop of Reward-Guided
 * Speculative Decoding (RSD, arXiv 2501.19324, Algorithm 1).
 *
 * One context serves a batch of independent rows.  Per step and per live row the library
 *   (1) decodes a draft step  y^_i <- m(x, y_{1:i-1})            (Algorithm 1, "Generate draft step"),
 *   (2) scores it             r_i  <- r(y^_i | x, y_{1:i-1})     (Algorithm 1, "Compute reward"),
 *   (3) gates it              accept iff r_i >= delta            (Table 1, binary step; Algorithm 2),
 *   (4) re-decodes rejected rows with the target  y_i <- M(x, y_{1:i-1}),
 *   (5) commits y_i and stops rows on EOS / step budget          (Algorithm 1, "if s in y_i: break").
 * m, M and r are Llama-style decoder-only transformers; r carries a scalar head in place of
 * lm_head (Appendix B.3) whose sigmoid lies in [0,1] (Section 3, "Models").
 *
 * Conventions
 *   - Every function returns an int status: 0 = RSD_OK, negative = error.  Nothing throws, aborts
 *     or exits.  rsd_last_error() returns a library-owned description of the last failure.
 *   - "device" pointers are CUDA device pointers valid on the context's GPU; "host" pointers are
 *     ordinary host memory.  The library allocates NO device memory: weights, KV pools and the
 *     workspace are allocated by the caller and only borrowed until rsd_destroy().
 *   - All work is enqueued on the stream given to each call.  Calls that return host values
 *     synchronise that stream before returning.
 *   - One context must be used by one host thread at a time.
 *   - There is no CPU fallback: without a CUDA device every compute call fails with RSD_ERR_CUDA.
 */
#ifndef RSD_H
#define RSD_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct rsd_ctx rsd_ctx; /* opaque, owned by the library */

enum {
  RSD_OK = 0,
  RSD_ERR_ARG = -1,         /* bad argument / inconsistent shapes                         */
  RSD_ERR_STATE = -2,       /* call out of order (e.g. step before prefill)               */
  RSD_ERR_OOM_PAGES = -3,   /* a KV page pool or the workspace is too small; the rows' state is
                               unchanged, but only rsd_prefill / rsd_reset are valid afterwards */
  RSD_ERR_CUDA = -4,        /* a CUDA call failed; only rsd_destroy is valid afterwards   */
  RSD_ERR_TIMEOUT = -5,     /* a bounded device-side wait expired                         */
  RSD_ERR_UNSUPPORTED = -6  /* shape or option the kernels do not cover                   */
};

enum { RSD_F32 = 0, RSD_BF16 = 1, RSD_F16 = 2 /* KV caches only */, RSD_F16_EXT = 3 /* fp16 cache whose pages carry
       two more blocks with the low halves of keys and values; queries and softmax weights as hi + lo */ };
enum { RSD_DRAFT = 0, RSD_PRM = 1, RSD_TARGET = 2 };
enum { RSD_HEAD_LM = 0, RSD_HEAD_REWARD_SIGMOID = 1, RSD_HEAD_REWARD_RAW = 2 };

/* Weighting functions omega(r) of Table 1, used by the acceptance criterion of Algorithm 2. */
enum {
  RSD_OMEGA_CONSTANT = 0, /* omega = p               (p passed as delta)                   */
  RSD_OMEGA_STEP = 1,     /* omega = 1(r >= delta)   (the paper's default)                 */
  RSD_OMEGA_CLIP = 2,     /* omega = min(1, max(0, r))                                     */
  RSD_OMEGA_RATIO = 3,    /* omega = max(0, r / (1 + r))                                   */
  RSD_OMEGA_LOGISTIC = 4  /* omega = 1 / (1 + exp(-alpha (r - delta)))                     */
};

/* One transformer.  All pointers are DEVICE pointers, borrowed, read-only, row-major, of element
 * type `dtype` (fp32 or bfloat16), never copied or repacked by the library.
 *   y = W x with W stored [out_features, in_features].                                      */
typedef struct {
  int32_t n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ffn, vocab, dtype;
  float rope_theta, rms_eps;
  int32_t head_kind;          /* RSD_HEAD_*                                                  */
  const void* tok_embed;      /* [vocab, d_model]                                            */
  const void* final_norm;     /* [d_model]                                                   */
  const void* head;           /* [vocab, d_model] (lm_head) or [d_model] (reward projection) */
  const void* const* wqkv;    /* host array of n_layers device pointers:
                                 [(H + 2 KV) * head_dim, d_model], rows = Wq | Wk | Wv       */
  const void* const* wo;      /* per layer [d_model, H * head_dim]                           */
  const void* const* wgu;     /* per layer [2 * d_ffn, d_model], rows = Wgate | Wup          */
  const void* const* wdown;   /* per layer [d_model, d_ffn]                                  */
  const void* const* norm1;   /* per layer [d_model], RMSNorm gain before attention          */
  const void* const* norm2;   /* per layer [d_model], RMSNorm gain before the MLP            */
} rsd_model;

typedef struct {
  int32_t max_batch;          /* rows B, 1..1024                                             */
  int32_t max_seq_tokens;     /* per-row capacity of prompt + response                       */
  int32_t max_step_tokens;    /* cap on the tokens of one step                               */
  int32_t max_steps;          /* N of Algorithm 1: a row stops after this many steps         */
  int32_t page_tokens;        /* KV page size; must be 16                                    */
  int32_t step_end_id;        /* token that ends a step (the delimiter belongs to the step)  */
  int32_t eos_id;             /* EOS token s of Algorithm 1; -1 = none                       */
  int32_t step_end_mod;       /* 0 = off; m > 0: a token ends a step iff id % m == step_end_id % m */
  float temperature;          /* 0 = greedy; > 0 = Gumbel-max sampling at this temperature   */
  uint64_t seed;              /* Philox key of the sampling noise                            */
  int32_t omega_kind;         /* RSD_OMEGA_*; RSD_OMEGA_STEP reproduces the paper's default  */
  float omega_alpha;          /* alpha of RSD_OMEGA_LOGISTIC                                 */
  int32_t max_chunk_tokens;   /* tokens pushed through a model per multi-token pass; 0 = 4096 */
  int32_t debug_flags;        /* RSD_DEBUG_*                                                 */
  int32_t kv_extended;        /* bf16 models only; per model.  1: keys and values are cached as fp16 hi + lo
                                 pairs (twice the KV bytes) and queries / softmax weights enter the attention
                                 products as hi + lo pairs (attention accurate to ~2^-20).  2: plain fp16 keys
                                 and values, fp16 queries and softmax weights.  0 (default): by depth -- plain
                                 fp16 for models of up to 48 layers, the pairs for deeper ones, whose logits
                                 would otherwise leave the 3e-2 band around an exact reference (measured at 80
                                 layers: 5e-2 to 7e-2 with the plain cache, 2e-3 with the pairs)                  */
  int32_t prm_shares_draft;   /* 1: merged serving (Appendix B.3: the PRM is a projection layer on a language
                                 model's final layer; Section 4 on merging PRM and policy): the PRM is its
                                 final_norm and scalar head on the DRAFT's trunk.  r_i is read after one
                                 single-token pass of the draft over the last token of the draft step,
                                 from the draft's own cache; the PRM keeps no cache and its separate
                                 scoring pass disappears.  The prm descriptor must repeat the draft's
                                 dimensions and dtype; its layer arrays and kv_pool[RSD_PRM] may be NULL.
                                 Results equal those of a separate PRM whose trunk weights are the draft's */
  int32_t sd_tokens;          /* k, 0..16.  k > 0: RSD combined with speculative decoding (Section 4, discussion
                                 item on combining RSD with SD: a rejected step, which the target must write
                                 anyway, is rewritten by draft-then-verify decoding).  The target's step of a
                                 rejected row is then written in rounds: the draft proposes up to k tokens, the
                                 target evaluates its own choice at all k positions in ONE pass and the choices
                                 are written while every earlier one equalled the proposal (at least one, at
                                 most k tokens per round).  Sampling noise is keyed by (model, row, position), so
                                 the step is token for token the one plain target decoding writes; only the
                                 number of target passes changes.  The workspace grows with k (logits of k
                                 positions per row)                                                           */
  /* caller-allocated device memory, sizes as reported by rsd_query_sizes (or larger)        */
  void* kv_pool[3];           /* RSD_DRAFT / RSD_PRM / RSD_TARGET                            */
  size_t kv_bytes[3];
  void* workspace;
  size_t workspace_bytes;
} rsd_config;

enum {
  RSD_DEBUG_KEEP_LOGITS = 1, /* keep every decode iteration's logits for rsd_debug_get_logits      */
  RSD_DEBUG_NO_GRAPHS = 2,   /* launch decode iterations kernel by kernel instead of as CUDA graphs */
  RSD_DEBUG_PERSISTENT_DECODE = 4, /* alternative decode path for bf16 models at up to 64 rows: the layers of a
                                decode iteration run as ONE persistent kernel (one CTA per SM, grid barriers
                                between the phases) instead of kernel by kernel.  Same results; slower than
                                the default on the measured shapes, kept for study                    */
  RSD_DEBUG_MEGA_PROFILE = 8, /* the persistent decode kernel records global-timer stamps around its grid
                                barriers (rsd_debug_mega_profile)                                     */
  RSD_DEBUG_NO_F16_DENSE = 16 /* keep bf16 hi + lo operand pairs in the passes of more than 128 tokens too
                                (by default a bf16 model that uses the pairs gets fp16 copies of its layer
                                matrices in the workspace, up to 20 GB a model, and those passes run on them
                                with one fp16 activation operand: half the tensor-core work)             */
};

/* Fills cfg->kv_bytes[] (enough pages for max_batch rows of max_seq_tokens) and
 * cfg->workspace_bytes for these three models.  Host only.  RSD_ERR_ARG on bad shapes.
 * The workspace includes room for fp16 copies of the layer matrices of the bf16 models whose
 * passes of more than 128 tokens run on them (see RSD_DEBUG_NO_F16_DENSE): up to the size of
 * the model's layers again, for models of up to 20 GB.  rsd_load_models fills the copies; the
 * caller's weights are only ever read.                                                        */
int rsd_query_sizes(const rsd_model* draft, const rsd_model* prm, const rsd_model* target, rsd_config* cfg);

/* Creates a context on the current CUDA device from a filled rsd_config.  The KV pools and the
 * workspace must stay alive and untouched by the caller until rsd_destroy.                   */
int rsd_create(const rsd_config* cfg, rsd_ctx** out);

/* rsd_load_models(draft, prm, target): records the three borrowed weight sets, validates shapes
 * (GQA divisibility, head_dim 64 or 128, K dimensions a multiple of the vector width) and lays
 * out the workspace.  Sampling is restricted to ids below the smallest of the three vocabularies
 * so every token is valid for every embedding.  Once per context: a second successful load is
 * refused with RSD_ERR_STATE (the captured decode graphs keep the first models' pointers); use a
 * new context for other models.                                                              */
int rsd_load_models(rsd_ctx*, const rsd_model* draft, const rsd_model* prm, const rsd_model* target);

/* rsd_prefill(prompts): starts B rows from ragged prompts (z_1 = x).  `tokens` is a HOST array of
 * offsets[B] ids, row b owning [offsets[b], offsets[b+1]).  The draft caches each prompt without
 * its last token, the PRM the whole prompt, the target nothing (it catches up when a row is first
 * rejected).  Drops any rows of an earlier call.                                             */
int rsd_prefill(rsd_ctx*, const int32_t* tokens, const int32_t* offsets, int32_t B, void* cuda_stream);

/* rsd_step(delta): one pass of the loop body of Algorithm 1 over all rows.  Outputs are HOST
 * arrays (any may be NULL): step_tokens [B, max_step_tokens] (y_i, zero padded), step_len [B],
 * rewards [B] (r_i of the draft step), accept [B] (1 = draft step kept), live [B] (row continues).
 * Rows that were already stopped report step_len 0, reward 0, accept 0.  Synchronises.       */
int rsd_step(rsd_ctx*, float delta, void* cuda_stream, int32_t* step_tokens, int32_t* step_len,
             float* rewards, uint8_t* accept, uint8_t* live);

/* rsd_step with queued rejections.  Rows are independent in Algorithm 1, and a batched target pass
 * reads all of M's weights however few rows were rejected (the FLOPs of Section 3.3 count tokens, the
 * clock counts weight passes).  Here a row whose draft step is rejected WAITS -- its draft step is
 * dropped from the draft and PRM caches, it takes no part in later draft phases -- while accepted
 * rows go on; in the call in which min_target_rows rows wait (or every live row does) the target
 * catches up on and writes y_i for all waiting rows, in ascending row order.  Every row's own
 * sequence of steps is the one rsd_step would give it; min_target_rows = 1 is rsd_step.
 * Outputs as rsd_step, per call: a row that waits reports step_len 0, accept 0, live 1 and
 * waiting 1 (HOST [B], may be NULL); rewards[b] is the reward of row b's latest draft step; a row
 * served by the target reports its step with accept 0 in the call of that pass.
 * RSD_ERR_ARG when min_target_rows < 1.                                                        */
int rsd_step_queued(rsd_ctx*, float delta, int32_t min_target_rows, void* cuda_stream, int32_t* step_tokens,
                    int32_t* step_len, float* rewards, uint8_t* accept, uint8_t* live, uint8_t* waiting);

/* rsd_step / rsd_step_queued (min_target_rows = 1 is rsd_step) with DEVICE output arrays (any may be NULL), filled
 * on the stream in order with the call's kernels: for callers that keep the step's results on the GPU.  The call
 * still synchronises the stream while it runs (the host sizes the ragged passes from device counters).        */
int rsd_step_device(rsd_ctx*, float delta, int32_t min_target_rows, void* cuda_stream, int32_t* step_tokens,
                    int32_t* step_len, float* rewards, uint8_t* accept, uint8_t* live, uint8_t* waiting);

/* Reward of each row's latest step that the TARGET wrote (HOST out [B]; NaN for a row without one, or whose step has
 * not been scored yet).  Algorithm 1 gates on the draft step's reward only; the paper's comparison of draft-step and
 * target-step rewards inside RSD (Section 2, figure on reward distributions) reads this value too.  It costs
 * nothing: the PRM has to cache a target-written step before it scores the row's next draft step, and the reward
 * head is read at that step's last token on the way, so the value appears one call after the step was written.
 * Not available with prm_shares_draft (no PRM pass).  Synchronises the device.                                 */
int rsd_get_target_step_rewards(rsd_ctx*, float* out);

/* Counters of the work done since rsd_prefill / rsd_reset.  Index 0 draft, 1 PRM, 2 target.
 * flops_paper follows Section 3.3: 2N per inference token of an N-parameter model (all
 * parameters, embedding and head included), counting every token the draft or the target
 * generated (discarded draft steps too) and every token the PRM processed.  flops_all_tokens
 * bills 2N for every token pushed through any model, prompts and catch-up included.         */
typedef struct {
  uint64_t gen_tokens[3];
  uint64_t ingest_tokens[3];
  uint64_t score_tokens;
  uint64_t steps, accepted_steps, rejected_steps, discarded_draft_tokens;
  double flops_paper, flops_all_tokens;
  /* speculative decoding of rejected steps (sd_tokens > 0): rounds summed over rows, tokens the draft proposed,
     proposals the target's choice equalled, positions the target evaluated.  flops_paper then bills the draft
     its proposals as well and the target every evaluated position instead of every generated token.          */
  uint64_t sd_rounds, sd_proposed, sd_matched, sd_verified;
} rsd_counters;
int rsd_flops_counters(rsd_ctx*, rsd_counters* out);

int rsd_reset(rsd_ctx*);    /* drops rows and returns every KV page; keeps the models        */
int rsd_destroy(rsd_ctx*);
const char* rsd_last_error(const rsd_ctx*); /* ctx may be NULL: error of the last failed create */

/* ---- parity hooks ------------------------------------------------------------------------- */

/* Teacher forcing for the NEXT rsd_step only: tokens [B, max_step_tokens] and len [B] (HOST) replace
 * what model `which` (RSD_DRAFT or RSD_TARGET) samples; len[b] = 0 leaves row b free.  The sampled
 * ids remain readable through rsd_debug_get_sampled.  accept [B] (HOST, may be NULL; 0/1, other
 * values = do not force) overrides the gate when which == RSD_PRM (tokens/len ignored).      */
int rsd_debug_force(rsd_ctx*, int which, const int32_t* tokens, const int32_t* len, const uint8_t* accept);

/* Speculative decoding of rejected steps, for the NEXT step only: props [B, max_step_tokens, sd_tokens] (HOST)
 * replaces what the draft proposes -- entry (b, r, j) is proposal j of row b's r-th round -- for rows with
 * on[b] != 0 (HOST [B]).  Needs sd_tokens > 0 and RSD_DEBUG_KEEP_LOGITS, else RSD_ERR_STATE.                 */
int rsd_debug_force_sd(rsd_ctx*, const int32_t* props, const uint8_t* on);

/* Logits of the last rsd_step's decode iterations of model `which`, when RSD_DEBUG_KEEP_LOGITS
 * is set: out is a HOST array [B, max_step_tokens, vocab(which)] (row b, iteration j).        */
int rsd_debug_get_logits(rsd_ctx*, int which, float* out);
/* Ids sampled (before forcing) in the last rsd_step: HOST out [B, max_step_tokens].           */
int rsd_debug_get_sampled(rsd_ctx*, int which, int32_t* out);

/* Integer state, HOST outputs (any may be NULL): z_len [B], kv_len [3, B], n_pages [3, B],
 * page_table [3, B, max_pages] with max_pages = ceil(max_seq_tokens / page_tokens), next_page [3],
 * rej_idx [B] (ascending rows that waited for the target after the last step's gate -- with rsd_step
 * the rows rejected in that step -- first *n_rej entries valid).                                */
int rsd_debug_get_state(rsd_ctx*, int32_t* z_len, int32_t* kv_len, int32_t* n_pages, int32_t* page_table,
                        int32_t* next_page, int32_t* rej_idx, int32_t* n_rej);

/* Timing of the weight GEMMs inside rsd_prefill / rsd_step with CUDA events on the caller's stream:
 * every `stride`-th GEMM launch is bracketed by two events (stride 0 switches timing off; at most
 * 8192 launches are held between two synchronisation points of a step).  Each call first returns
 * what was gathered since the previous call -- summed device time in ms, summed algorithmic bytes
 * (weights + input read once, output written once, or read and written when accumulated into) and
 * the number of timed launches -- then clears the totals and installs the new stride.  HOST outputs,
 * any may be NULL.  Synchronises the device.                                                   */
int rsd_debug_gemm_timing(rsd_ctx*, int32_t stride, double* ms, double* bytes, uint64_t* launches);
/* The dense launches (more than 128 rows of x: prefill, PRM scoring, sync and catch-up passes) among the launches
 * timed by rsd_debug_gemm_timing since the previous call of THIS function, in two classes -- index 0: plain bf16
 * operand, index 1: hi + lo operand pair (twice the tensor-core work per algorithmic flop) --: summed device time in
 * ms, summed algorithmic flops 2 M N K and the number of launches; the totals are cleared.  Call it before the
 * rsd_debug_gemm_timing call that closes the period.  HOST arrays of two elements, any may be NULL.               */
int rsd_debug_gemm_timing_dense(rsd_ctx*, double* ms, double* flops, uint64_t* launches);
/* Device time of the phases of rsd_step, from CUDA events on the caller's stream, summed over the
 * steps since the previous call: out[7] (HOST, may be NULL) = draft sync, draft decode, PRM scoring,
 * gate + routing, target catch-up, target decode, commit, in ms.  Each call returns and clears the
 * sums, then switches the timing on (enable != 0) or off.                                       */
int rsd_debug_phase_ms(rsd_ctx*, int32_t enable, double* out);
/* Number of kernels this library has enqueued in this process so far.                          */
uint64_t rsd_debug_launch_count(void);
/* Timeline of the last launch of the persistent decode kernel of model `which` (RSD_DRAFT or RSD_TARGET),
 * recorded by its first CTA when RSD_DEBUG_MEGA_PROFILE is set: stamps[0] = kernel start, then for every
 * grid barrier the global-timer value (ns) when the CTA's phase work was done and when the barrier let it
 * go, in phase order (embedding; per layer: qkv, attention, wo, residual + norm, gate/up + SwiGLU, down,
 * residual + norm), last the kernel's end.  stamps (HOST, `capacity` words) receives *n_out values.
 * Synchronises the device.  RSD_ERR_STATE when the flag was not set.                            */
int rsd_debug_mega_profile(rsd_ctx*, int which, uint64_t* stamps, int32_t capacity, int32_t* n_out);

/* ---- single kernels (sweeps and unit parity); all pointers DEVICE unless noted ------------ */

/* y[M, N] (fp32) = (accumulate ? y : 0) + (x + x_lo)[M, K] * W[N, K]^T, W and x of element type `dtype`.
 * x_lo (bf16 only, may be NULL) is the low half of a split-precision activation: x = bf16(a),
 * x_lo = bf16(a - x), both multiplied on the tensor cores and added, so `a` enters with ~16 bits.
 * impl: 0 = pick by shape, 1 = split-K SIMT GEMV path, 2 = tcgen05/TMEM/TMA path (bf16 only,
 * K % 8 == 0, 16-byte aligned rows), 3 = the same with one CTA per output tile (no split along K),
 * 4 = the dense form of the passes of more than 128 tokens: W and x hold FP16 (dtype still RSD_BF16: the element
 * size), x_lo NULL, M > 128, one fp16 operand per activation on the persistent tcgen05 kernel.  `scratch` (scratch_bytes from rsd_k_gemm_scratch_bytes)
 * holds split-K partial sums and tile counters; its first 4 KiB + 256 B must be zero before the
 * first call; the counters are left zero by every call and the int at byte 4096 becomes non-zero
 * if a bounded device-side wait of the tcgen05 path expired (RSD_ERR_TIMEOUT condition).                                                      */
int rsd_k_gemm(const void* W, const void* x, const void* x_lo, float* y, int32_t M, int32_t N, int32_t K, int32_t dtype,
               int32_t accumulate, int32_t impl, void* scratch, size_t scratch_bytes, void* cuda_stream);
size_t rsd_k_gemm_scratch_bytes(int32_t M, int32_t N, int32_t K);
/* Failure path of the tcgen05 GEMM without a fault: launches one CTA of the kernel in a mode in which its copy
 * engine issues nothing, so the first pipeline stage never fills, the MMA warp's bounded wait (cut to a few thousand
 * polls here) runs out, the CTA raises the error flag, releases its other warps, frees its tensor memory and
 * returns with nothing in flight.  Returns RSD_ERR_TIMEOUT (the expected outcome; rsd_last_error(NULL) names the
 * wait) after clearing the flag, so the same scratch serves rsd_k_gemm afterwards.  W [128, 64] and x [16, 64]
 * bf16 and y [16, 128] fp32 are DEVICE buffers that are mapped but neither read nor written; scratch as for
 * rsd_k_gemm with M = 16.  Synchronises the stream.                                                          */
int rsd_debug_gemm_wait_probe(const void* W, const void* x, float* y, void* scratch, size_t scratch_bytes,
                              void* cuda_stream);

/* Paged-KV grouped-query decode attention: one query per row.  q [B, H, hd] fp32; kv pool of pages,
 * each page = keys [KV][16 tokens][hd] followed by values transposed [KV][hd][16 tokens], of
 * `dtype` (RSD_F32, RSD_BF16, RSD_F16 or RSD_F16_EXT, which adds the blocks keys_lo and values_lo after the
 * first two); page_table [B, max_pages]; ctx_len [B] (number of cached
 * positions attended; rows with ctx_len < 1 are skipped); out [B, H, hd] fp32.  16-bit caches with
 * H / KV <= 8 take the tensor-core split-context kernel, everything else a generic kernel.  The
 * step loop keeps fp16 caches for bf16 models (same bytes, three more mantissa bits).                                   */
int rsd_k_attn_decode(const float* q, const void* kv_pool, const int32_t* page_table, const int32_t* ctx_len,
                      float* out, int32_t B, int32_t H, int32_t KV, int32_t hd, int32_t max_pages,
                      int32_t dtype, void* scratch, size_t scratch_bytes, void* cuda_stream);
size_t rsd_k_attn_decode_scratch_bytes(int32_t B, int32_t H, int32_t hd, int32_t max_ctx);

/* Causal attention of a ragged list of T new tokens over the same paged cache (prefill, PRM step scoring,
 * catch-up): entry t belongs to row tok_row[t] (entries sorted by row, then position; tok_row < 0 is
 * skipped) and attends positions [0, tok_pos[t]] of that row, whose keys and values (those of the new
 * tokens included) are already in the pages.  q and out are [T, H, hd] fp32.  fp16 caches with
 * hd = 128, H / KV <= 8 and T >= 64 take the tcgen05 kernel (operands and accumulators in tensor
 * memory, pages fetched by TMA: kv_pool must be 16-byte aligned), other 16-bit caches with
 * H / KV <= 8 the mma.sync kernel, everything else the generic one.  (Inside rsd_prefill / rsd_step
 * a bounded device-side wait of the tcgen05 kernel that runs out makes the call return
 * RSD_ERR_TIMEOUT; this stand-alone entry has no error word to report it in.)                      */
int rsd_k_attn_chunk(const float* q, const void* kv_pool, const int32_t* page_table, const int32_t* tok_row,
                     const int32_t* tok_pos, float* out, int32_t T, int32_t H, int32_t KV, int32_t hd,
                     int32_t max_pages, int32_t dtype, void* cuda_stream);

/* Gate + compaction (Table 1 binary step; Algorithm 1 else-branch batched over rows):
 * accept[b] = live[b] && rewards[b] >= delta; rej_idx [B] receives the ascending list of live
 * rejected rows, *n_rej (device) their count.  B up to 2^24.  scratch: 4 * ceil(B / 1024) bytes. */
int rsd_k_gate_compact(const float* rewards, const uint8_t* live, float delta, uint8_t* accept,
                       int32_t* rej_idx, int32_t* n_rej, int32_t B, void* scratch, size_t scratch_bytes,
                       void* cuda_stream);

/* The same gate + compaction for callers that cannot allocate device memory -- a serving process
 * whose GPU memory was handed out once at start-up, a tenant held to a fixed memory budget, code in
 * a section where an allocation (which may stall the device) is not allowed.  (The paper has no
 * counterpart to this call: it is a packaging variant of rsd_k_gate_compact, not part of the method.)
 * Its scratch is a fixed 4 KiB array inside the library's device image, present on every GPU that
 * loads the library until the process ends, so the caller passes only inputs and outputs and the
 * call performs no cudaMalloc / cudaFree.  B must lie in 1..RSD_GATE_STATIC_MAX_ROWS, otherwise
 * RSD_ERR_ARG is returned and rsd_k_gate_compact_static_error() says why.
 *   - The first call on each device looks up the array's device address (with that device
 *     current); make that first call before starting any stream capture.
 *   - All calls share the one array, which keeps the previous call's contents; none of it needs
 *     clearing between calls (every counter a call reads is written by that call first).  Two
 *     calls that overlap on the GPU -- different streams without ordering, or different host
 *     threads -- race on it and give wrong lists: order them on one stream or with events.
 *   - Pointers are DEVICE pointers as for rsd_k_gate_compact; results are identical to it.       */
#define RSD_GATE_STATIC_MAX_ROWS (1 << 20)
int rsd_k_gate_compact_static(const float* rewards, const uint8_t* live, float delta, uint8_t* accept,
                              int32_t* rej_idx, int32_t* n_rej, int32_t B, void* cuda_stream);
const char* rsd_k_gate_compact_static_error(void); /* text of its last failure (any thread's), copied for
                                                      the calling thread: valid until that thread's next call */

/* out[t, :] = x[t, :] * gain / sqrt(mean(x^2) + eps), x fp32 [T, d], out of element type `dtype`. */
int rsd_k_rmsnorm(const float* x, const void* gain, void* out, int32_t T, int32_t d, float eps,
                  int32_t dtype, void* cuda_stream);
/* Rotary embedding in place on v [T, n_heads, hd] fp32 at positions pos [T]: pairs (i, i + hd/2). */
int rsd_k_rope(float* v, const int32_t* pos, int32_t T, int32_t n_heads, int32_t hd, float theta,
               void* cuda_stream);
/* out[t, f] = silu(gu[t, f]) * gu[t, F + f]; gu fp32 [T, 2F], out of element type `dtype`.     */
int rsd_k_swiglu(const float* gu, void* out, int32_t T, int32_t F, int32_t dtype, void* cuda_stream);
/* Gate/up projection of the SwiGLU MLP with the nonlinearity in the GEMM epilogue (tcgen05 path, bf16):
 * act[m, f] = silu(g[m, f]) * u[m, f], [g | u] = (x + x_lo)[M, K] * Wgu[2F, K]^T with Wgu rows = Wgate | Wup,
 * written as the split-precision pair act_hi = bf16(act), act_lo = bf16(act - act_hi), both [M, F].
 * F % 64 == 0, K % 8 == 0, 16-byte aligned rows.  x_lo and act_lo may both be NULL when M > 128: the operand is
 * then plain bf16 and only act_hi = bf16(act) is written (half the tensor-core work).  `scratch`: at least
 * rsd_k_gemm_scratch_bytes(M, 2F, K) bytes, zero on first use (it carries the kernel's error flag).
 * RSD_ERR_UNSUPPORTED for other shapes.                                                         */
int rsd_k_gemm_gu(const void* Wgu, const void* x, const void* x_lo, void* act_hi, void* act_lo, int32_t M, int32_t F,
                  int32_t K, void* scratch, size_t scratch_bytes, void* cuda_stream);
/* token[b] = argmax over v < v_limit of logits[b, v] / T + g, g = -log(-log u) with u the Philox
 * uniform of (seed; counter = (v / 4, pos[b] + 1, row[b], model_id), word v % 4), or the plain
 * argmax when temperature == 0; ties to the lowest id.  pos[b] is the position of the token fed to
 * the model, the sampled token sits at pos[b] + 1.  row[b] < 0 skips slot b.  logits fp32 [B, V].
 * scratch: 8 * B bytes, 8-byte aligned (per-slot packed maxima the vocabulary chunks fold into).  */
int rsd_k_sample(const float* logits, int32_t B, int32_t V, int32_t v_limit, float temperature,
                 uint64_t seed, int32_t model_id, const int32_t* row, const int32_t* pos, int32_t* token,
                 void* scratch, size_t scratch_bytes, void* cuda_stream);
/* Philox4x32-10 blocks: out[i] = philox(ctr[i], key), ctr [n, 4], key [2], out [n, 4] (uint32). */
int rsd_k_philox(const uint32_t* ctr, const uint32_t* key, uint32_t* out, int32_t n, void* cuda_stream);

#ifdef __cplusplus
}
#endif
#endif /* RSD_H */
