/* TEST INFRASTRUCTURE -- CPU oracle for the Reward-Guided Speculative Decoding step loop.
 *
 * Plain, slow, obviously-correct C.  Weights arrive as fp32 arrays (for 16-bit configurations
 * they hold the bfloat16-rounded values, which fp32 represents exactly); every activation,
 * accumulation, softmax and rotary angle is computed in fp64.  Nothing here is blocked, fused or
 * reordered beyond what the definitions state.  OpenMP only spreads independent outputs over
 * host cores.  This file shares no code with the CUDA library and must never be linked,
 * imported or executed by it: it exists so tests and the benchmark's CPU leg can check the GPU.
 *
 * What is implemented, with the passage of the paper each part follows:
 *   - the three "Llama-style" decoder-only transformers m (draft), M (target) and r (PRM) of
 *     Section 2 "Notations" / Section 3 "Models": RMSNorm, rotary embeddings, grouped-query
 *     causal attention, SwiGLU MLP, untied lm_head;
 *   - the PRM head of Appendix B.3 ("Model Merge": a projection layer on top of the last
 *     transformer layer mapping the hidden state to a scalar, in place of lm_head), squashed by a
 *     sigmoid so the score lies in [0,1] as Section 3 "Models" states;
 *   - the weighting functions omega(r) of Table 1 and the acceptance criterion of Algorithm 2;
 *   - token sampling: greedy (temperature 0, Section 3 "Default Setting") and Gumbel-max at a
 *     temperature, with noise from Philox4x32-10 (Salmon et al., SC'11).
 * The step loop of Algorithm 1 itself is written in Python (rsd_loop.py) on top of these calls.
 *
 * Parity pins live in tests/test_oracle_*.py: a third-party Llama implementation, library
 * attention / normalisation routines, closed forms and invariants.  No function here is unpinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef struct {
  int32_t n_layers, d_model, n_heads, n_kv_heads, head_dim, d_ffn, vocab, head_kind;
  double rope_theta, rms_eps;
} orc_shape;

typedef struct {
  const float *wq, *wk, *wv, *wo, *wgate, *wup, *wdown, *norm1, *norm2;
} orc_layer;

/* ---------------------------------------------------------------- elementary pieces -------- */

/* RMSNorm: out_i = x_i * g_i / sqrt(mean(x^2) + eps). */
void orc_rmsnorm(const double* x, const float* g, int d, double eps, double* out) {
  double ss = 0.0;
  for (int i = 0; i < d; ++i) ss += x[i] * x[i];
  double inv = 1.0 / sqrt(ss / (double)d + eps);
  for (int i = 0; i < d; ++i) out[i] = x[i] * inv * (double)g[i];
}

/* Y[t, r] = sum_c W[r, c] * X[t, c]   (W row-major [rows, cols], fp32 values, fp64 sums). */
void orc_matmul(const float* W, int rows, int cols, const double* X, int T, double* Y) {
#pragma omp parallel for schedule(static)
  for (int r = 0; r < rows; ++r) {
    const float* w = W + (size_t)r * cols;
    for (int t = 0; t < T; ++t) {
      const double* x = X + (size_t)t * cols;
      double acc = 0.0;
      for (int c = 0; c < cols; ++c) acc += (double)w[c] * x[c];
      Y[(size_t)t * rows + r] = acc;
    }
  }
}

/* Rotary embedding of one head vector at position pos: pairs (i, i + hd/2) are rotated by
 * angle pos * theta^(-2i/hd). */
void orc_rope(double* v, int head_dim, int pos, double theta) {
  int half = head_dim / 2;
  for (int i = 0; i < half; ++i) {
    double ang = (double)pos * pow(theta, -2.0 * (double)i / (double)head_dim);
    double c = cos(ang), s = sin(ang);
    double a = v[i], b = v[i + half];
    v[i] = a * c - b * s;
    v[i + half] = b * c + a * s;
  }
}

void orc_embed(const float* tok_embed, const int32_t* tokens, int T, int d, double* x) {
  for (int t = 0; t < T; ++t)
    for (int i = 0; i < d; ++i) x[(size_t)t * d + i] = (double)tok_embed[(size_t)tokens[t] * d + i];
}

/* ---------------------------------------------------------------- one decoder layer -------- */

/* Runs T new tokens, sitting at positions start_pos .. start_pos+T-1 of one sequence, through one
 * layer.  x [T, d] is the residual stream, updated in place.  kcache / vcache are
 * [capacity, n_kv_heads*head_dim] fp64 arrays of this layer for this sequence; entries below
 * start_pos must already hold the keys (after RoPE) and values of the earlier positions, and the
 * entries of the new positions are written here.  Query head j reads KV head j / (H / KV). */
void orc_layer_forward(const orc_shape* s, const orc_layer* L, double* x, int T, int start_pos,
                       double* kcache, double* vcache) {
  const int d = s->d_model, H = s->n_heads, KV = s->n_kv_heads, hd = s->head_dim, F = s->d_ffn;
  const int qd = H * hd, kvd = KV * hd, group = H / KV;
  double* h = (double*)malloc(sizeof(double) * (size_t)T * d);
  double* q = (double*)malloc(sizeof(double) * (size_t)T * qd);
  double* k = (double*)malloc(sizeof(double) * (size_t)T * kvd);
  double* v = (double*)malloc(sizeof(double) * (size_t)T * kvd);
  double* att = (double*)malloc(sizeof(double) * (size_t)T * qd);
  double* proj = (double*)malloc(sizeof(double) * (size_t)T * d);
  double* gate = (double*)malloc(sizeof(double) * (size_t)T * F);
  double* up = (double*)malloc(sizeof(double) * (size_t)T * F);

  for (int t = 0; t < T; ++t) orc_rmsnorm(x + (size_t)t * d, L->norm1, d, s->rms_eps, h + (size_t)t * d);
  orc_matmul(L->wq, qd, d, h, T, q);
  orc_matmul(L->wk, kvd, d, h, T, k);
  orc_matmul(L->wv, kvd, d, h, T, v);
  for (int t = 0; t < T; ++t) {
    int pos = start_pos + t;
    for (int j = 0; j < H; ++j) orc_rope(q + (size_t)t * qd + (size_t)j * hd, hd, pos, s->rope_theta);
    for (int j = 0; j < KV; ++j) orc_rope(k + (size_t)t * kvd + (size_t)j * hd, hd, pos, s->rope_theta);
    memcpy(kcache + (size_t)pos * kvd, k + (size_t)t * kvd, sizeof(double) * kvd);
    memcpy(vcache + (size_t)pos * kvd, v + (size_t)t * kvd, sizeof(double) * kvd);
  }
  const double inv_sqrt = 1.0 / sqrt((double)hd);
#pragma omp parallel for collapse(2) schedule(dynamic)
  for (int t = 0; t < T; ++t) {
    for (int j = 0; j < H; ++j) {
      int pos = start_pos + t, g = j / group;
      const double* qv = q + (size_t)t * qd + (size_t)j * hd;
      double* sc = (double*)malloc(sizeof(double) * (size_t)(pos + 1));
      double mx = -INFINITY;
      for (int p = 0; p <= pos; ++p) {
        const double* kv = kcache + (size_t)p * kvd + (size_t)g * hd;
        double a = 0.0;
        for (int i = 0; i < hd; ++i) a += qv[i] * kv[i];
        sc[p] = a * inv_sqrt;
        if (sc[p] > mx) mx = sc[p];
      }
      double den = 0.0;
      for (int p = 0; p <= pos; ++p) { sc[p] = exp(sc[p] - mx); den += sc[p]; }
      double* o = att + (size_t)t * qd + (size_t)j * hd;
      for (int i = 0; i < hd; ++i) o[i] = 0.0;
      for (int p = 0; p <= pos; ++p) {
        const double* vv = vcache + (size_t)p * kvd + (size_t)g * hd;
        double w = sc[p] / den;
        for (int i = 0; i < hd; ++i) o[i] += w * vv[i];
      }
      free(sc);
    }
  }
  orc_matmul(L->wo, d, qd, att, T, proj);
  for (size_t i = 0; i < (size_t)T * d; ++i) x[i] += proj[i];

  for (int t = 0; t < T; ++t) orc_rmsnorm(x + (size_t)t * d, L->norm2, d, s->rms_eps, h + (size_t)t * d);
  orc_matmul(L->wgate, F, d, h, T, gate);
  orc_matmul(L->wup, F, d, h, T, up);
  for (size_t i = 0; i < (size_t)T * F; ++i) {
    double a = gate[i];
    gate[i] = (a / (1.0 + exp(-a))) * up[i]; /* silu(gate) * up */
  }
  orc_matmul(L->wdown, d, F, gate, T, proj);
  for (size_t i = 0; i < (size_t)T * d; ++i) x[i] += proj[i];

  free(h); free(q); free(k); free(v); free(att); free(proj); free(gate); free(up);
}

/* ---------------------------------------------------------------- heads -------------------- */

/* logits = W_lm * RMSNorm(x; final_norm) for one position. */
void orc_head_logits(const orc_shape* s, const float* final_norm, const float* head, const double* x,
                     double* logits) {
  double* h = (double*)malloc(sizeof(double) * (size_t)s->d_model);
  orc_rmsnorm(x, final_norm, s->d_model, s->rms_eps, h);
  orc_matmul(head, s->vocab, s->d_model, h, 1, logits);
  free(h);
}

/* PRM score of one position: w_r . RMSNorm(x; final_norm), through a sigmoid when
 * head_kind == 1 (scores in [0,1]); head_kind == 2 leaves the raw scalar (outcome reward models,
 * Section 4 "general-domain" experiment, score on the whole real line). */
double orc_head_reward(const orc_shape* s, const float* final_norm, const float* head, const double* x) {
  double* h = (double*)malloc(sizeof(double) * (size_t)s->d_model);
  orc_rmsnorm(x, final_norm, s->d_model, s->rms_eps, h);
  double a = 0.0;
  for (int i = 0; i < s->d_model; ++i) a += (double)head[i] * h[i];
  free(h);
  if (s->head_kind == 2) return a;
  return 1.0 / (1.0 + exp(-a));
}

/* ---------------------------------------------------------------- random numbers ----------- */

/* Philox4x32-10: ten rounds of  (c0,c1,c2,c3) <- (hi(M1*c2)^c1^k0, lo(M1*c2), hi(M0*c0)^c3^k1, lo(M0*c0)),
 * the key advancing by the Weyl constants after each round. */
void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
  uint32_t c[4] = {ctr[0], ctr[1], ctr[2], ctr[3]};
  uint32_t k[2] = {key[0], key[1]};
  for (int round = 0; round < 10; ++round) {
    if (round > 0) { k[0] += 0x9E3779B9u; k[1] += 0xBB67AE85u; }
    uint64_t prod0 = (uint64_t)c[0] * 0xD2511F53ull;
    uint64_t prod1 = (uint64_t)c[2] * 0xCD9E8D57ull;
    uint32_t hi0 = (uint32_t)(prod0 >> 32), lo0 = (uint32_t)(prod0 & 0xFFFFFFFFull);
    uint32_t hi1 = (uint32_t)(prod1 >> 32), lo1 = (uint32_t)(prod1 & 0xFFFFFFFFull);
    uint32_t n[4] = {hi1 ^ c[1] ^ k[0], lo1, hi0 ^ c[3] ^ k[1], lo0};
    memcpy(c, n, sizeof(c));
  }
  memcpy(out, c, sizeof(c));
}

/* 32 random bits -> uniform on (0,1): the top 23 bits, centred in their cell, so that the value
 * (2k+1) / 2^24 is also exact in fp32 and never 0 or 1. */
double orc_uniform_from_bits(uint32_t x) { return ((double)(x >> 9) + 0.5) * (1.0 / 8388608.0); }

/* Uniform draw attached to (seed, stream, row, position, index): counter = (index/4, position,
 * row, stream), key = the two halves of the seed, word index%4 of the block. */
double orc_uniform(uint64_t seed, uint32_t stream, uint32_t row, uint32_t position, uint32_t index) {
  uint32_t ctr[4] = {index / 4u, position, row, stream};
  uint32_t key[2] = {(uint32_t)(seed & 0xFFFFFFFFull), (uint32_t)(seed >> 32)};
  uint32_t o[4];
  orc_philox4x32_10(ctr, key, o);
  return orc_uniform_from_bits(o[index % 4u]);
}

/* ---------------------------------------------------------------- sampling ----------------- */

/* Next-token choice over ids [0, v_limit).  temperature == 0: argmax of the logits (Section 3,
 * "Default Setting": temperature 0 for RSD).  temperature > 0: Gumbel-max, i.e.
 * argmax_v(logit_v / T + g_v) with g_v = -log(-log u_v), which draws from softmax(logits / T).
 * u_v is the uniform of (seed, stream = model id, row, position of the token being generated, v).
 * Ties go to the lowest id.  *margin receives (best - second best) of the compared scores. */
int32_t orc_sample(const double* logits, int v_limit, double temperature, uint64_t seed, uint32_t model_id,
                   uint32_t row, uint32_t position, double* margin) {
  double best = -INFINITY, second = -INFINITY;
  int32_t arg = 0;
  for (int v = 0; v < v_limit; ++v) {
    double sc;
    if (temperature > 0.0) {
      double u = orc_uniform(seed, model_id, row, position, (uint32_t)v);
      sc = logits[v] / temperature + (-log(-log(u)));
    } else {
      sc = logits[v];
    }
    if (sc > best) { second = best; best = sc; arg = v; }
    else if (sc > second) { second = sc; }
  }
  if (margin) *margin = best - second;
  return arg;
}

/* ---------------------------------------------------------------- acceptance --------------- */

/* Weighting functions of Table 1.  kind: 0 constant p (param a), 1 binary step 1(r >= delta)
 * (param a = delta), 2 clip(r, 0, 1), 3 max(0, r / (1 + r)), 4 logistic 1/(1+exp(-alpha (r-delta)))
 * (a = delta, b = alpha). */
double orc_omega(int kind, double r, double a, double b) {
  switch (kind) {
    case 0: return a;
    case 1: return (r >= a) ? 1.0 : 0.0;
    case 2: return fmin(1.0, fmax(0.0, r));
    case 3: return fmax(0.0, r / (1.0 + r));
    case 4: return 1.0 / (1.0 + exp(-b * (r - a)));
    default: return 0.0;
  }
}

/* Acceptance criterion of Algorithm 2: omega(r) in {0,1} decides by itself; otherwise accept iff
 * omega(r) >= u for a uniform u on (0,1) supplied by the caller. */
int orc_accept(int kind, double r, double a, double b, double u) {
  double w = orc_omega(kind, r, a, b);
  if (w == 0.0) return 0;
  if (w == 1.0) return 1;
  return (w >= u) ? 1 : 0;
}
