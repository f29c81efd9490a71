/*
 * CPU oracle for one continuous-batching decode step over 4-bit group-quantised
 * weights and a paged KV pool.
 *
 * THIS FILE IS TEST INFRASTRUCTURE.  It is the slow, plain definition that the
 * CUDA library is compared against; the product never calls it and shares no
 * code, header, table or helper with it.  Only the tests, the smoke check and
 * the CPU-baseline leg of the benchmark load it.
 *
 * What it defines.  The paper's scheduler (Algorithm 1) produces, at every
 * token boundary, one token for each request r of the active batch B by
 * GenerateToken(r, KVCache[r]).  The paper runs 4-bit quantised models
 * (Section 4, "Setup") and delegates the forward pass to its model library, so
 * the forward pass written here is the standard pre-norm decoder of the model
 * families in Table 1, with the storage format and the rounding points fixed as
 * follows (all accumulations in fp64, results rounded to bf16 with
 * round-to-nearest-even exactly where stated):
 *
 *   weight   w[j][k] = fl32(scale[j][k/64] * q[j][k] + bias[j][k/64]),
 *            q in 0..15, element k of a row in word k>>3, bits 4*(k&7)..+3
 *   x      = bf16(dequant(embed row tok_r))
 *   layer: y   = bf16(x * rsqrt(mean(x^2)+eps) * w_attn)
 *          qkv = bf16(Wqkv y)
 *          q,k = bf16(RMSNorm_128(head) * w_q|k)           (only if qk_norm)
 *          q,k = bf16(rope(head, position len_r))           pairs (i, i+64)
 *          append k, v at token slot len_r of the request's blocks
 *          s_t = q.k_t / sqrt(128), t = 0..len_r ; P = softmax(s)
 *          a   = bf16(sum_t P_t v_t)        kv head = q head / (nq/nkv)
 *          x   = bf16(x + bf16(Wo a))
 *          y   = bf16(RMSNorm(x) * w_mlp)
 *          h   = bf16(silu(bf16(Wg y)) * bf16(Wu y)),  silu(g) = g/(1+exp(-g))
 *          x   = bf16(x + bf16(Wd h))
 *          MoE layer: z = Wr y (unrounded), pi = softmax(z), top-k (lower index
 *          wins ties), renormalised if norm_topk_prob;
 *          x = bf16(x + bf16(sum_k pi_k * bf16(Wd_e(k) h_e(k))))
 *   logits = fl32(Wlm bf16(RMSNorm(x) * w_final)) ; next = argmax, lowest index
 *
 * Each request is computed independently of its batch-mates.
 *
 * Pins (tests/test_oracle_*.py): bf16 rounding against a library conversion and
 * closed-form ties; dequant against the closed form on all 16 codes; the
 * quantised matmul against an explicit float matrix product; RMSNorm, RoPE,
 * SiLU and softmax attention against invariants and a naive full-matrix form;
 * the paged gather against a contiguous layout under block permutations; batch
 * invariance; MoE against its dense special case; the whole step against an
 * independently written numpy restatement on toy shapes.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#define ORC_OK 0
#define ORC_ERR_ARG (-1)
#define ORC_ERR_ALLOC (-2)

typedef struct {
  int32_t n_layers, hidden, n_q_heads, n_kv_heads, head_dim;
  int32_t mlp_inter, vocab;
  int32_t group_size, bits;
  int32_t qk_norm, tie_embeddings;
  float rms_eps;
  int32_t n_experts, top_k, expert_inter, norm_topk_prob;
  int32_t max_batch, max_positions;
} orc_shape;

typedef struct {
  const uint32_t* q;
  const uint16_t* scales;
  const uint16_t* biases;
} orc_qtensor;

typedef struct {
  const uint16_t *attn_norm, *mlp_norm, *q_norm, *k_norm;
  orc_qtensor wqkv, wo, w_gate_up, w_down;
  const uint16_t* router;
  orc_qtensor experts_gate_up, experts_down;
} orc_layer;

typedef struct {
  const orc_layer* layers;
  const uint16_t* final_norm;
  orc_qtensor embed, lm_head;
  const float* rope_cos_sin; /* [max_positions][64][2] = cos, sin */
} orc_weights;

/* ------------------------------------------------------------------ bf16 */

/* bf16 bits -> value (exact). */
float orc_bf16_to_float(uint16_t h) {
  uint32_t u = ((uint32_t)h) << 16;
  float f;
  memcpy(&f, &u, 4);
  return f;
}

/* Nearest bf16 to a double, ties to even, one rounding straight from fp64.
 * bf16 = 1 sign, 8 exponent, 7 fraction bits; normal exponents -126..127,
 * subnormal spacing 2^-133. */
uint16_t orc_bf16_round(double v) {
  uint16_t sign = signbit(v) ? 0x8000u : 0u;
  if (isnan(v)) return 0x7fc0u;
  double a = fabs(v);
  if (isinf(a)) return (uint16_t)(sign | 0x7f80u);
  if (a == 0.0) return sign;
  int e;
  (void)frexp(a, &e);  /* a = m * 2^e, m in [0.5, 1) */
  int lead = e - 1;    /* exponent of the leading bit */
  if (lead < -126) lead = -126;
  double ulp = ldexp(1.0, lead - 7);
  double r = nearbyint(a / ulp) * ulp; /* default mode: ties to even; a/ulp is exact */
  if (r >= ldexp(1.0, 128)) return (uint16_t)(sign | 0x7f80u);
  float f = (float)r; /* exact: at most 8 significant bits */
  uint32_t u;
  memcpy(&u, &f, 4);
  return (uint16_t)(sign | (uint16_t)(u >> 16));
}

void orc_bf16_round_array(const double* in, int64_t n, uint16_t* out) {
  for (int64_t i = 0; i < n; ++i) out[i] = orc_bf16_round(in[i]);
}

static inline double bf(uint16_t h) { return (double)orc_bf16_to_float(h); }

/* ------------------------------------------------- 4-bit affine group-64 */

static inline uint32_t nibble(const uint32_t* qrow, int64_t k) {
  return (qrow[k >> 3] >> (4 * (k & 7))) & 0xFu;
}

/* Setup-time quantiser (not on the decode path).  Per group of 64 input
 * features: bias = bf16(min), scale = bf16((max-min)/15) in fp32 arithmetic,
 * code = clamp(rne((w-bias)/scale), 0, 15) in fp32 arithmetic; a flat group
 * (or a scale that rounds to zero) takes scale 1 and code 0. */
void orc_quantize_q4(const float* w, int64_t N, int64_t K, uint32_t* q, uint16_t* scales,
                     uint16_t* biases) {
  int64_t G = K / 64;
#pragma omp parallel for schedule(static)
  for (int64_t j = 0; j < N; ++j) {
    for (int64_t g = 0; g < G; ++g) {
      const float* p = w + j * K + g * 64;
      float lo = p[0], hi = p[0];
      for (int i = 1; i < 64; ++i) {
        if (p[i] < lo) lo = p[i];
        if (p[i] > hi) hi = p[i];
      }
      uint16_t bb = orc_bf16_round((double)lo);
      float d = (hi - lo) / 15.0f;
      uint16_t sb = orc_bf16_round((double)d);
      float s = orc_bf16_to_float(sb);
      float b = orc_bf16_to_float(bb);
      int flat = !(s > 0.0f);
      if (flat) {
        sb = 0x3f80u; /* 1.0 */
        s = 1.0f;
      }
      scales[j * G + g] = sb;
      biases[j * G + g] = bb;
      for (int wd = 0; wd < 8; ++wd) {
        uint32_t word = 0;
        for (int i = 0; i < 8; ++i) {
          uint32_t code = 0;
          if (!flat) {
            float t = (p[wd * 8 + i] - b) / s;
            float r = nearbyintf(t);
            if (r < 0.0f) r = 0.0f;
            if (r > 15.0f) r = 15.0f;
            code = (uint32_t)r;
          }
          word |= code << (4 * i);
        }
        q[j * (K / 8) + g * 8 + wd] = word;
      }
    }
  }
}

/* w[j][k] = fl32(scale*q + bias): one rounding, which fmaf gives by definition. */
static inline float dequant_one(const orc_qtensor* t, int64_t K, int64_t j, int64_t k) {
  int64_t G = K / 64;
  float s = orc_bf16_to_float(t->scales[j * G + (k >> 6)]);
  float b = orc_bf16_to_float(t->biases[j * G + (k >> 6)]);
  return fmaf(s, (float)nibble(t->q + j * (K / 8), k), b);
}

void orc_dequant_q4(const uint32_t* q, const uint16_t* scales, const uint16_t* biases, int64_t N,
                    int64_t K, float* out) {
  orc_qtensor t = {q, scales, biases};
#pragma omp parallel for schedule(static)
  for (int64_t j = 0; j < N; ++j)
    for (int64_t k = 0; k < K; ++k) out[j * K + k] = dequant_one(&t, K, j, k);
}

/* The definition accumulates in fp64.  A second build of this file with
 * -DORC_SENSITIVITY_PROBE_FP32 (made and loaded only by tests/fp32_probe.py, never by
 * oracle/build.py) accumulates the projections in fp32 instead: the tests use that
 * variant to measure how far any fp32-accumulating implementation drifts from the
 * definition once bf16 rounding decisions start to differ.  It is not the oracle. */
/* out[r][j] = sum_k w[j][k] * x[r][k], k ascending, fp64, for rows j in
 * [row0, row0+N) of a tensor with K input features.  x is bf16 [n][K]. */
static int q4_matmul_rows(const orc_qtensor* t, int64_t row0, int64_t N, int64_t K,
                          const uint16_t* x, int32_t n, double* out, int64_t out_stride) {
  double* xt = (double*)malloc(sizeof(double) * (size_t)K * (size_t)n); /* [k][r] */
  if (!xt) return ORC_ERR_ALLOC;
  for (int32_t r = 0; r < n; ++r)
    for (int64_t k = 0; k < K; ++k) xt[k * n + r] = bf(x[(int64_t)r * K + k]);
  int fail = 0;
#pragma omp parallel
  {
    float* wrow = (float*)malloc(sizeof(float) * (size_t)K);
    double* acc = (double*)malloc(sizeof(double) * (size_t)n);
    if (!wrow || !acc) {
#pragma omp atomic write
      fail = 1;
    } else {
#pragma omp for schedule(static)
      for (int64_t j = 0; j < N; ++j) {
        for (int64_t k = 0; k < K; ++k) wrow[k] = dequant_one(t, K, row0 + j, k);
        for (int32_t r = 0; r < n; ++r) acc[r] = 0.0;
#ifdef ORC_SENSITIVITY_PROBE_FP32
        for (int64_t k = 0; k < K; ++k) {
          const double* xk = xt + k * n;
          for (int32_t r = 0; r < n; ++r) acc[r] = (double)((float)acc[r] + wrow[k] * (float)xk[r]);
        }
#else
        for (int64_t k = 0; k < K; ++k) {
          double wk = (double)wrow[k];
          const double* xk = xt + k * n;
          for (int32_t r = 0; r < n; ++r) acc[r] += wk * xk[r];
        }
#endif
        for (int32_t r = 0; r < n; ++r) out[(int64_t)r * out_stride + j] = acc[r];
      }
    }
    free(wrow);
    free(acc);
  }
  free(xt);
  return fail ? ORC_ERR_ALLOC : ORC_OK;
}

int orc_q4_matmul(const uint32_t* q, const uint16_t* scales, const uint16_t* biases, int64_t N,
                  int64_t K, const uint16_t* x, int32_t n, double* out) {
  orc_qtensor t = {q, scales, biases};
  return q4_matmul_rows(&t, 0, N, K, x, n, out, N);
}

/* ---------------------------------------------------------------- RMSNorm */

/* y = bf16(x * (mean(x^2)+eps)^-1/2 * w) per row of length H. */
void orc_rmsnorm(const uint16_t* x, const uint16_t* w, float eps, int32_t n, int32_t H,
                 uint16_t* y) {
  for (int32_t r = 0; r < n; ++r) {
    double ss = 0.0;
    for (int32_t i = 0; i < H; ++i) {
      double v = bf(x[(int64_t)r * H + i]);
      ss += v * v;
    }
    double inv = 1.0 / sqrt(ss / (double)H + (double)eps);
    for (int32_t i = 0; i < H; ++i)
      y[(int64_t)r * H + i] = orc_bf16_round(bf(x[(int64_t)r * H + i]) * inv * bf(w[i]));
  }
}

/* ------------------------------------------------------------------- RoPE */

/* Rotate one head of even length d in place at a position whose table row is
 * cs = [d/2][2] (cos, sin), pairing element i with i + d/2. */
void orc_rope(uint16_t* head, const float* cs, int32_t d) {
  int32_t h = d / 2;
  for (int32_t i = 0; i < h; ++i) {
    double a = bf(head[i]), b = bf(head[i + h]);
    double c = (double)cs[2 * i], s = (double)cs[2 * i + 1];
    head[i] = orc_bf16_round(a * c - b * s);
    head[i + h] = orc_bf16_round(b * c + a * s);
  }
}

/* ------------------------------------------------------------ paged KV pool */
/* Pool layout: [layer][kv(0=K,1=V)][block][kv_head][slot][head_dim] bf16;
 * one block id names the same block in every layer. */

static inline int64_t pool_off(int32_t num_blocks, int32_t nkv, int32_t bs, int32_t d,
                               int32_t layer, int32_t kv, int32_t block, int32_t head,
                               int32_t slot) {
  return (((((int64_t)layer * 2 + kv) * num_blocks + block) * nkv + head) * bs + slot) * d;
}

/* Copy tokens 0..len-1 of one (layer, kv head) into contiguous [len][d]. */
void orc_kv_gather(const uint16_t* pool, int32_t num_blocks, int32_t nkv, int32_t bs, int32_t d,
                   int32_t layer, int32_t head, const int32_t* block_table, int32_t len,
                   uint16_t* k_out, uint16_t* v_out) {
  for (int32_t t = 0; t < len; ++t) {
    int32_t blk = block_table[t / bs], slot = t % bs;
    memcpy(k_out + (int64_t)t * d, pool + pool_off(num_blocks, nkv, bs, d, layer, 0, blk, head, slot),
           sizeof(uint16_t) * (size_t)d);
    memcpy(v_out + (int64_t)t * d, pool + pool_off(num_blocks, nkv, bs, d, layer, 1, blk, head, slot),
           sizeof(uint16_t) * (size_t)d);
  }
}

void orc_kv_append(uint16_t* pool, int32_t num_blocks, int32_t nkv, int32_t bs, int32_t d,
                   int32_t layer, int32_t head, const int32_t* block_table, int32_t pos,
                   const uint16_t* k, const uint16_t* v) {
  int32_t blk = block_table[pos / bs], slot = pos % bs;
  memcpy(pool + pool_off(num_blocks, nkv, bs, d, layer, 0, blk, head, slot), k,
         sizeof(uint16_t) * (size_t)d);
  memcpy(pool + pool_off(num_blocks, nkv, bs, d, layer, 1, blk, head, slot), v,
         sizeof(uint16_t) * (size_t)d);
}

/* -------------------------------------------------------------- attention */

/* One query head against contiguous K, V [T][d]:
 * out = bf16(sum_t softmax_t(q.k_t / sqrt(d)) v_t). */
int orc_attention_head(const uint16_t* q, const uint16_t* K, const uint16_t* V, int32_t T,
                       int32_t d, uint16_t* out) {
  double* s = (double*)malloc(sizeof(double) * (size_t)T);
  double* acc = (double*)calloc((size_t)d, sizeof(double));
  if (!s || !acc) {
    free(s);
    free(acc);
    return ORC_ERR_ALLOC;
  }
  double scale = 1.0 / sqrt((double)d), m = -INFINITY;
  for (int32_t t = 0; t < T; ++t) {
    double dot = 0.0;
    for (int32_t i = 0; i < d; ++i) dot += bf(q[i]) * bf(K[(int64_t)t * d + i]);
    s[t] = dot * scale;
    if (s[t] > m) m = s[t];
  }
  double Z = 0.0;
  for (int32_t t = 0; t < T; ++t) {
    s[t] = exp(s[t] - m);
    Z += s[t];
  }
  for (int32_t t = 0; t < T; ++t) {
    double p = s[t] / Z;
    for (int32_t i = 0; i < d; ++i) acc[i] += p * bf(V[(int64_t)t * d + i]);
  }
  for (int32_t i = 0; i < d; ++i) out[i] = orc_bf16_round(acc[i]);
  free(s);
  free(acc);
  return ORC_OK;
}

/* Decode attention for a batch over the paged pool (new token already
 * appended): q bf16 [n][nq][d] -> out bf16 [n][nq][d]; request r attends to
 * tokens 0..lens[r] inclusive. */
int orc_attention_paged(const uint16_t* q, const uint16_t* pool, int32_t num_blocks, int32_t nq,
                        int32_t nkv, int32_t bs, int32_t d, int32_t layer, int32_t n,
                        const int32_t* lens, const int32_t* block_tables, int32_t max_blocks,
                        uint16_t* out) {
  int32_t G = nq / nkv;
  int fail = 0;
#pragma omp parallel for schedule(dynamic, 1) collapse(2)
  for (int32_t r = 0; r < n; ++r) {
    for (int32_t h = 0; h < nkv; ++h) {
      int32_t T = lens[r] + 1;
      uint16_t* Kc = (uint16_t*)malloc(sizeof(uint16_t) * (size_t)T * (size_t)d);
      uint16_t* Vc = (uint16_t*)malloc(sizeof(uint16_t) * (size_t)T * (size_t)d);
      if (!Kc || !Vc) {
#pragma omp atomic write
        fail = 1;
      } else {
        orc_kv_gather(pool, num_blocks, nkv, bs, d, layer, h, block_tables + (int64_t)r * max_blocks,
                      T, Kc, Vc);
        for (int32_t g = 0; g < G; ++g) {
          int32_t qh = h * G + g;
          if (orc_attention_head(q + ((int64_t)r * nq + qh) * d, Kc, Vc, T, d,
                                 out + ((int64_t)r * nq + qh) * d) != ORC_OK) {
#pragma omp atomic write
            fail = 1;
          }
        }
      }
      free(Kc);
      free(Vc);
    }
  }
  return fail ? ORC_ERR_ALLOC : ORC_OK;
}

/* ------------------------------------------------------------- SiLU gating */

/* h = bf16(g/(1+exp(-g)) * u) elementwise. */
void orc_silu_mul(const uint16_t* g, const uint16_t* u, int64_t n, uint16_t* h) {
  for (int64_t i = 0; i < n; ++i) {
    double gv = bf(g[i]);
    h[i] = orc_bf16_round(gv / (1.0 + exp(-gv)) * bf(u[i]));
  }
}

/* ------------------------------------------------------------------ argmax */

void orc_argmax(const float* logits, int32_t n, int64_t V, int32_t* out) {
  for (int32_t r = 0; r < n; ++r) {
    const float* p = logits + (int64_t)r * V;
    int64_t best = 0;
    for (int64_t j = 1; j < V; ++j)
      if (p[j] > p[best]) best = j; /* strict: the lowest index keeps a tie */
    out[r] = (int32_t)best;
  }
}

/* ------------------------------------------------------------- MoE routing */

/* z fp64 [E] -> the top_k experts by softmax probability (lower index wins a
 * tie) and their weights, renormalised to sum 1 if norm is set. */
void orc_moe_route(const double* z, int32_t E, int32_t top_k, int32_t norm, int32_t* idx,
                   double* wgt) {
  double m = z[0];
  for (int32_t e = 1; e < E; ++e)
    if (z[e] > m) m = z[e];
  double Z = 0.0;
  for (int32_t e = 0; e < E; ++e) Z += exp(z[e] - m);
  double tot = 0.0;
  for (int32_t k = 0; k < top_k; ++k) {
    int32_t best = -1;
    for (int32_t e = 0; e < E; ++e) {
      int taken = 0;
      for (int32_t j = 0; j < k; ++j) taken |= (idx[j] == e);
      if (taken) continue;
      if (best < 0 || z[e] > z[best]) best = e;
    }
    idx[k] = best;
    wgt[k] = exp(z[best] - m) / Z;
    tot += wgt[k];
  }
  if (norm)
    for (int32_t k = 0; k < top_k; ++k) wgt[k] /= tot;
}

/* ------------------------------------------------------------ decode step */

static void round_rows(const double* in, int64_t cnt, uint16_t* out) {
  orc_bf16_round_array(in, cnt, out);
}

/* x <- bf16(x + bf16(delta)) */
static void residual_add(uint16_t* x, const double* delta, int64_t cnt) {
  for (int64_t i = 0; i < cnt; ++i) x[i] = orc_bf16_round(bf(x[i]) + bf(orc_bf16_round(delta[i])));
}

/* One decode step for n requests.  lens[r] = tokens already cached for request
 * r (its new token takes position lens[r]); the pool receives the new K, V.
 * layer_limit < n_layers runs only the first layer_limit layers before the
 * final norm and LM head (used to time a bounded sample).  taps, if given, is
 * bf16 [n_layers+1][n][H]: the hidden state after the embedding and after each
 * layer run.  Returns 0 or a negative error. */
int orc_decode_step(const orc_shape* sh, const orc_weights* w, uint16_t* pool, int32_t num_blocks,
                    int32_t block_size, int32_t n, const int32_t* lens, const int32_t* last_tokens,
                    const int32_t* block_tables, int32_t max_blocks, int32_t layer_limit,
                    int32_t* next_tokens, float* logits_out, uint16_t* taps) {
  if (!sh || !w || !pool || n < 0) return ORC_ERR_ARG;
  if (n == 0) return ORC_OK;
  const int32_t H = sh->hidden, d = sh->head_dim, nq = sh->n_q_heads, nkv = sh->n_kv_heads;
  const int32_t I = sh->mlp_inter, V = sh->vocab, L = sh->n_layers, E = sh->n_experts;
  const int32_t Ie = sh->expert_inter, top_k = sh->top_k;
  if (sh->group_size != 64 || sh->bits != 4 || d % 2 || nq % nkv) return ORC_ERR_ARG;
  if (layer_limit < 0 || layer_limit > L) layer_limit = L;
  for (int32_t r = 0; r < n; ++r) {
    if (lens[r] < 0 || lens[r] >= sh->max_positions) return ORC_ERR_ARG;
    if ((int64_t)max_blocks * block_size < (int64_t)lens[r] + 1) return ORC_ERR_ARG;
    if (last_tokens[r] < 0 || last_tokens[r] >= V) return ORC_ERR_ARG;
  }
  const int32_t Nqkv = (nq + 2 * nkv) * d;
  int64_t widest = H;
  if (Nqkv > widest) widest = Nqkv;
  if (2 * (int64_t)I > widest) widest = 2 * (int64_t)I;
  if (2 * (int64_t)Ie > widest) widest = 2 * (int64_t)Ie;
  if ((int64_t)nq * d > widest) widest = (int64_t)nq * d;

  uint16_t* x = (uint16_t*)malloc(sizeof(uint16_t) * (size_t)n * H);
  uint16_t* y = (uint16_t*)malloc(sizeof(uint16_t) * (size_t)n * H);
  uint16_t* qkv = (uint16_t*)malloc(sizeof(uint16_t) * (size_t)n * Nqkv);
  uint16_t* qh = (uint16_t*)malloc(sizeof(uint16_t) * (size_t)n * nq * d);
  uint16_t* att = (uint16_t*)malloc(sizeof(uint16_t) * (size_t)n * nq * d);
  uint16_t* gu = (uint16_t*)malloc(sizeof(uint16_t) * (size_t)n * (size_t)widest);
  uint16_t* hh = (uint16_t*)malloc(sizeof(uint16_t) * (size_t)n * (size_t)widest);
  double* acc = (double*)malloc(sizeof(double) * (size_t)n * (size_t)(V > widest ? V : widest));
  double* mix = (double*)malloc(sizeof(double) * (size_t)n * H);
  int rc = ORC_OK;
  if (!x || !y || !qkv || !qh || !att || !gu || !hh || !acc || !mix) {
    rc = ORC_ERR_ALLOC;
    goto done;
  }

  /* embedding */
  for (int32_t r = 0; r < n; ++r)
    for (int32_t k = 0; k < H; ++k)
      x[(int64_t)r * H + k] = orc_bf16_round((double)dequant_one(&w->embed, H, last_tokens[r], k));
  if (taps) memcpy(taps, x, sizeof(uint16_t) * (size_t)n * H);

  for (int32_t l = 0; l < layer_limit; ++l) {
    const orc_layer* lw = &w->layers[l];
    /* attention block */
    orc_rmsnorm(x, lw->attn_norm, sh->rms_eps, n, H, y);
    if ((rc = q4_matmul_rows(&lw->wqkv, 0, Nqkv, H, y, n, acc, Nqkv)) != ORC_OK) goto done;
    round_rows(acc, (int64_t)n * Nqkv, qkv);
    for (int32_t r = 0; r < n; ++r) {
      uint16_t* row = qkv + (int64_t)r * Nqkv;
      const float* cs = w->rope_cos_sin + (int64_t)lens[r] * d; /* (d/2) pairs of (cos, sin) */
      for (int32_t hd = 0; hd < nq + nkv; ++hd) { /* q heads then k heads */
        uint16_t* head = row + (int64_t)hd * d;
        if (sh->qk_norm) {
          uint16_t tmp[1024];
          if (d > 1024) {
            rc = ORC_ERR_ARG;
            goto done;
          }
          orc_rmsnorm(head, hd < nq ? lw->q_norm : lw->k_norm, sh->rms_eps, 1, d, tmp);
          memcpy(head, tmp, sizeof(uint16_t) * (size_t)d);
        }
        orc_rope(head, cs, d);
      }
      memcpy(qh + (int64_t)r * nq * d, row, sizeof(uint16_t) * (size_t)nq * d);
      for (int32_t hk = 0; hk < nkv; ++hk)
        orc_kv_append(pool, num_blocks, nkv, block_size, d, l, hk,
                      block_tables + (int64_t)r * max_blocks, lens[r], row + (int64_t)(nq + hk) * d,
                      row + (int64_t)(nq + nkv + hk) * d);
    }
    if ((rc = orc_attention_paged(qh, pool, num_blocks, nq, nkv, block_size, d, l, n, lens,
                                  block_tables, max_blocks, att)) != ORC_OK)
      goto done;
    if ((rc = q4_matmul_rows(&lw->wo, 0, H, (int64_t)nq * d, att, n, acc, H)) != ORC_OK) goto done;
    residual_add(x, acc, (int64_t)n * H);

    /* MLP block */
    orc_rmsnorm(x, lw->mlp_norm, sh->rms_eps, n, H, y);
    if (E == 0) {
      if ((rc = q4_matmul_rows(&lw->w_gate_up, 0, 2 * (int64_t)I, H, y, n, acc, 2 * (int64_t)I)) !=
          ORC_OK)
        goto done;
      round_rows(acc, (int64_t)n * 2 * I, gu);
      for (int32_t r = 0; r < n; ++r)
        orc_silu_mul(gu + (int64_t)r * 2 * I, gu + (int64_t)r * 2 * I + I, I, hh + (int64_t)r * I);
      if ((rc = q4_matmul_rows(&lw->w_down, 0, H, I, hh, n, acc, H)) != ORC_OK) goto done;
      residual_add(x, acc, (int64_t)n * H);
    } else {
      /* routed experts: each request alone through its top_k experts */
      for (int32_t r = 0; r < n; ++r) {
        const uint16_t* yr = y + (int64_t)r * H;
        double z[4096];
        int32_t idx[64];
        double pw[64];
        if (E > 4096 || top_k > 64 || top_k > E) {
          rc = ORC_ERR_ARG;
          goto done;
        }
        for (int32_t e = 0; e < E; ++e) {
          double s = 0.0;
          for (int32_t k = 0; k < H; ++k) s += bf(lw->router[(int64_t)e * H + k]) * bf(yr[k]);
          z[e] = s;
        }
        orc_moe_route(z, E, top_k, sh->norm_topk_prob, idx, pw);
        for (int32_t k = 0; k < H; ++k) mix[(int64_t)r * H + k] = 0.0;
        for (int32_t kk = 0; kk < top_k; ++kk) {
          int32_t e = idx[kk];
          if ((rc = q4_matmul_rows(&lw->experts_gate_up, (int64_t)e * 2 * Ie, 2 * (int64_t)Ie, H, yr,
                                   1, acc, 2 * (int64_t)Ie)) != ORC_OK)
            goto done;
          round_rows(acc, 2 * (int64_t)Ie, gu);
          orc_silu_mul(gu, gu + Ie, Ie, hh);
          if ((rc = q4_matmul_rows(&lw->experts_down, (int64_t)e * H, H, Ie, hh, 1, acc, H)) != ORC_OK)
            goto done;
          for (int32_t k = 0; k < H; ++k)
            mix[(int64_t)r * H + k] += pw[kk] * bf(orc_bf16_round(acc[k]));
        }
      }
      residual_add(x, mix, (int64_t)n * H);
    }
    if (taps) memcpy(taps + (int64_t)(l + 1) * n * H, x, sizeof(uint16_t) * (size_t)n * H);
  }

  /* final norm, LM head, greedy token */
  orc_rmsnorm(x, w->final_norm, sh->rms_eps, n, H, y);
  if ((rc = q4_matmul_rows(&w->lm_head, 0, V, H, y, n, acc, V)) != ORC_OK) goto done;
  {
    float* lg = logits_out ? logits_out : (float*)malloc(sizeof(float) * (size_t)n * V);
    if (!lg) {
      rc = ORC_ERR_ALLOC;
      goto done;
    }
    for (int64_t i = 0; i < (int64_t)n * V; ++i) lg[i] = (float)acc[i];
    if (next_tokens) orc_argmax(lg, n, V, next_tokens);
    if (!logits_out) free(lg);
  }

done:
  free(x);
  free(y);
  free(qkv);
  free(qh);
  free(att);
  free(gu);
  free(hh);
  free(acc);
  free(mix);
  return rc;
}

int orc_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}
