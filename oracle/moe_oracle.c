/*
 * CPU oracle for the MoE verification layer -- TEST INFRASTRUCTURE ONLY.
 *
 * This file is the slow, plain, fp64 statement of what the verification-pass
 * MoE layer computes for gamma draft-tree tokens.  Only the test-suite, the
 * smoke check and the bench's CPU-baseline leg may call it; the product
 * (CUDA) path shares no code with it and must never route through it.
 *
 * What it follows:
 *   - Sec. 1 / Sec. 3 of the paper: a router assigns every token a top-k
 *     subset S_l(x_t) of the E experts of layer l.
 *   - Eq. 1: verification touches the union  E_verify = U_t S_l(x_t); its
 *     cardinality (the paper's "average active experts" metric, Table 1/3
 *     captions) is what this oracle reports as n_active.
 *   - Sec. 3 ("verification can reuse expert weights"): every expert of the
 *     union is applied to all tokens routed to it, so a weight row is decoded
 *     once and reused.
 *   - Fig. 1(c): one FP8 DeepSeek-V3.1 expert is 3*7168*2048 bytes = 44.04 MB;
 *     oracle_expert_code_bytes() reproduces that figure.
 * The paper does not print the expert FFN; the form used here is the gated
 * SwiGLU FFN  down( silu(gate x) * (up x) )  without biases, routed outputs
 * combined with the renormalised top-k router weights, plus always-on shared
 * experts with weight 1 (Table 13: "256 routed + 1 shared").
 *
 * Everything is evaluated in double precision directly from the raw input
 * bytes with the decoders below.  There is no blocking, fusion or reordering:
 * loops run in the order of the definition.  OpenMP (optional) only splits
 * independent output rows between threads.
 *
 * Every function here is pinned by tests that do not depend on this file's
 * own arithmetic (library decoders, float64 matmul, brute force, closed
 * forms); none is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORC_W_FP32 = 0, ORC_W_BF16 = 1, ORC_W_FP8E4M3_B128 = 2, ORC_W_MXFP4 = 3 };
enum { ORC_ACT_FP32 = 0, ORC_ACT_BF16 = 1 };
enum { ORC_SCORE_SOFTMAX = 0, ORC_SCORE_SIGMOID = 1 };

typedef struct {
  int32_t H, I, E, top_k, n_shared;
  int32_t wfmt, afmt, score;
  double routed_scale;
  int32_t ffn_kind; /* 0: bias-free SwiGLU (the benchmark configurations); 1: GPT-OSS form, see expert_ffn */
  int32_t n_group;  /* > 0: group-limited routing, see oracle_topk_grouped (score must be sigmoid) */
  int32_t topk_group;
  int32_t act_quant; /* 0: activations as given; 1, 2: FP8 activations with 1x128 scales, see oracle_act_quant */
} oracle_cfg;

/* All pointers are HOST pointers.  Layouts (K = contraction dim, contiguous):
 *   w_gate, w_up [E, I, H]; w_down [E, H, I]
 *   fp32 / bf16        : plain elements
 *   fp8 e4m3 + b128    : 1 byte per element, scales fp32 [E, ceil(N/128), ceil(K/128)]
 *   mxfp4              : byte i of a row = elements 2i (low nibble), 2i+1 (high nibble);
 *                        scales u8 e8m0 [E, N, K/32]
 *   shared experts use the same layouts with leading dim n_shared.            */
typedef struct {
  const float *router_w; /* [E,H] fp32 */
  const void *w_gate, *w_up, *w_down;
  const void *s_gate, *s_up, *s_down;
  const void *sh_gate, *sh_up, *sh_down;
  const void *sh_s_gate, *sh_s_up, *sh_s_down;
  const float *b_gate, *b_up, *b_down; /* ffn_kind 1: fp32 biases [E,I], [E,I], [E,H]; NULL = zero */
  const float *router_bias;            /* n_group > 0: fp32 score-correction bias [E]; NULL = zero */
} oracle_layer;

/* ---------------------------------------------------------------- decoders */

/* bf16 is the upper half of an IEEE binary32. */
double oracle_decode_bf16(uint16_t b) {
  uint32_t u = ((uint32_t)b) << 16;
  float f;
  memcpy(&f, &u, 4);
  return (double)f;
}

/* e4m3 "fn": 1 sign, 4 exponent (bias 7), 3 mantissa bits; no infinities;
 * exponent 15 with mantissa 7 is NaN; exponent 0 is subnormal (m * 2^-9). */
double oracle_decode_e4m3(uint8_t b) {
  int s = b >> 7, e = (b >> 3) & 15, m = b & 7;
  double v;
  if (e == 15 && m == 7) return NAN;
  if (e == 0)
    v = ldexp((double)m, -9);
  else
    v = ldexp(1.0 + (double)m / 8.0, e - 7);
  return s ? -v : v;
}

/* e2m1: 1 sign, 2 exponent (bias 1), 1 mantissa bit -> 0, .5, 1, 1.5, 2, 3, 4, 6 */
double oracle_decode_e2m1(uint8_t nib) {
  int s = (nib >> 3) & 1, e = (nib >> 1) & 3, m = nib & 1;
  double v = (e == 0) ? 0.5 * (double)m : ldexp(1.0 + 0.5 * (double)m, e - 1);
  return s ? -v : v;
}

/* e8m0: unsigned power-of-two scale 2^(b-127); 0xFF is NaN. */
double oracle_decode_e8m0(uint8_t b) {
  if (b == 0xFF) return NAN;
  return ldexp(1.0, (int)b - 127);
}

static double decode_act(const void *x, int afmt, size_t idx) {
  if (afmt == ORC_ACT_FP32) return (double)((const float *)x)[idx];
  return oracle_decode_bf16(((const uint16_t *)x)[idx]);
}

/* Decode row n of the [N,K] matrix of expert e into out[K]. */
static void decode_row(int wfmt, const void *w, const void *s, int64_t e, int64_t N, int64_t K,
                       int64_t n, double *out) {
  if (wfmt == ORC_W_FP32) {
    const float *p = (const float *)w + (e * N + n) * K;
    for (int64_t k = 0; k < K; ++k) out[k] = (double)p[k];
  } else if (wfmt == ORC_W_BF16) {
    const uint16_t *p = (const uint16_t *)w + (e * N + n) * K;
    for (int64_t k = 0; k < K; ++k) out[k] = oracle_decode_bf16(p[k]);
  } else if (wfmt == ORC_W_FP8E4M3_B128) {
    const uint8_t *p = (const uint8_t *)w + (e * N + n) * K;
    int64_t nb = (N + 127) / 128, kb = (K + 127) / 128;
    const float *sc = (const float *)s + (e * nb + n / 128) * kb;
    for (int64_t k = 0; k < K; ++k) out[k] = oracle_decode_e4m3(p[k]) * (double)sc[k / 128];
  } else { /* MXFP4 */
    const uint8_t *p = (const uint8_t *)w + (e * N + n) * (K / 2);
    const uint8_t *sc = (const uint8_t *)s + (e * N + n) * (K / 32);
    for (int64_t k = 0; k < K; ++k) {
      uint8_t byte = p[k >> 1];
      uint8_t nib = (k & 1) ? (uint8_t)(byte >> 4) : (uint8_t)(byte & 15);
      out[k] = oracle_decode_e2m1(nib) * oracle_decode_e8m0(sc[k / 32]);
    }
  }
}

/* Exposed so tests can pin the row decoder against library casts. */
void oracle_decode_weight_row(int32_t wfmt, const void *w, const void *s, int64_t e, int64_t N,
                              int64_t K, int64_t n, double *out) {
  decode_row(wfmt, w, s, e, N, K, n, out);
}

/* Bytes of weight codes of one expert (3 matrices of I*H elements) -- Fig. 1(c). */
int64_t oracle_expert_code_bytes(const oracle_cfg *c) {
  int64_t el = 3 * (int64_t)c->H * c->I;
  switch (c->wfmt) {
    case ORC_W_FP32: return el * 4;
    case ORC_W_BF16: return el * 2;
    case ORC_W_FP8E4M3_B128: return el;
    default: return el / 2;
  }
}

/* Bytes of scale factors of one expert. */
int64_t oracle_expert_scale_bytes(const oracle_cfg *c) {
  int64_t H = c->H, I = c->I;
  if (c->wfmt == ORC_W_FP8E4M3_B128) {
    int64_t hb = (H + 127) / 128, ib = (I + 127) / 128;
    return 3 * hb * ib * 4;
  }
  if (c->wfmt == ORC_W_MXFP4) return 3 * H * I / 32;
  return 0;
}

/* ------------------------------------------------------------------ router */

/* logits[t,e] = sum_h x[t,h] * Wr[e,h], summed in index order (Sec. 1: the router's
 * per-token scores over the E experts, from which each token's top-k experts are taken). */
void oracle_router_logits(const oracle_cfg *c, const void *x, const float *router_w, int32_t gamma,
                          double *logits) {
  int64_t H = c->H, E = c->E;
#pragma omp parallel for schedule(static)
  for (int64_t t = 0; t < gamma; ++t)
    for (int64_t e = 0; e < E; ++e) {
      double acc = 0.0;
      for (int64_t h = 0; h < H; ++h)
        acc += decode_act(x, c->afmt, (size_t)(t * H + h)) * (double)router_w[e * H + h];
      logits[t * E + e] = acc;
    }
}

/* Top-k on the raw logits: order experts by (logit descending, id ascending)
 * and keep the first k.  Weights over the selected experts:
 *   softmax: w_j = exp(l_j - l_max) / sum_{j<k} exp(l_j - l_max)
 *   sigmoid: s_j = 1/(1+exp(-l_j)),  w_j = c * s_j / (sum_j s_j + 1e-20)
 * gap[t] = l_(k) - l_(k+1) (inf when k == E): the decision margin of token t. */
void oracle_topk(const oracle_cfg *c, const double *logits, int32_t gamma, int32_t *ids, double *w,
                 double *gap) {
  int E = c->E, k = c->top_k;
  for (int t = 0; t < gamma; ++t) {
    const double *l = logits + (int64_t)t * E;
    char *taken = (char *)calloc((size_t)E, 1);
    for (int j = 0; j < k; ++j) {
      int best = -1;
      for (int e = 0; e < E; ++e) {
        if (taken[e]) continue;
        if (best < 0 || l[e] > l[best]) best = e; /* strict '>' keeps the lower id on ties */
      }
      taken[best] = 1;
      ids[t * k + j] = best;
    }
    if (gap) {
      int nxt = -1;
      for (int e = 0; e < E; ++e) {
        if (taken[e]) continue;
        if (nxt < 0 || l[e] > l[nxt]) nxt = e;
      }
      gap[t] = (nxt < 0) ? INFINITY : l[ids[t * k + k - 1]] - l[nxt];
    }
    free(taken);
    if (c->score == ORC_SCORE_SOFTMAX) {
      double lmax = l[ids[t * k]], den = 0.0;
      for (int j = 0; j < k; ++j) den += exp(l[ids[t * k + j]] - lmax);
      for (int j = 0; j < k; ++j) w[t * k + j] = exp(l[ids[t * k + j]] - lmax) / den;
    } else {
      double den = 0.0;
      for (int j = 0; j < k; ++j) den += 1.0 / (1.0 + exp(-l[ids[t * k + j]]));
      for (int j = 0; j < k; ++j)
        w[t * k + j] = c->routed_scale * (1.0 / (1.0 + exp(-l[ids[t * k + j]]))) / (den + 1e-20);
    }
  }
}

/* Group-limited routing of the published DeepSeek-V3 models (not in the paper, whose routing is a
 * plain top-k): s_e = sigmoid(l_e); c_e = s_e + bias_e; the E experts form n_group contiguous
 * groups; a group's score is the sum of its two largest c (its only c when it has one expert);
 * the topk_group best groups are kept (score descending, index ascending); among their experts the
 * top k by (c descending, id ascending) are selected, in that order; weights use the unbiased
 * scores: w_j = routed_scale * s_j / (sum_j s_j + 1e-20).
 * gap[t] = the smaller of the two decision margins (k-th vs next c among kept experts; last kept
 * vs first dropped group score; inf where there is no alternative). */
void oracle_topk_grouped(const oracle_cfg *c, const double *logits, const float *bias, int32_t gamma,
                         int32_t *ids, double *w, double *gap) {
  int E = c->E, k = c->top_k, ng = c->n_group, kg = c->topk_group, gs = E / ng;
  double *sc = (double *)malloc(sizeof(double) * (size_t)E);
  double *cc = (double *)malloc(sizeof(double) * (size_t)E);
  double *G = (double *)malloc(sizeof(double) * (size_t)ng);
  char *keep = (char *)malloc((size_t)ng);
  char *taken = (char *)malloc((size_t)E);
  for (int t = 0; t < gamma; ++t) {
    const double *l = logits + (int64_t)t * E;
    for (int e = 0; e < E; ++e) {
      sc[e] = 1.0 / (1.0 + exp(-l[e]));
      cc[e] = sc[e] + (bias ? (double)bias[e] : 0.0);
    }
    for (int g = 0; g < ng; ++g) {
      int b1 = -1, b2 = -1;
      for (int e = g * gs; e < (g + 1) * gs; ++e)
        if (b1 < 0 || cc[e] > cc[b1]) b1 = e;
      for (int e = g * gs; e < (g + 1) * gs; ++e)
        if (e != b1 && (b2 < 0 || cc[e] > cc[b2])) b2 = e;
      G[g] = cc[b1] + (b2 >= 0 ? cc[b2] : 0.0);
      keep[g] = 0;
    }
    double gmargin = INFINITY;
    int last_kept = -1;
    for (int j = 0; j < kg; ++j) {
      int best = -1;
      for (int g = 0; g < ng; ++g)
        if (!keep[g] && (best < 0 || G[g] > G[best])) best = g;
      keep[best] = 1;
      last_kept = best;
    }
    for (int g = 0; g < ng; ++g)
      if (!keep[g] && G[last_kept] - G[g] < gmargin) gmargin = G[last_kept] - G[g];
    memset(taken, 0, (size_t)E);
    for (int j = 0; j < k; ++j) {
      int best = -1;
      for (int e = 0; e < E; ++e) {
        if (taken[e] || !keep[e / gs]) continue;
        if (best < 0 || cc[e] > cc[best]) best = e;
      }
      taken[best] = 1;
      ids[t * k + j] = best;
    }
    if (gap) {
      int nxt = -1;
      for (int e = 0; e < E; ++e) {
        if (taken[e] || !keep[e / gs]) continue;
        if (nxt < 0 || cc[e] > cc[nxt]) nxt = e;
      }
      double m = (nxt < 0) ? INFINITY : cc[ids[t * k + k - 1]] - cc[nxt];
      gap[t] = m < gmargin ? m : gmargin;
    }
    double den = 0.0;
    for (int j = 0; j < k; ++j) den += sc[ids[t * k + j]];
    for (int j = 0; j < k; ++j) w[t * k + j] = c->routed_scale * sc[ids[t * k + j]] / (den + 1e-20);
  }
  free(sc); free(cc); free(G); free(keep); free(taken);
}

/* Eq. 1: the union of the per-token expert sets, and the token->expert
 * grouping.  union_ids ascending [U]; offsets [U+1] exclusive scan of the
 * per-expert token counts in that order; perm[A] lists the assignments
 * a = t*k + j sorted by expert id, ties kept in increasing a (stable);
 * inv_perm[a] is the position of a in perm.  Returns U. */
int32_t oracle_union_perm(int32_t E, int32_t k, int32_t gamma, const int32_t *ids,
                          int32_t *union_ids, int32_t *offsets, int32_t *perm, int32_t *inv_perm) {
  int A = gamma * k, U = 0, pos = 0;
  for (int e = 0; e < E; ++e) {
    int cnt = 0;
    for (int a = 0; a < A; ++a)
      if (ids[a] == e) {
        if (perm) perm[pos] = a;
        if (inv_perm) inv_perm[a] = pos;
        ++pos;
        ++cnt;
      }
    if (cnt) {
      if (union_ids) union_ids[U] = e;
      if (offsets) offsets[U] = pos - cnt;
      ++U;
    }
  }
  if (offsets) offsets[U] = pos;
  return U;
}

/* ------------------------------------------------- FP8 activations (1x128) */

/* Nearest e4m3 code of a finite float, ties to the even code, magnitudes above
 * 448 saturate to 448.  Written as a search over the 127 finite magnitudes of
 * the decoder above. */
uint8_t oracle_encode_e4m3(float f) {
  double a = fabs((double)f);
  int lo = 0;
  if (a >= 448.0) {
    lo = 0x7E;
  } else {
    while (lo < 0x7E && oracle_decode_e4m3((uint8_t)(lo + 1)) <= a) ++lo; /* value(lo) <= a < value(lo + 1) */
    double dl = a - oracle_decode_e4m3((uint8_t)lo), dh = oracle_decode_e4m3((uint8_t)(lo + 1)) - a;
    if (dh < dl || (dh == dl && (lo & 1))) ++lo;
  }
  return (uint8_t)(lo | (signbit(f) ? 0x80 : 0));
}

/* Not in the paper (which does not print the expert FFN): deployed DeepSeek-V3
 * inference feeds every expert GEMM with FP8 activations, quantised on the fly
 * per token and per block of 128 consecutive elements of the contraction axis:
 *   amax = max |x_i| over the block,   s = amax / 448   (mode 1, binary32)
 *                                      s = 2^ceil(log2(amax / 448))   (mode 2, power-of-two scales)
 *   code_i = e4m3( x_i / s ),   the GEMM sees  decode(code_i) * s.
 * An all-zero block takes s = 1.  The scale, the division and the rounding are
 * binary32 operations (the codes are integers decided by floating point, so
 * the precision is part of the definition); the last block may be shorter. */
void oracle_act_quant(const float *x, int64_t n, int32_t mode, uint8_t *codes, float *scales) {
  for (int64_t b0 = 0; b0 < n; b0 += 128) {
    int64_t b1 = b0 + 128 < n ? b0 + 128 : n;
    float amax = 0.0f;
    for (int64_t i = b0; i < b1; ++i) {
      float a = fabsf(x[i]);
      if (a > amax) amax = a;
    }
    float s = 1.0f;
    if (amax > 0.0f) {
      s = amax / 448.0f;
      if (mode == 2) {
        int e;
        float fr = frexpf(s, &e); /* s = fr * 2^e, fr in [0.5, 1) */
        s = ldexpf(1.0f, fr == 0.5f ? e - 1 : e);
      }
    }
    scales[b0 / 128] = s;
    for (int64_t i = b0; i < b1; ++i) codes[i] = oracle_encode_e4m3(x[i] / s);
  }
}

/* x (length n, values representable in binary32) -> the values the GEMM sees, in place */
static void act_qdq(double *x, int64_t n, int32_t mode) {
  float *xf = (float *)malloc(sizeof(float) * (size_t)n);
  uint8_t *q = (uint8_t *)malloc((size_t)n);
  float *sc = (float *)malloc(sizeof(float) * (size_t)((n + 127) / 128));
  for (int64_t i = 0; i < n; ++i) xf[i] = (float)x[i];
  oracle_act_quant(xf, n, mode, q, sc);
  for (int64_t i = 0; i < n; ++i) x[i] = oracle_decode_e4m3(q[i]) * (double)sc[i / 128];
  free(xf);
  free(q);
  free(sc);
}

/* --------------------------------------------------------------- expert FFN */

/* Apply expert e (of the tensor set wg/wu/wd with scales sg/su/sd) to m
 * tokens: xs[m][H] -> out[m][H] with out = Wd * ( silu(Wg x) * (Wu x) ),
 * silu(z) = z / (1 + exp(-z)).  Each weight row is decoded once.
 * ffn_kind 1 (the published GPT-OSS expert; not in the paper, which does not print the FFN):
 *   g = min(Wg x + bg, 7),  u = clamp(Wu x + bu, -7, 7),
 *   h = g * sigmoid(1.702 g) * (u + 1),  out = Wd h + bd          (bg, bu, bd may be NULL = 0).
 * act_quant != 0: both GEMM inputs, x and h (rounded to binary32 first), are replaced by their
 * FP8 1x128 quantisation (oracle_act_quant). */
static void expert_ffn(const oracle_cfg *c, const void *wg, const void *wu, const void *wd,
                       const void *sg, const void *su, const void *sd, int64_t e, int m,
                       const double *xs, double *out, const float *bg, const float *bu,
                       const float *bd) {
  int64_t H = c->H, I = c->I;
  double *hbuf = (double *)malloc(sizeof(double) * (size_t)m * (size_t)I);
  double *xq = NULL;
  if (c->act_quant) {
    xq = (double *)malloc(sizeof(double) * (size_t)m * (size_t)H);
    memcpy(xq, xs, sizeof(double) * (size_t)m * (size_t)H);
    for (int r = 0; r < m; ++r) act_qdq(xq + (int64_t)r * H, H, c->act_quant);
    xs = xq;
  }
#pragma omp parallel
  {
    double *rg = (double *)malloc(sizeof(double) * (size_t)(H > I ? H : I));
    double *ru = (double *)malloc(sizeof(double) * (size_t)H);
#pragma omp for schedule(static)
    for (int64_t i = 0; i < I; ++i) {
      decode_row(c->wfmt, wg, sg, e, I, H, i, rg);
      decode_row(c->wfmt, wu, su, e, I, H, i, ru);
      for (int r = 0; r < m; ++r) {
        const double *xv = xs + (int64_t)r * H;
        double g = 0.0, p = 0.0;
        for (int64_t h = 0; h < H; ++h) g += rg[h] * xv[h];
        for (int64_t h = 0; h < H; ++h) p += ru[h] * xv[h];
        if (c->ffn_kind == 1) {
          if (bg) g += (double)bg[e * I + i];
          if (bu) p += (double)bu[e * I + i];
          if (g > 7.0) g = 7.0;
          if (p > 7.0) p = 7.0;
          if (p < -7.0) p = -7.0;
          hbuf[(int64_t)r * I + i] = g / (1.0 + exp(-1.702 * g)) * (p + 1.0);
        } else {
          hbuf[(int64_t)r * I + i] = g / (1.0 + exp(-g)) * p;
        }
      }
    }
#pragma omp single
    {
      if (c->act_quant)
        for (int r = 0; r < m; ++r) act_qdq(hbuf + (int64_t)r * I, I, c->act_quant);
    }
#pragma omp for schedule(static)
    for (int64_t n = 0; n < H; ++n) {
      decode_row(c->wfmt, wd, sd, e, H, I, n, rg);
      for (int r = 0; r < m; ++r) {
        const double *hv = hbuf + (int64_t)r * I;
        double o = 0.0;
        for (int64_t i = 0; i < I; ++i) o += rg[i] * hv[i];
        if (c->ffn_kind == 1 && bd) o += (double)bd[e * H + n];
        out[(int64_t)r * H + n] = o;
      }
    }
    free(rg);
    free(ru);
  }
  free(hbuf);
  free(xq);
}

/* Exposed single-expert FFN on already-decoded double inputs (pins). */
void oracle_expert_ffn(const oracle_cfg *c, const oracle_layer *L, int32_t shared, int32_t e,
                       int32_t m, const double *xs, double *out) {
  if (shared)
    expert_ffn(c, L->sh_gate, L->sh_up, L->sh_down, L->sh_s_gate, L->sh_s_up, L->sh_s_down, e, m,
               xs, out, NULL, NULL, NULL);
  else
    expert_ffn(c, L->w_gate, L->w_up, L->w_down, L->s_gate, L->s_up, L->s_down, e, m, xs, out, L->b_gate, L->b_up,
               L->b_down);
}

/* ------------------------------------------------------------- whole layer */

/* The routed MoE layer over gamma tokens.
 *   y64[t,:] = sum_j w[t,j] * FFN_{ids[t,j]}(x_t) + sum_s FFN_shared_s(x_t)
 * evaluated expert by expert over the union (Eq. 1), each expert applied to
 * all of its tokens at once.  override_w (may be NULL) replaces the router
 * weights in the combine (used to test linearity in the combine weights).
 * skip_ffn != 0 stops after routing/grouping (y64 untouched).
 * Any output pointer may be NULL.  Returns U, or -1 on bad arguments. */
int32_t oracle_moe_verify(const oracle_cfg *c, const oracle_layer *L, const void *x, int32_t gamma,
                          const double *override_w, int32_t skip_ffn, double *y64,
                          int32_t *topk_ids, double *topk_w, int32_t *union_ids, int32_t *offsets,
                          int32_t *perm, int32_t *inv_perm, double *gap, double *logits_out) {
  if (!c || !L || !x || gamma < 1 || c->top_k < 1 || c->top_k > c->E) return -1;
  int64_t H = c->H;
  int E = c->E, k = c->top_k, A = gamma * k;
  double *logits = (double *)malloc(sizeof(double) * (size_t)gamma * (size_t)E);
  int32_t *ids = (int32_t *)malloc(sizeof(int32_t) * (size_t)A);
  double *w = (double *)malloc(sizeof(double) * (size_t)A);
  int32_t *uni = (int32_t *)malloc(sizeof(int32_t) * (size_t)E);
  int32_t *off = (int32_t *)malloc(sizeof(int32_t) * (size_t)(E + 1));
  int32_t *pm = (int32_t *)malloc(sizeof(int32_t) * (size_t)A);
  int32_t *ipm = (int32_t *)malloc(sizeof(int32_t) * (size_t)A);

  oracle_router_logits(c, x, L->router_w, gamma, logits);
  if (c->n_group > 0) oracle_topk_grouped(c, logits, L->router_bias, gamma, ids, w, gap);
  else oracle_topk(c, logits, gamma, ids, w, gap);
  int U = oracle_union_perm(E, k, gamma, ids, uni, off, pm, ipm);

  if (logits_out) memcpy(logits_out, logits, sizeof(double) * (size_t)gamma * (size_t)E);
  if (topk_ids) memcpy(topk_ids, ids, sizeof(int32_t) * (size_t)A);
  if (topk_w) memcpy(topk_w, w, sizeof(double) * (size_t)A);
  if (union_ids) memcpy(union_ids, uni, sizeof(int32_t) * (size_t)U);
  if (offsets) memcpy(offsets, off, sizeof(int32_t) * (size_t)(U + 1));
  if (perm) memcpy(perm, pm, sizeof(int32_t) * (size_t)A);
  if (inv_perm) memcpy(inv_perm, ipm, sizeof(int32_t) * (size_t)A);

  if (!skip_ffn && y64) {
    const double *cw = override_w ? override_w : w;
    double *xd = (double *)malloc(sizeof(double) * (size_t)gamma * (size_t)H);
    for (int64_t i = 0; i < (int64_t)gamma * H; ++i) xd[i] = decode_act(x, c->afmt, (size_t)i);
    double *xs = (double *)malloc(sizeof(double) * (size_t)gamma * (size_t)H);
    double *os = (double *)malloc(sizeof(double) * (size_t)gamma * (size_t)H);
    memset(y64, 0, sizeof(double) * (size_t)gamma * (size_t)H);
    for (int u = 0; u < U; ++u) {
      int m = off[u + 1] - off[u];
      for (int r = 0; r < m; ++r) {
        int t = pm[off[u] + r] / k;
        memcpy(xs + (int64_t)r * H, xd + (int64_t)t * H, sizeof(double) * (size_t)H);
      }
      expert_ffn(c, L->w_gate, L->w_up, L->w_down, L->s_gate, L->s_up, L->s_down, uni[u], m, xs,
                 os, L->b_gate, L->b_up, L->b_down);
      for (int r = 0; r < m; ++r) {
        int a = pm[off[u] + r], t = a / k;
        for (int64_t n = 0; n < H; ++n) y64[(int64_t)t * H + n] += cw[a] * os[(int64_t)r * H + n];
      }
    }
    for (int s = 0; s < c->n_shared; ++s) {
      expert_ffn(c, L->sh_gate, L->sh_up, L->sh_down, L->sh_s_gate, L->sh_s_up, L->sh_s_down, s,
                 gamma, xd, os, NULL, NULL, NULL);
      for (int64_t i = 0; i < (int64_t)gamma * H; ++i) y64[i] += os[i];
    }
    free(xd);
    free(xs);
    free(os);
  }
  free(logits);
  free(ids);
  free(w);
  free(uni);
  free(off);
  free(pm);
  free(ipm);
  return U;
}

/* Brute-force dense evaluation (tiny inputs only): every one of the E experts
 * is applied to every token and weighted by the gate g[t,e], which is the
 * router weight if e is among the token's top-k and 0 otherwise; shared
 * experts are added with weight 1.  No union, no grouping, no permutation. */
int32_t oracle_moe_dense(const oracle_cfg *c, const oracle_layer *L, const void *x, int32_t gamma,
                         double *y64) {
  if (!c || !L || !x || !y64 || gamma < 1) return -1;
  int64_t H = c->H;
  int E = c->E, k = c->top_k;
  double *logits = (double *)malloc(sizeof(double) * (size_t)gamma * (size_t)E);
  int32_t *ids = (int32_t *)malloc(sizeof(int32_t) * (size_t)gamma * (size_t)k);
  double *w = (double *)malloc(sizeof(double) * (size_t)gamma * (size_t)k);
  double *gate = (double *)calloc((size_t)gamma * (size_t)E, sizeof(double));
  oracle_router_logits(c, x, L->router_w, gamma, logits);
  if (c->n_group > 0) oracle_topk_grouped(c, logits, L->router_bias, gamma, ids, w, NULL);
  else oracle_topk(c, logits, gamma, ids, w, NULL);
  for (int t = 0; t < gamma; ++t)
    for (int j = 0; j < k; ++j) gate[(int64_t)t * E + ids[t * k + j]] = w[t * k + j];
  double *xd = (double *)malloc(sizeof(double) * (size_t)H);
  double *o = (double *)malloc(sizeof(double) * (size_t)H);
  memset(y64, 0, sizeof(double) * (size_t)gamma * (size_t)H);
  for (int t = 0; t < gamma; ++t) {
    for (int64_t h = 0; h < H; ++h) xd[h] = decode_act(x, c->afmt, (size_t)(t * H + h));
    for (int e = 0; e < E; ++e) {
      expert_ffn(c, L->w_gate, L->w_up, L->w_down, L->s_gate, L->s_up, L->s_down, e, 1, xd, o, L->b_gate, L->b_up,
                 L->b_down);
      for (int64_t n = 0; n < H; ++n) y64[(int64_t)t * H + n] += gate[(int64_t)t * E + e] * o[n];
    }
    for (int s = 0; s < c->n_shared; ++s) {
      expert_ffn(c, L->sh_gate, L->sh_up, L->sh_down, L->sh_s_gate, L->sh_s_up, L->sh_s_down, s, 1,
                 xd, o, NULL, NULL, NULL);
      for (int64_t n = 0; n < H; ++n) y64[(int64_t)t * H + n] += o[n];
    }
  }
  free(logits);
  free(ids);
  free(w);
  free(gate);
  free(xd);
  free(o);
  return 0;
}

int32_t oracle_num_threads(void) {
#ifdef _OPENMP
  return (int32_t)omp_get_max_threads();
#else
  return 1;
#endif
}

/* ------------------------------------------------- cost-aware draft selection */

/* Algorithm 1 (cost-aware draft selection), Eqs. 7-10 -- the step that runs before the
 * verification pass and shrinks its expert union.
 *
 * Tree of n nodes in topological order (parent[i] < i, parent[root] = -1); P[i] is the
 * cumulative draft probability of node i; pred[i] is the predicted expert set of node i
 * over all MoE layers as a bitmap of W 32-bit words (bit (l*E + e) = pair (l, e), Eq. 4);
 * buffer0 is the initial expert buffer B_0 (W words, may be NULL = empty).
 *   E_traj(i)  = OR of pred over the path root -> i                      (Eq. 7)
 *   dCost(i|B) = | E_traj(i) \ B |                                       (Eq. 8)
 *   score(i)   = P(i) / (dCost + eps)                                    (Eq. 9)
 * gamma rounds: score every unselected node, take the arg-max (exact ties: the lowest
 * index, so a parent precedes its children), add it to S and OR its E_traj into B.
 * global_cost != 0 is the ablation variant of Eq. 10: the cost is |E_traj(i)| and the
 * buffer is not updated.  Scores are evaluated in IEEE binary32 (one rounded add, one
 * rounded divide), the precision in which the arg-max is decided.
 * Outputs: selected[gamma] node indices in selection order; costs[gamma] the cost each had
 * when chosen (may be NULL); buffer_out (W words, may be NULL) the final buffer.
 * Returns the number selected (min(gamma, n)) or -1 on bad arguments. */
int32_t oracle_select_drafts(int32_t n, int32_t W, const int32_t *parent, const float *P,
                             const uint32_t *pred, const uint32_t *buffer0, int32_t gamma,
                             float eps, int32_t global_cost, int32_t *selected, int32_t *costs,
                             uint32_t *buffer_out) {
  if (n < 1 || W < 1 || gamma < 1 || !parent || !P || !pred || !selected) return -1;
  uint32_t *traj = (uint32_t *)malloc(sizeof(uint32_t) * (size_t)n * (size_t)W);
  uint32_t *B = (uint32_t *)calloc((size_t)W, sizeof(uint32_t));
  char *taken = (char *)calloc((size_t)n, 1);
  if (buffer0) memcpy(B, buffer0, sizeof(uint32_t) * (size_t)W);
  for (int i = 0; i < n; ++i) {
    if (parent[i] >= i) { free(traj); free(B); free(taken); return -1; }
    for (int w = 0; w < W; ++w)
      traj[(size_t)i * W + w] =
          pred[(size_t)i * W + w] | (parent[i] >= 0 ? traj[(size_t)parent[i] * W + w] : 0u);
  }
  int count = 0;
  while (count < gamma && count < n) {
    int best = -1, best_cost = 0;
    float best_score = 0.f;
    for (int i = 0; i < n; ++i) {
      if (taken[i]) continue;
      int cost = 0;
      for (int w = 0; w < W; ++w) {
        uint32_t v = traj[(size_t)i * W + w];
        if (!global_cost) v &= ~B[w];
        while (v) { v &= v - 1; ++cost; }
      }
      volatile float den = (float)cost + eps; /* rounded to binary32 before the divide */
      float score = P[i] / den;
      if (best < 0 || score > best_score) { best = i; best_score = score; best_cost = cost; }
    }
    taken[best] = 1;
    selected[count] = best;
    if (costs) costs[count] = best_cost;
    if (!global_cost)
      for (int w = 0; w < W; ++w) B[w] |= traj[(size_t)best * W + w];
    ++count;
  }
  if (buffer_out) memcpy(buffer_out, B, sizeof(uint32_t) * (size_t)W);
  free(traj);
  free(B);
  free(taken);
  return count;
}
