/*
 * CPU oracle for the per-window 8-bit decode step of Gated DeltaNet (scalar
 * gate) and Kimi Delta Attention (per-channel gate) recurrent states.
 *
 * THIS FILE IS TEST INFRASTRUCTURE.  It is the slow, plain statement of what
 * the method computes, written from the paper, and is what the GPU library is
 * checked against.  Only the tests, the smoke check and the benchmark's CPU
 * baseline leg may build or call it; the product never does.  It shares no
 * code, header, table or helper with the CUDA path.
 *
 * Orientation (Sec. 3.1, Eq. 1): one head has state S in R^{d_k x d_v},
 * stored row-major S[i*d_v + j] with i the key index and j the value index;
 * the readout is o = S^T q.
 *
 * Arithmetic: IEEE binary32, round to nearest even, compiled with
 * -ffp-contract=off so that a product is fused with an addition only where
 * fmaf() is written.  bf16 inputs and fp16 compensators are widened exactly.
 *
 * The boundary-state term of the readout, (B/127) Z^T (C Gamma x) in Appendix
 * B.3, is an integer payload times a vector.  The paper leaves its arithmetic
 * open; here the vector C Gamma x is taken in block fixed point (30 bits below
 * the power of two that bounds its largest entry) and the products with the
 * 8-bit codes are accumulated exactly, as integers.  The term is then free of
 * summation order, and it is more accurate than an fp32 accumulation.
 *
 * Summation order.  The paper never says in which order a sum is taken, yet
 * the 8-bit codes and the fp16 compensators are step functions of fp32
 * values, so the order has to be part of the definition.  Every reduction in
 * this file goes through csum_dot()/csum_abs(): the terms are taken in
 * consecutive blocks of eight; inside a block the even-numbered and the
 * odd-numbered terms are accumulated separately, left to right (first product
 * rounded, the others folded in with fmaf), and the two halves are added; the
 * block results are then added as a balanced binary tree over the block index
 * (neighbours first).  (Two interleaved chains per block are what a two-wide
 * fp32 fused multiply-add gives.)  Two other builds of this file exist to
 * measure what that choice and the fixed-point readout are worth:
 *   -DLQO_WIDE   every such sum is taken left to right in binary64 and
 *                rounded once (the fixed-point readout is kept);
 *   -DLQO_PLAIN  the same, and the readout is the plain definition as well:
 *                sum_i Z_ij x_i with x in binary32 as computed, no fixed-point
 *                grid, accumulated left to right in binary64 together with
 *                the compensator and record terms (records oldest first),
 *                rounded once.  Same constants, same start vectors.
 * A result of the defining build that differs from the PLAIN build's does
 * so because of summation order and the fixed-point grid, nothing else.
 *
 * Parity status of the pieces (what pins each is listed in the tests):
 *   reference recurrence, windowed decode, reconstruction, quantizer,
 *   smoothing, rank-r fit as a Frobenius minimiser        : pinned
 *   the constants n_iter, the start vectors of the power iteration, the 1e-30
 *   and 1e-6 guards of its orthonormalisation, the 1e-6 smoothing floor, the
 *   summation tree, the 30-bit fixed-point grid of the readout vector,
 *   the grouping of the readout's terms                    : parity unpinned
 *   (the paper fixes none of them; they are this build's definition).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

#if defined(LQO_PLAIN) && !defined(LQO_WIDE)
#define LQO_WIDE
#endif

enum { LQO_GATE_SCALAR = 0, LQO_GATE_DIAG = 1 };

typedef struct {
  int batch;     /* sequences                                              */
  int heads_v;   /* value heads per sequence (one state each)               */
  int heads_qk;  /* query/key heads per sequence; heads_v % heads_qk == 0   */
  int d_k, d_v;  /* state is d_k x d_v                                      */
  int W;         /* window length p                                         */
  int r;         /* Compensator Tokens per state                            */
  int n_iter;    /* power-iteration steps per compensator (>= 1)            */
  int gate;      /* LQO_GATE_SCALAR (GDN) or LQO_GATE_DIAG (KDA)            */
  int smooth;    /* 1: residual smoothing (Sec. 3.4); 0: c == 1             */
  int delta;     /* 1: delta rule, read vector b = alpha (.) k (DeltaNet, Gated DeltaNet, KDA);
                    0: b = 0, so u = v (linear attention, RetNet, Mamba2, GLA, RWKV6, HGRN2: Table 4) */
  int rec16;     /* 1: the buffered records are kept in fp16 as in the paper's storage accounting (kt, u and, for the
                    diagonal gate, alpha are rounded when a record is appended; the scalar gate's decay stays
                    fp32); 0: fp32 records */
  int state_bf16; /* 1: "per-window BF16" (the -w baseline of Fig. 3 and Table 2): the boundary state is the dense
                    state rounded to bfloat16 element by element, with no scale, smoothing or compensator;
                    needs the S0 array of lqo_state, whose entries are then bfloat16 values; 0: the 8-bit
                    representation (or, with S0 given, no quantization at all) */
} lqo_shape;

typedef struct {
  int8_t *codes;        /* [B,Hv,d_k,d_v]  Z                                */
  float *col_scale;     /* [B,Hv,d_v]      code step B_j/127, per value ch. */
  float *row_smooth;    /* [B,Hv,d_k]      c, per key row                   */
  uint16_t *comp_k;     /* [B,Hv,r,d_k]    fp16 bit patterns                */
  uint16_t *comp_u;     /* [B,Hv,r,d_v]    fp16 bit patterns                */
  float *buf_k;         /* [B,Hv,W,d_k]    write keys beta*k                */
  float *buf_u;         /* [B,Hv,W,d_v]    corrections u                    */
  float *buf_a;         /* [B,Hv,W] (scalar gate) or [B,Hv,W,d_k] (diag)    */
  int32_t *win_pos;     /* [B]             records buffered, 0..W-1 at rest */
  float *S0;            /* [B,Hv,d_k,d_v]  only for the no-quantization mode*/
} lqo_state;

/* ------------------------------------------------------------------ */
/* number formats                                                      */
/* ------------------------------------------------------------------ */

static float bits_f32(uint32_t u) { float f; memcpy(&f, &u, 4); return f; }
static uint32_t f32_bits(float f) { uint32_t u; memcpy(&u, &f, 4); return u; }

/* bf16 is the upper half of a binary32. */
static float bf16_to_f32(uint16_t h) { return bits_f32((uint32_t)h << 16); }

/* binary32 -> bfloat16, round to nearest even (used by the bf16-state baseline). */
uint16_t lqo_f32_to_bf16(float f) {
  uint32_t x = f32_bits(f);
  if ((x & 0x7FFFFFFFu) > 0x7F800000u) return (uint16_t)((x >> 16) | 0x0040u);
  uint32_t keep = x >> 16, rest = x & 0xFFFFu;
  if (rest > 0x8000u || (rest == 0x8000u && (keep & 1u))) keep++;
  return (uint16_t)keep;
}

/* binary16 -> binary32, exact. */
float lqo_f16_to_f32(uint16_t h) {
  uint32_t sign = (uint32_t)(h & 0x8000u) << 16;
  int e = (h >> 10) & 0x1F;
  uint32_t m = h & 0x3FFu;
  if (e == 31) return bits_f32(sign | 0x7F800000u | (m << 13));
  if (e == 0) {
    /* subnormal: m * 2^-24, exact in binary32 */
    float mag = (float)m * 5.9604644775390625e-08f;
    return sign ? -mag : mag;
  }
  return bits_f32(sign | ((uint32_t)(e - 15 + 127) << 23) | (m << 13));
}

/* binary32 -> binary16, round to nearest even; overflow goes to infinity
 * (callers that must not overflow clamp to +-65504 first). */
uint16_t lqo_f32_to_f16(float f) {
  uint32_t x = f32_bits(f);
  uint16_t sign = (uint16_t)((x >> 16) & 0x8000u);
  uint32_t mag = x & 0x7FFFFFFFu;
  if (mag > 0x7F800000u) return (uint16_t)(sign | 0x7E00u);          /* NaN  */
  if (mag >= 0x477FF000u) return (uint16_t)(sign | 0x7C00u);         /* >= 65520 */
  if (mag <= 0x33000000u) return sign;                               /* <= 2^-25 */
  int e = (int)(mag >> 23) - 127;
  uint32_t m24 = (mag & 0x7FFFFFu) | 0x800000u;  /* 1.m as a 24-bit integer */
  int drop;            /* low bits of m24 that do not fit                    */
  uint32_t out;
  if (e >= -14) {
    drop = 13;
    out = ((uint32_t)(e + 15) << 10) + ((m24 >> 13) - 0x400u);
  } else {
    drop = 13 + (-14 - e);
    out = m24 >> drop;
  }
  uint32_t rem = m24 & ((1u << drop) - 1u), half = 1u << (drop - 1);
  if (rem > half || (rem == half && (out & 1u))) out++;  /* a carry moves into the exponent */
  return (uint16_t)(sign | out);
}

static float clamp_f16_range(float x) { return fminf(fmaxf(x, -65504.0f), 65504.0f); }
/* the fp32 value of x after a round trip through saturating fp16 storage */
static float as_stored_f16(float x) { return lqo_f16_to_f32(lqo_f32_to_f16(clamp_f16_range(x))); }

/* ------------------------------------------------------------------ */
/* the one place where sums are taken                                  */
/* ------------------------------------------------------------------ */

/* sum_i a[i]*b[i], i = 0..n-1 */
float lqo_csum_dot(const float *a, const float *b, int n) {
#ifdef LQO_WIDE
  double acc = 0.0;
  for (int i = 0; i < n; i++) acc += (double)a[i] * (double)b[i];
  return (float)acc;
#else
  if (n <= 0) return 0.0f;
  int nblk = (n + 7) / 8, width = 1;
  while (width < nblk) width *= 2;
  float *part = (float *)malloc(sizeof(float) * (size_t)width);
  for (int c = 0; c < width; c++) {
    float acc = 0.0f;
    if (c < nblk) {
      int lo = 8 * c, hi = lo + 8 < n ? lo + 8 : n;
      float even = a[lo] * b[lo], odd = 0.0f;
      for (int i = lo + 2; i < hi; i += 2) even = fmaf(a[i], b[i], even);
      if (lo + 1 < hi) {
        odd = a[lo + 1] * b[lo + 1];
        for (int i = lo + 3; i < hi; i += 2) odd = fmaf(a[i], b[i], odd);
      }
      acc = even + odd;
    }
    part[c] = acc;
  }
  for (; width > 1; width /= 2)
    for (int c = 0; c < width / 2; c++) part[c] = part[2 * c] + part[2 * c + 1];
  float s = part[0];
  free(part);
  return s;
#endif
}

/* sum_i |x[i]|, same order */
float lqo_csum_abs(const float *x, int n) {
#ifdef LQO_WIDE
  double acc = 0.0;
  for (int i = 0; i < n; i++) acc += fabs((double)x[i]);
  return (float)acc;
#else
  if (n <= 0) return 0.0f;
  int nblk = (n + 7) / 8, width = 1;
  while (width < nblk) width *= 2;
  float *part = (float *)malloc(sizeof(float) * (size_t)width);
  for (int c = 0; c < width; c++) {
    float acc = 0.0f;
    if (c < nblk) {
      int lo = 8 * c, hi = lo + 8 < n ? lo + 8 : n;
      float even = fabsf(x[lo]), odd = 0.0f;
      for (int i = lo + 2; i < hi; i += 2) even = even + fabsf(x[i]);
      for (int i = lo + 1; i < hi; i += 2) odd = odd + fabsf(x[i]);
      acc = even + odd;
    }
    part[c] = acc;
  }
  for (; width > 1; width /= 2)
    for (int c = 0; c < width / 2; c++) part[c] = part[2 * c] + part[2 * c + 1];
  float s = part[0];
  free(part);
  return s;
#endif
}

/* column j of a row-major d_k x d_v matrix, gathered so that it can be summed */
static void column_of(const float *M, int d_k, int d_v, int j, float *out) {
  for (int i = 0; i < d_k; i++) out[i] = M[(size_t)i * d_v + j];
}

/* ------------------------------------------------------------------ */
/* block fixed point for the readout vector                            */
/* ------------------------------------------------------------------ */

/* X_i = rint(x_i * 2^(29-e)) with 2^e <= max|x| < 2^(e+1), so that |X_i| <= 2^30; returns 2^(e-29), the
 * factor that takes integers back (0 when the vector is zero or below 2^-96, in which case X = 0). */
static float block_fixed_point(const float *x, int n, int32_t *X) {
  float xmax = 0.0f;
  for (int i = 0; i < n; i++) xmax = fmaxf(xmax, fabsf(x[i]));
  if (!(xmax >= 0x1p-96f)) {
    for (int i = 0; i < n; i++) X[i] = 0;
    return 0.0f;
  }
  int e = (int)((f32_bits(xmax) >> 23) & 0xFF) - 127;       /* floor(log2 xmax); xmax is a normal number */
  float scale = bits_f32((uint32_t)(29 - e + 127) << 23);   /* 2^(29-e) */
  for (int i = 0; i < n; i++) X[i] = (int32_t)rintf(x[i] * scale);
  return bits_f32((uint32_t)(e - 29 + 127) << 23);          /* 2^(e-29) */
}

/* ------------------------------------------------------------------ */
/* per-head views                                                      */
/* ------------------------------------------------------------------ */

typedef struct {
  int8_t *Z; float *B, *c; uint16_t *ck, *cu; float *bk, *bu, *ba; float *S0;
} head_view;

static head_view view_of(const lqo_shape *sh, const lqo_state *st, int b, int h) {
  size_t bh = (size_t)b * sh->heads_v + h;
  size_t K = sh->d_k, V = sh->d_v, W = sh->W, r = sh->r;
  size_t na = sh->gate == LQO_GATE_DIAG ? K : 1;
  head_view hv;
  hv.Z = st->codes ? st->codes + bh * K * V : NULL;
  hv.B = st->col_scale ? st->col_scale + bh * V : NULL;
  hv.c = st->row_smooth ? st->row_smooth + bh * K : NULL;
  hv.ck = st->comp_k ? st->comp_k + bh * r * K : NULL;
  hv.cu = st->comp_u ? st->comp_u + bh * r * V : NULL;
  hv.bk = st->buf_k + bh * W * K;
  hv.bu = st->buf_u + bh * W * V;
  hv.ba = st->buf_a + bh * W * na;
  hv.S0 = st->S0 ? st->S0 + bh * K * V : NULL;
  return hv;
}

/* decay of record j as a d_k vector (a scalar gate is the same value on every key channel) */
static void record_decay(const lqo_shape *sh, const head_view *hv, int j, float *out) {
  for (int i = 0; i < sh->d_k; i++)
    out[i] = sh->gate == LQO_GATE_DIAG ? hv->ba[(size_t)j * sh->d_k + i] : hv->ba[j];
}

/* the token's inputs for value head h of sequence b, widened to binary32 */
typedef struct { float *q, *k, *v, *a; float beta; } token_in;

static token_in token_alloc(const lqo_shape *sh) {
  token_in t;
  t.q = (float *)malloc(sizeof(float) * sh->d_k);
  t.k = (float *)malloc(sizeof(float) * sh->d_k);
  t.a = (float *)malloc(sizeof(float) * sh->d_k);
  t.v = (float *)malloc(sizeof(float) * sh->d_v);
  t.beta = 0.0f;
  return t;
}
static void token_free(token_in *t) { free(t->q); free(t->k); free(t->a); free(t->v); }

static void token_load(const lqo_shape *sh, int b, int h, const uint16_t *q, const uint16_t *k,
                       const uint16_t *v, const uint16_t *beta, const uint16_t *alpha, token_in *t) {
  int K = sh->d_k, V = sh->d_v;
  int group = sh->heads_v / sh->heads_qk;
  size_t qk_off = ((size_t)b * sh->heads_qk + h / group) * K;  /* value head h reads q/k head h/group */
  size_t bh = (size_t)b * sh->heads_v + h;
  for (int i = 0; i < K; i++) {
    t->q[i] = bf16_to_f32(q[qk_off + i]);
    t->k[i] = bf16_to_f32(k[qk_off + i]);
    t->a[i] = sh->gate == LQO_GATE_DIAG ? bf16_to_f32(alpha[bh * K + i]) : bf16_to_f32(alpha[bh]);
  }
  for (int j = 0; j < V; j++) t->v[j] = bf16_to_f32(v[bh * V + j]);
  t->beta = bf16_to_f32(beta[bh]);
}

/* ------------------------------------------------------------------ */
/* Eq. 1 with the GDN / KDA coefficients of Table 4 (Appendix A):      */
/*   write key kt = beta*k, read vector b = alpha (.) k,               */
/*   u = v - S^T b,  S <- Diag(alpha) S + kt u^T,  o = S^T q           */
/* ------------------------------------------------------------------ */
static void head_ref_step(const lqo_shape *sh, float *S, const token_in *t, float *o) {
  int K = sh->d_k, V = sh->d_v;
  float *kt = (float *)malloc(sizeof(float) * K), *bv = (float *)malloc(sizeof(float) * K);
  float *col = (float *)malloc(sizeof(float) * K), *u = (float *)malloc(sizeof(float) * V);
  for (int i = 0; i < K; i++) { kt[i] = t->beta * t->k[i]; bv[i] = t->a[i] * t->k[i]; }
  for (int j = 0; j < V; j++) {
    column_of(S, K, V, j, col);
    u[j] = sh->delta ? t->v[j] - lqo_csum_dot(col, bv, K) : t->v[j];   /* b = 0: nothing is read back */
  }
  for (int i = 0; i < K; i++)
    for (int j = 0; j < V; j++) S[(size_t)i * V + j] = fmaf(kt[i], u[j], t->a[i] * S[(size_t)i * V + j]);
  for (int j = 0; j < V; j++) {
    column_of(S, K, V, j, col);
    o[j] = lqo_csum_dot(col, t->q, K);
  }
  free(kt); free(bv); free(col); free(u);
}

/* ------------------------------------------------------------------ */
/* Reconstruction of the state after the n buffered records, Eq. 7      */
/* (Eq. 4 when there is no smoothing and no compensator):               */
/*   S_n = Gamma_{1:n} [ C dequant(Z) + Kc Uc^T ] + sum_j Gamma_{j+1:n} kt_j u_j^T
 * with dequant(Z) = (Z/127) B (Appendix B.3; B/127 is what is stored).  The cumulative decays are
 * built up record by record from the newest one, as Appendix B.2 describes. */
/* ------------------------------------------------------------------ */
static void head_reconstruct(const lqo_shape *sh, const head_view *hv, int n, float *S) {
  int K = sh->d_k, V = sh->d_v, r = sh->r;
  float *gam = (float *)malloc(sizeof(float) * K);               /* Gamma_{j+1:n}, ends as Gamma_{1:n} */
  float *kd = (float *)malloc(sizeof(float) * (size_t)(n > 0 ? n : 1) * K); /* Gamma_{j+1:n} kt_j       */
  float *dec = (float *)malloc(sizeof(float) * K);
  for (int i = 0; i < K; i++) gam[i] = 1.0f;
  for (int j = n - 1; j >= 0; j--) {
    record_decay(sh, hv, j, dec);
    for (int i = 0; i < K; i++) {
      kd[(size_t)j * K + i] = gam[i] * hv->bk[(size_t)j * K + i];
      gam[i] = gam[i] * dec[i];
    }
  }
  for (int i = 0; i < K; i++)
    for (int j = 0; j < V; j++) {
      float base;
      if (hv->S0) {
        base = hv->S0[(size_t)i * V + j];                        /* quantization switched off */
      } else {
        float s = hv->B[j];                                       /* the stored step B_j/127 */
        base = hv->c[i] * ((float)hv->Z[(size_t)i * V + j] * s);
        for (int h = 0; h < r; h++)
          base = fmaf(lqo_f16_to_f32(hv->ck[(size_t)h * K + i]), lqo_f16_to_f32(hv->cu[(size_t)h * V + j]), base);
      }
      float x = gam[i] * base;
      for (int jj = 0; jj < n; jj++) x = fmaf(kd[(size_t)jj * K + i], hv->bu[(size_t)jj * V + j], x);
      S[(size_t)i * V + j] = x;
    }
  free(gam); free(kd); free(dec);
}

/* ------------------------------------------------------------------ */
/* Window-boundary quantization of a dense state M (destroyed):        */
/*   r Compensator Tokens, Eqs. 5-6: K~ U~^T is a rank-r fit of M in    */
/*   the Frobenius norm, found by power iteration on all r vectors at   */
/*   once and removed with the values that are actually stored (fp16);  */
/*   smoothing scales c, Sec. 3.4 (square root of the row mean |.|);    */
/*   per-value-channel symmetric 8-bit codes, Appendix B.3.             */
/* ------------------------------------------------------------------ */

/* Start vector h of the power iteration when no buffered record supplies one: entry j is -1 where j and h
 * share an odd number of set bits, else +1 (the Walsh functions: h = 0 is the all-equal vector, different h
 * are orthogonal).  Data-independent, so that the fit has one result per input. */
static float walsh_entry(int h, int j) {
  int x = h & j, odd = 0;
  while (x) { odd ^= 1; x &= x - 1; }
  return odd ? -1.0f : 1.0f;
}

/* Orthonormal basis Q of the span of the r vectors X[0..r-1] (each of length len), taken in order:
 * q_h = (x_h - sum_{j<h} L_hj q_j) / L_hh with L the Cholesky factor of the Gram matrix X^T X.  One pass of
 * dot products serves all r vectors.  A vector that is zero (squared length below 1e-30), or that the vectors
 * before it span already (what is left of its squared length is not above 1e-6 of it: fp32 cannot tell such a
 * remainder from rounding noise), gives q_h = 0 and alive[h] = 0. */
static void orthonormalize(const float *X, int len, int r, float *Q, int *alive) {
  float *G = (float *)malloc(sizeof(float) * (size_t)r * r), *L = (float *)calloc((size_t)r * r, sizeof(float));
  float *inv = (float *)malloc(sizeof(float) * (size_t)r);
  for (int a = 0; a < r; a++)
    for (int b = 0; b <= a; b++) G[a * r + b] = lqo_csum_dot(X + (size_t)a * len, X + (size_t)b * len, len);
  for (int h = 0; h < r; h++) {
    for (int j = 0; j < h; j++) {
      float s = G[h * r + j];
      for (int m = 0; m < j; m++) s = fmaf(-L[h * r + m], L[j * r + m], s);
      L[h * r + j] = s * inv[j];                          /* inv[j] = 0 for a vector that was dropped */
    }
    float d = G[h * r + h];
    for (int m = 0; m < h; m++) d = fmaf(-L[h * r + m], L[h * r + m], d);
    alive[h] = G[h * r + h] >= 1e-30f && d > 1e-6f * G[h * r + h];
    inv[h] = alive[h] ? 1.0f / sqrtf(d) : 0.0f;
  }
  for (int i = 0; i < len; i++)
    for (int h = 0; h < r; h++) {
      float x = X[(size_t)h * len + i];
      for (int j = 0; j < h; j++) x = fmaf(-L[h * r + j], Q[(size_t)j * len + i], x);
      Q[(size_t)h * len + i] = x * inv[h];
    }
  free(G); free(L); free(inv);
}

/* The paper says the compensators are "fitted with power iteration" and no more.  Here all r vectors are iterated
 * together (power iteration on a subspace): T = M W, orthonormalize; W = M^T T, orthonormalize; ... n_iter
 * times, ending on the key side.  The columns of W start from the value sides u of the newest buffered records
 * (column h from the (h+1)-th newest: they dominate the state that is being fitted), from Walsh vectors
 * where there is no such record.  The key sides are then rounded to fp16, and value side h is the least-squares
 * answer for what is left after components 0..h-1 as stored:
 *   u_h = (M - sum_{a<h} k_a u_a^T)^T k_h = M^T k_h - sum_{a<h} u_a (k_a^T k_h),
 * rounded to fp16 in turn.  `starts` holds `nstarts` rows of d_v floats, oldest first (the u part of the record
 * buffer), or is NULL. */
static void head_quantize(const lqo_shape *sh, float *M, const head_view *hv, const float *starts, int nstarts) {
  int K = sh->d_k, V = sh->d_v, r = sh->r;
  float *col = (float *)malloc(sizeof(float) * K);

  if (r > 0) {
    float *Wv = (float *)malloc(sizeof(float) * (size_t)r * V), *Xv = (float *)malloc(sizeof(float) * (size_t)r * V);
    float *T = (float *)malloc(sizeof(float) * (size_t)r * K), *Q = (float *)malloc(sizeof(float) * (size_t)r * K);
    float *kf = (float *)malloc(sizeof(float) * (size_t)r * K), *uf = (float *)malloc(sizeof(float) * (size_t)r * V);
    float *g = (float *)malloc(sizeof(float) * (size_t)r * r);
    int *alive = (int *)malloc(sizeof(int) * (size_t)r);
    for (int h = 0; h < r; h++)
      for (int j = 0; j < V; j++)
        Wv[(size_t)h * V + j] = (starts && h < nstarts) ? starts[(size_t)(nstarts - 1 - h) * V + j] : walsh_entry(h, j);
    for (int it = 0; it < sh->n_iter; it++) {
      for (int h = 0; h < r; h++)
        for (int i = 0; i < K; i++) T[(size_t)h * K + i] = lqo_csum_dot(M + (size_t)i * V, Wv + (size_t)h * V, V);   /* T = M W */
      orthonormalize(T, K, r, Q, alive);
      if (it + 1 < sh->n_iter) {
        for (int j = 0; j < V; j++) {
          column_of(M, K, V, j, col);
          for (int h = 0; h < r; h++) Xv[(size_t)h * V + j] = lqo_csum_dot(col, Q + (size_t)h * K, K);                /* W = M^T T */
        }
        orthonormalize(Xv, V, r, Wv, alive);
      }
    }
    /* key sides as stored */
    for (int h = 0; h < r; h++)
      for (int i = 0; i < K; i++) {
        uint16_t bits = alive[h] ? lqo_f32_to_f16(clamp_f16_range(Q[(size_t)h * K + i])) : 0;
        hv->ck[(size_t)h * K + i] = bits;
        kf[(size_t)h * K + i] = lqo_f16_to_f32(bits);
      }
    for (int a = 0; a < r; a++)
      for (int b = a + 1; b < r; b++) g[a * r + b] = lqo_csum_dot(kf + (size_t)a * K, kf + (size_t)b * K, K);
    /* value sides */
    for (int j = 0; j < V; j++) {
      column_of(M, K, V, j, col);
      for (int h = 0; h < r; h++) {
        float x = lqo_csum_dot(col, kf + (size_t)h * K, K);
        for (int a = 0; a < h; a++) x = fmaf(-uf[(size_t)a * V + j], g[a * r + h], x);
        uint16_t bits = alive[h] ? lqo_f32_to_f16(clamp_f16_range(x)) : 0;   /* a dropped component is all zero bits */
        hv->cu[(size_t)h * V + j] = bits;
        uf[(size_t)h * V + j] = lqo_f16_to_f32(bits);
      }
    }
    /* the residual R = M - K~ U~^T with the stored values */
    for (int i = 0; i < K; i++)
      for (int j = 0; j < V; j++) {
        float x = M[(size_t)i * V + j];
        for (int h = 0; h < r; h++) x = fmaf(-kf[(size_t)h * K + i], uf[(size_t)h * V + j], x);
        M[(size_t)i * V + j] = x;
      }
    free(Wv); free(Xv); free(T); free(Q); free(kf); free(uf); free(g); free(alive);
  }

  /* M is now the residual R.  Smooth the key rows, then quantize each value channel. */
  for (int i = 0; i < K; i++) {
    float ci = 1.0f;
    if (sh->smooth) {
      float mean_abs = lqo_csum_abs(M + (size_t)i * V, V) / (float)V;
      ci = fmaxf(sqrtf(mean_abs), 1e-6f);
    }
    hv->c[i] = ci;
    float inv_c = 1.0f / ci;
    for (int j = 0; j < V; j++) M[(size_t)i * V + j] = M[(size_t)i * V + j] * inv_c;
  }
  for (int j = 0; j < V; j++) {
    float amax = 0.0f;
    for (int i = 0; i < K; i++) amax = fmaxf(amax, fabsf(M[(size_t)i * V + j]));
    hv->B[j] = amax / 127.0f;                 /* stored as the step of the code: dequant = Z * step */
    float inv = amax > 0.0f ? 127.0f / amax : 0.0f;
    for (int i = 0; i < K; i++) {
      float z = rintf(M[(size_t)i * V + j] * inv);          /* ties to even */
      z = fminf(fmaxf(z, -127.0f), 127.0f);
      hv->Z[(size_t)i * V + j] = (int8_t)z;
    }
  }
  free(col);
}

/* the boundary state without the 8-bit quantizer: the dense state itself, or (per-window BF16) each element
 * rounded to the nearest bfloat16, ties to even */
static void head_store_dense(const lqo_shape *sh, const float *S, const head_view *hv) {
  size_t KV = (size_t)sh->d_k * sh->d_v;
  for (size_t e = 0; e < KV; e++) hv->S0[e] = sh->state_bf16 ? bf16_to_f32(lqo_f32_to_bf16(S[e])) : S[e];
}

/* boundary: rebuild S_W from the window representation and start the next window from it */
static void head_flush(const lqo_shape *sh, const head_view *hv, int n) {
  int K = sh->d_k, V = sh->d_v;
  float *S = (float *)malloc(sizeof(float) * (size_t)K * V);
  head_reconstruct(sh, hv, n, S);
  if (hv->S0) head_store_dense(sh, S, hv);
  else head_quantize(sh, S, hv, hv->bu, n);
  free(S);
}

/* ------------------------------------------------------------------ */
/* One decode token inside a window: the readout of Eq. 10 applied to   */
/* x = alpha (.) k (for the correction u, Eq. 3) and to x = alpha (.) q */
/* (for the output, using S_l^T q = S_{l-1}^T (alpha (.) q) + u (kt^T q)). */
/* n records are already buffered; the new record goes to slot n.       */
/* ------------------------------------------------------------------ */
static void head_decode(const lqo_shape *sh, const head_view *hv, int n, const token_in *t, float *o) {
  int K = sh->d_k, V = sh->d_v, r = sh->r;
  float *kt = (float *)malloc(sizeof(float) * K), *g = (float *)malloc(sizeof(float) * K);
  float *gk = (float *)malloc(sizeof(float) * K), *gq = (float *)malloc(sizeof(float) * K);
  float *dec = (float *)malloc(sizeof(float) * K), *col = (float *)malloc(sizeof(float) * K);
  float *pk = (float *)malloc(sizeof(float) * (n + r + 1)), *pq = (float *)malloc(sizeof(float) * (n + r + 1));
  float *ck = (float *)malloc(sizeof(float) * K);
  float *u = (float *)malloc(sizeof(float) * V);

  for (int i = 0; i < K; i++) { kt[i] = t->beta * t->k[i]; g[i] = t->a[i]; }

  /* real records, newest first; g is the decay from just after record j through the current token */
  for (int j = n - 1; j >= 0; j--) {
    for (int i = 0; i < K; i++) { gk[i] = g[i] * t->k[i]; gq[i] = g[i] * t->q[i]; }
    pk[j] = lqo_csum_dot(hv->bk + (size_t)j * K, gk, K);
    pq[j] = lqo_csum_dot(hv->bk + (size_t)j * K, gq, K);
    record_decay(sh, hv, j, dec);
    for (int i = 0; i < K; i++) g[i] = g[i] * dec[i];
  }
  /* g = Gamma_{1:l}: what the boundary state and its compensators have decayed by */
  for (int i = 0; i < K; i++) { gk[i] = g[i] * t->k[i]; gq[i] = g[i] * t->q[i]; }

  float *ptk = pk + n, *ptq = pq + n;      /* compensator projections */
  if (!hv->S0)
    for (int h = 0; h < r; h++) {
      for (int i = 0; i < K; i++) ck[i] = lqo_f16_to_f32(hv->ck[(size_t)h * K + i]);
      ptk[h] = lqo_csum_dot(ck, gk, K);
      ptq[h] = lqo_csum_dot(ck, gq, K);
    }

  float ktq = lqo_csum_dot(kt, t->q, K);

  /* boundary-state term: (B/127) Z^T (C Gamma x), the vector in block fixed point and the sum exact;
   * with quantization off it is S0^T (Gamma x) in fp32 */
  float *xk = (float *)malloc(sizeof(float) * K), *xq = (float *)malloc(sizeof(float) * K);
  int32_t *Xk = (int32_t *)malloc(sizeof(int32_t) * K), *Xq = (int32_t *)malloc(sizeof(int32_t) * K);
  for (int i = 0; i < K; i++) {
    xk[i] = hv->S0 ? gk[i] : hv->c[i] * gk[i];
    xq[i] = hv->S0 ? gq[i] : hv->c[i] * gq[i];
  }
  float back_k = 0.0f, back_q = 0.0f;
  if (!hv->S0) { back_k = block_fixed_point(xk, K, Xk); back_q = block_fixed_point(xq, K, Xq); }
  for (int j = 0; j < V; j++) {
    float rk, rq;
    if (hv->S0) {
      column_of(hv->S0, K, V, j, col);
      rk = lqo_csum_dot(col, xk, K);
      rq = lqo_csum_dot(col, xq, K);
    } else {
#ifdef LQO_PLAIN
      /* Eq. 10 as it stands: (B/127) Z^T (C Gamma x) + Uc (Kc^T Gamma x) + sum_j u_j (kt_j^T Gamma x), one sum */
      double ak = 0.0, aq = 0.0;
      for (int i = 0; i < K; i++) {
        ak += (double)hv->Z[(size_t)i * V + j] * (double)xk[i];
        aq += (double)hv->Z[(size_t)i * V + j] * (double)xq[i];
      }
      ak *= (double)hv->B[j];
      aq *= (double)hv->B[j];
      for (int h = 0; h < r; h++) {
        double uc = (double)lqo_f16_to_f32(hv->cu[(size_t)h * V + j]);
        ak += uc * (double)ptk[h];
        aq += uc * (double)ptq[h];
      }
      for (int jj = 0; jj < n; jj++) {
        ak += (double)hv->bu[(size_t)jj * V + j] * (double)pk[jj];
        aq += (double)hv->bu[(size_t)jj * V + j] * (double)pq[jj];
      }
      rk = (float)ak;
      rq = (float)aq;
      (void)Xk; (void)Xq; (void)back_k; (void)back_q;
#else
      int64_t tk = 0, tq = 0;
      for (int i = 0; i < K; i++) {
        tk += (int64_t)hv->Z[(size_t)i * V + j] * Xk[i];
        tq += (int64_t)hv->Z[(size_t)i * V + j] * Xq[i];
      }
      float s = hv->B[j];
      rk = s * ((float)tk * back_k);
      rq = s * ((float)tq * back_q);
      for (int h = 0; h < r; h++) {
        float uc = lqo_f16_to_f32(hv->cu[(size_t)h * V + j]);
        rk = fmaf(uc, ptk[h], rk);
        rq = fmaf(uc, ptq[h], rq);
      }
#endif
    }
#ifdef LQO_PLAIN
    if (hv->S0)
#endif
    {
      /* the records' terms: their own sum, from the newest record back, added as one number */
      float sk = 0.0f, sq = 0.0f;
      for (int jj = n - 1; jj >= 0; jj--) {
        sk = fmaf(hv->bu[(size_t)jj * V + j], pk[jj], sk);
        sq = fmaf(hv->bu[(size_t)jj * V + j], pq[jj], sq);
      }
      rk = rk + sk;
      rq = rq + sq;
    }
    u[j] = sh->delta ? t->v[j] - rk : t->v[j];   /* Eq. 3: u = v - S_{l-1}^T b, b = alpha (.) k or 0 */
    o[j] = fmaf(u[j], ktq, rq);          /* o = S_{l-1}^T (alpha (.) q) + u (kt^T q) */
  }

  /* append the record (alpha, kt, u) */
  /* (fp16 records: what is stored is the rounded value, widened again; o above used the unrounded u) */
  if (sh->gate == LQO_GATE_DIAG)
    for (int i = 0; i < K; i++) hv->ba[(size_t)n * K + i] = sh->rec16 ? as_stored_f16(t->a[i]) : t->a[i];
  else hv->ba[n] = t->a[0];
  for (int i = 0; i < K; i++) hv->bk[(size_t)n * K + i] = sh->rec16 ? as_stored_f16(kt[i]) : kt[i];
  for (int j = 0; j < V; j++) hv->bu[(size_t)n * V + j] = sh->rec16 ? as_stored_f16(u[j]) : u[j];

  free(kt); free(g); free(gk); free(gq); free(dec); free(col); free(pk); free(pq); free(ck); free(u);
  free(xk); free(xq); free(Xk); free(Xq);
}

/* ------------------------------------------------------------------ */
/* batch drivers (exported)                                            */
/* ------------------------------------------------------------------ */

static int shape_ok(const lqo_shape *sh) {
  return sh && sh->batch >= 0 && sh->heads_v > 0 && sh->heads_qk > 0 && sh->heads_v % sh->heads_qk == 0 &&
         sh->d_k > 0 && sh->d_v > 0 && sh->W > 0 && sh->r >= 0 && sh->n_iter >= 1 &&
         (sh->gate == LQO_GATE_SCALAR || sh->gate == LQO_GATE_DIAG) && (sh->delta == 0 || sh->delta == 1) &&
         (sh->rec16 == 0 || sh->rec16 == 1) && (sh->state_bf16 == 0 || sh->state_bf16 == 1);
}
/* per-window BF16 lives in the S0 array and has no compensators */
static int state_ok(const lqo_shape *sh, const lqo_state *st) {
  return !sh->state_bf16 || (st && st->S0 && sh->r == 0);
}

int lqo_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* Eq. 1 on a dense fp32 state (the unquantized trajectory). */
int lqo_ref_step_f32(const lqo_shape *sh, float *S, const uint16_t *q, const uint16_t *k, const uint16_t *v,
                     const uint16_t *beta, const uint16_t *alpha, float *o) {
  if (!shape_ok(sh)) return 1;
  long nh = (long)sh->batch * sh->heads_v;
#pragma omp parallel for schedule(dynamic, 1)
  for (long bh = 0; bh < nh; bh++) {
    int b = (int)(bh / sh->heads_v), h = (int)(bh % sh->heads_v);
    token_in t = token_alloc(sh);
    token_load(sh, b, h, q, k, v, beta, alpha, &t);
    head_ref_step(sh, S + (size_t)bh * sh->d_k * sh->d_v, &t, o + (size_t)bh * sh->d_v);
    token_free(&t);
  }
  return 0;
}

/* Eq. 2 with bf16 as the storage format: the state is rounded to bf16 after every token;
 * the output is read from the updated state before it is rounded. */
int lqo_ref_step_bf16(const lqo_shape *sh, uint16_t *S16, const uint16_t *q, const uint16_t *k, const uint16_t *v,
                      const uint16_t *beta, const uint16_t *alpha, float *o) {
  if (!shape_ok(sh)) return 1;
  long nh = (long)sh->batch * sh->heads_v;
  size_t KV = (size_t)sh->d_k * sh->d_v;
#pragma omp parallel for schedule(dynamic, 1)
  for (long bh = 0; bh < nh; bh++) {
    int b = (int)(bh / sh->heads_v), h = (int)(bh % sh->heads_v);
    token_in t = token_alloc(sh);
    token_load(sh, b, h, q, k, v, beta, alpha, &t);
    float *S = (float *)malloc(sizeof(float) * KV);
    for (size_t e = 0; e < KV; e++) S[e] = bf16_to_f32(S16[(size_t)bh * KV + e]);
    head_ref_step(sh, S, &t, o + (size_t)bh * sh->d_v);
    for (size_t e = 0; e < KV; e++) S16[(size_t)bh * KV + e] = lqo_f32_to_bf16(S[e]);
    free(S);
    token_free(&t);
  }
  return 0;
}

/* dense fp32 state -> window representation with an empty window */
int lqo_quantize_state(const lqo_shape *sh, const float *S, lqo_state *st) {
  if (!shape_ok(sh) || !state_ok(sh, st)) return 1;
  long nh = (long)sh->batch * sh->heads_v;
  size_t KV = (size_t)sh->d_k * sh->d_v;
#pragma omp parallel for schedule(dynamic, 1)
  for (long bh = 0; bh < nh; bh++) {
    head_view hv = view_of(sh, st, (int)(bh / sh->heads_v), (int)(bh % sh->heads_v));
    if (hv.S0) { head_store_dense(sh, S + (size_t)bh * KV, &hv); continue; }
    float *M = (float *)malloc(sizeof(float) * KV);
    memcpy(M, S + (size_t)bh * KV, sizeof(float) * KV);
    head_quantize(sh, M, &hv, NULL, 0);
    free(M);
  }
  for (int b = 0; b < sh->batch; b++) st->win_pos[b] = 0;
  return 0;
}

/* window representation -> the dense state it stands for right now (all buffered records applied) */
int lqo_dequantize_state(const lqo_shape *sh, const lqo_state *st, float *S) {
  if (!shape_ok(sh) || !state_ok(sh, st)) return 1;
  long nh = (long)sh->batch * sh->heads_v;
  size_t KV = (size_t)sh->d_k * sh->d_v;
#pragma omp parallel for schedule(dynamic, 1)
  for (long bh = 0; bh < nh; bh++) {
    int b = (int)(bh / sh->heads_v);
    head_view hv = view_of(sh, st, b, (int)(bh % sh->heads_v));
    head_reconstruct(sh, &hv, st->win_pos[b], S + (size_t)bh * KV);
  }
  return 0;
}

/* Flush sequences whose window is full (force == 0) or that hold any record (force != 0). */
int lqo_window_flush(const lqo_shape *sh, lqo_state *st, int force) {
  if (!shape_ok(sh) || !state_ok(sh, st)) return 1;
  long nh = (long)sh->batch * sh->heads_v;
#pragma omp parallel for schedule(dynamic, 1)
  for (long bh = 0; bh < nh; bh++) {
    int b = (int)(bh / sh->heads_v);
    int n = st->win_pos[b];
    if (n == sh->W || (force && n > 0)) {
      head_view hv = view_of(sh, st, b, (int)(bh % sh->heads_v));
      head_flush(sh, &hv, n);
    }
  }
  for (int b = 0; b < sh->batch; b++) {
    int n = st->win_pos[b];
    if (n == sh->W || (force && n > 0)) st->win_pos[b] = 0;
  }
  return 0;
}

/* One decode token for every (sequence, value head); a window that becomes full is flushed at once
 * (Eq. 4: the state is materialised and quantized only at l = p). */
int lqo_decode_step(const lqo_shape *sh, lqo_state *st, const uint16_t *q, const uint16_t *k, const uint16_t *v,
                    const uint16_t *beta, const uint16_t *alpha, float *o) {
  if (!shape_ok(sh) || !state_ok(sh, st)) return 1;
  for (int b = 0; b < sh->batch; b++)
    if (st->win_pos[b] < 0 || st->win_pos[b] >= sh->W) return 2;
  long nh = (long)sh->batch * sh->heads_v;
#pragma omp parallel for schedule(dynamic, 1)
  for (long bh = 0; bh < nh; bh++) {
    int b = (int)(bh / sh->heads_v), h = (int)(bh % sh->heads_v);
    head_view hv = view_of(sh, st, b, h);
    token_in t = token_alloc(sh);
    token_load(sh, b, h, q, k, v, beta, alpha, &t);
    head_decode(sh, &hv, st->win_pos[b], &t, o + (size_t)bh * sh->d_v);
    token_free(&t);
  }
  for (int b = 0; b < sh->batch; b++) st->win_pos[b] += 1;
  return lqo_window_flush(sh, st, 0);
}
