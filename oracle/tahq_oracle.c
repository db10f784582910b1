/*
 * TAH-Quant boundary codec -- CPU ORACLE (test infrastructure, not the product).
 *
 * Plain scalar C, one loop per step, in the order the paper gives the steps
 * (Sec. 3.1 tiles -> Sec. 3.2 entropy + top-p% allocation -> Sec. 3.3 outlier
 * test, pivot swap, Hadamard, asymmetric quantiser -> Sec. 3.4 packing; the
 * receiver of Algorithm 1 line 5 runs the inverse).  No blocking, no fusion,
 * no vectorisation: a reader should be able to tick every line off against
 * the paper.  Where the paper leaves a choice open (constants, tie rules,
 * rounding, byte layout) the choice is stated in the comment of the step.
 *
 * Pinned by tests/test_oracle_*.py (Hadamard orthogonality against an explicit
 * Sylvester matrix, closed-form entropies, brute-force allocation, textbook
 * min-max quantisation, published Philox known answers, size accounting of
 * Sec. 3.4, error bounds).  The encoded bytes of a whole realistic tensor are
 * "parity unpinned": the paper prints no worked example of an encoded tile, so
 * whole-buffer bytes are pinned only through those per-step checks.
 *
 * Build: gcc -O2 -std=c11 -ffp-contract=off -fno-fast-math -fopenmp -fPIC -shared
 */
#include "tahq_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------ */
/* Number formats                                                      */
/* ------------------------------------------------------------------ */

static uint32_t f32_bits(float x) { uint32_t u; memcpy(&u, &x, 4); return u; }
static float bits_f32(uint32_t u) { float x; memcpy(&x, &u, 4); return x; }

/* binary32 -> binary16, round-to-nearest-even, gradual underflow, overflow to
 * infinity (callers clamp to the finite range first). */
uint16_t tahqo_f32_to_f16(float x) {
  uint32_t u = f32_bits(x);
  uint32_t sign = (u >> 16) & 0x8000u;
  uint32_t mag = u & 0x7fffffffu;
  if (mag >= 0x7f800000u) return (uint16_t)(sign | (mag > 0x7f800000u ? 0x7e00u : 0x7c00u));
  /* Express |x| as an integer number n of half-precision quanta, rounding once. */
  int e = (int)(mag >> 23) - 127;              /* unbiased exponent of |x| (for normals) */
  if (mag < 0x00800000u) return (uint16_t)sign; /* fp32 subnormal: far below 2^-25 -> 0   */
  if (e >= 16) return (uint16_t)(sign | 0x7c00u);
  uint32_t sig = (mag & 0x7fffffu) | 0x800000u; /* 24-bit significand, value = sig * 2^(e-23) */
  int shift;                                    /* bits of sig dropped by the target format   */
  if (e >= -14) shift = 13;                     /* normal half: keeps 11 significant bits     */
  else shift = 13 + (-14 - e);                  /* subnormal half: quantum is fixed at 2^-24  */
  if (shift > 25) return (uint16_t)sign;        /* below half of the smallest subnormal       */
  uint32_t kept = sig >> shift;
  uint32_t rem = sig & ((1u << shift) - 1u);
  uint32_t half = 1u << (shift - 1);
  if (rem > half || (rem == half && (kept & 1u))) kept += 1u;
  uint32_t h;
  if (e >= -14) {
    /* kept is in [2^10, 2^11]; adding the exponent field lets a carry bump the exponent. */
    h = ((uint32_t)(e + 15) << 10) + (kept - 0x400u);
  } else {
    h = kept;                                   /* subnormal (or 0x400 = smallest normal)     */
  }
  if (h >= 0x7c00u) h = 0x7c00u;
  return (uint16_t)(sign | h);
}

float tahqo_f16_to_f32(uint16_t h) {
  uint32_t sign = ((uint32_t)h & 0x8000u) << 16;
  uint32_t ex = (h >> 10) & 0x1fu;
  uint32_t fr = h & 0x3ffu;
  float mag;
  if (ex == 0) mag = ldexpf((float)fr, -24);
  else if (ex == 31) mag = fr ? NAN : INFINITY;
  else mag = ldexpf((float)(fr | 0x400u), (int)ex - 25);
  return bits_f32(f32_bits(mag) | sign);
}

/* binary32 -> bfloat16, round-to-nearest-even (receiver output when dtype is bf16). */
uint16_t tahqo_f32_to_bf16(float x) {
  uint32_t u = f32_bits(x);
  if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x40u);
  uint32_t lsb = (u >> 16) & 1u;
  u += 0x7fffu + lsb;
  return (uint16_t)(u >> 16);
}

static float bf16_to_f32(uint16_t b) { return bits_f32((uint32_t)b << 16); }

/* ------------------------------------------------------------------ */
/* Layout of the packed buffer (Sec. 3.4: one contiguous uint8 stream  */
/* whose size depends on the configuration only, never on the data)    */
/* ------------------------------------------------------------------ */

#define TAHQO_ALIGN 128u
#define TAHQO_HEADER_BYTES 128u
#define TAHQO_MAGIC 0x51484154u /* bytes 'T','A','H','Q' */

static uint64_t align_up(uint64_t x) { return (x + (TAHQO_ALIGN - 1)) & ~(uint64_t)(TAHQO_ALIGN - 1); }

int tahqo_layout_of(const tahqo_params *p, tahqo_layout *L) {
  if (!p || !L) return 1;
  uint32_t G = p->tile;
  if (G < 8 || G > 128 || (G & (G - 1))) return 1;          /* Sylvester H_G needs a power of two */
  if (p->dtype > 1 || p->rounding > 1) return 1;
  if (p->tokens == 0 || p->hidden == 0 || p->hidden % G) return 1;
  uint64_t S = p->group_tokens ? p->group_tokens : p->tokens;
  if (p->tokens % S) return 1;
  uint32_t beta = p->budget_millibits;
  if (beta < 2000 || beta > 8000) return 1;
  uint32_t lo = beta / 1000, f = beta % 1000;
  uint64_t M = p->hidden / G;                                 /* quantisation tiles per token */
  uint32_t A = p->alloc_tile ? p->alloc_tile : G;             /* allocation-tile width (Sec. 3.2) */
  if (A % G || A > p->hidden || p->hidden % A) return 1;
  uint64_t m = A / G;                                         /* quantisation tiles per allocation tile */
  L->n_tiles = p->tokens * M;
  L->tiles_per_group = S * M;
  L->n_groups = p->tokens / S;
  /* "the SM allocation tiles of every sample" (M = C/A here): top-p% of them, p = f/10 percent, never
   * more than the budget allows; every quantisation tile inside a chosen allocation tile gets hi */
  uint64_t alloc_per_group = S * (p->hidden / A);
  L->k_hi = ((alloc_per_group * (uint64_t)f) / 1000u) * m;
  L->lo_bits = lo;
  L->hi_bits = f ? lo + 1 : lo;
  L->payload_bytes = L->n_groups * (uint64_t)(G / 8) * (L->tiles_per_group * lo + L->k_hi);
  L->off_bitmap = TAHQO_HEADER_BYTES;
  L->off_scale_zero = align_up(L->off_bitmap + (L->n_tiles + 7) / 8);
  L->off_pivot = align_up(L->off_scale_zero + 4 * L->n_tiles);
  L->off_payload = align_up(L->off_pivot + L->n_tiles);
  L->total_bytes = align_up(L->off_payload + L->payload_bytes);
  return 0;
}

size_t tahqo_packed_bound(const tahqo_params *p) {
  tahqo_layout L;
  if (tahqo_layout_of(p, &L)) return 0;
  return (size_t)L.total_bytes;
}

static void put32(uint8_t *b, uint32_t v) { for (int i = 0; i < 4; i++) b[i] = (uint8_t)(v >> (8 * i)); }
static void put64(uint8_t *b, uint64_t v) { for (int i = 0; i < 8; i++) b[i] = (uint8_t)(v >> (8 * i)); }
static uint32_t get32(const uint8_t *b) { uint32_t v = 0; for (int i = 0; i < 4; i++) v |= (uint32_t)b[i] << (8 * i); return v; }
static uint64_t get64(const uint8_t *b) { uint64_t v = 0; for (int i = 0; i < 8; i++) v |= (uint64_t)b[i] << (8 * i); return v; }

static void write_header(const tahqo_params *p, const tahqo_layout *L, uint8_t *h) {
  memset(h, 0, TAHQO_HEADER_BYTES);
  put32(h + 0, TAHQO_MAGIC);
  put32(h + 4, 1u); /* format version */
  put32(h + 8, p->dtype);
  put32(h + 12, p->rounding);
  put64(h + 16, p->tokens);
  put32(h + 24, p->hidden);
  put32(h + 28, p->tile);
  put32(h + 32, (uint32_t)(L->tiles_per_group / (p->hidden / p->tile))); /* resolved S */
  put32(h + 36, p->budget_millibits);
  put32(h + 40, f32_bits(p->tau));
  put32(h + 44, f32_bits(p->eps_l1));
  put32(h + 48, f32_bits(p->eps_log));
  put32(h + 52, f32_bits(p->eps_ratio));
  put64(h + 56, p->seed);
  put64(h + 64, L->n_tiles);
  put64(h + 72, L->payload_bytes);
  put64(h + 80, L->total_bytes);
  put32(h + 88, (p->alloc_tile && p->alloc_tile != p->tile) ? p->alloc_tile : 0u);   /* 0: A = G */
}

/* ------------------------------------------------------------------ */
/* Steps                                                               */
/* ------------------------------------------------------------------ */

/* Fixed pairwise summation tree over n values: neighbours first, then
 * neighbours of the partial sums, ... (a partial sum without a neighbour
 * waits for the next level).  Fixing the order makes every score a single
 * well-defined binary32 number (the paper does not give an order). */
float tahqo_treesum(const float *x, uint32_t n) {
  float small[128] = {0};
  float *t = n <= 128 ? small : (float *)malloc((size_t)n * sizeof(float));
  for (uint32_t i = 0; i < n; i++) t[i] = x[i];
  for (uint32_t h = 1; h < n; h *= 2)
    for (uint32_t i = 0; i + h < n; i += 2 * h) t[i] = t[i] + t[i + h];
  float r = t[0];
  if (t != small) free(t);
  return r;
}

/* log2 of a positive normal binary32 number: exponent + u*Q(u), u = mantissa-1
 * in [0,1), Q a fixed degree-5 polynomial (Horner, fused multiply-adds).
 * |error| < 3e-6 (plus half an ulp of the result) against log2; exact at powers of two.  The paper's "log" has
 * no stated base or evaluation; a fixed formula makes the ranking of Sec. 3.2
 * reproducible bit for bit, and the base only rescales the score. */
static float oracle_lg2(float x) {
  uint32_t xi = f32_bits(x);
  int e = (int)(xi >> 23) - 127;
  float m = bits_f32((xi & 0x007fffffu) | 0x3f800000u);
  float u = m - 1.0f;
  float q = -0x1.a762d6p-6f;
  q = fmaf(q, u, 0x1.f2e252p-4f);
  q = fmaf(q, u, -0x1.1c9334p-2f);
  q = fmaf(q, u, 0x1.d487c6p-2f);
  q = fmaf(q, u, -0x1.6fb0bcp-1f);
  q = fmaf(q, u, 0x1.714aa0p+0f);
  return fmaf(u, q, (float)e);
}

void tahqo_lg2_array(const float *x, float *y, size_t n) {
  for (size_t i = 0; i < n; i++) y[i] = oracle_lg2(x[i]);
}

/* Eq. 1 and Eq. 2 on one raw (untransformed) tile.  Eq. 2 is printed without
 * a minus sign, but the text under it says the score is high for evenly
 * spread energy and low for a sharp outlier, which is Shannon's sign; the
 * score is therefore -sum p log2(p + varsigma). */
float tahqo_score(const float *tile, uint32_t G, float eps_l1, float eps_log) {
  /* G is the width of the allocation tile the score is taken over (A of Sec. 3.2; = the quantisation
   * tile by default) */
  float sa[128] = {0}, st[128] = {0};
  float *a = G <= 128 ? sa : (float *)malloc((size_t)G * sizeof(float));
  float *term = G <= 128 ? st : (float *)malloc((size_t)G * sizeof(float));
  for (uint32_t k = 0; k < G; k++) a[k] = fabsf(tile[k]);
  float L1 = tahqo_treesum(a, G);
  float inv = 1.0f / (L1 + eps_l1);
  for (uint32_t k = 0; k < G; k++) {
    float p = a[k] * inv;                     /* Eq. 1 */
    term[k] = p * oracle_lg2(p + eps_log);    /* summand of Eq. 2 */
  }
  float r = 0.0f - tahqo_treesum(term, G);
  if (a != sa) { free(a); free(term); }
  return r;
}

/* Sec. 3.2 "Top-p% tile selection" inside one ranking group: sort the tiles by
 * score (highest first; equal scores keep the lower tile index first) and give
 * the first k_hi the higher width. */
typedef struct { float score; uint64_t idx; } ranked;
static int ranked_cmp(const void *pa, const void *pb) {
  const ranked *a = (const ranked *)pa, *b = (const ranked *)pb;
  if (a->score > b->score) return -1;
  if (a->score < b->score) return 1;
  return (a->idx > b->idx) - (a->idx < b->idx);
}
void tahqo_allocate(const float *score, uint64_t n, uint64_t k_hi, uint8_t *is_hi) {
  ranked *r = (ranked *)malloc((size_t)n * sizeof(ranked));
  for (uint64_t i = 0; i < n; i++) { r[i].score = score[i]; r[i].idx = i; is_hi[i] = 0; }
  qsort(r, (size_t)n, sizeof(ranked), ranked_cmp);
  for (uint64_t i = 0; i < k_hi; i++) is_hi[r[i].idx] = 1;
  free(r);
}

/* Eq. 3: ratio of the largest to the second-largest magnitude against tau.
 * d is the first index that attains the maximum; the "second largest" is the
 * largest magnitude among the other G-1 positions.  r > tau is tested without
 * a division as |a(1)| > tau * (|a(2)| + varrho). */
void tahqo_pivot(const float *tile, uint32_t G, float tau, float eps_ratio, uint32_t *d, int *flag) {
  uint32_t dd = 0;
  float a1 = fabsf(tile[0]);
  for (uint32_t k = 1; k < G; k++)
    if (fabsf(tile[k]) > a1) { a1 = fabsf(tile[k]); dd = k; }
  float a2 = 0.0f;
  for (uint32_t k = 0; k < G; k++)
    if (k != dd && fabsf(tile[k]) > a2) a2 = fabsf(tile[k]);
  float t1 = a2 + eps_ratio;
  float t2 = tau * t1;
  *d = dd;
  *flag = a1 > t2;
}

/* Eq. 4: alpha P_d (1/sqrt G) H_G with H_G the Sylvester matrix, applied as the
 * in-place butterfly (strides 1, 2, 4, ...), then one multiply by (float)(1/sqrt G).
 * H_G is symmetric, so the receiver applies the same butterfly and the same swap. */
static void butterfly_scale(float *x, uint32_t G) {
  for (uint32_t h = 1; h < G; h *= 2)
    for (uint32_t i = 0; i < G; i++)
      if (!(i & h)) {
        float a = x[i], b = x[i + h];
        x[i] = a + b;
        x[i + h] = a - b;
      }
  float c = (float)(1.0 / sqrt((double)G));
  for (uint32_t i = 0; i < G; i++) x[i] = x[i] * c;
}
void tahqo_swap_hadamard(float *x, uint32_t G, uint32_t d) {
  float t = x[0]; x[0] = x[d]; x[d] = t;       /* P_d */
  butterfly_scale(x, G);
}

/* "Standard asymmetric quantizer" of Sec. 3.3 as min-max affine quantisation:
 * zero-point z = min (kept in the value domain), scale s = (max - z)/(2^b - 1),
 * both stored in binary16 (16 + 16 + 1 + 6 bits of metadata per 64-wide tile is
 * the 0.61 bits/element of Sec. 3.4); the encoder quantises against the STORED
 * z and s so that sender and receiver use the same numbers. */
void tahqo_range(const float *v, uint32_t G, uint32_t bits, uint16_t *s_h, uint16_t *z_h) {
  float mn = v[0], mx = v[0];
  for (uint32_t k = 1; k < G; k++) { if (v[k] < mn) mn = v[k]; if (v[k] > mx) mx = v[k]; }
  mn = mn + 0.0f;                                /* -0 -> +0 */
  if (mn < -65504.0f) mn = -65504.0f;
  if (mn > 65504.0f) mn = 65504.0f;
  uint16_t zh = tahqo_f32_to_f16(mn);
  float z = tahqo_f16_to_f32(zh);
  float qmax = (float)((1u << bits) - 1u);
  float s = (mx - z) / qmax;
  if (!(s > 0.0f)) s = 0.0f;                     /* stored z may sit above max on a flat tile */
  if (s > 65504.0f) s = 65504.0f;
  *s_h = tahqo_f32_to_f16(s);
  *z_h = zh;
}

/* Philox4x32 with 10 rounds (Salmon et al., SC'11), the counter-based generator
 * behind the optional stochastic rounding. */
void tahqo_philox4x32_10(const uint32_t key[2], const uint32_t ctr[4], uint32_t out[4]) {
  uint32_t k0 = key[0], k1 = key[1];
  uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
  for (int r = 0; r < 10; r++) {
    uint64_t p0 = (uint64_t)0xD2511F53u * c0;
    uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
    uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
    uint32_t n1 = (uint32_t)p1;
    uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
    uint32_t n3 = (uint32_t)p0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    k0 += 0x9E3779B9u; k1 += 0xBB67AE85u;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* q_k = clamp(round((v_k - z) / s), 0, 2^b - 1), the division done as a
 * multiplication by the binary32 reciprocal of the stored scale.  The
 * difference d = v_k - z is a binary32 subtraction; the product d * inv_s is
 * taken EXACTLY (two binary32 factors multiply exactly in binary64) and rounded
 * once, to the nearest integer, ties to even.
 * rounding 0: as above.  rounding 1: floor(y + u) on the binary32 product y,
 * u uniform in [0,1) with 24 bits, taken from word (i mod 4) of
 * Philox(key = seed, counter = i/4) where i = first_elem + k is the element's
 * index in the whole tensor. */
void tahqo_quantise(const float *v, uint32_t G, uint32_t bits, uint16_t s_h, uint16_t z_h,
                    uint32_t rounding, uint64_t seed, uint64_t first_elem, uint32_t *q) {
  float s = tahqo_f16_to_f32(s_h), z = tahqo_f16_to_f32(z_h);
  float inv_s = s > 0.0f ? 1.0f / s : 0.0f;
  float qmax = (float)((1u << bits) - 1u);
  for (uint32_t k = 0; k < G; k++) {
    float d = v[k] - z;
    if (rounding == 0) {
      double y = (double)d * (double)inv_s;       /* exact */
      if (!(y > 0.0)) y = 0.0;
      if (y > (double)qmax) y = (double)qmax;
      q[k] = (uint32_t)rint(y);                    /* default rounding mode: nearest, ties to even */
    } else {
      float y = d * inv_s;
      if (!(y > 0.0f)) y = 0.0f;
      if (y > qmax) y = qmax;
      uint64_t i = first_elem + k, c = i / 4;
      uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
      uint32_t ctr[4] = { (uint32_t)c, (uint32_t)(c >> 32), 0u, 0u };
      uint32_t w[4];
      tahqo_philox4x32_10(key, ctr, w);
      float u = (float)(w[i & 3] >> 8) * 0x1p-24f;
      float r = floorf(y + u);
      if (r > qmax) r = qmax;
      q[k] = (uint32_t)r;
    }
  }
}

/* ------------------------------------------------------------------ */
/* Whole-tensor encode                                                 */
/* ------------------------------------------------------------------ */

static void load_tile(const tahqo_params *p, const void *in, uint64_t t, float *x) {
  uint32_t G = p->tile;
  /* row-major [tokens x hidden] with G | hidden: tile t is elements [t*G, (t+1)*G) (Sec. 3.1) */
  if (p->dtype == TAHQO_F32) {
    const float *src = (const float *)in + t * G;
    for (uint32_t k = 0; k < G; k++) x[k] = src[k];
  } else {
    const uint16_t *src = (const uint16_t *)in + t * G;
    for (uint32_t k = 0; k < G; k++) x[k] = bf16_to_f32(src[k]);
  }
}

/* Little-endian bit stream: code k of a b-bit tile occupies stream bits [k*b, (k+1)*b). */
static void put_bits(uint8_t *dst, uint64_t bitpos, uint32_t nbits, uint32_t v) {
  for (uint32_t j = 0; j < nbits; j++, bitpos++)
    if ((v >> j) & 1u) dst[bitpos >> 3] |= (uint8_t)(1u << (bitpos & 7));
}
static uint32_t get_bits(const uint8_t *src, uint64_t bitpos, uint32_t nbits) {
  uint32_t v = 0;
  for (uint32_t j = 0; j < nbits; j++, bitpos++)
    v |= (uint32_t)((src[bitpos >> 3] >> (bitpos & 7)) & 1u) << j;
  return v;
}

int tahqo_encode(const tahqo_params *p, const void *in, uint8_t *packed, size_t cap) {
  tahqo_layout L;
  if (tahqo_layout_of(p, &L) || !in || !packed) return 1;
  if (cap < L.total_bytes) return 3;
  const uint32_t G = p->tile;
  const uint64_t n = L.n_tiles, ng = L.tiles_per_group;
  memset(packed, 0, (size_t)L.total_bytes);
  write_header(p, &L, packed);

  /* Sec. 3.2: entropy score of every allocation tile (A consecutive channels of one token = m
   * consecutive quantisation tiles), top-p% of them per sample, and the chosen width for every
   * quantisation tile inside. */
  uint8_t *is_hi = (uint8_t *)calloc((size_t)n, 1);
  if (L.k_hi > 0) {
    const uint32_t A = p->alloc_tile ? p->alloc_tile : G;
    const uint64_t m = A / G, na = n / m, nag = ng / m;
    float *score = (float *)malloc((size_t)na * sizeof(float));
    uint8_t *a_hi = (uint8_t *)calloc((size_t)na, 1);
#pragma omp parallel for schedule(static)
    for (int64_t t = 0; t < (int64_t)na; t++) {
      float *x = (float *)malloc((size_t)A * sizeof(float));
      for (uint64_t j = 0; j < m; j++) load_tile(p, in, (uint64_t)t * m + j, x + j * G);
      score[t] = tahqo_score(x, A, p->eps_l1, p->eps_log);
      free(x);
    }
#pragma omp parallel for schedule(static)
    for (int64_t g = 0; g < (int64_t)L.n_groups; g++)
      tahqo_allocate(score + (uint64_t)g * nag, nag, L.k_hi / m, a_hi + (uint64_t)g * nag);
    for (uint64_t t = 0; t < n; t++) is_hi[t] = a_hi[t / m];
    free(a_hi);
    free(score);
  }

  /* Byte offset of every tile's codes: exclusive running sum of G*b/8. */
  uint64_t *offset = (uint64_t *)malloc((size_t)n * sizeof(uint64_t));
  uint64_t run = 0;
  for (uint64_t t = 0; t < n; t++) {
    offset[t] = run;
    run += (uint64_t)(G / 8) * (is_hi[t] ? L.hi_bits : L.lo_bits);
    if (is_hi[t]) packed[L.off_bitmap + (t >> 3)] |= (uint8_t)(1u << (t & 7));
  }

  /* Sec. 3.3 per tile, then Sec. 3.4 packing. */
#pragma omp parallel for schedule(static)
  for (int64_t ti = 0; ti < (int64_t)n; ti++) {
    uint64_t t = (uint64_t)ti;
    float x[128];
    uint32_t q[128];
    load_tile(p, in, t, x);
    uint32_t d; int flag;
    tahqo_pivot(x, G, p->tau, p->eps_ratio, &d, &flag);
    if (flag) tahqo_swap_hadamard(x, G, d);
    uint32_t b = is_hi[t] ? L.hi_bits : L.lo_bits;
    uint16_t sh, zh;
    tahqo_range(x, G, b, &sh, &zh);
    tahqo_quantise(x, G, b, sh, zh, p->rounding, p->seed, t * G, q);
    uint8_t *sz = packed + L.off_scale_zero + 4 * t;
    sz[0] = (uint8_t)sh; sz[1] = (uint8_t)(sh >> 8);
    sz[2] = (uint8_t)zh; sz[3] = (uint8_t)(zh >> 8);
    packed[L.off_pivot + t] = flag ? (uint8_t)(0x80u | d) : 0;
    uint8_t *dst = packed + L.off_payload + offset[t];
    for (uint32_t k = 0; k < G; k++) put_bits(dst, (uint64_t)k * b, b, q[k]);
  }
  free(offset);
  free(is_hi);
  return 0;
}

/* ------------------------------------------------------------------ */
/* Whole-tensor decode (Algorithm 1, line 5)                           */
/* ------------------------------------------------------------------ */

int tahqo_decode(const tahqo_params *p, const uint8_t *packed, size_t bytes, void *out) {
  tahqo_layout L;
  if (tahqo_layout_of(p, &L) || !packed || !out) return 1;
  if (bytes < L.total_bytes) return 3;
  /* the header must describe the same configuration */
  if (get32(packed) != TAHQO_MAGIC || get32(packed + 4) != 1u || get32(packed + 8) != p->dtype ||
      get64(packed + 16) != p->tokens || get32(packed + 24) != p->hidden ||
      get32(packed + 28) != p->tile || get32(packed + 36) != p->budget_millibits ||
      get64(packed + 64) != L.n_tiles || get64(packed + 72) != L.payload_bytes)
    return 6;
  const uint32_t G = p->tile;
  const uint64_t n = L.n_tiles;
  uint64_t *offset = (uint64_t *)malloc((size_t)n * sizeof(uint64_t));
  uint64_t run = 0;
  for (uint64_t t = 0; t < n; t++) {
    int hi = (packed[L.off_bitmap + (t >> 3)] >> (t & 7)) & 1;
    offset[t] = run;
    run += (uint64_t)(G / 8) * (hi ? L.hi_bits : L.lo_bits);
  }
  int bad = run != L.payload_bytes;
#pragma omp parallel for schedule(static)
  for (int64_t ti = 0; ti < (int64_t)n; ti++) {
    if (bad) continue;
    uint64_t t = (uint64_t)ti;
    int hi = (packed[L.off_bitmap + (t >> 3)] >> (t & 7)) & 1;
    uint32_t b = hi ? L.hi_bits : L.lo_bits;
    const uint8_t *sz = packed + L.off_scale_zero + 4 * t;
    float s = tahqo_f16_to_f32((uint16_t)(sz[0] | (sz[1] << 8)));
    float z = tahqo_f16_to_f32((uint16_t)(sz[2] | (sz[3] << 8)));
    uint8_t pv = packed[L.off_pivot + t];
    const uint8_t *src = packed + L.off_payload + offset[t];
    float x[128];
    for (uint32_t k = 0; k < G; k++) {
      uint32_t q = get_bits(src, (uint64_t)k * b, b);
      x[k] = fmaf((float)q, s, z);                 /* z + q*s, one rounding */
    }
    if (pv & 0x80u) {
      uint32_t d = pv & 0x7fu;
      butterfly_scale(x, G);                        /* (1/sqrt G) H_G^T, H_G symmetric */
      float tmp = x[0]; x[0] = x[d]; x[d] = tmp;    /* P_d is its own inverse */
    }
    if (p->dtype == TAHQO_F32) {
      float *dst = (float *)out + t * G;
      for (uint32_t k = 0; k < G; k++) dst[k] = x[k];
    } else {
      uint16_t *dst = (uint16_t *)out + t * G;
      for (uint32_t k = 0; k < G; k++) dst[k] = tahqo_f32_to_bf16(x[k]);
    }
  }
  free(offset);
  return bad ? 6 : 0;
}
