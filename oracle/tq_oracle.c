/*
 * tq_oracle.c -- plain CPU oracle for int4 KV-cache quantisation and single-query attention.
 *
 * TEST INFRASTRUCTURE, NOT PRODUCT CODE.  Only the test-suite, the smoke check and the
 * benchmark's CPU-baseline leg may call into this file.  It shares no code, header, table
 * or helper with the CUDA library and must never be used as a fallback for it.
 *
 * What it implements (paper passages):
 *   - per-group asymmetric int4 quantiser, group g = 32 along head_dim       (Sec. 2.1, Eq. 2-3)
 *   - two codes per byte, low nibble = even element                           (Sec. 2.1; nibble
 *     order as implied by the masks of Eq. 4)
 *   - dequant4:  x^ = (q - z) * s                                             (Eq. 3, Sec. 3.1)
 *   - single-query attention softmax(alpha * q K^T) V over dequantised K, V   (Algorithm 1, whose
 *     result is exactly this definition; written here as the plain two-pass definition in fp64)
 *   - split partials (o_c, m_c, l_c) and their reduction                      (Sec. 3.2, Eq. 5)
 *   - GQA head map kv_head = head / (H_q / H_kv)                              (Sec. 3.1)
 *   - sliding window: only the last w tokens are attended                     (Appendix A)
 *   - KV cache size model                                                     (Eq. 1, Table 4)
 *
 * Precision: the quantiser is an encoding and runs in IEEE binary32, round-to-nearest-even,
 * one rounding per written operation, true division, no fused multiply-add (compile with
 * -ffp-contract=off and without -ffast-math).  Attention runs in fp64 on the exact values of
 * the stored codes, scales and zeros.
 *
 * Readings of the paper where it is silent (each is also what the CUDA library does):
 *   scale and zero are stored as fp16 (needed for the stated 3.2x at g = 32); the zero-point is
 *   real-valued, not rounded to an integer; z and q are computed from the STORED (fp16-rounded)
 *   scale; rounding of x/s + z is half-to-even; a group whose scale rounds to zero in fp16
 *   stores s = 1, z = -min and all codes 0; z is clamped to the finite fp16 range.
 *
 * Pins (tests/test_oracle_*.py): fp16 conversions against an independent implementation over
 * all 65536 halves and over ties; Eq. 4 identity over all 65536 words; pack/unpack round trip;
 * Eq. 1 / Table 4 closed forms; |x - x^| <= s/2; nearest-code brute force; constant groups;
 * softmax weights sum to 1; constant-V, S = 1, q = 0, permutation, split and GQA invariances;
 * a blocked log-sum-exp evaluation written in the tests; a library fp64 attention on the
 * dequantised values; the windowed form against full attention over a cache cut to the window.
 * The bit-level operation ORDER of the quantiser (which of several mathematically equal float32
 * evaluation orders) is this build's reading and cannot be pinned
 * by the paper, which prints no worked example.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#define TQO_GROUP 32

/* ---------------------------------------------------------------- fp16 <-> fp32, bit level */

float tqo_half_to_float(uint16_t h) {
  uint32_t sign = (uint32_t)(h & 0x8000u) << 16;
  uint32_t e = (h >> 10) & 0x1Fu;
  uint32_t m = h & 0x3FFu;
  uint32_t bits;
  if (e == 0) {
    if (m == 0) {
      bits = sign;
    } else { /* subnormal half: m * 2^-24, normalise */
      int sh = 0;
      while (!(m & 0x400u)) { m <<= 1; ++sh; }
      m &= 0x3FFu;
      bits = sign | ((uint32_t)(127 - 15 + 1 - sh) << 23) | (m << 13);
    }
  } else if (e == 31) {
    bits = sign | 0x7F800000u | (m << 13);
  } else {
    bits = sign | ((e + 127 - 15) << 23) | (m << 13);
  }
  float f;
  memcpy(&f, &bits, 4);
  return f;
}

/* binary32 -> binary16, round to nearest, ties to even; overflow gives infinity */
uint16_t tqo_float_to_half(float f) {
  uint32_t x;
  memcpy(&x, &f, 4);
  uint16_t sign = (uint16_t)((x >> 16) & 0x8000u);
  x &= 0x7FFFFFFFu;
  if (x >= 0x7F800000u) return (uint16_t)(sign | (x > 0x7F800000u ? 0x7E00u : 0x7C00u));
  if (x >= 0x477FF000u) return (uint16_t)(sign | 0x7C00u); /* >= 65520 rounds to inf */
  if (x < 0x38800000u) {                                   /* below 2^-14: subnormal half */
    int e = (int)(x >> 23);
    int shift = 126 - e; /* result = mantissa24 / 2^shift in units of 2^-24 */
    if (e == 0 || shift > 25) return sign;
    uint32_t m = (x & 0x7FFFFFu) | 0x800000u;
    uint32_t r = m >> shift;
    uint32_t rem = m & ((1u << shift) - 1u);
    uint32_t halfway = 1u << (shift - 1);
    if (rem > halfway || (rem == halfway && (r & 1u))) ++r;
    return (uint16_t)(sign | r);
  }
  uint32_t r = (x - 0x38000000u) >> 13;
  uint32_t rem = x & 0x1FFFu;
  if (rem > 0x1000u || (rem == 0x1000u && (r & 1u))) ++r;
  return (uint16_t)(sign | r);
}

/* ---------------------------------------------------------------- sizes (Eq. 1, Sec. 2.1) */

/* bytes of one K or V vector of d elements in the int4 format: d/2 code bytes + fp16 scale
 * and fp16 zero per group of 32 (20 bytes per 32 elements => 3.2x against fp16). */
int64_t tqo_int4_vector_bytes(int64_t d) { return d / 2 + (d / TQO_GROUP) * 2 + (d / TQO_GROUP) * 2; }

/* Eq. 1: 2 * L * H_kv * S * d * b bytes for K and V together, fp16 (b = 2). */
int64_t tqo_fp16_cache_bytes(int64_t L, int64_t H_kv, int64_t S, int64_t d) { return 2 * L * H_kv * S * d * 2; }

int64_t tqo_int4_cache_bytes(int64_t L, int64_t H_kv, int64_t S, int64_t d) {
  return 2 * L * H_kv * S * tqo_int4_vector_bytes(d);
}

/* ---------------------------------------------------------------- quantiser (Eq. 2-3) */

/* One group of 32 fp16 inputs -> 32 codes (one per byte, unpacked), fp16 scale, fp16 zero. */
void tqo_quantize_group(const uint16_t* x16, uint8_t* codes, uint16_t* scale16, uint16_t* zero16) {
  float x[TQO_GROUP];
  float mn, mx;
  for (int i = 0; i < TQO_GROUP; ++i) x[i] = tqo_half_to_float(x16[i]);
  mn = x[0];
  mx = x[0];
  for (int i = 1; i < TQO_GROUP; ++i) {
    if (x[i] < mn) mn = x[i];
    if (x[i] > mx) mx = x[i];
  }
  float range = mx - mn;
  float s32 = range / 15.0f;               /* s = (max - min) / 15 */
  uint16_t s16 = tqo_float_to_half(s32);   /* stored scale */
  if ((s16 & 0x7FFFu) == 0) {              /* degenerate: scale rounds to zero */
    *scale16 = 0x3C00u;                    /* 1.0 */
    *zero16 = tqo_float_to_half(0.0f - mn);
    for (int i = 0; i < TQO_GROUP; ++i) codes[i] = 0;
    return;
  }
  float sf = tqo_half_to_float(s16);
  float z32 = (0.0f - mn) / sf;            /* z = -min / s, with the stored s */
  if (z32 > 65504.0f) z32 = 65504.0f;
  if (z32 < -65504.0f) z32 = -65504.0f;
  uint16_t z16 = tqo_float_to_half(z32);
  float zf = tqo_half_to_float(z16);
  for (int i = 0; i < TQO_GROUP; ++i) {
    float t = x[i] / sf;
    float u = t + zf;
    float r = rintf(u);                    /* half-to-even under the default rounding mode */
    if (!(r >= 0.0f)) r = 0.0f;            /* also catches NaN */
    if (r > 15.0f) r = 15.0f;
    codes[i] = (uint8_t)(int)r;
  }
  *scale16 = s16;
  *zero16 = z16;
}

/* two codes per byte: byte b = code[2b] | code[2b+1] << 4 */
void tqo_pack_nibbles(const uint8_t* codes, int64_t n, uint8_t* packed) {
  for (int64_t b = 0; b < n / 2; ++b) packed[b] = (uint8_t)((codes[2 * b] & 0xF) | ((codes[2 * b + 1] & 0xF) << 4));
}

void tqo_unpack_nibbles(const uint8_t* packed, int64_t n, uint8_t* codes) {
  for (int64_t b = 0; b < n / 2; ++b) {
    codes[2 * b] = packed[b] & 0xF;
    codes[2 * b + 1] = packed[b] >> 4;
  }
}

/* rows: [n_rows][d] fp16 -> packed [n_rows][d/2], scale/zero [n_rows][d/32] */
void tqo_quantize_rows(const uint16_t* x16, int64_t n_rows, int64_t d, uint8_t* packed, uint16_t* scale16,
                       uint16_t* zero16) {
  int64_t ng = d / TQO_GROUP;
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < n_rows; ++r) {
    uint8_t codes[TQO_GROUP];
    for (int64_t g = 0; g < ng; ++g) {
      tqo_quantize_group(x16 + r * d + g * TQO_GROUP, codes, scale16 + r * ng + g, zero16 + r * ng + g);
      tqo_pack_nibbles(codes, TQO_GROUP, packed + r * (d / 2) + g * (TQO_GROUP / 2));
    }
  }
}

/* dequant4 of one row into fp64: x^[c] = (q[c] - z[c/32]) * s[c/32], exact in fp64 */
void tqo_dequant_row(const uint8_t* packed, const uint16_t* scale16, const uint16_t* zero16, int64_t d, double* out) {
  for (int64_t c = 0; c < d; ++c) {
    uint8_t byte = packed[c / 2];
    int code = (c & 1) ? (byte >> 4) : (byte & 0xF);
    double s = (double)tqo_half_to_float(scale16[c / TQO_GROUP]);
    double z = (double)tqo_half_to_float(zero16[c / TQO_GROUP]);
    out[c] = ((double)code - z) * s;
  }
}

void tqo_dequant_rows(const uint8_t* packed, const uint16_t* scale16, const uint16_t* zero16, int64_t n_rows,
                      int64_t d, double* out) {
  int64_t ng = d / TQO_GROUP;
#pragma omp parallel for schedule(static)
  for (int64_t r = 0; r < n_rows; ++r)
    tqo_dequant_row(packed + r * (d / 2), scale16 + r * ng, zero16 + r * ng, d, out + r * d);
}

/* Append T new tokens per (b, kv head) at position lens[b]; lens[b] += T.  A sequence that
 * would overflow S_cap is left untouched and its bit is set in the returned mask count.
 * cache arrays: packed [B][H_kv][S_cap][d/2], scale/zero [B][H_kv][S_cap][d/32];
 * x_new: [B][H_kv][T][d] fp16.  Returns the number of sequences skipped for overflow. */
int tqo_quantize_append(uint8_t* packed, uint16_t* scale16, uint16_t* zero16, int32_t* lens, int64_t B, int64_t H_kv,
                        int64_t S_cap, int64_t d, const uint16_t* x_new, int64_t T, int update_lens) {
  int64_t ng = d / TQO_GROUP;
  int skipped = 0;
  for (int64_t b = 0; b < B; ++b) {
    int64_t len = lens[b];
    if (len < 0 || len + T > S_cap) { ++skipped; continue; }
    for (int64_t h = 0; h < H_kv; ++h) {
      int64_t row0 = (b * H_kv + h) * S_cap + len;
      tqo_quantize_rows(x_new + ((b * H_kv + h) * T) * d, T, d, packed + row0 * (d / 2), scale16 + row0 * ng,
                        zero16 + row0 * ng);
    }
    if (update_lens) lens[b] = (int32_t)(len + T);
  }
  return skipped;
}

/* ---------------------------------------------------------------- attention */

typedef struct {
  const uint8_t *k_packed, *v_packed;  /* [B][H_kv][S_cap][d/2] */
  const uint16_t *k_scale, *k_zero;    /* [B][H_kv][S_cap][d/32] */
  const uint16_t *v_scale, *v_zero;
  const int32_t* lens;                 /* [B] */
  int64_t B, H_kv, S_cap, d;
} tqo_cache;

static void fill_cache(tqo_cache* c, const uint8_t* kp, const uint16_t* ks, const uint16_t* kz, const uint8_t* vp,
                       const uint16_t* vs, const uint16_t* vz, const int32_t* lens, int64_t B, int64_t H_kv,
                       int64_t S_cap, int64_t d) {
  c->k_packed = kp; c->k_scale = ks; c->k_zero = kz;
  c->v_packed = vp; c->v_scale = vs; c->v_zero = vz;
  c->lens = lens; c->B = B; c->H_kv = H_kv; c->S_cap = S_cap; c->d = d;
}

static void dequant_token(const tqo_cache* c, int is_v, int64_t b, int64_t kvh, int64_t i, double* out) {
  int64_t ng = c->d / TQO_GROUP;
  int64_t row = (b * c->H_kv + kvh) * c->S_cap + i;
  if (is_v)
    tqo_dequant_row(c->v_packed + row * (c->d / 2), c->v_scale + row * ng, c->v_zero + row * ng, c->d, out);
  else
    tqo_dequant_row(c->k_packed + row * (c->d / 2), c->k_scale + row * ng, c->k_zero + row * ng, c->d, out);
}

/* Two-pass definition on tokens [t0, t1) of sequence b for query head h.
 * Writes the normalised output o (d doubles), the maximum score m and the sum of exponentials l
 * (the partial triple of Sec. 3.2).  An empty range gives o = 0, m = -inf, l = 0.
 * If weights != NULL it receives the t1 - t0 softmax weights p_i / l. */
static void attend_range(const tqo_cache* c, const uint16_t* q16, int64_t H_q, double alpha, int64_t b, int64_t h,
                         int64_t t0, int64_t t1, double* o, double* m_out, double* l_out, double* weights) {
  int64_t d = c->d;
  int64_t kvh = h / (H_q / c->H_kv); /* GQA map */
  int64_t n = t1 > t0 ? t1 - t0 : 0;
  for (int64_t x = 0; x < d; ++x) o[x] = 0.0;
  if (n == 0) { *m_out = -INFINITY; *l_out = 0.0; return; }
  double* a = (double*)malloc((size_t)n * sizeof(double));
  double* row = (double*)malloc((size_t)d * sizeof(double));
  double* qd = (double*)malloc((size_t)d * sizeof(double));
  for (int64_t x = 0; x < d; ++x) qd[x] = (double)tqo_half_to_float(q16[(b * H_q + h) * d + x]);
  double M = -INFINITY;
  for (int64_t i = 0; i < n; ++i) {
    dequant_token(c, 0, b, kvh, t0 + i, row);
    double dot = 0.0;
    for (int64_t x = 0; x < d; ++x) dot += qd[x] * row[x];
    a[i] = alpha * dot;
    if (a[i] > M) M = a[i];
  }
  double L = 0.0;
  for (int64_t i = 0; i < n; ++i) { a[i] = exp(a[i] - M); L += a[i]; }
  for (int64_t i = 0; i < n; ++i) {
    double w = a[i] / L;
    if (weights) weights[i] = w;
    dequant_token(c, 1, b, kvh, t0 + i, row);
    for (int64_t x = 0; x < d; ++x) o[x] += w * row[x];
  }
  *m_out = M;
  *l_out = L;
  free(a); free(row); free(qd);
}

/* out: [B][H_q][d] fp64.  Heads h in [h_begin, h_end) only (others untouched); sequences with
 * lens[b] == 0 give zeros. */
void tqo_attention(const uint8_t* kp, const uint16_t* ks, const uint16_t* kz, const uint8_t* vp, const uint16_t* vs,
                   const uint16_t* vz, const int32_t* lens, int64_t B, int64_t H_kv, int64_t S_cap, int64_t d,
                   const uint16_t* q16, int64_t H_q, double alpha, int64_t h_begin, int64_t h_end, double* out) {
  tqo_cache c;
  fill_cache(&c, kp, ks, kz, vp, vs, vz, lens, B, H_kv, S_cap, d);
  int64_t nh = h_end - h_begin;
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t bh = 0; bh < B * nh; ++bh) {
    int64_t b = bh / nh, h = h_begin + bh % nh;
    double m, l;
    attend_range(&c, q16, H_q, alpha, b, h, 0, lens[b], out + (b * H_q + h) * d, &m, &l, NULL);
  }
}

/* Sliding window (Appendix A): sequence b attends tokens [max(0, lens[b] - window), lens[b]);
 * window <= 0 means all tokens.  out: [B][H_q][d] fp64. */
void tqo_attention_window(const uint8_t* kp, const uint16_t* ks, const uint16_t* kz, const uint8_t* vp,
                          const uint16_t* vs, const uint16_t* vz, const int32_t* lens, int64_t B, int64_t H_kv,
                          int64_t S_cap, int64_t d, const uint16_t* q16, int64_t H_q, double alpha, int64_t window,
                          double* out) {
  tqo_cache c;
  fill_cache(&c, kp, ks, kz, vp, vs, vz, lens, B, H_kv, S_cap, d);
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t bh = 0; bh < B * H_q; ++bh) {
    int64_t b = bh / H_q, h = bh % H_q;
    int64_t begin = (window > 0 && window < lens[b]) ? lens[b] - window : 0;
    double m, l;
    attend_range(&c, q16, H_q, alpha, b, h, begin, lens[b], out + (b * H_q + h) * d, &m, &l, NULL);
  }
}

/* softmax weights of one (b, h): weights[lens[b]] */
void tqo_attention_weights(const uint8_t* kp, const uint16_t* ks, const uint16_t* kz, const uint8_t* vp,
                           const uint16_t* vs, const uint16_t* vz, const int32_t* lens, int64_t B, int64_t H_kv,
                           int64_t S_cap, int64_t d, const uint16_t* q16, int64_t H_q, double alpha, int64_t b,
                           int64_t h, double* weights) {
  tqo_cache c;
  fill_cache(&c, kp, ks, kz, vp, vs, vz, lens, B, H_kv, S_cap, d);
  double m, l;
  double* o = (double*)malloc((size_t)d * sizeof(double));
  attend_range(&c, q16, H_q, alpha, b, h, 0, lens[b], o, &m, &l, weights);
  free(o);
}

/* Partials of Sec. 3.2 for caller-given split boundaries: bounds is [B][C+1], split c of
 * sequence b covers tokens [bounds[b][c], bounds[b][c+1]).
 * o_part [B][H_q][C][d], m_part, l_part [B][H_q][C]. */
void tqo_attention_partials(const uint8_t* kp, const uint16_t* ks, const uint16_t* kz, const uint8_t* vp,
                            const uint16_t* vs, const uint16_t* vz, const int32_t* lens, int64_t B, int64_t H_kv,
                            int64_t S_cap, int64_t d, const uint16_t* q16, int64_t H_q, double alpha, int64_t C,
                            const int32_t* bounds, double* o_part, double* m_part, double* l_part) {
  tqo_cache c;
  fill_cache(&c, kp, ks, kz, vp, vs, vz, lens, B, H_kv, S_cap, d);
#pragma omp parallel for schedule(dynamic, 1)
  for (int64_t idx = 0; idx < B * H_q * C; ++idx) {
    int64_t s = idx % C, h = (idx / C) % H_q, b = idx / (C * H_q);
    attend_range(&c, q16, H_q, alpha, b, h, bounds[b * (C + 1) + s], bounds[b * (C + 1) + s + 1],
                 o_part + idx * d, m_part + idx, l_part + idx, NULL);
  }
}

/* Eq. 5: o = sum_c l_c e^{m_c - m_g} o_c / sum_c l_c e^{m_c - m_g}; splits with l_c = 0 are
 * skipped; if every split is empty the output is zero. */
void tqo_combine(const double* o_part, const double* m_part, const double* l_part, int64_t B, int64_t H_q, int64_t C,
                 int64_t d, double* out) {
  for (int64_t bh = 0; bh < B * H_q; ++bh) {
    const double* m = m_part + bh * C;
    const double* l = l_part + bh * C;
    double mg = -INFINITY;
    for (int64_t c = 0; c < C; ++c)
      if (l[c] > 0.0 && m[c] > mg) mg = m[c];
    double den = 0.0;
    for (int64_t x = 0; x < d; ++x) out[bh * d + x] = 0.0;
    if (mg == -INFINITY) continue;
    for (int64_t c = 0; c < C; ++c) {
      if (!(l[c] > 0.0)) continue;
      double w = l[c] * exp(m[c] - mg);
      den += w;
      for (int64_t x = 0; x < d; ++x) out[bh * d + x] += w * o_part[(bh * C + c) * d + x];
    }
    for (int64_t x = 0; x < d; ++x) out[bh * d + x] /= den;
  }
}

int tqo_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}
