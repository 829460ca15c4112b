/*
 * CPU oracle for the QK4PV8 mixed-precision attention forward.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, step-by-step CPU
 * statement of what the CUDA library must compute.  It shares no code with the
 * CUDA path and must never be linked or imported by it.  It follows the paper's
 * Algorithm 1 and Sections 2.1 / 4.1-4.3 / 5.3 in the paper's order, emulating
 * every rounding explicitly:
 *   - all arithmetic is IEEE binary32, round-to-nearest-even, no FMA contraction
 *     (compile with -ffp-contract=off), except where "double" is written out;
 *   - quantizer outputs (means, tensor scales, E4M3 block scales, E2M1 codes,
 *     E4M3 V codes, BF16 compensation vector) are defined bit by bit;
 *   - the attention main loop is defined up to FP32 summation order.
 *
 * Pins (tests/test_oracle_*.py): brute-force nearest-value enumeration of all
 * 16 E2M1 and 256 E4M3 codes, exact integer column sums, Eq. 8 identity in
 * FP64, the identity-quantizer special case against textbook FP64 softmax
 * attention, softmax rows summing to one, traversal-order invariance in FP64;
 * the reverse block order, the fixed scale 448 of P-hat (codes of a worked row,
 * subnormal codes included) and the GQA head mapping against NumPy statements
 * of the same steps on operands built code by code; the NVFP4 + NVFP4 assignment
 * (token-axis V quantizer, block-scaled P) against NumPy statements of its steps.
 * Parity unpinned (the paper prints no worked example for them, they are
 * readings fixed by this file): the per-tensor scale recipe, reciprocal-multiply
 * element scaling, the unit in which the compensation vector is stored, FP32
 * summation orders.
 *
 * Build: gcc -O2 -std=c11 -ffp-contract=off -fno-fast-math -fopenmp -shared -fPIC
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#define D 128          /* head dimension (the paper evaluates d = 128 only, Section 7.1) */
#define G 16           /* NVFP4 block size along the head dimension (Section 2.1, Eq. 1) */
#define NBLK (D / G)   /* 8 scale factors per (token, head) row */

/* ------------------------------------------------------------------------- */
/* number formats                                                            */
/* ------------------------------------------------------------------------- */

float mpfa_oracle_bf16_to_f32(uint16_t h) {
  uint32_t u = (uint32_t)h << 16;
  float f;
  memcpy(&f, &u, 4);
  return f;
}

/* FP32 -> BF16, round to nearest even (inputs are never NaN on this path). */
uint16_t mpfa_oracle_f32_to_bf16(float f) {
  uint32_t u;
  memcpy(&u, &f, 4);
  uint32_t lsb = (u >> 16) & 1u;
  u += 0x7FFFu + lsb;
  return (uint16_t)(u >> 16);
}

/* E4M3 ("fn" flavour: bias 7, no infinity, largest finite value 448, S.1111.111 = NaN). */
float mpfa_oracle_e4m3_decode(uint8_t c) {
  int s = c >> 7, e = (c >> 3) & 15, m = c & 7;
  float v = (e == 0) ? ldexpf((float)m, -9) : ldexpf((float)(8 + m), e - 10);
  return s ? -v : v;
}

/* FP32 -> E4M3, round to nearest even, saturating to +-448 (never produces NaN).
 * Step: scale the magnitude so that one code step is 1.0, round with rint()
 * (ties to even integer == ties to even code, because codes are consecutive
 * integers in magnitude order), let a mantissa carry roll into the exponent. */
uint8_t mpfa_oracle_e4m3_encode(float x) {
  uint8_t sign = signbit(x) ? 0x80 : 0;
  float a = fabsf(x);
  int code;
  if (!(a < 464.0f)) {            /* >= midpoint above 448, or NaN: saturate */
    code = 0x7E;
  } else if (a < 0.015625f) {     /* below 2^-6: subnormal step 2^-9 */
    code = (int)rintf(a * 512.0f);           /* 0..8; 8 is the first normal 0x08 */
  } else {
    int ex;
    float fr = frexpf(a, &ex);               /* a = fr * 2^ex, fr in [0.5,1) */
    int e = ex - 1;                          /* a = (2 fr) * 2^e, 2fr in [1,2) */
    int q = (int)rintf((fr * 2.0f - 1.0f) * 8.0f);   /* exact products; 0..8 */
    code = ((e + 7) << 3) + q;               /* q == 8 carries into the exponent */
    if (code > 0x7E) code = 0x7E;
  }
  return (uint8_t)(sign | code);
}

/* E2M1: magnitudes {0, .5, 1, 1.5, 2, 3, 4, 6} = codes 0..7, bit 3 = sign. */
float mpfa_oracle_e2m1_decode(uint8_t c) {
  static const float mag[8] = {0.0f, 0.5f, 1.0f, 1.5f, 2.0f, 3.0f, 4.0f, 6.0f};
  float v = mag[c & 7];
  return (c & 8) ? -v : v;
}

/* FP32 -> E2M1, round to nearest even code, saturating to +-6, sign bit kept
 * (a negative input that rounds to zero gives code 0x8). */
uint8_t mpfa_oracle_e2m1_encode(float y) {
  uint8_t sign = signbit(y) ? 8 : 0;
  float a = fabsf(y);
  int code;
  if (!(a < 5.0f)) {                 /* 5.0 is the 4|6 midpoint and ties to 4 (even code) */
    code = (a == 5.0f) ? 6 : 7;
  } else if (a < 2.0f) {
    code = (int)rintf(a * 2.0f);     /* step 0.5: 0..4 */
  } else if (a < 4.0f) {
    code = 2 + (int)rintf(a);        /* step 1: 2,3,4 -> codes 4,5,6 */
  } else {
    code = 4 + (int)rintf(a * 0.5f); /* [4,5): a/2 in [2,2.5) -> 2 -> code 6 */
  }
  return (uint8_t)(sign | code);
}

/* ------------------------------------------------------------------------- */
/* stage 1: statistics and quantizers (Algorithm 1 lines 1-5)                 */
/* ------------------------------------------------------------------------- */

/* Eq. 7: mean over the N valid tokens, per (batch, head, channel).
 * x: BF16 [B, N, H, D]; mean: FP32 [B, H, D].  FP64 sum, one rounding to FP32. */
void mpfa_oracle_means(const uint16_t *x, int B, int N, int H, float *mean) {
#pragma omp parallel for collapse(2) schedule(static)
  for (int b = 0; b < B; ++b)
    for (int h = 0; h < H; ++h) {
      double s[D];
      for (int c = 0; c < D; ++c) s[c] = 0.0;
      for (int t = 0; t < N; ++t) {   /* tokens ascending, one running FP64 sum per channel */
        const uint16_t *row = x + (((size_t)b * N + t) * H + h) * D;
        for (int c = 0; c < D; ++c) s[c] += (double)mpfa_oracle_bf16_to_f32(row[c]);
      }
      for (int c = 0; c < D; ++c) mean[((size_t)b * H + h) * D + c] = (float)(s[c] / (double)N);
    }
}

/* Same column sums in exact fixed point (units of 2^-40), used only to pin
 * the claim that the FP64 sum above is exact for the generator's inputs. */
void mpfa_oracle_colsum_fixed(const uint16_t *x, int B, int N, int H, int64_t *sum) {
  for (int b = 0; b < B; ++b)
    for (int h = 0; h < H; ++h)
      for (int c = 0; c < D; ++c) {
        int64_t s = 0;
        for (int t = 0; t < N; ++t) {
          double v = (double)mpfa_oracle_bf16_to_f32(x[(((size_t)b * N + t) * H + h) * D + c]);
          s += (int64_t)ldexp(v, 40);
        }
        sum[((size_t)b * H + h) * D + c] = s;
      }
}

/* Per-tensor scale (one per batch element): d = max|x - mean| / (6 * 448).
 * The paper has only the E4M3 block scale; this extra FP32 factor maps the
 * largest block scale of the tensor onto 448 so the E4M3 range is used fully. */
void mpfa_oracle_tensor_scale(const uint16_t *x, const float *mean, int B, int N, int H, float *d) {
  for (int b = 0; b < B; ++b) {
    float amax = 0.0f;
    for (int t = 0; t < N; ++t)
      for (int h = 0; h < H; ++h)
        for (int c = 0; c < D; ++c) {
          float xc = mpfa_oracle_bf16_to_f32(x[(((size_t)b * N + t) * H + h) * D + c]) -
                     mean[((size_t)b * H + h) * D + c];
          float a = fabsf(xc);
          if (a > amax) amax = a;
        }
    d[b] = (amax > 0.0f) ? amax / 2688.0f : 1.0f;
  }
}

/* Eq. 1 with the E4M3 rounding of the block scale made explicit.
 * x: BF16 [B, N, H, D] (token-major, as produced by the model);
 * codes: [B, H, N, D/2] two E2M1 codes per byte, even channel in the low nibble;
 * sf:    [B, H, N, 8] unsigned E4M3 block-scale codes. */
void mpfa_oracle_quantize_nvfp4(const uint16_t *x, const float *mean, const float *d, int B, int N,
                                int H, uint8_t *codes, uint8_t *sf) {
#pragma omp parallel for collapse(2) schedule(static)
  for (int b = 0; b < B; ++b)
    for (int t = 0; t < N; ++t)
      for (int h = 0; h < H; ++h) {
        const uint16_t *row = x + (((size_t)b * N + t) * H + h) * D;
        const float *mu = mean + ((size_t)b * H + h) * D;
        uint8_t *crow = codes + (((size_t)b * H + h) * N + t) * (D / 2);
        uint8_t *srow = sf + (((size_t)b * H + h) * N + t) * NBLK;
        float e = 6.0f * d[b];
        for (int g = 0; g < NBLK; ++g) {
          float xc[G];
          float a = 0.0f;
          for (int i = 0; i < G; ++i) {
            xc[i] = mpfa_oracle_bf16_to_f32(row[g * G + i]) - mu[g * G + i];   /* centering */
            if (fabsf(xc[i]) > a) a = fabsf(xc[i]);
          }
          float r = a / e;                                   /* s_g = amax / rho, in units of d */
          uint8_t sc = mpfa_oracle_e4m3_encode(r);           /* rounded to E4M3, <= 448 */
          float s = mpfa_oracle_e4m3_decode(sc) * d[b];      /* the scale the MMA reconstructs with */
          float inv = 1.0f / s;
          if (!(s > 0.0f) || isinf(inv)) inv = 0.0f;
          srow[g] = sc;
          for (int i = 0; i < G; i += 2) {
            uint8_t lo = mpfa_oracle_e2m1_encode(xc[i] * inv);
            uint8_t hi = mpfa_oracle_e2m1_encode(xc[i + 1] * inv);
            crow[(g * G + i) / 2] = (uint8_t)(lo | (hi << 4));
          }
        }
      }
}

/* Eq. 9: Delta_S[b, hq, j] = qmean[b, hq, :] . (K[b, j, hkv, :] - kmean[b, hkv, :]),
 * stored in the unit of the block-scaled MMA output (true logit / (dQ dK)) and
 * rounded once to BF16 (Section 4.3: "one BF16 rounding").
 * FP64 accumulation, channels ascending.  delta: BF16 [B, Hq, N]. */
void mpfa_oracle_delta_s(const uint16_t *k, const float *q_mean, const float *k_mean, const float *dq,
                         const float *dk, int B, int N, int Hq, int Hkv, uint16_t *delta) {
  int grp = Hq / Hkv;
#pragma omp parallel for collapse(2) schedule(static)
  for (int b = 0; b < B; ++b)
    for (int t = 0; t < N; ++t)
      for (int hq = 0; hq < Hq; ++hq) {
        int hk = hq / grp;
        const uint16_t *row = k + (((size_t)b * N + t) * Hkv + hk) * D;
        const float *mu = k_mean + ((size_t)b * Hkv + hk) * D;
        const float *qm = q_mean + ((size_t)b * Hq + hq) * D;
        double s = 0.0;
        for (int c = 0; c < D; ++c) {
          float kc = mpfa_oracle_bf16_to_f32(row[c]) - mu[c];
          s += (double)qm[c] * (double)kc;
        }
        float v = (float)(s / ((double)dq[b] * (double)dk[b]));
        delta[((size_t)b * Hq + hq) * N + t] = mpfa_oracle_f32_to_bf16(v);
      }
}

/* Algorithm 1 line 4: V is not centered; code = E4M3(v * (1 / v_scale)).
 * v: BF16 [B, N, H, D]; out: [B, H, N, D]. */
void mpfa_oracle_quantize_v(const uint16_t *v, int B, int N, int H, float v_scale, uint8_t *out) {
  float inv = 1.0f / v_scale;
#pragma omp parallel for collapse(2) schedule(static)
  for (int b = 0; b < B; ++b)
    for (int t = 0; t < N; ++t)
      for (int h = 0; h < H; ++h)
        for (int c = 0; c < D; ++c)
          out[(((size_t)b * H + h) * N + t) * D + c] =
              mpfa_oracle_e4m3_encode(mpfa_oracle_bf16_to_f32(v[(((size_t)b * N + t) * H + h) * D + c]) * inv);
}

/* ------------------------------------------------------------------------- */
/* stage 2: attention main loop (Algorithm 1 lines 6-20)                      */
/* ------------------------------------------------------------------------- */

static float e2m1_pair_lo[256], e2m1_pair_hi[256], e4m3_tab[256];
static int tables_ready = 0;
static void init_tables(void) {
  if (tables_ready) return;
  for (int i = 0; i < 256; ++i) {
    e2m1_pair_lo[i] = mpfa_oracle_e2m1_decode((uint8_t)(i & 15));
    e2m1_pair_hi[i] = mpfa_oracle_e2m1_decode((uint8_t)(i >> 4));
    e4m3_tab[i] = mpfa_oracle_e4m3_decode((uint8_t)i);
  }
  tables_ready = 1;
}

/* Eq. 10 / Eq. 11: logits of one query row against keys [0, n_keys), in the
 * unit of the block-scaled MMA (true logit / (dQ dK)):
 *   acc = Delta_S[j]                        (rank-one seed; 0 without compensation)
 *   acc += (sQ_g * sK_g) * sum_i q_gi k_gi  for g = 0..7
 * The 16-term inner sum is exact in FP32 (multiples of 1/4 below 2^10), the
 * scale product is exact (4 x 4 significant bits). */
static void logits_row_q4(const uint8_t *qc, const uint8_t *qs, const uint8_t *kc, const uint8_t *ks,
                          const uint16_t *delta, int n_keys, float *s) {
  float qv[D], qsc[NBLK];
  for (int i = 0; i < D / 2; ++i) {
    qv[2 * i] = e2m1_pair_lo[qc[i]];
    qv[2 * i + 1] = e2m1_pair_hi[qc[i]];
  }
  for (int g = 0; g < NBLK; ++g) qsc[g] = e4m3_tab[qs[g]];
  for (int j = 0; j < n_keys; ++j) {
    const uint8_t *kr = kc + (size_t)j * (D / 2);
    const uint8_t *sr = ks + (size_t)j * NBLK;
    float acc = delta ? mpfa_oracle_bf16_to_f32(delta[j]) : 0.0f;
    for (int g = 0; g < NBLK; ++g) {
      float dot = 0.0f;
      for (int i = 0; i < G / 2; ++i) {
        uint8_t byte = kr[g * (G / 2) + i];
        dot += qv[g * G + 2 * i] * e2m1_pair_lo[byte];
        dot += qv[g * G + 2 * i + 1] * e2m1_pair_hi[byte];
      }
      acc += (qsc[g] * e4m3_tab[sr[g]]) * dot;
    }
    s[j] = acc;
  }
}

/* exp2 of an FP32 argument, correctly rounded to FP32 via double. */
static float exp2_f32(float x) { return (float)exp2((double)x); }

typedef struct {
  float m;      /* running maximum, in logit units of s[] */
  float l;      /* running sum of unquantized P */
  float o[D];   /* running sum of P_hat * V (P_hat carries the factor 448) */
} softmax_state;

/* Online softmax + PV over keys [k0, k1) of one row (Algorithm 1 lines 8-16,
 * Eq. 3-6), KV blocks of `block` keys aligned to multiples of `block` counted
 * from key 0, visited in descending order when `reverse` (Section 4.1).
 * s: logits in MMA units; lam: lambda' = softmax_scale * log2(e) * dQ * dK.
 * v: E4M3 codes [n, D] (v_f32 == NULL) or FP32 values [n, D].
 * p_fp8: quantize P to E4M3 with the fixed scale 448 (else keep FP32 P * 448).
 * phat_out (optional, inspection only): receives, per key index, the E4M3 code
 * the loop gave that key's P when its block was visited.
 * Inspection hooks, used only by mpfa_oracle_phat_rows (NULL / -1 everywhere
 * else, where they change nothing): q_out receives the FP32 value 448 P that
 * was encoded; flip_key >= 0 moves that one key's code by flip_dir steps
 * (to show what a one-step difference in a single P-hat does to a row). */
static void online_softmax_pv_x(const float *s, int k0, int k1, float lam, const uint8_t *v,
                                const float *v_f32, int block, int reverse, int p_fp8,
                                softmax_state *st, uint8_t *phat_out, float *q_out, int flip_key, int flip_dir);

static void online_softmax_pv(const float *s, int k0, int k1, float lam, const uint8_t *v,
                              const float *v_f32, int block, int reverse, int p_fp8,
                              softmax_state *st, uint8_t *phat_out) {
  online_softmax_pv_x(s, k0, k1, lam, v, v_f32, block, reverse, p_fp8, st, phat_out, NULL, -1, 0);
}

static void online_softmax_pv_x(const float *s, int k0, int k1, float lam, const uint8_t *v,
                                const float *v_f32, int block, int reverse, int p_fp8,
                                softmax_state *st, uint8_t *phat_out, float *q_out, int flip_key, int flip_dir) {
  st->m = -INFINITY;
  st->l = 0.0f;
  for (int c = 0; c < D; ++c) st->o[c] = 0.0f;
  if (k1 <= k0) return;
  int jb0 = k0 / block, jb1 = (k1 - 1) / block;
  float *p = (float *)malloc(sizeof(float) * (size_t)block);
  for (int step = 0; step <= jb1 - jb0; ++step) {
    int jb = reverse ? jb1 - step : jb0 + step;
    int a = jb * block < k0 ? k0 : jb * block;
    int b = (jb + 1) * block > k1 ? k1 : (jb + 1) * block;
    float rowmax = -INFINITY;
    for (int j = a; j < b; ++j)
      if (s[j] > rowmax) rowmax = s[j];
    float m_new = st->m > rowmax ? st->m : rowmax;
    if (m_new == -INFINITY) continue;
    float mlam = m_new * lam;
    float alpha = (st->m == -INFINITY) ? 0.0f : exp2_f32((st->m - m_new) * lam);
    float rowsum = 0.0f;
    for (int j = a; j < b; ++j) {
      p[j - a] = exp2_f32(fmaf(s[j], lam, -mlam));        /* P = 2^(lam S - lam m) <= 1 */
      rowsum += p[j - a];                                  /* l uses the unquantized P */
    }
    st->l = alpha * st->l + rowsum;
    float acc[D];
    for (int c = 0; c < D; ++c) acc[c] = alpha * st->o[c];
    for (int j = a; j < b; ++j) {
      float ph = p[j - a] * 448.0f;
      if (p_fp8) {
        uint8_t code = mpfa_oracle_e4m3_encode(ph);
        if (q_out) q_out[j] = ph;
        if (j == flip_key) {
          int c2 = (int)code + flip_dir;
          code = (uint8_t)(c2 < 0 ? 0 : (c2 > 0x7E ? 0x7E : c2));
        }
        if (phat_out) phat_out[j] = code;
        ph = e4m3_tab[code];
      }
      if (v_f32) {
        const float *vr = v_f32 + (size_t)j * D;
        for (int c = 0; c < D; ++c) acc[c] += ph * vr[c];
      } else {
        const uint8_t *vr = v + (size_t)j * D;
        for (int c = 0; c < D; ++c) acc[c] += ph * e4m3_tab[vr[c]];
      }
    }
    for (int c = 0; c < D; ++c) st->o[c] = acc[c];
    st->m = m_new;
  }
  free(p);
}

/* Number of keys a query row may see. Causal masks are bottom-right aligned. */
static int visible_keys(int i, int Nq, int Nkv, int causal) {
  if (!causal) return Nkv;
  int n = i + Nkv - Nq + 1;
  return n < 0 ? 0 : (n > Nkv ? Nkv : n);
}

/* QK4PV8 prefill for a list of rows.  rows: int32 [n_rows, 3] = (b, hq, i).
 * Quantized inputs are the logical row-major arrays written by the quantizers
 * above.  delta may be NULL (no compensation).  out_f32: [n_rows, D] before the
 * final BF16 rounding, out_bf16: [n_rows, D]. */
static void prefill_rows_impl(const uint8_t *q_codes, const uint8_t *q_sf, const uint8_t *k_codes,
                              const uint8_t *k_sf, const uint8_t *v_codes, const uint16_t *delta,
                              const float *dq, const float *dk, float v_scale, float softmax_scale,
                              int causal, int Nq, int Nkv, int Hq, int Hkv, int block_kv, int reverse,
                              int p_fp8, int delta_elementwise, const int32_t *rows, int n_rows,
                              float *out_f32, uint16_t *out_bf16) {
  init_tables();
  int grp = Hq / Hkv;
#pragma omp parallel for schedule(dynamic, 1)
  for (int r = 0; r < n_rows; ++r) {
    int b = rows[3 * r], hq = rows[3 * r + 1], i = rows[3 * r + 2];
    int hk = hq / grp;
    int n = visible_keys(i, Nq, Nkv, causal);
    float *s = (float *)malloc(sizeof(float) * (size_t)(n > 0 ? n : 1));
    logits_row_q4(q_codes + (((size_t)b * Hq + hq) * Nq + i) * (D / 2),
                  q_sf + (((size_t)b * Hq + hq) * Nq + i) * NBLK,
                  k_codes + ((size_t)b * Hkv + hk) * Nkv * (D / 2),
                  k_sf + ((size_t)b * Hkv + hk) * Nkv * NBLK,
                  (delta && !delta_elementwise) ? delta + ((size_t)b * Hq + hq) * Nkv : NULL, n, s);
    if (delta && delta_elementwise) {
      /* Section 7.4, element-wise placement: the same BF16 term added to the finished FP32 score */
      const uint16_t *dr = delta + ((size_t)b * Hq + hq) * Nkv;
      for (int j = 0; j < n; ++j) s[j] = s[j] + mpfa_oracle_bf16_to_f32(dr[j]);
    }
    float lam = ((softmax_scale * 1.4426950408889634f) * dq[b]) * dk[b];
    softmax_state st;
    online_softmax_pv(s, 0, n, lam, v_codes + ((size_t)b * Hkv + hk) * Nkv * D, NULL, block_kv,
                      reverse, p_fp8, &st, NULL);
    for (int c = 0; c < D; ++c) {
      float o = (st.l > 0.0f) ? st.o[c] / (448.0f * st.l) * v_scale : 0.0f;
      out_f32[(size_t)r * D + c] = o;
      out_bf16[(size_t)r * D + c] = mpfa_oracle_f32_to_bf16(o);
    }
    free(s);
  }
}

void mpfa_oracle_prefill_rows(const uint8_t *q_codes, const uint8_t *q_sf, const uint8_t *k_codes,
                              const uint8_t *k_sf, const uint8_t *v_codes, const uint16_t *delta,
                              const float *dq, const float *dk, float v_scale, float softmax_scale,
                              int causal, int B, int Nq, int Nkv, int Hq, int Hkv, int block_kv,
                              int reverse, int p_fp8, const int32_t *rows, int n_rows, float *out_f32,
                              uint16_t *out_bf16) {
  (void)B;
  prefill_rows_impl(q_codes, q_sf, k_codes, k_sf, v_codes, delta, dq, dk, v_scale, softmax_scale, causal, Nq, Nkv,
                    Hq, Hkv, block_kv, reverse, p_fp8, 0, rows, n_rows, out_f32, out_bf16);
}

/* Ablation variant (Section 7.4, compensation placement): identical to the function above except that
 * Delta_S is not the seed of the score accumulator but is added, in FP32, to the finished score of the
 * block-scaled products ("element-wise placement uses FP32 scalar addition").  The BF16 values of Delta_S
 * are the same in both placements here, so the two differ by where one FP32 rounding falls. */
void mpfa_oracle_prefill_rows_elementwise(const uint8_t *q_codes, const uint8_t *q_sf, const uint8_t *k_codes,
                                          const uint8_t *k_sf, const uint8_t *v_codes, const uint16_t *delta,
                                          const float *dq, const float *dk, float v_scale, float softmax_scale,
                                          int causal, int B, int Nq, int Nkv, int Hq, int Hkv, int block_kv,
                                          int reverse, int p_fp8, const int32_t *rows, int n_rows,
                                          float *out_f32, uint16_t *out_bf16) {
  (void)B;
  prefill_rows_impl(q_codes, q_sf, k_codes, k_sf, v_codes, delta, dq, dk, v_scale, softmax_scale, causal, Nq, Nkv,
                    Hq, Hkv, block_kv, reverse, p_fp8, 1, rows, n_rows, out_f32, out_bf16);
}

/* QK4PV8 decode (Section 5.3): one query token per request against its first
 * seq_len keys, split into consecutive `split`-token ranges counted from key 0;
 * each range runs the main loop above on its own, the partial states are merged
 * by log-sum-exp with ranges ascending.
 * q_codes [B, Hq, D/2], q_sf [B, Hq, 8]; K/V/delta are the logical per-request
 * arrays [B, Hkv, Lmax, ...] (the page table only relocates data and is
 * resolved by the caller). */
void mpfa_oracle_decode(const uint8_t *q_codes, const uint8_t *q_sf, const uint8_t *k_codes,
                        const uint8_t *k_sf, const uint8_t *v_codes, const uint16_t *delta,
                        const float *dq, const float *dk, float v_scale, float softmax_scale,
                        const int32_t *seq_lens, int B, int Lmax, int Hq, int Hkv, int block_kv,
                        int split, int reverse, int p_fp8, float *out_f32, uint16_t *out_bf16) {
  init_tables();
  int grp = Hq / Hkv;
#pragma omp parallel for collapse(2) schedule(dynamic, 1)
  for (int b = 0; b < B; ++b)
    for (int hq = 0; hq < Hq; ++hq) {
      int hk = hq / grp;
      int L = seq_lens[b];
      float *s = (float *)malloc(sizeof(float) * (size_t)(L > 0 ? L : 1));
      logits_row_q4(q_codes + ((size_t)b * Hq + hq) * (D / 2), q_sf + ((size_t)b * Hq + hq) * NBLK,
                    k_codes + ((size_t)b * Hkv + hk) * Lmax * (D / 2),
                    k_sf + ((size_t)b * Hkv + hk) * Lmax * NBLK,
                    delta ? delta + ((size_t)b * Hq + hq) * Lmax : NULL, L, s);
      float lam = ((softmax_scale * 1.4426950408889634f) * dq[b]) * dk[b];
      int n_split = (L + split - 1) / split;
      softmax_state *parts = (softmax_state *)malloc(sizeof(softmax_state) * (size_t)(n_split > 0 ? n_split : 1));
      float M = -INFINITY;
      for (int sp = 0; sp < n_split; ++sp) {
        int k0 = sp * split, k1 = (sp + 1) * split > L ? L : (sp + 1) * split;
        online_softmax_pv(s, k0, k1, lam, v_codes + ((size_t)b * Hkv + hk) * Lmax * D, NULL, block_kv,
                          reverse, p_fp8, &parts[sp], NULL);
        if (parts[sp].m > M) M = parts[sp].m;
      }
      float l = 0.0f, o[D];
      for (int c = 0; c < D; ++c) o[c] = 0.0f;
      for (int sp = 0; sp < n_split; ++sp) {
        if (parts[sp].m == -INFINITY) continue;
        float w = exp2_f32((parts[sp].m - M) * lam);
        l += w * parts[sp].l;
        for (int c = 0; c < D; ++c) o[c] += w * parts[sp].o[c];
      }
      for (int c = 0; c < D; ++c) {
        float r = (l > 0.0f) ? o[c] / (448.0f * l) * v_scale : 0.0f;
        out_f32[((size_t)b * Hq + hq) * D + c] = r;
        out_bf16[((size_t)b * Hq + hq) * D + c] = mpfa_oracle_f32_to_bf16(r);
      }
      free(parts);
      free(s);
    }
}

/* The same main loop with every quantizer replaced by the identity: FP32 logits
 * from FP32 q.k dot products (FP64 accumulate, one rounding), FP32 V, FP32 P.
 * Used to pin the loop itself against textbook softmax attention.
 * q [n_rows, D], k [Nkv, D], v [Nkv, D] FP32; n_vis[r] = keys visible to row r. */
void mpfa_oracle_mainloop_identity(const float *q, const float *k, const float *v, const int32_t *n_vis,
                                   int n_rows, int Nkv, float softmax_scale, int block_kv, int reverse,
                                   float *out_f32, float *rowsum_norm) {
  init_tables();
  (void)Nkv;
  for (int r = 0; r < n_rows; ++r) {
    int n = n_vis[r];
    float *s = (float *)malloc(sizeof(float) * (size_t)(n > 0 ? n : 1));
    for (int j = 0; j < n; ++j) {
      double a = 0.0;
      for (int c = 0; c < D; ++c) a += (double)q[(size_t)r * D + c] * (double)k[(size_t)j * D + c];
      s[j] = (float)a;
    }
    float lam = softmax_scale * 1.4426950408889634f;
    softmax_state st;
    online_softmax_pv(s, 0, n, lam, NULL, v, block_kv, reverse, 0, &st, NULL);
    for (int c = 0; c < D; ++c) out_f32[(size_t)r * D + c] = (st.l > 0.0f) ? st.o[c] / (448.0f * st.l) : 0.0f;
    /* sum over keys of the final normalised probabilities, for the rows-sum-to-one pin */
    double tot = 0.0;
    for (int j = 0; j < n; ++j) tot += exp2((double)s[j] * lam - (double)st.m * lam);
    rowsum_norm[r] = (st.l > 0.0f) ? (float)(tot / (double)st.l) : 0.0f;
    free(s);
  }
}

/* Eq. 2 in FP64 on unquantized BF16 inputs, for the rows listed: the "exact"
 * reference used only for reported error columns and oracle pins.
 * q [B,Nq,Hq,D], k, v [B,Nkv,Hkv,D] BF16; out FP64 [n_rows, D]. */
void mpfa_oracle_exact_rows(const uint16_t *q, const uint16_t *k, const uint16_t *v, float softmax_scale,
                            int causal, int B, int Nq, int Nkv, int Hq, int Hkv, const int32_t *rows,
                            int n_rows, double *out) {
  (void)B;
  int grp = Hq / Hkv;
#pragma omp parallel for schedule(dynamic, 1)
  for (int r = 0; r < n_rows; ++r) {
    int b = rows[3 * r], hq = rows[3 * r + 1], i = rows[3 * r + 2];
    int hk = hq / grp;
    int n = visible_keys(i, Nq, Nkv, causal);
    double *s = (double *)malloc(sizeof(double) * (size_t)(n > 0 ? n : 1));
    const uint16_t *qr = q + (((size_t)b * Nq + i) * Hq + hq) * D;
    double mx = -INFINITY;
    for (int j = 0; j < n; ++j) {
      const uint16_t *kr = k + (((size_t)b * Nkv + j) * Hkv + hk) * D;
      double a = 0.0;
      for (int c = 0; c < D; ++c)
        a += (double)mpfa_oracle_bf16_to_f32(qr[c]) * (double)mpfa_oracle_bf16_to_f32(kr[c]);
      s[j] = a * (double)softmax_scale;
      if (s[j] > mx) mx = s[j];
    }
    double l = 0.0, o[D];
    for (int c = 0; c < D; ++c) o[c] = 0.0;
    for (int j = 0; j < n; ++j) {
      double p = exp(s[j] - mx);
      l += p;
      const uint16_t *vr = v + (((size_t)b * Nkv + j) * Hkv + hk) * D;
      for (int c = 0; c < D; ++c) o[c] += p * (double)mpfa_oracle_bf16_to_f32(vr[c]);
    }
    for (int c = 0; c < D; ++c) out[(size_t)r * D + c] = (l > 0.0) ? o[c] / l : 0.0;
    free(s);
  }
}

/* Logits of listed rows, exposed so tests can pin Eq. 10/11 against an integer
 * dot product and the Eq. 8 identity.  s_out: [n_rows, Nkv] (all keys, no mask). */
void mpfa_oracle_logits_rows(const uint8_t *q_codes, const uint8_t *q_sf, const uint8_t *k_codes,
                             const uint8_t *k_sf, const uint16_t *delta, int Nq, int Nkv, int Hq, int Hkv,
                             const int32_t *rows, int n_rows, float *s_out) {
  init_tables();
  int grp = Hq / Hkv;
  for (int r = 0; r < n_rows; ++r) {
    int b = rows[3 * r], hq = rows[3 * r + 1], i = rows[3 * r + 2];
    int hk = hq / grp;
    logits_row_q4(q_codes + (((size_t)b * Hq + hq) * Nq + i) * (D / 2),
                  q_sf + (((size_t)b * Hq + hq) * Nq + i) * NBLK,
                  k_codes + ((size_t)b * Hkv + hk) * Nkv * (D / 2), k_sf + ((size_t)b * Hkv + hk) * Nkv * NBLK,
                  delta ? delta + ((size_t)b * Hq + hq) * Nkv : NULL, Nkv, s_out + (size_t)r * Nkv);
  }
}

/* Inspection entry point for the pins: the E4M3 codes of P-hat that the main
 * loop assigns to every visible key of the listed rows (Section 4.1: fixed
 * scale 448, quantized against the running maximum of the traversal), plus the
 * final (m, l) of each row.  Same calls as prefill_rows_impl; nothing is
 * computed differently unless flip_key >= 0.  codes_out: [n_rows, Nkv] (keys a row
 * cannot see stay 0), ml_out: [n_rows, 2]; optional q_out [n_rows, Nkv] (the FP32
 * values 448 P that were encoded) and o_out [n_rows, D] (outputs, v_scale = 1). */
void mpfa_oracle_phat_rows(const uint8_t *q_codes, const uint8_t *q_sf, const uint8_t *k_codes,
                           const uint8_t *k_sf, const uint8_t *v_codes, const uint16_t *delta,
                           const float *dq, const float *dk, float softmax_scale, int causal, int Nq, int Nkv,
                           int Hq, int Hkv, int block_kv, int reverse, const int32_t *rows, int n_rows,
                           uint8_t *codes_out, float *ml_out, float *q_out, float *o_out, int flip_key, int flip_dir) {
  init_tables();
  int grp = Hq / Hkv;
  for (int r = 0; r < n_rows; ++r) {
    int b = rows[3 * r], hq = rows[3 * r + 1], i = rows[3 * r + 2];
    int hk = hq / grp;
    int n = visible_keys(i, Nq, Nkv, causal);
    float *s = (float *)malloc(sizeof(float) * (size_t)(n > 0 ? n : 1));
    logits_row_q4(q_codes + (((size_t)b * Hq + hq) * Nq + i) * (D / 2),
                  q_sf + (((size_t)b * Hq + hq) * Nq + i) * NBLK,
                  k_codes + ((size_t)b * Hkv + hk) * Nkv * (D / 2), k_sf + ((size_t)b * Hkv + hk) * Nkv * NBLK,
                  delta ? delta + ((size_t)b * Hq + hq) * Nkv : NULL, n, s);
    float lam = ((softmax_scale * 1.4426950408889634f) * dq[b]) * dk[b];
    softmax_state st;
    memset(codes_out + (size_t)r * Nkv, 0, (size_t)Nkv);
    if (q_out) memset(q_out + (size_t)r * Nkv, 0, sizeof(float) * (size_t)Nkv);
    online_softmax_pv_x(s, 0, n, lam, v_codes + ((size_t)b * Hkv + hk) * Nkv * D, NULL, block_kv, reverse, 1, &st,
                        codes_out + (size_t)r * Nkv, q_out ? q_out + (size_t)r * Nkv : NULL, flip_key, flip_dir);
    ml_out[2 * r] = st.m;
    ml_out[2 * r + 1] = st.l;
    if (o_out)   /* the row's output before the BF16 rounding, v_scale = 1 */
      for (int c = 0; c < D; ++c) o_out[(size_t)r * D + c] = (st.l > 0.0f) ? st.o[c] / (448.0f * st.l) : 0.0f;
    free(s);
  }
}

/* ------------------------------------------------------------------------- */
/* precision-assignment variant: NVFP4 Q K^T with BF16 P V (Section 3.1)      */
/* ------------------------------------------------------------------------- */

/* One of the paper's four precision assignments (Section 3.1, Section 7.2): the logits are the same
 * NVFP4 + rank-one logits as in the method, but P is carried to the second MMA in BF16 and V stays in
 * BF16 (the unquantized input).  Per KV block (reverse order, as in the method):
 *   m_new = max(m, rowmax);  P = 2^(lam S - lam m_new) in FP32;  l = alpha l + sum P (FP32 P);
 *   P_b = BF16_RNE(P);  O = alpha O + sum_k P_b[k] V[k] (FP32, k ascending);  out = O / l.
 * No scale 448 is involved (BF16 has the range); reading taken: P is rounded once, to nearest even.
 * v: BF16 [B, Nkv, Hkv, D] as given to stage 1. */
void mpfa_oracle_prefill_rows_pv_bf16(const uint8_t *q_codes, const uint8_t *q_sf, const uint8_t *k_codes,
                                      const uint8_t *k_sf, const uint16_t *v, const uint16_t *delta, const float *dq,
                                      const float *dk, float softmax_scale, int causal, int Nq, int Nkv, int Hq, int Hkv,
                                      int block_kv, const int32_t *rows, int n_rows, float *out_f32, uint16_t *out_bf16) {
  init_tables();
  int grp = Hq / Hkv;
#pragma omp parallel for schedule(dynamic, 1)
  for (int r = 0; r < n_rows; ++r) {
    int b = rows[3 * r], hq = rows[3 * r + 1], i = rows[3 * r + 2];
    int hk = hq / grp;
    int n = visible_keys(i, Nq, Nkv, causal);
    float *s = (float *)malloc(sizeof(float) * (size_t)(n > 0 ? n : 1));
    float *p = (float *)malloc(sizeof(float) * (size_t)block_kv);
    logits_row_q4(q_codes + (((size_t)b * Hq + hq) * Nq + i) * (D / 2), q_sf + (((size_t)b * Hq + hq) * Nq + i) * NBLK,
                  k_codes + ((size_t)b * Hkv + hk) * Nkv * (D / 2), k_sf + ((size_t)b * Hkv + hk) * Nkv * NBLK,
                  delta ? delta + ((size_t)b * Hq + hq) * Nkv : NULL, n, s);
    float lam = ((softmax_scale * 1.4426950408889634f) * dq[b]) * dk[b];
    float m = -INFINITY, l = 0.0f, o[D];
    for (int c = 0; c < D; ++c) o[c] = 0.0f;
    for (int jb = n > 0 ? (n - 1) / block_kv : -1; jb >= 0; --jb) {
      int a = jb * block_kv, e = (jb + 1) * block_kv > n ? n : (jb + 1) * block_kv;
      float rowmax = -INFINITY;
      for (int j = a; j < e; ++j)
        if (s[j] > rowmax) rowmax = s[j];
      float m_new = m > rowmax ? m : rowmax;
      if (m_new == -INFINITY) continue;
      float mlam = m_new * lam;
      float alpha = (m == -INFINITY) ? 0.0f : exp2_f32((m - m_new) * lam);
      float rowsum = 0.0f;
      for (int j = a; j < e; ++j) {
        p[j - a] = exp2_f32(fmaf(s[j], lam, -mlam));
        rowsum += p[j - a];
      }
      l = alpha * l + rowsum;
      for (int c = 0; c < D; ++c) o[c] = alpha * o[c];
      for (int j = a; j < e; ++j) {
        float pb = mpfa_oracle_bf16_to_f32(mpfa_oracle_f32_to_bf16(p[j - a]));
        const uint16_t *vr = v + (((size_t)b * Nkv + j) * Hkv + hk) * D;
        for (int c = 0; c < D; ++c) o[c] += pb * mpfa_oracle_bf16_to_f32(vr[c]);
      }
      m = m_new;
    }
    for (int c = 0; c < D; ++c) {
      float x = (l > 0.0f) ? o[c] / l : 0.0f;
      out_f32[(size_t)r * D + c] = x;
      out_bf16[(size_t)r * D + c] = mpfa_oracle_f32_to_bf16(x);
    }
    free(p);
    free(s);
  }
}

/* ------------------------------------------------------------------------- */
/* precision-assignment variant: NVFP4 Q K^T with NVFP4 P V (Section 3.1)     */
/* ------------------------------------------------------------------------- */

/* V for a block-scaled second MMA: the contraction runs over the keys, so the 16-element blocks of
 * Eq. 1 lie along the token axis (tokens 16 g .. 16 g + 15 of one channel; tokens past N count as zero).
 * Same recipe as the Q/K quantizer with the caller's tensor scale d in place of a statistic and no
 * centering:  r = amax / (6 d);  sc = E4M3(r);  s = decode(sc) d;  code = E2M1(x (1 / s)).
 * v: BF16 [B, N, H, D];  codes: [B, H, D, NB, 8] (NB = ceil(N / 16); two E2M1 codes per byte, the even
 * token of the block in the low nibble);  sf: [B, H, D, NB]. */
void mpfa_oracle_quantize_v_fp4(const uint16_t *v, int B, int N, int H, float d, uint8_t *codes, uint8_t *sf) {
  int NB = (N + G - 1) / G;
#pragma omp parallel for collapse(2) schedule(static)
  for (int b = 0; b < B; ++b)
    for (int h = 0; h < H; ++h)
      for (int c = 0; c < D; ++c)
        for (int g = 0; g < NB; ++g) {
          float x[G];
          float a = 0.0f;
          for (int i = 0; i < G; ++i) {
            int t = g * G + i;
            x[i] = t < N ? mpfa_oracle_bf16_to_f32(v[(((size_t)b * N + t) * H + h) * D + c]) : 0.0f;
            if (fabsf(x[i]) > a) a = fabsf(x[i]);
          }
          float e = 6.0f * d;
          float r = a / e;
          uint8_t sc = mpfa_oracle_e4m3_encode(r);
          float s = mpfa_oracle_e4m3_decode(sc) * d;
          float inv = 1.0f / s;
          if (!(s > 0.0f) || isinf(inv)) inv = 0.0f;
          size_t blk = (((size_t)b * H + h) * D + c) * NB + g;
          sf[blk] = sc;
          for (int i = 0; i < G; i += 2) {
            uint8_t lo = mpfa_oracle_e2m1_encode(x[i] * inv);
            uint8_t hi = mpfa_oracle_e2m1_encode(x[i + 1] * inv);
            codes[blk * (G / 2) + i / 2] = (uint8_t)(lo | (hi << 4));
          }
        }
}

/* The fourth precision assignment of Section 3.1 / 7.2: logits as in the method; P and V both enter the
 * second MMA as NVFP4 operands.  The paper gives no arithmetic for it; reading taken, per KV block
 * (reverse order) and row:
 *   m_new, alpha, P = 2^(lam S - lam m_new), l = alpha l + sum P           as in the method;
 *   q = 448 P (P <= 1, so the tensor scale of P is fixed at 1 / (6 * 448) and needs no statistic, like the
 *   fixed 448 of the FP8 path: a block's scale amax_P / (6 d_P) is then 448 amax_P = max q <= 448);
 *   per 16 keys (blocks aligned to multiples of 16; keys the row cannot see count as 0):
 *     sc = E4M3(max q);  s = decode(sc);  code_j = E2M1(q_j (6 / s))     (6 / s = 0 when s = 0);
 *   O = alpha O + sum over the 16-key blocks of (s s_V[c]) * sum_j code_j vcode_j[c]
 *       (the block-scaled MMA: exact 16-term dot product, one scale product per block, FP32 adds, blocks
 *       ascending);
 *   out = O / (6 * 448 * l) * d_V.
 * v_codes / v_sf: as written by mpfa_oracle_quantize_v_fp4 for the same N = Nkv.
 * Inspection outputs (optional): pcodes_out [n_rows, Nkv] E2M1 codes of P, psf_out [n_rows, ceil(Nkv/16)] block
 * scale codes, y_out [n_rows, Nkv] the FP32 values q (6 / s) that were encoded, amax_out [n_rows, ceil(Nkv/16)] the
 * FP32 block maxima that were encoded.  Inspection switches (-1 everywhere else, where they change nothing):
 * flip_key >= 0 moves that key's E2M1 code by flip_dir steps; flip_blk >= 0 moves that block's scale code by
 * flip_blk_dir steps before its codes are made (to show what a one-step difference in a single decision does to a
 * row). */
void mpfa_oracle_prefill_rows_pv_fp4(const uint8_t *q_codes, const uint8_t *q_sf, const uint8_t *k_codes,
                                     const uint8_t *k_sf, const uint8_t *v_codes, const uint8_t *v_sf,
                                     const uint16_t *delta, const float *dq, const float *dk, float v_gscale,
                                     float softmax_scale, int causal, int Nq, int Nkv, int Hq, int Hkv, int block_kv,
                                     const int32_t *rows, int n_rows, float *out_f32, uint16_t *out_bf16,
                                     uint8_t *pcodes_out, uint8_t *psf_out, float *y_out, float *amax_out,
                                     int flip_key, int flip_dir, int flip_blk, int flip_blk_dir) {
  init_tables();
  int grp = Hq / Hkv;
  int NB = (Nkv + G - 1) / G;
#pragma omp parallel for schedule(dynamic, 1)
  for (int r = 0; r < n_rows; ++r) {
    int b = rows[3 * r], hq = rows[3 * r + 1], i = rows[3 * r + 2];
    int hk = hq / grp;
    int n = visible_keys(i, Nq, Nkv, causal);
    float *s = (float *)malloc(sizeof(float) * (size_t)(n > 0 ? n : 1));
    float *q = (float *)malloc(sizeof(float) * (size_t)(block_kv + G));
    logits_row_q4(q_codes + (((size_t)b * Hq + hq) * Nq + i) * (D / 2), q_sf + (((size_t)b * Hq + hq) * Nq + i) * NBLK,
                  k_codes + ((size_t)b * Hkv + hk) * Nkv * (D / 2), k_sf + ((size_t)b * Hkv + hk) * Nkv * NBLK,
                  delta ? delta + ((size_t)b * Hq + hq) * Nkv : NULL, n, s);
    if (pcodes_out) memset(pcodes_out + (size_t)r * Nkv, 0, (size_t)Nkv);
    if (psf_out) memset(psf_out + (size_t)r * NB, 0, (size_t)NB);
    if (y_out) memset(y_out + (size_t)r * Nkv, 0, sizeof(float) * (size_t)Nkv);
    if (amax_out) memset(amax_out + (size_t)r * NB, 0, sizeof(float) * (size_t)NB);
    float lam = ((softmax_scale * 1.4426950408889634f) * dq[b]) * dk[b];
    float m = -INFINITY, l = 0.0f, o[D];
    for (int c = 0; c < D; ++c) o[c] = 0.0f;
    const uint8_t *vc = v_codes + ((size_t)b * Hkv + hk) * D * NB * (G / 2);
    const uint8_t *vs = v_sf + ((size_t)b * Hkv + hk) * D * NB;
    for (int jb = n > 0 ? (n - 1) / block_kv : -1; jb >= 0; --jb) {
      int a = jb * block_kv, e = (jb + 1) * block_kv > n ? n : (jb + 1) * block_kv;
      float rowmax = -INFINITY;
      for (int j = a; j < e; ++j)
        if (s[j] > rowmax) rowmax = s[j];
      float m_new = m > rowmax ? m : rowmax;
      if (m_new == -INFINITY) continue;
      float mlam = m_new * lam;
      float alpha = (m == -INFINITY) ? 0.0f : exp2_f32((m - m_new) * lam);
      float rowsum = 0.0f;
      for (int j = a; j < e; ++j) {
        float p = exp2_f32(fmaf(s[j], lam, -mlam));
        rowsum += p;
        q[j - a] = p * 448.0f;
      }
      for (int j = e; j < a + block_kv + G; ++j) q[j - a] = 0.0f;   /* keys the row cannot see */
      l = alpha * l + rowsum;
      for (int c = 0; c < D; ++c) o[c] = alpha * o[c];
      for (int g0 = a; g0 < e; g0 += G) {                         /* a is a multiple of 16 */
        float amax = 0.0f;
        for (int j = 0; j < G; ++j)
          if (q[g0 - a + j] > amax) amax = q[g0 - a + j];
        uint8_t sc = mpfa_oracle_e4m3_encode(amax);
        if (amax_out) amax_out[(size_t)r * NB + g0 / G] = amax;
        if (g0 / G == flip_blk) {
          int c2 = (int)sc + flip_blk_dir;
          sc = (uint8_t)(c2 < 0 ? 0 : (c2 > 0x7E ? 0x7E : c2));
        }
        float sp = e4m3_tab[sc];
        float inv = sp > 0.0f ? 6.0f / sp : 0.0f;
        float pv[G];
        for (int j = 0; j < G; ++j) {
          uint8_t code = mpfa_oracle_e2m1_encode(q[g0 - a + j] * inv);
          if (y_out && g0 + j < Nkv) y_out[(size_t)r * Nkv + g0 + j] = q[g0 - a + j] * inv;
          if (g0 + j == flip_key) {
            int c2 = (int)code + flip_dir;
            code = (uint8_t)(c2 < 0 ? 0 : (c2 > 7 ? 7 : c2));
          }
          pv[j] = mpfa_oracle_e2m1_decode(code);
          if (pcodes_out && g0 + j < Nkv) pcodes_out[(size_t)r * Nkv + g0 + j] = code;
        }
        if (psf_out) psf_out[(size_t)r * NB + g0 / G] = sc;
        int gi = g0 / G;
        for (int c = 0; c < D; ++c) {
          const uint8_t *vb = vc + ((size_t)c * NB + gi) * (G / 2);
          float dot = 0.0f;
          for (int j = 0; j < G / 2; ++j) {
            dot += pv[2 * j] * e2m1_pair_lo[vb[j]];
            dot += pv[2 * j + 1] * e2m1_pair_hi[vb[j]];
          }
          o[c] += (sp * e4m3_tab[vs[(size_t)c * NB + gi]]) * dot;
        }
      }
      m = m_new;
    }
    for (int c = 0; c < D; ++c) {
      float x = (l > 0.0f) ? o[c] / (2688.0f * l) * v_gscale : 0.0f;
      out_f32[(size_t)r * D + c] = x;
      out_bf16[(size_t)r * D + c] = mpfa_oracle_f32_to_bf16(x);
    }
    free(q);
    free(s);
  }
}
