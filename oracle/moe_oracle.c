/*
 * CPU oracle for the routed-MoE expert path.  TEST INFRASTRUCTURE ONLY: it is
 * called by the tests, the smoke check and the bench's CPU-baseline leg, never by
 * the library.  It shares no code with the CUDA path.
 *
 * The method computes exactly the plain MoE forward (Section 2.1 of the paper: a
 * router picks the top-k routed experts of every token, the token's activation
 * goes through each of them, the outputs are combined), so the oracle is that
 * definition written out, step by step, with double accumulators:
 *
 *   plan     counts / exclusive offsets / stable permutation of the routed rows
 *            (the per-expert packed layout of Section 2.4) and the tile table
 *            whose length is the footprint x_moe of Section 6.2
 *   ffn      per routed row, SwiGLU expert FFN: silu(x Wg) * (x Wu), then Wd
 *            (the "two grouped GEMMs, activation functions" of Section 7.1)
 *   combine  y[t] = sum_j w[t,j] * d[row(t,j)], slots in order
 *
 * Parity pins (see tests/test_oracle_pins.py): the plan equals a stable argsort
 * and a brute-force rescan; the FFN equals a float64 library MLP for E=1,k=1;
 * the whole equals dense every-expert evaluation in float64; e4m3 decode equals
 * the library's table for all 256 codes; the rounding switches of the FFN (e4m3 per
 * row and 128 columns, bf16 of the intermediate, bf16 of the output) equal the
 * library casts applied to the un-rounded values.  The paper prints no worked numeric
 * example of this path, so numeric parity against the paper itself is unpinned.
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

#ifdef _OPENMP
#include <omp.h>
#endif

enum { ORC_BF16 = 0, ORC_E4M3 = 1 };
enum { ROUND_NONE = 0, ROUND_BF16 = 1, ROUND_E4M3_1X128 = 2 };

int orc_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}

/* ------------------------------------------------------------------ number formats */

float orc_bf16_to_f32(uint16_t b) {
  uint32_t u = ((uint32_t)b) << 16;
  float f;
  memcpy(&f, &u, 4);
  return f;
}

/* fp32 -> bf16, round to nearest, ties to even (NaN kept quiet) */
uint16_t orc_f32_to_bf16(float f) {
  uint32_t u;
  memcpy(&u, &f, 4);
  if ((u & 0x7fffffffu) > 0x7f800000u) return (uint16_t)((u >> 16) | 0x40);
  uint32_t lsb = (u >> 16) & 1u;
  u += 0x7fffu + lsb;
  return (uint16_t)(u >> 16);
}

/* OCP E4M3FN: 1 sign, 4 exponent (bias 7), 3 mantissa; no infinity; S.1111.111 is NaN;
 * largest finite 448. */
float orc_e4m3_to_f32(uint8_t c) {
  int s = c >> 7, e = (c >> 3) & 15, m = c & 7;
  double v;
  if (e == 15 && m == 7) return NAN;
  if (e == 0) v = ldexp((double)m, -9);            /* subnormal: m/8 * 2^-6 */
  else v = ldexp(1.0 + m / 8.0, e - 7);
  return (float)(s ? -v : v);
}

/* fp32 -> e4m3, round to nearest even, saturating to +-448 (NaN -> 0x7f).
 * Written as a search over the 127 finite magnitudes so it can be checked by eye. */
uint8_t orc_f32_to_e4m3(float f) {
  if (f != f) return 0x7f;
  uint8_t sign = (uint8_t)(signbit(f) ? 0x80 : 0);
  double a = fabs((double)f);
  if (a >= 448.0) return (uint8_t)(sign | 0x7e);
  int best = 0;
  double bestd = a;                                  /* distance to code 0 (value 0) */
  for (int c = 1; c <= 0x7e; ++c) {
    double d = fabs(a - (double)orc_e4m3_to_f32((uint8_t)c));
    if (d < bestd || (d == bestd && (c & 1) == 0)) { bestd = d; best = c; }
  }
  return (uint8_t)(sign | best);
}

/* Quantise one group of n fp32 values to e4m3 with one fp32 scale:
 * scale = amax/448 (1 when amax == 0), code = rn(v * (448/amax)). */
void orc_quant_group(const float* v, int n, uint8_t* q, float* scale) {
  float amax = 0.f;
  for (int i = 0; i < n; ++i) { float a = fabsf(v[i]); if (a > amax) amax = a; }
  if (amax == 0.f) {
    *scale = 1.0f;
    for (int i = 0; i < n; ++i) q[i] = 0;
    return;
  }
  *scale = amax / 448.0f;
  float inv = 448.0f / amax;
  for (int i = 0; i < n; ++i) q[i] = orc_f32_to_e4m3(v[i] * inv);
}

/* ------------------------------------------------------------------ router (C1 reading) */

/* softmax over all E experts in fp32 with max subtraction, then the k largest
 * probabilities (ties to the lower expert id), slots in that order, weights
 * renormalised over the selected k. */
int orc_router(const float* logits, int T, int E, int k, int32_t* ids, float* w) {
  if (k > E || k <= 0) return -1;
  float* p = (float*)malloc(sizeof(float) * (size_t)E);
  char* used = (char*)malloc((size_t)E);
  if (!p || !used) return -2;
  for (int t = 0; t < T; ++t) {
    const float* z = logits + (size_t)t * E;
    float mx = z[0];
    for (int e = 1; e < E; ++e) if (z[e] > mx) mx = z[e];
    float sum = 0.f;
    for (int e = 0; e < E; ++e) { p[e] = expf(z[e] - mx); sum += p[e]; }
    for (int e = 0; e < E; ++e) p[e] = p[e] / sum;
    memset(used, 0, (size_t)E);
    float ssel = 0.f;
    for (int j = 0; j < k; ++j) {
      int arg = -1;
      for (int e = 0; e < E; ++e)
        if (!used[e] && (arg < 0 || p[e] > p[arg])) arg = e;
      used[arg] = 1;
      ids[(size_t)t * k + j] = arg;
      w[(size_t)t * k + j] = p[arg];
      ssel += p[arg];
    }
    for (int j = 0; j < k; ++j) w[(size_t)t * k + j] = w[(size_t)t * k + j] / ssel;
  }
  free(p);
  free(used);
  return 0;
}

/* ------------------------------------------------------------------ plan */

/* counts[e] = #{i : ids[i] = e}; offsets = exclusive scan with offsets[E] = R;
 * rows of one expert keep ascending flat index i = t*k + j (stable packing).
 * Returns 0, or -(i+1) for the first out-of-range id. */
int orc_plan(const int32_t* ids, int R, int E, int32_t* counts, int32_t* offsets,
             int32_t* sorted_to_flat, int32_t* flat_to_sorted) {
  for (int e = 0; e < E; ++e) counts[e] = 0;
  for (int i = 0; i < R; ++i) {
    if (ids[i] < 0 || ids[i] >= E) return -(i + 1);
    counts[ids[i]] += 1;
  }
  offsets[0] = 0;
  for (int e = 0; e < E; ++e) offsets[e + 1] = offsets[e] + counts[e];
  for (int e = 0; e < E; ++e) {
    int r = 0;
    for (int i = 0; i < R; ++i) {
      if (ids[i] != e) continue;
      int p = offsets[e] + r;
      sorted_to_flat[p] = i;
      flat_to_sorted[i] = p;
      r += 1;
    }
  }
  return 0;
}

/* Tile table: for every expert with rows, ceil(m_e / M_t) tiles of (expert, first
 * sorted row, valid rows).  The return value is x_moe (Section 6.2).  Output
 * arrays may be NULL to only count. */
int orc_tiles(const int32_t* counts, int E, int Mt, int32_t* t_expert, int32_t* t_row0,
              int32_t* t_rows) {
  int x = 0, off = 0;
  for (int e = 0; e < E; ++e) {
    for (int r0 = 0; r0 < counts[e]; r0 += Mt) {
      if (t_expert) {
        t_expert[x] = e;
        t_row0[x] = off + r0;
        t_rows[x] = counts[e] - r0 < Mt ? counts[e] - r0 : Mt;
      }
      x += 1;
    }
    off += counts[e];
  }
  return x;
}

/* ------------------------------------------------------------------ expert FFN */

typedef struct {
  int E, k, H, I, dtype;
  const void* w_gate_up;   /* [E, 2I, H]: math W_gate[h, c] = storage[e][c][h]        */
  const void* w_down;      /* [E, H, I]:  math W_down[c, h] = storage[e][h][c]        */
  const float* s_gate_up;  /* [E, 2I/128, H/128] (e4m3 only)                          */
  const float* s_down;     /* [E, H/128, I/128]  (e4m3 only)                          */
} orc_weights_t;

/* all 256 e4m3 codes decoded once by orc_e4m3_to_f32 (filled before any parallel region) */
static float e4m3_tab[256];
static int e4m3_tab_ready = 0;
static void e4m3_tab_init(void) {
  if (e4m3_tab_ready) return;
  for (int c = 0; c < 256; ++c) e4m3_tab[c] = orc_e4m3_to_f32((uint8_t)c);
  e4m3_tab_ready = 1;
}

static inline double load_el(const void* base, size_t idx, int dtype) {
  if (dtype == ORC_BF16) return (double)orc_bf16_to_f32(((const uint16_t*)base)[idx]);
  return (double)e4m3_tab[((const uint8_t*)base)[idx]];
}

/* One routed row: x is row `tok` of X ([T,H] stored dtype, x_scale [T,H/128] for e4m3);
 * d_out receives H fp32 values.  a holds I floats, xd holds H doubles (scratch). */
static void ffn_one(const orc_weights_t* W, const void* X, const float* x_scale, int tok,
                    int e, int round_A, int round_D, float* a, double* xd, float* d_out) {
  const int H = W->H, I = W->I, dt = W->dtype;
  const size_t w1 = (size_t)e * 2 * I * H, w2 = (size_t)e * H * I;
  const int HB = H / 128, IB = I / 128;
  /* the stored activation row, upcast exactly (code * scale for e4m3) */
  for (int h = 0; h < H; ++h) {
    xd[h] = load_el(X, (size_t)tok * H + h, dt);
    if (dt == ORC_E4M3) xd[h] *= (double)x_scale[(size_t)tok * HB + h / 128];
  }
  for (int c = 0; c < I; ++c) {
    double g = 0.0, u = 0.0;
    for (int h = 0; h < H; ++h) {
      double wg = load_el(W->w_gate_up, w1 + (size_t)c * H + h, dt);
      double wu = load_el(W->w_gate_up, w1 + (size_t)(I + c) * H + h, dt);
      if (dt == ORC_E4M3) {
        wg *= (double)W->s_gate_up[((size_t)e * (2 * I / 128) + c / 128) * HB + h / 128];
        wu *= (double)W->s_gate_up[((size_t)e * (2 * I / 128) + (I + c) / 128) * HB + h / 128];
      }
      g += xd[h] * wg;
      u += xd[h] * wu;
    }
    float gf = (float)g, uf = (float)u;
    double silu = (double)gf / (1.0 + exp(-(double)gf));
    a[c] = (float)(silu * (double)uf);
  }
  if (round_A == ROUND_BF16) {
    for (int c = 0; c < I; ++c) a[c] = orc_bf16_to_f32(orc_f32_to_bf16(a[c]));
  } else if (round_A == ROUND_E4M3_1X128) {
    /* the one on-path quantisation of the FP8 encoding: 1x128 groups along I */
    uint8_t q[128];
    for (int b = 0; b < IB; ++b) {
      float sc;
      orc_quant_group(a + b * 128, 128, q, &sc);
      for (int i = 0; i < 128; ++i) a[b * 128 + i] = orc_e4m3_to_f32(q[i]) * sc;
    }
  }
  for (int h = 0; h < H; ++h) {
    double d = 0.0;
    for (int c = 0; c < I; ++c) {
      double wd = load_el(W->w_down, w2 + (size_t)h * I + c, dt);
      if (dt == ORC_E4M3) wd *= (double)W->s_down[((size_t)e * (H / 128) + h / 128) * IB + c / 128];
      d += (double)a[c] * wd;
    }
    float df = (float)d;
    if (round_D == ROUND_BF16) df = orc_bf16_to_f32(orc_f32_to_bf16(df));
    d_out[h] = df;
  }
}

/* FFN for a list of routed rows given as (token, expert) pairs.
 * D_out is [n_rows, H] fp32; A_out (may be NULL) is [n_rows, I] fp32. */
int orc_ffn_rows(const orc_weights_t* W, const void* X, const float* x_scale,
                 const int32_t* row_token, const int32_t* row_expert, int n_rows,
                 int round_A, int round_D, float* D_out, float* A_out) {
  int err = 0;
  e4m3_tab_init();
#pragma omp parallel
  {
    float* a = (float*)malloc(sizeof(float) * (size_t)W->I);
    double* xd = (double*)malloc(sizeof(double) * (size_t)W->H);
#pragma omp for schedule(dynamic, 1)
    for (int r = 0; r < n_rows; ++r) {
      int e = row_expert[r];
      if (!a || !xd || e < 0 || e >= W->E) { err = -1; continue; }
      ffn_one(W, X, x_scale, row_token[r], e, round_A, round_D, a, xd, D_out + (size_t)r * W->H);
      if (A_out) memcpy(A_out + (size_t)r * W->I, a, sizeof(float) * (size_t)W->I);
    }
    free(a);
    free(xd);
  }
  return err;
}

/* ------------------------------------------------------------------ combine */

/* y[t,:] = sum_{j=0}^{k-1} w[t,j] * D[row_of[t*k+j], :], slots added in order, double
 * accumulator.  row_of maps a flat routed index to a row of D (the flat->sorted
 * permutation for a packed D, or the identity for a D kept in flat order). */
int orc_combine(const float* D, const float* w, const int32_t* row_of, int T, int k, int H,
                float* y) {
#pragma omp parallel for schedule(static)
  for (int t = 0; t < T; ++t) {
    for (int h = 0; h < H; ++h) {
      double acc = 0.0;
      for (int j = 0; j < k; ++j) {
        size_t i = (size_t)t * k + j;
        acc += (double)w[i] * (double)D[(size_t)row_of[i] * H + h];
      }
      y[(size_t)t * H + h] = (float)acc;
    }
  }
  return 0;
}
