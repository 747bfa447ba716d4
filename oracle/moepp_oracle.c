/*
 * CPU oracle for one MoE++ layer (arXiv 2410.07348), forward pass.
 * TEST INFRASTRUCTURE ONLY -- see moepp_oracle.h for the rules it lives under.
 *
 * Compiled twice: -DORACLE_REAL=float  -DORACLE_PFX=oracle_f32_
 *                 -DORACLE_REAL=double -DORACLE_PFX=oracle_f64_
 * Every intermediate value has type `real`.  Loops follow the equations term by
 * term; the only concession to speed is an OpenMP loop over tokens (tokens are
 * independent in the layer) and a simd reduction on the innermost dot product.
 */
#include "moepp_oracle.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>
#ifdef _OPENMP
#include <omp.h>
#endif

#ifndef ORACLE_REAL
#error "define ORACLE_REAL and ORACLE_PFX"
#endif
typedef ORACLE_REAL real;
#define CAT_(a, b) a##b
#define CAT(a, b) CAT_(a, b)
#define FN(name) CAT(ORACLE_PFX, name)

#ifdef ORACLE_MAIN_TU
void oracle_capacities(const oracle_config* c, int32_t* cap_ffn, int32_t* cap_zc) {
  *cap_ffn = INT32_MAX;
  *cap_zc = INT32_MAX;
  if (c->capacity_factor <= 0.0f) return;
  const double tau = c->tau > 0.0f ? (double)c->tau : 1.0;
  const double slots = (double)c->T * (double)c->top_k;
  const double denom = tau * c->n_ffn + (double)(c->n_zero + c->n_copy + c->n_const);
  const double cf = ceil((double)c->capacity_factor * tau * slots / denom);
  const double cz = ceil((double)c->capacity_factor * slots / denom);
  *cap_ffn = cf > 2147483647.0 ? INT32_MAX : (int32_t)cf;
  *cap_zc = cz > 2147483647.0 ? INT32_MAX : (int32_t)cz;
}

int oracle_num_threads(void) {
#ifdef _OPENMP
  return omp_get_max_threads();
#else
  return 1;
#endif
}
#endif

static real r_exp(real z) { return (sizeof(real) == sizeof(float)) ? (real)expf((float)z) : (real)exp((double)z); }

/* widen one bf16 bit pattern: bf16 is the upper half of an IEEE float */
static float bf16_bits_to_float(uint16_t b) {
  uint32_t u = ((uint32_t)b) << 16;
  float f;
  memcpy(&f, &u, sizeof f);
  return f;
}

static int n_experts(const oracle_config* c) { return c->n_ffn + c->n_zero + c->n_copy + c->n_const; }

static int bad_config(const oracle_config* c) {
  if (!c) return 1;
  if (c->T < 0 || c->D <= 0 || c->F < 0) return 1;
  if (c->n_ffn < 0 || c->n_zero < 0 || c->n_copy < 0 || c->n_const < 0) return 1;
  if (n_experts(c) <= 0) return 1;
  if (c->top_k < 1 || c->top_k > n_experts(c)) return 1;
  if (c->row_align < 1) return 1;
  if (c->n_ffn > 0 && c->F <= 0) return 1;
  return 0;
}

/* dot product of a weight row (float or bf16 bits) with a vector of reals */
static real dot_w(const void* W, int64_t row, int n, int is_bf16, const real* u) {
  real acc = 0;
  if (is_bf16) {
    const uint16_t* w = (const uint16_t*)W + row * (int64_t)n;
#pragma omp simd reduction(+ : acc)
    for (int d = 0; d < n; ++d) acc += (real)bf16_bits_to_float(w[d]) * u[d];
  } else {
    const float* w = (const float*)W + row * (int64_t)n;
#pragma omp simd reduction(+ : acc)
    for (int d = 0; d < n; ++d) acc += (real)w[d] * u[d];
  }
  return acc;
}

/* ---- Eq. 2 and Eq. 6: router logits of one token ------------------------------------------ */
static void logits_token(const oracle_config* c, const float* x_t, const float* W_r, const float* W_g,
                         const float* prev_t, const float* bias, real* G_t) {
  const int N = n_experts(c), D = c->D;
  for (int i = 0; i < N; ++i) {
    real g = 0;
#pragma omp simd reduction(+ : g)
    for (int d = 0; d < D; ++d) g += (real)W_r[(int64_t)i * D + d] * (real)x_t[d]; /* W x */
    if (W_g && prev_t) {
      real r = 0;
      for (int j = 0; j < N; ++j) r += (real)W_g[i * N + j] * (real)prev_t[j]; /* W_g G(x^{j-1}) */
      g += r;
    }
    if (bias) g += (real)bias[i];
    G_t[i] = g;
  }
}

int FN(router_logits)(const oracle_config* c, const float* x, const float* W_r, const float* W_g,
                      const float* prev, const float* bias, float* G) {
  if (bad_config(c) || !x || !W_r || !G) return 1;
  if ((W_g == NULL) != (prev == NULL)) return 1;
  const int N = n_experts(c);
#pragma omp parallel for schedule(static)
  for (int t = 0; t < c->T; ++t) {
    real g[256];
    logits_token(c, x + (int64_t)t * c->D, W_r, W_g, prev ? prev + (int64_t)t * N : NULL, bias, g);
    for (int i = 0; i < N; ++i) G[(int64_t)t * N + i] = (float)g[i];
  }
  return 0;
}

/* ---- Eq. 1: softmax over all N experts, top-K picked on the logits -------------------------- */
static void softmax_all(const real* g, int N, real* P) {
  real m = g[0];
  for (int i = 1; i < N; ++i)
    if (g[i] > m) m = g[i];
  real s = 0;
  for (int i = 0; i < N; ++i) {
    P[i] = r_exp(g[i] - m);
    s += P[i];
  }
  for (int i = 0; i < N; ++i) P[i] = P[i] / s;
}

static void topk_token(const oracle_config* c, const real* g, const real* P, const int32_t* forced, int32_t* idx_t,
                       real* w_t) {
  const int N = n_experts(c), K = c->top_k;
  char taken[256];
  memset(taken, 0, sizeof taken);
  for (int k = 0; k < K; ++k) {
    int best = -1;
    if (forced) {
      best = forced[k];
    } else {
      for (int i = 0; i < N; ++i) {
        if (taken[i]) continue;
        if (best < 0 || g[i] > g[best]) best = i; /* strict '>' keeps the lower index on ties */
      }
    }
    taken[best] = 1;
    idx_t[k] = best;
    w_t[k] = P[best];
  }
  if (c->renorm_topk) {
    real s = 0;
    for (int k = 0; k < K; ++k) s += w_t[k];
    for (int k = 0; k < K; ++k) w_t[k] = w_t[k] / s;
  }
}

int FN(gate_topk)(const oracle_config* c, const float* G, int32_t* idx, float* w, float* P_out) {
  if (bad_config(c) || !G || !idx || !w) return 1;
  const int N = n_experts(c), K = c->top_k;
  if (N > 256) return 1;
#pragma omp parallel for schedule(static)
  for (int t = 0; t < c->T; ++t) {
    real g[256], P[256], wt[256];
    for (int i = 0; i < N; ++i) g[i] = (real)G[(int64_t)t * N + i];
    softmax_all(g, N, P);
    topk_token(c, g, P, NULL, idx + (int64_t)t * K, wt);
    for (int k = 0; k < K; ++k) w[(int64_t)t * K + k] = (float)wt[k];
    if (P_out)
      for (int i = 0; i < N; ++i) P_out[(int64_t)t * N + i] = (float)P[i];
  }
  return 0;
}

/* ---- grouping tables: FFN slots only, expert-major, ascending slot id inside an expert ------ */
int FN(tables)(const oracle_config* c, const int32_t* idx, int32_t* counts, int32_t* offsets, int32_t* row_of_slot,
               int32_t* slot_of_row) {
  if (bad_config(c) || !idx || !counts || !offsets) return 1;
  const int N = n_experts(c), K = c->top_k, A = c->row_align;
  const int64_t S = (int64_t)c->T * K;
  const int64_t M_cap = S + (int64_t)c->n_ffn * (A - 1);
  for (int e = 0; e < N; ++e) counts[e] = 0;
  for (int64_t s = 0; s < S; ++s) {
    if (idx[s] < 0 || idx[s] >= N) return 2;
    counts[idx[s]] += 1;
  }
  int32_t cap_ffn, cap_zc;
  oracle_capacities(c, &cap_ffn, &cap_zc);
  offsets[0] = 0;
  for (int e = 0; e < c->n_ffn; ++e) {
    const int kept = counts[e] < cap_ffn ? counts[e] : cap_ffn; /* Eq. 8: at most cap_ffn slots are served */
    offsets[e + 1] = offsets[e] + ((kept + A - 1) / A) * A;
  }
  if (!row_of_slot && !slot_of_row) return 0;
  if (slot_of_row)
    for (int64_t r = 0; r < M_cap; ++r) slot_of_row[r] = -1;
  int32_t* seen = (int32_t*)calloc((size_t)N, sizeof(int32_t));
  for (int64_t s = 0; s < S; ++s) { /* slot order = the order in which experts fill up */
    const int e = idx[s];
    const int32_t cap = e < c->n_ffn ? cap_ffn : cap_zc;
    int32_t row;
    if (seen[e] >= cap) {
      row = -2; /* dropped */
    } else if (e < c->n_ffn) {
      row = offsets[e] + seen[e];
      if (slot_of_row) slot_of_row[row] = (int32_t)s;
    } else {
      row = -1; /* zero-computation slots own no row */
    }
    seen[e] += 1;
    if (row_of_slot) row_of_slot[s] = row;
  }
  free(seen);
  return 0;
}

int FN(permute_rows)(const oracle_config* c, const float* x, const int32_t* slot_of_row, int64_t n_rows,
                     float* x_perm) {
  if (bad_config(c) || !x || !slot_of_row || !x_perm) return 1;
  const int D = c->D, K = c->top_k;
  for (int64_t r = 0; r < n_rows; ++r) {
    const int32_t s = slot_of_row[r];
    for (int d = 0; d < D; ++d) x_perm[r * D + d] = (s < 0) ? 0.0f : x[(int64_t)(s / K) * D + d];
  }
  return 0;
}

/* ---- Eq. 5: [alpha1, alpha2] = Softmax(W_c x) for one constant expert ----------------------- */
static void alpha_token(const oracle_config* c, const float* x_t, const float* W_c_e, real* a) {
  const int D = c->D;
  real z0 = 0, z1 = 0;
#pragma omp simd reduction(+ : z0, z1)
  for (int d = 0; d < D; ++d) {
    z0 += (real)W_c_e[d] * (real)x_t[d];
    z1 += (real)W_c_e[D + d] * (real)x_t[d];
  }
  real z[2] = {z0, z1};
  softmax_all(z, 2, a);
}

int FN(const_alpha)(const oracle_config* c, const float* x, const float* W_c, float* alpha) {
  if (bad_config(c) || !x || !alpha) return 1;
  if (c->n_const > 0 && !W_c) return 1;
#pragma omp parallel for schedule(static)
  for (int t = 0; t < c->T; ++t)
    for (int q = 0; q < c->n_const; ++q) {
      real a[2];
      alpha_token(c, x + (int64_t)t * c->D, W_c + (int64_t)q * 2 * c->D, a);
      alpha[((int64_t)t * c->n_const + q) * 2 + 0] = (float)a[0];
      alpha[((int64_t)t * c->n_const + q) * 2 + 1] = (float)a[1];
    }
  return 0;
}

/* ---- FFN expert: W_down ( silu(W_gate x) * (W_up x) ), silu(z) = z / (1 + exp(-z)) ---------- */
static void ffn_real(const oracle_config* c, const real* u, const void* Wg_e, const void* Wu_e, const void* Wd_e,
                     real* h, real* out) {
  const int D = c->D, F = c->F, b = c->ffn_w_bf16;
  for (int f = 0; f < F; ++f) {
    const real g = dot_w(Wg_e, f, D, b, u);
    const real up = dot_w(Wu_e, f, D, b, u);
    h[f] = (g / ((real)1 + r_exp(-g))) * up;
  }
  for (int d = 0; d < D; ++d) out[d] = dot_w(Wd_e, d, F, b, h);
}

int FN(ffn_token)(const oracle_config* c, const float* x_row, const void* Wg_e, const void* Wu_e, const void* Wd_e,
                  float* out_row) {
  if (bad_config(c) || !x_row || !Wg_e || !Wu_e || !Wd_e || !out_row) return 1;
  real* buf = (real*)malloc(sizeof(real) * (size_t)(2 * c->D + c->F));
  real *u = buf, *o = buf + c->D, *h = buf + 2 * c->D;
  for (int d = 0; d < c->D; ++d) u[d] = (real)x_row[d];
  ffn_real(c, u, Wg_e, Wu_e, Wd_e, h, o);
  for (int d = 0; d < c->D; ++d) out_row[d] = (float)o[d];
  free(buf);
  return 0;
}

static const void* expert_w(const void* W, int e, int64_t elems, int is_bf16) {
  return (const char*)W + (int64_t)e * elems * (is_bf16 ? 2 : 4);
}

int FN(grouped_ffn)(const oracle_config* c, const float* x_perm, const int32_t* offsets, const int32_t* counts,
                    const void* W_gate, const void* W_up, const void* W_down, float* y_perm) {
  if (bad_config(c) || !x_perm || !offsets || !counts || !y_perm) return 1;
  const int64_t DF = (int64_t)c->D * c->F;
  for (int e = 0; e < c->n_ffn; ++e) {
    const void* wg = expert_w(W_gate, e, DF, c->ffn_w_bf16);
    const void* wu = expert_w(W_up, e, DF, c->ffn_w_bf16);
    const void* wd = expert_w(W_down, e, DF, c->ffn_w_bf16);
#pragma omp parallel for schedule(dynamic, 4)
    for (int r = offsets[e]; r < offsets[e] + counts[e]; ++r)
      FN(ffn_token)(c, x_perm + (int64_t)r * c->D, wg, wu, wd, y_perm + (int64_t)r * c->D);
  }
  return 0;
}

/* ---- Eq. 1 sum with Eq. 3 (zero), Eq. 4 (copy), Eq. 5 (constant) in place ------------------- */
int FN(combine)(const oracle_config* c, const float* x, const float* y_perm, const int32_t* idx, const float* w,
                const int32_t* row_of_slot, const float* alpha, const float* v, float* y) {
  if (bad_config(c) || !x || !idx || !w || !y) return 1;
  const int D = c->D, K = c->top_k;
  const int zero0 = c->n_ffn, copy0 = zero0 + c->n_zero, const0 = copy0 + c->n_copy;
#pragma omp parallel for schedule(static)
  for (int t = 0; t < c->T; ++t) {
    const float* xt = x + (int64_t)t * D;
    for (int d = 0; d < D; ++d) {
      real acc = c->add_residual ? (real)xt[d] : (real)0;
      for (int k = 0; k < K; ++k) {
        const int e = idx[(int64_t)t * K + k];
        const real g = (real)w[(int64_t)t * K + k];
        real contrib;
        if (row_of_slot[(int64_t)t * K + k] == -2) {
          contrib = 0; /* Eq. 8: dropped at a full expert */
        } else if (e < zero0) {
          contrib = (real)y_perm[(int64_t)row_of_slot[(int64_t)t * K + k] * D + d];
        } else if (e < copy0) {
          contrib = 0; /* Eq. 3 */
        } else if (e < const0) {
          contrib = (real)xt[d]; /* Eq. 4 */
        } else {               /* Eq. 5 */
          const int q = e - const0;
          const real a1 = (real)alpha[((int64_t)t * c->n_const + q) * 2 + 0];
          const real a2 = (real)alpha[((int64_t)t * c->n_const + q) * 2 + 1];
          contrib = a1 * (real)xt[d] + a2 * (real)v[(int64_t)q * D + d];
        }
        acc += g * contrib;
      }
      y[(int64_t)t * D + d] = (float)acc;
    }
  }
  return 0;
}

/* ---- the whole layer by the definition: y = sum_i g_i E_i(x), no grouping -------------------- */
int FN(layer_forward)(const oracle_config* c, const float* x, const float* W_r, const float* W_g, const float* prev,
                      const float* bias, const float* W_c, const float* v, const void* W_gate, const void* W_up,
                      const void* W_down, const int32_t* forced_idx, const int32_t* tokens, int32_t n_tokens,
                      float* logits, int32_t* idx, float* w, float* y) {
  if (bad_config(c) || !x || !W_r || !logits || !idx || !w || !y) return 1;
  if ((W_g == NULL) != (prev == NULL)) return 1;
  const int N = n_experts(c), D = c->D, F = c->F, K = c->top_k;
  if (N > 256) return 1;
  if (c->n_const > 0 && (!W_c || !v)) return 1;
  if (c->n_ffn > 0 && (!W_gate || !W_up || !W_down)) return 1;
  const int zero0 = c->n_ffn, copy0 = zero0 + c->n_zero, const0 = copy0 + c->n_copy;
  const int64_t DF = (int64_t)D * F;

  /* routing for every token (cheap), so that logits / idx / w are complete */
#pragma omp parallel for schedule(static)
  for (int t = 0; t < c->T; ++t) {
    real g[256], P[256], wt[256];
    logits_token(c, x + (int64_t)t * D, W_r, W_g, prev ? prev + (int64_t)t * N : NULL, bias, g);
    /* the next layer (Eq. 6) and the top-K both see the logits as stored, in float */
    for (int i = 0; i < N; ++i) {
      logits[(int64_t)t * N + i] = (float)g[i];
      g[i] = (real)logits[(int64_t)t * N + i];
    }
    softmax_all(g, N, P);
    topk_token(c, g, P, forced_idx ? forced_idx + (int64_t)t * K : NULL, idx + (int64_t)t * K, wt);
    for (int k = 0; k < K; ++k) w[(int64_t)t * K + k] = (float)wt[k];
  }

  /* Eq. 8: serve slots in slot order; a slot that finds its expert full is dropped */
  int32_t cap_ffn, cap_zc;
  oracle_capacities(c, &cap_ffn, &cap_zc);
  char* dropped = (char*)calloc((size_t)c->T * K + 1, 1);
  if (c->capacity_factor > 0.0f) {
    int32_t seen[256];
    memset(seen, 0, sizeof seen);
    for (int64_t s = 0; s < (int64_t)c->T * K; ++s) {
      const int e = idx[s];
      if (seen[e] >= (e < zero0 ? cap_ffn : cap_zc)) dropped[s] = 1;
      seen[e] += 1;
    }
  }

  const int n_out = tokens ? n_tokens : c->T;
#pragma omp parallel
  {
    real* buf = (real*)malloc(sizeof(real) * (size_t)(3 * D + F));
    real *u = buf, *e_out = buf + D, *acc = buf + 2 * D, *h = buf + 3 * D;
#pragma omp for schedule(dynamic, 1)
    for (int j = 0; j < n_out; ++j) {
      const int t = tokens ? tokens[j] : j;
      const float* xt = x + (int64_t)t * D;
      for (int d = 0; d < D; ++d) {
        u[d] = (real)xt[d];
        acc[d] = c->add_residual ? u[d] : (real)0;
      }
      for (int k = 0; k < K; ++k) {
        const int e = idx[(int64_t)t * K + k];
        /* the weight as stored (float), the same value the combine step is handed */
        const real g = (real)w[(int64_t)t * K + k];
        if (dropped[(int64_t)t * K + k]) continue;
        if (e < zero0) {
          ffn_real(c, u, expert_w(W_gate, e, DF, c->ffn_w_bf16), expert_w(W_up, e, DF, c->ffn_w_bf16),
                   expert_w(W_down, e, DF, c->ffn_w_bf16), h, e_out);
        } else if (e < copy0) {
          for (int d = 0; d < D; ++d) e_out[d] = 0; /* Eq. 3 */
        } else if (e < const0) {
          for (int d = 0; d < D; ++d) e_out[d] = u[d]; /* Eq. 4 */
        } else {                                       /* Eq. 5 */
          const int q = e - const0;
          real a[2];
          alpha_token(c, xt, W_c + (int64_t)q * 2 * D, a);
          for (int d = 0; d < D; ++d) e_out[d] = a[0] * u[d] + a[1] * (real)v[(int64_t)q * D + d];
        }
        for (int d = 0; d < D; ++d) acc[d] += g * e_out[d];
      }
      for (int d = 0; d < D; ++d) y[(int64_t)j * D + d] = (float)acc[d];
    }
    free(buf);
  }
  free(dropped);
  return 0;
}

/* ---- Eq. 7: heterogeneous load-balance statistics ------------------------------------------------ */
int FN(balance_stats)(const oracle_config* c, const float* G, const int32_t* idx, float* f, float* Pm,
                      float* loss) {
  if (bad_config(c) || !G || !idx || !f || !Pm || !loss) return 1;
  const int N = n_experts(c), K = c->top_k;
  if (N > 256) return 1;
  const real tau = c->tau > 0.0f ? (real)c->tau : (real)1;
  real fs[256], ps[256];
  for (int i = 0; i < N; ++i) { fs[i] = 0; ps[i] = 0; }
  for (int t = 0; t < c->T; ++t) {
    real g[256], P[256];
    for (int i = 0; i < N; ++i) g[i] = (real)G[(int64_t)t * N + i];
    softmax_all(g, N, P);
    for (int i = 0; i < N; ++i) ps[i] += P[i];
    for (int k = 0; k < K; ++k) fs[idx[(int64_t)t * K + k]] += 1; /* token t selects this expert */
  }
  real L = 0;
  for (int i = 0; i < N; ++i) {
    const real fi = c->T > 0 ? fs[i] / (real)c->T : 0, pi = c->T > 0 ? ps[i] / (real)c->T : 0;
    const real eta = i < c->n_ffn ? (real)1 : tau;
    f[i] = (float)fi;
    Pm[i] = (float)pi;
    L += eta * fi * pi;
  }
  *loss = (float)L;
  return 0;
}

/* ---- Eq. 7 differentiated with respect to the router logits ----------------------------------------
 * L_b = sum_i eta_i f_i P_i, P_i = (1/T) sum_t softmax(G_t)_i.  f_i counts selections and is piecewise
 * constant in G, so only P_i carries a gradient:
 *   d(scale L_b)/dG[t,j] = (scale/T) P_tj (c_j - sum_i c_i P_ti),  c_i = eta_i f_i.
 * accumulate != 0 adds to dG instead of overwriting it. */
int FN(balance_backward)(const oracle_config* c, const float* G, const float* f, float scale, int accumulate,
                         float* dG) {
  if (bad_config(c) || !G || !f || !dG) return 1;
  const int N = n_experts(c);
  if (N > 256) return 1;
  const real tau = c->tau > 0.0f ? (real)c->tau : (real)1;
  real ci[256];
  for (int i = 0; i < N; ++i) ci[i] = (i < c->n_ffn ? (real)1 : tau) * (real)f[i];
  for (int t = 0; t < c->T; ++t) {
    real g[256], P[256];
    for (int i = 0; i < N; ++i) g[i] = (real)G[(int64_t)t * N + i];
    softmax_all(g, N, P);
    real dot = 0;
    for (int i = 0; i < N; ++i) dot += ci[i] * P[i];
    for (int j = 0; j < N; ++j) {
      const real v = (real)scale / (real)c->T * P[j] * (ci[j] - dot);
      float* out = dG + (int64_t)t * N + j;
      *out = accumulate ? (float)((real)*out + v) : (float)v;
    }
  }
  return 0;
}

/* ==== backward pass: chain rule through Eq. 1-6, token by token ===================================== */

/* gradient accumulators for the weights, in `real`, rounded to float once at the end */
static real* zeros_real(size_t n) { return (real*)calloc(n > 0 ? n : 1, sizeof(real)); }
static void store_f32(float* dst, const real* src, size_t n) {
  if (!dst) return;
  for (size_t i = 0; i < n; ++i) dst[i] = (float)src[i];
}

/* one FFN expert on token u: forward values kept, then the gradient of dc = dL/d(out) */
static void ffn_backward_token(const oracle_config* c, const real* u, const float* Wg, const float* Wu,
                               const float* Wd, const real* dc, real* du, real* gWg, real* gWu, real* gWd,
                               real* out, real* scratch) {
  const int D = c->D, F = c->F;
  real *gt = scratch, *up = scratch + F, *sg = scratch + 2 * F, *h = scratch + 3 * F, *dh = scratch + 4 * F;
  for (int f = 0; f < F; ++f) {
    real a = 0, b = 0;
    for (int d = 0; d < D; ++d) {
      a += (real)Wg[(int64_t)f * D + d] * u[d];
      b += (real)Wu[(int64_t)f * D + d] * u[d];
    }
    gt[f] = a;
    up[f] = b;
    sg[f] = (real)1 / ((real)1 + r_exp(-a)); /* sigmoid */
    h[f] = a * sg[f] * b;                     /* silu(gate) * up */
  }
  for (int d = 0; d < D; ++d) {
    real o = 0;
    for (int f = 0; f < F; ++f) o += (real)Wd[(int64_t)d * F + f] * h[f];
    out[d] = o;
  }
  if (!dc) return;
  for (int f = 0; f < F; ++f) {
    real a = 0;
    for (int d = 0; d < D; ++d) a += dc[d] * (real)Wd[(int64_t)d * F + f];
    dh[f] = a;
  }
  for (int d = 0; d < D; ++d)
    for (int f = 0; f < F; ++f) gWd[(int64_t)d * F + f] += dc[d] * h[f];
  for (int f = 0; f < F; ++f) {
    const real d_up = dh[f] * gt[f] * sg[f];
    /* d silu(z)/dz = s + z s (1 - s) */
    const real d_gt = dh[f] * up[f] * (sg[f] + gt[f] * sg[f] * ((real)1 - sg[f]));
    for (int d = 0; d < D; ++d) {
      gWg[(int64_t)f * D + d] += d_gt * u[d];
      gWu[(int64_t)f * D + d] += d_up * u[d];
      du[d] += d_gt * (real)Wg[(int64_t)f * D + d] + d_up * (real)Wu[(int64_t)f * D + d];
    }
  }
}

int FN(layer_backward)(const oracle_config* c, const float* x, const float* W_r, const float* W_g, const float* prev,
                       const float* bias, const float* W_c, const float* v, const float* W_gate, const float* W_up,
                       const float* W_down, const int32_t* idx, const float* dy, const float* dlogits, float* dx,
                       float* dprev, float* dW_r, float* dW_g, float* dbias, float* dW_c, float* dv, float* dW_gate,
                       float* dW_up, float* dW_down) {
  if (bad_config(c) || !x || !W_r || !idx || !dy || !dx || !dW_r) return 1;
  if ((W_g == NULL) != (prev == NULL)) return 1;
  const int N = n_experts(c), D = c->D, F = c->F, K = c->top_k, T = c->T;
  if (N > 256 || c->ffn_w_bf16) return 1;
  const int zero0 = c->n_ffn, copy0 = zero0 + c->n_zero, const0 = copy0 + c->n_copy;
  const int64_t DF = (int64_t)D * F;

  real* gWr = zeros_real((size_t)N * D);
  real* gWgate = zeros_real((size_t)c->n_ffn * DF), *gWup = zeros_real((size_t)c->n_ffn * DF);
  real* gWdown = zeros_real((size_t)c->n_ffn * DF);
  real* gWg = zeros_real((size_t)N * N), *gb = zeros_real((size_t)N);
  real* gWc = zeros_real((size_t)c->n_const * 2 * D), *gv = zeros_real((size_t)c->n_const * D);
  real* buf = (real*)malloc(sizeof(real) * (size_t)(4 * D + 5 * F + 8));
  real *u = buf, *du = buf + D, *dc = buf + 2 * D, *out = buf + 3 * D, *scratch = buf + 4 * D;

  /* Eq. 8: which slots were dropped (same rule as the forward pass) */
  int32_t cap_ffn, cap_zc;
  oracle_capacities(c, &cap_ffn, &cap_zc);
  char* dropped = (char*)calloc((size_t)T * K + 1, 1);
  if (c->capacity_factor > 0.0f) {
    int32_t seen[256];
    memset(seen, 0, sizeof seen);
    for (int64_t s = 0; s < (int64_t)T * K; ++s) {
      const int e = idx[s];
      if (seen[e] >= (e < zero0 ? cap_ffn : cap_zc)) dropped[s] = 1;
      seen[e] += 1;
    }
  }

  for (int t = 0; t < T; ++t) {
    const float* xt = x + (int64_t)t * D;
    const float* dyt = dy + (int64_t)t * D;
    real g[256], P[256], wk[256], dw[256], dG[256];
    logits_token(c, xt, W_r, W_g, prev ? prev + (int64_t)t * N : NULL, bias, g);
    for (int i = 0; i < N; ++i) g[i] = (real)(float)g[i]; /* the forward pass stores the logits in float */
    softmax_all(g, N, P);
    real S = 0;
    for (int k = 0; k < K; ++k) S += P[idx[(int64_t)t * K + k]];
    for (int k = 0; k < K; ++k) {
      wk[k] = P[idx[(int64_t)t * K + k]];
      if (c->renorm_topk) wk[k] = wk[k] / S;
      wk[k] = (real)(float)wk[k]; /* stored in float by the forward pass */
    }
    for (int d = 0; d < D; ++d) {
      u[d] = (real)xt[d];
      du[d] = c->add_residual ? (real)dyt[d] : (real)0; /* y = x + ... */
    }
    for (int k = 0; k < K; ++k) {
      const int e = idx[(int64_t)t * K + k];
      dw[k] = 0;
      if (dropped[(int64_t)t * K + k]) continue;
      for (int d = 0; d < D; ++d) dc[d] = wk[k] * (real)dyt[d]; /* dL/d E_k(x) */
      if (e < zero0) {
        ffn_backward_token(c, u, W_gate + e * DF, W_up + e * DF, W_down + e * DF, dc, du, gWgate + e * DF,
                           gWup + e * DF, gWdown + e * DF, out, scratch);
        for (int d = 0; d < D; ++d) dw[k] += (real)dyt[d] * out[d];
      } else if (e < copy0) {
        /* Eq. 3: E = 0, nothing flows */
      } else if (e < const0) { /* Eq. 4: E = x */
        for (int d = 0; d < D; ++d) {
          dw[k] += (real)dyt[d] * u[d];
          du[d] += dc[d];
        }
      } else { /* Eq. 5: E = a1 x + a2 v, a = softmax(W_c x) */
        const int q = e - const0;
        const float* Wc = W_c + (int64_t)q * 2 * D;
        const float* vq = v + (int64_t)q * D;
        real a[2];
        alpha_token(c, xt, Wc, a);
        real da1 = 0, da2 = 0;
        for (int d = 0; d < D; ++d) {
          dw[k] += (real)dyt[d] * (a[0] * u[d] + a[1] * (real)vq[d]);
          da1 += dc[d] * u[d];
          da2 += dc[d] * (real)vq[d];
          du[d] += a[0] * dc[d];
          gv[(int64_t)q * D + d] += a[1] * dc[d];
        }
        const real mean = a[0] * da1 + a[1] * da2; /* softmax backward over the two mixing logits */
        const real dz0 = a[0] * (da1 - mean), dz1 = a[1] * (da2 - mean);
        for (int d = 0; d < D; ++d) {
          gWc[((int64_t)q * 2 + 0) * D + d] += dz0 * u[d];
          gWc[((int64_t)q * 2 + 1) * D + d] += dz1 * u[d];
          du[d] += dz0 * (real)Wc[d] + dz1 * (real)Wc[D + d];
        }
      }
    }
    /* gate: w_k = P[idx_k] (/ sum over the picks if renormalised); softmax over all N */
    real dP[256];
    for (int i = 0; i < N; ++i) dP[i] = 0;
    if (c->renorm_topk) {
      real dot = 0;
      for (int k = 0; k < K; ++k) dot += dw[k] * wk[k];
      for (int k = 0; k < K; ++k) dP[idx[(int64_t)t * K + k]] += (dw[k] - dot) / S;
    } else {
      for (int k = 0; k < K; ++k) dP[idx[(int64_t)t * K + k]] += dw[k];
    }
    real dotP = 0;
    for (int i = 0; i < N; ++i) dotP += dP[i] * P[i];
    for (int i = 0; i < N; ++i) {
      dG[i] = P[i] * (dP[i] - dotP);
      if (dlogits) dG[i] += (real)dlogits[(int64_t)t * N + i]; /* the next layer's gating residual reads G */
    }
    /* router: G = W_r x + W_g G_prev + b */
    for (int i = 0; i < N; ++i) {
      for (int d = 0; d < D; ++d) {
        gWr[(int64_t)i * D + d] += dG[i] * u[d];
        du[d] += dG[i] * (real)W_r[(int64_t)i * D + d];
      }
      gb[i] += dG[i];
    }
    if (W_g) {
      for (int j = 0; j < N; ++j) {
        real a = 0;
        for (int i = 0; i < N; ++i) {
          a += dG[i] * (real)W_g[i * N + j];
          gWg[i * N + j] += dG[i] * (real)prev[(int64_t)t * N + j];
        }
        if (dprev) dprev[(int64_t)t * N + j] = (float)a;
      }
    }
    for (int d = 0; d < D; ++d) dx[(int64_t)t * D + d] = (float)du[d];
  }
  store_f32(dW_r, gWr, (size_t)N * D);
  store_f32(dW_g, gWg, (size_t)N * N);
  store_f32(dbias, gb, (size_t)N);
  store_f32(dW_c, gWc, (size_t)c->n_const * 2 * D);
  store_f32(dv, gv, (size_t)c->n_const * D);
  store_f32(dW_gate, gWgate, (size_t)c->n_ffn * DF);
  store_f32(dW_up, gWup, (size_t)c->n_ffn * DF);
  store_f32(dW_down, gWdown, (size_t)c->n_ffn * DF);
  free(gWr); free(gWgate); free(gWup); free(gWdown); free(gWg); free(gb); free(gWc); free(gv); free(buf);
  free(dropped);
  return 0;
}
