/*
 * CPU oracle for the forward pass of one MoE++ layer (arXiv 2410.07348).
 *
 * TEST INFRASTRUCTURE ONLY.  This is a plain, slow, token-by-token restatement
 * of the paper's definitions.  It exists so that the CUDA library can be checked
 * against something that is obviously the paper's mathematics.  It shares no
 * code, header, table or helper with the CUDA library, and nothing in the
 * product path may call it.
 *
 * Every function exists twice: oracle_f32_<name> does all arithmetic in float,
 * oracle_f64_<name> does all arithmetic in double (inputs and outputs are float
 * arrays either way).  The f64 build is the referee used for parity; the f32
 * build bounds how much of a difference is just rounding.
 *
 * Expert index space (the paper lists the kinds as Zero/Copy/Constant, Table 2):
 *   [0, n_ffn)                    FFN experts
 *   [n_ffn, +n_zero)              zero experts      Eq. 3
 *   [.., +n_copy)                 copy experts      Eq. 4
 *   [.., +n_const)                constant experts  Eq. 5
 * N = n_ffn + n_zero + n_copy + n_const.
 *
 * Readings of points the paper leaves open (each is also listed in the design
 * notes of the repository):
 *   - gate weight = softmax over ALL N logits, then masked to the top-K (Eq. 1
 *     as printed); no renormalisation unless renorm_topk is set.
 *   - top-K is taken on the logits; larger logit first, equal logits -> lower
 *     expert index first.
 *   - the gating residual (Eq. 6) consumes the previous layer's full
 *     pre-softmax logits.
 *   - each constant expert owns its own W_c (2 x D) and v (D).
 *   - the FFN expert is a bias-free SwiGLU: W_down (silu(W_gate x) * (W_up x)).
 *   - no capacity limit unless capacity_factor > 0.  With a limit (Eq. 8), slots are served in slot
 *     order (token-major, then pick order); a slot that arrives at a full expert is dropped: it
 *     contributes nothing to y (the token passes on through the residual stream), owns no row
 *     (row_of_slot = -2) and causes no FFN work.  expert_counts stay the selection counts.
 *
 * Parity pins: see tests/test_oracle_*.py.  No function here is unpinned.
 */
#ifndef MOEPP_ORACLE_H
#define MOEPP_ORACLE_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct {
  int32_t T, D, F;
  int32_t n_ffn, n_zero, n_copy, n_const;
  int32_t top_k;
  int32_t renorm_topk;  /* 0: Eq. 1 as printed; 1: divide the K weights by their sum */
  int32_t row_align;    /* each FFN expert's row segment is padded to a multiple of this (>= 1) */
  int32_t add_residual; /* 1: y = x + Eq. 1 (used only when layers are stacked) */
  int32_t ffn_w_bf16;   /* 0: FFN weights are float; 1: they are bf16 bit patterns (uint16_t) */
  float tau;            /* Eq. 7 / Eq. 8: weight of the zero-computation experts; <= 0 means 1 */
  float capacity_factor; /* Eq. 8 gamma; <= 0: no capacity limit (nothing is dropped) */
} oracle_config;

/* Eq. 8 with T read as the number of routing slots T*K (for K = 1 the printed formula), rounded up:
 *   FFN expert:              ceil(gamma * tau * T*K / (tau * N_FFN + N_ZC))
 *   zero-computation expert: ceil(gamma *       T*K / (tau * N_FFN + N_ZC))
 * Both are INT32_MAX when capacity_factor <= 0. */
void oracle_capacities(const oracle_config* c, int32_t* cap_ffn, int32_t* cap_zc);

int oracle_num_threads(void);

#define ORACLE_DECLARE(P)                                                                          \
  /* Eq. 2 / Eq. 6 (+ optional bias, which is not part of the method): G[t,i]. */                  \
  int P##router_logits(const oracle_config* c, const float* x, const float* W_r,                   \
                       const float* W_g, const float* prev, const float* bias, float* G);          \
  /* Eq. 1 gate: softmax over all N, top-K on logits.  P_out may be NULL. */                       \
  int P##gate_topk(const oracle_config* c, const float* G, int32_t* idx, float* w, float* P_out);  \
  /* Grouping tables for FFN slots only.  row_of_slot: row | -1 (zero-computation slot) | -2 (dropped, Eq. 8). */                                                        \
  int P##tables(const oracle_config* c, const int32_t* idx, int32_t* counts, int32_t* offsets,     \
                int32_t* row_of_slot, int32_t* slot_of_row);                                       \
  /* x_perm[row] = x[slot_of_row[row] / K]; rows with slot -1 are set to 0. */                     \
  int P##permute_rows(const oracle_config* c, const float* x, const int32_t* slot_of_row,          \
                      int64_t n_rows, float* x_perm);                                              \
  /* Eq. 5 mixing weights: alpha[t,c,:] = softmax(W_c^(c) x_t). */                                 \
  int P##const_alpha(const oracle_config* c, const float* x, const float* W_c, float* alpha);      \
  /* One FFN expert on one token. */                                                               \
  int P##ffn_token(const oracle_config* c, const float* x_row, const void* Wg_e,                   \
                   const void* Wu_e, const void* Wd_e, float* out_row);                            \
  /* FFN expert e on every row of its segment [offsets[e], offsets[e]+counts[e]). */               \
  int P##grouped_ffn(const oracle_config* c, const float* x_perm, const int32_t* offsets,          \
                     const int32_t* counts, const void* W_gate, const void* W_up,                  \
                     const void* W_down, float* y_perm);                                           \
  /* Eq. 1 sum over the K slots with Eq. 3-5 applied in place. */                                  \
  int P##combine(const oracle_config* c, const float* x, const float* y_perm, const int32_t* idx,  \
                 const float* w, const int32_t* row_of_slot, const float* alpha, const float* v,   \
                 float* y);                                                                        \
  /* Eq. 7: f[i] = share of tokens that select expert i, P[i] = mean softmax weight of expert i,            \
     loss = sum_i eta_i f[i] P[i] with eta = 1 (FFN) or tau (zero-computation). */                           \
  int P##balance_stats(const oracle_config* c, const float* G, const int32_t* idx, float* f, float* Pm,     \
                       float* loss);                                                                        \
  int P##balance_backward(const oracle_config* c, const float* G, const float* f, float scale,             \
                          int accumulate, float* dG);                                                       \
  /* Whole layer by the definition, token by token, without any grouping.                          \
     tokens==NULL: all T tokens, y is [T,D]; else y is [n_tokens,D] for the listed tokens.         \
     forced_idx (may be NULL) replaces the top-K choice; the weights still come from the           \
     oracle's own softmax.  logits/idx/w are always produced for all T tokens. */                  \
  int P##layer_forward(const oracle_config* c, const float* x, const float* W_r,                   \
                       const float* W_g, const float* prev, const float* bias, const float* W_c,   \
                       const float* v, const void* W_gate, const void* W_up, const void* W_down,   \
                       const int32_t* forced_idx, const int32_t* tokens, int32_t n_tokens,         \
                       float* logits, int32_t* idx, float* w, float* y);

/* Backward pass of the layer: the gradient of a scalar L with respect to every input, given
 * dy = dL/dy [T,D] and (may be NULL) dlogits = dL/dlogits [T,N] arriving from the next layer's
 * gating residual (Eq. 6).  It is the chain rule written out token by token for Eq. 1-6 with the picks
 * `idx` held fixed (top-K itself has no gradient; slots dropped by Eq. 8 have none either).
 * All gradient outputs are float arrays of the shape of the thing they belong to; dprev, dW_g, dbias may be
 * NULL when the layer has no such input.  FFN weights must be float here. */
#define ORACLE_DECLARE_BWD(P)                                                                          \
  int P##layer_backward(const oracle_config* c, const float* x, const float* W_r, const float* W_g,    \
                        const float* prev, const float* bias, const float* W_c, const float* v,        \
                        const float* W_gate, const float* W_up, const float* W_down,                   \
                        const int32_t* idx, const float* dy, const float* dlogits, float* dx,          \
                        float* dprev, float* dW_r, float* dW_g, float* dbias, float* dW_c, float* dv,  \
                        float* dW_gate, float* dW_up, float* dW_down);

ORACLE_DECLARE(oracle_f32_)
ORACLE_DECLARE(oracle_f64_)
ORACLE_DECLARE_BWD(oracle_f32_)
ORACLE_DECLARE_BWD(oracle_f64_)

#ifdef __cplusplus
}
#endif
#endif
