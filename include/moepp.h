/*
 * moepp.h -- C ABI of the MoE++ heterogeneous expert layer (forward pass) for NVIDIA B200 (sm_100a).
 *
 * The layer is the one defined in "MoE++: Accelerating Mixture-of-Experts Methods with
 * Zero-Computation Experts" (arXiv 2410.07348):
 *   Eq. 1  y = sum_i g_i E_i(x),  g_i = Softmax(G(x))_i if i is among the Top-K logits, else 0
 *   Eq. 2  vanilla router G(x) = W x
 *   Eq. 3  zero expert      E(x) = 0
 *   Eq. 4  copy expert      E(x) = x
 *   Eq. 5  constant expert  E(x) = a1 x + a2 v,  [a1, a2] = Softmax(W_c x)
 *   Eq. 6  gating residual  G(x^j) = W^j x^j + W_g^j G(x^{j-1})   (first layer: no residual term)
 * FFN experts are bias-free SwiGLU networks: W_down (silu(W_gate x) * (W_up x)).
 *
 * Conventions shared by every call
 *   - All pointers are DEVICE pointers owned by the caller unless a parameter says "host".
 *     The library allocates nothing and frees nothing.  Work is enqueued on `stream`
 *     (a cudaStream_t passed as void*; NULL = the default stream) and the call returns
 *     without synchronising.
 *   - Row-major everywhere.  T tokens, D model width, F FFN width, K = top_k,
 *     N = n_ffn + n_zero + n_copy + n_const experts, indexed in that order
 *     (FFN | zero | copy | constant).  Slot s = t*K + k is the k-th pick of token t.
 *   - `dtype` is the storage type of x, y, x_perm, h, y_perm and the FFN weights.
 *     Router weights, logits, gate weights, W_c, v and all accumulation are float.
 *   - Activation, FFN-weight and topk_idx pointers must be 16-byte aligned; D and F must be
 *     multiples of 8 (MOEPP_ERR_ALIGN otherwise).
 *   - M_cap = T*K + n_ffn*(row_align-1) is the row capacity of the grouped buffers.
 *   - Errors are returned, never thrown: argument errors are found on the host before
 *     anything is launched; MOEPP_ERR_CUDA wraps a failed launch.  T == 0 is valid and does nothing.
 *   - Limits: N <= 64, 1 <= K <= min(N, 8), N + 2*n_const <= 128.
 *   - Expert capacity (Eq. 8), only when capacity_factor > 0: with S = T*K routing slots an FFN expert
 *     serves at most ceil(gamma*tau*S / (tau*n_ffn + n_zc)) slots and a zero-computation expert at most
 *     ceil(gamma*S / (tau*n_ffn + n_zc)) (Eq. 8 with its T read as the number of routing slots; for K = 1
 *     it is the printed formula).  Slots are served in slot order; a slot that arrives at a full expert
 *     is dropped: row_of_slot = -2, no grouped row, no FFN work, no contribution to y (the token passes
 *     on through the residual stream).  expert_counts always are the selection counts; expert_offsets
 *     count served slots only.
 */
#ifndef MOEPP_H
#define MOEPP_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  MOEPP_OK = 0,
  MOEPP_ERR_INVALID_ARG = 1,
  MOEPP_ERR_UNSUPPORTED = 2,
  MOEPP_ERR_ALIGN = 3,
  MOEPP_ERR_WORKSPACE = 4,
  MOEPP_ERR_CUDA = 5,
  MOEPP_ERR_TIMEOUT = 6
} moepp_status;

typedef enum { MOEPP_F32 = 0, MOEPP_BF16 = 1 } moepp_dtype;

/* flags */
#define MOEPP_FLAG_LOGITS_GIVEN 1 /* moepp_route reads `logits` instead of computing Eq. 2 / Eq. 6 */
#define MOEPP_FLAG_SIMT_FFN 2     /* bf16 only: run the FFN on the plain FMA kernel (cross-check path) */
#define MOEPP_FLAG_FUSED_GATHER 8  /* moepp_layer_forward, bf16: GEMM 1 fetches its rows from x with TMA gather loads
                                      and x_perm is never built (measured slower than the staged default on B200) */
#define MOEPP_FLAG_FFN_SINGLE_CTA 4 /* bf16 only: 128x256 tiles on single CTAs instead of 256x256 on CTA pairs */
#define MOEPP_FLAG_SAVE_PREACT 16 /* moepp_layer_forward: also keep the SwiGLU pre-activations (gate and up, [M_cap, F]
                                     each) in the workspace, which grows accordingly; moepp_layer_backward then skips
                                     their recomputation.  Not with MOEPP_FLAG_FFN_SINGLE_CTA / MOEPP_FLAG_FUSED_GATHER. */
#define MOEPP_FLAG_ACCUM_GRADS 32 /* moepp_layer_backward / moepp_stack_backward: ADD the weight gradients (dW_r, dW_g,
                                     dbias, dW_c, dv, dW_gate, dW_up, dW_down) to what the buffers hold instead of
                                     overwriting them (gradient accumulation over micro-batches); dx and dprev are
                                     always overwritten */

typedef struct {
  int32_t T, D, F;
  int32_t n_ffn, n_zero, n_copy, n_const; /* expert index order: FFN | zero | copy | constant */
  int32_t top_k;                          /* the paper uses 2 in every layer */
  int32_t dtype;                          /* moepp_dtype */
  int32_t renorm_topk;                    /* 0: Eq. 1 as printed; 1: divide the K gate weights by their sum */
  int32_t row_align;                      /* 1: dense grouped layout; >1: pad each expert's rows to a multiple */
  int32_t add_residual;                   /* 0: y is Eq. 1; 1: y = x + Eq. 1 (for stacking layers) */
  int32_t flags;                          /* MOEPP_FLAG_* */
  float tau;                              /* Eq. 7 / Eq. 8: weight of the zero-computation experts; <= 0 means 1 */
  float capacity_factor;                  /* Eq. 8 gamma; <= 0 (default): no capacity limit, nothing is dropped */
} moepp_config;

typedef struct {
  const float* W_r;         /* [N, D]            Eq. 2 / Eq. 6 */
  const float* W_g;         /* [N, N] or NULL    Eq. 6 */
  const float* W_c;         /* [n_const, 2, D]   Eq. 5 (each constant expert has its own) */
  const float* v;           /* [n_const, D]      Eq. 5 */
  const float* router_bias; /* [N] or NULL; not part of the method, only shapes the load in benchmarks */
  const void* W_gate;       /* [n_ffn, F, D] */
  const void* W_up;         /* [n_ffn, F, D] */
  const void* W_down;       /* [n_ffn, D, F] */
} moepp_weights;

const char* moepp_status_string(moepp_status s);

/* Bytes of device scratch moepp_layer_forward needs for this configuration (a pure host computation). */
moepp_status moepp_workspace_bytes(const moepp_config* cfg, size_t* bytes);

/*
 * Router (Eq. 2, Eq. 6), gate (Eq. 1) and, if alpha is wanted, the constant experts' mixing weights (Eq. 5).
 *   logits[t,i] = W_r[i,:].x[t,:] (+ W_g[i,:].prev_logits[t,:]) (+ router_bias[i])
 *   P = softmax(logits[t,:]) over all N; the K largest logits are picked, larger first, equal
 *   logits -> lower index first; topk_w = P at the picks (divided by their sum if renorm_topk).
 *   expert_counts[e] = number of slots routed to e (all N experts);
 *   expert_offsets[e] = first grouped row of FFN expert e, expert_offsets[n_ffn] = rows in use;
 *   each expert's segment is its count rounded up to row_align.
 * W_g and prev_logits are both NULL (first layer) or both set.  alpha may be NULL (then W_c is unused).
 * With MOEPP_FLAG_LOGITS_GIVEN `logits` is an input and W_r, W_g, prev_logits, router_bias are ignored.
 */
moepp_status moepp_route(const moepp_config* cfg, const void* x, const float* W_r, const float* W_g,
                         const float* prev_logits, const float* router_bias, const float* W_c,
                         float* logits,           /* [T, N] out (in with MOEPP_FLAG_LOGITS_GIVEN) */
                         int32_t* topk_idx,       /* [T, K] out */
                         float* topk_w,           /* [T, K] out */
                         int32_t* expert_counts,  /* [N] out */
                         int32_t* expert_offsets, /* [n_ffn + 1] out */
                         float* alpha,            /* [T, n_const, 2] out, or NULL */
                         void* stream);

/*
 * Grouping of the FFN slots only; zero-computation slots get no row (the efficiency argument of the
 * paper's Section 3.4 made literal).  Rows are expert-major and, inside an expert, ascend in slot id.
 *   row_of_slot[s] = grouped row of slot s, or -1 for a zero-computation slot, or -2 for a slot dropped
 *                    at a full expert (Eq. 8; never without capacity_factor)
 *   slot_of_row[r] = slot held by row r, or -1 for a pad row / a row beyond expert_offsets[n_ffn]
 *   x_perm[r,:]    = x[slot_of_row[r] / K, :]; pad rows inside a segment are zero-filled; rows at or
 *                    beyond expert_offsets[n_ffn] are left untouched.
 */
moepp_status moepp_permute(const moepp_config* cfg, const void* x, const int32_t* topk_idx,
                           const int32_t* expert_offsets,
                           int32_t* row_of_slot, /* [T, K] out */
                           int32_t* slot_of_row, /* [M_cap] out */
                           void* x_perm,         /* [M_cap, D] out */
                           void* stream);

/*
 * Grouped SwiGLU FFN: for each FFN expert e and each row r in [expert_offsets[e], expert_offsets[e+1])
 *   h[r,:] = silu(W_gate[e] x_perm[r,:]) * (W_up[e] x_perm[r,:]);  y_perm[r,:] = W_down[e] h[r,:].
 * bf16: tcgen05 tensor-core kernels fed by TMA, float accumulation in tensor memory, h and y_perm
 * rounded once to bf16.  f32: FMA kernels.  h_ws is caller-provided scratch of M_cap*F elements.
 */
moepp_status moepp_grouped_ffn(const moepp_config* cfg, const void* x_perm, const int32_t* expert_offsets,
                               const void* W_gate, const void* W_up, const void* W_down,
                               void* h_ws,   /* [M_cap, F] scratch */
                               void* y_perm, /* [M_cap, D] out */
                               void* stream);

/*
 * Weighted combine (Eq. 1) with the zero-computation experts applied in place:
 *   y[t,:] = (x[t,:] if add_residual) + sum_k topk_w[t,k] * c(t,k),
 *   c = y_perm[row_of_slot[t,k],:] (FFN) | 0 (Eq. 3) | x[t,:] (Eq. 4) | a1 x[t,:] + a2 v[q,:] (Eq. 5).
 * alpha may be NULL; the mixing weights are then computed here from W_c and x.
 */
moepp_status moepp_combine(const moepp_config* cfg, const void* x, const void* y_perm, const int32_t* topk_idx,
                           const float* topk_w, const int32_t* row_of_slot,
                           const float* alpha, /* [T, n_const, 2] or NULL */
                           const float* W_c, const float* v,
                           void* y, /* [T, D] out */
                           void* stream);

/*
 * One whole layer: route -> permute -> grouped FFN -> combine, on one stream, without host
 * synchronisation.  prev_logits is NULL for the first layer (then W_g must be NULL too).
 * logits_out ([T, N], may be NULL) receives this layer's logits for the next layer's Eq. 6.
 * workspace: device scratch of at least moepp_workspace_bytes(), 256-byte aligned.
 */
moepp_status moepp_layer_forward(const moepp_config* cfg, const moepp_weights* weights, const void* x,
                                 const float* prev_logits, void* y, float* logits_out, void* workspace,
                                 size_t workspace_bytes, void* stream);

/*
 * The same layer for a caller whose activations live in HOST memory (pinned memory for the copies
 * to be asynchronous): x_host, prev_logits_host (or NULL), y_host and logits_out_host (or NULL) are
 * host pointers; weights and workspace stay on the device.  The workspace must be
 * moepp_workspace_bytes_host() large; copies and kernels are enqueued on `stream`, and the host
 * buffers are valid once the stream has been synchronised.
 */
moepp_status moepp_workspace_bytes_host(const moepp_config* cfg, size_t* bytes);
moepp_status moepp_layer_forward_host(const moepp_config* cfg, const moepp_weights* weights, const void* x_host,
                                      const float* prev_logits_host, void* y_host, float* logits_out_host,
                                      void* workspace, size_t workspace_bytes, void* stream);

/*
 * Heterogeneous load-balance statistics (Eq. 7), by-products of the router:
 *   f[i] = expert_counts[i] / T   share of tokens that select expert i (sums to K)
 *   P[i] = (1/T) sum_t Softmax(logits[t,:])_i
 *   *loss = sum_i eta_i f[i] P[i],  eta_i = 1 for FFN experts and tau for zero-computation experts.
 * f, P ([N] each) and loss ([1]) are device pointers.  The reduction order is fixed: results are
 * reproducible from run to run.
 */
moepp_status moepp_balance_stats(const moepp_config* cfg, const float* logits, const int32_t* expert_counts, float* f,
                                 float* P, float* loss, void* stream);

/*
 * Gradient of scale * L_b (Eq. 7; the paper adds beta * L_b to the training loss, Sec. 3.4) with respect to
 * the router logits.  f_i only counts selections, so it is held fixed and the gradient flows through P_i:
 *   dlogits[t, j] (+)= (scale / T) P_tj (c_j - sum_i c_i P_ti),  P_t = softmax(logits[t, :]),  c_i = eta_i f_i.
 *   logits [T, N] float (device), f [N] float (device; what moepp_balance_stats wrote)
 *   dlogits [T, N] float (device): overwritten, or added to when accumulate != 0 -- e.g. on top of the dprev
 *   the next layer's moepp_layer_backward produced, before it is passed on as dlogits_next.
 */
moepp_status moepp_balance_backward(const moepp_config* cfg, const float* logits, const float* f, float scale,
                                    int32_t accumulate, float* dlogits, void* stream);

/*
 * A stack of n_layers layers that share one configuration (the gating residual of Eq. 6 carries the
 * logits from layer to layer): layer j reads x^j and the logits of layer j-1 and produces
 * x^{j+1} = (x^j if add_residual) + Eq. 1 and its own logits.  layers[j] holds layer j's weights; a layer
 * whose W_g is NULL ignores the incoming logits (layer 1 of a model, Eq. 6 case j = 1).  prev_logits
 * feeds layers[0] and may be NULL when layers[0].W_g is NULL.  y receives the last layer's output,
 * logits_out (may be NULL) the last layer's logits.  Workspace: moepp_stack_workspace_bytes().
 * The _host variant takes host pointers for x, prev_logits, y and logits_out (pinned memory for
 * asynchronous copies): x goes to the device once, y comes back once, the layers in between stay on
 * the device.  For T >= 4096 (and no capacity limit) the tokens are cut into 2 or 4 chunks (equal ones, or
 * 1/8, 3/8, 3/8, 1/8 when the stack's arithmetic outlasts the copies) that are pipelined: one chunk computes on `stream` while the next is copied in and the previous is copied out
 * on two internal streams; these streams and the events that order them are created and released
 * inside the call (no device memory is allocated), `stream` is made to wait for the last copy, and the
 * results are the same bits as without chunking.  Workspace: moepp_stack_workspace_bytes_host().
 */
moepp_status moepp_stack_workspace_bytes(const moepp_config* cfg, int32_t n_layers, size_t* bytes);
moepp_status moepp_stack_forward(const moepp_config* cfg, const moepp_weights* layers, int32_t n_layers, const void* x,
                                 const float* prev_logits, void* y, float* logits_out, void* workspace,
                                 size_t workspace_bytes, void* stream);
moepp_status moepp_stack_workspace_bytes_host(const moepp_config* cfg, int32_t n_layers, size_t* bytes);
moepp_status moepp_stack_forward_host(const moepp_config* cfg, const moepp_weights* layers, int32_t n_layers,
                                      const void* x_host, const float* prev_logits_host, void* y_host,
                                      float* logits_out_host, void* workspace, size_t workspace_bytes, void* stream);

/*
 * Backward pass of one layer: the chain rule through Eq. 1-6 with the top-K picks held fixed (the
 * selection is piecewise constant).  The paper trains the layer with ordinary back-propagation and
 * prints no formulas for it; these are the derivatives of the forward pass above.
 *
 * Every pointer of moepp_grads is device memory the caller owns; every gradient is OVERWRITTEN
 * (with MOEPP_FLAG_ACCUM_GRADS the weight gradients are added to instead).  Weight gradients are float whatever cfg->dtype is; dx has cfg->dtype.
 */
typedef struct {
  void* dx;       /* [T, D]  dL/dx, cfg->dtype */
  float* dprev;   /* [T, N]  dL/dprev_logits; required when weights->W_g is set, else ignored */
  float* dW_r;    /* [N, D] */
  float* dW_g;    /* [N, N]  may be NULL */
  float* dbias;   /* [N]     may be NULL */
  float* dW_c;    /* [n_const, 2, D]  required when n_const > 0 */
  float* dv;      /* [n_const, D]     required when n_const > 0 */
  float* dW_gate; /* [n_ffn, F, D]    required when n_ffn > 0 */
  float* dW_up;   /* [n_ffn, F, D] */
  float* dW_down; /* [n_ffn, D, F] */
} moepp_grads;

/* Bytes of device scratch moepp_layer_backward needs on top of the forward workspace. */
moepp_status moepp_backward_workspace_bytes(const moepp_config* cfg, size_t* bytes);

/*
 * Device pointers.  `fwd_workspace` is the workspace moepp_layer_forward filled for the SAME cfg, weights,
 * x and prev_logits (it holds the picks, gate weights, row tables, grouped activations and the SwiGLU
 * output); it is read, not written.  `logits` is what that forward call returned in logits_out, or NULL
 * if logits_out was NULL there (the copy in the workspace is used).
 *   dy           [T, D] cfg->dtype   dL/dy
 *   dlogits_next [T, N] float or NULL: dL/dlogits arriving from the next layer's gating residual (Eq. 6)
 * Steps: combine backward (dL/dE_k = w_k dy to the grouped rows, dL/dw_k = <dy, E_k(x)>; Eq. 3 passes
 * nothing, Eq. 4 passes w dy to x, Eq. 5 also feeds dv and the two mixing logits), gate backward (softmax
 * over all N, renormalisation if on), the expert FFNs (SwiGLU pre-activations recomputed from x_perm),
 * the router (dW_r, dW_g, dbias, dprev) and dx.  Slots dropped by Eq. 8 carry no gradient.
 * bf16: the FFN GEMMs run on the tensor cores, operands read in place (the transposed products take their tiles
 * MN-major); a row_align that is a multiple of 64 saves the weight-gradient kernel the clearing of one tile tail
 * per output tile.  Float storage: FMA units.  Float accumulation either way.
 * With MOEPP_FLAG_SAVE_PREACT (set in the forward call too) the pre-activations are read from fwd_workspace
 * instead of being recomputed.
 * MOEPP_FLAG_FUSED_GATHER is refused (that forward path does not keep x_perm).
 * Errors: as moepp_layer_forward; MOEPP_ERR_WORKSPACE when either workspace is too small.
 */
moepp_status moepp_layer_backward(const moepp_config* cfg, const moepp_weights* weights, const void* x,
                                  const float* prev_logits, const float* logits, const void* dy,
                                  const float* dlogits_next, const void* fwd_workspace, size_t fwd_workspace_bytes,
                                  const moepp_grads* grads, void* bwd_workspace, size_t bwd_workspace_bytes,
                                  void* stream);

/*
 * dst[i, :] = src[row_index[i], :] for i < n_rows; a negative index gives a row of zeros.  Rows of row_elems elements
 * of `dtype`, row size a multiple of 16 bytes, device pointers.  The paper has no counterpart: this is the row
 * regrouping an expert-parallel deployment (Sec. 3.4: FFN experts spread over GPUs, zero-computation experts on
 * every GPU) needs between the all-to-all exchange and the grouped FFN, see paper_2410_07348_b200/expert_parallel.py.
 */
moepp_status moepp_gather_rows(const void* src, const int32_t* row_index, int64_t n_rows, int32_t row_elems,
                               int32_t dtype, void* dst, void* stream);

/*
 * The stack of moepp_stack_forward in a form that can be differentiated, and its backward pass: a training
 * step's worth of the layer (the paper trains all layers jointly on the language-model loss plus beta times
 * the sum of the layers' Eq. 7 losses, Sec. 3.4; it prints no backward formulas).
 *
 * moepp_stack_forward_train computes what moepp_stack_forward computes (same kernels, same bits) but gives every
 * layer its own slot in `workspace` (moepp_stack_train_workspace_bytes: n_layers layer workspaces, outputs and
 * logits), so that nothing a backward pass needs is overwritten.
 *
 * moepp_stack_backward walks the layers last to first with moepp_layer_backward's arithmetic: layer j's dx is
 * layer j-1's dy, layer j's dprev is what reaches layer j-1's logits through Eq. 6.
 *   x, prev_logits       the inputs the forward call had
 *   dy [T, D]            dL/d(output of the last layer);  dlogits_last [T, N] or NULL: dL/d(its logits)
 *   balance_scale        beta: if non-zero, beta * dL_b/dlogits (Eq. 7, moepp_balance_backward) of EVERY layer is
 *                        added to that layer's logit gradient; balance_loss_out ([n_layers] float, device, may be
 *                        NULL) then receives each layer's L_b
 *   grads[n_layers]      one gradient set per layer, all weight gradients overwritten; dx and dprev are taken
 *                        from grads[0] only (gradients with respect to x and prev_logits); the others' dx / dprev
 *                        fields are ignored (the call keeps those intermediates in its own scratch)
 *   bwd_workspace        moepp_stack_backward_workspace_bytes
 * All pointers are device memory; nothing is allocated.  Flags as in moepp_layer_forward / moepp_layer_backward
 * (MOEPP_FLAG_SAVE_PREACT must be the same in both calls).
 */
moepp_status moepp_stack_train_workspace_bytes(const moepp_config* cfg, int32_t n_layers, size_t* bytes);
moepp_status moepp_stack_forward_train(const moepp_config* cfg, const moepp_weights* layers, int32_t n_layers,
                                       const void* x, const float* prev_logits, void* y, float* logits_out,
                                       void* workspace, size_t workspace_bytes, void* stream);
moepp_status moepp_stack_backward_workspace_bytes(const moepp_config* cfg, int32_t n_layers, size_t* bytes);
moepp_status moepp_stack_backward(const moepp_config* cfg, const moepp_weights* layers, int32_t n_layers, const void* x,
                                  const float* prev_logits, const void* dy, const float* dlogits_last,
                                  float balance_scale, float* balance_loss_out, const void* train_workspace,
                                  size_t train_workspace_bytes, const moepp_grads* grads, void* bwd_workspace,
                                  size_t bwd_workspace_bytes, void* stream);

/*
 * moepp_grouped_ffn without a scratch argument.  (The paper has no counterpart to this call: it exists
 * for the way this library is embedded, not for the method.)
 *
 * Who needs it: code that is handed input and output buffers and nothing else, and that may not
 * create device memory itself -- for example an operator plugged into a serving runtime whose
 * memory planner owns every byte of the GPU and offers the operator no workspace slot, or a
 * latency-critical loop in which a device allocation (which can stall the whole device) is
 * off limits.  Such a caller cannot supply the [M_cap, F] intermediate that moepp_grouped_ffn wants.
 *
 * Here the intermediate lives in a fixed array of MOEPP_STATIC_SCRATCH_BYTES bytes inside the
 * library's device image.  Consequences a caller must know:
 *   - every GPU that loads the library sets that many bytes aside until the process exits;
 *   - M_cap * F * sizeof(element) must not exceed MOEPP_STATIC_SCRATCH_BYTES; a larger problem is
 *     refused with MOEPP_ERR_WORKSPACE before anything is launched;
 *   - the first call on each device looks up the array's device address (a one-time runtime query,
 *     made with that device current); make that first call outside any stream capture;
 *   - all calls, on all streams, share the one array, and it keeps whatever the previous call left
 *     there.  Nothing in it has to start at zero (every row the second GEMM reads for a live output
 *     row was written by the first GEMM of the same call), so it is not cleared; but two calls that
 *     overlap on the GPU (different streams, or different host threads) race on it.  Serialise them.
 *   - the call itself allocates nothing and frees nothing, like the rest of the library.
 * Arguments, layouts, results and status codes are otherwise those of moepp_grouped_ffn.
 */
#define MOEPP_STATIC_SCRATCH_BYTES (32u << 20)
moepp_status moepp_grouped_ffn_static(const moepp_config* cfg, const void* x_perm, const int32_t* expert_offsets,
                                      const void* W_gate, const void* W_up, const void* W_down,
                                      void* y_perm, /* [M_cap, D] out */
                                      void* stream);

/*
 * Device-side waits in the tensor-core kernels are bounded.  If one ever runs out, the kernel
 * stops early and records a non-zero code; this call copies the code to *code (host pointer),
 * clears it, and synchronises the device while doing so.  0 = no kernel gave up.
 */
moepp_status moepp_device_error(int32_t* code);

#ifdef __cplusplus
}
#endif
#endif /* MOEPP_H */
