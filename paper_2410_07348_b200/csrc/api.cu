// C-ABI layer: argument validation on the host, workspace carving, and the five calls of the layer.
// Nothing here allocates memory or synchronises the stream.
#include <cmath>
#include <cstring>

#include "common.cuh"

using namespace moepp;

namespace {

constexpr size_t kAlign = 256;
inline size_t align_up(size_t v) { return (v + kAlign - 1) / kAlign * kAlign; }
inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// Checks the configuration and fills the internal dimension record.
moepp_status make_dims(const moepp_config* c, Dims* d) {
  if (c == nullptr) return MOEPP_ERR_INVALID_ARG;
  if (c->T < 0 || c->D <= 0 || c->F < 0) return MOEPP_ERR_INVALID_ARG;
  if (c->n_ffn < 0 || c->n_zero < 0 || c->n_copy < 0 || c->n_const < 0) return MOEPP_ERR_INVALID_ARG;
  const long long N = (long long)c->n_ffn + c->n_zero + c->n_copy + c->n_const;
  if (N <= 0) return MOEPP_ERR_INVALID_ARG;
  if (N > kMaxExperts || N + 2 * c->n_const > kMaxRouteRows) return MOEPP_ERR_UNSUPPORTED;
  if (c->top_k < 1 || c->top_k > N) return MOEPP_ERR_INVALID_ARG;
  if (c->top_k > kMaxTopK) return MOEPP_ERR_UNSUPPORTED;
  if (c->dtype != MOEPP_F32 && c->dtype != MOEPP_BF16) return MOEPP_ERR_INVALID_ARG;
  if (c->row_align < 1 || c->row_align > 4096) return MOEPP_ERR_INVALID_ARG;
  if (c->n_ffn > 0 && c->F <= 0) return MOEPP_ERR_INVALID_ARG;
  if (c->D % 8 != 0 || c->F % 8 != 0) return MOEPP_ERR_ALIGN;
  const long long S = (long long)c->T * c->top_k;
  const long long M_cap = S + (long long)c->n_ffn * (c->row_align - 1);
  if (M_cap > 0x7fffffffLL) return MOEPP_ERR_UNSUPPORTED;  // rows and slots are int32
  d->T = c->T; d->D = c->D; d->F = c->F;
  d->n_ffn = c->n_ffn; d->n_zero = c->n_zero; d->n_copy = c->n_copy; d->n_const = c->n_const;
  d->N = (int)N; d->K = c->top_k;
  d->dtype = c->dtype; d->renorm = c->renorm_topk ? 1 : 0; d->row_align = c->row_align;
  d->add_residual = c->add_residual ? 1 : 0; d->flags = c->flags;
  d->M_cap = M_cap;
  d->tau = c->tau > 0.f ? c->tau : 1.f;
  d->cap_on = c->capacity_factor > 0.f ? 1 : 0;
  d->cap_ffn = d->cap_zc = 0x7fffffff;
  if (d->cap_on) {  // Eq. 8 over the T*K routing slots, rounded up
    const double denom = (double)d->tau * c->n_ffn + (double)(c->n_zero + c->n_copy + c->n_const);
    const double cf = ceil((double)c->capacity_factor * d->tau * (double)S / denom);
    const double cz = ceil((double)c->capacity_factor * (double)S / denom);
    d->cap_ffn = cf > 2147483647.0 ? 0x7fffffff : (int)cf;
    d->cap_zc = cz > 2147483647.0 ? 0x7fffffff : (int)cz;
  }
  return MOEPP_OK;
}

inline moepp_status from_cuda(cudaError_t e) { return e == cudaSuccess ? MOEPP_OK : MOEPP_ERR_CUDA; }

// Regions of the layer workspace, in order.  `host_io` adds device staging for x, prev, y.
struct Carve {
  size_t logits, topk_idx, topk_w, counts, offsets, alpha, row_of_slot, slot_of_row, x_perm, h, y_perm;
  size_t gate, up;  // SwiGLU pre-activations, only with MOEPP_FLAG_SAVE_PREACT
  size_t x_dev, prev_dev, y_dev;
  size_t total;
};

Carve carve(const Dims& d, bool host_io) {
  Carve c{};
  size_t off = 0;
  auto take = [&](size_t bytes) {
    const size_t at = off;
    off += align_up(bytes > 0 ? bytes : 1);
    return at;
  };
  const size_t es = elem_size(d.dtype);
  const size_t S = (size_t)d.T * d.K;
  c.logits = take(sizeof(float) * (size_t)d.T * d.N);
  c.topk_idx = take(sizeof(int32_t) * S);
  c.topk_w = take(sizeof(float) * S);
  c.counts = take(sizeof(int32_t) * d.N);
  c.offsets = take(sizeof(int32_t) * (d.n_ffn + 1));
  c.alpha = take(sizeof(float) * (size_t)d.T * d.n_const * 2);
  c.row_of_slot = take(sizeof(int32_t) * S);
  c.slot_of_row = take(sizeof(int32_t) * (size_t)d.M_cap);
  c.x_perm = take(es * (size_t)d.M_cap * d.D);
  c.h = take(es * (size_t)d.M_cap * d.F);
  c.y_perm = take(es * (size_t)d.M_cap * d.D);
  if (d.flags & MOEPP_FLAG_SAVE_PREACT) {
    c.gate = take(es * (size_t)d.M_cap * d.F);
    c.up = take(es * (size_t)d.M_cap * d.F);
  }
  if (host_io) {
    c.x_dev = take(es * (size_t)d.T * d.D);
    c.prev_dev = take(sizeof(float) * (size_t)d.T * d.N);
    c.y_dev = take(es * (size_t)d.T * d.D);
  }
  c.total = off;
  return c;
}

moepp_status ffn_dispatch(const Dims& d, const void* x_perm, const int32_t* offsets, const void* W_gate,
                          const void* W_up, const void* W_down, void* h, void* y_perm, cudaStream_t st,
                          void* gate_out = nullptr, void* up_out = nullptr) {
  if (d.n_ffn == 0 || d.T == 0) return MOEPP_OK;
  if (d.dtype == MOEPP_BF16 && !(d.flags & MOEPP_FLAG_SIMT_FFN)) {
    const cudaError_t e =
        (d.flags & MOEPP_FLAG_FFN_SINGLE_CTA)
            ? launch_ffn_tcgen05(d, x_perm, offsets, W_gate, W_up, W_down, h, y_perm, st)
            : launch_ffn_tcgen05_pair(d, x_perm, offsets, W_gate, W_up, W_down, h, y_perm, st, gate_out, up_out);
    // a shape the TMA tensor maps cannot describe runs on the FMA kernels instead
    if (e != cudaErrorNotSupported) return from_cuda(e);
  }
  return from_cuda(launch_ffn_simt(d, x_perm, offsets, W_gate, W_up, W_down, h, y_perm, st, gate_out, up_out));
}

moepp_status layer_on_device(const Dims& d, const Carve& c, const moepp_weights* w, const void* x,
                             const float* prev, void* y, float* logits_out, char* ws, cudaStream_t st) {
  float* logits = logits_out ? logits_out : reinterpret_cast<float*>(ws + c.logits);
  int32_t* topk_idx = reinterpret_cast<int32_t*>(ws + c.topk_idx);
  float* topk_w = reinterpret_cast<float*>(ws + c.topk_w);
  int32_t* counts = reinterpret_cast<int32_t*>(ws + c.counts);
  int32_t* offsets = reinterpret_cast<int32_t*>(ws + c.offsets);
  float* alpha = d.n_const > 0 ? reinterpret_cast<float*>(ws + c.alpha) : nullptr;
  int32_t* row_of_slot = reinterpret_cast<int32_t*>(ws + c.row_of_slot);
  int32_t* slot_of_row = reinterpret_cast<int32_t*>(ws + c.slot_of_row);
  void* x_perm = ws + c.x_perm;
  void* h = ws + c.h;
  void* y_perm = ws + c.y_perm;

  cudaError_t e = launch_route(d, x, w->W_r, w->W_g, prev, w->router_bias, w->W_c, logits, topk_idx, topk_w, counts,
                               offsets, alpha, st);
  if (e != cudaSuccess) return MOEPP_ERR_CUDA;
  // optional: GEMM 1 gathers its rows from x itself, so the grouped copy of x is never built
  const bool fused_gather = d.dtype == MOEPP_BF16 && (d.flags & MOEPP_FLAG_FUSED_GATHER) && !(d.flags & MOEPP_FLAG_SIMT_FFN);
  e = launch_permute(d, x, topk_idx, offsets, row_of_slot, slot_of_row, fused_gather ? nullptr : x_perm, st);
  if (e != cudaSuccess) return MOEPP_ERR_CUDA;
  if (fused_gather) {
    if (d.n_ffn > 0 && d.T > 0) {
      e = launch_ffn_tcgen05_gather(d, x, slot_of_row, offsets, w->W_gate, w->W_up, w->W_down, h, y_perm, st);
      if (e == cudaErrorNotSupported) return MOEPP_ERR_UNSUPPORTED;
      if (e != cudaSuccess) return MOEPP_ERR_CUDA;
    }
  } else {
    const bool keep = (d.flags & MOEPP_FLAG_SAVE_PREACT) != 0;
    const moepp_status s = ffn_dispatch(d, x_perm, offsets, w->W_gate, w->W_up, w->W_down, h, y_perm, st,
                                        keep ? ws + c.gate : nullptr, keep ? ws + c.up : nullptr);
    if (s != MOEPP_OK) return s;
  }
  e = launch_combine(d, x, y_perm, topk_idx, topk_w, row_of_slot, alpha, w->W_c, w->v, y, st);
  return from_cuda(e);
}

moepp_status check_layer_args(const Dims& d, const moepp_weights* w, const void* x, const float* prev, const void* y,
                              const void* ws) {
  if (w == nullptr || ws == nullptr) return MOEPP_ERR_INVALID_ARG;
  if (d.T > 0 && (x == nullptr || y == nullptr)) return MOEPP_ERR_INVALID_ARG;
  if (d.flags & MOEPP_FLAG_LOGITS_GIVEN) return MOEPP_ERR_INVALID_ARG;  // a whole layer computes its own logits
  if ((d.flags & MOEPP_FLAG_SAVE_PREACT) && (d.flags & (MOEPP_FLAG_FFN_SINGLE_CTA | MOEPP_FLAG_FUSED_GATHER)))
    return MOEPP_ERR_INVALID_ARG;  // only the default and the FMA kernels store the pre-activations
  if (w->W_r == nullptr) return MOEPP_ERR_INVALID_ARG;
  if (d.T > 0 && (w->W_g == nullptr) != (prev == nullptr)) return MOEPP_ERR_INVALID_ARG;
  if (d.n_const > 0 && (w->W_c == nullptr || w->v == nullptr)) return MOEPP_ERR_INVALID_ARG;
  if (d.n_ffn > 0 && (w->W_gate == nullptr || w->W_up == nullptr || w->W_down == nullptr))
    return MOEPP_ERR_INVALID_ARG;
  if (!aligned16(w->W_r) || !aligned16(w->W_c) || !aligned16(w->v) || !aligned16(w->W_gate) ||
      !aligned16(w->W_up) || !aligned16(w->W_down))
    return MOEPP_ERR_ALIGN;
  if ((reinterpret_cast<uintptr_t>(ws) & (kAlign - 1)) != 0) return MOEPP_ERR_ALIGN;
  return MOEPP_OK;
}

}  // namespace

extern "C" {

const char* moepp_status_string(moepp_status s) {
  switch (s) {
    case MOEPP_OK: return "ok";
    case MOEPP_ERR_INVALID_ARG: return "invalid argument";
    case MOEPP_ERR_UNSUPPORTED: return "unsupported configuration";
    case MOEPP_ERR_ALIGN: return "pointer or dimension not aligned";
    case MOEPP_ERR_WORKSPACE: return "workspace too small";
    case MOEPP_ERR_CUDA: return "CUDA error at launch";
    case MOEPP_ERR_TIMEOUT: return "a device-side wait ran out";
  }
  return "unknown status";
}

moepp_status moepp_workspace_bytes(const moepp_config* cfg, size_t* bytes) {
  Dims d;
  const moepp_status s = make_dims(cfg, &d);
  if (s != MOEPP_OK) return s;
  if (bytes == nullptr) return MOEPP_ERR_INVALID_ARG;
  *bytes = carve(d, false).total;
  return MOEPP_OK;
}

moepp_status moepp_workspace_bytes_host(const moepp_config* cfg, size_t* bytes) {
  Dims d;
  const moepp_status s = make_dims(cfg, &d);
  if (s != MOEPP_OK) return s;
  if (bytes == nullptr) return MOEPP_ERR_INVALID_ARG;
  *bytes = carve(d, true).total;
  return MOEPP_OK;
}

moepp_status moepp_route(const moepp_config* cfg, const void* x, const float* W_r, const float* W_g,
                         const float* prev_logits, const float* router_bias, const float* W_c, float* logits,
                         int32_t* topk_idx, float* topk_w, int32_t* expert_counts, int32_t* expert_offsets,
                         float* alpha, void* stream) {
  Dims d;
  const moepp_status s = make_dims(cfg, &d);
  if (s != MOEPP_OK) return s;
  if (expert_counts == nullptr || expert_offsets == nullptr) return MOEPP_ERR_INVALID_ARG;
  if (d.T > 0 && (logits == nullptr || topk_idx == nullptr || topk_w == nullptr)) return MOEPP_ERR_INVALID_ARG;
  const bool given = (d.flags & MOEPP_FLAG_LOGITS_GIVEN) != 0;
  if (given) {
    W_r = nullptr; W_g = nullptr; prev_logits = nullptr; router_bias = nullptr;
  } else {
    if (W_r == nullptr) return MOEPP_ERR_INVALID_ARG;
    if (d.T > 0 && (W_g == nullptr) != (prev_logits == nullptr)) return MOEPP_ERR_INVALID_ARG;
  }
  if (d.n_const == 0) alpha = nullptr;
  if (alpha != nullptr && W_c == nullptr) return MOEPP_ERR_INVALID_ARG;
  const bool needs_x = !given || alpha != nullptr;
  if (needs_x && d.T > 0 && x == nullptr) return MOEPP_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(W_r) || !aligned16(W_c)) return MOEPP_ERR_ALIGN;
  return from_cuda(launch_route(d, x, W_r, W_g, prev_logits, router_bias, W_c, logits, topk_idx, topk_w,
                                expert_counts, expert_offsets, alpha, static_cast<cudaStream_t>(stream)));
}

moepp_status moepp_permute(const moepp_config* cfg, const void* x, const int32_t* topk_idx,
                           const int32_t* expert_offsets, int32_t* row_of_slot, int32_t* slot_of_row, void* x_perm,
                           void* stream) {
  Dims d;
  const moepp_status s = make_dims(cfg, &d);
  if (s != MOEPP_OK) return s;
  if (expert_offsets == nullptr) return MOEPP_ERR_INVALID_ARG;
  if (d.T > 0 && (x == nullptr || topk_idx == nullptr || row_of_slot == nullptr)) return MOEPP_ERR_INVALID_ARG;
  if (d.M_cap > 0 && (slot_of_row == nullptr || x_perm == nullptr)) return MOEPP_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(x_perm) || !aligned16(topk_idx)) return MOEPP_ERR_ALIGN;
  return from_cuda(launch_permute(d, x, topk_idx, expert_offsets, row_of_slot, slot_of_row, x_perm,
                                  static_cast<cudaStream_t>(stream)));
}

moepp_status moepp_gather_rows(const void* src, const int32_t* row_index, int64_t n_rows, int32_t row_elems,
                               int32_t dtype, void* dst, void* stream) {
  if (n_rows < 0 || row_elems <= 0 || (dtype != MOEPP_F32 && dtype != MOEPP_BF16)) return MOEPP_ERR_INVALID_ARG;
  const size_t row_bytes = (size_t)row_elems * elem_size(dtype);
  if (row_bytes % 16 != 0) return MOEPP_ERR_ALIGN;
  if (n_rows > 0 && (src == nullptr || row_index == nullptr || dst == nullptr)) return MOEPP_ERR_INVALID_ARG;
  if (!aligned16(src) || !aligned16(dst)) return MOEPP_ERR_ALIGN;
  return from_cuda(launch_gather_rows(src, row_index, n_rows, row_bytes, dst, static_cast<cudaStream_t>(stream)));
}

moepp_status moepp_grouped_ffn(const moepp_config* cfg, const void* x_perm, const int32_t* expert_offsets,
                               const void* W_gate, const void* W_up, const void* W_down, void* h_ws, void* y_perm,
                               void* stream) {
  Dims d;
  const moepp_status s = make_dims(cfg, &d);
  if (s != MOEPP_OK) return s;
  if (expert_offsets == nullptr) return MOEPP_ERR_INVALID_ARG;
  if (d.T > 0 && d.n_ffn > 0 && (x_perm == nullptr || h_ws == nullptr || y_perm == nullptr))
    return MOEPP_ERR_INVALID_ARG;
  if (d.n_ffn > 0 && (W_gate == nullptr || W_up == nullptr || W_down == nullptr)) return MOEPP_ERR_INVALID_ARG;
  if (!aligned16(x_perm) || !aligned16(W_gate) || !aligned16(W_up) || !aligned16(W_down) || !aligned16(h_ws) ||
      !aligned16(y_perm))
    return MOEPP_ERR_ALIGN;
  return ffn_dispatch(d, x_perm, expert_offsets, W_gate, W_up, W_down, h_ws, y_perm,
                      static_cast<cudaStream_t>(stream));
}

moepp_status moepp_combine(const moepp_config* cfg, const void* x, const void* y_perm, const int32_t* topk_idx,
                           const float* topk_w, const int32_t* row_of_slot, const float* alpha, const float* W_c,
                           const float* v, void* y, void* stream) {
  Dims d;
  const moepp_status s = make_dims(cfg, &d);
  if (s != MOEPP_OK) return s;
  if (d.T > 0 && (x == nullptr || topk_idx == nullptr || topk_w == nullptr || row_of_slot == nullptr || y == nullptr))
    return MOEPP_ERR_INVALID_ARG;
  if (d.T > 0 && d.n_ffn > 0 && y_perm == nullptr) return MOEPP_ERR_INVALID_ARG;
  if (d.n_const > 0 && (v == nullptr || (alpha == nullptr && W_c == nullptr))) return MOEPP_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(y_perm) || !aligned16(y) || !aligned16(v) || !aligned16(W_c))
    return MOEPP_ERR_ALIGN;
  return from_cuda(launch_combine(d, x, y_perm, topk_idx, topk_w, row_of_slot, alpha, W_c, v, y,
                                  static_cast<cudaStream_t>(stream)));
}

moepp_status moepp_layer_forward(const moepp_config* cfg, const moepp_weights* weights, const void* x,
                                 const float* prev_logits, void* y, float* logits_out, void* workspace,
                                 size_t workspace_bytes, void* stream) {
  Dims d;
  moepp_status s = make_dims(cfg, &d);
  if (s != MOEPP_OK) return s;
  s = check_layer_args(d, weights, x, prev_logits, y, workspace);
  if (s != MOEPP_OK) return s;
  if (!aligned16(x) || !aligned16(y)) return MOEPP_ERR_ALIGN;
  const Carve c = carve(d, false);
  if (workspace_bytes < c.total) return MOEPP_ERR_WORKSPACE;
  return layer_on_device(d, c, weights, x, prev_logits, y, logits_out, static_cast<char*>(workspace),
                         static_cast<cudaStream_t>(stream));
}

moepp_status moepp_layer_forward_host(const moepp_config* cfg, const moepp_weights* weights, const void* x_host,
                                      const float* prev_logits_host, void* y_host, float* logits_out_host,
                                      void* workspace, size_t workspace_bytes, void* stream) {
  Dims d;
  moepp_status s = make_dims(cfg, &d);
  if (s != MOEPP_OK) return s;
  s = check_layer_args(d, weights, x_host, prev_logits_host, y_host, workspace);
  if (s != MOEPP_OK) return s;
  const Carve c = carve(d, true);
  if (workspace_bytes < c.total) return MOEPP_ERR_WORKSPACE;
  if (d.T == 0) return MOEPP_OK;
  char* ws = static_cast<char*>(workspace);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t es = elem_size(d.dtype);
  const size_t act_bytes = es * (size_t)d.T * d.D, lg_bytes = sizeof(float) * (size_t)d.T * d.N;
  if (cudaMemcpyAsync(ws + c.x_dev, x_host, act_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess)
    return MOEPP_ERR_CUDA;
  const float* prev_dev = nullptr;
  if (prev_logits_host != nullptr) {
    if (cudaMemcpyAsync(ws + c.prev_dev, prev_logits_host, lg_bytes, cudaMemcpyHostToDevice, st) != cudaSuccess)
      return MOEPP_ERR_CUDA;
    prev_dev = reinterpret_cast<const float*>(ws + c.prev_dev);
  }
  s = layer_on_device(d, c, weights, ws + c.x_dev, prev_dev, ws + c.y_dev, nullptr, ws, st);
  if (s != MOEPP_OK) return s;
  if (cudaMemcpyAsync(y_host, ws + c.y_dev, act_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return MOEPP_ERR_CUDA;
  if (logits_out_host != nullptr &&
      cudaMemcpyAsync(logits_out_host, ws + c.logits, lg_bytes, cudaMemcpyDeviceToHost, st) != cudaSuccess)
    return MOEPP_ERR_CUDA;
  return MOEPP_OK;
}

// Workspace of a stack: one layer workspace, two activation buffers and two logits buffers to ping-pong
// between layers (plus, for host I/O, nothing more: the first activation buffer receives x).
static size_t stack_extra_bytes(const Dims& d, size_t* act, size_t* lg) {
  *act = align_up(elem_size(d.dtype) * (size_t)d.T * d.D + 1);
  *lg = align_up(sizeof(float) * (size_t)d.T * d.N + 1);
  return 2 * (*act) + 2 * (*lg);
}

moepp_status moepp_stack_workspace_bytes(const moepp_config* cfg, int32_t n_layers, size_t* bytes) {
  Dims d;
  const moepp_status s = make_dims(cfg, &d);
  if (s != MOEPP_OK) return s;
  if (bytes == nullptr || n_layers < 1) return MOEPP_ERR_INVALID_ARG;
  size_t act, lg;
  *bytes = carve(d, false).total + stack_extra_bytes(d, &act, &lg);
  return MOEPP_OK;
}

static moepp_status stack_on_device(const Dims& d, const moepp_weights* layers, int32_t n_layers, const void* x,
                                    const float* prev_logits, void* y, float* logits_out, char* ws, cudaStream_t st) {
  const Carve c = carve(d, false);
  size_t act, lg;
  stack_extra_bytes(d, &act, &lg);
  char* extra = ws + c.total;
  void* xbuf[2] = {extra, extra + act};
  float* lbuf[2] = {reinterpret_cast<float*>(extra + 2 * act), reinterpret_cast<float*>(extra + 2 * act + lg)};
  const void* cur_x = x;
  const float* cur_prev = prev_logits;
  for (int j = 0; j < n_layers; ++j) {
    const bool last = (j == n_layers - 1);
    void* out_y = last ? y : xbuf[j & 1];
    float* out_l = (last && logits_out != nullptr) ? logits_out : lbuf[j & 1];
    const moepp_weights* w = &layers[j];
    const float* prev = (w->W_g != nullptr) ? cur_prev : nullptr;
    const moepp_status s = check_layer_args(d, w, cur_x, prev, out_y, ws);
    if (s != MOEPP_OK) return s;
    const moepp_status r = layer_on_device(d, c, w, cur_x, prev, out_y, out_l, ws, st);
    if (r != MOEPP_OK) return r;
    cur_x = out_y;
    cur_prev = out_l;
  }
  return MOEPP_OK;
}

moepp_status moepp_stack_forward(const moepp_config* cfg, const moepp_weights* layers, int32_t n_layers, const void* x,
                                 const float* prev_logits, void* y, float* logits_out, void* workspace,
                                 size_t workspace_bytes, void* stream) {
  Dims d;
  const moepp_status s = make_dims(cfg, &d);
  if (s != MOEPP_OK) return s;
  if (layers == nullptr || n_layers < 1 || workspace == nullptr) return MOEPP_ERR_INVALID_ARG;
  if (d.T > 0 && (x == nullptr || y == nullptr)) return MOEPP_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(y)) return MOEPP_ERR_ALIGN;
  if ((reinterpret_cast<uintptr_t>(workspace) & (kAlign - 1)) != 0) return MOEPP_ERR_ALIGN;
  size_t act, lg;
  if (workspace_bytes < carve(d, false).total + stack_extra_bytes(d, &act, &lg)) return MOEPP_ERR_WORKSPACE;
  if (d.T > 0 && layers[0].W_g != nullptr && prev_logits == nullptr) return MOEPP_ERR_INVALID_ARG;
  return stack_on_device(d, layers, n_layers, x, prev_logits, y, logits_out, static_cast<char*>(workspace),
                         static_cast<cudaStream_t>(stream));
}

// ---- stack with host activations: token chunks pipelined over copy-in, compute and copy-out ----------------
// Tokens are independent through a stack (no capacity limit), so the batch is cut into chunks: while one chunk
// computes on the caller's stream, the next one is copied in and the previous one copied out on two internal
// streams.  Every chunk owns its own slice of the workspace.
namespace {

struct HostChunks {
  int n;           // number of chunks
  int begin[4];    // first token of each chunk
  int tokens[4];   // tokens of each chunk (multiples of 128; the last chunk takes the rest)
};

// Large batches are cut into 4 chunks (2 from 4096 tokens on).  Where the stack's arithmetic outlasts the copies
// (about n_layers * F * K >= 16384 at PCIe 5 and bf16 tensor speed) the cut is 1/8, 3/8, 3/8, 1/8: a short copy-in
// before compute starts, a short copy-out tail, and middle chunks whose GEMMs run at nearly the full batch's
// efficiency.  Otherwise the copies are the bound and equal chunks keep both copy directions busy longest.
HostChunks host_chunks(const Dims& d, int n_layers) {
  HostChunks h{};
  h.n = 1; h.begin[0] = 0; h.tokens[0] = d.T;
  if (d.cap_on || d.T < 4096) return h;  // Eq. 8 shares one capacity among all tokens: keep the batch whole
  auto up128 = [](long long v) { return (int)((v + 127) / 128 * 128); };
  const bool compute_bound = (long long)n_layers * d.F * d.K >= 16384;
  int want[4], n;
  if (d.T >= 16384) {
    n = 4;
    if (compute_bound) {
      want[0] = up128(d.T / 8); want[1] = up128(3LL * d.T / 8); want[2] = want[1];
    } else {
      want[0] = want[1] = want[2] = up128((d.T + 3) / 4);
    }
    want[3] = d.T;
  } else {
    n = 2;
    want[0] = up128(d.T / 2); want[1] = d.T;
  }
  int at = 0;
  h.n = 0;
  for (int i = 0; i < n && at < d.T; ++i) {
    const int tok = (i + 1 < n && at + want[i] < d.T) ? want[i] : d.T - at;
    h.begin[h.n] = at; h.tokens[h.n] = tok;
    at += tok;
    ++h.n;
  }
  return h;
}

// A chunk holds a fraction of every expert's rows, so the 256-row tiles of the CTA-pair kernels would be padded
// more heavily: chunks run the 128-row single-CTA kernels (the same arithmetic per element, the same bits).
Dims chunk_dims(const Dims& d, int tokens, bool chunked) {
  Dims c = d;
  c.T = tokens;
  c.M_cap = (long long)tokens * d.K + (long long)d.n_ffn * (d.row_align - 1);
  if (chunked && !(d.flags & (MOEPP_FLAG_SAVE_PREACT | MOEPP_FLAG_FUSED_GATHER))) c.flags |= MOEPP_FLAG_FFN_SINGLE_CTA;
  return c;
}

// workspace of one chunk: layer workspace + ping-pong buffers + staging of x, y, prev, last logits
size_t chunk_ws_bytes(const Dims& c) {
  size_t act, lg;
  const size_t extra = stack_extra_bytes(c, &act, &lg);
  return carve(c, false).total + extra + 2 * act + 2 * lg;
}

}  // namespace

moepp_status moepp_stack_workspace_bytes_host(const moepp_config* cfg, int32_t n_layers, size_t* bytes) {
  Dims d;
  const moepp_status s = make_dims(cfg, &d);
  if (s != MOEPP_OK) return s;
  if (bytes == nullptr || n_layers < 1) return MOEPP_ERR_INVALID_ARG;
  const HostChunks h = host_chunks(d, n_layers);
  size_t total = 0;
  for (int i = 0; i < h.n; ++i) total += chunk_ws_bytes(chunk_dims(d, h.tokens[i], h.n > 1));
  *bytes = total;
  return MOEPP_OK;
}

moepp_status moepp_stack_forward_host(const moepp_config* cfg, const moepp_weights* layers, int32_t n_layers,
                                      const void* x_host, const float* prev_logits_host, void* y_host,
                                      float* logits_out_host, void* workspace, size_t workspace_bytes, void* stream) {
  Dims d;
  const moepp_status s = make_dims(cfg, &d);
  if (s != MOEPP_OK) return s;
  if (layers == nullptr || n_layers < 1 || workspace == nullptr) return MOEPP_ERR_INVALID_ARG;
  if (d.T > 0 && (x_host == nullptr || y_host == nullptr)) return MOEPP_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(workspace) & (kAlign - 1)) != 0) return MOEPP_ERR_ALIGN;
  size_t need = 0;
  {
    const moepp_status w = moepp_stack_workspace_bytes_host(cfg, n_layers, &need);
    if (w != MOEPP_OK) return w;
  }
  if (workspace_bytes < need) return MOEPP_ERR_WORKSPACE;
  if (d.T > 0 && layers[0].W_g != nullptr && prev_logits_host == nullptr) return MOEPP_ERR_INVALID_ARG;
  if (d.T == 0) return MOEPP_OK;

  const HostChunks h = host_chunks(d, n_layers);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const size_t es = elem_size(d.dtype);
  constexpr int kMaxChunks = 8;
  cudaStream_t s_in = nullptr, s_out = nullptr;
  cudaEvent_t ev_start = nullptr, ev_out = nullptr, ev_in[kMaxChunks] = {}, ev_done[kMaxChunks] = {};
  const bool piped = h.n > 1;
  moepp_status result = MOEPP_OK;
  auto fail = [&](moepp_status code) { if (result == MOEPP_OK) result = code; };

  if (piped) {  // two internal streams and a handful of events, created and released inside this call
    bool ok = cudaStreamCreateWithFlags(&s_in, cudaStreamNonBlocking) == cudaSuccess &&
              cudaStreamCreateWithFlags(&s_out, cudaStreamNonBlocking) == cudaSuccess &&
              cudaEventCreateWithFlags(&ev_start, cudaEventDisableTiming) == cudaSuccess &&
              cudaEventCreateWithFlags(&ev_out, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; ok && i < h.n; ++i)
      ok = cudaEventCreateWithFlags(&ev_in[i], cudaEventDisableTiming) == cudaSuccess &&
           cudaEventCreateWithFlags(&ev_done[i], cudaEventDisableTiming) == cudaSuccess;
    if (!ok) fail(MOEPP_ERR_CUDA);
    // the internal streams start after whatever the caller queued before this call
    if (result == MOEPP_OK && (cudaEventRecord(ev_start, st) != cudaSuccess ||
                               cudaStreamWaitEvent(s_in, ev_start, 0) != cudaSuccess ||
                               cudaStreamWaitEvent(s_out, ev_start, 0) != cudaSuccess))
      fail(MOEPP_ERR_CUDA);
  }

  char* ws = static_cast<char*>(workspace);
  for (int i = 0; i < h.n && result == MOEPP_OK; ++i) {
    const int t_begin = h.begin[i], tok = h.tokens[i];
    const Dims c = chunk_dims(d, tok, h.n > 1);
    size_t act, lg;
    const size_t extra = stack_extra_bytes(c, &act, &lg);
    const size_t base = carve(c, false).total + extra;
    char* x_dev = ws + base;
    char* y_dev = x_dev + act;
    float* p_dev = reinterpret_cast<float*>(y_dev + act);
    float* l_dev = reinterpret_cast<float*>(y_dev + act + lg);
    const size_t act_bytes = es * (size_t)tok * d.D, lg_bytes = sizeof(float) * (size_t)tok * d.N;
    const char* xh = static_cast<const char*>(x_host) + es * (size_t)t_begin * d.D;
    char* yh = static_cast<char*>(y_host) + es * (size_t)t_begin * d.D;
    cudaStream_t cin = piped ? s_in : st, cout = piped ? s_out : st;

    if (cudaMemcpyAsync(x_dev, xh, act_bytes, cudaMemcpyHostToDevice, cin) != cudaSuccess) { fail(MOEPP_ERR_CUDA); break; }
    const float* prev = nullptr;
    if (prev_logits_host != nullptr) {
      if (cudaMemcpyAsync(p_dev, prev_logits_host + (size_t)t_begin * d.N, lg_bytes, cudaMemcpyHostToDevice, cin) !=
          cudaSuccess) { fail(MOEPP_ERR_CUDA); break; }
      prev = p_dev;
    }
    if (piped && (cudaEventRecord(ev_in[i], s_in) != cudaSuccess || cudaStreamWaitEvent(st, ev_in[i], 0) != cudaSuccess)) {
      fail(MOEPP_ERR_CUDA); break;
    }
    const moepp_status r = stack_on_device(c, layers, n_layers, x_dev, prev, y_dev, l_dev, ws, st);
    if (r != MOEPP_OK) { fail(r); break; }
    if (piped && (cudaEventRecord(ev_done[i], st) != cudaSuccess ||
                  cudaStreamWaitEvent(s_out, ev_done[i], 0) != cudaSuccess)) { fail(MOEPP_ERR_CUDA); break; }
    if (cudaMemcpyAsync(yh, y_dev, act_bytes, cudaMemcpyDeviceToHost, cout) != cudaSuccess) { fail(MOEPP_ERR_CUDA); break; }
    if (logits_out_host != nullptr &&
        cudaMemcpyAsync(logits_out_host + (size_t)t_begin * d.N, l_dev, lg_bytes, cudaMemcpyDeviceToHost, cout) !=
            cudaSuccess) { fail(MOEPP_ERR_CUDA); break; }
    ws += chunk_ws_bytes(c);
  }

  if (piped) {
    // the caller's stream ends after the last copy out; then the internal objects go (the runtime frees them
    // once the work queued on them has finished)
    if (s_out != nullptr && ev_out != nullptr) {
      if (cudaEventRecord(ev_out, s_out) != cudaSuccess || cudaStreamWaitEvent(st, ev_out, 0) != cudaSuccess)
        fail(MOEPP_ERR_CUDA);
    }
    for (int i = 0; i < h.n; ++i) {
      if (ev_in[i]) cudaEventDestroy(ev_in[i]);
      if (ev_done[i]) cudaEventDestroy(ev_done[i]);
    }
    if (ev_start) cudaEventDestroy(ev_start);
    if (ev_out) cudaEventDestroy(ev_out);
    if (s_in) cudaStreamDestroy(s_in);
    if (s_out) cudaStreamDestroy(s_out);
  }
  return result;
}

moepp_status moepp_balance_stats(const moepp_config* cfg, const float* logits, const int32_t* expert_counts, float* f,
                                 float* P, float* loss, void* stream) {
  Dims d;
  const moepp_status s = make_dims(cfg, &d);
  if (s != MOEPP_OK) return s;
  if (expert_counts == nullptr || f == nullptr || P == nullptr || loss == nullptr) return MOEPP_ERR_INVALID_ARG;
  if (d.T > 0 && logits == nullptr) return MOEPP_ERR_INVALID_ARG;
  return from_cuda(launch_balance_stats(d, logits, expert_counts, f, P, loss, static_cast<cudaStream_t>(stream)));
}

moepp_status moepp_balance_backward(const moepp_config* cfg, const float* logits, const float* f, float scale,
                                    int32_t accumulate, float* dlogits, void* stream) {
  Dims d;
  const moepp_status s = make_dims(cfg, &d);
  if (s != MOEPP_OK) return s;
  if (f == nullptr) return MOEPP_ERR_INVALID_ARG;
  if (d.T > 0 && (logits == nullptr || dlogits == nullptr)) return MOEPP_ERR_INVALID_ARG;
  return from_cuda(launch_balance_backward(d, logits, f, scale, accumulate != 0, dlogits,
                                           static_cast<cudaStream_t>(stream)));
}

// Device scratch of the backward pass, carved like the forward workspace.
struct BwdCarve {
  size_t dYp, gate, up, dXp, dw, dGz, cx, cvq, part, split, segs, total;
};

static BwdCarve carve_backward(const Dims& d) {
  BwdCarve c{};
  size_t off = 0;
  auto take = [&](size_t bytes) {
    const size_t at = off;
    off += align_up(bytes > 0 ? bytes : 1);
    return at;
  };
  const size_t es = elem_size(d.dtype);
  const size_t R = (size_t)d.N + 2 * (size_t)d.n_const;
  c.dYp = take(es * (size_t)d.M_cap * d.D);
  c.gate = take(es * (size_t)d.M_cap * d.F);
  c.up = take(es * (size_t)d.M_cap * d.F);
  c.dXp = take(es * (size_t)d.M_cap * d.D);
  c.dw = take(sizeof(float) * (size_t)d.T * d.K);
  c.dGz = take(sizeof(float) * (size_t)d.T * R);
  c.cx = take(sizeof(float) * (size_t)d.T);
  c.cvq = take(sizeof(float) * (size_t)d.T * d.n_const);
  c.part = take(sizeof(float) * backward_part_floats(d));
  c.split = take(2 * (size_t)d.T * 128);
  c.segs = take(sizeof(int32_t) * (kMaxExperts + 1));
  c.total = off;
  return c;
}

moepp_status moepp_backward_workspace_bytes(const moepp_config* cfg, size_t* bytes) {
  Dims d;
  const moepp_status s = make_dims(cfg, &d);
  if (s != MOEPP_OK) return s;
  if (bytes == nullptr) return MOEPP_ERR_INVALID_ARG;
  *bytes = carve_backward(d).total;
  return MOEPP_OK;
}

// One layer's backward pass on validated dimensions: argument checks for the gradient set, then the launches.
static moepp_status layer_backward_on_device(const Dims& d, const moepp_weights* weights, const void* x,
                                             const float* prev_logits, const float* logits, const void* dy,
                                             const float* dlogits_next, const char* fw, const moepp_grads& g, char* bw,
                                             cudaStream_t st) {
  const moepp_status s = check_layer_args(d, weights, x, prev_logits, dy, fw);
  if (s != MOEPP_OK) return s;
  if (g.dW_r == nullptr || (d.T > 0 && g.dx == nullptr)) return MOEPP_ERR_INVALID_ARG;
  if (d.T > 0 && weights->W_g != nullptr && g.dprev == nullptr) return MOEPP_ERR_INVALID_ARG;
  if (d.n_const > 0 && (g.dW_c == nullptr || g.dv == nullptr)) return MOEPP_ERR_INVALID_ARG;
  if (d.n_ffn > 0 && (g.dW_gate == nullptr || g.dW_up == nullptr || g.dW_down == nullptr))
    return MOEPP_ERR_INVALID_ARG;
  if (!aligned16(dy) || !aligned16(g.dx) || !aligned16(x)) return MOEPP_ERR_ALIGN;
  const Carve c = carve(d, false);
  const BwdCarve bc = carve_backward(d);
  ForwardState fs{};
  fs.logits = logits != nullptr ? logits : reinterpret_cast<const float*>(fw + c.logits);
  fs.topk_idx = reinterpret_cast<const int32_t*>(fw + c.topk_idx);
  fs.topk_w = reinterpret_cast<const float*>(fw + c.topk_w);
  fs.offsets = reinterpret_cast<const int32_t*>(fw + c.offsets);
  fs.alpha = reinterpret_cast<const float*>(fw + c.alpha);
  fs.row_of_slot = reinterpret_cast<const int32_t*>(fw + c.row_of_slot);
  fs.slot_of_row = reinterpret_cast<const int32_t*>(fw + c.slot_of_row);
  fs.x_perm = fw + c.x_perm;
  fs.h = fw + c.h;
  fs.y_perm = fw + c.y_perm;
  const bool kept = (d.flags & MOEPP_FLAG_SAVE_PREACT) != 0;
  fs.gate = kept ? fw + c.gate : nullptr;
  fs.up = kept ? fw + c.up : nullptr;
  BackwardScratch b{};
  b.dYp = bw + bc.dYp; b.gate = bw + bc.gate; b.up = bw + bc.up; b.dXp = bw + bc.dXp;
  b.dw = reinterpret_cast<float*>(bw + bc.dw);
  b.dGz = reinterpret_cast<float*>(bw + bc.dGz);
  b.cx = reinterpret_cast<float*>(bw + bc.cx);
  b.cvq = reinterpret_cast<float*>(bw + bc.cvq);
  b.part = reinterpret_cast<float*>(bw + bc.part);
  b.split = bw + bc.split;
  b.segs = reinterpret_cast<int32_t*>(bw + bc.segs);
  return from_cuda(launch_layer_backward(d, fs, *weights, x, prev_logits, dy, dlogits_next, b, g, st));
}

moepp_status moepp_layer_backward(const moepp_config* cfg, const moepp_weights* weights, const void* x,
                                  const float* prev_logits, const float* logits, const void* dy,
                                  const float* dlogits_next, const void* fwd_workspace, size_t fwd_workspace_bytes,
                                  const moepp_grads* grads, void* bwd_workspace, size_t bwd_workspace_bytes,
                                  void* stream) {
  Dims d;
  const moepp_status s = make_dims(cfg, &d);
  if (s != MOEPP_OK) return s;
  if (grads == nullptr || bwd_workspace == nullptr) return MOEPP_ERR_INVALID_ARG;
  if (d.flags & MOEPP_FLAG_FUSED_GATHER) return MOEPP_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(bwd_workspace) & (kAlign - 1)) != 0) return MOEPP_ERR_ALIGN;
  if (fwd_workspace_bytes < carve(d, false).total || bwd_workspace_bytes < carve_backward(d).total)
    return MOEPP_ERR_WORKSPACE;
  return layer_backward_on_device(d, weights, x, prev_logits, logits, dy, dlogits_next,
                                  static_cast<const char*>(fwd_workspace), *grads, static_cast<char*>(bwd_workspace),
                                  static_cast<cudaStream_t>(stream));
}

// ---- a stack that can be differentiated: every layer keeps its own workspace, output and logits ------------
// slot j = [layer workspace | y of layer j | logits of layer j]
static size_t train_slot_bytes(const Dims& d, size_t* act, size_t* lg) {
  stack_extra_bytes(d, act, lg);
  return carve(d, false).total + *act + *lg;
}

moepp_status moepp_stack_train_workspace_bytes(const moepp_config* cfg, int32_t n_layers, size_t* bytes) {
  Dims d;
  const moepp_status s = make_dims(cfg, &d);
  if (s != MOEPP_OK) return s;
  if (bytes == nullptr || n_layers < 1) return MOEPP_ERR_INVALID_ARG;
  size_t act, lg;
  *bytes = (size_t)n_layers * train_slot_bytes(d, &act, &lg);
  return MOEPP_OK;
}

moepp_status moepp_stack_forward_train(const moepp_config* cfg, const moepp_weights* layers, int32_t n_layers,
                                       const void* x, const float* prev_logits, void* y, float* logits_out,
                                       void* workspace, size_t workspace_bytes, void* stream) {
  Dims d;
  const moepp_status s = make_dims(cfg, &d);
  if (s != MOEPP_OK) return s;
  if (layers == nullptr || n_layers < 1 || workspace == nullptr) return MOEPP_ERR_INVALID_ARG;
  if (d.T > 0 && (x == nullptr || y == nullptr)) return MOEPP_ERR_INVALID_ARG;
  if (d.flags & MOEPP_FLAG_FUSED_GATHER) return MOEPP_ERR_INVALID_ARG;
  if (!aligned16(x) || !aligned16(y)) return MOEPP_ERR_ALIGN;
  if ((reinterpret_cast<uintptr_t>(workspace) & (kAlign - 1)) != 0) return MOEPP_ERR_ALIGN;
  size_t act, lg;
  const size_t slot = train_slot_bytes(d, &act, &lg);
  if (workspace_bytes < (size_t)n_layers * slot) return MOEPP_ERR_WORKSPACE;
  if (d.T > 0 && layers[0].W_g != nullptr && prev_logits == nullptr) return MOEPP_ERR_INVALID_ARG;
  const Carve c = carve(d, false);
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  char* ws = static_cast<char*>(workspace);
  const void* cur_x = x;
  const float* cur_prev = prev_logits;
  for (int j = 0; j < n_layers; ++j) {
    char* sl = ws + (size_t)j * slot;
    const bool last = (j == n_layers - 1);
    void* out_y = last ? y : static_cast<void*>(sl + c.total);
    float* out_l = reinterpret_cast<float*>(sl + c.total + act);
    const moepp_weights* w = &layers[j];
    const float* prev = (w->W_g != nullptr) ? cur_prev : nullptr;
    moepp_status r = check_layer_args(d, w, cur_x, prev, out_y, sl);
    if (r != MOEPP_OK) return r;
    r = layer_on_device(d, c, w, cur_x, prev, out_y, out_l, sl, st);
    if (r != MOEPP_OK) return r;
    cur_x = out_y;
    cur_prev = out_l;
  }
  if (logits_out != nullptr && d.T > 0 &&
      cudaMemcpyAsync(logits_out, cur_prev, sizeof(float) * (size_t)d.T * d.N, cudaMemcpyDeviceToDevice, st) !=
          cudaSuccess)
    return MOEPP_ERR_CUDA;
  return MOEPP_OK;
}

// backward scratch of a stack: one layer's scratch, two dx and two dlogits buffers to ping-pong between layers,
// and the Eq. 7 statistics of the layer in hand (f, P, loss)
static size_t stack_backward_bytes(const Dims& d, size_t* act, size_t* lg, size_t* stats) {
  stack_extra_bytes(d, act, lg);
  *stats = align_up(sizeof(float) * (2 * (size_t)d.N + 1));
  return carve_backward(d).total + 2 * (*act) + 2 * (*lg) + *stats;
}

moepp_status moepp_stack_backward_workspace_bytes(const moepp_config* cfg, int32_t n_layers, size_t* bytes) {
  Dims d;
  const moepp_status s = make_dims(cfg, &d);
  if (s != MOEPP_OK) return s;
  if (bytes == nullptr || n_layers < 1) return MOEPP_ERR_INVALID_ARG;
  size_t act, lg, stats;
  *bytes = stack_backward_bytes(d, &act, &lg, &stats);
  return MOEPP_OK;
}

moepp_status moepp_stack_backward(const moepp_config* cfg, const moepp_weights* layers, int32_t n_layers, const void* x,
                                  const float* prev_logits, const void* dy, const float* dlogits_last,
                                  float balance_scale, float* balance_loss_out, const void* train_workspace,
                                  size_t train_workspace_bytes, const moepp_grads* grads, void* bwd_workspace,
                                  size_t bwd_workspace_bytes, void* stream) {
  Dims d;
  const moepp_status s = make_dims(cfg, &d);
  if (s != MOEPP_OK) return s;
  if (layers == nullptr || grads == nullptr || n_layers < 1 || train_workspace == nullptr || bwd_workspace == nullptr)
    return MOEPP_ERR_INVALID_ARG;
  if (d.flags & MOEPP_FLAG_FUSED_GATHER) return MOEPP_ERR_INVALID_ARG;
  if ((reinterpret_cast<uintptr_t>(train_workspace) & (kAlign - 1)) != 0 ||
      (reinterpret_cast<uintptr_t>(bwd_workspace) & (kAlign - 1)) != 0)
    return MOEPP_ERR_ALIGN;
  size_t act, lg, stats;
  const size_t slot = train_slot_bytes(d, &act, &lg);
  if (train_workspace_bytes < (size_t)n_layers * slot) return MOEPP_ERR_WORKSPACE;
  if (bwd_workspace_bytes < stack_backward_bytes(d, &act, &lg, &stats)) return MOEPP_ERR_WORKSPACE;
  const Carve c = carve(d, false);
  const size_t bc_total = carve_backward(d).total;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const char* ws = static_cast<const char*>(train_workspace);
  char* bw = static_cast<char*>(bwd_workspace);
  void* dxbuf[2] = {bw + bc_total, bw + bc_total + act};
  float* dlbuf[2] = {reinterpret_cast<float*>(bw + bc_total + 2 * act),
                     reinterpret_cast<float*>(bw + bc_total + 2 * act + lg)};
  float* st_f = reinterpret_cast<float*>(bw + bc_total + 2 * act + 2 * lg);
  float* st_P = st_f + d.N;
  float* st_loss = st_P + d.N;
  const size_t lg_bytes = sizeof(float) * (size_t)d.T * d.N;
  const bool balance = balance_scale != 0.f;

  for (int j = n_layers - 1; j >= 0; --j) {
    const char* sl = ws + (size_t)j * slot;
    const moepp_weights* w = &layers[j];
    const bool last = (j == n_layers - 1);
    const void* x_j = j == 0 ? x : static_cast<const void*>(ws + (size_t)(j - 1) * slot + c.total);
    const float* in_logits = j == 0 ? prev_logits : reinterpret_cast<const float*>(ws + (size_t)(j - 1) * slot + c.total + act);
    const float* prev_j = (w->W_g != nullptr) ? in_logits : nullptr;
    const float* logits_j = reinterpret_cast<const float*>(sl + c.total + act);
    const void* dy_j = last ? dy : dxbuf[(j + 1) & 1];
    // what arrives at this layer's logits from above: the next layer's dprev, or the caller's dlogits_last
    const float* dl = last ? dlogits_last : (layers[j + 1].W_g != nullptr ? dlbuf[(j + 1) & 1] : nullptr);
    if (balance && d.T > 0) {  // + balance_scale * dL_b/dlogits of this layer (Eq. 7)
      const int32_t* counts = reinterpret_cast<const int32_t*>(sl + c.counts);
      if (launch_balance_stats(d, logits_j, counts, st_f, st_P, st_loss, st) != cudaSuccess) return MOEPP_ERR_CUDA;
      if (balance_loss_out != nullptr &&
          cudaMemcpyAsync(balance_loss_out + j, st_loss, sizeof(float), cudaMemcpyDeviceToDevice, st) != cudaSuccess)
        return MOEPP_ERR_CUDA;
      float* mine = dlbuf[(j + 1) & 1];
      if (last && dl != nullptr) {
        if (cudaMemcpyAsync(mine, dl, lg_bytes, cudaMemcpyDeviceToDevice, st) != cudaSuccess) return MOEPP_ERR_CUDA;
      }
      if (launch_balance_backward(d, logits_j, st_f, balance_scale, dl != nullptr ? 1 : 0, mine, st) != cudaSuccess)
        return MOEPP_ERR_CUDA;
      dl = mine;
    }
    moepp_grads g = grads[j];
    if (j > 0) {
      g.dx = dxbuf[j & 1];
      g.dprev = (w->W_g != nullptr) ? dlbuf[j & 1] : nullptr;
    }
    const moepp_status r = layer_backward_on_device(d, w, x_j, prev_j, logits_j, dy_j, dl, sl, g, bw, st);
    if (r != MOEPP_OK) return r;
  }
  return MOEPP_OK;
}

moepp_status moepp_device_error(int32_t* code) {
  if (code == nullptr) return MOEPP_ERR_INVALID_ARG;
  const cudaError_t e = read_and_clear_device_error(code);
  if (e != cudaSuccess) return MOEPP_ERR_CUDA;
  return *code == 0 ? MOEPP_OK : MOEPP_ERR_TIMEOUT;
}

}  // extern "C"
