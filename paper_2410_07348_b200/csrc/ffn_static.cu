// Grouped SwiGLU FFN for callers that cannot provide scratch memory: the [M_cap, F] intermediate lives
// in a fixed array that is part of this library's device image instead of a caller buffer.
//
// The array below is reserved on every GPU that loads the library, from load until the process exits.
// In host code its name is only a handle for the runtime, not an address a kernel can use, so the
// device address is looked up once per device with cudaGetSymbolAddress and that pointer is what the
// kernels receive.
#include <mutex>

#include "common.cuh"

namespace {

static __device__ __align__(256) unsigned char g_ffn_static_scratch[MOEPP_STATIC_SCRATCH_BYTES];

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
void* g_scratch_addr[kMaxDevices] = {};

// Device address of the scratch array on the current device (looked up on the first call per device).
cudaError_t scratch_address(void** out) {
  int dev = 0;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return e;
  if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
  std::lock_guard<std::mutex> lock(g_setup_mutex);
  if (g_scratch_addr[dev] == nullptr) {
    void* p = nullptr;
    e = cudaGetSymbolAddress(&p, g_ffn_static_scratch);
    if (e != cudaSuccess) return e;
    if (p == nullptr) return cudaErrorInvalidSymbol;
    g_scratch_addr[dev] = p;
  }
  *out = g_scratch_addr[dev];
  return cudaSuccess;
}

inline bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace

extern "C" moepp_status moepp_grouped_ffn_static(const moepp_config* c, const void* x_perm,
                                                 const int32_t* expert_offsets, const void* W_gate, const void* W_up,
                                                 const void* W_down, void* y_perm, void* stream) {
  using namespace moepp;
  // the same configuration rules as every other call
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
  const long long M_cap = (long long)c->T * c->top_k + (long long)c->n_ffn * (c->row_align - 1);
  if (M_cap > 0x7fffffffLL) return MOEPP_ERR_UNSUPPORTED;

  // the intermediate must fit the fixed array
  const unsigned long long need = (unsigned long long)M_cap * (unsigned long long)c->F * elem_size(c->dtype);
  if (need > (unsigned long long)MOEPP_STATIC_SCRATCH_BYTES) return MOEPP_ERR_WORKSPACE;

  if (expert_offsets == nullptr) return MOEPP_ERR_INVALID_ARG;
  if (c->T > 0 && c->n_ffn > 0 &&
      (x_perm == nullptr || y_perm == nullptr || W_gate == nullptr || W_up == nullptr || W_down == nullptr))
    return MOEPP_ERR_INVALID_ARG;
  if (!aligned16(x_perm) || !aligned16(W_gate) || !aligned16(W_up) || !aligned16(W_down) || !aligned16(y_perm))
    return MOEPP_ERR_ALIGN;
  if (c->T == 0 || c->n_ffn == 0) return MOEPP_OK;

  Dims d{};
  d.tau = 1.f; d.cap_on = 0; d.cap_ffn = d.cap_zc = 0x7fffffff;
  d.T = c->T; d.D = c->D; d.F = c->F;
  d.n_ffn = c->n_ffn; d.n_zero = c->n_zero; d.n_copy = c->n_copy; d.n_const = c->n_const;
  d.N = (int)N; d.K = c->top_k;
  d.dtype = c->dtype; d.renorm = c->renorm_topk ? 1 : 0; d.row_align = c->row_align;
  d.add_residual = c->add_residual ? 1 : 0; d.flags = c->flags;
  d.M_cap = M_cap;

  void* h = nullptr;
  if (scratch_address(&h) != cudaSuccess) return MOEPP_ERR_CUDA;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  cudaError_t e;
  if (d.dtype == MOEPP_BF16 && !(d.flags & MOEPP_FLAG_SIMT_FFN)) {
    e = (d.flags & MOEPP_FLAG_FFN_SINGLE_CTA)
            ? launch_ffn_tcgen05(d, x_perm, expert_offsets, W_gate, W_up, W_down, h, y_perm, st)
            : launch_ffn_tcgen05_pair(d, x_perm, expert_offsets, W_gate, W_up, W_down, h, y_perm, st);
    if (e == cudaErrorNotSupported) return MOEPP_ERR_UNSUPPORTED;
  } else {
    e = launch_ffn_simt(d, x_perm, expert_offsets, W_gate, W_up, W_down, h, y_perm, st);
  }
  return e == cudaSuccess ? MOEPP_OK : MOEPP_ERR_CUDA;
}
