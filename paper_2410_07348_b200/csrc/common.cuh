// Internal declarations shared by the kernels and the C-ABI layer of the MoE++ forward library.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "moepp.h"

namespace moepp {

constexpr int kMaxExperts = 64;     // N
constexpr int kMaxTopK = 8;         // K
constexpr int kMaxRouteRows = 128;  // N + 2 * n_const

struct Dims {
  int T, D, F;
  int n_ffn, n_zero, n_copy, n_const, N, K;
  int dtype, renorm, row_align, add_residual, flags;
  long long M_cap;
  float tau;             // Eq. 7 / Eq. 8
  int cap_on;            // Eq. 8 active
  int cap_ffn, cap_zc;   // slots an FFN / a zero-computation expert serves (INT_MAX when off)
  __host__ __device__ int zero0() const { return n_ffn; }
  __host__ __device__ int copy0() const { return n_ffn + n_zero; }
  __host__ __device__ int const0() const { return n_ffn + n_zero + n_copy; }
};

inline size_t elem_size(int dtype) { return dtype == MOEPP_BF16 ? 2 : 4; }

// ---- kernel launchers (each enqueues on `st` and returns the launch status) -------------------
cudaError_t launch_route(const Dims& d, const void* x, const float* W_r, const float* W_g, const float* prev,
                         const float* bias, const float* W_c, float* logits, int32_t* topk_idx, float* topk_w,
                         int32_t* counts, int32_t* offsets, float* alpha, cudaStream_t st);

// bf16 router with the projection on the tensor cores; cudaErrorNotSupported when it does not apply.
cudaError_t launch_route_tc(const Dims& d, const void* x, const float* W_r, const float* W_g, const float* prev,
                            const float* bias, const float* W_c, float* logits, int32_t* topk_idx, float* topk_w,
                            int32_t* counts, float* alpha, cudaStream_t st);

cudaError_t launch_permute(const Dims& d, const void* x, const int32_t* topk_idx, const int32_t* offsets,
                           int32_t* row_of_slot, int32_t* slot_of_row, void* x_perm, cudaStream_t st);

cudaError_t launch_gather_rows(const void* src, const int32_t* index, long long n_rows, size_t row_bytes, void* dst,
                               cudaStream_t st);

// gate_out / up_out (both or neither): the SwiGLU pre-activations [M_cap, F] are stored as well
cudaError_t launch_ffn_simt(const Dims& d, const void* x_perm, const int32_t* offsets, const void* W_gate,
                            const void* W_up, const void* W_down, void* h, void* y_perm, cudaStream_t st,
                            void* gate_out = nullptr, void* up_out = nullptr);

// bf16 tensor-core path; returns cudaErrorNotSupported if the tensor maps cannot be encoded.
cudaError_t launch_ffn_tcgen05(const Dims& d, const void* x_perm, const int32_t* offsets, const void* W_gate,
                               const void* W_up, const void* W_down, void* h, void* y_perm, cudaStream_t st);

// single-CTA kernels with GEMM 1 gathering its rows from x through slot_of_row (x_perm is never built)
cudaError_t launch_ffn_tcgen05_gather(const Dims& d, const void* x, const int32_t* slot_of_row, const int32_t* offsets,
                                      const void* W_gate, const void* W_up, const void* W_down, void* h, void* y_perm,
                                      cudaStream_t st);

// the same on CTA pairs (cta_group::2, 256 x 256 tiles)
cudaError_t launch_ffn_tcgen05_pair(const Dims& d, const void* x_perm, const int32_t* offsets, const void* W_gate,
                                    const void* W_up, const void* W_down, void* h, void* y_perm, cudaStream_t st,
                                    void* gate_out = nullptr, void* up_out = nullptr);

cudaError_t launch_balance_stats(const Dims& d, const float* logits, const int32_t* counts, float* f, float* P,
                                 float* loss, cudaStream_t st);

cudaError_t launch_balance_backward(const Dims& d, const float* logits, const float* f, float scale, int accumulate,
                                    float* dlogits, cudaStream_t st);

cudaError_t launch_combine(const Dims& d, const void* x, const void* y_perm, const int32_t* topk_idx,
                           const float* topk_w, const int32_t* row_of_slot, const float* alpha, const float* W_c,
                           const float* v, void* y, cudaStream_t st);

// ---- backward pass ---------------------------------------------------------------------------------
// What the forward pass left in its workspace (all device pointers).
struct ForwardState {
  const float* logits;
  const int32_t* topk_idx;
  const float* topk_w;
  const int32_t* offsets;
  const float* alpha;
  const int32_t* row_of_slot;
  const int32_t* slot_of_row;
  const void* x_perm;
  const void* h;
  const void* y_perm;
  const void* gate;  // SwiGLU pre-activations [M_cap, F] if the forward pass kept them, else nullptr
  const void* up;
};

// Device scratch of one backward pass.
struct BackwardScratch {
  void *dYp, *gate, *up, *dXp;  // grouped rows, activation dtype: [M_cap, D], [M_cap, F] x 2, [M_cap, D]
  float* dw;                    // [T, K]
  float* dGz;                   // [T, R], R = N + 2 n_const: dL/dlogits, then dL/d(mixing logits)
  float* cx;                    // [T]
  float* cvq;                   // [T, n_const]
  float* part;                  // partial sums of the reductions over tokens (see backward_part_floats)
  void* split;                  // [T, 128] bf16: a small float factor as hi (columns 0..63) + lo (64..127) terms
  int32_t* segs;                // [65] token segments of the tensor-core reduction
};

// Token segments of the tensor-core reductions (whole 64-token tiles each, at most 64 segments).
int backward_token_segments(const Dims& d, int* tokens_per_segment);
size_t backward_part_floats(const Dims& d);

// part[seg, m, n] = sum over the tokens t of segment seg of P[t, m] Q[t, n] on the tensor cores:
// P [T, 128] bf16 (hi | lo columns), Q [T, D] bf16, part [n_seg, 128, D] float.  cudaErrorNotSupported if the
// tensor maps cannot be encoded.
cudaError_t launch_token_outer_tc(const Dims& d, const void* P, const void* Q, float* part, const int32_t* segs,
                                  int n_seg, cudaStream_t st);

int backward_token_chunks(const Dims& d, int* chunk_tokens);

// gate_in / up_in: pre-activations kept by the forward pass (nullptr: they are recomputed into gate_buf / up_buf)
cudaError_t launch_ffn_backward_simt(const Dims& d, const void* x_perm, const int32_t* offsets, const void* W_gate,
                                     const void* W_up, const void* W_down, const void* h, const void* dy_perm,
                                     void* gate_buf, void* up_buf, void* dx_perm, float* dW_gate, float* dW_up,
                                     float* dW_down, cudaStream_t st, const void* gate_in = nullptr,
                                     const void* up_in = nullptr);

// The same on the tensor cores (bf16 storage); cudaErrorNotSupported otherwise.
cudaError_t launch_ffn_backward_tc(const Dims& d, const void* x_perm, const int32_t* offsets, const void* W_gate,
                                   const void* W_up, const void* W_down, const void* h, const void* dy_perm,
                                   void* gate_buf, void* up_buf, void* dx_perm, float* dW_gate, float* dW_up,
                                   float* dW_down, cudaStream_t st, const void* gate_in = nullptr,
                                   const void* up_in = nullptr);

// C[r, :] = A[r, :] B[e]^T on the forward tensor-core kernel (A [M_cap, Kd], B [n_ffn, Nout, Kd], bf16)
cudaError_t launch_grouped_gemm_tcgen05(const Dims& d, const void* A, const void* B, void* C, const int32_t* offsets,
                                        int Nout, int Kd, cudaStream_t st);

// Whole backward pass of one layer; grads are overwritten.
cudaError_t launch_layer_backward(const Dims& d, const ForwardState& fs, const moepp_weights& w, const void* x,
                                  const float* prev, const void* dy, const float* dlogits_next,
                                  const BackwardScratch& b, const moepp_grads& g, cudaStream_t st);

// Error word written by kernels whose bounded waits ran out (0 = fine).
cudaError_t read_and_clear_device_error(int32_t* code);
int32_t* device_error_word();  // device address of that word on the current device (nullptr on failure)

// ---- small device helpers -----------------------------------------------------------------------
__device__ __forceinline__ float bf16_lo(uint32_t u) { return __uint_as_float(u << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t u) { return __uint_as_float(u & 0xffff0000u); }
__device__ __forceinline__ uint32_t pack_bf16(float a, float b) {
  __nv_bfloat162 p = __floats2bfloat162_rn(a, b);
  return *reinterpret_cast<uint32_t*>(&p);
}

// 8 consecutive elements of a row as floats (16 bytes of bf16, or 32 bytes of float).
template <typename T>
struct Vec8;
template <>
struct Vec8<__nv_bfloat16> {
  static __device__ __forceinline__ void load(const __nv_bfloat16* p, float (&f)[8]) {
    const uint4 u = *reinterpret_cast<const uint4*>(p);
    f[0] = bf16_lo(u.x); f[1] = bf16_hi(u.x); f[2] = bf16_lo(u.y); f[3] = bf16_hi(u.y);
    f[4] = bf16_lo(u.z); f[5] = bf16_hi(u.z); f[6] = bf16_lo(u.w); f[7] = bf16_hi(u.w);
  }
  static __device__ __forceinline__ void store(__nv_bfloat16* p, const float (&f)[8]) {
    uint4 u;
    u.x = pack_bf16(f[0], f[1]); u.y = pack_bf16(f[2], f[3]); u.z = pack_bf16(f[4], f[5]); u.w = pack_bf16(f[6], f[7]);
    *reinterpret_cast<uint4*>(p) = u;
  }
};
template <>
struct Vec8<float> {
  static __device__ __forceinline__ void load(const float* p, float (&f)[8]) {
    const float4 a = *reinterpret_cast<const float4*>(p);
    const float4 b = *reinterpret_cast<const float4*>(p + 4);
    f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w; f[4] = b.x; f[5] = b.y; f[6] = b.z; f[7] = b.w;
  }
  static __device__ __forceinline__ void store(float* p, const float (&f)[8]) {
    *reinterpret_cast<float4*>(p) = make_float4(f[0], f[1], f[2], f[3]);
    *reinterpret_cast<float4*>(p + 4) = make_float4(f[4], f[5], f[6], f[7]);
  }
};

}  // namespace moepp
