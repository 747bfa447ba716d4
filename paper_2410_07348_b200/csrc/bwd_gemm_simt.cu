// Grouped GEMMs of the backward pass on plain FMA units (float storage, and the cross-check for bf16).
//   rows-kernel : C[r, n] = sum_k A[r, k] * B_e(k, n) (+ a second product A2 . B2_e) for every row r of expert e's
//                 segment; B_e is addressed through strides, so W or W^T are the same kernel.  An optional
//                 epilogue turns dH into the SwiGLU input gradients in place.
//   wgrad-kernel: C_e[m, n] = sum over the rows r of expert e's segment of A[r, m] * B[r, n].
// 64x64 output tile, 16-wide k step, 4x4 outputs per thread, float accumulation.
#include "common.cuh"

namespace moepp {
namespace {

constexpr int TM = 64, TN = 64, TK = 16;

__device__ __forceinline__ float ldf(const float* p) { return *p; }
__device__ __forceinline__ float ldf(const __nv_bfloat16* p) { return __bfloat162float(*p); }
__device__ __forceinline__ void stf(float* p, float v) { *p = v; }
__device__ __forceinline__ void stf(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

struct RowsArgs {
  const void *A, *B, *A2, *B2;   // second product optional (A2 == nullptr)
  void* C;
  void *gate, *up;               // SwiGLU-backward epilogue: dGate / dUp out (C unused)
  const void *gate_in, *up_in;   // ... and the pre-activations it reads (may be the same buffers)
  const int32_t* offsets;
  int n_ffn, Nout, Kd;
  long long a_rs, c_rs;          // row strides of A (and A2) and C
  long long b_es, b_ks, b_ns;    // B_e(k, n) = B[e*b_es + k*b_ks + n*b_ns]
};

// EPI 0: store C;  EPI 1: C is dH: dGate = dH * up * silu'(gate), dUp = dH * silu(gate), written over gate / up
template <typename T, int EPI>
__global__ void __launch_bounds__(256) bwd_rows_kernel(RowsArgs a) {
  __shared__ float As[TK][TM + 4], Bs[TK][TN + 4];
  int e = 0, tile0 = 0, row0 = 0, row_end = 0;
  {
    bool found = false;
    for (e = 0; e < a.n_ffn; ++e) {
      const int b = a.offsets[e], en = a.offsets[e + 1], nt = (en - b + TM - 1) / TM;
      if ((int)blockIdx.x < tile0 + nt) { row0 = b + ((int)blockIdx.x - tile0) * TM; row_end = en; found = true; break; }
      tile0 += nt;
    }
    if (!found) return;
  }
  const int n0 = blockIdx.y * TN, tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  float acc[4][4] = {};
  for (int pass = 0; pass < 2; ++pass) {
    const T* A = static_cast<const T*>(pass ? a.A2 : a.A);
    const T* B = static_cast<const T*>(pass ? a.B2 : a.B);
    if (A == nullptr) break;
    const T* Be = B + (size_t)e * a.b_es;
    for (int k0 = 0; k0 < a.Kd; k0 += TK) {
      __syncthreads();
      for (int i = tid; i < TM * TK; i += 256) {
        const int m = i / TK, k = i % TK;
        As[k][m] = (row0 + m < row_end && k0 + k < a.Kd) ? ldf(A + (size_t)(row0 + m) * a.a_rs + k0 + k) : 0.f;
      }
      for (int i = tid; i < TN * TK; i += 256) {
        const int n = i % TN, k = i / TN;
        Bs[k][n] = (n0 + n < a.Nout && k0 + k < a.Kd) ? ldf(Be + (size_t)(k0 + k) * a.b_ks + (size_t)(n0 + n) * a.b_ns) : 0.f;
      }
      __syncthreads();
#pragma unroll
      for (int kk = 0; kk < TK; ++kk) {
        const float4 av = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
        const float4 bv = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
        const float am[4] = {av.x, av.y, av.z, av.w}, bm[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(am[i], bm[j], acc[i][j]);
      }
    }
  }
#pragma unroll
  for (int i = 0; i < 4; ++i) {
    const int r = row0 + ty * 4 + i;
    if (r >= row_end) continue;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int n = n0 + tx * 4 + j;
      if (n >= a.Nout) continue;
      const size_t at = (size_t)r * a.c_rs + n;
      if (EPI == 0) {
        stf(static_cast<T*>(a.C) + at, acc[i][j]);
      } else {
        T* gp = static_cast<T*>(a.gate) + at;
        T* up = static_cast<T*>(a.up) + at;
        const float g = ldf(static_cast<const T*>(a.gate_in) + at), u = ldf(static_cast<const T*>(a.up_in) + at);
        const float s = 1.f / (1.f + expf(-g)), dh = acc[i][j];
        stf(gp, dh * u * (s + g * s * (1.f - s)));
        stf(up, dh * g * s);
      }
    }
  }
}

// C_e[m, n] = sum_{r in segment e} A[r*a_rs + m] * B[r*b_rs + n];  C is float, [n_ffn][Mout][Nout]
template <typename T>
__global__ void __launch_bounds__(256)
bwd_wgrad_kernel(const T* __restrict__ A, const T* __restrict__ B, float* __restrict__ C,
                 const int32_t* __restrict__ offsets, int Mout, int Nout, long long a_rs, long long b_rs,
                 int accumulate) {
  __shared__ float As[TK][TM + 4], Bs[TK][TN + 4];
  const int e = blockIdx.z, m0 = blockIdx.x * TM, n0 = blockIdx.y * TN;
  const int r_begin = offsets[e], r_end = offsets[e + 1];
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  float acc[4][4] = {};
  for (int r0 = r_begin; r0 < r_end; r0 += TK) {
    __syncthreads();
    for (int i = tid; i < TM * TK; i += 256) {
      const int m = i % TM, k = i / TM;
      As[k][m] = (r0 + k < r_end && m0 + m < Mout) ? ldf(A + (size_t)(r0 + k) * a_rs + m0 + m) : 0.f;
    }
    for (int i = tid; i < TN * TK; i += 256) {
      const int n = i % TN, k = i / TN;
      Bs[k][n] = (r0 + k < r_end && n0 + n < Nout) ? ldf(B + (size_t)(r0 + k) * b_rs + n0 + n) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < TK; ++kk) {
      const float4 av = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
      const float4 bv = *reinterpret_cast<const float4*>(&Bs[kk][tx * 4]);
      const float am[4] = {av.x, av.y, av.z, av.w}, bm[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(am[i], bm[j], acc[i][j]);
    }
  }
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int m = m0 + ty * 4 + i, n = n0 + tx * 4 + j;
      if (m < Mout && n < Nout) {
        float* dst = C + ((size_t)e * Mout + m) * Nout + n;
        *dst = accumulate ? *dst + acc[i][j] : acc[i][j];
      }
    }
}

template <typename T>
cudaError_t run_rows(const Dims& d, RowsArgs a, bool swiglu_bwd, cudaStream_t st) {
  dim3 grid((unsigned)((d.M_cap + TM - 1) / TM + d.n_ffn), (unsigned)((a.Nout + TN - 1) / TN));
  if (swiglu_bwd) bwd_rows_kernel<T, 1><<<grid, 256, 0, st>>>(a);
  else bwd_rows_kernel<T, 0><<<grid, 256, 0, st>>>(a);
  return cudaGetLastError();
}

}  // namespace

namespace {

template <typename T>
cudaError_t ffn_backward_t(const Dims& d, const void* x_perm, const int32_t* offsets, const void* W_gate,
                           const void* W_up, const void* W_down, const void* h, const void* dy_perm, void* gate_buf,
                           void* up_buf, void* dx_perm, float* dW_gate, float* dW_up, float* dW_down,
                           cudaStream_t st, const void* gate_in, const void* up_in) {
  const long long D = d.D, F = d.F;
  const int accum = (d.flags & MOEPP_FLAG_ACCUM_GRADS) ? 1 : 0;
  cudaError_t err;
  if (gate_in == nullptr) {
    // 1-2. SwiGLU pre-activations again: gate = Xp W_gate^T, up = Xp W_up^T
    RowsArgs a{};
    a.offsets = offsets; a.n_ffn = d.n_ffn;
    a.A = x_perm; a.a_rs = D; a.Kd = d.D; a.Nout = d.F; a.c_rs = F; a.b_es = F * D; a.b_ks = 1; a.b_ns = D;
    a.B = W_gate; a.C = gate_buf;
    if ((err = run_rows<T>(d, a, false, st)) != cudaSuccess) return err;
    a.B = W_up; a.C = up_buf;
    if ((err = run_rows<T>(d, a, false, st)) != cudaSuccess) return err;
    gate_in = gate_buf;
    up_in = up_buf;
  }
  // 3. dW_down[e] = dYp_e^T H_e
  dim3 gdn((unsigned)((d.D + TM - 1) / TM), (unsigned)((d.F + TN - 1) / TN), (unsigned)d.n_ffn);
  bwd_wgrad_kernel<T><<<gdn, 256, 0, st>>>(static_cast<const T*>(dy_perm), static_cast<const T*>(h), dW_down, offsets,
                                           d.D, d.F, D, F, accum);
  if ((err = cudaGetLastError()) != cudaSuccess) return err;
  // 4. dH = dYp W_down, turned in place into dGate, dUp
  RowsArgs b{};
  b.offsets = offsets; b.n_ffn = d.n_ffn;
  b.A = dy_perm; b.a_rs = D; b.Kd = d.D; b.Nout = d.F; b.c_rs = F; b.B = W_down; b.b_es = D * F; b.b_ks = F; b.b_ns = 1;
  b.gate = gate_buf; b.up = up_buf; b.gate_in = gate_in; b.up_in = up_in;
  if ((err = run_rows<T>(d, b, true, st)) != cudaSuccess) return err;
  // 5. dW_gate[e] = dGate_e^T Xp_e, dW_up[e] = dUp_e^T Xp_e
  dim3 gup((unsigned)((d.F + TM - 1) / TM), (unsigned)((d.D + TN - 1) / TN), (unsigned)d.n_ffn);
  bwd_wgrad_kernel<T><<<gup, 256, 0, st>>>(static_cast<const T*>(gate_buf), static_cast<const T*>(x_perm), dW_gate,
                                           offsets, d.F, d.D, F, D, accum);
  if ((err = cudaGetLastError()) != cudaSuccess) return err;
  bwd_wgrad_kernel<T><<<gup, 256, 0, st>>>(static_cast<const T*>(up_buf), static_cast<const T*>(x_perm), dW_up, offsets,
                                           d.F, d.D, F, D, accum);
  if ((err = cudaGetLastError()) != cudaSuccess) return err;
  // 6. dXp = dGate W_gate + dUp W_up
  RowsArgs c{};
  c.offsets = offsets; c.n_ffn = d.n_ffn;
  c.A = gate_buf; c.A2 = up_buf; c.a_rs = F; c.Kd = d.F; c.Nout = d.D; c.c_rs = D;
  c.B = W_gate; c.B2 = W_up; c.b_es = F * D; c.b_ks = D; c.b_ns = 1; c.C = dx_perm;
  return run_rows<T>(d, c, false, st);
}

}  // namespace

// FFN backward for every expert segment.  In: x_perm, h (both from the forward pass), dy_perm.  Scratch: gate_buf,
// up_buf [M_cap, F].  Out: dx_perm [M_cap, D] and the three float weight gradients.
cudaError_t launch_ffn_backward_simt(const Dims& d, const void* x_perm, const int32_t* offsets, const void* W_gate,
                                     const void* W_up, const void* W_down, const void* h, const void* dy_perm,
                                     void* gate_buf, void* up_buf, void* dx_perm, float* dW_gate, float* dW_up,
                                     float* dW_down, cudaStream_t st, const void* gate_in, const void* up_in) {
  if (d.n_ffn == 0) return cudaSuccess;
  const size_t wbytes = sizeof(float) * (size_t)d.n_ffn * d.D * d.F;
  cudaError_t err;  // experts without rows still get a defined (zero) gradient
  if ((d.T == 0 || d.M_cap == 0) && (d.flags & MOEPP_FLAG_ACCUM_GRADS)) return cudaSuccess;  // nothing to add
  if (d.T == 0 || d.M_cap == 0) {
    if ((err = cudaMemsetAsync(dW_gate, 0, wbytes, st)) != cudaSuccess) return err;
    if ((err = cudaMemsetAsync(dW_up, 0, wbytes, st)) != cudaSuccess) return err;
    return cudaMemsetAsync(dW_down, 0, wbytes, st);
  }
  return d.dtype == MOEPP_BF16
             ? ffn_backward_t<__nv_bfloat16>(d, x_perm, offsets, W_gate, W_up, W_down, h, dy_perm, gate_buf, up_buf,
                                             dx_perm, dW_gate, dW_up, dW_down, st, gate_in, up_in)
             : ffn_backward_t<float>(d, x_perm, offsets, W_gate, W_up, W_down, h, dy_perm, gate_buf, up_buf, dx_perm,
                                     dW_gate, dW_up, dW_down, st, gate_in, up_in);
}

}  // namespace moepp
