// Grouped SwiGLU FFN on plain FMA units: the float path of the library, and a cross-check for the
// tensor-core path.  For every FFN expert e and every row r of its segment:
//   h[r,:] = silu(W_gate[e] x_perm[r,:]) * (W_up[e] x_perm[r,:]),   y_perm[r,:] = W_down[e] h[r,:].
// 64x64 output tile per block, 16-wide k step, 4x4 outputs per thread, float accumulation.
#include "common.cuh"

namespace moepp {
namespace {

constexpr int BM = 64, BN = 64, BK = 16;

template <typename T>
__device__ __forceinline__ void load4(const T* p, float (&f)[4]);
template <>
__device__ __forceinline__ void load4<float>(const float* p, float (&f)[4]) {
  const float4 a = *reinterpret_cast<const float4*>(p);
  f[0] = a.x; f[1] = a.y; f[2] = a.z; f[3] = a.w;
}
template <>
__device__ __forceinline__ void load4<__nv_bfloat16>(const __nv_bfloat16* p, float (&f)[4]) {
  const uint2 u = *reinterpret_cast<const uint2*>(p);
  f[0] = bf16_lo(u.x); f[1] = bf16_hi(u.x); f[2] = bf16_lo(u.y); f[3] = bf16_hi(u.y);
}
__device__ __forceinline__ void store1(float* p, float v) { *p = v; }
__device__ __forceinline__ void store1(__nv_bfloat16* p, float v) { *p = __float2bfloat16_rn(v); }

// C[rows of expert e, Nout] = A[rows, Kd] . B_e[Nout, Kd]^T   (SWIGLU: silu(A.B0^T) * (A.B1^T))
template <typename T, bool SWIGLU>
__global__ void __launch_bounds__(256)
ffn_simt_kernel(const T* __restrict__ A, const T* __restrict__ B0, const T* __restrict__ B1, T* __restrict__ C,
                const int32_t* __restrict__ offsets, int n_ffn, int Nout, int Kd, T* __restrict__ G,
                T* __restrict__ U) {
  __shared__ float As[BK][BM + 4];
  __shared__ float Bs0[BK][BN + 4];
  __shared__ float Bs1[SWIGLU ? BK : 1][BN + 4];

  // which expert owns m-tile blockIdx.x
  int e = 0, tile0 = 0, row0 = 0, row_end = 0;
  {
    const int t = blockIdx.x;
    bool found = false;
    for (e = 0; e < n_ffn; ++e) {
      const int b = offsets[e], en = offsets[e + 1];
      const int nt = (en - b + BM - 1) / BM;
      if (t < tile0 + nt) {
        row0 = b + (t - tile0) * BM;
        row_end = en;
        found = true;
        break;
      }
      tile0 += nt;
    }
    if (!found) return;
  }
  const int n0 = blockIdx.y * BN;
  const T* Be0 = B0 + (size_t)e * Nout * Kd;
  const T* Be1 = SWIGLU ? (B1 + (size_t)e * Nout * Kd) : nullptr;

  const int tid = threadIdx.x;
  const int tx = tid & 15, ty = tid >> 4;       // 16 x 16 threads, each 4 x 4 outputs
  const int lr = tid >> 2, lk = (tid & 3) * 4;  // loader: row lr (0..63), k offset lk

  float acc0[4][4], acc1[4][4];
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) { acc0[i][j] = 0.f; acc1[i][j] = 0.f; }

  for (int k0 = 0; k0 < Kd; k0 += BK) {
    float a[4] = {0.f, 0.f, 0.f, 0.f}, b0[4] = {0.f, 0.f, 0.f, 0.f}, b1[4] = {0.f, 0.f, 0.f, 0.f};
    const bool k_ok = (k0 + lk) < Kd;
    if (k_ok && row0 + lr < row_end) load4<T>(A + (size_t)(row0 + lr) * Kd + k0 + lk, a);
    if (k_ok && n0 + lr < Nout) {
      load4<T>(Be0 + (size_t)(n0 + lr) * Kd + k0 + lk, b0);
      if (SWIGLU) load4<T>(Be1 + (size_t)(n0 + lr) * Kd + k0 + lk, b1);
    }
    __syncthreads();
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      As[lk + i][lr] = a[i];
      Bs0[lk + i][lr] = b0[i];
      if (SWIGLU) Bs1[lk + i][lr] = b1[i];
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < BK; ++kk) {
      const float4 av = *reinterpret_cast<const float4*>(&As[kk][ty * 4]);
      const float4 bv = *reinterpret_cast<const float4*>(&Bs0[kk][tx * 4]);
      const float am[4] = {av.x, av.y, av.z, av.w};
      const float bm[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc0[i][j] = fmaf(am[i], bm[j], acc0[i][j]);
      if (SWIGLU) {
        const float4 cv = *reinterpret_cast<const float4*>(&Bs1[kk][tx * 4]);
        const float cm[4] = {cv.x, cv.y, cv.z, cv.w};
#pragma unroll
        for (int i = 0; i < 4; ++i)
#pragma unroll
          for (int j = 0; j < 4; ++j) acc1[i][j] = fmaf(am[i], cm[j], acc1[i][j]);
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
      if (n >= Nout) continue;
      float val = acc0[i][j];
      if (SWIGLU && G != nullptr) {  // keep the pre-activations for the backward pass
        store1(G + (size_t)r * Nout + n, acc0[i][j]);
        store1(U + (size_t)r * Nout + n, acc1[i][j]);
      }
      if (SWIGLU) val = (val / (1.f + expf(-val))) * acc1[i][j];
      store1(C + (size_t)r * Nout + n, val);
    }
  }
}

template <typename T>
cudaError_t launch_t(const Dims& d, const void* x_perm, const int32_t* offsets, const void* W_gate, const void* W_up,
                     const void* W_down, void* h, void* y_perm, cudaStream_t st, void* gate_out, void* up_out) {
  const unsigned mt = (unsigned)((d.M_cap + BM - 1) / BM + d.n_ffn);
  dim3 g1(mt, (unsigned)((d.F + BN - 1) / BN)), g2(mt, (unsigned)((d.D + BN - 1) / BN));
  ffn_simt_kernel<T, true><<<g1, 256, 0, st>>>(static_cast<const T*>(x_perm), static_cast<const T*>(W_gate),
                                               static_cast<const T*>(W_up), static_cast<T*>(h), offsets, d.n_ffn,
                                               d.F, d.D, static_cast<T*>(gate_out), static_cast<T*>(up_out));
  cudaError_t err = cudaGetLastError();
  if (err != cudaSuccess) return err;
  ffn_simt_kernel<T, false><<<g2, 256, 0, st>>>(static_cast<const T*>(h), static_cast<const T*>(W_down), nullptr,
                                                static_cast<T*>(y_perm), offsets, d.n_ffn, d.D, d.F, nullptr,
                                                nullptr);
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_ffn_simt(const Dims& d, const void* x_perm, const int32_t* offsets, const void* W_gate,
                            const void* W_up, const void* W_down, void* h, void* y_perm, cudaStream_t st,
                            void* gate_out, void* up_out) {
  if (d.T == 0 || d.n_ffn == 0 || d.M_cap == 0) return cudaSuccess;
  return d.dtype == MOEPP_BF16
             ? launch_t<__nv_bfloat16>(d, x_perm, offsets, W_gate, W_up, W_down, h, y_perm, st, gate_out, up_out)
             : launch_t<float>(d, x_perm, offsets, W_gate, W_up, W_down, h, y_perm, st, gate_out, up_out);
}

}  // namespace moepp
