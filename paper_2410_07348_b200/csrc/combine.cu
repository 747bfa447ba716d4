// Weighted combine of the K picks of every token (Eq. 1) with the zero-computation experts applied
// in place: a zero slot is skipped (Eq. 3), a copy slot adds g*x (Eq. 4), a constant slot adds
// g*(a1 x + a2 v) (Eq. 5); only FFN slots read a grouped row.  One warp per token, 16-byte vectors.
#include "common.cuh"

namespace moepp {
namespace {

constexpr int kCombineThreads = 256;

// KMAX: compile-time bound on the picks per token (2 or kMaxTopK); U: column chunks per trip;
// MINB: blocks per SM the register allocation must allow.
template <typename XT, int KMAX, int U, int MINB>
__global__ void __launch_bounds__(kCombineThreads, MINB)
combine_kernel(Dims dm, const XT* __restrict__ x, const XT* __restrict__ y_perm, const int32_t* __restrict__ topk_idx,
               const float* __restrict__ topk_w, const int32_t* __restrict__ row_of_slot,
               const float* __restrict__ alpha, const float* __restrict__ W_c, const float* __restrict__ v,
               XT* __restrict__ y) {
  const int lane = threadIdx.x & 31;
  const long long t = (long long)blockIdx.x * (kCombineThreads / 32) + (threadIdx.x >> 5);
  if (t >= dm.T) return;
  const int K = dm.K, D = dm.D;
  const int zero0 = dm.zero0(), copy0 = dm.copy0(), const0 = dm.const0();
  const XT* xt = x + (size_t)t * D;

  // lane k holds pick k
  int e_l = -1, row_l = -1;
  float w_l = 0.f;
  if (lane < K) {
    e_l = topk_idx[t * K + lane];
    w_l = topk_w[t * K + lane];
    row_l = row_of_slot[t * K + lane];
  }
  // coefficient of x, and per-pick coefficient of v for constant picks
  float cx = dm.add_residual ? 1.f : 0.f;
  float cv[KMAX], wk[KMAX];
  int vq[KMAX], rows[KMAX];
#pragma unroll
  for (int k = 0; k < KMAX; ++k) {
    cv[k] = 0.f; vq[k] = -1; rows[k] = -1; wk[k] = 0.f;
    if (k < K) {
      const int e = __shfl_sync(0xffffffffu, e_l, k);
      const float g = __shfl_sync(0xffffffffu, w_l, k);
      const int row = __shfl_sync(0xffffffffu, row_l, k);
      if (row == -2) {
        // Eq. 8: dropped at a full expert, contributes nothing
      } else if (e < zero0) {
        rows[k] = row; wk[k] = g;
      } else if (e < copy0) {
        // Eq. 3: contributes nothing
      } else if (e < const0) {
        cx += g;  // Eq. 4
      } else {
        const int q = e - const0;
        float a1, a2;
        if (alpha != nullptr) {
          a1 = alpha[(t * dm.n_const + q) * 2 + 0];
          a2 = alpha[(t * dm.n_const + q) * 2 + 1];
        } else {  // Eq. 5: [a1, a2] = Softmax(W_c x), computed by the warp
          const float* w0 = W_c + (size_t)q * 2 * D;
          const float* w1 = w0 + D;
          float z0 = 0.f, z1 = 0.f;
          for (int d = lane * 8; d < D; d += 256) {
            float xv[8];
            Vec8<XT>::load(xt + d, xv);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              z0 = fmaf(__ldg(w0 + d + i), xv[i], z0);
              z1 = fmaf(__ldg(w1 + d + i), xv[i], z1);
            }
          }
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) {
            z0 += __shfl_xor_sync(0xffffffffu, z0, o);
            z1 += __shfl_xor_sync(0xffffffffu, z1, o);
          }
          const float mm = fmaxf(z0, z1);
          const float e0 = expf(z0 - mm), e1 = expf(z1 - mm);
          a1 = e0 / (e0 + e1);
          a2 = e1 / (e0 + e1);
        }
        cx += g * a1;
        cv[k] = g * a2;
        vq[k] = q;
      }
    }
  }

  XT* yt = y + (size_t)t * D;
  // U column chunks (256 elements each) per trip: all row loads of a trip are issued before any is used,
  // so a warp keeps up to U * (picks + 1) 16-byte loads in flight.
  for (int d0 = lane * 8; d0 < D; d0 += 256 * U) {
    float acc[U][8];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int d = d0 + 256 * u;
#pragma unroll
      for (int i = 0; i < 8; ++i) acc[u][i] = 0.f;
      if (d < D && cx != 0.f) {
        float xv[8];
        Vec8<XT>::load(xt + d, xv);
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[u][i] = cx * xv[i];
      }
    }
#pragma unroll
    for (int k = 0; k < KMAX; ++k) {
      if (k < K) {
        if (rows[k] >= 0) {
          float yv[U][8];
#pragma unroll
          for (int u = 0; u < U; ++u) {
            const int d = d0 + 256 * u;
            if (d < D) Vec8<XT>::load(y_perm + (size_t)rows[k] * D + d, yv[u]);
          }
#pragma unroll
          for (int u = 0; u < U; ++u)
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[u][i] = fmaf(wk[k], yv[u][i], acc[u][i]);
        } else if (vq[k] >= 0) {
#pragma unroll
          for (int u = 0; u < U; ++u) {
            const int d = d0 + 256 * u;
            if (d < D) {
              const float* vp = v + (size_t)vq[k] * D + d;
              const float4 a = __ldg(reinterpret_cast<const float4*>(vp));
              const float4 b = __ldg(reinterpret_cast<const float4*>(vp + 4));
              acc[u][0] = fmaf(cv[k], a.x, acc[u][0]); acc[u][1] = fmaf(cv[k], a.y, acc[u][1]);
              acc[u][2] = fmaf(cv[k], a.z, acc[u][2]); acc[u][3] = fmaf(cv[k], a.w, acc[u][3]);
              acc[u][4] = fmaf(cv[k], b.x, acc[u][4]); acc[u][5] = fmaf(cv[k], b.y, acc[u][5]);
              acc[u][6] = fmaf(cv[k], b.z, acc[u][6]); acc[u][7] = fmaf(cv[k], b.w, acc[u][7]);
            }
          }
        }
      }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int d = d0 + 256 * u;
      if (d < D) Vec8<XT>::store(yt + d, acc[u]);
    }
  }
}

}  // namespace

cudaError_t launch_combine(const Dims& d, const void* x, const void* y_perm, const int32_t* topk_idx,
                           const float* topk_w, const int32_t* row_of_slot, const float* alpha, const float* W_c,
                           const float* v, void* y, cudaStream_t st) {
  if (d.T == 0) return cudaSuccess;
  const int tokens_per_block = kCombineThreads / 32;
  const unsigned grid = (unsigned)((d.T + tokens_per_block - 1) / tokens_per_block);
#define MOEPP_COMBINE(XT, KMAX, U)  MOEPP_COMBINE2(XT, KMAX, U, 1)
#define MOEPP_COMBINE2(XT, KMAX, U, MINB)                                                                             \
  combine_kernel<XT, KMAX, U, MINB><<<grid, kCombineThreads, 0, st>>>(                                               \
      d, static_cast<const XT*>(x), static_cast<const XT*>(y_perm), topk_idx, topk_w, row_of_slot, alpha, W_c, \
      v, static_cast<XT*>(y))
  if (d.dtype == MOEPP_BF16) {
    // two chunks per trip at four blocks per SM (64 registers) keeps the most bytes in flight: measured best
    if (d.K <= 2) MOEPP_COMBINE2(__nv_bfloat16, 2, 2, 4);
    else MOEPP_COMBINE(__nv_bfloat16, kMaxTopK, 1);
  } else {
    if (d.K <= 2) MOEPP_COMBINE(float, 2, 2);
    else MOEPP_COMBINE(float, kMaxTopK, 1);
  }
#undef MOEPP_COMBINE
  return cudaGetLastError();
}

}  // namespace moepp
