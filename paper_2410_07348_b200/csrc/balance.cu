// Heterogeneous load-balance statistics (Eq. 7): f_i = share of tokens selecting expert i,
// P_i = mean softmax weight of expert i, L_b = sum_i eta_i f_i P_i with eta = 1 (FFN) or tau
// (zero-computation).  A training-time by-product of the router, far off the forward hot path:
// one CTA, fixed reduction order, so the result is reproducible bit for bit.
#include "common.cuh"

namespace moepp {
namespace {

constexpr int kBalThreads = 1024;

__global__ void __launch_bounds__(kBalThreads)
balance_stats_kernel(Dims dm, const float* __restrict__ logits, const int32_t* __restrict__ counts,
                     float* __restrict__ f, float* __restrict__ P, float* __restrict__ loss) {
  __shared__ float part[32][kMaxExperts];  // per-warp sums of the softmax columns
  __shared__ float col[kMaxExperts];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int N = dm.N;
  // lane i of a warp owns experts i and i + 32; a warp walks tokens warp, warp + 32, ...
  float acc0 = 0.f, acc1 = 0.f;
  for (long long t = warp; t < dm.T; t += 32) {
    const float g0 = (lane < N) ? logits[t * N + lane] : -INFINITY;
    const float g1 = (lane + 32 < N) ? logits[t * N + lane + 32] : -INFINITY;
    float m = fmaxf(g0, g1);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    const float p0 = (lane < N) ? expf(g0 - m) : 0.f, p1 = (lane + 32 < N) ? expf(g1 - m) : 0.f;
    float z = p0 + p1;
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
    acc0 += p0 / z;
    acc1 += p1 / z;
  }
  part[warp][lane] = acc0;
  part[warp][lane + 32] = acc1;
  __syncthreads();
  if (tid < N) {
    float s = 0.f;
    for (int w = 0; w < 32; ++w) s += part[w][tid];  // fixed order
    const float inv_T = dm.T > 0 ? 1.f / (float)dm.T : 0.f;
    const float pi = s * inv_T, fi = (float)counts[tid] * inv_T;
    P[tid] = pi;
    f[tid] = fi;
    col[tid] = (tid < dm.n_ffn ? 1.f : dm.tau) * fi * pi;
  }
  __syncthreads();
  if (tid == 0) {
    float L = 0.f;
    for (int i = 0; i < N; ++i) L += col[i];
    *loss = L;
  }
}

}  // namespace

cudaError_t launch_balance_stats(const Dims& d, const float* logits, const int32_t* counts, float* f, float* P,
                                 float* loss, cudaStream_t st) {
  balance_stats_kernel<<<1, kBalThreads, 0, st>>>(d, logits, counts, f, P, loss);
  return cudaGetLastError();
}

}  // namespace moepp
