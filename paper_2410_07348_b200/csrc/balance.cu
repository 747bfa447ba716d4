// Heterogeneous load-balance statistics (Eq. 7): f_i = share of tokens selecting expert i,
// P_i = mean softmax weight of expert i, L_b = sum_i eta_i f_i P_i with eta = 1 (FFN) or tau
// (zero-computation).  A training-time by-product of the router, off the forward hot path:
// one cluster of eight CTAs, fixed reduction order, so the result is reproducible bit for bit.
#include "common.cuh"

namespace moepp {
namespace {


constexpr int kBalanceCtas = 8;  // one thread-block cluster

__device__ __forceinline__ uint32_t cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// float at the same shared-memory offset in CTA `rank` of this cluster
__device__ __forceinline__ float ld_cluster_f32(const float* p, uint32_t rank) {
  uint32_t a = (uint32_t)__cvta_generic_to_shared(p), ra;
  float v;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(a), "r"(rank));
  asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(ra) : "memory");
  return v;
}

// A cluster of kBalanceCtas CTAs.  One thread per token (tokens strided over all threads of the cluster), NP >= N
// per-thread column accumulators in registers (fewer threads for larger NP so that they stay there), then a
// fixed-order reduction: lanes by shuffle tree, warps in index order, CTAs in rank order through distributed
// shared memory -- the same bits on every run.
template <int NP, int THREADS>
__global__ void __cluster_dims__(kBalanceCtas, 1, 1) __launch_bounds__(THREADS)
balance_stats_kernel(Dims dm, const float* __restrict__ logits, const int32_t* __restrict__ counts,
                     float* __restrict__ f, float* __restrict__ P, float* __restrict__ loss) {
  __shared__ float part[THREADS / 32][NP];  // per-warp sums of the softmax columns
  __shared__ float cta_col[NP];             // this CTA's sums, read by CTA 0 of the cluster
  __shared__ float col[NP];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint32_t rank = cluster_rank();
  const int N = dm.N;
  float acc[NP];
#pragma unroll
  for (int i = 0; i < NP; ++i) acc[i] = 0.f;
  for (long long t = (long long)rank * THREADS + tid; t < dm.T; t += (long long)kBalanceCtas * THREADS) {
    const float* row = logits + t * N;
    float g[NP];
#pragma unroll
    for (int i = 0; i < NP; ++i) g[i] = (i < N) ? __ldg(row + i) : -INFINITY;
    float m = g[0];
#pragma unroll
    for (int i = 1; i < NP; ++i) m = fmaxf(m, g[i]);
    float z = 0.f;
#pragma unroll
    for (int i = 0; i < NP; ++i) {
      g[i] = (i < N) ? expf(g[i] - m) : 0.f;
      z += g[i];
    }
    const float inv = 1.f / z;
#pragma unroll
    for (int i = 0; i < NP; ++i) acc[i] = fmaf(g[i], inv, acc[i]);
  }
#pragma unroll
  for (int i = 0; i < NP; ++i) {
    float a = acc[i];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
    if (lane == 0) part[warp][i] = a;
  }
  __syncthreads();
  if (tid < NP) {
    float s = 0.f;
    for (int w = 0; w < THREADS / 32; ++w) s += part[w][tid];  // fixed order
    cta_col[tid] = s;
  }
  cluster_sync_all();  // every CTA's sums are in place and visible
  if (rank == 0) {
    if (tid < N) {
      float s = 0.f;
      for (uint32_t r = 0; r < (uint32_t)kBalanceCtas; ++r) s += ld_cluster_f32(&cta_col[tid], r);  // fixed order
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
  cluster_sync_all();  // no CTA leaves while its shared memory may still be read
}

}  // namespace

namespace {

// Eq. 7 differentiated with respect to the logits, f held fixed (it only counts selections):
//   d(scale L_b)/dG[t, j] = (scale / T) P_tj (c_j - sum_i c_i P_ti),  c_i = eta_i f_i.
// One warp per token, lane l holds experts l and l + 32; written to dG or added to it.
__global__ void __launch_bounds__(256)
balance_bwd_kernel(Dims dm, const float* __restrict__ logits, const float* __restrict__ f, float scale,
                   int accumulate, float* __restrict__ dG) {
  const int lane = threadIdx.x & 31, N = dm.N;
  const long long t = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (t >= dm.T) return;
  const int i0 = lane, i1 = lane + 32;
  const float g0 = i0 < N ? logits[t * N + i0] : -INFINITY, g1 = i1 < N ? logits[t * N + i1] : -INFINITY;
  float m = fmaxf(g0, g1);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  const float e0 = i0 < N ? expf(g0 - m) : 0.f, e1 = i1 < N ? expf(g1 - m) : 0.f;
  float z = e0 + e1;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
  const float P0 = e0 / z, P1 = e1 / z;
  const float c0 = i0 < N ? (i0 < dm.n_ffn ? 1.f : dm.tau) * f[i0] : 0.f;
  const float c1 = i1 < N ? (i1 < dm.n_ffn ? 1.f : dm.tau) * f[i1] : 0.f;
  float dot = c0 * P0 + c1 * P1;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);
  const float k = scale / (float)dm.T;
  if (i0 < N) {
    const float v = k * P0 * (c0 - dot);
    dG[t * N + i0] = accumulate ? dG[t * N + i0] + v : v;
  }
  if (i1 < N) {
    const float v = k * P1 * (c1 - dot);
    dG[t * N + i1] = accumulate ? dG[t * N + i1] + v : v;
  }
}

}  // namespace

cudaError_t launch_balance_backward(const Dims& d, const float* logits, const float* f, float scale, int accumulate,
                                    float* dlogits, cudaStream_t st) {
  if (d.T == 0) return cudaSuccess;
  balance_bwd_kernel<<<(unsigned)((d.T + 7) / 8), 256, 0, st>>>(d, logits, f, scale, accumulate, dlogits);
  return cudaGetLastError();
}

cudaError_t launch_balance_stats(const Dims& d, const float* logits, const int32_t* counts, float* f, float* P,
                                 float* loss, cudaStream_t st) {
  if (d.N <= 16) balance_stats_kernel<16, 1024><<<kBalanceCtas, 1024, 0, st>>>(d, logits, counts, f, P, loss);
  else if (d.N <= 32) balance_stats_kernel<32, 512><<<kBalanceCtas, 512, 0, st>>>(d, logits, counts, f, P, loss);
  else balance_stats_kernel<64, 256><<<kBalanceCtas, 256, 0, st>>>(d, logits, counts, f, P, loss);
  return cudaGetLastError();
}

}  // namespace moepp
