// Router of the MoE++ layer: logits with the gating residual (Eq. 2, Eq. 6), softmax over all N
// experts and top-K on the logits (Eq. 1), per-expert slot counts, the FFN offset table, and the
// constant experts' mixing weights (Eq. 5).  One pass over x: the router rows W_r and the constant
// experts' W_c rows are stacked into one small matrix so that x is read from HBM exactly once.
#include "common.cuh"

namespace moepp {
namespace {

constexpr int kRouteThreads = 256;
constexpr int kRouteWarps = kRouteThreads / 32;
constexpr int kChunk = 256;  // elements of D handled per pass: 8 per lane

// RT: padded number of stacked rows (N + 2*n_const rounded up); TPW: tokens per warp.
template <typename XT, int RT, int TPW>
__global__ void __launch_bounds__(kRouteThreads)
route_kernel(Dims dm, const XT* __restrict__ x, const float* __restrict__ W_r, const float* __restrict__ W_g,
             const float* __restrict__ prev, const float* __restrict__ bias, const float* __restrict__ W_c,
             float* __restrict__ logits, int32_t* __restrict__ topk_idx, float* __restrict__ topk_w,
             int32_t* __restrict__ counts, float* __restrict__ alpha) {
  extern __shared__ __align__(16) float smem[];
  float* Ws = smem;                                                    // [RT][kChunk]
  float* sums = Ws + RT * kChunk;                                      // [warps][TPW][RT]
  int* s_cnt = reinterpret_cast<int*>(sums + kRouteWarps * TPW * RT);  // [kMaxExperts]

  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int N = dm.N, D = dm.D, K = dm.K;
  const bool logits_given = (dm.flags & MOEPP_FLAG_LOGITS_GIVEN) != 0;
  const bool want_alpha = (alpha != nullptr) && dm.n_const > 0;
  const int R = N + (want_alpha ? 2 * dm.n_const : 0);  // stacked rows in use
  const int r_first = logits_given ? N : 0;             // rows below this are not needed
  const bool need_proj = r_first < R;

  if (tid < kMaxExperts) s_cnt[tid] = 0;

  const long long tok0 = ((long long)blockIdx.x * kRouteWarps + warp) * TPW;
  float acc[TPW][RT];
#pragma unroll
  for (int j = 0; j < TPW; ++j)
#pragma unroll
    for (int r = 0; r < RT; ++r) acc[j][r] = 0.f;

  if (need_proj) {
    for (int d0 = 0; d0 < D; d0 += kChunk) {
      __syncthreads();
      // stage the chunk of the stacked weight matrix (rows outside [r_first, R) are zero)
      for (int i = tid; i < RT * (kChunk / 4); i += kRouteThreads) {
        const int r = i / (kChunk / 4), c = (i % (kChunk / 4)) * 4;
        float4 w4 = make_float4(0.f, 0.f, 0.f, 0.f);
        if (r >= r_first && r < R && d0 + c < D) {
          const float* src = (r < N) ? (W_r + (size_t)r * D) : (W_c + (size_t)(r - N) * D);
          w4 = *reinterpret_cast<const float4*>(src + d0 + c);
        }
        *reinterpret_cast<float4*>(Ws + r * kChunk + c) = w4;
      }
      __syncthreads();
      const int d = d0 + lane * 8;
      if (d < D) {
        float xv[TPW][8];
#pragma unroll
        for (int j = 0; j < TPW; ++j) {
          if (tok0 + j < dm.T) {
            Vec8<XT>::load(x + (size_t)(tok0 + j) * D + d, xv[j]);
          } else {
#pragma unroll
            for (int i = 0; i < 8; ++i) xv[j][i] = 0.f;
          }
        }
#pragma unroll
        for (int r = 0; r < RT; ++r) {
          const float4 wa = *reinterpret_cast<const float4*>(Ws + r * kChunk + lane * 8);
          const float4 wb = *reinterpret_cast<const float4*>(Ws + r * kChunk + lane * 8 + 4);
#pragma unroll
          for (int j = 0; j < TPW; ++j) {
            float a = acc[j][r];
            a = fmaf(wa.x, xv[j][0], a); a = fmaf(wa.y, xv[j][1], a);
            a = fmaf(wa.z, xv[j][2], a); a = fmaf(wa.w, xv[j][3], a);
            a = fmaf(wb.x, xv[j][4], a); a = fmaf(wb.y, xv[j][5], a);
            a = fmaf(wb.z, xv[j][6], a); a = fmaf(wb.w, xv[j][7], a);
            acc[j][r] = a;
          }
        }
      }
    }
    // sum the per-lane partials; lane (r mod 32) keeps row r
#pragma unroll
    for (int j = 0; j < TPW; ++j)
#pragma unroll
      for (int r = 0; r < RT; ++r) {
        float a = acc[j][r];
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
        if (lane == (r & 31)) sums[(warp * TPW + j) * RT + r] = a;
      }
  }
  __syncthreads();  // s_cnt zeroed, sums visible

  // ---- per token: residual + bias, softmax over all N, top-K on the logits, Eq. 5 weights -------
  for (int j = 0; j < TPW; ++j) {
    const long long t = tok0 + j;
    if (t >= dm.T) break;  // warp-uniform
    const float* s = sums + (warp * TPW + j) * RT;
    float g[2];
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int e = lane + 32 * h;
      g[h] = -INFINITY;
      if (e < N) {
        float val;
        if (logits_given) {
          val = logits[t * N + e];
        } else {
          val = s[e];
          if (W_g != nullptr) {
            float r = 0.f;
            for (int q = 0; q < N; ++q) r = fmaf(__ldg(W_g + e * N + q), __ldg(prev + t * N + q), r);
            val += r;
          }
          if (bias != nullptr) val += __ldg(bias + e);
          logits[t * N + e] = val;
        }
        g[h] = val;
      }
    }
    float m = fmaxf(g[0], g[1]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
    float p[2];
    p[0] = (lane < N) ? expf(g[0] - m) : 0.f;
    p[1] = (lane + 32 < N) ? expf(g[1] - m) : 0.f;
    float z = p[0] + p[1];
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) z += __shfl_xor_sync(0xffffffffu, z, o);
    p[0] = p[0] / z;
    p[1] = p[1] / z;

    float wk[kMaxTopK];
    int ik[kMaxTopK];
    float wsum = 0.f;
#pragma unroll
    for (int k = 0; k < kMaxTopK; ++k) {
      if (k < K) {
        // this lane's better candidate: larger logit, the lower index on ties
        float bv = g[0];
        int bi = lane;
        if (g[1] > g[0]) { bv = g[1]; bi = lane + 32; }
        if (bi >= N) bv = -INFINITY;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
          const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
          const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
          if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
        }
        const float pw = __shfl_sync(0xffffffffu, (bi >= 32) ? p[1] : p[0], bi & 31);
        ik[k] = bi;
        wk[k] = pw;
        wsum += pw;
        if ((bi & 31) == lane) g[bi >> 5] = -INFINITY;  // taken
      }
    }
    if (lane == 0) {
#pragma unroll
      for (int k = 0; k < kMaxTopK; ++k)
        if (k < K) {
          topk_idx[t * K + k] = ik[k];
          topk_w[t * K + k] = dm.renorm ? wk[k] / wsum : wk[k];
          atomicAdd(&s_cnt[ik[k]], 1);
        }
    }
    if (want_alpha && lane < dm.n_const) {
      const float z0 = s[N + 2 * lane], z1 = s[N + 2 * lane + 1];
      const float mm = fmaxf(z0, z1);
      const float e0 = expf(z0 - mm), e1 = expf(z1 - mm);
      const float inv = 1.f / (e0 + e1);
      alpha[(t * dm.n_const + lane) * 2 + 0] = e0 * inv;
      alpha[(t * dm.n_const + lane) * 2 + 1] = e1 * inv;
    }
  }
  __syncthreads();
  if (tid < N && s_cnt[tid] != 0) atomicAdd(&counts[tid], s_cnt[tid]);
}

// offsets[e] = first row of FFN expert e; every segment is its served count rounded up to row_align.
__global__ void route_offsets_kernel(const int32_t* __restrict__ counts, int32_t* __restrict__ offsets, int n_ffn,
                                     int row_align, int cap_ffn) {
  if (threadIdx.x == 0 && blockIdx.x == 0) {
    int run = 0;
    offsets[0] = 0;
    for (int e = 0; e < n_ffn; ++e) {
      const int served = counts[e] < cap_ffn ? counts[e] : cap_ffn;  // Eq. 8: a full expert serves no more
      run += (served + row_align - 1) / row_align * row_align;
      offsets[e + 1] = run;
    }
  }
}

template <typename XT, int RT, int TPW>
cudaError_t launch_route_t(const Dims& d, const void* x, const float* W_r, const float* W_g, const float* prev,
                           const float* bias, const float* W_c, float* logits, int32_t* topk_idx, float* topk_w,
                           int32_t* counts, float* alpha, cudaStream_t st) {
  const size_t smem =
      sizeof(float) * ((size_t)RT * kChunk + (size_t)kRouteWarps * TPW * RT) + sizeof(int) * kMaxExperts;
  auto kern = route_kernel<XT, RT, TPW>;
  cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (err != cudaSuccess) return err;
  const int tokens_per_block = kRouteWarps * TPW;
  const unsigned grid = (unsigned)((d.T + tokens_per_block - 1) / tokens_per_block);
  kern<<<grid, kRouteThreads, smem, st>>>(d, static_cast<const XT*>(x), W_r, W_g, prev, bias, W_c, logits, topk_idx,
                                          topk_w, counts, alpha);
  return cudaGetLastError();
}

template <typename XT>
cudaError_t launch_route_x(const Dims& d, int R, const void* x, const float* W_r, const float* W_g,
                           const float* prev, const float* bias, const float* W_c, float* logits, int32_t* topk_idx,
                           float* topk_w, int32_t* counts, float* alpha, cudaStream_t st) {
#define MOEPP_ROUTE_CASE(RT, TPW)                                                                                 \
  if (R <= RT)                                                                                                    \
    return launch_route_t<XT, RT, TPW>(d, x, W_r, W_g, prev, bias, W_c, logits, topk_idx, topk_w, counts, alpha, \
                                       st);
  MOEPP_ROUTE_CASE(8, 4)
  MOEPP_ROUTE_CASE(16, 4)
  MOEPP_ROUTE_CASE(24, 4)
  MOEPP_ROUTE_CASE(32, 2)
  MOEPP_ROUTE_CASE(64, 2)
  MOEPP_ROUTE_CASE(128, 1)
#undef MOEPP_ROUTE_CASE
  return cudaErrorInvalidValue;
}

}  // namespace

cudaError_t launch_route(const Dims& d, const void* x, const float* W_r, const float* W_g, const float* prev,
                         const float* bias, const float* W_c, float* logits, int32_t* topk_idx, float* topk_w,
                         int32_t* counts, int32_t* offsets, float* alpha, cudaStream_t st) {
  cudaError_t err = cudaMemsetAsync(counts, 0, sizeof(int32_t) * d.N, st);
  if (err != cudaSuccess) return err;
  bool done = false;
  if (d.T > 0) {  // bf16 activations: projection on the tensor cores
    err = launch_route_tc(d, x, W_r, W_g, prev, bias, W_c, logits, topk_idx, topk_w, counts,
                          d.n_const > 0 ? alpha : nullptr, st);
    if (err == cudaSuccess) done = true;
    else if (err != cudaErrorNotSupported) return err;
  }
  if (d.T > 0 && !done) {
    const int R = d.N + ((alpha != nullptr) ? 2 * d.n_const : 0);
    err = (d.dtype == MOEPP_BF16)
              ? launch_route_x<__nv_bfloat16>(d, R, x, W_r, W_g, prev, bias, W_c, logits, topk_idx, topk_w, counts,
                                              alpha, st)
              : launch_route_x<float>(d, R, x, W_r, W_g, prev, bias, W_c, logits, topk_idx, topk_w, counts, alpha,
                                      st);
    if (err != cudaSuccess) return err;
  }
  route_offsets_kernel<<<1, 32, 0, st>>>(counts, offsets, d.n_ffn, d.row_align, d.cap_ffn);
  return cudaGetLastError();
}

}  // namespace moepp
