// Backward pass of the layer outside the expert GEMMs: the chain rule through the combine (Eq. 1, Eq. 3-5), the
// gate (Eq. 1) and the router with its gating residual (Eq. 2, Eq. 6), with the picks held fixed.
//   combine_bwd : per token, dL/dE_k = w_k dy scattered to the grouped rows, dL/dw_k = <dy, E_k(x)>, the
//                 coefficient of dy that flows straight to x, and the constant experts' mixing gradients
//   gate_bwd    : dL/dG through the softmax over all N experts (and the optional renormalisation), plus the
//                 gradient the next layer sends back through its gating residual; dL/dG_prev = dG W_g
//   token_outer : sum over tokens of a[t, :]^T b[t, :] in fixed chunks (deterministic two-stage reduction),
//                 used for dW_r, dW_c, dW_g, dv
//   dx_assemble : dx = cx dy + [dG | dz] [W_r ; W_c] + the K grouped rows of dXp
#include "common.cuh"

namespace moepp {
namespace {

constexpr int kWarpsPerBlock = 8;

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// One warp per token.
//   dYp[row_k, :] = w_k dy            (FFN picks that were kept)
//   dw[t, k]      = <dy, E_k(x)>      (0 for zero experts and dropped slots)
//   cx[t]         = residual + sum of w_k over copy picks + sum of w_k a1 over constant picks
//   cvq[t, q]     = w_k a2 for the constant expert q the token picked, else 0
//   dGz[t, N + 2q + j] = dL/dz_j of constant expert q's mixing logits, else 0
template <typename XT>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
combine_bwd_kernel(Dims dm, int R, const XT* __restrict__ x, const XT* __restrict__ dy,
                   const XT* __restrict__ y_perm, const int32_t* __restrict__ topk_idx,
                   const float* __restrict__ topk_w, const int32_t* __restrict__ row_of_slot,
                   const float* __restrict__ alpha, const float* __restrict__ v, XT* __restrict__ dYp,
                   float* __restrict__ dw, float* __restrict__ cx_out, float* __restrict__ cvq,
                   float* __restrict__ dGz) {
  const int lane = threadIdx.x & 31;
  const long long t = (long long)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
  if (t >= dm.T) return;
  const int K = dm.K, D = dm.D, N = dm.N;
  const int zero0 = dm.zero0(), copy0 = dm.copy0(), const0 = dm.const0();
  const XT* xt = x + (size_t)t * D;
  const XT* dyt = dy + (size_t)t * D;

  for (int i = lane; i < 2 * dm.n_const; i += 32) dGz[t * R + N + i] = 0.f;
  for (int i = lane; i < dm.n_const; i += 32) cvq[t * dm.n_const + i] = 0.f;
  __syncwarp();

  float cx = dm.add_residual ? 1.f : 0.f;
  float dyx = 0.f;
  bool have_dyx = false;
  for (int k = 0; k < K; ++k) {
    const int e = topk_idx[t * K + k];
    const float g = topk_w[t * K + k];
    const int row = row_of_slot[t * K + k];
    float dwk = 0.f;
    if (row == -2 || (e >= zero0 && e < copy0)) {
      // dropped (Eq. 8) or a zero expert (Eq. 3): nothing flows
    } else if (e < zero0) {
      float acc = 0.f;
      for (int d = lane * 8; d < D; d += 256) {
        float dv8[8], yv[8], o[8];
        Vec8<XT>::load(dyt + d, dv8);
        Vec8<XT>::load(y_perm + (size_t)row * D + d, yv);
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          acc = fmaf(dv8[i], yv[i], acc);
          o[i] = g * dv8[i];
        }
        Vec8<XT>::store(dYp + (size_t)row * D + d, o);
      }
      dwk = warp_sum(acc);
    } else {
      if (!have_dyx) {
        float acc = 0.f;
        for (int d = lane * 8; d < D; d += 256) {
          float dv8[8], xv[8];
          Vec8<XT>::load(dyt + d, dv8);
          Vec8<XT>::load(xt + d, xv);
#pragma unroll
          for (int i = 0; i < 8; ++i) acc = fmaf(dv8[i], xv[i], acc);
        }
        dyx = warp_sum(acc);
        have_dyx = true;
      }
      if (e < const0) {  // Eq. 4
        dwk = dyx;
        cx += g;
      } else {  // Eq. 5
        const int q = e - const0;
        const float a1 = alpha[(t * dm.n_const + q) * 2 + 0], a2 = alpha[(t * dm.n_const + q) * 2 + 1];
        float acc = 0.f;
        for (int d = lane * 8; d < D; d += 256) {
          float dv8[8];
          Vec8<XT>::load(dyt + d, dv8);
#pragma unroll
          for (int i = 0; i < 8; ++i) acc = fmaf(dv8[i], __ldg(v + (size_t)q * D + d + i), acc);
        }
        const float dyv = warp_sum(acc);
        dwk = a1 * dyx + a2 * dyv;
        const float da1 = g * dyx, da2 = g * dyv, mean = a1 * da1 + a2 * da2;
        cx += g * a1;
        if (lane == 0) {
          cvq[t * dm.n_const + q] = g * a2;
          dGz[t * R + N + 2 * q + 0] = a1 * (da1 - mean);
          dGz[t * R + N + 2 * q + 1] = a2 * (da2 - mean);
        }
      }
    }
    if (lane == 0) dw[t * K + k] = dwk;
  }
  if (lane == 0) cx_out[t] = cx;
}

// Grouped rows no slot owns (padding up to row_align) get a zero gradient, so they add nothing to the GEMMs.
template <typename XT>
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
zero_pad_rows_kernel(const int32_t* __restrict__ slot_of_row, const int32_t* __restrict__ offsets, int n_ffn, int D,
                     XT* __restrict__ dYp) {
  const int lane = threadIdx.x & 31;
  const long long row = (long long)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
  if (row >= offsets[n_ffn] || slot_of_row[row] >= 0) return;
  const float z[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
  for (int d = lane * 8; d < D; d += 256) Vec8<XT>::store(dYp + (size_t)row * D + d, z);
}

// One warp per token; lane l holds experts l and l + 32.
//   P = softmax(logits[t, :]);  w_k = P[idx_k] (/ S, the sum over the picks, if renormalised)
//   dP[idx_k] = dw_k                      or (dw_k - sum_j dw_j w_j) / S when renormalised
//   dG = P (dP - <dP, P>) + dlogits_next;  dprev = dG W_g
__global__ void __launch_bounds__(kWarpsPerBlock * 32)
gate_bwd_kernel(Dims dm, int R, const float* __restrict__ logits, const int32_t* __restrict__ topk_idx,
                const float* __restrict__ topk_w, const float* __restrict__ dw,
                const float* __restrict__ dlogits_next, const float* __restrict__ W_g, float* __restrict__ dGz,
                float* __restrict__ dprev) {
  extern __shared__ float s_Wg[];  // [N, N] when W_g is given
  const int N = dm.N, K = dm.K;
  if (W_g != nullptr) {
    for (int i = threadIdx.x; i < N * N; i += blockDim.x) s_Wg[i] = W_g[i];
    __syncthreads();
  }
  const int lane = threadIdx.x & 31;
  const long long t = (long long)blockIdx.x * kWarpsPerBlock + (threadIdx.x >> 5);
  if (t >= dm.T) return;
  const int i0 = lane, i1 = lane + 32;
  const float g0 = i0 < N ? logits[t * N + i0] : -INFINITY;
  const float g1 = i1 < N ? logits[t * N + i1] : -INFINITY;
  float m = fmaxf(g0, g1);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  const float e0 = i0 < N ? expf(g0 - m) : 0.f, e1 = i1 < N ? expf(g1 - m) : 0.f;
  const float inv = 1.f / warp_sum(e0 + e1);
  const float P0 = e0 * inv, P1 = e1 * inv;

  // lane k holds pick k
  int e_l = -1;
  float dw_l = 0.f, w_l = 0.f;
  if (lane < K) {
    e_l = topk_idx[t * K + lane];
    dw_l = dw[t * K + lane];
    w_l = topk_w[t * K + lane];
  }
  float dot = 0.f, S = 1.f;
  if (dm.renorm) {
    dot = warp_sum(dw_l * w_l);
    float sp = 0.f;
    for (int k = 0; k < K; ++k) {
      const int e = __shfl_sync(0xffffffffu, e_l, k);
      sp += (e == i0 ? P0 : 0.f) + (e == i1 ? P1 : 0.f);
    }
    S = warp_sum(sp);
  }
  float dP0 = 0.f, dP1 = 0.f;
  for (int k = 0; k < K; ++k) {
    const int e = __shfl_sync(0xffffffffu, e_l, k);
    const float dk = __shfl_sync(0xffffffffu, dw_l, k);
    const float val = dm.renorm ? (dk - dot) / S : dk;
    if (e == i0) dP0 += val;
    if (e == i1) dP1 += val;
  }
  const float dotP = warp_sum(dP0 * P0 + dP1 * P1);
  float dG0 = P0 * (dP0 - dotP), dG1 = P1 * (dP1 - dotP);
  if (dlogits_next != nullptr) {
    if (i0 < N) dG0 += dlogits_next[t * N + i0];
    if (i1 < N) dG1 += dlogits_next[t * N + i1];
  }
  if (i0 < N) dGz[t * R + i0] = dG0;
  if (i1 < N) dGz[t * R + i1] = dG1;
  if (W_g != nullptr) {  // Eq. 6: G = ... + W_g G_prev
    float a0 = 0.f, a1 = 0.f;
    for (int i = 0; i < N; ++i) {
      const float gi = __shfl_sync(0xffffffffu, i < 32 ? dG0 : dG1, i & 31);
      if (i0 < N) a0 = fmaf(gi, s_Wg[i * N + i0], a0);
      if (i1 < N) a1 = fmaf(gi, s_Wg[i * N + i1], a1);
    }
    if (i0 < N) dprev[t * N + i0] = a0;
    if (i1 < N) dprev[t * N + i1] = a1;
  }
}

constexpr int kOm = 64, kOn = 64, kOk = 16;

__device__ __forceinline__ float ldf(const float* p) { return *p; }
__device__ __forceinline__ float ldf(const __nv_bfloat16* p) { return __bfloat162float(*p); }

// part[z, m, n] = sum over the tokens t of chunk z of A[t, m] * B[t, n]   (A float [T, M], B [T, Nout])
template <typename TB>
__global__ void __launch_bounds__(256)
token_outer_kernel(const float* __restrict__ A, const TB* __restrict__ B, float* __restrict__ part, int T, int M,
                   int Nout, long long a_rs, long long b_rs, int chunk) {
  __shared__ float As[kOk][kOm + 4], Bs[kOk][kOn + 4];
  const int m0 = blockIdx.x * kOm, n0 = blockIdx.y * kOn, z = blockIdx.z;
  const int t_begin = z * chunk, t_end = min(T, t_begin + chunk);
  const int tid = threadIdx.x, tx = tid & 15, ty = tid >> 4;
  float acc[4][4] = {};
  for (int t0 = t_begin; t0 < t_end; t0 += kOk) {
    __syncthreads();
    for (int i = tid; i < kOm * kOk; i += 256) {
      const int m = i % kOm, k = i / kOm;
      As[k][m] = (t0 + k < t_end && m0 + m < M) ? A[(size_t)(t0 + k) * a_rs + m0 + m] : 0.f;
    }
    for (int i = tid; i < kOn * kOk; i += 256) {
      const int n = i % kOn, k = i / kOn;
      Bs[k][n] = (t0 + k < t_end && n0 + n < Nout) ? ldf(B + (size_t)(t0 + k) * b_rs + n0 + n) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < kOk; ++kk) {
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
      if (m < M && n < Nout) part[((size_t)z * M + m) * Nout + n] = acc[i][j];
    }
}

// sum over z (in order) of part[z, i], written to out_a[i] for i < n_a and to out_b[i - n_a] after that
__global__ void __launch_bounds__(256) sum_parts_kernel(const float* __restrict__ part, float* __restrict__ out_a,
                                                        long long n_a, float* __restrict__ out_b, long long n, int Z,
                                                        int accumulate) {
  const long long i = (long long)blockIdx.x * 256 + threadIdx.x;
  if (i >= n) return;
  float s = 0.f;
  for (int z = 0; z < Z; ++z) s += part[(size_t)z * n + i];
  float* dst = i < n_a ? out_a + i : out_b + (i - n_a);
  *dst = accumulate ? *dst + s : s;
}

// out[i] = sum over tokens of A[t, i]; one block per column, fixed order of the partial sums
__global__ void __launch_bounds__(256) column_sum_kernel(const float* __restrict__ A, float* __restrict__ out, int T,
                                                         long long a_rs, int accumulate) {
  __shared__ float s[256];
  float acc = 0.f;
  for (int t = threadIdx.x; t < T; t += 256) acc += A[(size_t)t * a_rs + blockIdx.x];
  s[threadIdx.x] = acc;
  __syncthreads();
  for (int o = 128; o > 0; o >>= 1) {
    if ((int)threadIdx.x < o) s[threadIdx.x] += s[threadIdx.x + o];
    __syncthreads();
  }
  if (threadIdx.x == 0) out[blockIdx.x] = accumulate ? out[blockIdx.x] + s[0] : s[0];
}

constexpr int kDxTokens = 4;   // tokens per warp in dx_assemble
constexpr int kDxSlab = 256;   // columns per block
constexpr int kDxGroups = 4;   // groups of 32 tokens a block serves one after the other

// dx = cx dy + sum_r dGz[t, r] Wrow_r + sum over kept FFN picks of dXp[row_k, :],
// Wrow_r = W_r[r, :] for r < N and the flattened W_c rows after that.
// A block owns 256 columns (blockIdx.y) of 128 tokens (blockIdx.x): the R x 256 slab of the stacked weights is
// staged in shared memory once; the block then serves four groups of 32 tokens, each warp kDxTokens of them, a lane
// holding columns 4 lane .. 4 lane + 3 and 128 + 4 lane .. of the slab (conflict-free 16-byte shared loads).
template <typename XT>
__global__ void __launch_bounds__(kWarpsPerBlock * 32, 2)
dx_assemble_kernel(Dims dm, int R, const XT* __restrict__ dy, const float* __restrict__ cx,
                   const float* __restrict__ dGz, const float* __restrict__ W_r, const float* __restrict__ W_c,
                   const XT* __restrict__ dXp, const int32_t* __restrict__ topk_idx,
                   const int32_t* __restrict__ row_of_slot, XT* __restrict__ dx) {
  extern __shared__ __align__(16) float s_dx[];  // [R][256] weights; per warp [R][kDxTokens] coefficients
  const int lane = threadIdx.x & 31, wib = threadIdx.x >> 5;
  const int D = dm.D, N = dm.N, K = dm.K;
  const int d0 = blockIdx.y * kDxSlab;
  float* s_w = s_dx;
  float* s_c = s_dx + (size_t)R * kDxSlab + (size_t)wib * R * kDxTokens;
  for (int i = threadIdx.x; i < R * (kDxSlab / 4); i += kWarpsPerBlock * 32) {
    const int r = i / (kDxSlab / 4), c4 = (i % (kDxSlab / 4)) * 4;
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (d0 + c4 < D) {
      const float* wrow = r < N ? W_r + (size_t)r * D : W_c + (size_t)(r - N) * D;
      v = __ldg(reinterpret_cast<const float4*>(wrow + d0 + c4));
    }
    *reinterpret_cast<float4*>(s_w + (size_t)r * kDxSlab + c4) = v;
  }
  // rows of the first two picks and cx of every token this warp will serve (all groups), fetched up front
  __shared__ int s_rows[kWarpsPerBlock][kDxGroups * kDxTokens * 2];
  __shared__ float s_cx[kWarpsPerBlock][kDxGroups * kDxTokens];
  {
    const int grp = lane / (kDxTokens * 2), j = (lane / 2) % kDxTokens, k = lane & 1;
    const long long t = (((long long)blockIdx.x * kDxGroups + grp) * kWarpsPerBlock + wib) * kDxTokens + j;
    int row = -1;
    if (grp < kDxGroups && t < dm.T && k < K && topk_idx[t * K + k] < dm.n_ffn) row = row_of_slot[t * K + k];  // -2: dropped
    if (grp < kDxGroups) s_rows[wib][lane] = row;
    if (lane < kDxGroups * kDxTokens) {
      const long long tc = (((long long)blockIdx.x * kDxGroups + lane / kDxTokens) * kWarpsPerBlock + wib) * kDxTokens +
                           lane % kDxTokens;
      s_cx[wib][lane] = tc < dm.T ? cx[tc] : 0.f;
    }
  }
  __syncthreads();
  // the two 4-column groups of this lane
  const int ca = d0 + 4 * lane, cb = d0 + 128 + 4 * lane;
  const bool a_ok = ca < D, b_ok = cb < D;  // D is a multiple of 8, groups are 4-aligned
  auto load4 = [&](const XT* p, float (&v)[4]) {
    if (sizeof(XT) == 2) {
      const uint2 u = *reinterpret_cast<const uint2*>(p);
      v[0] = bf16_lo(u.x); v[1] = bf16_hi(u.x); v[2] = bf16_lo(u.y); v[3] = bf16_hi(u.y);
    } else {
      const float4 f = *reinterpret_cast<const float4*>(p);
      v[0] = f.x; v[1] = f.y; v[2] = f.z; v[3] = f.w;
    }
  };
  for (int grp = 0; grp < kDxGroups; ++grp) {
    const long long t0 = (((long long)blockIdx.x * kDxGroups + grp) * kWarpsPerBlock + wib) * kDxTokens;
    if (t0 >= dm.T) break;
    const int nt = (int)min((long long)kDxTokens, dm.T - t0);
    __syncwarp();
    for (int i = lane; i < R * kDxTokens; i += 32) {
      const int r = i / kDxTokens, j = i % kDxTokens;
      s_c[i] = j < nt ? dGz[(t0 + j) * R + r] : 0.f;
    }
    __syncwarp();
    // cx dy + the grouped rows of the kept FFN picks.  16-bit storage: the rows of dy and of the first two picks are
    // requested here as raw words and only unpacked after the weight loop, which covers their latency.
    constexpr bool kEarly = sizeof(XT) == 2;
    uint2 ra[kDxTokens][3], rb[kDxTokens][3];
    float acc[kDxTokens][8];
#pragma unroll
    for (int j = 0; j < kDxTokens; ++j) {
#pragma unroll
      for (int i = 0; i < 8; ++i) acc[j][i] = 0.f;
#pragma unroll
      for (int k = 0; k < 3; ++k) ra[j][k] = rb[j][k] = make_uint2(0u, 0u);  // bf16 zeros
      if (j < nt) {
        const int r0 = s_rows[wib][(grp * kDxTokens + j) * 2], r1 = s_rows[wib][(grp * kDxTokens + j) * 2 + 1];
        if (kEarly) {
          const XT* src = dy + (size_t)(t0 + j) * D;
          if (a_ok) ra[j][0] = *reinterpret_cast<const uint2*>(src + ca);
          if (b_ok) rb[j][0] = *reinterpret_cast<const uint2*>(src + cb);
          if (r0 >= 0) {
            src = dXp + (size_t)r0 * D;
            if (a_ok) ra[j][1] = *reinterpret_cast<const uint2*>(src + ca);
            if (b_ok) rb[j][1] = *reinterpret_cast<const uint2*>(src + cb);
          }
          if (r1 >= 0) {
            src = dXp + (size_t)r1 * D;
            if (a_ok) ra[j][2] = *reinterpret_cast<const uint2*>(src + ca);
            if (b_ok) rb[j][2] = *reinterpret_cast<const uint2*>(src + cb);
          }
        } else {
          const float c = s_cx[wib][grp * kDxTokens + j];
          float va[4] = {0.f, 0.f, 0.f, 0.f}, vb[4] = {0.f, 0.f, 0.f, 0.f};
          const XT* src = dy + (size_t)(t0 + j) * D;
          if (a_ok) load4(src + ca, va);
          if (b_ok) load4(src + cb, vb);
#pragma unroll
          for (int i = 0; i < 4; ++i) { acc[j][i] = c * va[i]; acc[j][4 + i] = c * vb[i]; }
#pragma unroll
          for (int k = 0; k < 2; ++k) {
            const int row = k ? r1 : r0;
            if (row < 0) continue;
            src = dXp + (size_t)row * D;
            if (a_ok) load4(src + ca, va);
            if (b_ok) load4(src + cb, vb);
#pragma unroll
            for (int i = 0; i < 4; ++i) { if (a_ok) acc[j][i] += va[i]; if (b_ok) acc[j][4 + i] += vb[i]; }
          }
        }
      }
    }
#pragma unroll 4
    for (int r = 0; r < R; ++r) {
      const float4 a = *reinterpret_cast<const float4*>(s_w + (size_t)r * kDxSlab + 4 * lane);
      const float4 b = *reinterpret_cast<const float4*>(s_w + (size_t)r * kDxSlab + 128 + 4 * lane);
      const float wv[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
      const float4 c0 = *reinterpret_cast<const float4*>(s_c + r * kDxTokens);
      const float cj[4] = {c0.x, c0.y, c0.z, c0.w};
#pragma unroll
      for (int j = 0; j < kDxTokens; ++j)
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[j][i] = fmaf(cj[j], wv[i], acc[j][i]);
    }
#pragma unroll
    for (int j = 0; j < kDxTokens; ++j) {
      if (j >= nt) continue;
      if (kEarly) {
        const float c = s_cx[wib][grp * kDxTokens + j];
        acc[j][0] += fmaf(c, bf16_lo(ra[j][0].x), bf16_lo(ra[j][1].x) + bf16_lo(ra[j][2].x));
        acc[j][1] += fmaf(c, bf16_hi(ra[j][0].x), bf16_hi(ra[j][1].x) + bf16_hi(ra[j][2].x));
        acc[j][2] += fmaf(c, bf16_lo(ra[j][0].y), bf16_lo(ra[j][1].y) + bf16_lo(ra[j][2].y));
        acc[j][3] += fmaf(c, bf16_hi(ra[j][0].y), bf16_hi(ra[j][1].y) + bf16_hi(ra[j][2].y));
        acc[j][4] += fmaf(c, bf16_lo(rb[j][0].x), bf16_lo(rb[j][1].x) + bf16_lo(rb[j][2].x));
        acc[j][5] += fmaf(c, bf16_hi(rb[j][0].x), bf16_hi(rb[j][1].x) + bf16_hi(rb[j][2].x));
        acc[j][6] += fmaf(c, bf16_lo(rb[j][0].y), bf16_lo(rb[j][1].y) + bf16_lo(rb[j][2].y));
        acc[j][7] += fmaf(c, bf16_hi(rb[j][0].y), bf16_hi(rb[j][1].y) + bf16_hi(rb[j][2].y));
      }
      for (int k = 2; k < K; ++k) {  // picks beyond the second
        if (topk_idx[(t0 + j) * K + k] >= dm.n_ffn) continue;
        const int row = row_of_slot[(t0 + j) * K + k];  // -2: dropped
        if (row < 0) continue;
        float va[4] = {0.f, 0.f, 0.f, 0.f}, vb[4] = {0.f, 0.f, 0.f, 0.f};
        const XT* src = dXp + (size_t)row * D;
        if (a_ok) load4(src + ca, va);
        if (b_ok) load4(src + cb, vb);
#pragma unroll
        for (int i = 0; i < 4; ++i) { acc[j][i] += va[i]; acc[j][4 + i] += vb[i]; }
      }
      XT* dst = dx + (size_t)(t0 + j) * D;
      if (sizeof(XT) == 2) {
        if (a_ok) *reinterpret_cast<uint2*>(dst + ca) = make_uint2(pack_bf16(acc[j][0], acc[j][1]), pack_bf16(acc[j][2], acc[j][3]));
        if (b_ok) *reinterpret_cast<uint2*>(dst + cb) = make_uint2(pack_bf16(acc[j][4], acc[j][5]), pack_bf16(acc[j][6], acc[j][7]));
      } else {
        if (a_ok) *reinterpret_cast<float4*>(dst + ca) = make_float4(acc[j][0], acc[j][1], acc[j][2], acc[j][3]);
        if (b_ok) *reinterpret_cast<float4*>(dst + cb) = make_float4(acc[j][4], acc[j][5], acc[j][6], acc[j][7]);
      }
    }
  }
}

constexpr int kOuterThreads = 128;

// part[z, m, n] = sum over the tokens t of chunk z of A[t, m] * B[t, n] for a SMALL M (a few dozen rows) and a wide,
// 8-aligned Nout: each thread keeps RT x 4 sums for 4 columns, the block covers 512 columns, and the rows of A
// are taken RT at a time (one pass when M <= RT; otherwise the chunk of B is read again from cache per group).
template <typename TB, int RT>
__global__ void __launch_bounds__(kOuterThreads)
token_outer_rows_kernel(const float* __restrict__ A, const TB* __restrict__ B, float* __restrict__ part, int T, int M,
                        int Nout, long long a_rs, long long b_rs, int chunk) {
  constexpr int TS = 32;  // tokens staged per trip
  constexpr int G = 8;    // tokens per group of loads in flight
  constexpr int W4 = sizeof(TB) == 2 ? 2 : 4;  // 32-bit words per 4 elements of B
  __shared__ __align__(16) float s_a[TS][RT];
  const int z = blockIdx.y, n = (blockIdx.x * kOuterThreads + threadIdx.x) * 4;
  const int t_begin = z * chunk, t_end = min(T, t_begin + chunk);
  const bool col_ok = n < Nout;  // Nout is a multiple of 4
  // raw words of B for one group of G tokens; the next group is requested before the current one is used
  auto fetch = [&](int t0, uint32_t (&raw)[G][W4]) {
#pragma unroll
    for (int j = 0; j < G; ++j) {
#pragma unroll
      for (int w = 0; w < W4; ++w) raw[j][w] = 0u;
      if (col_ok && t0 + j < t_end) {
        const TB* bp = B + (size_t)(t0 + j) * b_rs + n;
        if (W4 == 2) {
          const uint2 u = *reinterpret_cast<const uint2*>(bp);
          raw[j][0] = u.x; raw[j][1] = u.y;
        } else {
          const uint4 u = *reinterpret_cast<const uint4*>(bp);
          raw[j][0] = u.x; raw[j][1] = u.y; raw[j][W4 - 2] = u.z; raw[j][W4 - 1] = u.w;
        }
      }
    }
  };
  for (int m0 = 0; m0 < M; m0 += RT) {
    float acc[RT][4];
#pragma unroll
    for (int r = 0; r < RT; ++r) acc[r][0] = acc[r][1] = acc[r][2] = acc[r][3] = 0.f;
    uint32_t cur[G][W4], nxt[G][W4];
    fetch(t_begin, cur);
    for (int ts = t_begin; ts < t_end; ts += TS) {
      __syncthreads();
      for (int i = threadIdx.x; i < TS * RT; i += kOuterThreads) {
        const int tt = i / RT, r = i % RT;
        s_a[tt][r] = (ts + tt < t_end && m0 + r < M) ? A[(size_t)(ts + tt) * a_rs + m0 + r] : 0.f;
      }
      __syncthreads();
#pragma unroll 1
      for (int t8 = 0; t8 < TS; t8 += G) {  // not unrolled: the body is already several hundred FMAs
        fetch(ts + t8 + G, nxt);  // may reach into the next trip; beyond t_end it fetches nothing
#pragma unroll
        for (int j = 0; j < G; ++j) {
          float bv[4];
          if (W4 == 2) {
            bv[0] = bf16_lo(cur[j][0]); bv[1] = bf16_hi(cur[j][0]); bv[2] = bf16_lo(cur[j][1]); bv[3] = bf16_hi(cur[j][1]);
          } else {
            bv[0] = __uint_as_float(cur[j][0]); bv[1] = __uint_as_float(cur[j][1]);
            bv[2] = __uint_as_float(cur[j][W4 - 2]); bv[3] = __uint_as_float(cur[j][W4 - 1]);
          }
#pragma unroll
          for (int r4 = 0; r4 < RT; r4 += 4) {
            const float4 av = *reinterpret_cast<const float4*>(&s_a[t8 + j][r4]);
            const float ar[4] = {av.x, av.y, av.z, av.w};
#pragma unroll
            for (int r = 0; r < 4; ++r)
#pragma unroll
              for (int i = 0; i < 4; ++i) acc[r4 + r][i] = fmaf(ar[r], bv[i], acc[r4 + r][i]);
          }
        }
#pragma unroll
        for (int j = 0; j < G; ++j)
#pragma unroll
          for (int w = 0; w < W4; ++w) cur[j][w] = nxt[j][w];
      }
    }
    if (col_ok) {
#pragma unroll
      for (int r = 0; r < RT; ++r)
        if (m0 + r < M)
          *reinterpret_cast<float4*>(part + ((size_t)z * M + m0 + r) * Nout + n) =
              make_float4(acc[r][0], acc[r][1], acc[r][2], acc[r][3]);
    }
  }
}

}  // namespace

// Token segments of the tensor-core reductions: about four 128 x 256 tiles per SM in the grid, whole 64-token k
// tiles per segment, at most 64 segments (the kernel's segment table).
int backward_token_segments(const Dims& d, int* tokens_per_segment) {
  const int n_tiles = (d.D + 255) / 256;
  int want = (592 + n_tiles - 1) / n_tiles;
  if (want > 64) want = 64;
  int per = ((d.T + want - 1) / want + 63) / 64 * 64;
  if (per < 64) per = 64;
  if (tokens_per_segment != nullptr) *tokens_per_segment = per;
  return d.T > 0 ? (d.T + per - 1) / per : 1;
}

size_t backward_part_floats(const Dims& d) {
  const size_t R = (size_t)d.N + 2 * (size_t)d.n_const;
  const size_t widest = R * (size_t)d.D > (size_t)d.N * d.N ? R * (size_t)d.D : (size_t)d.N * d.N;
  const size_t fma = widest * (size_t)backward_token_chunks(d, nullptr);
  const size_t tc = (size_t)backward_token_segments(d, nullptr) * 128 * (size_t)d.D;
  return fma > tc ? fma : tc;
}

// Chunks of the reductions over tokens: enough of them that, with D / 512 column blocks each, about 900 CTAs are
// in the grid (two rounds of three CTAs per SM), but no chunk shorter than 64 tokens.
int backward_token_chunks(const Dims& d, int* chunk_tokens) {
  const int col_blocks = (d.D + 511) / 512;
  const int want = (888 + col_blocks - 1) / col_blocks;
  int chunk = (d.T + want - 1) / want;
  if (chunk < 64) chunk = 64;
  chunk = (chunk + 31) / 32 * 32;
  if (chunk_tokens != nullptr) *chunk_tokens = chunk;
  return d.T > 0 ? (d.T + chunk - 1) / chunk : 1;
}

namespace {

// A float factor [T, M] (M <= 64) as two bf16 terms per value: dst[t, m] = hi, dst[t, 64 + m] = lo, v = hi + lo up to
// 2^-17 relative; unused columns are zero.
__global__ void __launch_bounds__(256) split_bf16_kernel(const float* __restrict__ src, long long rs, int M, int T,
                                                         __nv_bfloat16* __restrict__ dst) {
  const long long i = (long long)blockIdx.x * 256 + threadIdx.x;
  const long long t = i >> 6;
  const int m = (int)(i & 63);
  if (t >= T) return;
  float hi = 0.f, lo = 0.f;
  if (m < M) {
    const float v = src[t * rs + m];
    hi = __bfloat162float(__float2bfloat16_rn(v));
    lo = v - hi;
  }
  dst[t * 128 + m] = __float2bfloat16_rn(hi);
  dst[t * 128 + 64 + m] = __float2bfloat16_rn(lo);
}

__global__ void token_segments_kernel(int32_t* __restrict__ segs, int T, int n_seg, int per) {
  const int i = threadIdx.x;
  if (i <= n_seg) segs[i] = min(T, i * per);
}

// out[m, n] = sum over segments (in order) of part[seg, m, n] + part[seg, 64 + m, n] for m < M, the first rows_a rows
// to out_a and the rest to out_b
__global__ void __launch_bounds__(256)
sum_split_parts_kernel(const float* __restrict__ part, float* __restrict__ out_a, int rows_a, float* __restrict__ out_b,
                       int M, int Nout, int n_seg, int accumulate) {
  const long long i = (long long)blockIdx.x * 256 + threadIdx.x;
  if (i >= (long long)M * Nout) return;
  const int m = (int)(i / Nout), n = (int)(i % Nout);
  float s = 0.f;
  for (int z = 0; z < n_seg; ++z) {
    const float* p = part + ((size_t)z * 128 + m) * Nout + n;
    s += p[0] + p[(size_t)64 * Nout];
  }
  float* dst = m < rows_a ? out_a + (size_t)m * Nout + n : out_b + (size_t)(m - rows_a) * Nout + n;
  *dst = accumulate ? *dst + s : s;
}

// The same reduction as token_outer on the tensor cores (bf16 activations, M <= 64, D wide enough to matter);
// cudaErrorNotSupported when it does not apply.
cudaError_t token_outer_tc(const Dims& d, const float* A, long long a_rs, int M, const void* B, const BackwardScratch& b,
                           float* out_a, int rows_a, float* out_b, cudaStream_t st) {
  if (d.dtype != MOEPP_BF16 || M > 64 || d.D < 256 || d.T < 1024) return cudaErrorNotSupported;
  int per;
  const int n_seg = backward_token_segments(d, &per);
  split_bf16_kernel<<<(unsigned)(((long long)d.T * 64 + 255) / 256), 256, 0, st>>>(
      A, a_rs, M, d.T, static_cast<__nv_bfloat16*>(b.split));
  cudaError_t err = cudaGetLastError();
  if (err != cudaSuccess) return err;
  token_segments_kernel<<<1, 128, 0, st>>>(b.segs, d.T, n_seg, per);
  if ((err = cudaGetLastError()) != cudaSuccess) return err;
  if ((err = launch_token_outer_tc(d, b.split, B, b.part, b.segs, n_seg, st)) != cudaSuccess) return err;
  const long long n = (long long)M * d.D;
  sum_split_parts_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(b.part, out_a, rows_a, out_b, M, d.D, n_seg,
                                                                      (d.flags & MOEPP_FLAG_ACCUM_GRADS) ? 1 : 0);
  return cudaGetLastError();
}

// out_a takes the first rows_a rows of the [M, Nout] product, out_b (if any) the rest
template <typename TB>
cudaError_t token_outer(const Dims& d, const float* A, long long a_rs, int M, const TB* B, long long b_rs, int Nout,
                        float* part, float* out_a, int rows_a, float* out_b, cudaStream_t st) {
  if (M == 0 || Nout == 0) return cudaSuccess;
  int chunk;
  const int Z = backward_token_chunks(d, &chunk);
  if (Nout % 8 == 0 && Nout >= 256 && b_rs % 8 == 0) {
    dim3 grid((unsigned)((Nout + 4 * kOuterThreads - 1) / (4 * kOuterThreads)), (unsigned)Z);
    if (M <= 8) token_outer_rows_kernel<TB, 8><<<grid, kOuterThreads, 0, st>>>(A, B, part, d.T, M, Nout, a_rs, b_rs, chunk);
    else if (M <= 16) token_outer_rows_kernel<TB, 16><<<grid, kOuterThreads, 0, st>>>(A, B, part, d.T, M, Nout, a_rs, b_rs, chunk);
    else token_outer_rows_kernel<TB, 24><<<grid, kOuterThreads, 0, st>>>(A, B, part, d.T, M, Nout, a_rs, b_rs, chunk);
  } else {
    dim3 grid((unsigned)((M + kOm - 1) / kOm), (unsigned)((Nout + kOn - 1) / kOn), (unsigned)Z);
    token_outer_kernel<TB><<<grid, 256, 0, st>>>(A, B, part, d.T, M, Nout, a_rs, b_rs, chunk);
  }
  cudaError_t err = cudaGetLastError();
  if (err != cudaSuccess) return err;
  const long long n = (long long)M * Nout;
  sum_parts_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(part, out_a, (long long)rows_a * Nout, out_b, n, Z,
                                                                (d.flags & MOEPP_FLAG_ACCUM_GRADS) ? 1 : 0);
  return cudaGetLastError();
}

template <typename XT>
cudaError_t layer_backward_t(const Dims& d, const ForwardState& fs, const moepp_weights& w, const XT* x,
                             const float* prev, const XT* dy, const float* dlogits_next, const BackwardScratch& b,
                             const moepp_grads& g, cudaStream_t st) {
  const int R = d.N + 2 * d.n_const;
  const unsigned token_blocks = (unsigned)((d.T + kWarpsPerBlock - 1) / kWarpsPerBlock);
  cudaError_t err;
  combine_bwd_kernel<XT><<<token_blocks, kWarpsPerBlock * 32, 0, st>>>(
      d, R, x, dy, static_cast<const XT*>(fs.y_perm), fs.topk_idx, fs.topk_w, fs.row_of_slot, fs.alpha, w.v,
      static_cast<XT*>(b.dYp), b.dw, b.cx, b.cvq, b.dGz);
  if ((err = cudaGetLastError()) != cudaSuccess) return err;
  if (d.n_ffn > 0 && d.M_cap > 0 && d.row_align > 1) {
    zero_pad_rows_kernel<XT><<<(unsigned)((d.M_cap + kWarpsPerBlock - 1) / kWarpsPerBlock), kWarpsPerBlock * 32, 0,
                               st>>>(fs.slot_of_row, fs.offsets, d.n_ffn, d.D, static_cast<XT*>(b.dYp));
    if ((err = cudaGetLastError()) != cudaSuccess) return err;
  }
  const size_t wg_smem = w.W_g != nullptr ? sizeof(float) * (size_t)d.N * d.N : 0;
  gate_bwd_kernel<<<token_blocks, kWarpsPerBlock * 32, wg_smem, st>>>(d, R, fs.logits, fs.topk_idx, fs.topk_w, b.dw,
                                                                       dlogits_next, w.W_g, b.dGz, g.dprev);
  if ((err = cudaGetLastError()) != cudaSuccess) return err;

  err = cudaErrorNotSupported;
  if (!(d.flags & MOEPP_FLAG_SIMT_FFN))
    err = launch_ffn_backward_tc(d, fs.x_perm, fs.offsets, w.W_gate, w.W_up, w.W_down, fs.h, b.dYp, b.gate, b.up,
                                 b.dXp, g.dW_gate, g.dW_up, g.dW_down, st, fs.gate, fs.up);
  if (err == cudaErrorNotSupported)
    err = launch_ffn_backward_simt(d, fs.x_perm, fs.offsets, w.W_gate, w.W_up, w.W_down, fs.h, b.dYp, b.gate, b.up,
                                   b.dXp, g.dW_gate, g.dW_up, g.dW_down, st, fs.gate, fs.up);
  if (err != cudaSuccess) return err;

  // router and constant-expert weights in one product: [dG | dz]^T x, rows 0..N-1 -> dW_r, the rest -> dW_c
  const bool fma_only = (d.flags & MOEPP_FLAG_SIMT_FFN) != 0;
  err = fma_only ? cudaErrorNotSupported : token_outer_tc(d, b.dGz, R, R, x, b, g.dW_r, d.N, g.dW_c, st);
  if (err == cudaErrorNotSupported) err = token_outer<XT>(d, b.dGz, R, R, x, d.D, d.D, b.part, g.dW_r, d.N, g.dW_c, st);
  if (err != cudaSuccess) return err;
  if (d.n_const > 0) {
    err = fma_only ? cudaErrorNotSupported : token_outer_tc(d, b.cvq, d.n_const, d.n_const, dy, b, g.dv, d.n_const, nullptr, st);
    if (err == cudaErrorNotSupported)
      err = token_outer<XT>(d, b.cvq, d.n_const, d.n_const, dy, d.D, d.D, b.part, g.dv, d.n_const, nullptr, st);
    if (err != cudaSuccess) return err;
  }
  if (w.W_g != nullptr && g.dW_g != nullptr) {
    if ((err = token_outer<float>(d, b.dGz, R, d.N, prev, d.N, d.N, b.part, g.dW_g, d.N, nullptr, st)) != cudaSuccess)
      return err;
  }
  if (g.dbias != nullptr) {
    column_sum_kernel<<<(unsigned)d.N, 256, 0, st>>>(b.dGz, g.dbias, d.T, R, (d.flags & MOEPP_FLAG_ACCUM_GRADS) ? 1 : 0);
    if ((err = cudaGetLastError()) != cudaSuccess) return err;
  }
  const int dx_tokens = kWarpsPerBlock * kDxTokens * kDxGroups;
  const dim3 dx_grid((unsigned)((d.T + dx_tokens - 1) / dx_tokens),
                     (unsigned)((d.D + kDxSlab - 1) / kDxSlab));
  const size_t dx_smem = sizeof(float) * ((size_t)R * kDxSlab + (size_t)kWarpsPerBlock * R * kDxTokens);
  if (dx_smem > 48 * 1024) {
    err = cudaFuncSetAttribute(dx_assemble_kernel<XT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)dx_smem);
    if (err != cudaSuccess) return err;
  }
  dx_assemble_kernel<XT><<<dx_grid, kWarpsPerBlock * 32, dx_smem, st>>>(
      d, R, dy, b.cx, b.dGz, w.W_r, w.W_c, static_cast<const XT*>(b.dXp), fs.topk_idx, fs.row_of_slot,
      static_cast<XT*>(g.dx));
  return cudaGetLastError();
}

}  // namespace

cudaError_t launch_layer_backward(const Dims& d, const ForwardState& fs, const moepp_weights& w, const void* x,
                                  const float* prev, const void* dy, const float* dlogits_next,
                                  const BackwardScratch& b, const moepp_grads& g, cudaStream_t st) {
  if (d.T == 0 && (d.flags & MOEPP_FLAG_ACCUM_GRADS)) return cudaSuccess;  // no tokens, nothing to add
  if (d.T == 0) {  // no tokens: every weight gradient is zero
    const int R2 = 2 * d.n_const;
    cudaError_t err;
    auto zero = [&](float* p, size_t n) { return (p == nullptr || n == 0) ? cudaSuccess : cudaMemsetAsync(p, 0, sizeof(float) * n, st); };
    if ((err = zero(g.dW_r, (size_t)d.N * d.D)) != cudaSuccess) return err;
    if ((err = zero(g.dW_g, (size_t)d.N * d.N)) != cudaSuccess) return err;
    if ((err = zero(g.dbias, (size_t)d.N)) != cudaSuccess) return err;
    if ((err = zero(g.dW_c, (size_t)R2 * d.D)) != cudaSuccess) return err;
    if ((err = zero(g.dv, (size_t)d.n_const * d.D)) != cudaSuccess) return err;
    return launch_ffn_backward_simt(d, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr, nullptr,
                                    nullptr, g.dW_gate, g.dW_up, g.dW_down, st);
  }
  return d.dtype == MOEPP_BF16
             ? layer_backward_t<__nv_bfloat16>(d, fs, w, static_cast<const __nv_bfloat16*>(x), prev,
                                               static_cast<const __nv_bfloat16*>(dy), dlogits_next, b, g, st)
             : layer_backward_t<float>(d, fs, w, static_cast<const float*>(x), prev, static_cast<const float*>(dy),
                                       dlogits_next, b, g, st);
}

}  // namespace moepp
