// Router of the MoE++ layer for bf16 activations, with the projection on the tensor cores.
//
// logits (Eq. 2, Eq. 6) need x . W^T for the N router rows and the 2*n_const rows of the constant
// experts' W_c (Eq. 5): a [T, D] x [D, R] product with R <= 128.  On CUDA cores that product costs more
// than reading x from HBM, so it runs as tcgen05 MMAs instead.  To keep the router in float, every
// float weight is split on the fly into three bf16 terms w = hi + mid + lo (each remainder is exact in
// float, so the three terms carry all 24 mantissa bits); x is bf16 already, every product is exact and
// the accumulation is float in tensor memory.
//
// One CTA per 128 tokens.  warp 0: TMA producer of x tiles (128 tokens x 64 k, 128-byte swizzle);
// warps 1-4: convert the matching 64-wide slice of the stacked weights into three bf16 operand tiles
// in shared memory (written directly in the swizzled K-major layout the MMA expects), then run the
// per-token epilogue; warp 5: allocates tensor memory and issues the MMAs (three per k-step, one per
// weight term, all accumulating into the same R columns).  Epilogue, one thread per token: gating
// residual and bias, softmax over all N experts, top-K on the logits with the lower index winning ties
// (Eq. 1), the constant experts' mixing weights, per-expert slot counts.
#include "common.cuh"
#include "tc_common.cuh"

namespace moepp {
namespace {

constexpr int kTileTokens = 128;
constexpr int kBK = 64;
constexpr int kThreadsR = 192;
constexpr int kABytesR = kTileTokens * kBK * 2;

template <int RP>
struct RouteTcSmem {
  static constexpr int kBSub = RP * 128;  // one weight term: RP rows of 64 bf16
  static constexpr int kStage = kABytesR + 3 * kBSub;
  static constexpr int kStages = (RP == 32) ? 3 : 2;  // 40 / 64 KiB per stage for 64 / 128 stacked rows
  static constexpr int kRing = kStages * kStage;
};

__device__ __forceinline__ void named_barrier_128() { asm volatile("bar.sync 1, 128;" ::: "memory"); }

template <int RP>
__global__ void __launch_bounds__(kThreadsR, RP <= 64 ? 2 : 1)
route_tc_kernel(const __grid_constant__ CUtensorMap tmX, Dims dm, const float* __restrict__ W_r,
                const float* __restrict__ W_g, const float* __restrict__ prev, const float* __restrict__ bias,
                const float* __restrict__ W_c, float* __restrict__ logits, int32_t* __restrict__ topk_idx,
                float* __restrict__ topk_w, int32_t* __restrict__ counts, float* __restrict__ alpha,
                int32_t* err_word) {
  using L = RouteTcSmem<RP>;
  constexpr int kStagesR = L::kStages;
  constexpr uint32_t kIdesc = umma_idesc_bf16(kTileTokens, RP);
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_full[kStagesR], bar_empty[kStagesR], bar_tmem_full, bar_drain;
  __shared__ uint32_t tmem_base_slot;
  __shared__ int s_cnt[kMaxExperts];
  __shared__ volatile int abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int N = dm.N, D = dm.D, K = dm.K;
  const bool want_alpha = (alpha != nullptr) && dm.n_const > 0;
  const int R = N + (want_alpha ? 2 * dm.n_const : 0);
  const int KB = (D + kBK - 1) / kBK;
  const long long t0 = (long long)blockIdx.x * kTileTokens;
  const int rows = (int)((dm.T - t0 < kTileTokens) ? (dm.T - t0) : kTileTokens);

  const uint32_t ring = (smem_u32(smem_raw) + 1023u) & ~1023u;
  uint8_t* ring_ptr = smem_raw + (ring - smem_u32(smem_raw));
  float* s_prev = reinterpret_cast<float*>(ring_ptr + L::kRing);  // [128][N + 1]
  float* s_Wg = s_prev + kTileTokens * (N + 1);                   // [N][N]
  float* s_bias = s_Wg + N * N;                                   // [N]

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < kStagesR; ++s) {
      mbar_init(smem_u32(&bar_full[s]), 1 + 128);  // the producer's expect_tx arrival + 128 converter threads
      mbar_init(smem_u32(&bar_empty[s]), 1);
    }
    mbar_init(smem_u32(&bar_tmem_full), 1);
    mbar_init(smem_u32(&bar_drain), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (threadIdx.x < kMaxExperts) s_cnt[threadIdx.x] = 0;
  if (warp == 5) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                 "r"(RP)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;

  if (warp == 0) {
    // ------------------------------ TMA producer: x tiles ---------------------------------------
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tmX) : "memory");
      int kb = 0;
      bool ok = true;
      for (; kb < KB; ++kb) {
        const uint32_t s = kb % kStagesR, ph = (kb / kStagesR) & 1u;
        if (!mbar_wait(smem_u32(&bar_empty[s]), ph ^ 1u, &abort_flag, 11, err_word)) { ok = false; break; }
        const uint32_t full = smem_u32(&bar_full[s]);
        mbar_expect_tx(full, kABytesR);
        tma_load_2d(ring + s * L::kStage, &tmX, kb * kBK, (int)t0, full);
      }
      if (!ok) {
        const int n_back = kb < kStagesR ? kb : kStagesR;
        for (int i = 1; i <= n_back; ++i) {
          const int j = kb - i;
          const uint32_t s = j % kStagesR, ph = (j / kStagesR) & 1u;
          for (int spin = 0; spin < 100000 && !mbar_try_wait(smem_u32(&bar_full[s]), ph); ++spin) __nanosleep(64);
        }
      }
    }
  } else if (warp == 5) {
    // ------------------------------ MMA issuer ----------------------------------------------------
    if (lane == 0) {
      bool ok = true;
      for (int kb = 0; kb < KB; ++kb) {
        const uint32_t s = kb % kStagesR, ph = (kb / kStagesR) & 1u;
        if (!mbar_wait(smem_u32(&bar_full[s]), ph, &abort_flag, 12, err_word)) { ok = false; break; }
        tc_fence_after();
        const uint32_t a_addr = ring + s * L::kStage, b_addr = a_addr + kABytesR;
        const uint64_t adesc = make_smem_desc(a_addr);
#pragma unroll
        for (int k = 0; k < kBK / 16; ++k) {
#pragma unroll
          for (int sp = 0; sp < 3; ++sp) {
            const uint64_t bdesc = make_smem_desc(b_addr + sp * L::kBSub);
            umma_bf16(tmem_base, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), kIdesc,
                      (kb | k | sp) != 0 ? 1u : 0u);
          }
        }
        umma_commit(smem_u32(&bar_empty[s]));
      }
      if (ok) {
        umma_commit(smem_u32(&bar_tmem_full));
      } else {
        umma_commit(smem_u32(&bar_drain));
        for (int spin = 0; spin < 100000 && !mbar_try_wait(smem_u32(&bar_drain), 0); ++spin) __nanosleep(64);
      }
    }
  } else {
    // ------------------------------ weight conversion, then the per-token epilogue ---------------
    const int tid_e = threadIdx.x - 32;  // 0..127
    // gating-residual operands of this tile (read again only by these 128 threads)
    if (W_g != nullptr) {
      for (int i = tid_e; i < N * N; i += 128) s_Wg[i] = W_g[i];
      for (int i = tid_e; i < rows * N; i += 128) s_prev[(i / N) * (N + 1) + (i % N)] = prev[t0 * N + i];
    }
    if (bias != nullptr)
      for (int i = tid_e; i < N; i += 128) s_bias[i] = bias[i];

    // Each thread owns CH 16-byte chunks (8 consecutive k of one stacked row) of every 64-wide slice.  The float
    // weights are fetched two slices ahead of their use, so that one L2 round trip is spread over two k steps
    // (with one slice of lookahead the loop ran at one L2 latency per step, twice the time x needs from HBM).
    constexpr int CH = RP * 8 / 128;
    constexpr int PF = 2;
    float wv[PF][CH][8];
    auto fetch = [&](int kb, float (&w)[CH][8]) {
#pragma unroll
      for (int j = 0; j < CH; ++j) {
        const int c = tid_e + j * 128, n = c >> 3, k0 = kb * kBK + (c & 7) * 8;
#pragma unroll
        for (int i = 0; i < 8; ++i) w[j][i] = 0.f;
        if (kb < KB && n < R && k0 < D) {
          const float* src = ((n < N) ? (W_r + (size_t)n * D) : (W_c + (size_t)(n - N) * D)) + k0;
          const float4 a = __ldg(reinterpret_cast<const float4*>(src));
          const float4 b = __ldg(reinterpret_cast<const float4*>(src + 4));
          w[j][0] = a.x; w[j][1] = a.y; w[j][2] = a.z; w[j][3] = a.w;
          w[j][4] = b.x; w[j][5] = b.y; w[j][6] = b.z; w[j][7] = b.w;
        }
      }
    };
#pragma unroll
    for (int u = 0; u < PF; ++u) fetch(u, wv[u]);
    bool ok = true;
    for (int kb0 = 0; kb0 < KB && ok; kb0 += PF) {
#pragma unroll
      for (int u = 0; u < PF; ++u) {
        const int kb = kb0 + u;
        if (kb >= KB || !ok) break;
        const uint32_t s = kb % kStagesR, ph = (kb / kStagesR) & 1u;
        if (!mbar_wait(smem_u32(&bar_empty[s]), ph ^ 1u, &abort_flag, 13, err_word)) { ok = false; break; }
        uint8_t* bbase = ring_ptr + s * L::kStage + kABytesR;
#pragma unroll
        for (int j = 0; j < CH; ++j) {
          const int c = tid_e + j * 128, n = c >> 3, kc = c & 7;
          float hi[8], mid[8], lo[8];
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            hi[i] = __bfloat162float(__float2bfloat16_rn(wv[u][j][i]));
            const float r1 = wv[u][j][i] - hi[i];  // exact
            mid[i] = __bfloat162float(__float2bfloat16_rn(r1));
            lo[i] = r1 - mid[i];                   // exact; rounded to bf16 when packed
          }
          const int off = (n >> 3) * 1024 + (n & 7) * 128 + ((kc ^ (n & 7)) << 4);
          *reinterpret_cast<uint4*>(bbase + off) = make_uint4(pack_bf16(hi[0], hi[1]), pack_bf16(hi[2], hi[3]),
                                                              pack_bf16(hi[4], hi[5]), pack_bf16(hi[6], hi[7]));
          *reinterpret_cast<uint4*>(bbase + L::kBSub + off) =
              make_uint4(pack_bf16(mid[0], mid[1]), pack_bf16(mid[2], mid[3]), pack_bf16(mid[4], mid[5]),
                         pack_bf16(mid[6], mid[7]));
          *reinterpret_cast<uint4*>(bbase + 2 * L::kBSub + off) =
              make_uint4(pack_bf16(lo[0], lo[1]), pack_bf16(lo[2], lo[3]), pack_bf16(lo[4], lo[5]),
                         pack_bf16(lo[6], lo[7]));
        }
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic-proxy writes -> visible to the MMA
        mbar_arrive(smem_u32(&bar_full[s]));
        fetch(kb + PF, wv[u]);
      }
    }
    if (ok) ok = mbar_wait(smem_u32(&bar_tmem_full), 0, &abort_flag, 14, err_word);
    named_barrier_128();
    const bool go = (abort_flag == 0);  // the same answer in all 128 threads
    if (go) {
      tc_fence_after();
      // all MMAs have retired: the ring is free and becomes the [128][RP + 1] staging of the sums
      float* s_log = reinterpret_cast<float*>(ring_ptr);
      const int q = warp & 3;
      const int r = q * 32 + lane;  // token row of this thread = its TMEM lane
      float* row = s_log + r * (RP + 1);
#pragma unroll 1
      for (int c = 0; c < RP; c += 16) {
        uint32_t v[16];
        tmem_ld16(tmem_base + ((uint32_t)(q * 32) << 16) + c, v);
        tmem_ld_wait();
        tmem_ld_pin(v);
#pragma unroll
        for (int i = 0; i < 16; ++i) row[c + i] = __uint_as_float(v[i]);
      }
      tc_fence_before();
      const long long t = t0 + r;
      const bool live = r < rows;
      if (live) {
        for (int e = 0; e < N; ++e) {
          float val = row[e];
          if (W_g != nullptr) {
            float a = 0.f;
            for (int j = 0; j < N; ++j) a = fmaf(s_Wg[e * N + j], s_prev[r * (N + 1) + j], a);
            val += a;
          }
          if (bias != nullptr) val += s_bias[e];
          row[e] = val;
        }
      }
      named_barrier_128();
      // the tile's logits are contiguous in global memory: coalesced copy
      for (int i = tid_e; i < rows * N; i += 128) logits[t0 * N + i] = s_log[(i / N) * (RP + 1) + (i % N)];
      if (live) {
        float m = row[0];
        for (int e = 1; e < N; ++e) m = fmaxf(m, row[e]);
        float z = 0.f;
        for (int e = 0; e < N; ++e) z += expf(row[e] - m);
        unsigned long long taken = 0ull;
        float wk[kMaxTopK];
        float wsum = 0.f;
#pragma unroll
        for (int k = 0; k < kMaxTopK; ++k) {
          wk[k] = 0.f;
          if (k < K) {
            int best = -1;
            float bv = 0.f;
            for (int e = 0; e < N; ++e) {
              if ((taken >> e) & 1ull) continue;
              const float val = row[e];
              if (best < 0 || val > bv) { best = e; bv = val; }  // strict '>' keeps the lower index on ties
            }
            taken |= 1ull << best;
            wk[k] = expf(bv - m) / z;
            wsum += wk[k];
            topk_idx[t * K + k] = best;
            atomicAdd(&s_cnt[best], 1);
          }
        }
#pragma unroll
        for (int k = 0; k < kMaxTopK; ++k)
          if (k < K) topk_w[t * K + k] = dm.renorm ? wk[k] / wsum : wk[k];
        if (want_alpha) {
          for (int qc = 0; qc < dm.n_const; ++qc) {
            const float z0 = row[N + 2 * qc], z1 = row[N + 2 * qc + 1];
            const float mm = fmaxf(z0, z1);
            const float e0 = expf(z0 - mm), e1 = expf(z1 - mm);
            const float inv = 1.f / (e0 + e1);
            alpha[(t * dm.n_const + qc) * 2 + 0] = e0 * inv;
            alpha[(t * dm.n_const + qc) * 2 + 1] = e1 * inv;
          }
        }
      }
      named_barrier_128();
      if (tid_e < N && s_cnt[tid_e] != 0) atomicAdd(&counts[tid_e], s_cnt[tid_e]);
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 5) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(RP) : "memory");
  }
}

template <int RP>
cudaError_t launch_rp(const CUtensorMap& tmX, const Dims& d, const float* W_r, const float* W_g, const float* prev,
                      const float* bias, const float* W_c, float* logits, int32_t* topk_idx, float* topk_w,
                      int32_t* counts, float* alpha, int32_t* err_word, cudaStream_t st) {
  const size_t extra = sizeof(float) * ((size_t)kTileTokens * (d.N + 1) + (size_t)d.N * d.N + d.N);
  const size_t smem = 1024 + RouteTcSmem<RP>::kRing + extra;
  auto kern = route_tc_kernel<RP>;
  cudaError_t err = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
  if (err != cudaSuccess) return err;
  const unsigned grid = (unsigned)((d.T + kTileTokens - 1) / kTileTokens);
  kern<<<grid, kThreadsR, smem, st>>>(tmX, d, W_r, W_g, prev, bias, W_c, logits, topk_idx, topk_w, counts, alpha,
                                      err_word);
  return cudaGetLastError();
}

}  // namespace

// Returns cudaErrorNotSupported when this path does not apply (the caller then uses the FMA kernel).
cudaError_t launch_route_tc(const Dims& d, const void* x, const float* W_r, const float* W_g, const float* prev,
                            const float* bias, const float* W_c, float* logits, int32_t* topk_idx, float* topk_w,
                            int32_t* counts, float* alpha, cudaStream_t st) {
  if (d.dtype != MOEPP_BF16 || (d.flags & MOEPP_FLAG_LOGITS_GIVEN) || d.T <= 0) return cudaErrorNotSupported;
  int32_t* err_word = device_error_word();
  CUtensorMap tmX;
  if (err_word == nullptr || !make_bf16_tile_map(&tmX, x, (uint64_t)d.T, (uint64_t)d.D, kTileTokens))
    return cudaErrorNotSupported;
  const int R = d.N + ((alpha != nullptr) ? 2 * d.n_const : 0);
  if (R <= 32) return launch_rp<32>(tmX, d, W_r, W_g, prev, bias, W_c, logits, topk_idx, topk_w, counts, alpha, err_word, st);
  if (R <= 64) return launch_rp<64>(tmX, d, W_r, W_g, prev, bias, W_c, logits, topk_idx, topk_w, counts, alpha, err_word, st);
  if (R <= 128) return launch_rp<128>(tmX, d, W_r, W_g, prev, bias, W_c, logits, topk_idx, topk_w, counts, alpha, err_word, st);
  return cudaErrorNotSupported;
}

}  // namespace moepp
