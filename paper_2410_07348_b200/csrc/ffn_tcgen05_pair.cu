// Grouped SwiGLU FFN on CTA pairs (tcgen05 cta_group::2): the same two GEMMs as ffn_tcgen05.cu,
//   GEMM 1  h[r,:]      = silu(x_perm[r,:] W_gate[e]^T) * (x_perm[r,:] W_up[e]^T)
//   GEMM 2  y_perm[r,:] = h[r,:] W_down[e]^T,
// with a 256 x 256 accumulator tile shared by the two CTAs of a cluster.  Each CTA stages its own 128
// rows of A and its own 128-row half of B (for GEMM 1: CTA 0 the W_gate rows, CTA 1 the matching W_up
// rows), so a CTA moves 32 KiB per 64-wide k step instead of 48 KiB and the ring holds 6 stages instead
// of 4.  The leader CTA's MMA thread issues tcgen05.mma.cta_group::2 (M = 256, N = 256, K = 16); each CTA
// ends up with its 128 rows x 256 columns of the accumulator in its own tensor memory and runs its own
// epilogue.  TMA loads of both CTAs complete on the leader's "full" barrier; the leader's tcgen05.commit
// arrives on the "empty" / "accumulator full" barriers of both CTAs; the epilogue warps of both CTAs
// arrive on the leader's "accumulator empty" barrier.  No multicast loads.  Every wait is bounded.
#include <cuda.h>

#include "common.cuh"
#include "tc_common.cuh"

namespace moepp {
namespace {

constexpr int BM2 = 256;       // rows per tile (both CTAs)
constexpr int BK = 64;
constexpr int UMMA_N = 256;
constexpr int kStages2 = 6;
constexpr int kHalfBytes = 128 * BK * 2;        // 16 KiB: one CTA's A rows, or its half of B
constexpr int kStageBytes2 = 2 * kHalfBytes;    // per CTA
constexpr int kThreads2 = 192;
constexpr int kTmemCols2 = 512;
constexpr int kSmemBytes2 = kStages2 * kStageBytes2 + 1024;
constexpr uint32_t kIdesc2 = umma_idesc_bf16(BM2, UMMA_N);

__device__ __forceinline__ uint32_t cluster_ctarank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
// address of the same shared-memory offset in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
  uint32_t r;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
  return r;
}
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release;\n\tbarrier.cluster.wait.acquire;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA tile load whose completion is counted on a barrier that may live in the pair's other CTA
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const CUtensorMap* tm, int c0, int c1,
                                                 uint32_t bar_cluster_addr) {
  asm volatile(
      "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], "
      "[%2];" ::"r"(dst),
      "l"(tm), "r"(bar_cluster_addr), "r"(c0), "r"(c1)
      : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc,
                                               uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
      : "memory");
}
// arrive (once the MMAs issued so far have retired) on the barrier at this offset in both CTAs of the pair
__device__ __forceinline__ void umma_commit_pair(uint32_t bar) {
  const uint16_t mask = 3;
  asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;" ::
                   "r"(bar), "h"(mask)
               : "memory");
}

__device__ __forceinline__ float silu_mul2(float g, float u) { return __fdividef(g, 1.f + __expf(-g)) * u; }

struct TileInfo2 {
  int e, row0, row_end, n0;
};

template <bool SWIGLU>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kThreads2, 1)
grouped_gemm_pair_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB0,
                         const __grid_constant__ CUtensorMap tmB1, __nv_bfloat16* __restrict__ C,
                         const int32_t* __restrict__ offsets, int n_ffn, int Nout, int Kd, int32_t* err_word,
                         __nv_bfloat16* __restrict__ G, __nv_bfloat16* __restrict__ U) {
  constexpr int BN_OUT = SWIGLU ? 128 : 256;
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_full[kStages2], bar_empty[kStages2], bar_tmem_full[2], bar_tmem_empty[2],
      bar_drain;
  __shared__ uint32_t tmem_base_slot;
  __shared__ int tile_start[kMaxExperts + 1];
  __shared__ int seg_begin[kMaxExperts + 1];
  __shared__ volatile int abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t rank = cluster_ctarank();
  const bool leader = rank == 0;
  const int pair_id = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;
  const uint32_t ring = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const int NT = (Nout + BN_OUT - 1) / BN_OUT;
  const int KB = (Kd + BK - 1) / BK;

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < kStages2; ++s) {
      mbar_init(smem_u32(&bar_full[s]), 1);   // leader: its producer's expect_tx arrival (bytes of both CTAs)
      mbar_init(smem_u32(&bar_empty[s]), 1);  // the leader's commit, delivered to both CTAs
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&bar_tmem_full[b]), 1);
      mbar_init(smem_u32(&bar_tmem_empty[b]), 8);  // leader: 4 epilogue warps of each CTA
    }
    mbar_init(smem_u32(&bar_drain), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    int run = 0;
    for (int e = 0; e < n_ffn; ++e) {
      const int b = offsets[e], en = offsets[e + 1];
      seg_begin[e] = b;
      tile_start[e] = run;
      run += ((en - b + BM2 - 1) / BM2) * NT;
    }
    seg_begin[n_ffn] = offsets[n_ffn];
    tile_start[n_ffn] = run;
  }
  if (warp == 1) {  // the same warp of both CTAs: 512 columns in each CTA's tensor memory
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                 "r"(kTmemCols2)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();  // both CTAs' barriers are initialised before anything arrives on them
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;
  const int total_tiles = tile_start[n_ffn];

  auto decode = [&](int L, int& e) -> TileInfo2 {
    while (L >= tile_start[e + 1]) ++e;
    const int local = L - tile_start[e];
    const int b = seg_begin[e], en = seg_begin[e + 1];
    const int mt = (en - b + BM2 - 1) / BM2;
    TileInfo2 ti;
    ti.e = e;
    ti.row0 = b + (local % mt) * BM2;
    ti.row_end = en;
    ti.n0 = (local / mt) * BN_OUT;
    return ti;
  };

  if (warp == 0) {
    // ---------------------------------- TMA producer (both CTAs) --------------------------------
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tmA) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tmB0) : "memory");
      if (SWIGLU) asm volatile("prefetch.tensormap [%0];" ::"l"(&tmB1) : "memory");
      const CUtensorMap* tmB = (SWIGLU && rank == 1) ? &tmB1 : &tmB0;
      uint32_t it = 0;
      int e = 0;
      bool ok = true;
      for (int L = pair_id; L < total_tiles && ok; L += n_pairs) {
        const TileInfo2 ti = decode(L, e);
        const int arow = ti.row0 + 128 * (int)rank;
        const int brow = ti.e * Nout + ti.n0 + (SWIGLU ? 0 : 128 * (int)rank);
        for (int kb = 0; kb < KB; ++kb, ++it) {
          const uint32_t s = it % kStages2, ph = (it / kStages2) & 1u;
          if (!mbar_wait(smem_u32(&bar_empty[s]), ph ^ 1u, &abort_flag, 21, err_word)) { ok = false; break; }
          const uint32_t full_local = smem_u32(&bar_full[s]);
          const uint32_t full_leader = map_to_cta(full_local, 0);
          const uint32_t a_dst = ring + s * kStageBytes2, b_dst = a_dst + kHalfBytes;
          if (leader) mbar_expect_tx(full_local, 2 * kStageBytes2);
          tma_load_2d_pair(a_dst, &tmA, kb * BK, arow, full_leader);
          tma_load_2d_pair(b_dst, tmB, kb * BK, brow, full_leader);
        }
      }
      if (!ok && leader) {  // give the copies already issued a bounded chance to land
        const uint32_t n_back = it < (uint32_t)kStages2 ? it : (uint32_t)kStages2;
        for (uint32_t i = 1; i <= n_back; ++i) {
          const uint32_t j = it - i, s = j % kStages2, ph = (j / kStages2) & 1u;
          for (int spin = 0; spin < 100000 && !mbar_try_wait(smem_u32(&bar_full[s]), ph); ++spin) __nanosleep(64);
        }
      }
    }
  } else if (warp == 1) {
    // ---------------------------------- MMA issuer (leader CTA only) ------------------------------
    if (lane == 0 && leader) {
      uint32_t it = 0, tile_iter = 0;
      bool ok = true;
      for (int L = pair_id; L < total_tiles && ok; L += n_pairs, ++tile_iter) {
        const uint32_t buf = tile_iter & 1u, tph = (tile_iter >> 1) & 1u;
        if (!mbar_wait(smem_u32(&bar_tmem_empty[buf]), tph ^ 1u, &abort_flag, 22, err_word)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * UMMA_N;
        for (int kb = 0; kb < KB; ++kb, ++it) {
          const uint32_t s = it % kStages2, ph = (it / kStages2) & 1u;
          if (!mbar_wait(smem_u32(&bar_full[s]), ph, &abort_flag, 23, err_word)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_addr = ring + s * kStageBytes2, b_addr = a_addr + kHalfBytes;
          const uint64_t adesc = make_smem_desc(a_addr), bdesc = make_smem_desc(b_addr);
#pragma unroll
          for (int k = 0; k < BK / 16; ++k)
            umma_bf16_pair(d_tmem, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), kIdesc2,
                           (kb | k) != 0 ? 1u : 0u);
          umma_commit_pair(smem_u32(&bar_empty[s]));
        }
        if (ok) umma_commit_pair(smem_u32(&bar_tmem_full[buf]));
      }
      if (!ok) {
        asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(
                         smem_u32(&bar_drain))
                     : "memory");
        for (int spin = 0; spin < 100000 && !mbar_try_wait(smem_u32(&bar_drain), 0); ++spin) __nanosleep(64);
      }
    }
  } else {
    // ---------------------------------- epilogue (both CTAs): this CTA's 128 rows ------------------
    const int q = warp & 3;
    uint32_t tile_iter = 0;
    int e = 0;
    bool ok = true;
    for (int L = pair_id; L < total_tiles && ok; L += n_pairs, ++tile_iter) {
      const TileInfo2 ti = decode(L, e);
      const uint32_t buf = tile_iter & 1u, tph = (tile_iter >> 1) & 1u;
      if (!mbar_wait(smem_u32(&bar_tmem_full[buf]), tph, &abort_flag, 24, err_word)) { ok = false; break; }
      tc_fence_after();
      const int grow = ti.row0 + 128 * (int)rank + q * 32 + lane;
      const bool row_ok = grow < ti.row_end;
      const uint32_t t_row = tmem_base + buf * UMMA_N + ((uint32_t)(q * 32) << 16);
      __nv_bfloat16* crow = C + (size_t)grow * Nout + ti.n0;
      if (SWIGLU) {
#pragma unroll 1
        for (int c = 0; c < 128; c += 16) {
          uint32_t g[16], u[16];
          tmem_ld16(t_row + c, g);
          tmem_ld16(t_row + 128 + c, u);
          tmem_ld_wait();
          tmem_ld_pin(g);
          tmem_ld_pin(u);
          uint32_t o[8];
#pragma unroll
          for (int i = 0; i < 8; ++i)
            o[i] = pack_bf16(silu_mul2(__uint_as_float(g[2 * i]), __uint_as_float(u[2 * i])),
                             silu_mul2(__uint_as_float(g[2 * i + 1]), __uint_as_float(u[2 * i + 1])));
          if (row_ok) {
            if (ti.n0 + c + 8 <= Nout) *reinterpret_cast<uint4*>(crow + c) = make_uint4(o[0], o[1], o[2], o[3]);
            if (ti.n0 + c + 16 <= Nout) *reinterpret_cast<uint4*>(crow + c + 8) = make_uint4(o[4], o[5], o[6], o[7]);
            if (G != nullptr) {  // keep the pre-activations for the backward pass
              uint32_t pg[8], pu[8];
#pragma unroll
              for (int i = 0; i < 8; ++i) {
                pg[i] = pack_bf16(__uint_as_float(g[2 * i]), __uint_as_float(g[2 * i + 1]));
                pu[i] = pack_bf16(__uint_as_float(u[2 * i]), __uint_as_float(u[2 * i + 1]));
              }
              const size_t at = (size_t)grow * Nout + ti.n0 + c;
              if (ti.n0 + c + 8 <= Nout) {
                *reinterpret_cast<uint4*>(G + at) = make_uint4(pg[0], pg[1], pg[2], pg[3]);
                *reinterpret_cast<uint4*>(U + at) = make_uint4(pu[0], pu[1], pu[2], pu[3]);
              }
              if (ti.n0 + c + 16 <= Nout) {
                *reinterpret_cast<uint4*>(G + at + 8) = make_uint4(pg[4], pg[5], pg[6], pg[7]);
                *reinterpret_cast<uint4*>(U + at + 8) = make_uint4(pu[4], pu[5], pu[6], pu[7]);
              }
            }
          }
        }
      } else {
#pragma unroll 1
        for (int c = 0; c < 256; c += 32) {
          uint32_t a[16], b[16];
          tmem_ld16(t_row + c, a);
          tmem_ld16(t_row + c + 16, b);
          tmem_ld_wait();
          tmem_ld_pin(a);
          tmem_ld_pin(b);
          uint32_t o[16];
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            o[i] = pack_bf16(__uint_as_float(a[2 * i]), __uint_as_float(a[2 * i + 1]));
            o[8 + i] = pack_bf16(__uint_as_float(b[2 * i]), __uint_as_float(b[2 * i + 1]));
          }
          if (row_ok) {
#pragma unroll
            for (int v = 0; v < 4; ++v)
              if (ti.n0 + c + 8 * v + 8 <= Nout)
                *reinterpret_cast<uint4*>(crow + c + 8 * v) =
                    make_uint4(o[4 * v], o[4 * v + 1], o[4 * v + 2], o[4 * v + 3]);
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive_cluster(map_to_cta(smem_u32(&bar_tmem_empty[buf]), 0));
    }
  }

  // Neither CTA may leave (or free tensor memory) while its partner can still read its shared memory,
  // write its tensor memory or arrive on its barriers.
  tc_fence_before();
  __syncthreads();
  cluster_sync_all();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols2) : "memory");
  }
}

}  // namespace

cudaError_t launch_ffn_tcgen05_pair(const Dims& d, const void* x_perm, const int32_t* offsets, const void* W_gate,
                                    const void* W_up, const void* W_down, void* h, void* y_perm, cudaStream_t st,
                                    void* gate_out, void* up_out) {
  if (d.T == 0 || d.n_ffn == 0 || d.M_cap == 0) return cudaSuccess;
  int dev = 0, sms = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (err != cudaSuccess) return err;
  int32_t* err_word = device_error_word();
  if (err_word == nullptr) return cudaErrorNotSupported;

  CUtensorMap mA1, mG, mU, mA2, mD;
  const uint64_t rows = (uint64_t)d.M_cap;
  if (!make_bf16_tile_map(&mA1, x_perm, rows, (uint64_t)d.D, 128) ||
      !make_bf16_tile_map(&mG, W_gate, (uint64_t)d.n_ffn * d.F, (uint64_t)d.D, 128) ||
      !make_bf16_tile_map(&mU, W_up, (uint64_t)d.n_ffn * d.F, (uint64_t)d.D, 128) ||
      !make_bf16_tile_map(&mA2, h, rows, (uint64_t)d.F, 128) ||
      !make_bf16_tile_map(&mD, W_down, (uint64_t)d.n_ffn * d.D, (uint64_t)d.F, 128))
    return cudaErrorNotSupported;

  auto k1 = grouped_gemm_pair_kernel<true>;
  auto k2 = grouped_gemm_pair_kernel<false>;
  err = cudaFuncSetAttribute(k1, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes2);
  if (err != cudaSuccess) return err;
  err = cudaFuncSetAttribute(k2, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes2);
  if (err != cudaSuccess) return err;

  // as many CTA pairs as can be resident at once (at most one CTA per SM)
  static int cached_pairs[64] = {};
  int pairs = (dev >= 0 && dev < 64) ? cached_pairs[dev] : 0;
  if (pairs == 0) {
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3((unsigned)(sms & ~1));
    lc.blockDim = dim3(kThreads2);
    lc.dynamicSmemBytes = kSmemBytes2;
    cudaLaunchAttribute at;
    at.id = cudaLaunchAttributeClusterDimension;
    at.val.clusterDim.x = 2; at.val.clusterDim.y = 1; at.val.clusterDim.z = 1;
    lc.attrs = &at;
    lc.numAttrs = 1;
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, k1, &lc) != cudaSuccess || n <= 0) {
      (void)cudaGetLastError();
      n = sms / 2;
    }
    pairs = n < sms / 2 ? n : sms / 2;
    if (pairs < 1) return cudaErrorNotSupported;
    if (dev >= 0 && dev < 64) cached_pairs[dev] = pairs;
  }
  const unsigned grid = (unsigned)(2 * pairs);
  k1<<<grid, kThreads2, kSmemBytes2, st>>>(mA1, mG, mU, static_cast<__nv_bfloat16*>(h), offsets, d.n_ffn, d.F, d.D,
                                            err_word, static_cast<__nv_bfloat16*>(gate_out),
                                            static_cast<__nv_bfloat16*>(up_out));
  err = cudaGetLastError();
  if (err != cudaSuccess) return err;
  k2<<<grid, kThreads2, kSmemBytes2, st>>>(mA2, mD, mD, static_cast<__nv_bfloat16*>(y_perm), offsets, d.n_ffn, d.D,
                                            d.F, err_word, nullptr, nullptr);
  return cudaGetLastError();
}

}  // namespace moepp
