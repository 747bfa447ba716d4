// Grouped GEMMs of the backward pass on the 5th-generation tensor cores (sm_100a), bf16 operands, float
// accumulation in tensor memory.  The same persistent, warp-specialised frame as the forward kernels (TMA
// producer warp, one MMA-issuing thread, four epilogue warps (eight in the DH mode), a 4-stage (DH: 3-stage)
// shared-memory ring, two 128 x 256
// accumulators in the 512 TMEM columns), with the operands read in the layout they already have in HBM:
// where the contraction runs over the dimension that is NOT contiguous in memory, the tile is loaded as it
// lies and handed to tcgen05.mma as an MN-major operand, so nothing is transposed in memory.
//
//   DH    : dH[r, f]   = sum_d dYp[r, d] W_down[e][d, f]            A K-major, B MN-major
//           epilogue: dGate = dH * up * silu'(gate), dUp = dH * silu(gate), written over gate / up
//   DX    : dXp[r, d]  = sum_f dGate[r, f] W_gate[e][f, d] + sum_f dUp[r, f] W_up[e][f, d]
//                                                                   A K-major, B MN-major, two k passes
//   WGRAD : dW[e][m, n] = sum over the rows r of expert e of P[r, m] Q[r, n]   A and B MN-major, float out
//           (the rows of an expert are the k range; where a segment is not a whole number of 64-row k tiles the
//           rows of its last tile that lie beyond it are cleared in shared memory before the MMAs)
// Every wait is bounded: a wait that runs out raises the error word and the CTA drains and leaves.
#include <cuda.h>

#include "common.cuh"
#include "tc_common.cuh"

namespace moepp {
namespace {

constexpr int BM = 128, BN = 256, BK = 64, UMMA_K = 16;
constexpr int kMaxStages = 4;
// The DH mode reads gate and up and writes dGate and dUp for every tile; where a tile has few k steps (small D) that
// epilogue is the bound, and the kernel trades one ring stage for the staging room of eight epilogue warps instead
// of four (EW = 8: 0.31 -> 0.22 ms at D = 768; at D = 4096 the four-warp, four-stage form is 6 % faster).
__host__ __device__ constexpr int stages_of(int ew) { return ew == 8 ? 3 : 4; }
constexpr int kABytes = BM * BK * 2;   // 16 KiB
constexpr int kBBytes = BN * BK * 2;   // 32 KiB
constexpr int kStageBytes = kABytes + kBBytes;
constexpr int kBoxBytes = 64 * BK * 2; // one 64 x 64 box of an MN-major operand: 8 KiB
__host__ __device__ constexpr int threads_of(int ew) { return 64 + 32 * ew; }
constexpr int kTmemCols = 512;
constexpr int kStagePitch = 36;  // floats per row of an epilogue warp's 32 x 32 staging piece (conflict-free)
__host__ __device__ constexpr int smem_bytes_of(int mode, int ew) {
  return stages_of(ew) * kStageBytes + 1024 + (mode == 0 ? ew * 32 * kStagePitch * 4 : 0);
}

enum Mode { DH = 0, DX = 1, WGRAD = 2 };

// MN-major operand, 128-byte swizzle: 64 elements along M/N are contiguous (one 128-byte row per k), eight k
// rows make a 1024-byte group (stride byte offset), and the next 64 elements along M/N start one box later
// (leading byte offset).
__device__ __forceinline__ uint64_t make_smem_desc_mn(uint32_t addr) {
  uint64_t d = 0;
  d |= (uint64_t)((addr & 0x3FFFFu) >> 4);
  d |= (uint64_t)(kBoxBytes >> 4) << 16;  // leading byte offset
  d |= (uint64_t)(1024 >> 4) << 32;       // stride byte offset
  d |= (uint64_t)1 << 46;
  d |= (uint64_t)2 << 61;
  return d;
}

struct TileInfo {
  int e, row0, row_end, m0, n0, kb_count;
  int second;  // WGRAD with two products in one launch: this tile belongs to the second (A from tmA1, C = C2)
};

struct Args {
  void* C;                 // DX: bf16 [M_cap, Nout];  WGRAD: float [n_ffn, Mout, Nout]
  float* C2;               // WGRAD: output of a second product P2^T Q sharing Q with the first (nullptr: none)
  __nv_bfloat16 *gate, *up;  // DH: dGate, dUp out
  const __nv_bfloat16 *gate_in, *up_in;  // DH: pre-activations in (may be the same buffers)
  const int32_t* offsets;
  int n_ffn, Mout, Nout, Kd;
  int accumulate;          // WGRAD: add to C instead of overwriting it
  int32_t* err_word;
};

template <int MODE, int EW>
__global__ void __launch_bounds__(threads_of(EW), 1)
bwd_gemm_kernel(const __grid_constant__ CUtensorMap tmA0, const __grid_constant__ CUtensorMap tmA1,
                const __grid_constant__ CUtensorMap tmB0, const __grid_constant__ CUtensorMap tmB1, const Args a) {
  constexpr bool A_MN = MODE == WGRAD;
  constexpr int kStages = stages_of(EW);
  constexpr int kEpiWarps = EW;
  // bit 15: A is MN-major, bit 16: B is MN-major
  constexpr uint32_t kIdesc = umma_idesc_bf16(BM, BN) | (A_MN ? (1u << 15) : 0u) | (1u << 16);
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_full[kMaxStages], bar_empty[kMaxStages], bar_tmem_full[2], bar_tmem_empty[2],
      bar_drain;
  __shared__ uint32_t tmem_base_slot;
  __shared__ int tile_start[kMaxExperts + 1];
  __shared__ int seg_begin[kMaxExperts + 1];
  __shared__ volatile int abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t ring = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const int NT = (a.Nout + BN - 1) / BN;
  const int MT1 = (a.Mout + BM - 1) / BM;                        // WGRAD: m tiles of one product
  const int MT = (MODE == WGRAD && a.C2 != nullptr) ? 2 * MT1 : MT1;  // ... of the launch
  const int KB = (a.Kd + BK - 1) / BK;    // DH, DX
  int32_t* const err_word = a.err_word;

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < kStages; ++s) {
      mbar_init(smem_u32(&bar_full[s]), 1);
      mbar_init(smem_u32(&bar_empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&bar_tmem_full[b]), 1);
      mbar_init(smem_u32(&bar_tmem_empty[b]), kEpiWarps);
    }
    mbar_init(smem_u32(&bar_drain), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    int run = 0;
    for (int e = 0; e < a.n_ffn; ++e) {
      const int b = a.offsets[e], en = a.offsets[e + 1];
      seg_begin[e] = b;
      tile_start[e] = run;
      run += (MODE == WGRAD ? MT : (en - b + BM - 1) / BM) * NT;
    }
    seg_begin[a.n_ffn] = a.offsets[a.n_ffn];
    tile_start[a.n_ffn] = run;
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;
  const int total_tiles = tile_start[a.n_ffn];

  auto decode = [&](int L, int& e) -> TileInfo {
    while (L >= tile_start[e + 1]) ++e;
    const int local = L - tile_start[e];
    const int b = seg_begin[e], en = seg_begin[e + 1];
    TileInfo ti;
    ti.e = e;
    ti.row_end = en;
    if (MODE == WGRAD) {
      ti.row0 = b;
      const int mt = local % MT;
      ti.second = mt >= MT1 ? 1 : 0;
      ti.m0 = (ti.second ? mt - MT1 : mt) * BM;
      ti.n0 = (local / MT) * BN;
      ti.kb_count = (en - b + BK - 1) / BK;
    } else {
      const int mt = (en - b + BM - 1) / BM;
      ti.row0 = b + (local % mt) * BM;
      ti.m0 = 0;
      ti.second = 0;
      ti.n0 = (local / mt) * BN;
      ti.kb_count = (MODE == DX ? 2 : 1) * KB;
    }
    return ti;
  };

  if (warp == 0) {
    // ---------------------------------- TMA producer ---------------------------------------------
    if (lane == 0) {
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tmA0) : "memory");
      asm volatile("prefetch.tensormap [%0];" ::"l"(&tmB0) : "memory");
      if (MODE != DH) asm volatile("prefetch.tensormap [%0];" ::"l"(&tmA1) : "memory");
      if (MODE == DX) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmB1) : "memory");
      }
      uint32_t it = 0;
      int e = 0;
      bool ok = true;
      for (int L = blockIdx.x; L < total_tiles && ok; L += gridDim.x) {
        const TileInfo ti = decode(L, e);
        for (int kb = 0; kb < ti.kb_count; ++kb, ++it) {
          const uint32_t s = it % kStages, ph = (it / kStages) & 1u;
          if (!mbar_wait(smem_u32(&bar_empty[s]), ph ^ 1u, &abort_flag, 31, err_word)) { ok = false; break; }
          const uint32_t full = smem_u32(&bar_full[s]);
          const uint32_t a_dst = ring + s * kStageBytes, b_dst = a_dst + kABytes;
          mbar_expect_tx(full, kStageBytes);
          if (MODE == WGRAD) {
            const int krow = ti.row0 + kb * BK;  // k runs over the expert's rows
#pragma unroll
            for (int j = 0; j < BM / 64; ++j)
              tma_load_2d(a_dst + j * kBoxBytes, ti.second ? &tmA1 : &tmA0, ti.m0 + 64 * j, krow, full);
#pragma unroll
            for (int j = 0; j < BN / 64; ++j) tma_load_2d(b_dst + j * kBoxBytes, &tmB0, ti.n0 + 64 * j, krow, full);
          } else {
            const bool second = MODE == DX && kb >= KB;
            const int kk = second ? kb - KB : kb;
            const CUtensorMap* mA = second ? &tmA1 : &tmA0;
            const CUtensorMap* mB = second ? &tmB1 : &tmB0;
            tma_load_2d(a_dst, mA, kk * BK, ti.row0, full);
            const int brow = ti.e * a.Kd + kk * BK;  // k runs over the rows of expert e's weight matrix
#pragma unroll
            for (int j = 0; j < BN / 64; ++j) tma_load_2d(b_dst + j * kBoxBytes, mB, ti.n0 + 64 * j, brow, full);
          }
        }
      }
      if (!ok) {  // give the copies already issued a bounded chance to land before the CTA leaves
        const uint32_t n_back = it < (uint32_t)kStages ? it : (uint32_t)kStages;
        for (uint32_t i = 1; i <= n_back; ++i) {
          const uint32_t j = it - i, s = j % kStages, ph = (j / kStages) & 1u;
          for (int spin = 0; spin < 100000 && !mbar_try_wait(smem_u32(&bar_full[s]), ph); ++spin) __nanosleep(64);
        }
      }
    }
  } else if (warp == 1) {
    // ---------------------------------- MMA issuer -----------------------------------------------
    // Where a WGRAD k tile reaches past the end of its segment (segments that are not whole 64-row tiles) the rows
    // beyond the end belong to the next expert, or to nobody: before the MMAs read the stage this thread clears
    // them in the A operand (so that they add nothing), and after the last segment also in the B operand (rows
    // nobody owns may hold anything, and 0 x NaN is not 0).
    if (lane == 0) {
      uint32_t it = 0, tile_iter = 0;
      int e = 0;
      bool ok = true;
      const int rows_in_use = seg_begin[a.n_ffn];
      for (int L = blockIdx.x; L < total_tiles && ok; L += gridDim.x, ++tile_iter) {
        const TileInfo ti = decode(L, e);
        const uint32_t buf = tile_iter & 1u, tph = (tile_iter >> 1) & 1u;
        if (!mbar_wait(smem_u32(&bar_tmem_empty[buf]), tph ^ 1u, &abort_flag, 32, err_word)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * BN;
        for (int kb = 0; kb < ti.kb_count; ++kb, ++it) {
          const uint32_t s = it % kStages, ph = (it / kStages) & 1u;
          if (!mbar_wait(smem_u32(&bar_full[s]), ph, &abort_flag, 33, err_word)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_addr = ring + s * kStageBytes, b_addr = a_addr + kABytes;
          if (MODE == WGRAD) {
            const int valid = (ti.row_end - ti.row0) - kb * BK;  // k rows of this tile that belong to the segment
            if (valid < BK) {
              // a k row is one 128-byte line of every 64-column box: lines [valid, 64) of the boxes concerned
              uint8_t* stage = smem_raw + (ring - smem_u32(smem_raw)) + s * kStageBytes;
              const int boxes = ti.row_end >= rows_in_use ? 6 : 2;  // A only, or A and B
              for (int box = 0; box < boxes; ++box) {
                uint4* p = reinterpret_cast<uint4*>(stage + box * kBoxBytes + valid * 128);
                for (int i = 0; i < (BK - valid) * 8; ++i) p[i] = make_uint4(0u, 0u, 0u, 0u);
              }
              asm volatile("fence.proxy.async.shared::cta;" ::: "memory");  // generic writes -> visible to the MMAs
            }
          }
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            // 16 k: K-major = 32 bytes inside the swizzle row; MN-major = 16 rows of 128 bytes
            const uint64_t adesc = A_MN ? make_smem_desc_mn(a_addr + k * (UMMA_K * 128))
                                        : make_smem_desc(a_addr) + (uint64_t)(2 * k);
            const uint64_t bdesc = make_smem_desc_mn(b_addr + k * (UMMA_K * 128));
            umma_bf16(d_tmem, adesc, bdesc, kIdesc, (kb | k) != 0 ? 1u : 0u);
          }
          umma_commit(smem_u32(&bar_empty[s]));
        }
        if (ok) umma_commit(smem_u32(&bar_tmem_full[buf]));
      }
      if (!ok) {
        umma_commit(smem_u32(&bar_drain));
        for (int spin = 0; spin < 100000 && !mbar_try_wait(smem_u32(&bar_drain), 0); ++spin) __nanosleep(64);
      }
    }
  } else {
    // ---------------------------------- epilogue: 4 warps, one TMEM lane quarter each --------------
    const int q = warp & 3;  // the TMEM lanes this warp may read: 32 q .. 32 q + 31
    // with eight epilogue warps (DH) the two warps of a lane quarter take half of the columns each
    const int c_lo = kEpiWarps == 8 ? ((warp - 2) >> 2) * (BN / 2) : 0, c_hi = kEpiWarps == 8 ? c_lo + BN / 2 : BN;
    uint32_t tile_iter = 0;
    int e = 0;
    bool ok = true;
    for (int L = blockIdx.x; L < total_tiles && ok; L += gridDim.x, ++tile_iter) {
      const TileInfo ti = decode(L, e);
      const uint32_t buf = tile_iter & 1u, tph = (tile_iter >> 1) & 1u;
      if (!mbar_wait(smem_u32(&bar_tmem_full[buf]), tph, &abort_flag, 34, err_word)) { ok = false; break; }
      tc_fence_after();
      const uint32_t t_row = tmem_base + buf * BN + ((uint32_t)(q * 32) << 16);
      if (MODE == WGRAD) {
        const int m = ti.m0 + q * 32 + lane;
        const bool row_ok = m < a.Mout;
        const bool empty = ti.kb_count == 0;  // an expert without rows: the accumulator was never written
        float* crow = (ti.second ? a.C2 : static_cast<float*>(a.C)) +
                      ((size_t)ti.e * a.Mout + (row_ok ? m : 0)) * a.Nout + ti.n0;
#pragma unroll 1
        for (int c = 0; c < BN; c += 16) {
          uint32_t r[16];
          tmem_ld16(t_row + c, r);
          tmem_ld_wait();
          tmem_ld_pin(r);
          if (row_ok) {
#pragma unroll
            for (int v = 0; v < 4; ++v)
              if (ti.n0 + c + 4 * v + 4 <= a.Nout) {
                float4 o = empty ? make_float4(0.f, 0.f, 0.f, 0.f)
                                 : make_float4(__uint_as_float(r[4 * v]), __uint_as_float(r[4 * v + 1]),
                                               __uint_as_float(r[4 * v + 2]), __uint_as_float(r[4 * v + 3]));
                float4* dst = reinterpret_cast<float4*>(crow + c + 4 * v);
                if (a.accumulate) {
                  const float4 old = *dst;
                  o.x += old.x; o.y += old.y; o.z += old.z; o.w += old.w;
                }
                *dst = o;
              }
          }
        }
      } else {
        const int grow = ti.row0 + q * 32 + lane;
        const bool row_ok = grow < ti.row_end;
        const size_t at = (size_t)(row_ok ? grow : 0) * a.Nout + ti.n0;
        if (MODE == DH) {
          // 32 columns at a time: the warp parks its 32 x 32 piece of dH in shared memory (a thread holds a row),
          // then works on it 8 rows at a time with 4 lanes per row and 8 columns per lane, so that the gate / up
          // reads and the dGate / dUp writes cover 64 contiguous bytes per row (8 lines per warp instruction instead
          // of 32).  gate / up of the next 32 columns are requested while the current ones are worked on.
          float* stage = reinterpret_cast<float*>(smem_raw + (ring - smem_u32(smem_raw)) + kStages * kStageBytes) +
                         (warp - 2) * (32 * kStagePitch);
          const int sub_row = lane >> 2, sub_col = (lane & 3) * 8;
          uint4 gq[4], uq[4], gn[4], un[4];
          auto fetch = [&](int c, uint4 (&g)[4], uint4 (&u)[4]) {
#pragma unroll
            for (int p = 0; p < 4; ++p) {
              g[p] = make_uint4(0u, 0u, 0u, 0u);
              u[p] = make_uint4(0u, 0u, 0u, 0u);
              const int gr = ti.row0 + q * 32 + p * 8 + sub_row;
              if (gr < ti.row_end && ti.n0 + c + sub_col + 8 <= a.Nout) {
                const size_t o = (size_t)gr * a.Nout + ti.n0 + c + sub_col;
                g[p] = *reinterpret_cast<const uint4*>(a.gate_in + o);
                u[p] = *reinterpret_cast<const uint4*>(a.up_in + o);
              }
            }
          };
          fetch(c_lo, gq, uq);
#pragma unroll 1
          for (int c = c_lo; c < c_hi; c += 32) {
            if (c + 32 < c_hi) fetch(c + 32, gn, un);
            uint32_t r0[16], r1[16];
            tmem_ld16(t_row + c, r0);
            tmem_ld16(t_row + c + 16, r1);
            tmem_ld_wait();
            tmem_ld_pin(r0);
            tmem_ld_pin(r1);
            float* mine = stage + lane * kStagePitch;
#pragma unroll
            for (int v = 0; v < 4; ++v) {
              *reinterpret_cast<uint4*>(mine + 4 * v) = make_uint4(r0[4 * v], r0[4 * v + 1], r0[4 * v + 2], r0[4 * v + 3]);
              *reinterpret_cast<uint4*>(mine + 16 + 4 * v) = make_uint4(r1[4 * v], r1[4 * v + 1], r1[4 * v + 2], r1[4 * v + 3]);
            }
            __syncwarp();
#pragma unroll
            for (int p = 0; p < 4; ++p) {
              const int gr = ti.row0 + q * 32 + p * 8 + sub_row;
              const float4 d0 = *reinterpret_cast<const float4*>(stage + (p * 8 + sub_row) * kStagePitch + sub_col);
              const float4 d1 = *reinterpret_cast<const float4*>(stage + (p * 8 + sub_row) * kStagePitch + sub_col + 4);
              if (gr >= ti.row_end || ti.n0 + c + sub_col + 8 > a.Nout) continue;
              const float dh[8] = {d0.x, d0.y, d0.z, d0.w, d1.x, d1.y, d1.z, d1.w};
              const uint32_t gw[4] = {gq[p].x, gq[p].y, gq[p].z, gq[p].w};
              const uint32_t uw[4] = {uq[p].x, uq[p].y, uq[p].z, uq[p].w};
              uint32_t og[4], ou[4];
#pragma unroll
              for (int i = 0; i < 4; ++i) {
                float dg2[2], du2[2];
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                  const float g = j ? bf16_hi(gw[i]) : bf16_lo(gw[i]);
                  const float u = j ? bf16_hi(uw[i]) : bf16_lo(uw[i]);
                  const float sg = __fdividef(1.f, 1.f + __expf(-g));
                  dg2[j] = dh[2 * i + j] * u * (sg + g * sg * (1.f - sg));
                  du2[j] = dh[2 * i + j] * g * sg;
                }
                og[i] = pack_bf16(dg2[0], dg2[1]);
                ou[i] = pack_bf16(du2[0], du2[1]);
              }
              const size_t o = (size_t)gr * a.Nout + ti.n0 + c + sub_col;
              *reinterpret_cast<uint4*>(a.gate + o) = make_uint4(og[0], og[1], og[2], og[3]);
              *reinterpret_cast<uint4*>(a.up + o) = make_uint4(ou[0], ou[1], ou[2], ou[3]);
            }
            __syncwarp();  // the piece is consumed before the next one overwrites it
#pragma unroll
            for (int p = 0; p < 4; ++p) { gq[p] = gn[p]; uq[p] = un[p]; }
          }
        } else {
#pragma unroll 1
          for (int c = 0; c < BN; c += 32) {
            uint32_t r0[16], r1[16];
            tmem_ld16(t_row + c, r0);
            tmem_ld16(t_row + c + 16, r1);
            tmem_ld_wait();
            tmem_ld_pin(r0);
            tmem_ld_pin(r1);
            uint32_t o[16];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              o[i] = pack_bf16(__uint_as_float(r0[2 * i]), __uint_as_float(r0[2 * i + 1]));
              o[8 + i] = pack_bf16(__uint_as_float(r1[2 * i]), __uint_as_float(r1[2 * i + 1]));
            }
            if (row_ok) {
              __nv_bfloat16* crow = static_cast<__nv_bfloat16*>(a.C) + at + c;
#pragma unroll
              for (int v = 0; v < 4; ++v)
                if (ti.n0 + c + 8 * v + 8 <= a.Nout)
                  *reinterpret_cast<uint4*>(crow + 8 * v) = make_uint4(o[4 * v], o[4 * v + 1], o[4 * v + 2], o[4 * v + 3]);
            }
          }
        }
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&bar_tmem_empty[buf]));
    }
  }

  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    __syncwarp();
    tc_fence_after();
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(kTmemCols) : "memory");
  }
}

}  // namespace

namespace {

template <int MODE, int EW = 4>
cudaError_t run(int sms, const CUtensorMap& a0, const CUtensorMap& a1, const CUtensorMap& b0, const CUtensorMap& b1,
                const Args& args, cudaStream_t st) {
  auto k = bwd_gemm_kernel<MODE, EW>;
  cudaError_t err = cudaFuncSetAttribute(k, cudaFuncAttributeMaxDynamicSharedMemorySize, smem_bytes_of(MODE, EW));
  if (err != cudaSuccess) return err;
  k<<<sms, threads_of(EW), smem_bytes_of(MODE, EW), st>>>(a0, a1, b0, b1, args);
  return cudaGetLastError();
}

}  // namespace

// The WGRAD mode with token segments in the place of expert segments: sum over tokens of P[t, :]^T Q[t, :].
cudaError_t launch_token_outer_tc(const Dims& d, const void* P, const void* Q, float* part, const int32_t* segs,
                                  int n_seg, cudaStream_t st) {
  int dev = 0, sms = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (err != cudaSuccess) return err;
  int32_t* err_word = device_error_word();
  if (err_word == nullptr || n_seg < 1 || n_seg > kMaxExperts) return cudaErrorNotSupported;
  CUtensorMap mP, mQ;
  if (!make_bf16_tile_map(&mP, P, (uint64_t)d.T, 128, 64) || !make_bf16_tile_map(&mQ, Q, (uint64_t)d.T, (uint64_t)d.D, 64))
    return cudaErrorNotSupported;
  Args a{};
  a.offsets = segs; a.n_ffn = n_seg; a.err_word = err_word;
  a.C = part; a.Mout = 128; a.Nout = d.D; a.Kd = 0;
  return run<WGRAD>(sms, mP, mP, mQ, mQ, a, st);
}

// bf16 FFN backward on the tensor cores.  cudaErrorNotSupported when it does not apply (storage type, shapes the
// tensor maps cannot describe): the caller then uses the FMA path.
cudaError_t launch_ffn_backward_tc(const Dims& d, const void* x_perm, const int32_t* offsets, const void* W_gate,
                                   const void* W_up, const void* W_down, const void* h, const void* dy_perm,
                                   void* gate_buf, void* up_buf, void* dx_perm, float* dW_gate, float* dW_up,
                                   float* dW_down, cudaStream_t st, const void* gate_in, const void* up_in) {
  if (d.dtype != MOEPP_BF16) return cudaErrorNotSupported;
  if (d.T == 0 || d.n_ffn == 0 || d.M_cap == 0) return cudaErrorNotSupported;
  int dev = 0, sms = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (err != cudaSuccess) return err;
  int32_t* err_word = device_error_word();
  if (err_word == nullptr) return cudaErrorNotSupported;

  const uint64_t rows = (uint64_t)d.M_cap, D = (uint64_t)d.D, F = (uint64_t)d.F, E = (uint64_t)d.n_ffn;
  CUtensorMap mDyK, mDyMN, mHMN, mXpMN, mGateK, mUpK, mGateMN, mUpMN, mWdMN, mWgMN, mWuMN;
  if (!make_bf16_tile_map(&mDyK, dy_perm, rows, D, BM) ||     // K-major A of DH
      !make_bf16_tile_map(&mDyMN, dy_perm, rows, D, 64) ||    // MN-major A of dW_down
      !make_bf16_tile_map(&mHMN, h, rows, F, 64) ||           // MN-major B of dW_down
      !make_bf16_tile_map(&mXpMN, x_perm, rows, D, 64) ||     // MN-major B of dW_gate, dW_up
      !make_bf16_tile_map(&mGateK, gate_buf, rows, F, BM) ||  // K-major A of DX
      !make_bf16_tile_map(&mUpK, up_buf, rows, F, BM) ||
      !make_bf16_tile_map(&mGateMN, gate_buf, rows, F, 64) || // MN-major A of dW_gate
      !make_bf16_tile_map(&mUpMN, up_buf, rows, F, 64) ||
      !make_bf16_tile_map(&mWdMN, W_down, E * D, F, 64) ||    // MN-major B of DH: k = d, n = f
      !make_bf16_tile_map(&mWgMN, W_gate, E * F, D, 64) ||    // MN-major B of DX: k = f, n = d
      !make_bf16_tile_map(&mWuMN, W_up, E * F, D, 64))
    return cudaErrorNotSupported;

  // 1. the SwiGLU pre-activations again, unless the forward pass kept them: gate = Xp W_gate^T, up = Xp W_up^T
  if (gate_in == nullptr) {
    if ((err = launch_grouped_gemm_tcgen05(d, x_perm, W_gate, gate_buf, offsets, d.F, d.D, st)) != cudaSuccess) return err;
    if ((err = launch_grouped_gemm_tcgen05(d, x_perm, W_up, up_buf, offsets, d.F, d.D, st)) != cudaSuccess) return err;
    gate_in = gate_buf;
    up_in = up_buf;
  }

  Args a{};
  a.offsets = offsets; a.n_ffn = d.n_ffn; a.err_word = err_word;
  // 2. dW_down[e] = dYp_e^T H_e
  a.accumulate = (d.flags & MOEPP_FLAG_ACCUM_GRADS) ? 1 : 0;
  a.C = dW_down; a.Mout = d.D; a.Nout = d.F; a.Kd = 0;
  if ((err = run<WGRAD>(sms, mDyMN, mDyMN, mHMN, mHMN, a, st)) != cudaSuccess) return err;
  // 3. dH = dYp W_down -> dGate, dUp in place
  a.C = nullptr; a.gate = static_cast<__nv_bfloat16*>(gate_buf); a.up = static_cast<__nv_bfloat16*>(up_buf);
  a.gate_in = static_cast<const __nv_bfloat16*>(gate_in); a.up_in = static_cast<const __nv_bfloat16*>(up_in);
  a.Mout = 0; a.Nout = d.F; a.Kd = d.D;
  err = d.D <= 2048 ? run<DH, 8>(sms, mDyK, mDyK, mWdMN, mWdMN, a, st) : run<DH, 4>(sms, mDyK, mDyK, mWdMN, mWdMN, a, st);
  if (err != cudaSuccess) return err;
  // 4. dW_gate[e] = dGate_e^T Xp_e and dW_up[e] = dUp_e^T Xp_e in one launch (they share the Xp tiles)
  a.gate = nullptr; a.up = nullptr; a.Mout = d.F; a.Nout = d.D; a.Kd = 0;
  a.C = dW_gate; a.C2 = dW_up;
  if ((err = run<WGRAD>(sms, mGateMN, mUpMN, mXpMN, mXpMN, a, st)) != cudaSuccess) return err;
  a.C2 = nullptr;
  // 5. dXp = dGate W_gate + dUp W_up
  a.C = dx_perm; a.Mout = 0; a.Nout = d.D; a.Kd = d.F;
  return run<DX>(sms, mGateK, mUpK, mWgMN, mWuMN, a, st);
}

}  // namespace moepp
