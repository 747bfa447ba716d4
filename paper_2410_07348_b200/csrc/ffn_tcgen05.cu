// Grouped SwiGLU FFN of the MoE++ layer on the 5th-generation tensor cores (sm_100a), bf16 in,
// float accumulation in tensor memory.  Two launches of one persistent, warp-specialised kernel:
//   GEMM 1  h[r,:]      = silu(x_perm[r,:] W_gate[e]^T) * (x_perm[r,:] W_up[e]^T)   (SwiGLU epilogue)
//   GEMM 2  y_perm[r,:] = h[r,:] W_down[e]^T
// for every FFN expert e and every row r of its segment [offsets[e], offsets[e+1]).
//
// Per CTA (one per SM): warp 0 = TMA producer, warp 1 = MMA issuer (tcgen05.mma, one thread),
// warps 2-5 = epilogue (tcgen05.ld -> registers -> global).  Operand tiles (128 rows x 64 k of A,
// 256 rows x 64 k of B, 128-byte swizzle) move through a 4-stage shared-memory ring guarded by
// mbarriers; the 128 x 256 float accumulator is double-buffered in the 512 TMEM columns so that the
// epilogue of one tile overlaps the MMAs of the next.  For GEMM 1 the 256 accumulator columns are
// 128 gate columns followed by the matching 128 up columns, so SwiGLU needs no second pass.
// The tile list depends on the routing (offsets lives on the device): every role walks the same
// static schedule tile = blockIdx.x + i * gridDim.x and decodes it from a small table in shared memory.
// Every wait is bounded: a wait that runs out raises an error word and the CTA drains and leaves.
#include <cuda.h>

#include "common.cuh"
#include "tc_common.cuh"

namespace moepp {

__device__ int32_t g_device_error = 0;

cudaError_t read_and_clear_device_error(int32_t* code) {
  cudaError_t e = cudaDeviceSynchronize();
  if (e != cudaSuccess) return e;
  e = cudaMemcpyFromSymbol(code, g_device_error, sizeof(int32_t));
  if (e != cudaSuccess) return e;
  const int32_t zero = 0;
  return cudaMemcpyToSymbol(g_device_error, &zero, sizeof(int32_t));
}

int32_t* device_error_word() {
  void* p = nullptr;
  return cudaGetSymbolAddress(&p, g_device_error) == cudaSuccess ? static_cast<int32_t*>(p) : nullptr;
}

namespace {

constexpr int BM = 128;      // rows per tile (UMMA M)
constexpr int BK = 64;       // k elements per stage: 128 bytes of bf16 = one swizzle row
constexpr int UMMA_N = 256;  // accumulator columns per tile
constexpr int UMMA_K = 16;   // k per tcgen05.mma for 16-bit operands
constexpr int kStages = 4;
constexpr int kABytes = BM * BK * 2;          // 16 KiB
constexpr int kBBytes = UMMA_N * BK * 2;      // 32 KiB
constexpr int kStageBytes = kABytes + kBBytes;
constexpr int kThreads = 192;
constexpr int kTmemCols = 512;
constexpr int kSmemBytes = kStages * kStageBytes + 1024;  // + slack to align the ring to 1024 B

constexpr uint32_t kIdesc = umma_idesc_bf16(BM, UMMA_N);

__device__ __forceinline__ float silu_mul(float g, float u) { return __fdividef(g, 1.f + __expf(-g)) * u; }

struct TileInfo {
  int e, row0, row_end, n0;
};

// SWIGLU: C has Nout columns, the tile covers 128 of them (gate | up in the accumulator).
// otherwise the tile covers 256 columns of C.
// GATHER: the A rows are not read from a grouped buffer but fetched straight from the token-major
// activations: row r of the tile is token slot_of_row[r] / K, loaded four rows at a time with TMA
// gather loads (tmA then describes x with a one-row box); pad rows and rows beyond the rows in use
// are pointed at row T, outside the tensor, and arrive as zeros.
template <bool SWIGLU, bool GATHER>
__global__ void __launch_bounds__(kThreads, 1)
grouped_gemm_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB0,
                    const __grid_constant__ CUtensorMap tmB1, __nv_bfloat16* __restrict__ C,
                    const int32_t* __restrict__ offsets, int n_ffn, int Nout, int Kd,
                    const int32_t* __restrict__ slot_of_row, int top_k, int n_tokens) {
  constexpr int BN_OUT = SWIGLU ? 128 : 256;
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_full[kStages], bar_empty[kStages], bar_tmem_full[2], bar_tmem_empty[2],
      bar_drain;
  __shared__ uint32_t tmem_base_slot;
  __shared__ int tile_start[kMaxExperts + 1];
  __shared__ int seg_begin[kMaxExperts + 1];
  __shared__ volatile int abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t ring = (smem_u32(smem_raw) + 1023u) & ~1023u;
  const int NT = (Nout + BN_OUT - 1) / BN_OUT;
  const int KB = (Kd + BK - 1) / BK;

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < kStages; ++s) {
      mbar_init(smem_u32(&bar_full[s]), 1);
      mbar_init(smem_u32(&bar_empty[s]), 1);
    }
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&bar_tmem_full[b]), 1);
      mbar_init(smem_u32(&bar_tmem_empty[b]), 4);
    }
    mbar_init(smem_u32(&bar_drain), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    int run = 0;
    for (int e = 0; e < n_ffn; ++e) {
      const int b = offsets[e], en = offsets[e + 1];
      seg_begin[e] = b;
      tile_start[e] = run;
      run += ((en - b + BM - 1) / BM) * NT;
    }
    seg_begin[n_ffn] = offsets[n_ffn];
    tile_start[n_ffn] = run;
  }
  if (warp == 1) {  // TMEM: all 512 columns (two accumulators)
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                 "r"(kTmemCols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = tmem_base_slot;
  const int total_tiles = tile_start[n_ffn];

  // decode a linear tile index; `e` only moves forward
  auto decode = [&](int L, int& e) -> TileInfo {
    while (L >= tile_start[e + 1]) ++e;
    const int local = L - tile_start[e];
    const int b = seg_begin[e], en = seg_begin[e + 1];
    const int mt = (en - b + BM - 1) / BM;
    TileInfo ti;
    ti.e = e;
    ti.row0 = b + (local % mt) * BM;
    ti.row_end = en;
    ti.n0 = (local / mt) * BN_OUT;
    return ti;
  };

  if (warp == 0) {
    // ---------------------------------- TMA producer ---------------------------------------------
    // one lane issues tile loads; with GATHER all 32 lanes work: lane l fetches rows 4l..4l+3 of the A tile
    if (GATHER || lane == 0) {
      if (lane == 0) {
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmA) : "memory");
        asm volatile("prefetch.tensormap [%0];" ::"l"(&tmB0) : "memory");
        if (SWIGLU) asm volatile("prefetch.tensormap [%0];" ::"l"(&tmB1) : "memory");
      }
      uint32_t it = 0;
      int e = 0;
      bool ok = true;
      const int rows_in_use = seg_begin[n_ffn];
      for (int L = blockIdx.x; L < total_tiles && ok; L += gridDim.x) {
        const TileInfo ti = decode(L, e);
        const int brow = ti.e * Nout + ti.n0;
        int tok[4] = {0, 0, 0, 0};
        if (GATHER) {
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const int r = ti.row0 + lane * 4 + i;
            const int slot = (r < rows_in_use) ? __ldg(slot_of_row + r) : -1;
            tok[i] = (slot >= 0) ? slot / top_k : n_tokens;  // row n_tokens lies outside x: zero fill
          }
        }
        for (int kb = 0; kb < KB; ++kb, ++it) {
          const uint32_t s = it % kStages, ph = (it / kStages) & 1u;
          bool got = mbar_wait(smem_u32(&bar_empty[s]), ph ^ 1u, &abort_flag, 1, &g_device_error);
          if (GATHER) got = __all_sync(0xffffffffu, got);
          if (!got) { ok = false; break; }
          const uint32_t full = smem_u32(&bar_full[s]);
          const uint32_t a_dst = ring + s * kStageBytes, b_dst = a_dst + kABytes;
          if (lane == 0) mbar_expect_tx(full, kStageBytes);
          if (GATHER) {
            asm volatile(
                "cp.async.bulk.tensor.2d.shared::cluster.global.tile::gather4.mbarrier::complete_tx::bytes "
                "[%0], [%1, {%3, %4, %5, %6, %7}], [%2];" ::"r"(a_dst + (uint32_t)lane * 512u),
                "l"(&tmA), "r"(full), "r"(kb * BK), "r"(tok[0]), "r"(tok[1]), "r"(tok[2]), "r"(tok[3])
                : "memory");
          } else {
            tma_load_2d(a_dst, &tmA, kb * BK, ti.row0, full);
          }
          if (lane == 0) {
            if (SWIGLU) {
              tma_load_2d(b_dst, &tmB0, kb * BK, brow, full);
              tma_load_2d(b_dst + kBBytes / 2, &tmB1, kb * BK, brow, full);
            } else {
              tma_load_2d(b_dst, &tmB0, kb * BK, brow, full);
            }
          }
        }
      }
      if (!ok && lane == 0) {  // give the copies already issued a bounded chance to land before the CTA leaves
        const uint32_t n_back = it < (uint32_t)kStages ? it : (uint32_t)kStages;
        for (uint32_t i = 1; i <= n_back; ++i) {
          const uint32_t j = it - i, s = j % kStages, ph = (j / kStages) & 1u;
          for (int spin = 0; spin < 100000 && !mbar_try_wait(smem_u32(&bar_full[s]), ph); ++spin) __nanosleep(64);
        }
      }
    }
  } else if (warp == 1) {
    // ---------------------------------- MMA issuer -----------------------------------------------
    if (lane == 0) {
      uint32_t it = 0, tile_iter = 0;
      bool ok = true;
      for (int L = blockIdx.x; L < total_tiles && ok; L += gridDim.x, ++tile_iter) {
        const uint32_t buf = tile_iter & 1u, tph = (tile_iter >> 1) & 1u;
        if (!mbar_wait(smem_u32(&bar_tmem_empty[buf]), tph ^ 1u, &abort_flag, 2, &g_device_error)) { ok = false; break; }
        tc_fence_after();
        const uint32_t d_tmem = tmem_base + buf * UMMA_N;
        for (int kb = 0; kb < KB; ++kb, ++it) {
          const uint32_t s = it % kStages, ph = (it / kStages) & 1u;
          if (!mbar_wait(smem_u32(&bar_full[s]), ph, &abort_flag, 3, &g_device_error)) { ok = false; break; }
          tc_fence_after();
          const uint32_t a_addr = ring + s * kStageBytes, b_addr = a_addr + kABytes;
          const uint64_t adesc = make_smem_desc(a_addr), bdesc = make_smem_desc(b_addr);
#pragma unroll
          for (int k = 0; k < BK / UMMA_K; ++k) {
            // advancing k by 16 elements = 32 bytes inside the 128-byte swizzle row: +2 in the address field
            umma_bf16(d_tmem, adesc + (uint64_t)(2 * k), bdesc + (uint64_t)(2 * k), kIdesc, (kb | k) != 0 ? 1u : 0u);
          }
          umma_commit(smem_u32(&bar_empty[s]));  // stage reusable once these MMAs have read it
        }
        if (ok) umma_commit(smem_u32(&bar_tmem_full[buf]));  // accumulator complete
      }
      if (!ok) {  // let issued MMAs retire (bounded) before TMEM is released
        umma_commit(smem_u32(&bar_drain));
        for (int spin = 0; spin < 100000 && !mbar_try_wait(smem_u32(&bar_drain), 0); ++spin) __nanosleep(64);
      }
    }
  } else {
    // ---------------------------------- epilogue: 4 warps, one TMEM lane quarter each --------------
    const int q = warp & 3;  // lanes [32q, 32q+32) are the ones this warp may read
    uint32_t tile_iter = 0;
    int e = 0;
    bool ok = true;
    for (int L = blockIdx.x; L < total_tiles && ok; L += gridDim.x, ++tile_iter) {
      const TileInfo ti = decode(L, e);
      const uint32_t buf = tile_iter & 1u, tph = (tile_iter >> 1) & 1u;
      if (!mbar_wait(smem_u32(&bar_tmem_full[buf]), tph, &abort_flag, 4, &g_device_error)) { ok = false; break; }
      tc_fence_after();
      const int grow = ti.row0 + q * 32 + lane;
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
            o[i] = pack_bf16(silu_mul(__uint_as_float(g[2 * i]), __uint_as_float(u[2 * i])),
                             silu_mul(__uint_as_float(g[2 * i + 1]), __uint_as_float(u[2 * i + 1])));
          if (row_ok) {
            if (ti.n0 + c + 8 <= Nout) *reinterpret_cast<uint4*>(crow + c) = make_uint4(o[0], o[1], o[2], o[3]);
            if (ti.n0 + c + 16 <= Nout) *reinterpret_cast<uint4*>(crow + c + 8) = make_uint4(o[4], o[5], o[6], o[7]);
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
                *reinterpret_cast<uint4*>(crow + c + 8 * v) = make_uint4(o[4 * v], o[4 * v + 1], o[4 * v + 2], o[4 * v + 3]);
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

// ---- host side: tensor maps ---------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

namespace {
EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (fn == nullptr) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// [rows, cols] bf16 row-major matrix, box = box_rows x 64 columns, 128-byte swizzle, zero fill outside
}  // namespace

bool make_bf16_tile_map(CUtensorMap* tm, const void* base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (fn == nullptr || rows == 0) return false;
  const cuuint64_t dims[2] = {cols, rows};
  const cuuint64_t strides[1] = {cols * 2};
  const cuuint32_t box[2] = {64u, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
            CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
            CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}


cudaError_t launch_ffn_tcgen05(const Dims& d, const void* x_perm, const int32_t* offsets, const void* W_gate,
                               const void* W_up, const void* W_down, void* h, void* y_perm, cudaStream_t st) {
  if (d.T == 0 || d.n_ffn == 0 || d.M_cap == 0) return cudaSuccess;
  int dev = 0, sms = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (err != cudaSuccess) return err;

  CUtensorMap mA1, mG, mU, mA2, mD;
  const uint64_t rows = (uint64_t)d.M_cap;
  if (!make_bf16_tile_map(&mA1, x_perm, rows, (uint64_t)d.D, BM) ||
      !make_bf16_tile_map(&mG, W_gate, (uint64_t)d.n_ffn * d.F, (uint64_t)d.D, 128) ||
      !make_bf16_tile_map(&mU, W_up, (uint64_t)d.n_ffn * d.F, (uint64_t)d.D, 128) ||
      !make_bf16_tile_map(&mA2, h, rows, (uint64_t)d.F, BM) ||
      !make_bf16_tile_map(&mD, W_down, (uint64_t)d.n_ffn * d.D, (uint64_t)d.F, 256))
    return cudaErrorNotSupported;

  auto k1 = grouped_gemm_kernel<true, false>;
  auto k2 = grouped_gemm_kernel<false, false>;
  err = cudaFuncSetAttribute(k1, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
  if (err != cudaSuccess) return err;
  err = cudaFuncSetAttribute(k2, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
  if (err != cudaSuccess) return err;

  k1<<<sms, kThreads, kSmemBytes, st>>>(mA1, mG, mU, static_cast<__nv_bfloat16*>(h), offsets, d.n_ffn, d.F, d.D,
                                        nullptr, 1, 0);
  err = cudaGetLastError();
  if (err != cudaSuccess) return err;
  k2<<<sms, kThreads, kSmemBytes, st>>>(mA2, mD, mD, static_cast<__nv_bfloat16*>(y_perm), offsets, d.n_ffn, d.D, d.F,
                                        nullptr, 1, 0);
  return cudaGetLastError();
}

// Plain grouped product on the same kernel: C[r, :] = A[r, :] B[e]^T for the rows r of expert e's segment,
// A [M_cap, Kd], B [n_ffn, Nout, Kd], C [M_cap, Nout], all bf16.
cudaError_t launch_grouped_gemm_tcgen05(const Dims& d, const void* A, const void* B, void* C, const int32_t* offsets,
                                        int Nout, int Kd, cudaStream_t st) {
  if (d.T == 0 || d.n_ffn == 0 || d.M_cap == 0) return cudaSuccess;
  int dev = 0, sms = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (err != cudaSuccess) return err;
  CUtensorMap mA, mB;
  if (!make_bf16_tile_map(&mA, A, (uint64_t)d.M_cap, (uint64_t)Kd, BM) ||
      !make_bf16_tile_map(&mB, B, (uint64_t)d.n_ffn * Nout, (uint64_t)Kd, 256))
    return cudaErrorNotSupported;
  auto k2 = grouped_gemm_kernel<false, false>;
  err = cudaFuncSetAttribute(k2, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
  if (err != cudaSuccess) return err;
  k2<<<sms, kThreads, kSmemBytes, st>>>(mA, mB, mB, static_cast<__nv_bfloat16*>(C), offsets, d.n_ffn, Nout, Kd, nullptr,
                                        1, 0);
  return cudaGetLastError();
}

// The same FFN with GEMM 1 reading its rows straight from x through slot_of_row (no grouped copy of x).
cudaError_t launch_ffn_tcgen05_gather(const Dims& d, const void* x, const int32_t* slot_of_row, const int32_t* offsets,
                                      const void* W_gate, const void* W_up, const void* W_down, void* h, void* y_perm,
                                      cudaStream_t st) {
  if (d.T == 0 || d.n_ffn == 0 || d.M_cap == 0) return cudaSuccess;
  int dev = 0, sms = 0;
  cudaError_t err = cudaGetDevice(&dev);
  if (err != cudaSuccess) return err;
  err = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (err != cudaSuccess) return err;

  CUtensorMap mX, mG, mU, mA2, mD;
  const uint64_t rows = (uint64_t)d.M_cap;
  if (!make_bf16_tile_map(&mX, x, (uint64_t)d.T, (uint64_t)d.D, 1) ||
      !make_bf16_tile_map(&mG, W_gate, (uint64_t)d.n_ffn * d.F, (uint64_t)d.D, 128) ||
      !make_bf16_tile_map(&mU, W_up, (uint64_t)d.n_ffn * d.F, (uint64_t)d.D, 128) ||
      !make_bf16_tile_map(&mA2, h, rows, (uint64_t)d.F, BM) ||
      !make_bf16_tile_map(&mD, W_down, (uint64_t)d.n_ffn * d.D, (uint64_t)d.F, 256))
    return cudaErrorNotSupported;

  auto k1 = grouped_gemm_kernel<true, true>;
  auto k2 = grouped_gemm_kernel<false, false>;
  err = cudaFuncSetAttribute(k1, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
  if (err != cudaSuccess) return err;
  err = cudaFuncSetAttribute(k2, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemBytes);
  if (err != cudaSuccess) return err;

  k1<<<sms, kThreads, kSmemBytes, st>>>(mX, mG, mU, static_cast<__nv_bfloat16*>(h), offsets, d.n_ffn, d.F, d.D,
                                        slot_of_row, d.K, d.T);
  err = cudaGetLastError();
  if (err != cudaSuccess) return err;
  k2<<<sms, kThreads, kSmemBytes, st>>>(mA2, mD, mD, static_cast<__nv_bfloat16*>(y_perm), offsets, d.n_ffn, d.D, d.F,
                                        nullptr, 1, 0);
  return cudaGetLastError();
}

}  // namespace moepp
