// Grouping of the FFN slots (zero-computation slots never get a row) and the row gather.
//   rank kernel  : stable rank of every FFN slot inside its expert -> row_of_slot, slot_of_row
//                  (up to 64 CTAs, each finds the rows before its slot range by counting them itself)
//   gather kernel: x_perm[row] = x[slot / K], 16-byte vectors, one warp per row
// The rank is deterministic (ascending slot id inside an expert): no atomics decide placement.
#include "common.cuh"

namespace moepp {
namespace {

constexpr int kRankThreads = 1024;
constexpr int kRankWarps = kRankThreads / 32;
constexpr int kRankSlotsPerCta = 2048;
constexpr int kRankMaxCtas = 64;

// CTA b owns the contiguous slot range [b*per_cta, (b+1)*per_cta).  Phase 0 counts, per FFN expert, the
// slots that precede the range (a plain shared-memory histogram of topk_idx[0, begin)): every CTA finds its
// own starting rows without any exchange between CTAs.  Then, inside the range, warp w owns a contiguous
// sub-range: pass 1 counts its slots per expert, a scan over (expert, warp) turns the counts into first
// rows, pass 2 hands out rows in slot order.
__global__ void __launch_bounds__(kRankThreads)
permute_rank_kernel(const int32_t* __restrict__ topk_idx, const int32_t* __restrict__ offsets, long long S,
                    long long per_cta, int n_ffn, int n_rank, int cap_ffn, int cap_zc,
                    int32_t* __restrict__ row_of_slot, int32_t* __restrict__ slot_of_row) {
  // n_rank: experts whose slots are ranked: the FFN experts, or all experts when a capacity limit (Eq. 8)
  // is active, because then the zero-computation experts fill up and drop slots too.
  __shared__ int base[kRankWarps][kMaxExperts];  // running rank (slots of this expert seen so far)
  __shared__ int before[kMaxExperts];
  __shared__ int seg0[kMaxExperts];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  for (int i = tid; i < kRankWarps * kMaxExperts; i += kRankThreads) (&base[0][0])[i] = 0;
  if (tid < kMaxExperts) {
    before[tid] = 0;
    seg0[tid] = (tid < n_ffn) ? offsets[tid] : 0;
  }
  __syncthreads();

  const long long c_begin = (long long)blockIdx.x * per_cta;
  const long long c_end = (c_begin + per_cta < S) ? c_begin + per_cta : S;

  // phase 0: slots before this CTA's range, per FFN expert (16 bytes per load)
  {
    const int4* v = reinterpret_cast<const int4*>(topk_idx);  // c_begin is a multiple of 4
    for (long long i = tid; i < c_begin / 4; i += kRankThreads) {
      const int4 q = __ldg(v + i);
      if (q.x < n_rank) atomicAdd(&before[q.x], 1);
      if (q.y < n_rank) atomicAdd(&before[q.y], 1);
      if (q.z < n_rank) atomicAdd(&before[q.z], 1);
      if (q.w < n_rank) atomicAdd(&before[q.w], 1);
    }
  }

  long long per_warp = (per_cta + kRankWarps - 1) / kRankWarps;
  per_warp = (per_warp + 31) / 32 * 32;
  const long long s_begin = c_begin + (long long)warp * per_warp;
  const long long s_end = (s_begin + per_warp < c_end) ? s_begin + per_warp : c_end;
  const unsigned lt_mask = (1u << lane) - 1u;

  for (long long s0 = s_begin; s0 < s_end; s0 += 32) {
    const long long s = s0 + lane;
    int e = (s < s_end) ? topk_idx[s] : -1;
    if (e >= n_rank) e = -1;
    const unsigned peers = __match_any_sync(0xffffffffu, e);
    if (e >= 0 && (peers & lt_mask) == 0) base[warp][e] += __popc(peers);
    __syncwarp();
  }
  __syncthreads();
  if (tid < n_rank) {
    int run = before[tid];
    for (int w = 0; w < kRankWarps; ++w) {
      const int c = base[w][tid];
      base[w][tid] = run;
      run += c;
    }
  }
  __syncthreads();
  for (long long s0 = s_begin; s0 < s_end; s0 += 32) {
    const long long s = s0 + lane;
    const bool live = s < s_end;
    int e = live ? topk_idx[s] : -1;
    if (e >= n_rank) e = -1;
    const unsigned peers = __match_any_sync(0xffffffffu, e);
    int row = -1;  // zero-computation slot: no row
    if (e >= 0) {
      const int rank = base[warp][e] + __popc(peers & lt_mask);
      if (rank >= (e < n_ffn ? cap_ffn : cap_zc)) row = -2;  // Eq. 8: the expert is full, the slot is dropped
      else if (e < n_ffn) row = seg0[e] + rank;
    }
    __syncwarp();
    if (e >= 0 && (peers & lt_mask) == 0) base[warp][e] += __popc(peers);
    __syncwarp();
    if (live) {
      row_of_slot[s] = row;
      if (row >= 0) slot_of_row[row] = (int32_t)s;
    }
  }
}

// One warp per grouped row.  Rows at or beyond offsets[n_ffn] are not touched.
template <typename XT>
__global__ void __launch_bounds__(256)
permute_gather_kernel(const XT* __restrict__ x, const int32_t* __restrict__ slot_of_row,
                      const int32_t* __restrict__ offsets, int n_ffn, int K, int D, long long M_cap,
                      XT* __restrict__ x_perm) {
  const int lane = threadIdx.x & 31;
  const long long row = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= M_cap) return;
  if (row >= __ldg(offsets + n_ffn)) return;
  const int slot = slot_of_row[row];
  constexpr int V = 16 / sizeof(XT);  // elements per 16-byte vector
  const int nvec = D / V;
  uint4* dst = reinterpret_cast<uint4*>(x_perm + (size_t)row * D);
  if (slot < 0) {
    for (int i = lane; i < nvec; i += 32) dst[i] = make_uint4(0u, 0u, 0u, 0u);
    return;
  }
  const uint4* src = reinterpret_cast<const uint4*>(x + (size_t)(slot / K) * D);
  int i = lane;
  for (; i + 96 < nvec; i += 128) {  // four loads in flight per lane
    const uint4 a = __ldg(src + i), b = __ldg(src + i + 32), c = __ldg(src + i + 64), e = __ldg(src + i + 96);
    dst[i] = a; dst[i + 32] = b; dst[i + 64] = c; dst[i + 96] = e;
  }
  for (; i < nvec; i += 32) dst[i] = __ldg(src + i);
}

// dst[i, :] = src[index[i], :] (zeros where index[i] < 0); one warp per row, rows of `bytes` bytes (multiple of 16)
__global__ void __launch_bounds__(256)
gather_rows_kernel(const uint4* __restrict__ src, const int32_t* __restrict__ index, long long n_rows, int vec_per_row,
                   uint4* __restrict__ dst) {
  const int lane = threadIdx.x & 31;
  const long long row = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  if (row >= n_rows) return;
  const int from = index[row];
  uint4* d = dst + (size_t)row * vec_per_row;
  if (from < 0) {
    for (int i = lane; i < vec_per_row; i += 32) d[i] = make_uint4(0u, 0u, 0u, 0u);
    return;
  }
  const uint4* s = src + (size_t)from * vec_per_row;
  int i = lane;
  for (; i + 96 < vec_per_row; i += 128) {  // four loads in flight per lane
    const uint4 a = __ldg(s + i), b = __ldg(s + i + 32), c = __ldg(s + i + 64), e = __ldg(s + i + 96);
    d[i] = a; d[i + 32] = b; d[i + 64] = c; d[i + 96] = e;
  }
  for (; i < vec_per_row; i += 32) d[i] = __ldg(s + i);
}

}  // namespace

cudaError_t launch_gather_rows(const void* src, const int32_t* index, long long n_rows, size_t row_bytes, void* dst,
                               cudaStream_t st) {
  if (n_rows == 0) return cudaSuccess;
  gather_rows_kernel<<<(unsigned)((n_rows + 7) / 8), 256, 0, st>>>(static_cast<const uint4*>(src), index, n_rows,
                                                                  (int)(row_bytes / 16), static_cast<uint4*>(dst));
  return cudaGetLastError();
}

cudaError_t launch_permute(const Dims& d, const void* x, const int32_t* topk_idx, const int32_t* offsets,
                           int32_t* row_of_slot, int32_t* slot_of_row, void* x_perm, cudaStream_t st) {
  if (d.M_cap > 0) {
    cudaError_t err = cudaMemsetAsync(slot_of_row, 0xff, sizeof(int32_t) * (size_t)d.M_cap, st);
    if (err != cudaSuccess) return err;
  }
  if (d.T == 0) return cudaSuccess;
  const long long S = (long long)d.T * d.K;
  long long n_cta = (S + kRankSlotsPerCta - 1) / kRankSlotsPerCta;
  if (n_cta > kRankMaxCtas) n_cta = kRankMaxCtas;
  long long per_cta = (S + n_cta - 1) / n_cta;
  per_cta = (per_cta + 1023) / 1024 * 1024;  // whole warps of 32 slots, and 16-byte loads in phase 0
  n_cta = (S + per_cta - 1) / per_cta;
  permute_rank_kernel<<<(unsigned)n_cta, kRankThreads, 0, st>>>(topk_idx, offsets, S, per_cta, d.n_ffn,
                                                                d.cap_on ? d.N : d.n_ffn, d.cap_ffn, d.cap_zc,
                                                                row_of_slot, slot_of_row);
  cudaError_t err = cudaGetLastError();
  if (err != cudaSuccess || d.n_ffn == 0 || d.M_cap == 0 || x_perm == nullptr) return err;  // nullptr: tables only
  const int rows_per_block = 8;
  const unsigned grid = (unsigned)((d.M_cap + rows_per_block - 1) / rows_per_block);
  if (d.dtype == MOEPP_BF16)
    permute_gather_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>(static_cast<const __nv_bfloat16*>(x), slot_of_row,
                                                               offsets, d.n_ffn, d.K, d.D, d.M_cap,
                                                               static_cast<__nv_bfloat16*>(x_perm));
  else
    permute_gather_kernel<float><<<grid, 256, 0, st>>>(static_cast<const float*>(x), slot_of_row, offsets, d.n_ffn,
                                                       d.K, d.D, d.M_cap, static_cast<float*>(x_perm));
  return cudaGetLastError();
}

}  // namespace moepp
