// Placement controls (Appendix "placement_control"): per trajectory, choose m = number of corrected
// valid positions, valid positions for the teacher-mode loss: uniformly (Random-TM) or without
// replacement with the positions' TV as weights (TV-Weighted-TM: the m smallest exponential-race keys
// -log U / TV, uniform fill if fewer than m positions have positive TV).
//
// One block per trajectory.  A position's key is a 64-bit integer that orders like
// (tier, float64 key value): bit 63 is the tier (0: weighted key, or any key in Random mode; 1: the
// uniform of a zero-TV position, used by the fill), the rest are the bits of the non-negative double.
// The m-th smallest key is found by an 8-pass radix select over the keys, which are recomputed in
// every pass (a Philox call and a logarithm: the whole call touches N scalars, nothing is worth
// storing); equal keys go to the lower index by an ordered count.
#include "saki_common.cuh"
#include <math_constants.h>

namespace saki {

constexpr int ST = 256;                              // threads per block
constexpr unsigned long long KEY_INVALID = ~0ull;    // not a valid position: never chosen (m <= number of valid positions)

__device__ __forceinline__ bool sel_valid(const SelectParams& P, int64_t i) {
  if (P.mask && P.mask[i] == 0) return false;
  const uint32_t unusable = SAKI_ROW_NONFINITE | SAKI_ROW_BAD_ID | SAKI_ROW_TIMEOUT | SAKI_ROW_NOT_COMPUTED;
  return !(P.rollout_status && (P.rollout_status[i] & unusable));
}
__device__ __forceinline__ unsigned long long sel_key(const SelectParams& P, int64_t i) {
  if (!sel_valid(P, i)) return KEY_INVALID;
  const double u = scalar_uniform(P.seed, P.row_offset + (uint64_t)i, STAGE_SELECT);
  if (P.mode == SAKI_SELECT_TV_WEIGHTED) {
    const double d = (double)P.tv[i];
    if (d > 0.0 && d < CUDART_INF) return (unsigned long long)__double_as_longlong(-log(u) / d);
    return (1ull << 63) | (unsigned long long)__double_as_longlong(u);
  }
  return (unsigned long long)__double_as_longlong(u);
}

// sum over the block, returned to every thread; `sh` holds ST/32 + 1 ints
__device__ __forceinline__ int block_sum_i(int v, int* sh) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  __syncthreads();
  if (lane == 0) sh[warp] = v;
  __syncthreads();
  int a = 0;
  for (int w = 0; w < ST / 32; ++w) a += sh[w];
  return a;
}

__global__ void __launch_bounds__(ST) select_kernel(const SelectParams P) {
  __shared__ int hist[256];
  __shared__ int sh[ST / 32 + 1];
  __shared__ int pick[2];        // the chosen digit of a pass and the count below it
  for (int64_t b = blockIdx.x; b < P.B; b += gridDim.x) {
    const int64_t lo = P.seq_start[b], hi = P.seq_start[b + 1];
    // m = corrected valid positions of the trajectory
    int cnt = 0;
    for (int64_t i = lo + threadIdx.x; i < hi; i += ST) cnt += (sel_valid(P, i) && P.corrected[i] != 0) ? 1 : 0;
    const int m = block_sum_i(cnt, sh);
    if (threadIdx.x == 0 && P.m) P.m[b] = m;
    if (m == 0) {
      for (int64_t i = lo + threadIdx.x; i < hi; i += ST) P.selected[i] = 0;
      continue;
    }
    // radix select of the m-th smallest key: after the passes, `prefix` is that key and `below` the
    // number of keys smaller than it
    unsigned long long prefix = 0ull;
    int below = 0;
    for (int pass = 0; pass < 8; ++pass) {
      const int shift = 56 - 8 * pass;
      const unsigned long long high_mask = pass == 0 ? 0ull : (~0ull << (shift + 8));
      hist[threadIdx.x] = 0;               // ST == 256 bins
      __syncthreads();
      for (int64_t i = lo + threadIdx.x; i < hi; i += ST) {
        const unsigned long long k = sel_key(P, i);
        if ((k & high_mask) == prefix) atomicAdd(&hist[(int)((k >> shift) & 0xffull)], 1);
      }
      __syncthreads();
      if (threadIdx.x == 0) {
        int acc = below, dgt = 0;
        for (; dgt < 255; ++dgt) {
          if (acc + hist[dgt] >= m) break;
          acc += hist[dgt];
        }
        pick[0] = dgt; pick[1] = acc;
      }
      __syncthreads();
      prefix |= (unsigned long long)pick[0] << shift;
      below = pick[1];
      __syncthreads();
    }
    // keys below the threshold are chosen; of the keys equal to it, the first (m - below) in index order
    int need = m - below;
    for (int64_t base = lo; base < hi; base += ST) {
      const int64_t i = base + threadIdx.x;
      const unsigned long long k = i < hi ? sel_key(P, i) : KEY_INVALID;
      const bool eq = (i < hi) && (k == prefix) && (k != KEY_INVALID);
      // ordered rank of this thread among the equal keys of the chunk
      const unsigned bal = __ballot_sync(0xffffffffu, eq);
      const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
      __syncthreads();
      if (lane == 0) sh[warp] = __popc(bal);
      __syncthreads();
      int before = 0, total = 0;
      for (int w = 0; w < ST / 32; ++w) { if (w < warp) before += sh[w]; total += sh[w]; }
      const int rank = before + __popc(bal & ((1u << lane) - 1u));
      if (i < hi) P.selected[i] = (k < prefix || (eq && rank < need)) ? 1 : 0;
      need = max(0, need - total);
    }
  }
}

cudaError_t launch_select(const SelectParams& p, cudaStream_t st, int* n_launches) {
  if (p.B <= 0) return cudaSuccess;
  const int grid = (int)std::min<int64_t>(p.B, 1 << 16);
  select_kernel<<<grid, ST, 0, st>>>(p);
  ++*n_launches;
  return cudaGetLastError();
}

}  // namespace saki
