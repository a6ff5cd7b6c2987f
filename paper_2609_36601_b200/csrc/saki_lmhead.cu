// The step in front of the routing path (Section 3.5 / Appendix K: the student drafts, the teacher
// verifies, and both leave full-vocabulary logits): logits = hidden x W^T as a bf16 GEMM on the 5th
// generation tensor cores, with what pass "lse" of the routing kernels needs from a row taken in the
// epilogue while the accumulator tile is still in tensor memory: the row maximum and the sum of
// exponentials (Section 3.1: p = softmax(logits / tau)), so that the logits are written once and one of
// the three later reads of a row can go.
//
// One persistent CTA per SM, tiles of 128 rows x 256 vocabulary columns, K in blocks of 64:
//   warp 0    one thread: TMA loads of the A (hidden) and B (weight) blocks into a 4-stage shared-memory ring
//             (128-byte swizzle; tensor maps cover this GPU's memory only; no multicast)
//   warp 1    allocates tensor memory; one thread issues tcgen05.mma (M 128, N 256, K 16, bf16 -> fp32) into one
//             of two accumulator buffers (2 x 256 columns), commits to the ring's "empty" barriers and,
//             after the last K block of a tile, to the accumulator's "full" barrier
//   warps 2-5 epilogue: tcgen05.ld of the thread's row (32 columns at a time), rounding to bf16, 16-byte
//             stores of the logits, and an online maximum / sum of 2^(logit * log2(e)/tau - max) over the
//             ROUNDED values (what the routing kernels will read); one (max, sum) pair per row and column
//             tile goes to a scratch array that a second small kernel folds into row_max and lse
// Every wait on an mbarrier is bounded; a wait that runs out sets an error word, and every role then
// leaves its loop, tensor memory is released and the kernel returns.
#include "saki_common.cuh"
#include <cuda.h>
#include <math_constants.h>
#include <algorithm>
#include <mutex>

namespace saki {

constexpr int LM_BM = 128, LM_BN = 256, LM_BK = 64, LM_STAGES = 4, LM_ACC = 2;
constexpr int LM_A_BYTES = LM_BM * LM_BK * 2, LM_B_BYTES = LM_BN * LM_BK * 2, LM_STAGE_BYTES = LM_A_BYTES + LM_B_BYTES;
constexpr int LM_THREADS = 192;
constexpr int LM_SMEM = LM_STAGES * LM_STAGE_BYTES + 256 + 1024;     // ring, barriers, slack for 1024-byte alignment
constexpr long long LM_WAIT_LIMIT = 4000000000LL;                    // ~2 s of SM cycles

struct LmParams {
  int64_t N;
  int32_t d, V;
  void* logits;            // [N, V] bf16, row stride ld_l elements
  int64_t ld_l;
  float* part;             // [N][n_tiles_n][2]: (max, sum) in base-2 units, per row and column tile
  float c;                 // log2(e) / temperature
  float* row_max_part;     // [N][n_tiles_n]: the tile's largest rounded logit
  int m_tiles, n_tiles, group_m;
  unsigned int* error;     // set to 1 if a wait ran out
};

__device__ __forceinline__ uint32_t lm_smem(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void lm_mbar_init(uint64_t* b, uint32_t n) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(lm_smem(b)), "r"(n));
}
__device__ __forceinline__ void lm_mbar_expect(uint64_t* b, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(lm_smem(b)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void lm_mbar_arrive(uint64_t* b) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(lm_smem(b)) : "memory");
}
__device__ __forceinline__ bool lm_try_wait(uint64_t* b, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
               : "=r"(ok) : "r"(lm_smem(b)), "r"(parity) : "memory");
  return ok != 0;
}
// bounded: false if the phase did not complete within the limit or another role has already given up
__device__ __forceinline__ bool lm_wait(uint64_t* b, uint32_t parity, volatile int* abort_flag) {
  if (lm_try_wait(b, parity)) return true;
  const long long t0 = clock64();
  while (!lm_try_wait(b, parity)) {
    if (*abort_flag) return false;
    if (clock64() - t0 > LM_WAIT_LIMIT) { *abort_flag = 1; return false; }
  }
  return true;
}
__device__ __forceinline__ void lm_tma_2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
  asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
               ::"r"(lm_smem(dst)), "l"(map), "r"(x), "r"(y), "r"(lm_smem(bar)) : "memory");
}
// shared-memory matrix descriptor: K-major operand, 128-byte swizzle, rows of 128 bytes, 8-row groups 1024 bytes apart
__device__ __forceinline__ uint64_t lm_desc(uint32_t smem_addr) {
  uint64_t d = 0;
  d |= (uint64_t)((smem_addr & 0x3FFFF) >> 4);          // start address
  d |= (uint64_t)1 << 16;                               // leading-dimension byte offset (unused with swizzle)
  d |= (uint64_t)(1024 >> 4) << 32;                     // stride-dimension byte offset: next group of 8 rows
  d |= (uint64_t)1 << 46;                               // descriptor version of this architecture
  d |= (uint64_t)2 << 61;                               // 128-byte swizzle
  return d;
}
// instruction descriptor: D fp32, A and B bf16, both K-major, N = 256, M = 128
constexpr uint32_t LM_IDESC = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(LM_BN >> 3) << 17) | ((uint32_t)(LM_BM >> 4) << 24);

__device__ __forceinline__ void lm_mma(uint32_t tmem_d, uint64_t da, uint64_t db, uint32_t accumulate) {
  asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
               "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
               ::"r"(tmem_d), "l"(da), "l"(db), "r"(LM_IDESC), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void lm_commit(uint64_t* bar) {   // the barrier gets an arrival when the MMAs issued so far are done
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(lm_smem(bar)) : "memory");
}
__device__ __forceinline__ void lm_ld32(uint32_t taddr, uint32_t (&r)[32]) {
  asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 "
               "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
               "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
               : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                 "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
                 "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
                 "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
               : "r"(taddr) : "memory");
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ float lm_ex2(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}

// tiles are numbered so that CTAs running side by side share weight tiles and stay inside a group of
// `group_m` row blocks whose hidden states fit in L2: within a group the column tile is the slow index
__device__ __forceinline__ void lm_tile(const LmParams& P, int t, int& m_blk, int& n_blk) {
  const int per_group = P.group_m * P.n_tiles;
  const int g = t / per_group, r = t - g * per_group;
  const int m0 = g * P.group_m, gm = min(P.group_m, P.m_tiles - m0);
  n_blk = r / gm;
  m_blk = m0 + (r - n_blk * gm);
}

__global__ void __launch_bounds__(LM_THREADS, 1) lmhead_kernel(const __grid_constant__ CUtensorMap map_a,
                                                               const __grid_constant__ CUtensorMap map_b, const LmParams P) {
  extern __shared__ unsigned char lm_raw[];
  unsigned char* base = (unsigned char*)(((uintptr_t)lm_raw + 1023) & ~(uintptr_t)1023);
  uint64_t* full = (uint64_t*)(base + LM_STAGES * LM_STAGE_BYTES);
  uint64_t* empty = full + LM_STAGES;
  uint64_t* tfull = empty + LM_STAGES;
  uint64_t* tempty = tfull + LM_ACC;
  uint32_t* tmem_slot = (uint32_t*)(tempty + LM_ACC);
  volatile int* abort_flag = (volatile int*)(tmem_slot + 1);
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int k_blocks = (P.d + LM_BK - 1) / LM_BK;
  // the last group of row blocks may be shorter: count the tiles exactly
  const int full_groups = P.m_tiles / P.group_m, rest_m = P.m_tiles - full_groups * P.group_m;
  const int total_tiles = (full_groups * P.group_m + rest_m) * P.n_tiles;

  if (tid == 0) {
    for (int s = 0; s < LM_STAGES; ++s) { lm_mbar_init(&full[s], 1); lm_mbar_init(&empty[s], 1); }
    for (int a = 0; a < LM_ACC; ++a) { lm_mbar_init(&tfull[a], 1); lm_mbar_init(&tempty[a], 4); }
    *abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(lm_smem(tmem_slot)), "r"(LM_ACC * LM_BN) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_base = *tmem_slot;

  if (warp == 0) {
    if (lane == 0) {            // ---- producer
      int stage = 0;
      uint32_t phase = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
        int m_blk, n_blk;
        lm_tile(P, t, m_blk, n_blk);
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!lm_wait(&empty[stage], phase ^ 1u, abort_flag)) { ok = false; break; }
          unsigned char* a = base + stage * LM_STAGE_BYTES;
          lm_mbar_expect(&full[stage], LM_STAGE_BYTES);
          lm_tma_2d(a, &map_a, kb * LM_BK, m_blk * LM_BM, &full[stage]);
          lm_tma_2d(a + LM_A_BYTES, &map_b, kb * LM_BK, n_blk * LM_BN, &full[stage]);
          if (++stage == LM_STAGES) { stage = 0; phase ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    if (lane == 0) {            // ---- MMA issuer
      int stage = 0, acc = 0;
      uint32_t phase = 0, acc_phase = 0;
      bool ok = true;
      for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
        if (!lm_wait(&tempty[acc], acc_phase ^ 1u, abort_flag)) break;      // the epilogue has drained this buffer
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t tmem_d = tmem_base + (uint32_t)(acc * LM_BN);
        for (int kb = 0; kb < k_blocks; ++kb) {
          if (!lm_wait(&full[stage], phase, abort_flag)) { ok = false; break; }
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t a_addr = lm_smem(base + stage * LM_STAGE_BYTES);
          const uint64_t da = lm_desc(a_addr), db = lm_desc(a_addr + LM_A_BYTES);
#pragma unroll
          for (int k = 0; k < LM_BK / 16; ++k)        // 32 bytes further along K inside the swizzled row: +2 in units of 16 bytes
            lm_mma(tmem_d, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), (kb | k) ? 1u : 0u);
          lm_commit(&empty[stage]);                   // the ring slot is free once these MMAs have read it
          if (++stage == LM_STAGES) { stage = 0; phase ^= 1u; }
        }
        if (!ok) break;
        lm_commit(&tfull[acc]);                       // the tile's accumulator is complete
        if (++acc == LM_ACC) { acc = 0; acc_phase ^= 1u; }
      }
    }
  } else {                      // ---- epilogue warps 2..5: TMEM lane quarter = warp % 4
    const int q = warp & 3;
    int acc = 0;
    uint32_t acc_phase = 0;
    for (int t = blockIdx.x; t < total_tiles; t += gridDim.x) {
      int m_blk, n_blk;
      lm_tile(P, t, m_blk, n_blk);
      if (!lm_wait(&tfull[acc], acc_phase, abort_flag)) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      const int64_t row = (int64_t)m_blk * LM_BM + q * 32 + lane;
      const int col_tile = n_blk * LM_BN;
      __nv_bfloat16* out = (__nv_bfloat16*)P.logits + row * P.ld_l + col_tile;
      float m = -CUDART_INF_F, s = 0.f, xmax = -CUDART_INF_F;
#pragma unroll 1
      for (int ch = 0; ch < LM_BN / 32; ++ch) {
        uint32_t r[32];
        lm_ld32(tmem_base + ((uint32_t)(q * 32) << 16) + (uint32_t)(acc * LM_BN + ch * 32), r);
        const int col0 = col_tile + ch * 32;
        if (col0 >= P.V) continue;                    // (warp-uniform) columns past the vocabulary: zero-filled weights
        uint32_t pk[16];
        float y[32];
        float cm = -CUDART_INF_F;
#pragma unroll
        for (int i = 0; i < 16; ++i) {
          const float a = __uint_as_float(r[2 * i]), b = __uint_as_float(r[2 * i + 1]);
          asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(pk[i]) : "f"(b), "f"(a));
          const float ra = __uint_as_float(pk[i] << 16), rb = __uint_as_float(pk[i] & 0xffff0000u);   // the stored values
          const bool va = col0 + 2 * i < P.V, vb = col0 + 2 * i + 1 < P.V;
          xmax = fmaxf(xmax, fmaxf(va ? ra : -CUDART_INF_F, vb ? rb : -CUDART_INF_F));
          y[2 * i] = va ? ra * P.c : -CUDART_INF_F;
          y[2 * i + 1] = vb ? rb * P.c : -CUDART_INF_F;
          cm = fmaxf(cm, fmaxf(y[2 * i], y[2 * i + 1]));
        }
        if (cm > m) { s *= lm_ex2(m - cm); m = cm; }  // (m = -inf at first: s is 0 and stays 0)
        float add = 0.f;
#pragma unroll
        for (int i = 0; i < 32; ++i) add += lm_ex2(y[i] - m);
        s += add;
        if (row < P.N) {
          const int n_valid = min(32, P.V - col0);    // V is a multiple of 8: whole 16-byte vectors
#pragma unroll
          for (int v = 0; v < 4; ++v)
            if (v * 8 < n_valid)
              *reinterpret_cast<uint4*>(out + ch * 32 + v * 8) = make_uint4(pk[4 * v], pk[4 * v + 1], pk[4 * v + 2], pk[4 * v + 3]);
        }
      }
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) lm_mbar_arrive(&tempty[acc]);    // this warp has read its quarter of the accumulator
      if (++acc == LM_ACC) { acc = 0; acc_phase ^= 1u; }
      if (row < P.N) {
        float* pp = P.part + (row * P.n_tiles + n_blk) * 2;
        pp[0] = m; pp[1] = s;
        P.row_max_part[row * P.n_tiles + n_blk] = xmax;
      }
    }
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (tid == 0 && *abort_flag) atomicExch(P.error, 1u);
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(LM_ACC * LM_BN) : "memory");
  }
}

// one warp per row: fold the per-tile pairs into the row's maximum logit and log-sum-exp
__global__ void lmhead_rows_kernel(const LmParams P, float* row_max, float* lse) {
  const int64_t row = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
  const int lane = threadIdx.x & 31;
  if (row >= P.N) return;
  const float* pp = P.part + row * P.n_tiles * 2;
  float m = -CUDART_INF_F, xm = -CUDART_INF_F;
  for (int t = lane; t < P.n_tiles; t += 32) { m = fmaxf(m, pp[2 * t]); xm = fmaxf(xm, P.row_max_part[row * P.n_tiles + t]); }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) { m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o)); xm = fmaxf(xm, __shfl_xor_sync(0xffffffffu, xm, o)); }
  double s = 0.0;
  for (int t = lane; t < P.n_tiles; t += 32) s += (double)pp[2 * t + 1] * exp2((double)pp[2 * t] - (double)m);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
  if (lane == 0) {
    const bool failed = *P.error != 0;     // a wait ran out in the GEMM: nothing of this call is to be trusted
    if (row_max) row_max[row] = failed ? CUDART_NAN_F : xm;
    if (lse) lse[row] = failed ? CUDART_NAN_F : (float)(((double)m + log2(s)) * 0.693147180559945309417232121458);
  }
}

// ---------------------------------------------------------------- host side
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  static std::once_flag once;
  std::call_once(once, [] {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
      fn = (EncodeTiledFn)p;
  });
  return fn;
}

// a [rows, d] bf16 matrix, d contiguous: boxes of 64 x box_rows elements, 128-byte swizzle, zero fill outside
static bool make_map(CUtensorMap* map, const void* ptr, int64_t rows, int64_t d, int64_t ld, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  const cuuint64_t dims[2] = {(cuuint64_t)d, (cuuint64_t)rows};
  const cuuint64_t strides[1] = {(cuuint64_t)ld * 2};
  const cuuint32_t box[2] = {(cuuint32_t)LM_BK, (cuuint32_t)box_rows};
  const cuuint32_t estr[2] = {1, 1};
  return fn(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

int64_t lmhead_scratch_bytes(int64_t N, int32_t V) {
  const int64_t n_tiles = (V + LM_BN - 1) / LM_BN;
  return N * n_tiles * 3 * (int64_t)sizeof(float) + 256;
}

cudaError_t launch_lmhead(const saki_lmhead_in& in, void* logits, int64_t ld_l, float* row_max, float* lse, void* scratch,
                          cudaStream_t st, const char** why) {
  *why = nullptr;
  CUtensorMap map_a, map_b;
  if (!make_map(&map_a, in.hidden, in.N, in.d, in.ld_h, LM_BM) || !make_map(&map_b, in.weight, in.V, in.d, in.ld_w, LM_BN)) {
    *why = "cuTensorMapEncodeTiled failed (pointers 16-byte aligned, strides multiples of 8 elements?)";
    return cudaErrorInvalidValue;
  }
  static std::mutex mu;
  static int attr_dev = -1, sms = 0;
  int dev = 0;
  cudaGetDevice(&dev);
  {
    std::lock_guard<std::mutex> lock(mu);
    if (attr_dev != dev) {
      cudaError_t e = cudaFuncSetAttribute(lmhead_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, LM_SMEM);
      if (e != cudaSuccess) return e;
      e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
      if (e != cudaSuccess) return e;
      attr_dev = dev;
    }
  }
  LmParams p;
  p.N = in.N; p.d = in.d; p.V = in.V; p.logits = logits; p.ld_l = ld_l;
  p.m_tiles = (int)((in.N + LM_BM - 1) / LM_BM);
  p.n_tiles = (in.V + LM_BN - 1) / LM_BN;
  // row blocks per group: their hidden states (128 x d x 2 bytes each) should fill about a quarter of a 126 MB L2
  const int64_t blk_bytes = (int64_t)LM_BM * in.d * 2;
  p.group_m = (int)std::max<int64_t>(1, std::min<int64_t>(p.m_tiles, (32LL << 20) / std::max<int64_t>(1, blk_bytes)));
  p.c = (float)(1.4426950408889634 / (double)in.temperature);
  p.error = (unsigned int*)scratch;
  p.part = (float*)((char*)scratch + 256);
  p.row_max_part = p.part + in.N * p.n_tiles * 2;
  cudaError_t e = cudaMemsetAsync(p.error, 0, sizeof(unsigned int), st);
  if (e != cudaSuccess) return e;
  const int64_t tiles = (int64_t)p.m_tiles * p.n_tiles;
  const int grid = (int)std::min<int64_t>(tiles, sms);
  lmhead_kernel<<<grid, LM_THREADS, LM_SMEM, st>>>(map_a, map_b, p);
  e = cudaGetLastError();
  if (e != cudaSuccess) return e;
  const int warps = 8;
  lmhead_rows_kernel<<<(unsigned)((in.N + warps - 1) / warps), warps * 32, 0, st>>>(p, row_max, lse);
  return cudaGetLastError();
}

}  // namespace saki
