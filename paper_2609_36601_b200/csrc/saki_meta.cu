// The trainer's step (Section 3.5): loss and gradient of the routed objective for freshly
// computed student logits, from the rollout's token-aligned metadata.
//
//   C = 0:  L = -A log pi(x)      Eqs. "k1_loss_token", "k1_advantage_token" (A from the rollout)
//   C = 1:  L = -log pi(v*)       Eq. "teacher_mode_loss"
//   g_j = grad_scale * coef * (pi_j - [j = tok]) / temperature,  (coef, tok) = (A, x) or (1, v*)
//
// Two kernels:
//   meta_stream_kernel   bf16 rows: one persistent CTA of 1024 threads per SM takes whole rows.  Per
//                        element the work is one exponential for the sum and one for the gradient,
//                        so the kernel is bound by HBM: a row is read from HBM once and its
//                        gradient written once.  Every lane owns 16-byte shared-memory slots that it
//                        fills itself with cp.async: the leading steps of a warp's segment stay
//                        resident for both passes, the rest streams through a ring (first touch
//                        from HBM, second from L2).  While pass "grad" of a row runs, the slots it
//                        frees already receive the next row.
//   meta_general_kernel  any dtype, V and layout; float64; one block per row.  Also takes the rows
//                        whose float32 sum overflowed in the streaming kernel (row list).
#include "saki_device.cuh"
#include <mutex>

namespace saki {

// ---------------------------------------------------------------- shared pieces
// what a row contributes, from its metadata alone (no logits)
struct MetaRow {
  int tok;          // supervised token, -1: the row contributes nothing
  float coef;       // A or 1
  uint32_t status;  // 0, MASKED, NOT_COMPUTED, NONFINITE (advantage), BAD_ID
};
__device__ __forceinline__ MetaRow meta_row(const MetaParams& P, int64_t row) {
  MetaRow m;
  m.tok = -1; m.coef = 0.f; m.status = 0;
  if (P.mask && P.mask[row] == 0) { m.status = SAKI_ROW_MASKED; return m; }
  const uint32_t unusable = SAKI_ROW_NONFINITE | SAKI_ROW_BAD_ID | SAKI_ROW_TIMEOUT | SAKI_ROW_NOT_COMPUTED;
  if (P.rollout_status && (P.rollout_status[row] & unusable)) { m.status = SAKI_ROW_NOT_COMPUTED; return m; }
  const bool c = P.corrected[row] != 0;
  const int tok = c ? P.teacher_top1[row] : P.proposal[row];
  const float coef = c ? 1.f : P.advantage[row];
  if (!(fabsf(coef) < CUDART_INF_F)) { m.status = SAKI_ROW_NONFINITE; return m; }
  if (tok < 0 || tok >= P.V) { m.status = SAKI_ROW_BAD_ID; return m; }
  m.tok = tok; m.coef = coef;
  return m;
}
__device__ __forceinline__ void meta_write(const MetaParams& P, int64_t row, float loss, float logp, uint32_t status) {
  if (P.out.loss) P.out.loss[row] = loss;
  if (P.out.logp_tok) P.out.logp_tok[row] = logp;
  if (P.out.row_status) P.out.row_status[row] = status;
  if (status & (SAKI_ROW_NONFINITE | SAKI_ROW_BAD_ID)) atomicAdd(P.flagged, 1ull);
}

// ---------------------------------------------------------------- general kernel (float64)
constexpr int MG_THREADS = 256;

__device__ __forceinline__ double block_sum_d(double v, double* sh) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  __syncthreads();
  if (lane == 0) sh[warp] = v;
  __syncthreads();
  double a = 0.0;
  for (int w = 0; w < MG_THREADS / 32; ++w) a += sh[w];   // fixed order
  return a;
}
__device__ __forceinline__ double block_max_d(double v, double* sh) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmax(v, __shfl_xor_sync(0xffffffffu, v, o));
  __syncthreads();
  if (lane == 0) sh[warp] = v;
  __syncthreads();
  double a = sh[0];
  for (int w = 1; w < MG_THREADS / 32; ++w) a = fmax(a, sh[w]);
  return a;
}

template <typename T>
__global__ void __launch_bounds__(MG_THREADS) meta_general_kernel(const MetaParams P) {
  __shared__ double sh[MG_THREADS / 32];
  const int64_t n_items = P.from_list ? (int64_t)*P.redo_count : P.n_rows;
  for (int64_t item = blockIdx.x; item < n_items; item += gridDim.x) {
    const int64_t row = P.from_list ? (int64_t)P.redo_list[item] : item;
    const T* s = (const T*)P.s + row * P.ld_s;
    T* g = (T*)P.dlogits + row * P.ld_g;
    const int V = P.V;
    MetaRow m = meta_row(P, row);
    const double rtau = 1.0 / (double)P.temperature;
    double mx = -CUDART_INF, bad = 0.0;
    if (m.tok >= 0) {
      for (int j = threadIdx.x; j < V; j += MG_THREADS) {
        const double z = (double)ld_as_float(s, j);
        if (!(fabs(z) < CUDART_INF)) bad = 1.0;
        mx = fmax(mx, z);
      }
      bad = block_max_d(bad, sh);
      mx = block_max_d(mx, sh);
      if (bad != 0.0) { m.tok = -1; m.status = SAKI_ROW_NONFINITE; }
    }
    if (m.tok < 0) {                       // contributes nothing: zero gradient row
      for (int j = threadIdx.x; j < V; j += MG_THREADS) st_from_float(g, j, 0.f);
      if (threadIdx.x == 0) meta_write(P, row, 0.f, 0.f, m.status);
      continue;
    }
    double sum = 0.0;
    for (int j = threadIdx.x; j < V; j += MG_THREADS) sum += exp(((double)ld_as_float(s, j) - mx) * rtau);
    sum = block_sum_d(sum, sh);
    const double lse = mx * rtau + log(sum);
    const double logp = (double)ld_as_float(s, m.tok) * rtau - lse;
    const double kg = (double)P.grad_scale * (double)m.coef * rtau;
    const double rs = 1.0 / sum;
    for (int j = threadIdx.x; j < V; j += MG_THREADS) {
      const double p = exp(((double)ld_as_float(s, j) - mx) * rtau) * rs;
      st_from_float(g, j, (float)(kg * (p - (j == m.tok ? 1.0 : 0.0))));
    }
    if (threadIdx.x == 0) meta_write(P, row, (float)(-(double)m.coef * logp), (float)logp, 0u);
  }
}

cudaError_t launch_meta_general(const MetaParams& p, int dtype, cudaStream_t st, int* n_launches) {
  if (p.n_rows <= 0) return cudaSuccess;
  const int grid = (int)std::min<int64_t>(p.n_rows, p.from_list ? 1184 : (1 << 20));
  if (dtype == SAKI_BF16) meta_general_kernel<__nv_bfloat16><<<grid, MG_THREADS, 0, st>>>(p);
  else meta_general_kernel<float><<<grid, MG_THREADS, 0, st>>>(p);
  ++*n_launches;
  return cudaGetLastError();
}

// ---------------------------------------------------------------- streaming kernel (bf16)
// The kernel is instantiated for 32 warps (one CTA per SM) and for 16 warps (two CTAs per SM, for short
// rows: one CTA's block barriers and scalar step run under the other's passes).
constexpr int MW_FULL = 32, MW_HALF = 16;
// rows up to this length take the 16-warp instance (M positions/s, one / two CTAs per SM: V = 8192 52 / 77,
// 32000 30.8 / 37.5, 50048 23.2 / 27.0, 65536 19.5 / 19.9, 131072 10.5 / 10.6, 151936 9.1 / 8.8)
constexpr int M_HALF_MAX_V = 98304;
constexpr int MKS = 13;                  // 512-byte steps of shared memory per warp (a step = 32 chunks of 8 elements)
constexpr int MNST = 5;                  // ring stages of a warp whose segment does not fit
constexpr int MRES = MKS - MNST;         // resident steps of such a warp
constexpr int M_MAX_STEPS = 64;          // V <= 64 * 32 * 8 * MW
__host__ __device__ constexpr int moff_red(int MW) { return MW * MKS * 512; }              // [3][MW] doubles: per-warp sum, shift, maximum
__host__ __device__ constexpr int moff_bc(int MW) { return moff_red(MW) + 3 * MW * 8; }    // [2][8] floats: the row's broadcast scalars, by row parity
__host__ __device__ constexpr int msmem_bytes(int MW) { return moff_bc(MW) + 2 * 8 * 4; }
constexpr uint32_t M_FILLER = 0xFF7FFF7Fu;           // two bf16 of the most negative finite value: exp -> 0

__device__ __forceinline__ void m_cp_async16(uint32_t dst, const void* src, uint64_t pol) {
  asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;"
               ::"r"(dst), "l"(__cvta_generic_to_global(src)), "l"(pol) : "memory");
}
__device__ __forceinline__ void m_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void m_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ uint4 m_lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
  return v;
}
__device__ __forceinline__ void m_sts128(uint32_t addr, uint32_t w) {
  asm volatile("st.shared.v4.u32 [%0], {%1, %1, %1, %1};" ::"r"(addr), "r"(w) : "memory");
}
__device__ __forceinline__ uint64_t m_policy_last() {
  uint64_t p;
  asm("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t m_policy_first() {
  uint64_t p;
  asm("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void m_st_stream(void* p, uint4 v, uint64_t pol) {
  asm volatile("st.global.L2::cache_hint.v4.b32 [%0], {%1, %2, %3, %4}, %5;"
               ::"l"(__cvta_generic_to_global(p)), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w), "l"(pol) : "memory");
}
__device__ __forceinline__ float m_pow2(float n) {   // 2^n for whole n, clamped to the normal float range
  const int i = (int)fminf(fmaxf(n, -126.f), 127.f);
  return __uint_as_float((uint32_t)(127 + i) << 23);
}

// One warp's view of a row: `steps` steps of 32 chunks, the first `res` of them resident.
struct MSeg { int c0, c1, steps, res; };

// Fills this lane's slot with the 16 bytes at byte offset `off` of the row at `row_base`, or with the
// filler where the row has no such chunk (off >= lim; lim = 0: no row).
__device__ __forceinline__ void m_fill(uint32_t slot, const char* row_base, uint32_t off, uint32_t lim, uint64_t pol) {
  if (off < lim) m_cp_async16(slot, row_base + off, pol);
  else m_sts128(slot, M_FILLER);
}

// Visits the warp's steps in order: body(words, byte offset of the chunk in its row, valid).  Every
// step commits one cp.async group.  A streamed step, once read, requests the streamed step MNST
// further on: of this pass, or past its end the first streamed steps of the pass that follows (over
// `wrap`: the same row again after pass "sum", the next row after pass "grad"; nullptr: none).  With
// REFILL, a resident step, once read, requests the same step of `wrap` (the next row).
template <bool REFILL, typename Body>
__device__ __forceinline__ void m_visit(const MSeg& sg, int lane, uint32_t base, const char* cur, const char* wrap,
                                        uint64_t pol_cur, uint64_t pol_wrap, uint64_t pol_res, uint32_t& ring_slot,
                                        Body&& body) {
  const uint32_t lim = (uint32_t)sg.c1 * 16u;
  const uint32_t lim_wrap = wrap != nullptr ? lim : 0u;
  const uint32_t wrap_back = (uint32_t)(MNST - (sg.steps - sg.res)) * 512u;   // (mod 2^32) from a step to the one it requests in the next pass
  const char* wb = wrap != nullptr ? wrap : cur;
  uint32_t off = (uint32_t)(sg.c0 + lane) * 16u;
  uint32_t slot = base;
#pragma unroll 1
  for (int k = 0; k < sg.steps; ++k, off += 512) {
    uint4 a;
    m_wait<MNST - 1>();
    if (k < sg.res) {
      a = m_lds128(slot);
      if (REFILL) m_fill(slot, wb, off, lim_wrap, pol_res);
      slot += 512;
    } else {
      a = m_lds128(ring_slot);
      if (k + MNST < sg.steps) m_fill(ring_slot, cur, off + MNST * 512u, lim, pol_cur);
      else m_fill(ring_slot, wb, off + wrap_back, lim_wrap, pol_wrap);
      ring_slot += 512;
      if (ring_slot == base + MKS * 512) ring_slot = base + MRES * 512;
    }
    m_commit();
    body(a, off, off < lim);
  }
}

template <int MW>
__global__ void __launch_bounds__(MW * 32, MW_FULL / MW) meta_stream_kernel(const MetaParams P) {
  constexpr int MOFF_RED = moff_red(MW), MOFF_BC = moff_bc(MW);
  extern __shared__ __align__(128) unsigned char msm[];
  const int tid = threadIdx.x, lane = tid & 31;
  const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);
  double* red = (double*)(msm + MOFF_RED);
  const int V = P.V, n_chunks = V / 8;
  // whole steps of 32 chunks, dealt out in order: steps_q to every warp, one more to the first steps_r
  // (a segment that ended inside a step would cost its warp a partly empty step in both passes)
  const int steps_all = (n_chunks + 31) / 32, steps_q = steps_all / MW, steps_r = steps_all - steps_q * MW;
  MSeg sg;
  sg.steps = steps_q + (warp < steps_r ? 1 : 0);
  sg.c0 = min(n_chunks, 32 * (warp * steps_q + min(warp, steps_r)));
  sg.c1 = min(n_chunks, sg.c0 + 32 * sg.steps);
  sg.res = sg.steps <= MKS ? sg.steps : MRES;
  const uint32_t base = smem_addr(msm) + (uint32_t)warp * (MKS * 512) + (uint32_t)lane * 16;   // this lane's slot of step 0
  uint32_t ring_slot = base + MRES * 512;
  const float c32 = (float)(1.4426950408889634 / (double)P.temperature);
  const double rtau = 1.0 / (double)P.temperature;
  const uint64_t pol_last = m_policy_last(), pol_first = m_policy_first();
  const bool few_groups = sg.steps - 1 < MNST;   // a short segment: its fills are fewer groups back than the waits assume

  auto row_base = [&](int64_t row) { return reinterpret_cast<const char*>((const __nv_bfloat16*)P.s + row * P.ld_s); };

  // first row of this CTA: request its resident steps and the first ring steps, one group per step
  if ((int64_t)blockIdx.x < P.n_rows) {
    const char* b0 = row_base(blockIdx.x);
    const uint32_t lim = (uint32_t)sg.c1 * 16u, off0 = (uint32_t)(sg.c0 + lane) * 16u;
    for (int k = 0; k < sg.res; ++k) { m_fill(base + k * 512, b0, off0 + k * 512u, lim, pol_first); m_commit(); }
    if (sg.res < sg.steps)
      for (int j = 0; j < MNST; ++j) {
        m_fill(ring_slot + j * 512, b0, off0 + (uint32_t)(sg.res + j) * 512u, lim, pol_last);
        m_commit();
      }
  }

  int rb = 0;
  for (int64_t row = blockIdx.x; row < P.n_rows; row += gridDim.x, rb ^= 1) {
    float* bc = (float*)(msm + MOFF_BC) + rb * 8;
    const char* cur = row_base(row);
    const int64_t next_row = row + gridDim.x;
    const char* nxt = next_row < P.n_rows ? row_base(next_row) : nullptr;
    __nv_bfloat16* g_out = (__nv_bfloat16*)P.dlogits + row * P.ld_g;
    // thread 0: what the row contributes; its loads are in flight during pass "sum"
    MetaRow m;
    m.tok = -1; m.coef = 0.f; m.status = 0;
    float s_tok = 0.f;
    if (tid == 0) {
      m = meta_row(P, row);
      if (m.tok >= 0) s_tok = __bfloat162float(((const __nv_bfloat16*)cur)[m.tok]);
    }

    // ------------------------------------------------ pass "sum": sum of 2^(c s + k) under a shift fixed
    // before the pass (k = -ceil(c m), m the largest of the warp's first 256 logits: an element of the
    // row, so nothing that matters underflows; a row whose maximum lies ~88 nats above m overflows
    // and goes to the float64 kernel), and the true maximum on the side (packed bf16)
    if (few_groups) m_wait<0>();
    float ksw = 1e30f;
    {
      m_wait<MNST - 1>();
      uint4 f = make_uint4(M_FILLER, M_FILLER, M_FILLER, M_FILLER);
      if (sg.c0 + lane < sg.c1) f = m_lds128(base);
      const float2 a = unpack_bf16x2(max_bf16x2(max_bf16x2(f.x, f.y), max_bf16x2(f.z, f.w)));
      float m0 = fmaxf(a.x, a.y);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) m0 = fmaxf(m0, __shfl_xor_sync(0xffffffffu, m0, o));
      if (sg.c0 < sg.c1) ksw = -ceilf(c32 * fmaxf(m0, -1e30f));
    }
    float2 S0 = splat(0.f), S1 = splat(0.f);
    uint32_t run = M_FILLER;
    const char* pf = sg.steps == sg.res ? nxt : nullptr;
    {
      const float2 cc = splat(c32), kk = splat(ksw);
      m_visit<false>(sg, lane, base, cur, cur, pol_last, pol_first, pol_first, ring_slot, [&](const uint4& w, uint32_t off, bool valid) {
        // a row that is entirely resident leaves L2 free: the next row's bytes of this step are sent on
        // their way into L2 (one lane per 128-byte line), so that HBM stays busy during this pass.  With
        // a streamed part kept in L2 between the passes the same prefetch evicts it (measured: -17 %).
        if (pf != nullptr && valid && (lane & 7) == 0) asm volatile("prefetch.global.L2 [%0];" ::"l"(pf + off));
        run = max_bf16x2(run, max_bf16x2(max_bf16x2(w.x, w.y), max_bf16x2(w.z, w.w)));
        S0 = fadd2(S0, ex2f2(ffma2(unpack_bf16x2(w.x), cc, kk)));
        S1 = fadd2(S1, ex2f2(ffma2(unpack_bf16x2(w.y), cc, kk)));
        S0 = fadd2(S0, ex2f2(ffma2(unpack_bf16x2(w.z), cc, kk)));
        S1 = fadd2(S1, ex2f2(ffma2(unpack_bf16x2(w.w), cc, kk)));
      });
    }
    {
      double ws = ((double)S0.x + (double)S0.y) + ((double)S1.x + (double)S1.y);
      const float2 r2 = unpack_bf16x2(run);
      float wm = fmaxf(r2.x, r2.y);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        ws += __shfl_xor_sync(0xffffffffu, ws, o);
        wm = fmaxf(wm, __shfl_xor_sync(0xffffffffu, wm, o));
      }
      if (lane == 0) { red[warp] = ws; red[MW + warp] = (double)ksw; red[2 * MW + warp] = (double)wm; }
    }
    __syncthreads();
    if (warp == 0) {
      // the row's shift is that of its true maximum; a warp's shift came from an element of the row, so
      // it is never below the row's and the factors are exact powers of two <= 1
      const int wl = lane < MW ? lane : 0;        // lanes beyond the warp count carry nothing
      float mx = lane < MW ? (float)red[2 * MW + wl] : -CUDART_INF_F;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
      const float kr = -ceilf(c32 * fmaxf(mx, -1e30f));
      const double kw = lane < MW ? red[MW + wl] : 1e30;
      double sum = kw < 1e29 ? red[wl] * (double)m_pow2(kr - (float)kw) : 0.0;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) sum += __shfl_xor_sync(0xffffffffu, sum, o);
      if (lane == 0) {
        float scale = 0.f, kg = 0.f;
        int tok = -1;
        if (m.tok >= 0) {
          if (!(sum > 0.0) || !(sum < CUDART_INF)) {
            // a non-finite logit, or float32 overflow on a finite row: the float64 kernel decides
            P.redo_list[atomicAdd(P.redo_count, 1u)] = (int32_t)row;
          } else {
            const double lse = LN2 * (log2(sum) - (double)kr);
            const double logp = (double)s_tok * rtau - lse;
            const double kgd = (double)P.grad_scale * (double)m.coef * rtau;
            kg = (float)kgd;
            scale = (float)(kgd / sum);
            tok = m.tok;
            meta_write(P, row, (float)(-(double)m.coef * logp), (float)logp, 0u);
          }
        } else {
          meta_write(P, row, 0.f, 0.f, m.status);
        }
        bc[0] = kr; bc[1] = scale; bc[2] = kg; bc[3] = __int_as_float(tok);
      }
    }
    __syncthreads();

    // ------------------------------------------------ pass "grad": g = scale 2^(c s + k) - kg [j = tok]
    {
      const float kr = bc[0], scale = bc[1], kg = bc[2];
      const int tok = __float_as_int(bc[3]);
      const uint32_t tok_off = tok >= 0 ? (uint32_t)(tok >> 3) * 16u : 0xffffffffu;   // byte offset of the supervised token's chunk
      const float2 cc = splat(c32), kk = splat(kr), sc = splat(scale);
      char* g_bytes = reinterpret_cast<char*>(g_out);
      m_visit<true>(sg, lane, base, cur, nxt, pol_first, pol_last, pol_first, ring_slot, [&](const uint4& w, uint32_t off, bool valid) {
        uint4 g = make_uint4(0u, 0u, 0u, 0u);
        if (tok >= 0) {    // a row that contributes nothing gets exact zeros, whatever its logits
          const uint32_t ww[4] = {w.x, w.y, w.z, w.w};
          uint32_t gp[4];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float2 e = fmul2(ex2f2(ffma2(unpack_bf16x2(ww[i]), cc, kk)), sc);
            gp[i] = pack_bf16x2(e.x, e.y);
          }
          if (off == tok_off) {   // the supervised token: subtract the one-hot part
            const int el = tok & 7, wi = el >> 1;
            const uint32_t word = wi == 0 ? ww[0] : wi == 1 ? ww[1] : wi == 2 ? ww[2] : ww[3];
            const float2 sf = unpack_bf16x2(word);
            const float e = ex2f(fmaf((el & 1) ? sf.y : sf.x, c32, kr));
            const uint32_t g16 = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(fmaf(e, scale, -kg)));
            const uint32_t old = wi == 0 ? gp[0] : wi == 1 ? gp[1] : wi == 2 ? gp[2] : gp[3];
            const uint32_t neu = (el & 1) ? ((old & 0x0000ffffu) | (g16 << 16)) : ((old & 0xffff0000u) | g16);
            if (wi == 0) gp[0] = neu; else if (wi == 1) gp[1] = neu; else if (wi == 2) gp[2] = neu; else gp[3] = neu;
          }
          g = make_uint4(gp[0], gp[1], gp[2], gp[3]);
        }
        if (valid) m_st_stream(g_bytes + off, g, pol_first);
      });
    }
  }
  m_wait<0>();
}

bool meta_stream_can_serve(const MetaParams& p, int dtype) {
  if (dtype != SAKI_BF16) return false;
  if (p.V < 2048 || p.V % 8 != 0 || p.V > M_MAX_STEPS * 32 * 8 * MW_FULL) return false;
  if (p.n_rows > 0x7fffffffLL) return false;
  auto al16 = [](const void* q) { return ((uintptr_t)q & 15) == 0; };
  if (!al16(p.s) || !al16(p.dlogits)) return false;
  if (p.ld_s % 8 || p.ld_g % 8) return false;
  return true;
}

template <int MW>
static cudaError_t launch_meta_stream_as(const MetaParams& p, cudaStream_t st) {
  static std::mutex mu;
  static int cached_dev = -1, cached_sms = 0;
  int dev = 0;
  cudaGetDevice(&dev);
  {
    std::lock_guard<std::mutex> lock(mu);
    if (cached_dev != dev) {
      cudaError_t e = cudaFuncSetAttribute(meta_stream_kernel<MW>, cudaFuncAttributeMaxDynamicSharedMemorySize, msmem_bytes(MW));
      if (e != cudaSuccess) return e;
      e = cudaDeviceGetAttribute(&cached_sms, cudaDevAttrMultiProcessorCount, dev);
      if (e != cudaSuccess) return e;
      cached_dev = dev;
    }
  }
  const int grid = (int)std::min<int64_t>(p.n_rows, (int64_t)cached_sms * (MW_FULL / MW));
  meta_stream_kernel<MW><<<grid, MW * 32, msmem_bytes(MW), st>>>(p);
  return cudaGetLastError();
}

cudaError_t launch_meta_stream(const MetaParams& p, cudaStream_t st, int* n_launches, bool* served) {
  *served = false;
  if (p.n_rows <= 0) { *served = true; return cudaSuccess; }
  const cudaError_t e = p.V <= M_HALF_MAX_V ? launch_meta_stream_as<MW_HALF>(p, st) : launch_meta_stream_as<MW_FULL>(p, st);
  ++*n_launches;
  *served = true;
  return e;
}

}  // namespace saki
