// One-row-per-SM kernel for bf16 rows.
//
// One persistent CTA of 1024 threads per SM routes whole rows, one after the
// other.  A row pair (student + teacher, e.g. 608 KB at V = 151936) does not
// fit on one SM, so it is kept in two places:
//   - the leading part of every warp's segment lives in shared memory
//     (192 KB per CTA), filled by per-warp 1-D bulk async copies that are
//     issued for the NEXT row as soon as the warp has read its resident part
//     for the last time;
//   - the rest is read from global memory in every pass.  Each row is touched
//     by one SM only, so after the first pass these reads are L2 hits; the
//     next row's share is pulled into L2 ahead of time with bulk L2 prefetches.
// HBM therefore sees each logit row once and the gradient row once.  All
// reductions stay inside the CTA (warp shuffles + shared memory), so a pass of
// ~150 k elements per SM amortises them.  Passes:
//   max      packed bf16 maxima of both rows (first touch of the L2 part)
//   lse      2 exponentials/element: log-sum-exps, moments of the logit
//            difference under p (initial guess of lambda), KL(T||p), argmax
//   solve    1 exponential/element per evaluation of KL(q_beta||p) and its
//            slope; Newton on sqrt(KL) in a bisection bracket (Eqs. "bridge",
//            "trust_region")
//   final    2 exponentials/element: TV = sum [q-p]_+ with per-warp ordered
//            partial sums for the inverse-CDF residual draw (Eqs. "accept",
//            "residual"), gradient row streamed out (Eq. "general_objective")
// Per-element work is float32 (packed f32x2 FMAs, ex2.approx); cross-thread
// combinations and per-row scalars are float64.
#include "saki_device.cuh"
#include <mutex>

namespace saki {

constexpr int RT = 1024;                // threads per CTA
constexpr int RW = RT / 32;             // warps per CTA
constexpr int KS_MAX = 6;               // resident steps per warp (a step = 32 chunks of 8 elements)
constexpr int RES_CHUNKS = KS_MAX * 32; // resident chunks per warp and row
constexpr int RNV = 8;                  // doubles per partial vector

constexpr int ROFF_S = 0;                                        // [RW][RES_CHUNKS] uint4
constexpr int ROFF_T = RW * RES_CHUNKS * 16;
constexpr int ROFF_RED = 2 * RW * RES_CHUNKS * 16;               // [RNV][RW] doubles
constexpr int ROFF_BC = ROFF_RED + RNV * RW * 8;                 // [BC_DOUBLES] doubles
constexpr int ROFF_WMAX = ROFF_BC + BC_DOUBLES * 8;              // [2][RW] floats
constexpr int ROFF_MBAR = ROFF_WMAX + 2 * RW * 4;
constexpr int RSMEM_BYTES = ROFF_MBAR + 16;

__device__ __forceinline__ void prefetch_l2(const void* src, uint32_t bytes) {
  asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
}
__device__ __forceinline__ uint4 ld_l2(const __nv_bfloat16* p) { return __ldcg(reinterpret_cast<const uint4*>(p)); }

__device__ __forceinline__ double warp_sum_d(double a) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
  return a;
}
__device__ __forceinline__ double warp_min_d(double a) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) a = fmin(a, __shfl_xor_sync(0xffffffffu, a, o));
  return a;
}
__device__ __forceinline__ float warp_max_f(float a) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) a = fmaxf(a, __shfl_xor_sync(0xffffffffu, a, o));
  return a;
}

struct Seg {   // this warp's share of a row, in chunks of 8 elements
  int c0, c1;          // [c0, c1)
  int steps, res;      // steps of 32 chunks; the first `res` of them are shared-memory resident
};

// Visits this thread's chunks in step order: body(a, b, chunk, valid) with the packed student /
// teacher words of the chunk.  Global (L2) chunks are fetched one step ahead.
template <typename Body>
__device__ __forceinline__ void for_each_chunk(const Seg& sg, int lane, const uint4* res_s, const uint4* res_t,
                                               const __nv_bfloat16* g_s, const __nv_bfloat16* g_t, Body&& body) {
  const uint4 sent = make_uint4(0xFF7FFF7Fu, 0xFF7FFF7Fu, 0xFF7FFF7Fu, 0xFF7FFF7Fu);   // exp -> 0, difference 0
#pragma unroll
  for (int k = 0; k < KS_MAX; ++k) {
    if (k < sg.res) {
      const int c = sg.c0 + k * 32 + lane;
      const bool valid = c < sg.c1;
      uint4 a = sent, b = sent;
      if (valid) { a = res_s[k * 32 + lane]; b = res_t[k * 32 + lane]; }
      body(a, b, c, valid);
    }
  }
  if (sg.steps > sg.res) {
    int c = sg.c0 + sg.res * 32 + lane;
    uint4 na = sent, nb = sent;
    if (c < sg.c1) { na = ld_l2(g_s + (size_t)c * 8); nb = ld_l2(g_t + (size_t)c * 8); }
    for (int k = sg.res; k < sg.steps; ++k) {
      const uint4 a = na, b = nb;
      const int cc = c;
      c += 32;
      na = sent; nb = sent;
      if (k + 1 < sg.steps && c < sg.c1) { na = ld_l2(g_s + (size_t)c * 8); nb = ld_l2(g_t + (size_t)c * 8); }
      body(a, b, cc, cc < sg.c1);
    }
  }
}

__global__ void __launch_bounds__(RT, 1) rowsm_kernel(const RowParams P) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const uint4* res_s = reinterpret_cast<const uint4*>(smem + ROFF_S) + warp * RES_CHUNKS;
  const uint4* res_t = reinterpret_cast<const uint4*>(smem + ROFF_T) + warp * RES_CHUNKS;
  double* red = (double*)(smem + ROFF_RED);
  double* bc = (double*)(smem + ROFF_BC);
  float* wmax = (float*)(smem + ROFF_WMAX);
  uint64_t* mbar = (uint64_t*)(smem + ROFF_MBAR);

  const int V = P.V;
  const int n_chunks = V / 8;
  const int cpw = (n_chunks + RW - 1) / RW;
  Seg sg;
  sg.c0 = min(n_chunks, warp * cpw);
  sg.c1 = min(n_chunks, sg.c0 + cpw);
  sg.steps = (sg.c1 - sg.c0 + 31) / 32;
  sg.res = min(sg.steps, KS_MAX);
  const int res_chunks = min(sg.c1 - sg.c0, sg.res * 32);          // resident chunks of this warp
  const uint32_t res_bytes = (uint32_t)res_chunks * 16u;
  const int l2_first = sg.c0 + res_chunks;                          // first chunk read from global memory
  const uint32_t l2_bytes = (uint32_t)max(0, sg.c1 - l2_first) * 16u;

  const float c32 = (float)(1.4426950408889634 / (double)P.temperature);     // log2(e)/temperature
  Consts K;
  K.tau = (double)P.temperature; K.rtau = 1.0 / K.tau; K.eps = (double)P.eps; K.c64 = (double)c32;
  K.rc64 = 1.0 / K.c64; K.grad_scale = (double)P.grad_scale; K.sqrt_eps = sqrtf(P.eps); K.V = V;

  auto row_ptrs = [&](int64_t row, const __nv_bfloat16*& s, const __nv_bfloat16*& t) {
    const int64_t b = row / P.K1;
    const int j = (int)(row - b * P.K1);
    s = (const __nv_bfloat16*)P.s + b * P.s_seq + (int64_t)j * P.s_pos;
    t = (const __nv_bfloat16*)P.t + b * P.t_seq + (int64_t)j * P.t_pos;
  };
  // lane 0 of each warp: fetch the warp's resident part of `row`, and pull the rest towards L2
  auto issue = [&](int64_t row) {
    const __nv_bfloat16 *s, *t;
    row_ptrs(row, s, t);
    mbar_expect_tx(mbar, 2u * res_bytes);
    if (res_bytes) {
      bulk_load((void*)res_s, s + (size_t)sg.c0 * 8, res_bytes, mbar);
      bulk_load((void*)res_t, t + (size_t)sg.c0 * 8, res_bytes, mbar);
    }
    if (l2_bytes) {
      prefetch_l2(s + (size_t)l2_first * 8, l2_bytes);
      prefetch_l2(t + (size_t)l2_first * 8, l2_bytes);
    }
  };
  // sum (or minimum, from component n_sum on) of n per-warp vectors: warp 0 ends up with the totals in v[]
  auto combine = [&](double* v, int n, int n_sum) {
    if (lane == 0) {
#pragma unroll
      for (int k = 0; k < RNV; ++k) if (k < n) red[k * RW + warp] = v[k];
    }
    __syncthreads();
    if (warp == 0) {
#pragma unroll
      for (int k = 0; k < RNV; ++k) if (k < n) v[k] = (k < n_sum) ? warp_sum_d(red[k * RW + lane]) : warp_min_d(red[k * RW + lane]);
    }
  };

  if (tid == 0) {
    mbar_init(mbar, RW);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  __syncthreads();
  if (lane == 0 && (int64_t)blockIdx.x < P.n_rows) issue(blockIdx.x);
  uint32_t phase = 0;
  bool dead = false;

  for (int64_t row = blockIdx.x; row < P.n_rows; row += gridDim.x) {
    const uint64_t rid = P.row_offset + (uint64_t)row;
    const int64_t seq = row / P.K1;
    const int pos = (int)(row - seq * P.K1);
    const bool bonus = P.spec && (pos == P.K1 - 1);
    const int x = bonus ? 0 : (P.spec ? P.proposal[seq * P.prop_ld + pos] : P.proposal[row]);
    const bool masked = (P.mask != nullptr) && (P.mask[row] == 0);
    const __nv_bfloat16 *g_s, *g_t;
    row_ptrs(row, g_s, g_t);
    __nv_bfloat16* g_out = P.dlogits ? (__nv_bfloat16*)P.dlogits + row * P.ld_g : nullptr;
    const int64_t next_row = row + gridDim.x;
    bool next_issued = false;

    bool timed_out = dead;
    if (!dead) {
      if (!mbar_wait_bounded(mbar, phase)) timed_out = true;
      else phase ^= 1u;
    }

    // ------------------------------------------------ pass "max"
    float my_mt;
    {
      uint32_t a = 0xFF7FFF7Fu, b = 0xFF7FFF7Fu;
      for_each_chunk(sg, lane, res_s, res_t, g_s, g_t, [&](const uint4& s4, const uint4& t4, int, bool) {
        a = max_bf16x2(max_bf16x2(a, max_bf16x2(s4.x, s4.y)), max_bf16x2(s4.z, s4.w));
        b = max_bf16x2(max_bf16x2(b, max_bf16x2(t4.x, t4.y)), max_bf16x2(t4.z, t4.w));
      });
      const float2 fa = unpack_bf16x2(a), fb = unpack_bf16x2(b);
      my_mt = fmaxf(fb.x, fb.y);
      const float wa = warp_max_f(fmaxf(fa.x, fa.y)), wb = warp_max_f(my_mt);
      if (lane == 0) { wmax[warp] = wa; wmax[RW + warp] = wb; }
    }
    const int any_timeout = __syncthreads_or(timed_out ? 1 : 0);
    if (any_timeout) dead = true;
    const float ms = warp_max_f(wmax[lane]), mt = warp_max_f(wmax[RW + lane]);
    const float k0 = -ceilf(c32 * fmaxf(ms, -1e30f)), k1 = -ceilf(c32 * fmaxf(mt, -1e30f));   // shifts: arguments <= 0

    // row scalars that do not depend on the passes
    if (tid == 32) bc[BC_UACC] = scalar_uniform(P.seed, rid, STAGE_ACCEPT);
    if (tid == 64) bc[BC_UDRAW] = scalar_uniform(P.seed, rid, bonus ? STAGE_BONUS : STAGE_RESIDUAL);
    if (tid == 96) {
      const bool ok = (x >= 0 && x < V);
      bc[BC_SX] = ok ? (double)__bfloat162float(g_s[x]) : 0.0;
      bc[BC_TX] = ok ? (double)__bfloat162float(g_t[x]) : 0.0;
    }

    // teacher argmax: threads that saw the row maximum look for its lowest index
    double cand = CUDART_INF;
    if (my_mt == mt) {
      for_each_chunk(sg, lane, res_s, res_t, g_s, g_t, [&](const uint4&, const uint4& t4, int c, bool valid) {
        if (valid) {
          const uint32_t w[4] = {t4.x, t4.y, t4.z, t4.w};
#pragma unroll
          for (int k = 3; k >= 0; --k) {
            const float2 f = unpack_bf16x2(w[k]);
            if (f.y == mt) cand = fmin(cand, (double)(c * 8 + 2 * k + 1));
            if (f.x == mt) cand = fmin(cand, (double)(c * 8 + 2 * k));
          }
        }
      });
    }

    // ------------------------------------------------ pass "lse"
    {
      float2 Ss = splat(0.f), St = splat(0.f), M1 = splat(0.f), M2 = splat(0.f), M3 = splat(0.f), N1 = splat(0.f);
      const float2 cc = splat(c32), kk0 = splat(k0), kk1 = splat(k1), neg1 = splat(-1.f);
      for_each_chunk(sg, lane, res_s, res_t, g_s, g_t, [&](const uint4& s4, const uint4& t4, int, bool) {
        const uint32_t sw[4] = {s4.x, s4.y, s4.z, s4.w}, tw[4] = {t4.x, t4.y, t4.z, t4.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float2 sf = unpack_bf16x2(sw[i]), tf = unpack_bf16x2(tw[i]);
          const float2 d = __ffma2_rn(sf, neg1, tf);
          const float2 es = ex2f2(__ffma2_rn(sf, cc, kk0));
          const float2 et = ex2f2(__ffma2_rn(tf, cc, kk1));
          Ss = __fadd2_rn(Ss, es);
          St = __fadd2_rn(St, et);
          const float2 t1 = __fmul2_rn(es, d);
          M1 = __fadd2_rn(M1, t1);
          const float2 t2 = __fmul2_rn(t1, d);
          M2 = __fadd2_rn(M2, t2);
          M3 = __ffma2_rn(t2, d, M3);
          N1 = __ffma2_rn(et, d, N1);
        }
      });
      auto tot = [](const float2 a) { return (double)a.x + (double)a.y; };
      double v[7] = {warp_sum_d(tot(Ss)), warp_sum_d(tot(St)), warp_sum_d(tot(M1)), warp_sum_d(tot(M2)),
                     warp_sum_d(tot(M3)), warp_sum_d(tot(N1)), warp_min_d(cand)};
      combine(v, 7, 6);
      if (tid == 0) scalar_after_lse(bc, v, K, k0, k1, x, bonus, masked, dead);
      __syncthreads();
    }

    // ------------------------------------------------ pass "solve" (repeated)
    while ((int)bc[BC_MODE] == MODE_SOLVE) {
      const float cb = (float)bc[BC_CB], kb = (float)bc[BC_KB];
      float2 S0 = splat(0.f), S1 = splat(0.f), S2 = splat(0.f);
      const float2 cc = splat(c32), cbb = splat(cb), kbb = splat(kb), neg1 = splat(-1.f);
      for_each_chunk(sg, lane, res_s, res_t, g_s, g_t, [&](const uint4& s4, const uint4& t4, int, bool) {
        const uint32_t sw[4] = {s4.x, s4.y, s4.z, s4.w}, tw[4] = {t4.x, t4.y, t4.z, t4.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float2 sf = unpack_bf16x2(sw[i]), tf = unpack_bf16x2(tw[i]);
          const float2 d = __ffma2_rn(sf, neg1, tf);
          const float2 e = ex2f2(__ffma2_rn(d, cbb, __ffma2_rn(sf, cc, kbb)));
          S0 = __fadd2_rn(S0, e);
          const float2 t1 = __fmul2_rn(e, d);
          S1 = __fadd2_rn(S1, t1);
          S2 = __ffma2_rn(t1, d, S2);
        }
      });
      auto tot = [](const float2 a) { return (double)a.x + (double)a.y; };
      double v[3] = {warp_sum_d(tot(S0)), warp_sum_d(tot(S1)), warp_sum_d(tot(S2))};
      combine(v, 3, 3);
      if (tid == 0) scalar_after_solve(bc, v, K, k0, k1, x, bonus, masked);
      __syncthreads();
    }

    // ------------------------------------------------ flagged row: zero outputs, zero gradient
    if ((int)bc[BC_MODE] == MODE_FLAGGED) {
      if (tid == 0) {
        write_row(P.out, row, zero_row((uint32_t)bc[BC_STATUS]), !P.spec);
        atomicAdd(P.flagged, 1ull);
      }
      if (g_out) {
        for (int k = 0; k < sg.steps; ++k) {
          const int c = sg.c0 + k * 32 + lane;
          if (c < sg.c1) __stcs(reinterpret_cast<uint4*>(g_out + (size_t)c * 8), make_uint4(0, 0, 0, 0));
        }
      }
      __syncwarp();
      if (lane == 0 && !dead && next_row < P.n_rows) {
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        issue(next_row);
      }
      __syncthreads();   // the broadcast area is rewritten by the next row
      continue;
    }

    // ------------------------------------------------ pass "final"
    const bool need_draw = bonus || bc[BC_CORR] != 0.0;
    const float cl = (float)bc[BC_CL], kq = (float)bc[BC_KQ];
    const float iq = (float)bc[BC_IQ], ip = (float)bc[BC_IP];
    const int tok = (int)bc[BC_TOK];
    const float KGf = (float)bc[BC_KG];
    const float kg = (float)(bc[BC_KG] * (double)ip);     // gradient entry = e_p * kg
    float warp_part;   // this warp's ordered weight for the inverse-CDF draw
    {
      const bool want_g = (g_out != nullptr);
      float2 Sq = splat(0.f), R = splat(0.f);
      const float2 cc = splat(c32), cll = splat(cl), kqq = splat(kq), kk0 = splat(k0), neg1 = splat(-1.f);
      const float2 iqq = splat(iq), nip = splat(-ip), kgg = splat(kg);
      int n_res_done = 0;
      for_each_chunk(sg, lane, res_s, res_t, g_s, g_t, [&](const uint4& s4, const uint4& t4, int c, bool valid) {
        const uint32_t sw[4] = {s4.x, s4.y, s4.z, s4.w}, tw[4] = {t4.x, t4.y, t4.z, t4.w};
        uint32_t gp[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float2 sf = unpack_bf16x2(sw[i]), tf = unpack_bf16x2(tw[i]);
          const float2 d = __ffma2_rn(sf, neg1, tf);
          const float2 ep = ex2f2(__ffma2_rn(sf, cc, kk0));
          const float2 eq = ex2f2(__ffma2_rn(d, cll, __ffma2_rn(sf, cc, kqq)));
          Sq = __fadd2_rn(Sq, eq);
          float2 r = __ffma2_rn(eq, iqq, __fmul2_rn(ep, nip));     // q_i - p_i
          r.x = fmaxf(r.x, 0.f); r.y = fmaxf(r.y, 0.f);
          R = __fadd2_rn(R, r);
          const float2 gv = __fmul2_rn(ep, kgg);
          gp[i] = pack_bf16x2(gv.x, gv.y);
        }
        if ((tok >> 3) == c && tok >= 0) {   // the supervised token is in this chunk: subtract the one-hot part
          const int e = tok & 7, wi = e >> 1;
          const uint32_t word = wi == 0 ? sw[0] : wi == 1 ? sw[1] : wi == 2 ? sw[2] : sw[3];
          const float2 sf = unpack_bf16x2(word);
          const float ep = ex2f(fmaf((e & 1) ? sf.y : sf.x, c32, k0));
          const uint32_t g16 = (uint32_t)__bfloat16_as_ushort(__float2bfloat16_rn(fmaf(ep, kg, -KGf)));
          const uint32_t old = wi == 0 ? gp[0] : wi == 1 ? gp[1] : wi == 2 ? gp[2] : gp[3];
          const uint32_t neu = (e & 1) ? ((old & 0x0000ffffu) | (g16 << 16)) : ((old & 0xffff0000u) | g16);
          if (wi == 0) gp[0] = neu; else if (wi == 1) gp[1] = neu; else if (wi == 2) gp[2] = neu; else gp[3] = neu;
        }
        if (want_g && valid) __stcs(reinterpret_cast<uint4*>(g_out + (size_t)c * 8), make_uint4(gp[0], gp[1], gp[2], gp[3]));
        // once the warp has read its resident part for the last time, the next row's may land there
        // (a row that still needs its draw re-reads the resident part: its copy is issued after the draw)
        if (++n_res_done == sg.res && !need_draw) {
          __syncwarp();
          if (lane == 0 && !dead && next_row < P.n_rows) {
            asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
            issue(next_row);
          }
          next_issued = true;
        }
      });
      if (!next_issued && !need_draw && lane == 0 && !dead && next_row < P.n_rows) issue(next_row);   // no elements
      const float sq_f = Sq.x + Sq.y, r_f = R.x + R.y;
      const double part = warp_sum_d((double)(bonus ? sq_f * iq : r_f));
      warp_part = (float)part;
      double v[3] = {warp_sum_d((double)sq_f), warp_sum_d((double)r_f), part};
      combine(v, 2, 2);
      if (lane == 0) red[2 * RW + warp] = part;     // ordered per-warp weights (read after the next barrier)
      if (tid == 0) {
        bc[BC_TV] = (bc[BC_LAMBDA] > 0.0) ? v[1] : 0.0;
        if (!need_draw) write_result(bc, P.out, !P.spec, row, 0, x, false, K.c64, g_s, g_t);
      }
    }
    (void)warp_part;

    // ------------------------------------------------ the draw (corrected and bonus rows only)
    if (need_draw) {
      __syncthreads();
      if (tid == 0) scalar_find_owner(bc, red + 2 * RW, RW);
      __syncthreads();
      if (warp == (int)bc[BC_OWNER_WARP]) {
        const double target = bc[BC_TARGET];
        const bool last_mode = bc[BC_TAKE_LAST] != 0.0;
        double running = bc[BC_BEFORE];
        int y = -1, last_pos = -1;
        const float2 cc = splat(c32), cll = splat(cl), kqq = splat(kq), kk0 = splat(k0), neg1 = splat(-1.f);
        for_each_chunk(sg, lane, res_s, res_t, g_s, g_t, [&](const uint4& s4, const uint4& t4, int c, bool valid) {
          if (y >= 0) return;
          const uint32_t sw[4] = {s4.x, s4.y, s4.z, s4.w}, tw[4] = {t4.x, t4.y, t4.z, t4.w};
          float w[8];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float2 sf = unpack_bf16x2(sw[i]), tf = unpack_bf16x2(tw[i]);
            const float2 d = __ffma2_rn(sf, neg1, tf);
            const float2 ep = ex2f2(__ffma2_rn(sf, cc, kk0));
            const float2 eq = ex2f2(__ffma2_rn(d, cll, __ffma2_rn(sf, cc, kqq)));
            w[2 * i] = bonus ? eq.x * iq : fmaxf(fmaf(eq.x, iq, -(ep.x * ip)), 0.f);
            w[2 * i + 1] = bonus ? eq.y * iq : fmaxf(fmaf(eq.y, iq, -(ep.y * ip)), 0.f);
          }
          double mine = 0.0;
#pragma unroll
          for (int i = 0; i < 8; ++i) mine += valid ? (double)w[i] : 0.0;
          double inc = mine;
#pragma unroll
          for (int o = 1; o < 32; o <<= 1) {
            const double up = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += up;
          }
          const unsigned posm = __ballot_sync(0xffffffffu, mine > 0.0);
          const unsigned hit = last_mode ? 0u : __ballot_sync(0xffffffffu, running + inc > target);
          int found = -1, lastp = -1;
          if (hit && lane == __ffs(hit) - 1) {           // walk the 8 elements of the crossing chunk
            double run = running + inc - mine;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
              run += (double)w[i];
              if (found < 0 && run > target) found = c * 8 + i;
            }
            if (found < 0) {                              // rounding: last positive element of the chunk
#pragma unroll
              for (int i = 0; i < 8; ++i) if (w[i] > 0.f) found = c * 8 + i;
            }
          }
          if (posm && lane == 31 - __clz(posm)) {
#pragma unroll
            for (int i = 0; i < 8; ++i) if (w[i] > 0.f) lastp = c * 8 + i;
          }
          if (hit) y = __shfl_sync(0xffffffffu, found, __ffs(hit) - 1);
          if (posm) last_pos = __shfl_sync(0xffffffffu, lastp, 31 - __clz(posm));
          running += __shfl_sync(0xffffffffu, inc, 31);
        });
        if (y < 0) y = (last_pos >= 0) ? last_pos : min(V - 1, sg.c1 * 8 - 1);
        if (lane == 0) write_result(bc, P.out, !P.spec, row, bonus ? 0 : 1, y, bonus, K.c64, g_s, g_t);
      }
      __syncwarp();
      if (lane == 0 && !dead && next_row < P.n_rows) {
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        issue(next_row);
      }
    }
    __syncthreads();   // the broadcast area and the partial-sum area are rewritten by the next row
  }

  // a CTA that gave up on a copy still waits (bounded) for what it has in flight before leaving
  if (dead && tid == 0) (void)mbar_wait_bounded(mbar, phase);
}

// ---------------------------------------------------------------- host side
bool rowsm_can_serve(const RowParams& p, int dtype) {
  if (dtype != SAKI_BF16) return false;
  if (p.V < 2048 || p.V % 8 != 0) return false;
  auto al16 = [](const void* q) { return ((uintptr_t)q & 15) == 0; };
  if (!al16(p.s) || !al16(p.t)) return false;
  if (p.s_seq % 8 || p.s_pos % 8 || p.t_seq % 8 || p.t_pos % 8) return false;
  if (p.dlogits && (!al16(p.dlogits) || p.ld_g % 8)) return false;
  return true;
}

cudaError_t launch_rowsm(const RowParams& p, cudaStream_t st, int* n_launches, bool* served) {
  *served = false;
  if (p.n_rows <= 0) { *served = true; return cudaSuccess; }
  static std::mutex mu;
  static int cached_dev = -1, cached_sms = 0;
  int dev = 0;
  cudaGetDevice(&dev);
  {
    std::lock_guard<std::mutex> lock(mu);
    if (cached_dev != dev) {
      cudaError_t e = cudaFuncSetAttribute(rowsm_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, RSMEM_BYTES);
      if (e != cudaSuccess) return e;
      e = cudaDeviceGetAttribute(&cached_sms, cudaDevAttrMultiProcessorCount, dev);
      if (e != cudaSuccess) return e;
      cached_dev = dev;
    }
  }
  const int grid = (int)(p.n_rows < cached_sms ? p.n_rows : cached_sms);
  rowsm_kernel<<<grid, RT, RSMEM_BYTES, st>>>(p);
  cudaError_t e = cudaGetLastError();
  if (e == cudaSuccess) { *served = true; if (n_launches) *n_launches += 1; }
  return e;
}

}  // namespace saki
