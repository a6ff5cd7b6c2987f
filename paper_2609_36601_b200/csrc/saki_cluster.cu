// Register-resident cluster kernel for bf16 rows: the latency path (calls of a few long rows).
//
// One vocabulary row per thread-block cluster of CS CTAs x 256 threads, two
// CTAs resident per SM.  Each CTA owns a contiguous slice of the row; each
// thread owns 80 contiguous elements of it, held for the whole row in
// registers as the raw packed bf16 pairs (40 + 40 registers), so the row pair
// is read from HBM exactly once.  The single shared-memory slot of a CTA is
// only the landing zone of the NEXT row's slice, fetched by one 1-D bulk
// async copy per row (cp.async.bulk + mbarrier) while the current row is
// being computed.  Passes over the registers:
//   lse      2 exponentials/element: both log-sum-exps (computed under the
//            CTA's own maxima rounded up to whole powers of two, then moved
//            exactly onto the row's maxima, which the CTAs exchange while the
//            pass runs), moments of the teacher-student logit difference under
//            p (initial guess of lambda), KL(T||p) (saturation test), teacher
//            argmax index
//   solve    1 exponential/element per evaluation of KL(q_beta||p) and the first
//            four cumulants of the logit difference under q_beta; lambda = root of
//            the fourth-order Taylor model inside a bisection bracket, one
//            evaluation for most rows (Eqs. "bridge", "trust_region")
//   final    2 exponentials/element: TV = sum [q-p]_+ with per-thread ordered
//            partial sums for the inverse-CDF residual draw (Eqs. "accept",
//            "residual"), and the gradient row written straight from
//            registers (Eq. "general_objective")
// Per-element work is float32 (packed f32x2 FMAs, ex2.approx); every
// cross-thread combination and every per-row scalar is float64.  Per-warp
// partial sums travel to all CTAs of the cluster as asynchronous
// distributed-shared-memory stores that complete on the receiver's mbarrier
// (no cluster barrier, no fence on the row loop); each CTA then forms the
// same scalars redundantly from the same numbers in the same order, so
// control flow is uniform across the cluster.
#include "saki_device.cuh"
#include <cooperative_groups.h>
#include <math_constants.h>
#include <mutex>

namespace cg = cooperative_groups;

namespace saki {

constexpr int CT = 256;                 // threads per CTA
constexpr int CW = CT / 32;             // warps per CTA
constexpr int CHUNKS = 10;              // 16-byte chunks (8 bf16) per thread per row
constexpr int EPT = CHUNKS * 8;         // elements per thread
constexpr int NPAIR = EPT / 2;          // packed registers per thread per row
constexpr int SLICE_CAP = CT * EPT;     // elements of one row a CTA can hold
constexpr int MAX_CS = 8;
constexpr int NSLOT = MAX_CS * CW;      // per-warp partial slots of a cluster
constexpr int NV = 8;                   // doubles per partial vector
constexpr uint32_t SENTINEL = 0xFF7FFF7Fu;   // two bf16 "most negative finite": exp -> 0, difference 0

constexpr int OFF_S = 0;
constexpr int OFF_T = SLICE_CAP * 2;
constexpr int OFF_RED = OFF_T + SLICE_CAP * 2;                  // [2][NV][NSLOT] doubles: per-warp partials
constexpr int OFF_MX = OFF_RED + 2 * NV * NSLOT * 8;            // [2][MAX_CS][2] doubles: per-CTA maxima
constexpr int OFF_GAT = OFF_MX + 2 * MAX_CS * 2 * 8;            // [NV] doubles: cluster totals
constexpr int OFF_BC = OFF_GAT + NV * 8;                        // [2][BC_DOUBLES] broadcast scalars
constexpr int OFF_WMAX = OFF_BC + 2 * BC_DOUBLES * 8;           // [2][2][CW] floats: per-warp maxima
constexpr int OFF_SCR = OFF_WMAX + 2 * 2 * CW * 4;              // [2][EPT] bf16: one thread's elements in index order
constexpr int OFF_MBAR = OFF_SCR + 2 * EPT * 2;                 // copy barrier, 2 exchange barriers, 2 maxima barriers
constexpr int SMEM_BYTES = OFF_MBAR + 5 * 8 + 8;
static_assert(OFF_MBAR % 8 == 0 && OFF_SCR % 16 == 0, "alignment");

template <int CS>
__global__ void __launch_bounds__(CT, 2) cluster_kernel(const RowParams P, const int n_clusters) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const unsigned rank = cg::this_cluster().block_rank();
  const int cluster_id = blockIdx.x / CS;

  const __nv_bfloat16* slot_s = (const __nv_bfloat16*)(smem + OFF_S);
  const __nv_bfloat16* slot_t = (const __nv_bfloat16*)(smem + OFF_T);
  double* red = (double*)(smem + OFF_RED);
  double* mx = (double*)(smem + OFF_MX);
  double* gat = (double*)(smem + OFF_GAT);
  float* wmax = (float*)(smem + OFF_WMAX);
  uint64_t* mbar = (uint64_t*)(smem + OFF_MBAR);   // [0] row copy, [1..2] partial exchange, [3..4] maxima exchange
  const uint32_t red_s = smem_addr(red), mx_s = smem_addr(mx), bar_s = smem_addr(mbar);

  const int V = P.V;
  const int slice_len = ((V + CS - 1) / CS + 7) & ~7;
  const int slice_start = (int)rank * slice_len;
  const int my_len = max(0, min(slice_len, V - slice_start));
  const uint32_t slice_bytes = (uint32_t)my_len * 2u;
  const int rot = (tid >> 2) & 1;          // chunk rotation: conflict-free 128-bit shared loads
  const int thr_first = tid * EPT;         // first element (within the slice) of this thread

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
  auto issue = [&](int64_t row) {   // one thread: fetch this CTA's slice of both rows
    const __nv_bfloat16 *s, *t;
    row_ptrs(row, s, t);
    mbar_expect_tx(&mbar[0], 2u * slice_bytes);
    if (slice_bytes) {
      bulk_load(smem + OFF_S, s + slice_start, slice_bytes, &mbar[0]);
      bulk_load(smem + OFF_T, t + slice_start, slice_bytes, &mbar[0]);
    }
  };
  // one exchange: every warp sends its N-vector to slot rank*CW+warp of red[p] in every CTA
  auto push = [&](const double* v, int n, int p) {
    if (lane < CS) {
      const uint32_t dst = map_to_rank(red_s + (uint32_t)(((p * NV) * NSLOT + rank * CW + warp) * 8), lane);
      const uint32_t bar = map_to_rank(bar_s + (uint32_t)((1 + p) * 8), lane);
#pragma unroll
      for (int k = 0; k < NV; ++k)
        if (k < n) st_async_f64(dst + (uint32_t)(k * NSLOT * 8), v[k], bar);
    }
  };
  // cluster total of component k (fixed order, the same in every CTA); is_min: minimum instead of sum
  auto gather = [&](int p, int k, bool is_min) {
    const double* base = red + (size_t)(p * NV + k) * NSLOT;
    double a = is_min ? CUDART_INF : 0.0;
    for (int slot = lane; slot < CS * CW; slot += 32) a = is_min ? fmin(a, base[slot]) : a + base[slot];
    return is_min ? warp_min(a) : warp_sum(a);
  };

  if (tid == 0) {
#pragma unroll
    for (int i = 0; i < 5; ++i) mbar_init(&mbar[i], 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  cg::this_cluster().sync();   // every CTA's barriers exist before any peer signals them
  if (tid == 0 && cluster_id < P.n_rows) issue(cluster_id);
  uint32_t phase = 0, xph0 = 0, xph1 = 0, mph0 = 0, mph1 = 0;
  int parity = 0, rb = 0;
  bool dead = false;   // a wait timed out: this CTA stops fetching and the cluster flags its rows

  for (int64_t row = cluster_id; row < P.n_rows; row += n_clusters, rb ^= 1) {
    double* bc = (double*)(smem + OFF_BC) + rb * BC_DOUBLES;
    const uint64_t rid = P.row_offset + (uint64_t)row;
    const int64_t seq = row / P.K1;
    const int pos = (int)(row - seq * P.K1);
    const bool bonus = P.spec && (pos == P.K1 - 1);
    const int x = bonus ? 0 : (P.spec ? P.proposal[seq * P.prop_ld + pos] : P.proposal[row]);
    const bool masked = (P.mask != nullptr) && (P.mask[row] == 0);
    const __nv_bfloat16 *g_s, *g_t;
    row_ptrs(row, g_s, g_t);
    __nv_bfloat16* g_out = P.dlogits ? (__nv_bfloat16*)P.dlogits + row * P.ld_g : nullptr;

    // ------------------------------------------------ stage: shared slot -> registers
    bool timed_out = dead;
    if (!dead) {
      if (!mbar_wait_bounded(&mbar[0], phase)) timed_out = true;
      else phase ^= 1u;
    }
    uint32_t sr[NPAIR], tr[NPAIR];
#pragma unroll
    for (int j = 0; j < CHUNKS; ++j) {
      int cj = j + rot;
      if (cj == CHUNKS) cj = 0;
      const int e0 = thr_first + cj * 8;
      uint4 a = make_uint4(SENTINEL, SENTINEL, SENTINEL, SENTINEL), b = a;
      if (e0 < my_len && !timed_out) {
        a = *reinterpret_cast<const uint4*>(slot_s + e0);
        b = *reinterpret_cast<const uint4*>(slot_t + e0);
      }
      sr[4 * j + 0] = a.x; sr[4 * j + 1] = a.y; sr[4 * j + 2] = a.z; sr[4 * j + 3] = a.w;
      tr[4 * j + 0] = b.x; tr[4 * j + 1] = b.y; tr[4 * j + 2] = b.z; tr[4 * j + 3] = b.w;
    }
    // maxima of this CTA's slice (packed bf16), via shuffles and one CTA barrier
    float my_mt;
    {
      uint32_t a = sr[0], b = tr[0];
#pragma unroll
      for (int i = 1; i < NPAIR; ++i) {
        a = max_bf16x2(a, sr[i]);
        b = max_bf16x2(b, tr[i]);
      }
      const float2 fb0 = unpack_bf16x2(b);
      my_mt = fmaxf(fb0.x, fb0.y);
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        a = max_bf16x2(a, __shfl_xor_sync(0xffffffffu, a, o));
        b = max_bf16x2(b, __shfl_xor_sync(0xffffffffu, b, o));
      }
      if (lane == 0) {
        const float2 fa = unpack_bf16x2(a), fb = unpack_bf16x2(b);
        wmax[(rb * 2 + 0) * CW + warp] = fmaxf(fa.x, fa.y);
        wmax[(rb * 2 + 1) * CW + warp] = fmaxf(fb.x, fb.y);
      }
    }
    const int any_timeout = __syncthreads_or(timed_out ? 1 : 0);   // also: every thread has drained the slot
    if (any_timeout) dead = true;
    if (tid == 0) {
      const int64_t next = row + n_clusters;
      if (!dead && next < P.n_rows) {
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        issue(next);
      }
      mbar_expect_tx(&mbar[3 + rb], (uint32_t)(CS * 16));          // maxima of all CTAs
      mbar_expect_tx(&mbar[1 + parity], (uint32_t)(CS * CW * 8 * 8));   // partials of pass "lse"
    }
    float ms_r = wmax[(rb * 2 + 0) * CW], mt_r = wmax[(rb * 2 + 1) * CW];
#pragma unroll
    for (int w = 1; w < CW; ++w) {
      ms_r = fmaxf(ms_r, wmax[(rb * 2 + 0) * CW + w]);
      mt_r = fmaxf(mt_r, wmax[(rb * 2 + 1) * CW + w]);
    }
    if (tid < CS) {   // this CTA's maxima to every CTA (a CTA that timed out sends NaN: the row is flagged)
      const uint32_t dst = map_to_rank(mx_s + (uint32_t)(((rb * MAX_CS) + rank) * 16), tid);
      const uint32_t bar = map_to_rank(bar_s + (uint32_t)((3 + rb) * 8), tid);
      st_async_f64(dst, dead ? CUDART_NAN : (double)ms_r, bar);
      st_async_f64(dst + 8, (double)mt_r, bar);
    }
    // whole-number shifts: every exponent argument is <= 0, and sums taken under different
    // shifts differ by exact powers of two
    const float k0r = -ceilf(c32 * fmaxf(ms_r, -1e30f)), k1r = -ceilf(c32 * fmaxf(mt_r, -1e30f));

    // row scalars that do not depend on the passes, fetched off the critical path
    if (tid == 32) bc[BC_UACC] = scalar_uniform(P.seed, rid, STAGE_ACCEPT);
    if (tid == 64) bc[BC_UDRAW] = scalar_uniform(P.seed, rid, bonus ? STAGE_BONUS : STAGE_RESIDUAL);
    if (tid == 96) {
      const bool ok = (x >= 0 && x < V);
      bc[BC_SX] = ok ? (double)__bfloat162float(g_s[x]) : 0.0;
      bc[BC_TX] = ok ? (double)__bfloat162float(g_t[x]) : 0.0;
    }

    // teacher argmax candidate of this thread (exact compare on stored values, lowest index)
    double cand = CUDART_INF;
    if (my_mt == mt_r) {
#pragma unroll
      for (int j = 0; j < CHUNKS; ++j) {
        int cj = j + rot;
        if (cj == CHUNKS) cj = 0;
        const int e0 = slice_start + thr_first + cj * 8;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const float2 f = unpack_bf16x2(tr[4 * j + k]);
          if (f.x == mt_r) cand = fmin(cand, (double)(e0 + 2 * k));
          if (f.y == mt_r) cand = fmin(cand, (double)(e0 + 2 * k + 1));
        }
      }
    }

    // ------------------------------------------------ pass "lse"
    float k0, k1;        // the row's shifts
    bool row_timeout;
    {
      float2 Ss = splat(0.f), St = splat(0.f), M1 = splat(0.f), M2 = splat(0.f), M3 = splat(0.f), M4 = splat(0.f),
             N1 = splat(0.f);
      const float2 cc = splat(c32), kk0 = splat(k0r), kk1 = splat(k1r), neg1 = splat(-1.f);
#pragma unroll
      for (int i = 0; i < NPAIR; ++i) {
        const float2 sf = unpack_fresh(sr[i]), tf = unpack_fresh(tr[i]);
        const float2 d = ffma2(sf, neg1, tf);
        const float2 es = ex2f2(ffma2(sf, cc, kk0));
        const float2 et = ex2f2(ffma2(tf, cc, kk1));
        Ss = fadd2(Ss, es);
        St = fadd2(St, et);
        const float2 t1 = fmul2(es, d);
        M1 = fadd2(M1, t1);
        const float2 t2 = fmul2(t1, d);
        M2 = fadd2(M2, t2);
        M3 = ffma2(t2, d, M3);
        M4 = ffma2(t2, fmul2(d, d), M4);
        N1 = ffma2(et, d, N1);
      }
      // the row's maxima have arrived meanwhile: move the partial sums onto the row's shifts
      bool mx_timeout = false;
      if (!mbar_wait_bounded(&mbar[3 + rb], rb ? mph1 : mph0)) mx_timeout = true;
      if (rb) mph1 ^= 1u; else mph0 ^= 1u;
      float gms = -CUDART_INF_F, gmt = -CUDART_INF_F;
      bool poisoned = mx_timeout;
#pragma unroll
      for (int r = 0; r < CS; ++r) {
        const double a = mx[(rb * MAX_CS + r) * 2 + 0], b = mx[(rb * MAX_CS + r) * 2 + 1];
        if (a != a) poisoned = true;
        gms = fmaxf(gms, (float)a); gmt = fmaxf(gmt, (float)b);
      }
      row_timeout = poisoned;
      if (mx_timeout) dead = true;
      k0 = -ceilf(c32 * fmaxf(gms, -1e30f)); k1 = -ceilf(c32 * fmaxf(gmt, -1e30f));
      const double fs = pow2_exact((int)(k0 - k0r)), ft = pow2_exact((int)(k1 - k1r));
      auto tot = [](const float2 a) { return (double)a.x + (double)a.y; };
      double v[8] = {fs * tot(Ss), ft * tot(St), fs * tot(M1), fs * tot(M2), fs * tot(M3), ft * tot(N1),
                     (mt_r == gmt) ? cand : CUDART_INF, fs * tot(M4)};
#pragma unroll
      for (int k = 0; k < 6; ++k) v[k] = warp_sum(v[k]);
      v[6] = warp_min(v[6]);
      v[7] = warp_sum(v[7]);
      push(v, 8, parity);
      if (warp < 8) {
        if (!mbar_wait_bounded(&mbar[1 + parity], parity ? xph1 : xph0)) dead = true;
        const double g = gather(parity, warp, warp == 6);
        if (lane == 0) gat[warp] = g;
      }
      if (parity) xph1 ^= 1u; else xph0 ^= 1u;
      parity ^= 1;
      __syncthreads();
      if (tid == 0) {
        scalar_after_lse(bc, gat, K, k0, k1, x, bonus, masked, row_timeout, gat + 7);
        if ((int)bc[BC_MODE] == MODE_SOLVE) mbar_expect_tx(&mbar[1 + parity], (uint32_t)(CS * CW * 5 * 8));
        else if ((int)bc[BC_MODE] == MODE_FINAL) mbar_expect_tx(&mbar[1 + parity], (uint32_t)(CS * CW * 3 * 8));
      }
      __syncthreads();
    }

    // ------------------------------------------------ pass "solve" (repeated)
    while ((int)bc[BC_MODE] == MODE_SOLVE) {
      const float cb = (float)bc[BC_CB], kb = (float)bc[BC_KB];
      float2 S0[2] = {splat(0.f), splat(0.f)}, S1[2] = {splat(0.f), splat(0.f)}, S2[2] = {splat(0.f), splat(0.f)},
             S3[2] = {splat(0.f), splat(0.f)}, S4[2] = {splat(0.f), splat(0.f)};
      const float2 cc = splat(c32), cbb = splat(cb), kbb = splat(kb), neg1 = splat(-1.f);
#pragma unroll
      for (int i = 0; i < NPAIR; ++i) {
        const int h = i & 1;
        const float2 sf = unpack_fresh(sr[i]), tf = unpack_fresh(tr[i]);
        const float2 d = ffma2(sf, neg1, tf);
        const float2 e = ex2f2(ffma2(d, cbb, ffma2(sf, cc, kbb)));
        S0[h] = fadd2(S0[h], e);
        const float2 t1 = fmul2(e, d);
        S1[h] = fadd2(S1[h], t1);
        const float2 t2 = fmul2(t1, d);
        S2[h] = fadd2(S2[h], t2);
        S3[h] = ffma2(t2, d, S3[h]);
        S4[h] = ffma2(t2, fmul2(d, d), S4[h]);
      }
      auto tot = [](const float2 (&a)[2]) { return ((double)a[0].x + (double)a[0].y) + ((double)a[1].x + (double)a[1].y); };
      double v[5] = {warp_sum(tot(S0)), warp_sum(tot(S1)), warp_sum(tot(S2)), warp_sum(tot(S3)), warp_sum(tot(S4))};
      push(v, 5, parity);
      if (warp < 5) {
        if (!mbar_wait_bounded(&mbar[1 + parity], parity ? xph1 : xph0)) dead = true;
        const double g = gather(parity, warp, false);
        if (lane == 0) gat[warp] = g;
      }
      if (parity) xph1 ^= 1u; else xph0 ^= 1u;
      parity ^= 1;
      __syncthreads();
      if (tid == 0) {
        scalar_after_solve4(bc, gat, K, k0, k1, x, bonus, masked);
        if ((int)bc[BC_MODE] == MODE_SOLVE) mbar_expect_tx(&mbar[1 + parity], (uint32_t)(CS * CW * 5 * 8));   // next evaluation
        else if ((int)bc[BC_MODE] == MODE_FINAL) mbar_expect_tx(&mbar[1 + parity], (uint32_t)(CS * CW * 3 * 8));   // pass "final"
      }
      __syncthreads();
    }

    // ------------------------------------------------ flagged row: zero outputs, zero gradient
    if ((int)bc[BC_MODE] == MODE_FLAGGED || (int)bc[BC_MODE] == MODE_REDO) {
      const bool redo = (int)bc[BC_MODE] == MODE_REDO;   // ill-conditioned for float32: the float64 kernel routes it
      if (rank == 0 && tid == 0) {
        if (redo) {
          const unsigned int slot = atomicAdd(P.redo_count, 1u);
          P.redo_list[slot] = (int32_t)row;
          if (P.redo_guess) P.redo_guess[slot] = (float)bc[BC_BETA];     // where the float64 kernel starts its iteration
        }
        else {
          write_row(P.out, row, zero_row((uint32_t)bc[BC_STATUS]), !P.spec);
          atomicAdd(P.flagged, 1ull);
        }
      }
      if (g_out && !redo) {
#pragma unroll
        for (int j = 0; j < CHUNKS; ++j) {
          int cj = j + rot;
          if (cj == CHUNKS) cj = 0;
          const int e0 = thr_first + cj * 8;
          if (e0 < my_len) *reinterpret_cast<uint4*>(g_out + slice_start + e0) = make_uint4(0, 0, 0, 0);
        }
      }
      continue;
    }

    // ------------------------------------------------ pass "final"
    const bool need_draw = bonus || bc[BC_CORR] != 0.0;
    float my_part;       // this thread's ordered weight for the inverse-CDF draw
    const float cl = (float)bc[BC_CL], kq = (float)bc[BC_KQ];
    const float iq = (float)bc[BC_IQ], ip = (float)bc[BC_IP];
    {
      const float KGf = (float)bc[BC_KG];
      const float kg = (float)(bc[BC_KG] * (double)ip);     // gradient entry = e_p * kg
      const bool want_g = (g_out != nullptr);
      float2 Sq[2] = {splat(0.f), splat(0.f)}, R[2] = {splat(0.f), splat(0.f)};
      const float2 cc = splat(c32), cll = splat(cl), kqq = splat(kq), kk0 = splat(k0), neg1 = splat(-1.f);
      const float2 iqq = splat(iq), nip = splat(-ip), kgg = splat(kg);
#pragma unroll
      for (int j = 0; j < CHUNKS; ++j) {
        uint32_t gp[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const int i = 4 * j + k, h = k & 1;
          const float2 sf = unpack_fresh(sr[i]), tf = unpack_fresh(tr[i]);
          const float2 d = ffma2(sf, neg1, tf);
          const float2 ep = ex2f2(ffma2(sf, cc, kk0));
          const float2 eq = ex2f2(ffma2(d, cll, ffma2(sf, cc, kqq)));
          Sq[h] = fadd2(Sq[h], eq);
          float2 r = ffma2(eq, iqq, fmul2(ep, nip));     // q_i - p_i
          r.x = fmaxf(r.x, 0.f); r.y = fmaxf(r.y, 0.f);
          R[h] = fadd2(R[h], r);
          const float2 gv = fmul2(ep, kgg);
          gp[k] = pack_bf16x2(gv.x, gv.y);
        }
        if (want_g) {
          int cj = j + rot;
          if (cj == CHUNKS) cj = 0;
          const int e0 = thr_first + cj * 8;
          if (e0 < my_len) *reinterpret_cast<uint4*>(g_out + slice_start + e0) = make_uint4(gp[0], gp[1], gp[2], gp[3]);
        }
      }
      const float sq_f = (Sq[0].x + Sq[0].y) + (Sq[1].x + Sq[1].y);
      const float r_f = (R[0].x + R[0].y) + (R[1].x + R[1].y);
      my_part = bonus ? sq_f * iq : r_f;
      // the thread that owns the supervised token subtracts the one-hot part of the gradient
      if (want_g) {
        const int tok = (int)bc[BC_TOK];
        const int loc = tok - slice_start - thr_first;
        if (tok >= 0 && loc >= 0 && loc < EPT && tok - slice_start < my_len) {
          const float ep = ex2f(fmaf(__bfloat162float(g_s[tok]), c32, k0));
          g_out[tok] = __float2bfloat16_rn(fmaf(ep, kg, -KGf));
        }
      }
      double v[3] = {warp_sum((double)sq_f), warp_sum((double)r_f), warp_sum((double)my_part)};
      push(v, 3, parity);
      if (warp == 0) {
        if (!mbar_wait_bounded(&mbar[1 + parity], parity ? xph1 : xph0)) dead = true;
        const double tv = gather(parity, 1, false);
        if (lane == 0) {
          bc[BC_TV] = (bc[BC_LAMBDA] > 0.0) ? tv : 0.0;
          if (need_draw) scalar_find_owner(bc, red + (size_t)(parity * NV + 2) * NSLOT, CS * CW);
          else if (rank == 0) write_result(bc, P.out, !P.spec, row, 0, x, false, K.c64, g_s, g_t);
        }
      }
      if (parity) xph1 ^= 1u; else xph0 ^= 1u;
      parity ^= 1;
    }

    // ------------------------------------------------ the draw (corrected and bonus rows only)
    if (need_draw) {
      __syncthreads();
      if ((int)rank * CW + warp == (int)bc[BC_OWNER_WARP]) {
        // inverse CDF inside the owning warp: lanes are in index order
        const double target = bc[BC_TARGET], before = bc[BC_BEFORE];
        const bool take_last = bc[BC_TAKE_LAST] != 0.0;
        double inc = (double)my_part;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
          const double up = __shfl_up_sync(0xffffffffu, inc, o);
          if (lane >= o) inc += up;
        }
        const unsigned posm = __ballot_sync(0xffffffffu, my_part > 0.f);
        const unsigned hit = take_last ? 0u : __ballot_sync(0xffffffffu, before + inc > target);
        int owner_lane;
        bool last_mode = take_last;
        if (hit) owner_lane = __ffs(hit) - 1;
        else { owner_lane = posm ? 31 - __clz(posm) : 0; last_mode = true; }
        // the owning thread lays its 80 elements out in index order; the warp walks them together
        uint32_t* scr_s = (uint32_t*)(smem + OFF_SCR);
        uint32_t* scr_t = scr_s + NPAIR;
        if (lane == owner_lane) {
#pragma unroll
          for (int j = 0; j < CHUNKS; ++j) {
            int cj = j + rot;
            if (cj == CHUNKS) cj = 0;
            *reinterpret_cast<uint4*>(scr_s + cj * 4) = make_uint4(sr[4 * j], sr[4 * j + 1], sr[4 * j + 2], sr[4 * j + 3]);
            *reinterpret_cast<uint4*>(scr_t + cj * 4) = make_uint4(tr[4 * j], tr[4 * j + 1], tr[4 * j + 2], tr[4 * j + 3]);
          }
        }
        __syncwarp();
        double running = __shfl_sync(0xffffffffu, before + inc - (double)my_part, owner_lane);
        const int first = slice_start + (warp * 32 + owner_lane) * EPT;
        const int n_el = max(0, min(EPT, slice_start + my_len - first));
        int y = -1, last_pos = -1;
        const __nv_bfloat16* es = (const __nv_bfloat16*)scr_s;
        const __nv_bfloat16* et = (const __nv_bfloat16*)scr_t;
        for (int base = 0; base < n_el && y < 0; base += 32) {
          const int e = base + lane;
          float w = 0.f;
          if (e < n_el) {
            const float sf = __bfloat162float(es[e]), tf = __bfloat162float(et[e]);
            const float d = tf - sf;
            const float ep = ex2f(fmaf(sf, c32, k0));
            const float eq = ex2f(fmaf(d, cl, fmaf(sf, c32, kq)));
            w = bonus ? eq * iq : fmaxf(fmaf(eq, iq, -(ep * ip)), 0.f);
          }
          double wi = (double)w;
#pragma unroll
          for (int o = 1; o < 32; o <<= 1) {
            const double up = __shfl_up_sync(0xffffffffu, wi, o);
            if (lane >= o) wi += up;
          }
          const unsigned pm = __ballot_sync(0xffffffffu, w > 0.f);
          const unsigned hm = last_mode ? 0u : __ballot_sync(0xffffffffu, running + wi > target);
          if (pm) last_pos = first + base + 31 - __clz(pm);
          if (hm) y = first + base + __ffs(hm) - 1;
          running += __shfl_sync(0xffffffffu, wi, 31);
        }
        if (y < 0) y = (last_pos >= 0) ? last_pos : min(V - 1, first + max(n_el - 1, 0));
        if (lane == 0) write_result(bc, P.out, !P.spec, row, bonus ? 0 : 1, y, bonus, K.c64, g_s, g_t);
      }
    }
  }

  // a CTA that gave up on a copy still waits (bounded) for what it has in flight before leaving
  if (dead && tid == 0) (void)mbar_wait_bounded(&mbar[0], phase);
  cg::this_cluster().sync();   // no CTA leaves while a peer may still write its shared memory
}

// ---------------------------------------------------------------- host side
static int pick_cs(int V) {
  int cs = 1;
  while (cs * SLICE_CAP < V) cs *= 2;
  return cs;
}

bool cluster_can_serve(const RowParams& p, int dtype) {
  if (dtype != SAKI_BF16) return false;
  if (p.V < 2048 || p.V % 8 != 0 || p.V > MAX_CS * SLICE_CAP) return false;
  if (p.n_rows > 0x7fffffffLL) return false;     // the redo list keeps row numbers in 32 bits
  auto al16 = [](const void* q) { return ((uintptr_t)q & 15) == 0; };
  if (!al16(p.s) || !al16(p.t)) return false;
  if (p.s_seq % 8 || p.s_pos % 8 || p.t_seq % 8 || p.t_pos % 8) return false;
  if (p.dlogits && (!al16(p.dlogits) || p.ld_g % 8)) return false;
  return true;
}

template <int CS>
static cudaError_t launch_cs(const RowParams& p, cudaStream_t st) {
  static std::mutex mu;
  static int cached_dev = -1, cached_clusters = 0;
  auto kern = cluster_kernel<CS>;
  int dev = 0;
  cudaGetDevice(&dev);
  cudaLaunchConfig_t cfg = {};
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = CS; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  cfg.blockDim = dim3(CT); cfg.dynamicSmemBytes = SMEM_BYTES; cfg.stream = st;
  cfg.attrs = at; cfg.numAttrs = 1;
  int n_clusters;
  {
    std::lock_guard<std::mutex> lock(mu);
    if (cached_dev != dev) {
      cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, SMEM_BYTES);
      if (e != cudaSuccess) return e;
      cfg.gridDim = dim3(CS * 64);
      int n = 0;
      e = cudaOccupancyMaxActiveClusters(&n, kern, &cfg);
      if (e != cudaSuccess) return e;
      if (n < 1) return cudaErrorLaunchOutOfResources;
      cached_clusters = n; cached_dev = dev;
    }
    n_clusters = cached_clusters;
  }
  if ((int64_t)n_clusters > p.n_rows) n_clusters = (int)p.n_rows;
  cfg.gridDim = dim3(CS * n_clusters);
  return cudaLaunchKernelEx(&cfg, kern, p, n_clusters);
}

cudaError_t launch_cluster(const RowParams& p, cudaStream_t st, int* n_launches, bool* served) {
  *served = false;
  if (p.n_rows <= 0) { *served = true; return cudaSuccess; }
  cudaError_t e;
  switch (pick_cs(p.V)) {
    case 1: e = launch_cs<1>(p, st); break;
    case 2: e = launch_cs<2>(p, st); break;
    case 4: e = launch_cs<4>(p, st); break;
    default: e = launch_cs<8>(p, st); break;
  }
  if (e == cudaSuccess) { *served = true; if (n_launches) *n_launches += 1; }
  return e;
}

}  // namespace saki
