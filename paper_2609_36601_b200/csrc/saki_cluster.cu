// Register-resident cluster kernel for bf16 rows (the hot path).
//
// One vocabulary row per thread-block cluster of CS CTAs x 256 threads, two
// CTAs resident per SM.  Each CTA owns a contiguous slice of the row; each
// thread owns 80 contiguous elements of it, held for the whole row in
// registers as the raw packed bf16 pairs (40 + 40 registers), so the row pair
// is read from HBM exactly once.  The single shared-memory slot of a CTA is
// only the landing zone of the NEXT row's slice, fetched by one 1-D bulk
// async copy per row (cp.async.bulk + mbarrier) while the current row is
// being computed.  Passes over the registers:
//   max      packed bf16 maxima of both rows
//   lse      2 exponentials/element: both log-sum-exps, moments of the
//            teacher-student logit difference under p (initial guess of
//            lambda), KL(T||p) (saturation test), teacher argmax index
//   solve    1 exponential/element per evaluation of KL(q_beta||p) and its
//            slope; Newton on sqrt(KL) inside a bisection bracket, typically
//            two evaluations (Eqs. "bridge", "trust_region")
//   final    2 exponentials/element: TV = sum [q-p]_+ with per-thread ordered
//            partial sums for the inverse-CDF residual draw (Eqs. "accept",
//            "residual"), and the gradient row written straight from
//            registers (Eq. "general_objective")
// Per-element work is float32 (packed f32x2 FMAs, ex2.approx); every
// cross-thread combination and every per-row scalar is float64.  Partial sums
// travel warp -> all CTAs of the cluster through distributed shared memory,
// one cluster barrier per pass; each CTA then forms the same scalars
// redundantly, so control flow is uniform across the cluster.
#include "saki_common.cuh"
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
constexpr int NV = 8;                   // doubles per partial-sum vector
constexpr uint32_t SENTINEL = 0xFF7FFF7Fu;   // two bf16 "most negative finite": exp -> 0, difference 0

constexpr int OFF_S = 0;
constexpr int OFF_T = SLICE_CAP * 2;
constexpr int OFF_RED = OFF_T + SLICE_CAP * 2;                  // [2][MAX_CS*CW][NV] doubles
constexpr int OFF_BC = OFF_RED + 2 * MAX_CS * CW * NV * 8;      // broadcast scalars
constexpr int BC_DOUBLES = 32;
constexpr int OFF_MBAR = OFF_BC + BC_DOUBLES * 8;
constexpr int SMEM_BYTES = OFF_MBAR + 16;

constexpr double LN2 = 0.693147180559945309417232121458;
constexpr long long WAIT_LIMIT_CYCLES = 4000000000LL;   // ~2 s: give up on a bulk copy

enum { MODE_SOLVE = 0, MODE_FINAL = 1, MODE_FLAGGED = 2 };
// broadcast slots
enum { BC_MODE = 0, BC_BETA, BC_CB, BC_KB, BC_LO, BC_HI, BC_ITER,       // solver
       BC_IQ, BC_IP, BC_KG, BC_TOK, BC_STATUS, BC_CORR, BC_LAMBDA,        // final pass
       BC_GLAM, BC_G0, BC_G1, BC_ACC, BC_LPX, BC_LTX, BC_LOSS, BC_VSTAR,
       BC_OWNER_WARP, BC_BEFORE, BC_TARGET, BC_TAKE_LAST, BC_MS, BC_MT, BC_BAD, BC_KL, BC_TV };

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ float ex2f(float x) {
  float y;
  asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
  return y;
}
__device__ __forceinline__ float2 unpack_bf16x2(uint32_t r) {
  return make_float2(__uint_as_float(r << 16), __uint_as_float(r & 0xffff0000u));
}
// Same, but opaque to the optimiser: each pass re-derives the floats from the
// packed registers instead of keeping 160 unpacked values alive across passes.
__device__ __forceinline__ float2 unpack_fresh(uint32_t r) {
  asm volatile("" : "+r"(r));
  return unpack_bf16x2(r);
}
__device__ __forceinline__ uint32_t max_bf16x2(uint32_t a, uint32_t b) {
  uint32_t d;
  asm("max.bf16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
  return d;
}
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {   // round to nearest even
  uint32_t d;
  asm("cvt.rn.bf16x2.f32 %0, %1, %2;" : "=r"(d) : "f"(hi), "f"(lo));
  return d;
}
__device__ __forceinline__ float2 ex2f2(float2 a) { return make_float2(ex2f(a.x), ex2f(a.y)); }
__device__ __forceinline__ float2 splat(float a) { return make_float2(a, a); }

// ---- bulk async copy global -> this CTA's shared memory, completion on an mbarrier ----
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count));
  asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void bulk_load(void* dst_smem, const void* src, uint32_t bytes, uint64_t* bar) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
               ::"r"(smem_addr(dst_smem)), "l"(src), "r"(bytes), "r"(smem_addr(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
  uint32_t ok;
  asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
               : "=r"(ok) : "r"(smem_addr(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// bounded wait: false if the copy did not land within the limit
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity) {
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (clock64() - t0 > WAIT_LIMIT_CYCLES) return false;
  }
  return true;
}

// ---- cluster-wide combination of per-thread partial vectors ----
// ops: components [0,NSUM) are summed, [NSUM,NSUM+NMAX) maximised, then NMIN minimised.
template <int NSUM, int NMAX, int NMIN>
__device__ __forceinline__ double comb(int k, double a, double b) {
  if (k < NSUM) return a + b;
  if (k < NSUM + NMAX) return fmax(a, b);
  return fmin(a, b);
}
template <int NSUM, int NMAX, int NMIN>
__device__ __forceinline__ double ident(int k) {
  if (k < NSUM) return 0.0;
  if (k < NSUM + NMAX) return -CUDART_INF;
  return CUDART_INF;
}

// After the call, warp 0 of every CTA holds the cluster-wide result in v[] (all
// lanes); the per-warp partials of every CTA sit in red[parity][rank*CW+warp][k].
template <int CS, int NSUM, int NMAX, int NMIN>
__device__ __forceinline__ void cluster_combine(double (&v)[NSUM + NMAX + NMIN], double* red, int parity,
                                                unsigned rank, int warp, int lane) {
  constexpr int N = NSUM + NMAX + NMIN;
  static_assert(N <= NV, "vector too long");
#pragma unroll
  for (int k = 0; k < N; ++k) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v[k] = comb<NSUM, NMAX, NMIN>(k, v[k], __shfl_xor_sync(0xffffffffu, v[k], o));
  }
  double* mine = red + ((size_t)parity * MAX_CS * CW + rank * CW + warp) * NV;
  if (CS == 1) {
    if (lane == 0) {
#pragma unroll
      for (int k = 0; k < N; ++k) mine[k] = v[k];
    }
    __syncthreads();
  } else {
    cg::cluster_group cl = cg::this_cluster();
    if (lane < CS) {
      double* dst = cl.map_shared_rank(mine, lane);
#pragma unroll
      for (int k = 0; k < N; ++k) dst[k] = v[k];
    }
    cl.sync();
  }
  if (warp == 0) {
    double acc[N];
#pragma unroll
    for (int k = 0; k < N; ++k) acc[k] = ident<NSUM, NMAX, NMIN>(k);
    for (int slot = lane; slot < CS * CW; slot += 32) {
      const double* src = red + ((size_t)parity * MAX_CS * CW + slot) * NV;
#pragma unroll
      for (int k = 0; k < N; ++k) acc[k] = comb<NSUM, NMAX, NMIN>(k, acc[k], src[k]);
    }
#pragma unroll
    for (int k = 0; k < N; ++k) {
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) acc[k] = comb<NSUM, NMAX, NMIN>(k, acc[k], __shfl_xor_sync(0xffffffffu, acc[k], o));
      v[k] = acc[k];
    }
  }
}

struct RowCtx {   // per-row values every thread needs (all cluster-uniform)
  int64_t row;
  uint64_t rid;
  int x;
  bool bonus, masked;
};

struct Consts {   // per-launch constants of the scalar phases
  double tau, eps, c64, grad_scale;
  uint64_t seed;
  int V;
};

// The scalar phases run on one thread per CTA, in float64, while all other
// threads hold the row in registers; they are kept out of line so that their
// register needs do not add to the row loop's.

// after pass "lse": log-sum-exps, saturation test, initial guess of lambda
__device__ __noinline__ void scalar_after_lse(volatile double* bc, const double* v, Consts K, float k0, float k1,
                                              int x, bool bonus, bool row_timeout) {
  const double SsT = v[0], StT = v[1], tau = K.tau, eps = K.eps;
  uint32_t status = 0;
  if (row_timeout) status = SAKI_ROW_TIMEOUT;
  else if (!isfinite(v[0] + v[1] + v[2] + v[3] + v[4] + v[5]) || !(SsT > 0.0) || !(StT > 0.0)) status = SAKI_ROW_NONFINITE;
  else if (!bonus && (x < 0 || x >= K.V)) status = SAKI_ROW_BAD_ID;
  bc[BC_STATUS] = (double)status;
  bc[BC_VSTAR] = (v[6] >= 0.0 && v[6] < (double)K.V) ? v[6] : 0.0;
  if (status) { bc[BC_MODE] = MODE_FLAGGED; return; }
  const double G0 = LN2 * (log2(SsT) - (double)k0), G1 = LN2 * (log2(StT) - (double)k1);
  bc[BC_G0] = G0; bc[BC_G1] = G1;
  double lam = -1.0;
  if (!(eps > 0.0)) { lam = 0.0; status |= SAKI_ROW_EPS_ZERO; }
  else {
    const double m1 = v[2] / SsT, m2 = v[3] / SsT, m3 = v[4] / SsT;
    const double kl1 = (v[5] / StT) / tau - (G1 - G0);       // KL(T || p)
    if (kl1 <= eps) { lam = 1.0; status |= SAKI_ROW_SATURATED; }
    else {
      // KL(beta) ~ beta^2/2 Var_p(d) + beta^3/3 kappa3_p(d)
      const double vd = fmax((m2 - m1 * m1) / (tau * tau), 1e-300);
      const double k3 = (m3 - 3.0 * m1 * m2 + 2.0 * m1 * m1 * m1) / (tau * tau * tau);
      double b = sqrt(2.0 * eps / vd);
      for (int it = 0; it < 3; ++it) {
        const double den = vd + (2.0 / 3.0) * fmin(b, 1.0) * k3;
        if (den > 0.25 * vd) b = sqrt(2.0 * eps / den);
      }
      if (!(b > 1e-7)) b = 1e-7;
      if (b > 0.98) b = 0.98;
      const float cb = (float)(K.c64 * b);
      const double be = (double)cb / K.c64;   // the coefficient the pass really evaluates
      bc[BC_MODE] = MODE_SOLVE; bc[BC_BETA] = be; bc[BC_CB] = (double)cb;
      bc[BC_KB] = (double)(float)((1.0 - be) * (double)k0 + be * (double)k1);
      bc[BC_LO] = 0.0; bc[BC_HI] = 1.0; bc[BC_ITER] = 0.0;
    }
  }
  bc[BC_STATUS] = (double)status;
  if (lam >= 0.0) {   // endpoint: no solve
    bc[BC_MODE] = MODE_FINAL; bc[BC_LAMBDA] = lam;
    bc[BC_GLAM] = lam == 0.0 ? G0 : G1;
  }
}

// after one evaluation of pass "solve": safeguarded Newton step on sqrt(KL)
__device__ __noinline__ void scalar_after_solve(volatile double* bc, const double* v, Consts K, float k0, float k1) {
  const double tau = K.tau, eps = K.eps;
  const double beta = bc[BC_BETA], G0 = bc[BC_G0];
  double lo = bc[BC_LO], hi = bc[BC_HI];
  const int iter = (int)bc[BC_ITER] + 1;
  const double G = LN2 * (log2(v[0]) - (double)(float)bc[BC_KB]);
  const double mu = v[1] / v[0], var = fmax(v[2] / v[0] - mu * mu, 0.0);
  const double kl = beta * mu / tau - G + G0;         // KL(q_beta || p)
  const double slope = beta * var / (tau * tau);      // d KL / d beta
  if (kl <= eps) lo = fmax(lo, beta); else hi = fmin(hi, beta);
  // KL is nearly quadratic in beta, so its square root is nearly linear
  double step;
  const double klp = fmax(kl, 1e-300);
  if (slope > 0.0 && isfinite(kl)) step = (sqrt(eps) - sqrt(klp)) * 2.0 * sqrt(klp) / slope;
  else step = 0.5 * (lo + hi) - beta;
  double nb = beta + step;
  bool bisected = false;
  if (!(nb > lo && nb < hi)) { nb = 0.5 * (lo + hi); bisected = true; }
  const bool done = (!bisected && fabs(nb - beta) <= 2e-4 * beta) || iter >= 40 || (hi - lo) < 1e-9;
  if (done) {
    const float cl = (float)(K.c64 * nb);
    const double lam = (double)cl / K.c64;
    const double dle = lam - beta;
    bc[BC_MODE] = MODE_FINAL; bc[BC_LAMBDA] = lam;
    // second-order prediction of G at lambda from this evaluation
    bc[BC_GLAM] = G + dle * mu / tau + 0.5 * dle * dle * var / (tau * tau);
  } else {
    const float cbn = (float)(K.c64 * nb);
    const double be = (double)cbn / K.c64;
    bc[BC_BETA] = be; bc[BC_CB] = (double)cbn;
    bc[BC_KB] = (double)(float)((1.0 - be) * (double)k0 + be * (double)k1);
    bc[BC_LO] = lo; bc[BC_HI] = hi; bc[BC_ITER] = (double)iter;
  }
}

// before pass "final": the coupling decision, the routed loss, the pass constants
__device__ __noinline__ void scalar_decide(volatile double* bc, Consts K, float k0, float k1, const __nv_bfloat16* g_s,
                                           const __nv_bfloat16* g_t, int x, uint64_t rid, bool bonus, bool masked) {
  const double lam = bc[BC_LAMBDA], G0 = bc[BC_G0], G1 = bc[BC_G1], Glam = bc[BC_GLAM];
  const double Lam = Glam - (1.0 - lam) * G0 - lam * G1;     // log Z(lambda)
  const int vstar = (int)bc[BC_VSTAR];
  double lp_x = 0.0, lT_x = 0.0, acc = 1.0;
  int corrected = 0;
  if (!bonus) {
    lp_x = LN2 * (K.c64 * (double)__bfloat162float(g_s[x])) - G0;
    lT_x = LN2 * (K.c64 * (double)__bfloat162float(g_t[x])) - G1;
    if (lam > 0.0) {
      acc = exp(fmin(0.0, lam * (lT_x - lp_x) - Lam));
      corrected = (scalar_uniform(K.seed, rid, STAGE_ACCEPT) < acc) ? 0 : 1;
    }
  }
  double loss = 0.0, coef = 0.0;
  int tok = -1;
  uint32_t status = (uint32_t)bc[BC_STATUS];
  if (masked) status |= SAKI_ROW_MASKED;
  else if (!bonus) {
    if (!corrected) { loss = (lp_x - lT_x) * lp_x; coef = -(lp_x - lT_x); tok = x; }
    else {
      const double lp_v = LN2 * (K.c64 * (double)__bfloat162float(g_s[vstar])) - G0;
      loss = -lp_v; coef = 1.0; tok = vstar;
    }
  }
  // final pass: q_i = e_q * iq, p_i = e_p * ip with exponent shifts kq, k0
  const float cl = (float)(K.c64 * lam);
  const float kq = (float)((1.0 - lam) * (double)k0 + lam * (double)k1);
  const double log2S0 = Glam / LN2 + (double)kq;             // predicted log2 of the sum of e_q
  const double log2Ss = G0 / LN2 + (double)k0;
  bc[BC_CB] = (double)cl; bc[BC_KB] = (double)kq;
  bc[BC_IQ] = (double)(float)exp2(-log2S0);
  bc[BC_IP] = (double)(float)exp2(-log2Ss);
  bc[BC_KG] = K.grad_scale * coef / K.tau;                   // gradient = KG * (p - onehot(tok))
  bc[BC_TOK] = (double)tok; bc[BC_STATUS] = (double)status; bc[BC_CORR] = (double)corrected;
  bc[BC_ACC] = acc; bc[BC_LPX] = lp_x; bc[BC_LTX] = lT_x; bc[BC_LOSS] = loss;
}

// after pass "final": KL and TV at lambda; for a draw, the warp that owns the target
__device__ __noinline__ void scalar_after_final(volatile double* bc, const double* v, const double* warp_part, int n_warps,
                                                Consts K, uint64_t rid, bool bonus) {
  const double lam = bc[BC_LAMBDA], G0 = bc[BC_G0], G1 = bc[BC_G1];
  const double Glam = (lam == 0.0) ? G0 : (lam == 1.0 ? G1 : LN2 * (log2(v[0]) - (double)(float)bc[BC_KB]));
  const double mu = v[1] / v[0];
  bc[BC_GLAM] = Glam;
  bc[BC_KL] = (lam > 0.0) ? (lam * mu / K.tau - Glam + G0) : 0.0;
  bc[BC_TV] = (lam > 0.0) ? v[2] : 0.0;
  bc[BC_OWNER_WARP] = -1.0;
  if (!(bonus || bc[BC_CORR] != 0.0)) return;
  // ordered scan of the per-warp weights (index order = CTA rank, then warp)
  double total = 0.0;
  for (int w = 0; w < n_warps; ++w) total += warp_part[w * NV + 3];
  const double u = scalar_uniform(K.seed, rid, bonus ? STAGE_BONUS : STAGE_RESIDUAL);
  const double target = u * total;
  int owner = -1;
  double before = 0.0;
  for (int w = 0; w < n_warps; ++w) {
    if (before + warp_part[w * NV + 3] > target) { owner = w; break; }
    before += warp_part[w * NV + 3];
  }
  double take_last = 0.0;
  if (owner < 0) {   // rounding left no crossing: last position with positive weight
    take_last = 1.0; before = 0.0;
    for (int w = n_warps - 1; w >= 0; --w) if (warp_part[w * NV + 3] > 0.0) { owner = w; break; }
    if (owner < 0) owner = 0;
  }
  bc[BC_OWNER_WARP] = (double)owner; bc[BC_BEFORE] = before; bc[BC_TARGET] = target; bc[BC_TAKE_LAST] = take_last;
}

__device__ __noinline__ void write_result(volatile double* bc, const RowParams& P, int64_t row, int corrected, int y,
                                          bool bonus, double c64, const __nv_bfloat16* g_s, const __nv_bfloat16* g_t) {
  RowResult r;
  const double lam = bc[BC_LAMBDA], G0 = bc[BC_G0], G1 = bc[BC_G1], Glam = bc[BC_GLAM];
  const double Lam = Glam - (1.0 - lam) * G0 - lam * G1;
  const double lp_x = bc[BC_LPX], lT_x = bc[BC_LTX];
  const double lp_y = LN2 * (c64 * (double)__bfloat162float(g_s[y])) - G0;
  const double lT_y = LN2 * (c64 * (double)__bfloat162float(g_t[y])) - G1;
  r.corrected = corrected; r.token = y; r.vstar = (int)bc[BC_VSTAR];
  r.lambda = (float)lam; r.kl = (float)bc[BC_KL]; r.tv = (float)bc[BC_TV];
  r.accept = bonus ? 0.f : (float)bc[BC_ACC];
  r.logp_x = (float)lp_x; r.logT_x = (float)lT_x;
  r.logq_x = bonus ? 0.f : (float)(lp_x + lam * (lT_x - lp_x) - Lam);
  r.logp_y = (float)lp_y; r.logq_y = (float)(lp_y + lam * (lT_y - lp_y) - Lam);
  r.loss = (float)bc[BC_LOSS]; r.status = (uint32_t)bc[BC_STATUS];
  write_row(P.out, row, r, !P.spec);
}

// the thread that owns the inverse-CDF target walks its elements in index order (from global memory: L2)
__device__ __noinline__ int rewalk(volatile double* bc, const __nv_bfloat16* g_s, const __nv_bfloat16* g_t, int first,
                                   int n_el, double running, bool last_mode, bool bonus, float c32, float k0, int V) {
  const float cl = (float)bc[BC_CB], kq = (float)bc[BC_KB], iq = (float)bc[BC_IQ], ip = (float)bc[BC_IP];
  const double target = bc[BC_TARGET];
  int y = -1, last_pos = -1;
  for (int e = 0; e < n_el; ++e) {
    const float sf = __bfloat162float(g_s[first + e]), tf = __bfloat162float(g_t[first + e]);
    const float d = tf - sf;
    const float ep = ex2f(fmaf(sf, c32, k0));
    const float eq = ex2f(fmaf(d, cl, fmaf(sf, c32, kq)));
    const float w = bonus ? eq * iq : fmaxf(fmaf(eq, iq, -(ep * ip)), 0.f);
    if (w > 0.f) last_pos = first + e;
    running += (double)w;
    if (!last_mode && running > target) { y = first + e; break; }
  }
  if (y < 0) y = (last_pos >= 0) ? last_pos : min(V - 1, first + max(n_el - 1, 0));
  return y;
}

template <int CS>
__global__ void __launch_bounds__(CT, 2) cluster_kernel(const RowParams P, const int n_clusters) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  unsigned rank = 0;
  if (CS > 1) rank = cg::this_cluster().block_rank();
  const int cluster_id = blockIdx.x / CS;

  const __nv_bfloat16* slot_s = (const __nv_bfloat16*)(smem + OFF_S);
  const __nv_bfloat16* slot_t = (const __nv_bfloat16*)(smem + OFF_T);
  double* red = (double*)(smem + OFF_RED);
  volatile double* bc = (volatile double*)(smem + OFF_BC);
  uint64_t* mbar = (uint64_t*)(smem + OFF_MBAR);

  const int V = P.V;
  const int slice_len = ((V + CS - 1) / CS + 7) & ~7;
  const int slice_start = (int)rank * slice_len;
  const int my_len = max(0, min(slice_len, V - slice_start));
  const uint32_t slice_bytes = (uint32_t)my_len * 2u;
  const int rot = (tid >> 2) & 1;          // chunk rotation: conflict-free 128-bit shared loads
  const int thr_first = tid * EPT;         // first element (within the slice) of this thread

  const float c32 = (float)(1.4426950408889634 / (double)P.temperature);     // log2(e)/temperature
  Consts K;
  K.tau = (double)P.temperature; K.eps = (double)P.eps; K.c64 = (double)c32; K.grad_scale = (double)P.grad_scale;
  K.seed = P.seed; K.V = V;

  auto row_ptrs = [&](int64_t row, const __nv_bfloat16*& s, const __nv_bfloat16*& t) {
    const int64_t b = row / P.K1;
    const int j = (int)(row - b * P.K1);
    s = (const __nv_bfloat16*)P.s + b * P.s_seq + (int64_t)j * P.s_pos;
    t = (const __nv_bfloat16*)P.t + b * P.t_seq + (int64_t)j * P.t_pos;
  };
  auto issue = [&](int64_t row) {   // one thread: fetch this CTA's slice of both rows
    const __nv_bfloat16 *s, *t;
    row_ptrs(row, s, t);
    mbar_expect_tx(mbar, 2u * slice_bytes);
    if (slice_bytes) {
      bulk_load(smem + OFF_S, s + slice_start, slice_bytes, mbar);
      bulk_load(smem + OFF_T, t + slice_start, slice_bytes, mbar);
    }
  };

  if (tid == 0) mbar_init(mbar, 1);
  __syncthreads();
  if (tid == 0 && cluster_id < P.n_rows) issue(cluster_id);
  uint32_t phase = 0;
  int parity = 0;
  bool dead = false;   // a bulk copy timed out: this CTA stops fetching and flags its rows

  for (int64_t row = cluster_id; row < P.n_rows; row += n_clusters) {
    RowCtx rc;
    rc.row = row;
    rc.rid = P.row_offset + (uint64_t)row;
    const int64_t seq = row / P.K1;
    const int pos = (int)(row - seq * P.K1);
    rc.bonus = P.spec && (pos == P.K1 - 1);
    rc.x = rc.bonus ? 0 : (P.spec ? P.proposal[seq * P.prop_ld + pos] : P.proposal[row]);
    rc.masked = (P.mask != nullptr) && (P.mask[row] == 0);
    const __nv_bfloat16 *g_s, *g_t;
    row_ptrs(row, g_s, g_t);
    __nv_bfloat16* g_out = P.dlogits ? (__nv_bfloat16*)P.dlogits + row * P.ld_g : nullptr;

    // ------------------------------------------------ stage: shared slot -> registers
    bool timed_out = dead;
    if (!dead) {
      if (!mbar_wait_bounded(mbar, phase)) timed_out = true;
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
    const int any_timeout = __syncthreads_or(timed_out ? 1 : 0);   // also: every thread has drained the slot
    if (any_timeout) dead = true;
    if (tid == 0 && !dead) {
      const int64_t next = row + n_clusters;
      if (next < P.n_rows) {
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        issue(next);
      }
    }

    // ------------------------------------------------ pass "max"
    float ms, mt;
    {
      uint32_t a = sr[0], b = tr[0];
#pragma unroll
      for (int i = 1; i < NPAIR; ++i) {
        a = max_bf16x2(a, sr[i]);
        b = max_bf16x2(b, tr[i]);
      }
      const float2 fa = unpack_bf16x2(a), fb = unpack_bf16x2(b);
      ms = fmaxf(fa.x, fa.y);
      mt = fmaxf(fb.x, fb.y);
    }
    const float my_mt = mt;
    {
      double v[3] = {dead ? 1.0 : 0.0, (double)ms, (double)mt};
      // component 0 is a flag: its maximum says whether any CTA of the cluster timed out
      cluster_combine<CS, 0, 3, 0>(v, red, parity, rank, warp, lane);
      parity ^= 1;
      if (tid == 0) { bc[BC_BAD] = v[0]; bc[BC_MS] = v[1]; bc[BC_MT] = v[2]; }
      __syncthreads();
      ms = (float)bc[BC_MS];
      mt = (float)bc[BC_MT];
    }
    const bool row_timeout = bc[BC_BAD] != 0.0;
    const float k0 = -(c32 * ms), k1 = -(c32 * mt);   // shifts: every exponent argument <= 0

    // teacher argmax: lowest index holding the row maximum (exact compare on stored values)
    double cand = CUDART_INF;
    if (my_mt == mt) {
#pragma unroll
      for (int j = 0; j < CHUNKS; ++j) {
        int cj = j + rot;
        if (cj == CHUNKS) cj = 0;
        const int e0 = slice_start + thr_first + cj * 8;
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const float2 f = unpack_bf16x2(tr[4 * j + k]);
          if (f.x == mt) cand = fmin(cand, (double)(e0 + 2 * k));
          if (f.y == mt) cand = fmin(cand, (double)(e0 + 2 * k + 1));
        }
      }
    }

    // ------------------------------------------------ pass "lse"
    {
      float2 Ss = splat(0.f), St = splat(0.f), M1 = splat(0.f), M2 = splat(0.f), M3 = splat(0.f), N1 = splat(0.f);
      const float2 cc = splat(c32), kk0 = splat(k0), kk1 = splat(k1), neg1 = splat(-1.f);
#pragma unroll
      for (int i = 0; i < NPAIR; ++i) {
        const float2 sf = unpack_fresh(sr[i]), tf = unpack_fresh(tr[i]);
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
      auto tot = [](const float2 a) { return (double)a.x + (double)a.y; };
      double v[7] = {tot(Ss), tot(St), tot(M1), tot(M2), tot(M3), tot(N1), cand};
      cluster_combine<CS, 6, 0, 1>(v, red, parity, rank, warp, lane);
      parity ^= 1;
      if (tid == 0) scalar_after_lse(bc, v, K, k0, k1, rc.x, rc.bonus, row_timeout);
      __syncthreads();
    }

    // ------------------------------------------------ pass "solve" (repeated)
    while ((int)bc[BC_MODE] == MODE_SOLVE) {
      const float cb = (float)bc[BC_CB], kb = (float)bc[BC_KB];
      float2 S0[2] = {splat(0.f), splat(0.f)}, S1[2] = {splat(0.f), splat(0.f)}, S2[2] = {splat(0.f), splat(0.f)};
      const float2 cc = splat(c32), cbb = splat(cb), kbb = splat(kb), neg1 = splat(-1.f);
#pragma unroll
      for (int i = 0; i < NPAIR; ++i) {
        const int h = i & 1;
        const float2 sf = unpack_fresh(sr[i]), tf = unpack_fresh(tr[i]);
        const float2 d = __ffma2_rn(sf, neg1, tf);
        const float2 e = ex2f2(__ffma2_rn(d, cbb, __ffma2_rn(sf, cc, kbb)));
        S0[h] = __fadd2_rn(S0[h], e);
        const float2 t1 = __fmul2_rn(e, d);
        S1[h] = __fadd2_rn(S1[h], t1);
        S2[h] = __ffma2_rn(t1, d, S2[h]);
      }
      auto tot = [](const float2 (&a)[2]) { return ((double)a[0].x + (double)a[0].y) + ((double)a[1].x + (double)a[1].y); };
      double v[3] = {tot(S0), tot(S1), tot(S2)};
      cluster_combine<CS, 3, 0, 0>(v, red, parity, rank, warp, lane);
      parity ^= 1;
      if (tid == 0) scalar_after_solve(bc, v, K, k0, k1);
      __syncthreads();
    }

    // ------------------------------------------------ flagged row: zero outputs, zero gradient
    if ((int)bc[BC_MODE] == MODE_FLAGGED) {
      if (rank == 0 && tid == 0) {
        write_row(P.out, row, zero_row((uint32_t)bc[BC_STATUS]), !P.spec);
        atomicAdd(P.flagged, 1ull);
      }
      if (g_out) {
#pragma unroll
        for (int j = 0; j < CHUNKS; ++j) {
          int cj = j + rot;
          if (cj == CHUNKS) cj = 0;
          const int e0 = thr_first + cj * 8;
          if (e0 < my_len) *reinterpret_cast<uint4*>(g_out + slice_start + e0) = make_uint4(0, 0, 0, 0);
        }
      }
      __syncthreads();
      continue;
    }

    // ------------------------------------------------ the coupling decision
    if (tid == 0) scalar_decide(bc, K, k0, k1, g_s, g_t, rc.x, rc.rid, rc.bonus, rc.masked);
    __syncthreads();

    // ------------------------------------------------ pass "final"
    float my_part;       // this thread's ordered weight for the inverse-CDF draw
    {
      const float cl = (float)bc[BC_CB], kq = (float)bc[BC_KB];
      const float iq = (float)bc[BC_IQ], ip = (float)bc[BC_IP];
      const float KGf = (float)bc[BC_KG];
      const float kg = (float)(bc[BC_KG] * (double)ip);     // gradient entry = e_p * kg
      const bool want_g = (g_out != nullptr);
      float2 Sq[2] = {splat(0.f), splat(0.f)}, S1[2] = {splat(0.f), splat(0.f)}, R[2] = {splat(0.f), splat(0.f)};
      const float2 cc = splat(c32), cll = splat(cl), kqq = splat(kq), kk0 = splat(k0), neg1 = splat(-1.f);
      const float2 iqq = splat(iq), nip = splat(-ip), kgg = splat(kg);
#pragma unroll
      for (int j = 0; j < CHUNKS; ++j) {
        uint32_t gp[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
          const int i = 4 * j + k, h = k & 1;
          const float2 sf = unpack_fresh(sr[i]), tf = unpack_fresh(tr[i]);
          const float2 d = __ffma2_rn(sf, neg1, tf);
          const float2 ep = ex2f2(__ffma2_rn(sf, cc, kk0));
          const float2 eq = ex2f2(__ffma2_rn(d, cll, __ffma2_rn(sf, cc, kqq)));
          Sq[h] = __fadd2_rn(Sq[h], eq);
          S1[h] = __ffma2_rn(eq, d, S1[h]);
          float2 r = __ffma2_rn(eq, iqq, __fmul2_rn(ep, nip));     // q_i - p_i
          r.x = fmaxf(r.x, 0.f); r.y = fmaxf(r.y, 0.f);
          R[h] = __fadd2_rn(R[h], r);
          const float2 gv = __fmul2_rn(ep, kgg);
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
      my_part = rc.bonus ? sq_f * iq : r_f;
      auto tot = [](const float2 (&a)[2]) { return ((double)a[0].x + (double)a[0].y) + ((double)a[1].x + (double)a[1].y); };
      double v[4] = {tot(Sq), tot(S1), (double)r_f, (double)my_part};
      // the thread that owns the supervised token subtracts the one-hot part of the gradient
      if (want_g) {
        const int tok = (int)bc[BC_TOK];
        const int loc = tok - slice_start - thr_first;
        if (tok >= 0 && loc >= 0 && loc < EPT && tok - slice_start < my_len) {
          const float ep = ex2f(fmaf(__bfloat162float(g_s[tok]), c32, k0));
          g_out[tok] = __float2bfloat16_rn(fmaf(ep, kg, -KGf));
        }
      }
      cluster_combine<CS, 4, 0, 0>(v, red, parity, rank, warp, lane);
      if (tid == 0)
        scalar_after_final(bc, v, red + (size_t)parity * MAX_CS * CW * NV, CS * CW, K, rc.rid, rc.bonus);
      parity ^= 1;
      __syncthreads();
    }

    // ------------------------------------------------ commit: write the row's outputs
    const bool need_draw = rc.bonus || bc[BC_CORR] != 0.0;
    if (!need_draw) {
      if (rank == 0 && tid == 0) write_result(bc, P, row, 0, rc.x, false, K.c64, g_s, g_t);
    } else if ((int)rank * CW + warp == (int)bc[BC_OWNER_WARP]) {
      // inverse CDF inside the owning warp: lanes are in index order
      const double target = bc[BC_TARGET], before = bc[BC_BEFORE];
      const bool take_last = bc[BC_TAKE_LAST] != 0.0;
      double inc = (double)my_part;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const double up = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += up;
      }
      const unsigned pos = __ballot_sync(0xffffffffu, my_part > 0.f);
      const unsigned hit = take_last ? 0u : __ballot_sync(0xffffffffu, before + inc > target);
      int owner_lane;
      bool last_mode = take_last;
      if (hit) owner_lane = __ffs(hit) - 1;
      else { owner_lane = pos ? 31 - __clz(pos) : 0; last_mode = true; }
      if (lane == owner_lane) {
        const int first = slice_start + thr_first;
        const int n_el = max(0, min(EPT, slice_start + my_len - first));
        const int y = rewalk(bc, g_s, g_t, first, n_el, before + inc - (double)my_part, last_mode, rc.bonus, c32, k0, V);
        write_result(bc, P, row, rc.bonus ? 0 : 1, y, rc.bonus, K.c64, g_s, g_t);
      }
    }
    __syncthreads();   // the broadcast slots are rewritten by the next row
  }

  // a CTA that gave up on a copy still waits (bounded) for what it has in flight before leaving
  if (dead && tid == 0) (void)mbar_wait_bounded(mbar, phase);
  if (CS > 1) cg::this_cluster().sync();   // no CTA leaves while a peer may still write its shared memory
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
