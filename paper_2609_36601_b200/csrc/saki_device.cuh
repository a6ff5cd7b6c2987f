// Device-side pieces shared by the two bf16 row kernels: packed-bf16 helpers,
// mbarrier / bulk-copy wrappers, the short float64 routines and the per-row
// scalar phases (lambda guess and solve step, coupling decision, result write).
#pragma once
#include "saki_common.cuh"
#include <math_constants.h>

namespace saki {

// Tolerances of the float32 solve (scalar_after_solve4), set against the float64 kernel on random rows (shapes,
// radii from 1e-3 to 3, temperatures 0.7 to 1.3): the direct value of KL from float32 sums is trusted where its
// error bound moves lambda by less than 4e-6 (its worst case is about twice the bound: 1e-5 let one call in fifty
// have a row more than 1e-5 off); the one-panel quadrature only up to beta = 0.25 (beyond, the slope of KL of a
// nearly one-hot row grows so fast over [0, beta] that the two rules agree to 1e-6 and are both 1e-4 off).
constexpr double KL_TOL_REL = 4e-6;
constexpr double QUAD_MAX_BETA = 0.25;
constexpr int BC_DOUBLES = 56;             // doubles of one broadcast area
constexpr double LN2 = 0.693147180559945309417232121458;
constexpr double INV_LN2 = 1.44269504088896340735992468100;
constexpr long long WAIT_LIMIT_CYCLES = 4000000000LL;   // ~2 s: give up on a wait

enum { MODE_SOLVE = 0, MODE_FINAL = 1, MODE_FLAGGED = 2, MODE_REDO = 3 };
// broadcast slots (one set per row buffer)
enum { BC_MODE = 0, BC_BETA, BC_CB, BC_KB, BC_LO, BC_HI, BC_ITER,                    // solver
       BC_CL, BC_KQ, BC_IQ, BC_IP, BC_KG, BC_TOK, BC_STATUS, BC_CORR, BC_LAMBDA,    // final pass
       BC_GLAM, BC_G0, BC_G1, BC_ACC, BC_LPX, BC_LTX, BC_LOSS, BC_VSTAR, BC_KL, BC_TV,
       BC_OWNER_WARP, BC_BEFORE, BC_TARGET, BC_TAKE_LAST, BC_RSS,
       BC_UACC, BC_UDRAW, BC_SX, BC_TX, BC_K0, BC_K1, BC_PMAX, BC_SV, BC_P2, BC_P3, BC_P4,
       BC_QSTATE, BC_E_BETA, BC_E_G, BC_E_G1, BC_E_G2, BC_E_G3, BC_E_G4, BC_E_I7,   // an evaluation waiting for its midpoint
       BC_COUNT };
static_assert(BC_COUNT <= BC_DOUBLES, "broadcast area too small");

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
// packed f32x2 arithmetic (one instruction for two lanes)
__device__ __forceinline__ float2 ffma2(float2 a, float2 b, float2 c) { return __ffma2_rn(a, b, c); }
__device__ __forceinline__ float2 fadd2(float2 a, float2 b) { return __fadd2_rn(a, b); }
__device__ __forceinline__ float2 fmul2(float2 a, float2 b) { return __fmul2_rn(a, b); }
__device__ __forceinline__ float2 ex2f2(float2 a) { return make_float2(ex2f(a.x), ex2f(a.y)); }
__device__ __forceinline__ float2 splat(float a) { return make_float2(a, a); }
// 2^x for a pair on the FMA pipe, for x <= 0 (clamped at -126: the result is then 2^-126, which the callers' sums
// ignore): x = n + f with n = round(x) by the magic-number addition, a degree-5 polynomial for 2^f on
// [-1/2, 1/2] (near-minimax, relative error 1.0e-7; 1.8e-7 as evaluated in float32: what ex2.approx gives),
// the exponent inserted by an integer add.  Twelve issue slots for two exponentials: worth it only where the
// special-function pipe is the tighter bound, and only for a share of the exponentials.
constexpr float EX2_C1 = 0.6931470632553101f, EX2_C2 = 0.24022242426872253f, EX2_C3 = 0.05550636723637581f,
                EX2_C4 = 0.009671509265899658f, EX2_C5 = 0.0013292919611558318f;
__device__ __forceinline__ float2 ex2_fma2(float2 x) {
  x.x = fmaxf(x.x, -126.f); x.y = fmaxf(x.y, -126.f);
  const float2 t = __fadd2_rn(x, make_float2(12582912.f, 12582912.f));              // 1.5 * 2^23: the low bits of t hold n
  const float2 nf = __fadd2_rn(t, make_float2(-12582912.f, -12582912.f));
  const float2 f = __ffma2_rn(nf, make_float2(-1.f, -1.f), x);
  float2 p = make_float2(EX2_C5, EX2_C5);
  p = __ffma2_rn(p, f, make_float2(EX2_C4, EX2_C4));
  p = __ffma2_rn(p, f, make_float2(EX2_C3, EX2_C3));
  p = __ffma2_rn(p, f, make_float2(EX2_C2, EX2_C2));
  p = __ffma2_rn(p, f, make_float2(EX2_C1, EX2_C1));
  p = __ffma2_rn(p, f, make_float2(1.f, 1.f));
  float2 r;
  r.x = __int_as_float(__float_as_int(p.x) + (__float_as_int(t.x) << 23));
  r.y = __int_as_float(__float_as_int(p.y) + (__float_as_int(t.y) << 23));
  return r;
}

// ---- short float64 routines for the scalar phases (one thread, latency-bound) ----
// log2(1 + (i+0.5)/16) and 2^(i/16), i = 0..15
static __constant__ double LOG2_CENTER[16] = {
    0.044394119358453436, 0.12928301694496647, 0.20945336562894978, 0.28540221886224837,
    0.3575520046180837,   0.42626475470209796, 0.4918530963296747,  0.5545888516776374,
    0.6147098441152082,   0.6724253419714956,  0.7279204545631992,  0.7813597135246596,
    0.8328900141647416,   0.8826430493618412,  0.9307373375628862,  0.9772799234999164};
static __constant__ double EXP2_SIXTEENTH[16] = {
    1.0,                1.0442737824274138, 1.0905077326652577, 1.1387886347566916,
    1.189207115002721,  1.241857812073484,  1.2968395546510096, 1.3542555469368927,
    1.4142135623730951, 1.4768261459394993, 1.5422108254079407, 1.6104903319492543,
    1.681792830507429,  1.7562521603732995, 1.8340080864093424, 1.9152065613971474};

__device__ __forceinline__ double rcp_fast(double x) {   // |x| within float range; rel. error ~1e-14
  double r = (double)__frcp_rn((float)x);
  r = r * (2.0 - x * r);
  return r * (2.0 - x * r);
}
// x > 0, normal.  Mantissa m in [1,2) is compared with the centre c of its sixteenth:
// log2 m = log2 c + (2/ln 2) atanh((m-c)/(m+c)), |(m-c)/(m+c)| <= 1/64: three series terms.
__device__ __forceinline__ double log2_fast(double x) {
  const long long bits = __double_as_longlong(x);
  const int e = (int)((bits >> 52) & 0x7ff) - 1023;
  const int i = (int)((bits >> 48) & 0xf);
  const double m = __longlong_as_double((bits & 0x000fffffffffffffLL) | 0x3ff0000000000000LL);
  const double c = 1.0 + ((double)i + 0.5) * 0.0625;
  const double s = (m - c) * rcp_fast(m + c);
  const double z = s * s;
  const double p = 1.0 + z * (1.0 / 3.0 + z * (1.0 / 5.0 + z * (1.0 / 7.0)));
  return ((double)e + LOG2_CENTER[i]) + (2.0 * INV_LN2) * s * p;
}
// any finite x; underflows to 0.  x = n + i/16 + f, |f| <= 1/32.
__device__ __forceinline__ double exp2_fast(double x) {
  if (x < -1020.0) return 0.0;
  if (x > 1020.0) x = 1020.0;
  const double t = rint(x * 16.0);
  const int ti = (int)t;
  const double y = (x - t * 0.0625) * LN2;                 // |y| <= 0.0217
  const double p = 1.0 + y * (1.0 + y * (0.5 + y * (1.0 / 6.0 + y * (1.0 / 24.0 + y * (1.0 / 120.0 + y * (1.0 / 720.0))))));
  const double r = p * EXP2_SIXTEENTH[ti & 15];
  return __longlong_as_double(__double_as_longlong(r) + ((long long)(ti >> 4) << 52));
}

__device__ __forceinline__ double pow2_exact(int n) {     // 2^n for n <= 0; 0 far below the float range
  return n < -120 ? 0.0 : (double)__uint_as_float((uint32_t)(127 + n) << 23);
}

// ---- mbarriers, bulk async copies, asynchronous distributed-shared-memory stores ----
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count));
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
__device__ __forceinline__ bool mbar_test_wait(uint64_t* bar, uint32_t parity) {   // never suspends the thread
  uint32_t ok;
  asm volatile("{\n\t.reg .pred p;\n\tmbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.u32 %0, 1, 0, p;\n\t}"
               : "=r"(ok) : "r"(smem_addr(bar)), "r"(parity) : "memory");
  return ok != 0;
}
// bounded wait: false if the phase did not complete within the limit (in SM cycles).  try_wait may itself
// suspend the thread for a while, so a limit shorter than the default is kept with the probe that does not.
__device__ __forceinline__ bool mbar_wait_bounded(uint64_t* bar, uint32_t parity, long long limit = WAIT_LIMIT_CYCLES) {
  if (limit < WAIT_LIMIT_CYCLES) {
    const long long t0 = clock64();
    while (!mbar_test_wait(bar, parity)) {
      if (clock64() - t0 > limit) return false;
    }
    return true;
  }
  if (mbar_try_wait(bar, parity)) return true;
  const long long t0 = clock64();
  while (!mbar_try_wait(bar, parity)) {
    if (clock64() - t0 > limit) return false;
  }
  return true;
}
__device__ __forceinline__ uint32_t map_to_rank(uint32_t local_smem_addr, uint32_t rank) {
  uint32_t r;
  asm("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_smem_addr), "r"(rank));
  return r;
}
// store 8 bytes into a peer CTA's shared memory; the peer's mbarrier counts the bytes
__device__ __forceinline__ void st_async_f64(uint32_t remote_addr, double v, uint32_t remote_bar) {
  asm volatile("st.async.weak.shared::cluster.mbarrier::complete_tx::bytes.b64 [%0], %1, [%2];"
               ::"r"(remote_addr), "l"(__double_as_longlong(v)), "r"(remote_bar) : "memory");
}

__device__ __forceinline__ double warp_sum(double a) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
  return a;
}
__device__ __forceinline__ double warp_min(double a) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) a = fmin(a, __shfl_xor_sync(0xffffffffu, a, o));
  return a;
}

struct Consts {   // per-launch constants of the scalar phases
  double tau, rtau, eps, c64, rc64, grad_scale;
  float sqrt_eps;
  int V;
};

// The scalar phases run on one thread per CTA, in float64, while all other
// threads hold the row in registers; they are kept out of line so that their
// register needs do not add to the row loop's.

// The coupling decision, the routed loss and the constants of pass "final".
__device__ __forceinline__ void decide(double* bc, const Consts& K, double lam, double Glam, double G0, double G1,
                                       double k0, double k1, double rSs, uint32_t status, int vstar, bool bonus,
                                       bool masked, int x) {
  const double Lam = Glam - (1.0 - lam) * G0 - lam * G1;     // log Z(lambda)
  double lp_x = 0.0, lT_x = 0.0, acc = 1.0;
  int corrected = 0;
  if (!bonus) {
    lp_x = LN2 * (K.c64 * bc[BC_SX]) - G0;
    lT_x = LN2 * (K.c64 * bc[BC_TX]) - G1;
    if (lam > 0.0) {
      acc = exp2_fast(fmin(0.0, lam * (lT_x - lp_x) - Lam) * INV_LN2);
      corrected = (bc[BC_UACC] < acc) ? 0 : 1;
    }
  }
  double loss = 0.0, coef = 0.0;   // a corrected row's loss, -log p(v*), is filled in when the row is written
  int tok = -1;
  if (masked) status |= SAKI_ROW_MASKED;
  else if (!bonus) {
    if (!corrected) { loss = (lp_x - lT_x) * lp_x; coef = -(lp_x - lT_x); tok = x; }
    else { coef = 1.0; tok = vstar; }
  }
  // final pass: q_i = e_q * iq, p_i = e_p * ip with exponent shifts kq, k0
  const float cl = (float)(K.c64 * lam);
  const float kq = (float)((1.0 - lam) * k0 + lam * k1);
  bc[BC_LAMBDA] = lam; bc[BC_GLAM] = Glam;
  bc[BC_CL] = (double)cl; bc[BC_KQ] = (double)kq;
  bc[BC_IQ] = (double)(float)exp2_fast(-(Glam * INV_LN2 + (double)kq));   // 1 / predicted sum of e_q
  bc[BC_IP] = (double)(float)rSs;                                           // 1 / sum of e_p
  bc[BC_KG] = K.grad_scale * coef * K.rtau;                  // gradient = KG * (p - onehot(tok))
  bc[BC_TOK] = (double)tok; bc[BC_STATUS] = (double)status; bc[BC_CORR] = (double)corrected;
  bc[BC_ACC] = acc; bc[BC_LPX] = lp_x; bc[BC_LTX] = lT_x; bc[BC_LOSS] = loss;
  bc[BC_MODE] = MODE_FINAL;
}

// after pass "lse": v = {Ss, St, M1, M2, M3, N1, argmax index} on the row's shifts k0, k1
// e_max: upper bound of the largest term of either sum (1 when the shifts come from the rows' maxima);
// overflow_redo: shifts that come from an estimate of the maxima can overflow on finite rows, so
// non-finite sums hand the row to the float64 kernel instead of flagging it.
// The reciprocal and the log-sum-exp of one row's sum S under shift k: the same instructions for the
// student and the teacher, so two lanes of a warp can do the two rows at once.
__device__ __forceinline__ void lse_of_sum(double S, double k, double& rS, double& G) {
  rS = rcp_fast(S);
  G = LN2 * (log2_fast(S) - k);
}
// The initial guess of lambda far from the student's end.  There the series in the cumulants of d under p is
// short of terms, but the other end is known: KL at beta = 1 is KL(T||p).  A fifth-order term is chosen so that
// the model meets it there, and the model's root is taken inside the bracket (0, 1) by safeguarded Newton (the
// model is negative at 0 and positive at 1, the row being short of the teacher endpoint).  On the sweep's rows
// at eps = 1 the median error of the guess goes from 5 % to 1.3 %; guesses below 0.45 (eps = 0.1 on most rows)
// are left to the series.  Out of line: rare on the headline workload, and the caller's code stays short.
static __device__ __noinline__ float anchored_guess(float b, float vd, float k3, float k4, float kl1, float ef) {
  const float a2 = 0.5f * vd, a3 = (1.f / 3.f) * k3, a4 = 0.125f * k4, a5 = kl1 - (a2 + a3 + a4);
  float lo = 0.f, hi = 1.f, x = fminf(b, 1.f);
#pragma unroll 1
  for (int it = 0; it < 8; ++it) {
    const float pv = x * x * (a2 + x * (a3 + x * (a4 + x * a5))) - ef;
    const float dv = x * (2.f * a2 + x * (3.f * a3 + x * (4.f * a4 + x * (5.f * a5))));
    if (pv > 0.f) hi = x; else lo = x;
    float nx = dv > 0.f ? x - __fdividef(pv, dv) : -1.f;
    if (!(nx > lo && nx < hi)) nx = 0.5f * (lo + hi);
    x = nx;
  }
  return x;
}

static __device__ __noinline__ void scalar_after_lse_tail(double* bc, const double* v, Consts K, float k0f, float k1f, int x,
                                                   bool bonus, bool masked, bool row_timeout, float e_max,
                                                   bool overflow_redo, double rSs, double rSt, double G0, double G1,
                                                   const double* m4_raw = nullptr) {
  const double SsT = v[0], StT = v[1], eps = K.eps, k0 = (double)k0f, k1 = (double)k1f;
  uint32_t status = 0;
  const double chk = ((v[0] + v[1]) + (v[2] + v[3])) + (v[4] + v[5]);
  if (row_timeout) status = SAKI_ROW_TIMEOUT;
  else if (!(fabs(chk) < CUDART_INF) || !(SsT > 0.0) || !(StT > 0.0)) {
    if (overflow_redo) { bc[BC_BETA] = -1.0; bc[BC_MODE] = MODE_REDO; return; }      // (no estimate of lambda to hand over)
    status = SAKI_ROW_NONFINITE;
  }
  else if (!bonus && (x < 0 || x >= K.V)) status = SAKI_ROW_BAD_ID;
  const int vstar = (v[6] >= 0.0 && v[6] < (double)K.V) ? (int)v[6] : 0;
  bc[BC_VSTAR] = (double)vstar;
  if (status) { bc[BC_STATUS] = (double)status; bc[BC_MODE] = MODE_FLAGGED; return; }
  bc[BC_G0] = G0; bc[BC_G1] = G1; bc[BC_RSS] = rSs;
  bc[BC_PMAX] = fmin(1.0, (double)e_max * fmax(rSs, rSt));      // upper bound of the largest probability of either row
  if (!(eps > 0.0)) {          // student-only endpoint
    bc[BC_KL] = 0.0;
    decide(bc, K, 0.0, G0, G0, G1, k0, k1, rSs, status | SAKI_ROW_EPS_ZERO, vstar, bonus, masked, x);
    return;
  }
  const double rtau = K.rtau;
  const double m1 = v[2] * rSs, m2 = v[3] * rSs, m3 = v[4] * rSs;
  const double kl1 = (v[5] * rSt) * rtau - (G1 - G0);       // KL(T || p)
  if (kl1 <= eps) {            // teacher endpoint
    bc[BC_KL] = kl1;
    decide(bc, K, 1.0, G1, G0, G1, k0, k1, rSs, status | SAKI_ROW_SATURATED, vstar, bonus, masked, x);
    return;
  }
  // initial guess from KL(beta) ~ beta^2/2 Var_p(d) + beta^3/3 kappa3_p(d) (+ beta^4/8 kappa4_p(d) where the
  // fourth moment is at hand); float32 is plenty
  const float rt = (float)rtau;
  const double var_p = m2 - m1 * m1, k3_p = m3 - 3.0 * m1 * m2 + 2.0 * m1 * m1 * m1;
  const float vd = fmaxf((float)var_p * rt * rt, 1e-30f);
  const float k3 = (float)k3_p * rt * rt * rt;
  double k4_p = 0.0;
  if (m4_raw) {
    const double m4 = *m4_raw * rSs, m1s = m1 * m1;
    k4_p = m4 - 4.0 * m3 * m1 - 3.0 * m2 * m2 + 12.0 * m2 * m1s - 6.0 * m1s * m1s;
  }
  const float k4 = (float)k4_p * (rt * rt) * (rt * rt);
  // second to fourth derivative of G at 0: they fix the slope b G2(b) of KL at the student's end, for
  // the quadrature of scalar_after_solve4
  const double rt2 = rtau * rtau;
  // (the cumulants come from raw moments: where the mean of d dwarfs its spread they have lost their
  // digits to cancellation, and a negative entry tells the quadrature to stand aside)
  bc[BC_P2] = (m1 * m1 <= 100.0 * var_p) ? var_p * rt2 : -1.0;
  bc[BC_P3] = k3_p * rt2 * rtau; bc[BC_P4] = k4_p * rt2 * rt2;
  const float e2 = 2.f * (float)eps;
  float b = sqrtf(__fdividef(e2, vd));
#pragma unroll
  for (int it = 0; it < 3; ++it) {
    const float bb = fminf(b, 1.f);
    const float den = vd + (2.f / 3.f) * bb * k3 + 0.25f * bb * bb * k4;
    if (den > 0.25f * vd) b = sqrtf(__fdividef(e2, den));
  }
  if (b > 0.45f) b = anchored_guess(b, vd, k3, k4, (float)kl1, (float)eps);
  if (!(b > 1e-7f)) b = 1e-7f;
  if (b > 0.98f) b = 0.98f;
  const float cb = (float)(K.c64 * (double)b);
  const double be = (double)cb * K.rc64;   // the coefficient the pass really evaluates
  bc[BC_STATUS] = (double)status;
  bc[BC_BETA] = be; bc[BC_CB] = (double)cb;
  bc[BC_KB] = (double)(float)((1.0 - be) * k0 + be * k1);
  bc[BC_LO] = 0.0; bc[BC_HI] = 1.0; bc[BC_ITER] = 0.0; bc[BC_QSTATE] = 0.0;
  bc[BC_MODE] = MODE_SOLVE;
}

static __device__ __noinline__ void scalar_after_lse(double* bc, const double* v, Consts K, float k0f, float k1f, int x,
                                              bool bonus, bool masked, bool row_timeout, const double* m4_raw = nullptr) {
  double rSs, rSt, G0, G1;
  lse_of_sum(v[0], (double)k0f, rSs, G0);
  lse_of_sum(v[1], (double)k1f, rSt, G1);
  scalar_after_lse_tail(bc, v, K, k0f, k1f, x, bonus, masked, row_timeout, 1.f, false, rSs, rSt, G0, G1, m4_raw);
}

// After one evaluation of pass "solve" that also carries the third and fourth moments:
// v = {S0, S1, S2, S3, S4}, S_k = sum of e_i d_i^k, d = t - s, e_i the shifted terms of q_beta.
// G(b) = log sum exp((s + b d)/tau) has the derivatives kappa_k(d; q_b) / tau^k, and
// KL(q_b || p) = b G'(b) - G(b) + G(0)  (Eqs. "bridge", "trust_region").  The fourth-order Taylor model
// of G around beta gives
//   KL(beta + h) = KL + h beta G2 + h^2 (beta G3 + G2)/2 + h^3 (beta G4/6 + G3/3) + h^4 G4/8,
// whose root is lambda up to a fifth-order term: with the initial guess a few percent off that is
// far below the resolution of the float32 sums, so one evaluation usually settles the row.  The
// size of the last kept term (with floors against accidentally small cumulants) decides whether
// another evaluation at the new point is needed.
static __device__ __noinline__ void scalar_after_solve4(double* bc, const double* v, Consts K, float k0f, float k1f, int x,
                                                 bool bonus, bool masked) {
  const double eps = K.eps, rtau = K.rtau;
  const double G0 = bc[BC_G0], kb = bc[BC_KB];
  double lo = bc[BC_LO], hi = bc[BC_HI];
  const int iter = (int)bc[BC_ITER] + 1;
  if (!(fabs((v[0] + v[1]) + (v[2] + v[3]) + v[4]) < CUDART_INF)) { bc[BC_BETA] = -1.0; bc[BC_MODE] = MODE_REDO; return; }   // float32 sums overflowed
  // this evaluation: log-partition and cumulants of d under q at bc[BC_BETA]
  double beta = bc[BC_BETA], G, G1, G2, G3, G4;
  bool well_conditioned;
  {
    const double r0 = rcp_fast(v[0]);
    G = LN2 * (log2_fast(v[0]) - kb);
    const double m1 = v[1] * r0, m2 = v[2] * r0, m3 = v[3] * r0, m4 = v[4] * r0;   // raw moments of d under q_beta
    const double m1s = m1 * m1;
    const double var = fmax(m2 - m1s, 0.0);
    const double k3 = m3 - 3.0 * m2 * m1 + 2.0 * m1s * m1;
    const double k4 = m4 - 4.0 * m3 * m1 - 3.0 * m2 * m2 + 12.0 * m2 * m1s - 6.0 * m1s * m1s;
    const double rt2 = rtau * rtau;
    G1 = m1 * rtau; G2 = var * rt2; G3 = k3 * rt2 * rtau; G4 = k4 * rt2 * rt2;
    well_conditioned = m1s <= 100.0 * var;      // else the cumulants have lost their digits to cancellation
  }
  // KL(q_beta || p).  Directly, beta G1 - G + G(0) is a difference of O(1) numbers known to a few 1e-7
  // x (largest probability) from float32 sums: good for radii of 1e-2 and more, useless for 1e-4.  But
  // KL(beta) is also the integral of its slope f(b) = b G2(b) from 0, and f and its first two
  // derivatives are known at both ends (cumulants of d under p from pass "lse", under q_beta from this
  // evaluation; at 0 also the third), each to ~1e-6 RELATIVE: two-point Hermite quadrature.  The rule
  // with three derivatives at 0 and two at beta (exact for degree 6) is taken for small radii when the
  // symmetric rule with two derivatives at each end (exact for degree 5) agrees with it to 2e-6.  Where
  // it does not (heavy tails of d: the integrand is no polynomial of that degree over [0, beta]) and
  // the direct value cannot do either, one more evaluation at beta/2 splits the integral in two panels.
  double kl;
  bool by_quadrature = false;
  const bool quad_ok = eps < 0.02 && bc[BC_P2] >= 0.0;
  const double f0p = bc[BC_P2], f0pp = 2.0 * bc[BC_P3], f0ppp = 3.0 * bc[BC_P4];
  auto rule7 = [&](double b, double g2, double g3, double g4) {   // integral over [0, b], three derivatives known at 0
    const double f1 = b * g2, f1p = g2 + b * g3, f1pp = 2.0 * g3 + b * g4, h2 = b * b;
    return (3.0 / 7.0) * b * f1 + h2 * ((1.0 / 7.0) * f0p - (1.0 / 14.0) * f1p) +
           h2 * b * ((2.0 / 105.0) * f0pp + (1.0 / 210.0) * f1pp) + h2 * h2 * (1.0 / 840.0) * f0ppp;
  };
  if ((int)bc[BC_QSTATE] == 1) {
    // this was the midpoint: panel [0, m] by the rule above, panel [m, beta] by the symmetric rule
    const double m = beta, mG2 = G2, mG3 = G3, mG4 = G4;
    const bool m_ok = well_conditioned;
    beta = bc[BC_E_BETA]; G = bc[BC_E_G]; G1 = bc[BC_E_G1]; G2 = bc[BC_E_G2]; G3 = bc[BC_E_G3]; G4 = bc[BC_E_G4];
    bc[BC_QSTATE] = 0.0;
    const double fa = m * mG2, fap = mG2 + m * mG3, fapp = 2.0 * mG3 + m * mG4;
    const double fb = beta * G2, fbp = G2 + beta * G3, fbpp = 2.0 * G3 + beta * G4;
    const double h = beta - m;
    const double two = rule7(m, mG2, mG3, mG4) + 0.5 * h * (fa + fb) + h * h * 0.1 * (fap - fbp) +
                       h * h * h * (1.0 / 120.0) * (fapp + fbpp);
    kl = beta * G1 - G + G0;
    // one panel was off by about |two - one|; two panels are closer by the seventh power of two or so
    if (m_ok && two > 0.0 && fabs(two - bc[BC_E_I7]) <= 1e-4 * two) { kl = two; by_quadrature = true; }
  } else {
    kl = beta * G1 - G + G0;
    if (quad_ok && well_conditioned) {
      const double f1 = beta * G2, f1p = G2 + beta * G3, f1pp = 2.0 * G3 + beta * G4;
      const double h2 = beta * beta;
      const double i6 = 0.5 * beta * f1 + h2 * 0.1 * (f0p - f1p) + h2 * beta * (1.0 / 120.0) * (f0pp + f1pp);
      const double i7 = rule7(beta, G2, G3, G4);
      if (i7 > 0.0 && fabs(i7 - i6) <= 2e-6 * i7 && beta <= QUAD_MAX_BETA) { kl = i7; by_quadrature = true; }
      else if (i7 > 0.0 && 3e-7 * (eps < 5e-3 ? 1.0 : bc[BC_PMAX]) > (eps < 5e-3 ? 2e-6 : KL_TOL_REL) * beta * G2 && iter < 38) {
        // neither form will do (see the second-tier test below): evaluate at beta/2 first
        bc[BC_QSTATE] = 1.0;
        bc[BC_E_BETA] = beta; bc[BC_E_G] = G; bc[BC_E_G1] = G1; bc[BC_E_G2] = G2; bc[BC_E_G3] = G3; bc[BC_E_G4] = G4;
        bc[BC_E_I7] = i7;
        const float cbm = (float)(K.c64 * 0.5 * beta);
        const double bm = (double)cbm * K.rc64;
        bc[BC_BETA] = bm; bc[BC_CB] = (double)cbm;
        bc[BC_KB] = (double)(float)((1.0 - bm) * (double)k0f + bm * (double)k1f);
        bc[BC_ITER] = (double)iter;
        return;
      }
    }
  }
  const double slope = beta * G2;                       // d KL / d beta
  const double Gq = by_quadrature ? beta * G1 + G0 - kl : G;   // log-partition consistent with the KL used
  if (kl <= eps) lo = fmax(lo, beta); else hi = fmin(hi, beta);
  const double c2 = 0.5 * (beta * G3 + G2), c3 = beta * G4 * (1.0 / 6.0) + G3 * (1.0 / 3.0), c4 = 0.125 * G4;
  double h;
  float trunc = 0.f;
  if (slope > 1e-30 && kl > 1e-30 && kl < 1e30) {
    // the steps are corrections: float32 from here, once eps - KL is formed in float64
    const float f0 = (float)(eps - kl), a1 = (float)slope, a2 = (float)c2, a3 = (float)c3, a4 = (float)c4;
    const float rk = sqrtf((float)kl);
    float hf = __fdividef(f0 * (2.f * rk), (K.sqrt_eps + rk) * a1);     // Newton on sqrt(KL): the starting point
#pragma unroll
    for (int it = 0; it < 3; ++it) {
      const float pv = hf * (a1 + hf * (a2 + hf * (a3 + hf * a4))) - f0;
      const float dv = a1 + hf * (2.f * a2 + hf * (3.f * a3 + hf * (4.f * a4)));
      if (dv > 0.25f * a1) hf -= __fdividef(pv, dv);
    }
    const float h2 = hf * hf;
    trunc = fmaxf(fabsf(a4), fmaxf(fabsf(a3), 0.5f * fabsf(a2))) * h2 * h2;
    h = (double)hf;
  } else { h = 0.5 * (lo + hi) - beta; trunc = 1e30f; }
  double nb = beta + h;
  bool bisected = false;
  if (!(nb > lo && nb < hi)) { nb = 0.5 * (lo + hi); bisected = true; }
  // accepted when the bound on the dropped terms (a generous one: the last kept coefficient in place of the
  // next) moves lambda by less than 1e-7; measured against the float64 kernel, the error of lambda is the
  // same at 3e-8, 1e-7 (and grows from 3e-7 on)
  const bool done = (!bisected && trunc <= 1e-7f * (float)slope) || iter >= 40 || (hi - lo) < 1e-9;
  // The float32 sums resolve KL to a few 1e-7 x (largest probability).  Where that would move lambda by
  // more than the tolerance (a very flat KL: nearly one-hot rows), or the solve did not converge, the row
  // is handed to the float64 kernel.
  // Below 5e-3 the direct value, where the quadrature was not taken, is held to a fifth of the tolerance
  // and to the worst case of its error: 3e-7 absolute (a flat row, where ex2.approx errs the same way on
  // every element).
  const double kl_tol = (eps < 5e-3 ? 2e-6 : KL_TOL_REL) * slope;
  const double kl_err = 3e-7 * (eps < 5e-3 ? 1.0 : bc[BC_PMAX]);
  if (done && ((!by_quadrature && kl_err > kl_tol) || iter >= 40)) {
    bc[BC_BETA] = iter >= 40 ? -1.0 : nb;     // what float32 made of lambda: the float64 kernel starts there
    bc[BC_MODE] = MODE_REDO;
    return;
  }
  if (done) {
    float cl = (float)(K.c64 * nb);
    {   // rounded so that (c - cl) + cl = c exactly in float32: pass "final" of the row-per-SM kernel forms the
        // exponent of q as (c - cl) s + cl t
      const float cf = (float)K.c64, ccl = cf - cl;
      cl = cf - ccl;
    }
    const double lam = (double)cl * K.rc64;
    const double dl = lam - beta;
    // the model's predictions at lambda
    bc[BC_KL] = kl + dl * (slope + dl * (c2 + dl * (c3 + dl * c4)));
    const double Glam = Gq + dl * (G1 + dl * (0.5 * G2 + dl * ((1.0 / 6.0) * G3 + dl * (1.0 / 24.0) * G4)));
    decide(bc, K, lam, Glam, G0, bc[BC_G1], (double)k0f, (double)k1f, bc[BC_RSS], (uint32_t)bc[BC_STATUS],
           (int)bc[BC_VSTAR], bonus, masked, x);
  } else {
    const float cbn = (float)(K.c64 * nb);
    const double be = (double)cbn * K.rc64;
    bc[BC_BETA] = be; bc[BC_CB] = (double)cbn;
    bc[BC_KB] = (double)(float)((1.0 - be) * (double)k0f + be * (double)k1f);
    bc[BC_LO] = lo; bc[BC_HI] = hi; bc[BC_ITER] = (double)iter;
  }
}

// for a draw: the warp that owns the inverse-CDF target (ordered scan of per-warp weights)
static __device__ __noinline__ void scalar_find_owner(double* bc, const double* warp_part, int n_warps) {
  double total = 0.0;
  for (int w = 0; w < n_warps; ++w) total += warp_part[w];
  const double target = bc[BC_UDRAW] * total;
  int owner = -1;
  double before = 0.0;
  for (int w = 0; w < n_warps; ++w) {
    if (before + warp_part[w] > target) { owner = w; break; }
    before += warp_part[w];
  }
  double take_last = 0.0;
  if (owner < 0) {   // rounding left no crossing: last position with positive weight
    take_last = 1.0; before = 0.0;
    for (int w = n_warps - 1; w >= 0; --w) if (warp_part[w] > 0.0) { owner = w; break; }
    if (owner < 0) owner = 0;
  }
  bc[BC_OWNER_WARP] = (double)owner; bc[BC_BEFORE] = before; bc[BC_TARGET] = target; bc[BC_TAKE_LAST] = take_last;
}

// tv: the row's total variation (the caller may hold it before bc[BC_TV] is written)
static __device__ __noinline__ void write_result_tv(const double* bc, saki_out out, bool write_loss, int64_t row, int corrected,
                                             int y, bool bonus, double c64, const __nv_bfloat16* g_s,
                                             const __nv_bfloat16* g_t, double tv) {
  RowResult r;
  const double lam = bc[BC_LAMBDA], G0 = bc[BC_G0], G1 = bc[BC_G1], Glam = bc[BC_GLAM];
  const double Lam = Glam - (1.0 - lam) * G0 - lam * G1;
  const double lp_x = bc[BC_LPX], lT_x = bc[BC_LTX];
  const uint32_t status = (uint32_t)bc[BC_STATUS];
  r.corrected = corrected; r.token = y; r.vstar = (int)bc[BC_VSTAR];
  r.lambda = (float)lam; r.kl = (float)bc[BC_KL]; r.tv = (float)tv;
  r.accept = bonus ? 0.f : (float)bc[BC_ACC];
  r.logp_x = (float)lp_x; r.logT_x = (float)lT_x;
  r.logq_x = bonus ? 0.f : (float)(lp_x + lam * (lT_x - lp_x) - Lam);
  r.loss = (float)bc[BC_LOSS];
  if (corrected || bonus) {
    const double lp_y = LN2 * (c64 * (double)__bfloat162float(g_s[y])) - G0;
    const double lT_y = LN2 * (c64 * (double)__bfloat162float(g_t[y])) - G1;
    r.logp_y = (float)lp_y; r.logq_y = (float)(lp_y + lam * (lT_y - lp_y) - Lam); r.logT_y = (float)lT_y;
    if (corrected && !(status & SAKI_ROW_MASKED))   // teacher-mode loss: -log p(v*)
      r.loss = (float)-(LN2 * (c64 * (double)__bfloat162float(g_s[r.vstar])) - G0);
  } else { r.logp_y = r.logp_x; r.logq_y = r.logq_x; r.logT_y = r.logT_x; }
  r.status = status;
  write_row(out, row, r, write_loss);
}
__device__ __forceinline__ void write_result(const double* bc, saki_out out, bool write_loss, int64_t row, int corrected,
                                             int y, bool bonus, double c64, const __nv_bfloat16* g_s,
                                             const __nv_bfloat16* g_t) {
  write_result_tv(bc, out, write_loss, row, corrected, y, bonus, c64, g_s, g_t, bc[BC_TV]);
}


}  // namespace saki
