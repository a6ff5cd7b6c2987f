// Vocabulary-sharded routing: every rank holds a contiguous slice [v0, v0 + V_local) of each logit row
// (as a tensor-parallel lm-head produces them) and the row is routed without ever gathering it.  The work
// is cut into stages; in each stage a rank reduces its slice to a few numbers per row (a "partial", a
// kernel here), the ranks exchange the partials (the caller's all-gather: ~100 bytes per row and stage),
// and every rank combines them, in rank order, into the same per-row state (a kernel here, and the same
// function compiled for the host).  What is computed is the definition (Eqs. "bridge", "trust_region",
// "accept", "residual", "k1_loss_token", "teacher_mode_loss", "general_objective"); sums, scalars and every
// combine in float64.  An evaluation
// of q_beta costs every rank a pass over its slice and the ranks an exchange, so the solver makes each one
// count: it carries the first four cumulants of the logit difference, the first guess is the root of the
// fourth-order series of KL(q_beta||p) at beta = 0, and each wave moves to the root of the fourth-order model
// at its beta (inside a bisection bracket); a step shorter than VS_SETTLE_STEP is taken without another look.
//   stage A  maxima, teacher argmax, the two sums of exponentials and the moments of the logit
//            difference under p (four) and T (one), each under the slice's own shift; the combine rescales
//   stage B  one evaluation of q_beta per wave: sum e delta^k, k = 0..4; repeated until every
//            row's lambda has settled (two waves as a rule)
//   stage C  the slice's share of TV = sum [q - p]_+ and of KL(q||p), the student's logit at the teacher's
//            argmax; the combine decides acceptance and finds the rank that owns the inverse-CDF target
//   stage D  the gradient slice, and on the owning rank the residual draw; the last combine writes the outputs
// Two families of slice kernels: float64 throughout (one block of 16 warps per row; any dtype, any alignment),
// and, further down, float32 per element for aligned bf16 slices.
#include "saki_device.cuh"
#include <math_constants.h>
#include <cmath>

namespace saki {

// per-row state, in doubles (the same on every rank after each combine)
enum { VS_MODE = 0,      // 0 solving, 1 settled, 2 flagged
       VS_STATUS, VS_MS, VS_MT, VS_VSTAR, VS_LSE_S, VS_LSE_T, VS_SX, VS_TX, VS_SV,
       VS_BETA, VS_LO, VS_HI, VS_ITER, VS_LAM, VS_LOGZ, VS_KL, VS_TV, VS_ACC, VS_CORR,
       VS_OWNER, VS_BEFORE, VS_TARGET, VS_TAKE_LAST, VS_TOK, VS_COEF, VS_LOSS, VS_Y, VS_SY, VS_TY,
       VS_F64,        // 1: the row is ill-conditioned for the float32 slice kernels, the float64 ones take it
       VS_COUNT };
static_assert(VS_COUNT <= SAKI_VSHARD_STATE, "state record too small");
enum { VS_SOLVING = 0, VS_SETTLED = 1, VS_FLAGGED = 2 };

struct VsConsts {
  int64_t N;
  int32_t V, world;
  double eps, tau;
  uint64_t seed, row_offset;
  const int32_t* proposal;
  const uint8_t* mask;
  int fast;          // the float32 slice kernels may be at work (a property of the call, the same on every rank)
};

// the second to fourth cumulants of delta from the sums  a_k = sum w delta^k, k = 0..4
__host__ __device__ inline void vs_cumulants(double a0, double a1, double a2, double a3, double a4, double& k2, double& k3,
                                             double& k4) {
  const double m1 = a1 / a0, r2 = a2 / a0, r3 = a3 / a0, r4 = a4 / a0;
  const double mu2 = r2 - m1 * m1;
  const double mu3 = r3 - 3.0 * m1 * r2 + 2.0 * m1 * m1 * m1;
  const double mu4 = r4 - 4.0 * m1 * r3 + 6.0 * m1 * m1 * r2 - 3.0 * m1 * m1 * m1 * m1;
  k2 = mu2; k3 = mu3; k4 = mu4 - 3.0 * mu2 * mu2;
}
// a wave's step shorter than this is taken without another evaluation: the model's error in lambda is of
// the order of (k5 / k2) step^4 / 24
constexpr double VS_SETTLE_STEP = 3e-3;

// ---------------------------------------------------------------- the combine steps (host and device)
// `part`: [world][N][SAKI_VSHARD_PARTIALS] gathered partials; row i of rank r at part[(r * N + i) * P].
__host__ __device__ inline void vs_combine_a(const VsConsts& c, int64_t i, const double* part, double* st) {
  const int P = SAKI_VSHARD_PARTIALS;
  for (int k = 0; k < SAKI_VSHARD_STATE; ++k) st[k] = 0.0;
  double ms = -INFINITY, mt = -INFINITY, am = 2147483647.0;
  bool finite = true;
  for (int r = 0; r < c.world; ++r) {
    const double* p = part + ((int64_t)r * c.N + i) * P;
    if (p[3] == 0.0) finite = false;
    if (p[0] > ms) ms = p[0];
    if (p[1] > mt || (p[1] == mt && p[2] < am)) { mt = p[1]; am = p[2]; }   // lowest index among ties
  }
  const int x = c.proposal[i];
  uint32_t status = 0;
  if (!finite || !(ms > -INFINITY) || !(mt > -INFINITY)) status = SAKI_ROW_NONFINITE;
  else if (x < 0 || x >= c.V) status = SAKI_ROW_BAD_ID;
  st[VS_MS] = ms; st[VS_MT] = mt; st[VS_VSTAR] = am < 2147483647.0 ? am : 0.0;
  if (status) { st[VS_STATUS] = (double)status; st[VS_MODE] = VS_FLAGGED; return; }
  double Ss = 0.0, St = 0.0, Td = 0.0, Sd = 0.0, Sd2 = 0.0, Sd3 = 0.0, Sd4 = 0.0, sx = 0.0, tx = 0.0;
  for (int r = 0; r < c.world; ++r) {      // rank order: the summation order is part of the protocol
    const double* p = part + ((int64_t)r * c.N + i) * P;
    const double fs = exp((p[0] - ms) / c.tau), ft = exp((p[1] - mt) / c.tau);
    if (p[4] > 0.0) { Ss += fs * p[4]; Sd += fs * p[7]; Sd2 += fs * p[8]; Sd3 += fs * p[12]; Sd4 += fs * p[13]; }
    if (p[5] > 0.0) { St += ft * p[5]; Td += ft * p[6]; }
    sx += p[9]; tx += p[10];
  }
  const double lse_s = ms / c.tau + log(Ss), lse_t = mt / c.tau + log(St);
  st[VS_LSE_S] = lse_s; st[VS_LSE_T] = lse_t; st[VS_SX] = sx; st[VS_TX] = tx;
  if (!(c.eps > 0.0)) { st[VS_STATUS] = (double)SAKI_ROW_EPS_ZERO; st[VS_MODE] = VS_SETTLED; return; }   // lambda = 0, log Z = 0
  const double cc = lse_t - lse_s;                       // d = delta - cc with delta = (t - s) / tau
  const double kl1 = Td / St - cc;                       // KL(T || p)
  if (kl1 <= c.eps) {                                    // teacher endpoint: q = T, log Z(1) = 0
    st[VS_LAM] = 1.0; st[VS_STATUS] = (double)SAKI_ROW_SATURATED; st[VS_MODE] = VS_SETTLED;
    return;
  }
  // First guess: d KL(q_beta||p) / d beta = beta Var_{q_beta}(d) and the variance under q_beta is
  // k2 + k3 beta + k4 beta^2 / 2 + ... in the cumulants of d under p (those of delta: d differs by a constant),
  // so KL = k2 beta^2 / 2 + k3 beta^3 / 3 + k4 beta^4 / 8 + ...; the root of that polynomial at eps, by Newton
  // from the root of its first term.
  double k2, k3, k4;
  vs_cumulants(Ss, Sd, Sd2, Sd3, Sd4, k2, k3, k4);
  double beta = sqrt(2.0 * c.eps / fmax(k2, 1e-300));
  if (!(beta > 0.0 && beta < 1.0)) beta = 0.5;
  {
    double b = beta;
    bool ok = true;
    for (int it = 0; it < 12 && ok; ++it) {
      const double f = b * b * (0.5 * k2 + b * (k3 / 3.0 + b * 0.125 * k4)) - c.eps;
      const double fp = b * (k2 + b * (k3 + b * 0.5 * k4));
      if (!(fp > 0.0)) { ok = false; break; }
      const double nb = b - f / fp;
      if (!(nb > 0.0 && nb < 1.0)) { ok = false; break; }
      const bool done = fabs(nb - b) < 1e-9;
      b = nb;
      if (done) break;
    }
    if (ok) beta = b;
  }
  st[VS_BETA] = beta; st[VS_LO] = 0.0; st[VS_HI] = 1.0; st[VS_MODE] = VS_SOLVING;
}

// One wave of the solver: from the sums at beta, KL(q_beta||p), the cumulants of d under q_beta and with them
// the model  KL(beta + h) = KL(beta) + int_0^h (beta + u) (k2 + k3 u + k4 u^2 / 2) du;  h = its root at eps (Newton
// from the first-order step), kept inside the bisection bracket.  Returns 1 if the row needs another wave.
__host__ __device__ inline int vs_combine_b(const VsConsts& c, int64_t i, const double* part, double* st) {
  if ((int)st[VS_MODE] != VS_SOLVING) return 0;
  const int P = SAKI_VSHARD_PARTIALS;
  double a0 = 0.0, a1 = 0.0, a2 = 0.0, a3 = 0.0, a4 = 0.0;
  for (int r = 0; r < c.world; ++r) {
    const double* p = part + ((int64_t)r * c.N + i) * P;
    a0 += p[0]; a1 += p[1]; a2 += p[2]; a3 += p[3]; a4 += p[4];
  }
  const double beta = st[VS_BETA], cc = st[VS_LSE_T] - st[VS_LSE_S];
  const double kb = ((1.0 - beta) * st[VS_MS] + beta * st[VS_MT]) / c.tau;    // the shift the partials were taken under
  double k2, k3, k4;
  vs_cumulants(a0, a1, a2, a3, a4, k2, k3, k4);
  const double E = a1 / a0 - cc;
  const double logZ = log(a0) + kb - (1.0 - beta) * st[VS_LSE_S] - beta * st[VS_LSE_T];
  const double kl = beta * E - logZ;
  double lo = st[VS_LO], hi = st[VS_HI];
  if (kl <= c.eps) lo = beta; else hi = beta;
  const int it = (int)st[VS_ITER] + 1;
  double h = (c.eps - kl) / (beta * k2);
  {
    double u = h;
    bool ok = isfinite(u);
    for (int n = 0; n < 12 && ok; ++n) {
      const double g = kl - c.eps + beta * u * (k2 + u * (0.5 * k3 + u * k4 / 6.0)) + u * u * (0.5 * k2 + u * (k3 / 3.0 + u * 0.125 * k4));
      const double gp = (beta + u) * (k2 + u * (k3 + u * 0.5 * k4));
      if (!(gp > 0.0)) { ok = false; break; }
      const double nu = u - g / gp;
      if (!isfinite(nu)) { ok = false; break; }
      const bool done = fabs(nu - u) < 1e-15;
      u = nu;
      if (done) break;
    }
    if (ok && fabs(u) <= 2.0 * fabs(h) + 1e-300) h = u;     // the model's root, unless it ran away from the first-order step
  }
  const bool inside = isfinite(h) && beta + h > lo && beta + h < hi;
  if (hi - lo < 1e-13 || it >= 100) h = 0.0;
  else if (!(inside && fabs(h) < VS_SETTLE_STEP)) {
    st[VS_BETA] = inside ? beta + h : 0.5 * (lo + hi);
    st[VS_LO] = lo; st[VS_HI] = hi; st[VS_ITER] = (double)it;
    return 1;
  }
  if (c.fast && st[VS_F64] == 0.0) {
    // The float32 slice kernels resolve KL to a few 1e-7 x (largest probability of either row).  Where that
    // would move lambda by more than a tenth of its tolerance (a very flat KL: nearly one-hot rows, whose TV
    // and acceptance probability move many times faster than lambda) the row goes on in float64.
    const double pmax = fmin(1.0, exp(fmax(st[VS_MS] / c.tau - st[VS_LSE_S], st[VS_MT] / c.tau - st[VS_LSE_T])));
    if (3e-7 * pmax > 1e-6 * beta * k2) {
      st[VS_F64] = 1.0;
      st[VS_BETA] = inside ? beta + h : beta;
      st[VS_LO] = 0.0; st[VS_HI] = 1.0; st[VS_ITER] = (double)it;     // the bracket came from float32 sums: start it over
      return 1;
    }
  }
  st[VS_LAM] = beta + h;
  st[VS_LOGZ] = logZ + h * (E + h * (0.5 * k2 + h * (k3 / 6.0 + h * k4 / 24.0)));   // log Z along beta: the cumulant series of d under q_beta
  st[VS_MODE] = VS_SETTLED;
  return 0;
}

// TV, KL, the coupling decision, the routed loss and the owner of the residual draw
__host__ __device__ inline void vs_combine_c(const VsConsts& c, int64_t i, const double* part, double* st) {
  if ((int)st[VS_MODE] == VS_FLAGGED) return;
  const int P = SAKI_VSHARD_PARTIALS;
  double tv = 0.0, kl = 0.0, sv = 0.0;
  for (int r = 0; r < c.world; ++r) {
    const double* p = part + ((int64_t)r * c.N + i) * P;
    tv += p[0]; kl += p[1]; sv += p[2];
  }
  const double lam = st[VS_LAM], logZ = st[VS_LOGZ];
  const int x = c.proposal[i];
  const uint64_t rid = c.row_offset + (uint64_t)i;
  const double lp_x = st[VS_SX] / c.tau - st[VS_LSE_S], lT_x = st[VS_TX] / c.tau - st[VS_LSE_T];
  double acc = 1.0;
  int corrected = 0;
  if (lam > 0.0) {
    acc = exp(fmin(0.0, lam * (lT_x - lp_x) - logZ));
    corrected = (scalar_uniform(c.seed, rid, STAGE_ACCEPT) < acc) ? 0 : 1;
  } else { tv = 0.0; kl = 0.0; }
  st[VS_SV] = sv; st[VS_TV] = tv; st[VS_KL] = kl; st[VS_ACC] = acc; st[VS_CORR] = (double)corrected;
  st[VS_OWNER] = -1.0; st[VS_Y] = (double)x; st[VS_SY] = st[VS_SX]; st[VS_TY] = st[VS_TX];
  if (corrected) {        // inverse CDF in index order: slices are contiguous, so rank order is index order
    const double target = scalar_uniform(c.seed, rid, STAGE_RESIDUAL) * tv;
    int owner = -1;
    double before = 0.0;
    for (int r = 0; r < c.world; ++r) {
      const double w = part[((int64_t)r * c.N + i) * P];
      if (before + w > target) { owner = r; break; }
      before += w;
    }
    double take_last = 0.0;
    if (owner < 0) {      // rounding left no crossing: the last index with positive weight
      take_last = 1.0; before = 0.0;
      for (int r = c.world - 1; r >= 0; --r) if (part[((int64_t)r * c.N + i) * P] > 0.0) { owner = r; break; }
      if (owner < 0) owner = c.world - 1;
    }
    st[VS_OWNER] = (double)owner; st[VS_BEFORE] = before; st[VS_TARGET] = target; st[VS_TAKE_LAST] = take_last;
  }
  const bool masked = c.mask != nullptr && c.mask[i] == 0;
  uint32_t status = (uint32_t)st[VS_STATUS];
  double loss = 0.0, coef = 0.0;
  int tok = -1;
  if (masked) status |= SAKI_ROW_MASKED;
  else if (!corrected) { loss = (lp_x - lT_x) * lp_x; coef = -(lp_x - lT_x); tok = x; }
  else { loss = -(sv / c.tau - st[VS_LSE_S]); coef = 1.0; tok = (int)st[VS_VSTAR]; }
  st[VS_STATUS] = (double)status; st[VS_LOSS] = loss; st[VS_COEF] = coef; st[VS_TOK] = (double)tok;
}

// the drawn token and the per-position outputs
__host__ __device__ inline void vs_combine_d(const VsConsts& c, int64_t i, const double* part, double* st, const saki_out& o) {
  if ((int)st[VS_MODE] == VS_FLAGGED) { write_row(o, i, zero_row((uint32_t)st[VS_STATUS]), true); return; }
  const int P = SAKI_VSHARD_PARTIALS;
  if (st[VS_CORR] != 0.0) {
    double y = -1.0, sy = 0.0, ty = 0.0;
    for (int r = 0; r < c.world; ++r) {
      const double* p = part + ((int64_t)r * c.N + i) * P;
      if (p[0] >= 0.0) { y = p[0]; sy = p[1]; ty = p[2]; }
    }
    st[VS_Y] = y; st[VS_SY] = sy; st[VS_TY] = ty;
  }
  const double lam = st[VS_LAM], logZ = st[VS_LOGZ];
  RowResult r;
  r.corrected = (int)st[VS_CORR]; r.token = (int)st[VS_Y]; r.vstar = (int)st[VS_VSTAR];
  r.lambda = (float)lam; r.kl = (float)st[VS_KL]; r.tv = (float)st[VS_TV]; r.accept = (float)st[VS_ACC];
  const double lp_x = st[VS_SX] / c.tau - st[VS_LSE_S], lT_x = st[VS_TX] / c.tau - st[VS_LSE_T];
  const double lp_y = st[VS_SY] / c.tau - st[VS_LSE_S], lT_y = st[VS_TY] / c.tau - st[VS_LSE_T];
  r.logp_x = (float)lp_x; r.logT_x = (float)lT_x; r.logq_x = (float)(lp_x + lam * (lT_x - lp_x) - logZ);
  r.logp_y = (float)lp_y; r.logT_y = (float)lT_y; r.logq_y = (float)(lp_y + lam * (lT_y - lp_y) - logZ);
  r.loss = (float)st[VS_LOSS]; r.status = (uint32_t)st[VS_STATUS];
  write_row(o, i, r, true);
}

// ---------------------------------------------------------------- partial kernels: one block per row
constexpr int VT = 512, VW = VT / 32;

template <int NV>
__device__ __forceinline__ void vs_block_sum(double (&v)[NV], double* sh) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int k = 0; k < NV; ++k) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v[k] += __shfl_xor_sync(0xffffffffu, v[k], o);
  }
  if (lane == 0) {
#pragma unroll
    for (int k = 0; k < NV; ++k) sh[k * VW + warp] = v[k];
  }
  __syncthreads();
#pragma unroll
  for (int k = 0; k < NV; ++k) {
    double a = 0.0;
#pragma unroll
    for (int w = 0; w < VW; ++w) a += sh[k * VW + w];
    v[k] = a;
  }
  __syncthreads();
}

struct VsSlice {
  const void *s, *t;
  int64_t ld_s, ld_t, N;
  int32_t V_local, v0, rank;
  double tau;
  const int32_t* proposal;
};

// The residual draw on the rank that owns the inverse-CDF target (all threads of the block call; NW warps).
// Every warp adds up the residual weights of its contiguous segment; the warp whose segment holds the target
// (segments in index order) walks it 32 elements at a time.  float64, whichever kernel family calls.
template <typename T, int NW>
__device__ __forceinline__ void vs_draw(const T* s, const T* t, int Vl, double rtau, const double* st, double* red, int* stoken) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const double lam = st[VS_LAM], lse_s = st[VS_LSE_S], lse_t = st[VS_LSE_T], logZ = st[VS_LOGZ];
  const double target = st[VS_TARGET];
  const bool take_last = st[VS_TAKE_LAST] != 0.0;
  const int seg = (Vl + NW - 1) / NW, v_lo = min(Vl, warp * seg), v_hi = min(Vl, v_lo + seg);
  auto weight = [&](int v) {
    const double lp = (double)ld_as_float(s, v) * rtau - lse_s, lT = (double)ld_as_float(t, v) * rtau - lse_t;
    return fmax(exp(lp + lam * (lT - lp) - logZ) - exp(lp), 0.0);
  };
  double wsum = 0.0;
  for (int v = v_lo + lane; v < v_hi; v += 32) wsum += weight(v);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) wsum += __shfl_xor_sync(0xffffffffu, wsum, o);
  if (lane == 0) red[warp] = wsum;
  __syncthreads();
  // the first warp whose running total passes the target; none (rounding, or the rule "last positive
  // element"): the last warp with weight
  double before = st[VS_BEFORE];
  int own_w = -1, last_w = -1;
  for (int w = 0; w < NW; ++w) {
    if (red[w] > 0.0) last_w = w;
    if (own_w < 0 && !take_last && before + red[w] > target) own_w = w;
    if (own_w < 0) before += red[w];
  }
  const bool walk_last = own_w < 0;
  if (walk_last) own_w = last_w;
  if (warp == own_w) {
    double running = before;
    int last_pos = -1, found = -1;
    for (int v0 = v_lo; v0 < v_hi && found < 0; v0 += 32) {
      const int v = v0 + lane;
      const double r = v < v_hi ? weight(v) : 0.0;
      double inc = r;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const double up = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += up;
      }
      const unsigned pos = __ballot_sync(0xffffffffu, r > 0.0);
      const unsigned hit = walk_last ? 0u : __ballot_sync(0xffffffffu, (running + inc > target) && v < v_hi);
      if (pos) last_pos = v0 + 31 - __clz(pos);
      if (hit) found = v0 + __ffs(hit) - 1;
      running += __shfl_sync(0xffffffffu, inc, 31);
    }
    if (found < 0) found = last_pos >= 0 ? last_pos : max(v_hi - 1, 0);   // rounding: the last element with weight in the segment
    if (lane == 0) *stoken = found;
  }
  if (own_w < 0 && tid == 0) *stoken = max(Vl - 1, 0);   // no weight anywhere in the slice
}

template <typename T>
__global__ void __launch_bounds__(VT) vs_partial_kernel(const VsSlice S, const int stage, const double* state, double* partial,
                                                        void* dlogits, const int64_t ld_g, const double grad_scale,
                                                        const bool only_flagged) {
  __shared__ double red[7 * VW];
  __shared__ float smax[2][VW];
  __shared__ int sarg[VW];
  __shared__ int stoken;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int Vl = S.V_local;
  const double rtau = 1.0 / S.tau;
  for (int64_t row = blockIdx.x; row < S.N; row += gridDim.x) {
    const T* s = (const T*)S.s + row * S.ld_s;
    const T* t = (const T*)S.t + row * S.ld_t;
    double* out = partial + row * SAKI_VSHARD_PARTIALS;
    const double* st = state ? state + row * SAKI_VSHARD_STATE : nullptr;
    if (only_flagged && !(st != nullptr && st[VS_F64] != 0.0)) continue;   // the float32 kernel has this row
    if (stage == 0) {
      // ---- stage A: maxima and argmax, then the sums under this slice's own shifts
      float ms = -CUDART_INF_F, mt = -CUDART_INF_F;
      int am = 0x7fffffff, finite = 1;
      for (int v = tid; v < Vl; v += VT) {
        const float a = ld_as_float(s, v), c = ld_as_float(t, v);
        finite &= (isfinite(a) && isfinite(c)) ? 1 : 0;
        ms = fmaxf(ms, a);
        if (c > mt) { mt = c; am = v; }
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        ms = fmaxf(ms, __shfl_xor_sync(0xffffffffu, ms, o));
        const float omt = __shfl_xor_sync(0xffffffffu, mt, o);
        const int oam = __shfl_xor_sync(0xffffffffu, am, o);
        if (omt > mt || (omt == mt && oam < am)) { mt = omt; am = oam; }
      }
      if (lane == 0) { smax[0][warp] = ms; smax[1][warp] = mt; sarg[warp] = am; }
      finite = __syncthreads_and(finite);
      ms = smax[0][0]; mt = smax[1][0]; am = sarg[0];
      for (int w = 1; w < VW; ++w) {
        ms = fmaxf(ms, smax[0][w]);
        if (smax[1][w] > mt || (smax[1][w] == mt && sarg[w] < am)) { mt = smax[1][w]; am = sarg[w]; }
      }
      __syncthreads();
      double a[7] = {0.0, 0.0, 0.0, 0.0, 0.0, 0.0, 0.0};
      if (finite && Vl > 0) {
        const double zms = (double)ms * rtau, zmt = (double)mt * rtau;
        for (int v = tid; v < Vl; v += VT) {
          const double zs = (double)ld_as_float(s, v) * rtau, zt = (double)ld_as_float(t, v) * rtau;
          const double es = exp(zs - zms), et = exp(zt - zmt), dl = zt - zs, ed = es * dl, ed2 = ed * dl;
          a[0] += es; a[1] += et; a[2] += et * dl; a[3] += ed; a[4] += ed2; a[5] += ed2 * dl; a[6] += ed2 * dl * dl;
        }
      }
      vs_block_sum<7>(a, red);
      if (tid == 0) {
        const int x = S.proposal[row] - S.v0;
        const bool own = x >= 0 && x < Vl;
        out[0] = (double)ms; out[1] = (double)mt; out[2] = am == 0x7fffffff ? 2147483647.0 : (double)(S.v0 + am);
        out[3] = finite ? 1.0 : 0.0;
        out[4] = a[0]; out[5] = a[1]; out[6] = a[2]; out[7] = a[3]; out[8] = a[4];
        out[9] = own ? (double)ld_as_float(s, x) : 0.0; out[10] = own ? (double)ld_as_float(t, x) : 0.0;
        out[11] = own ? 1.0 : 0.0;
        out[12] = a[5]; out[13] = a[6]; out[14] = 0.0; out[15] = 0.0;
      }
    } else if (stage == 1) {
      // ---- stage B: one evaluation at the row's current beta, under the row's global shift
      double a[5] = {0.0, 0.0, 0.0, 0.0, 0.0};
      if ((int)st[VS_MODE] == VS_SOLVING) {
        const double beta = st[VS_BETA];
        const double kb = ((1.0 - beta) * st[VS_MS] + beta * st[VS_MT]) * rtau;
        for (int v = tid; v < Vl; v += VT) {
          const double zs = (double)ld_as_float(s, v) * rtau, zt = (double)ld_as_float(t, v) * rtau;
          const double dl = zt - zs, e = exp(zs + beta * dl - kb), ed = e * dl, ed2 = ed * dl;
          a[0] += e; a[1] += ed; a[2] += ed2; a[3] += ed2 * dl; a[4] += ed2 * dl * dl;
        }
      }
      vs_block_sum<5>(a, red);
      if (tid == 0) {
        for (int k = 0; k < SAKI_VSHARD_PARTIALS; ++k) out[k] = 0.0;
        out[0] = a[0]; out[1] = a[1]; out[2] = a[2]; out[3] = a[3]; out[4] = a[4];
      }
    } else if (stage == 2) {
      // ---- stage C: the slice's share of TV and KL(q||p); the student's logit at the teacher's argmax
      double a[2] = {0.0, 0.0};
      const bool live = (int)st[VS_MODE] == VS_SETTLED;
      const double lam = st[VS_LAM];
      if (live && lam > 0.0) {
        const double lse_s = st[VS_LSE_S], lse_t = st[VS_LSE_T], logZ = st[VS_LOGZ];
        // per-warp segments in index order, summed in warp order: close to the index-order sum of the definition
        const int seg = (Vl + VW - 1) / VW, v_lo = warp * seg, v_hi = min(Vl, v_lo + seg);
        for (int v = v_lo + lane; v < v_hi; v += 32) {
          const double lp = (double)ld_as_float(s, v) * rtau - lse_s, lT = (double)ld_as_float(t, v) * rtau - lse_t;
          const double lq = lp + lam * (lT - lp) - logZ, q = exp(lq);
          a[0] += fmax(q - exp(lp), 0.0);
          a[1] += q * (lq - lp);
        }
      }
      vs_block_sum<2>(a, red);
      if (tid == 0) {
        for (int k = 0; k < SAKI_VSHARD_PARTIALS; ++k) out[k] = 0.0;
        const int vs = (int)st[VS_VSTAR] - S.v0;
        out[0] = a[0]; out[1] = a[1];
        out[2] = (live && vs >= 0 && vs < Vl) ? (double)ld_as_float(s, vs) : 0.0;
      }
    } else {
      // ---- stage D: the gradient slice; on the owning rank the residual draw
      const int mode = (int)st[VS_MODE];
      T* g = dlogits ? (T*)dlogits + row * ld_g : nullptr;
      if (g) {
        const double sc = mode == VS_FLAGGED ? 0.0 : grad_scale * st[VS_COEF] * rtau;
        const double lse_s = st[VS_LSE_S];
        const int tok = mode == VS_FLAGGED ? -1 : (int)st[VS_TOK] - S.v0;
        for (int v = tid; v < Vl; v += VT) {
          double gv = 0.0;
          if (sc != 0.0) gv = sc * (exp((double)ld_as_float(s, v) * rtau - lse_s) - (v == tok ? 1.0 : 0.0));
          if constexpr (sizeof(T) == 2) {
            // float64 -> bf16, round to nearest even: through a float rounded to odd (truncate, and keep in the
            // last bit whether anything was cut off), which the second rounding cannot mistake for a tie
            float f = __double2float_rz(gv);
            if ((double)f != gv) f = __uint_as_float(__float_as_uint(f) | 1u);
            g[v] = __float2bfloat16_rn(f);
          } else g[v] = (float)gv;
        }
      }
      if (tid == 0) stoken = -1;
      __syncthreads();
      const bool mine = mode == VS_SETTLED && st[VS_CORR] != 0.0 && (int)st[VS_OWNER] == S.rank;
      if (mine) vs_draw<T, VW>(s, t, Vl, rtau, st, red, &stoken);
      __syncthreads();
      if (tid == 0) {
        for (int k = 0; k < SAKI_VSHARD_PARTIALS; ++k) out[k] = 0.0;
        out[0] = -1.0;
        if (mine && stoken >= 0 && stoken < Vl) {
          out[0] = (double)(S.v0 + stoken);
          out[1] = (double)ld_as_float(s, stoken); out[2] = (double)ld_as_float(t, stoken);
        }
      }
      __syncthreads();
    }
  }
}

// ---------------------------------------------------------------- the float32 slice kernels
// The same partials for bf16 slices that start on a 16-byte boundary, with the per-element arithmetic of the
// row-per-SM kernel: packed f32x2 FMAs, ex2.approx under whole-number exponent shifts (the factor between such
// a shift and the one the partial is defined under is applied once per row, in float64), float32 sums per thread,
// float64 across threads.  One block of four warps per row slice, several blocks per SM.  A row whose state says
// VS_F64 is left to the float64 kernel, which is launched behind this one for those rows only.
constexpr int FT = 128, FW = FT / 32;
constexpr uint32_t VF_FILLER = 0xFF7FFF7Fu;       // two bf16 of the most negative finite value
constexpr double VF_LOG2E = 1.4426950408889634;

template <int NV>
__device__ __forceinline__ void vf_block_sum(double (&v)[NV], double* sh) {   // the totals are valid in thread 0
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int k = 0; k < NV; ++k) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v[k] += __shfl_xor_sync(0xffffffffu, v[k], o);
  }
  if (lane == 0) {
#pragma unroll
    for (int k = 0; k < NV; ++k) sh[k * FW + warp] = v[k];
  }
  __syncthreads();
  if (threadIdx.x == 0) {
#pragma unroll
    for (int k = 0; k < NV; ++k) {
      double a = 0.0;
#pragma unroll
      for (int w = 0; w < FW; ++w) a += sh[k * FW + w];
      v[k] = a;
    }
  }
  __syncthreads();
}
__device__ __forceinline__ uint4 vf_ld(const __nv_bfloat16* p) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p));
  return v;
}
__device__ __forceinline__ double vf_tot(const float2 a) { return (double)a.x + (double)a.y; }
// sums of e (d - D)^k, k = 0..4, to sums of e d^k (in place): the kernels take the moments about a constant near the
// mean of the logit difference, where float32 products keep their digits; the partials are defined about zero
__device__ __forceinline__ void vf_uncentre(double D, double a0, double& a1, double& a2, double& a3, double& a4) {
  const double D2 = D * D, D3 = D2 * D, D4 = D2 * D2;
  a4 = a4 + 4.0 * D * a3 + 6.0 * D2 * a2 + 4.0 * D3 * a1 + D4 * a0;
  a3 = a3 + 3.0 * D * a2 + 3.0 * D2 * a1 + D3 * a0;
  a2 = a2 + 2.0 * D * a1 + D2 * a0;
  a1 = a1 + D * a0;
}

// The residual draw of the float32 kernels on the owning rank (all threads of the block call): weights
// [q - p]_+ per element in float32 (in units of fq, like stage C), sums in float64.  Every warp adds up its
// contiguous range of chunks; the warp that holds the target walks its range 32 chunks at a time, the lane whose
// chunk holds it walks the chunk's 8 elements.
__device__ __forceinline__ void vf_draw(const __nv_bfloat16* s, const __nv_bfloat16* t, int n_chunks, float c32, double c64,
                                        double tau, const double* st, double* red, int* stoken) {
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const double lam = st[VS_LAM], target = st[VS_TARGET];
  const bool take_last = st[VS_TAKE_LAST] != 0.0;
  float cl = (float)(c64 * lam);
  const float ccl = c32 - cl;
  cl = c32 - ccl;
  const float msf = (float)st[VS_MS], mtf = (float)st[VS_MT];
  // (the log-sum-exps relative to the maxima: what the sums of 2^(c s'), 2^(c t') came to)
  const double ls = st[VS_LSE_S] - st[VS_MS] / tau, lt = st[VS_LSE_T] - st[VS_MT] / tau;
  const double kp2 = ls * VF_LOG2E, kq2 = ((1.0 - lam) * ls + lam * lt + st[VS_LOGZ]) * VF_LOG2E;
  const float kpi = floorf((float)kp2 - 1e-3f), kqi = floorf((float)kq2 - 1e-3f);
  const double fp = exp2((double)kpi - kp2), fq = exp2((double)kqi - kq2);
  const float2 cc = splat(c32), cll = splat(cl), ccll = splat(ccl), kpp = splat(-kpi), kqq = splat(-kqi);
  const float2 nms = splat(-msf), nmt = splat(-mtf);
  const float2 nrho = splat(-(float)(fp / fq));
  auto weights = [&](int c, float (&w)[8]) {
    const uint4 s4 = vf_ld(s + (size_t)c * 8), t4 = vf_ld(t + (size_t)c * 8);
    const uint32_t sw[4] = {s4.x, s4.y, s4.z, s4.w}, tw[4] = {t4.x, t4.y, t4.z, t4.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 sf = fadd2(unpack_bf16x2(sw[i]), nms), tf = fadd2(unpack_bf16x2(tw[i]), nmt);
      const float2 ep = ex2f2(ffma2(sf, cc, kpp));
      const float2 eq = ex2f2(ffma2(tf, cll, ffma2(sf, ccll, kqq)));
      const float2 r = ffma2(ep, nrho, eq);
      w[2 * i] = fmaxf(r.x, 0.f); w[2 * i + 1] = fmaxf(r.y, 0.f);
    }
  };
  auto total = [&](const float (&w)[8]) { return fq * (double)(((w[0] + w[1]) + (w[2] + w[3])) + ((w[4] + w[5]) + (w[6] + w[7]))); };
  const int seg = (n_chunks + FW - 1) / FW, c_lo = min(n_chunks, warp * seg), c_hi = min(n_chunks, c_lo + seg);
  double wsum = 0.0;
  for (int c = c_lo + lane; c < c_hi; c += 32) {
    float w[8];
    weights(c, w);
    wsum += total(w);
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) wsum += __shfl_xor_sync(0xffffffffu, wsum, o);
  if (lane == 0) red[warp] = wsum;
  __syncthreads();
  double before = st[VS_BEFORE];
  int own_w = -1, last_w = -1;
  for (int w = 0; w < FW; ++w) {
    if (red[w] > 0.0) last_w = w;
    if (own_w < 0 && !take_last && before + red[w] > target) own_w = w;
    if (own_w < 0) before += red[w];
  }
  const bool walk_last = own_w < 0;
  if (walk_last) own_w = last_w;
  if (warp == own_w) {
    double running = before;
    int found = -1, last_c = -1;
    for (int c0 = c_lo; c0 < c_hi && found < 0; c0 += 32) {
      const int c = c0 + lane;
      float w[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
      if (c < c_hi) weights(c, w);
      const double mine = total(w);
      double inc = mine;
#pragma unroll
      for (int o = 1; o < 32; o <<= 1) {
        const double up = __shfl_up_sync(0xffffffffu, inc, o);
        if (lane >= o) inc += up;
      }
      const unsigned pos = __ballot_sync(0xffffffffu, mine > 0.0);
      const unsigned hit = walk_last ? 0u : __ballot_sync(0xffffffffu, running + inc > target);
      if (pos) last_c = c0 + 31 - __clz(pos);
      if (hit) {
        const int src = __ffs(hit) - 1;
        int f = -1;
        if (lane == src) {
          double run = running + inc - mine;
#pragma unroll
          for (int i = 0; i < 8; ++i) {
            run += fq * (double)w[i];
            if (f < 0 && run > target) f = c * 8 + i;
          }
          if (f < 0) {                                // rounding inside the chunk: its last element with weight
#pragma unroll
            for (int i = 0; i < 8; ++i) if (w[i] > 0.f) f = c * 8 + i;
          }
        }
        found = __shfl_sync(0xffffffffu, f, src);
      }
      running += __shfl_sync(0xffffffffu, inc, 31);
    }
    if (found < 0 && last_c >= 0) {                   // no crossing: the last element with weight in the range
      float w[8];
      weights(last_c, w);
#pragma unroll
      for (int i = 0; i < 8; ++i) if (w[i] > 0.f) found = last_c * 8 + i;
    }
    if (found < 0) found = max(c_hi * 8 - 1, 0);
    if (lane == 0) *stoken = found;
  }
  if (own_w < 0 && tid == 0) *stoken = max(n_chunks * 8 - 1, 0);   // no weight anywhere in the slice
}

template <int STAGE>
__global__ void __launch_bounds__(FT) vs_fast_kernel(const VsSlice S, const double* state, double* partial, void* dlogits,
                                                     const int64_t ld_g, const double grad_scale) {
  __shared__ double red[7 * FW];
  __shared__ float smax[2][FW];
  __shared__ int sarg[FW];
  __shared__ int stoken;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int Vl = S.V_local, n_chunks = Vl >> 3;
  const double rtau = 1.0 / S.tau;
  const float c32 = (float)(VF_LOG2E / S.tau);
  const double c64 = (double)c32;                  // the multiplier the elements really see
  const float2 cc = splat(c32), neg1 = splat(-1.f);
  // Every element enters as its distance below the row's maxima, s' = s - max s and t' = t - max t (exact in
  // float32 for bf16 logits): exponents are then sums of small terms, and the logit difference d' = t' - s'
  // is taken about the difference of the maxima, so float32 products keep their digits whatever offsets the two
  // models' logits carry.  Partials that are defined about zero are converted in float64, once per row.
  for (int64_t row = blockIdx.x; row < S.N; row += gridDim.x) {
    const __nv_bfloat16* s = (const __nv_bfloat16*)S.s + row * S.ld_s;
    const __nv_bfloat16* t = (const __nv_bfloat16*)S.t + row * S.ld_t;
    double* out = partial + row * SAKI_VSHARD_PARTIALS;
    const double* st = state ? state + row * SAKI_VSHARD_STATE : nullptr;
    if (STAGE > 0 && st[VS_F64] != 0.0) continue;
    if (STAGE == 0) {
      // ---- stage A, first sweep: the slice's maxima, and the first chunk that holds the teacher's
      uint32_t run_s = VF_FILLER;
      float mt_run = -CUDART_INF_F;
      int arg_c = 0x7fffffff;
      for (int c = tid; c < n_chunks; c += FT) {
        const uint4 s4 = vf_ld(s + (size_t)c * 8), t4 = vf_ld(t + (size_t)c * 8);
        run_s = max_bf16x2(run_s, max_bf16x2(max_bf16x2(s4.x, s4.y), max_bf16x2(s4.z, s4.w)));
        const float2 cmt = unpack_bf16x2(max_bf16x2(max_bf16x2(t4.x, t4.y), max_bf16x2(t4.z, t4.w)));
        const float cm = fmaxf(cmt.x, cmt.y);
        if (cm > mt_run) { mt_run = cm; arg_c = c; }
      }
      const float2 rs2 = unpack_bf16x2(run_s);
      float ms = fmaxf(rs2.x, rs2.y), mt = mt_run;
      int ac = arg_c;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        ms = fmaxf(ms, __shfl_xor_sync(0xffffffffu, ms, o));
        const float omt = __shfl_xor_sync(0xffffffffu, mt, o);
        const int oac = __shfl_xor_sync(0xffffffffu, ac, o);
        if (omt > mt || (omt == mt && oac < ac)) { mt = omt; ac = oac; }
      }
      if (lane == 0) { smax[0][warp] = ms; smax[1][warp] = mt; sarg[warp] = ac; }
      __syncthreads();
      ms = smax[0][0]; mt = smax[1][0]; ac = sarg[0];
#pragma unroll
      for (int w = 1; w < FW; ++w) {
        ms = fmaxf(ms, smax[0][w]);
        if (smax[1][w] > mt || (smax[1][w] == mt && sarg[w] < ac)) { mt = smax[1][w]; ac = sarg[w]; }
      }
      __syncthreads();
      if (n_chunks == 0) { ms = -CUDART_INF_F; mt = -CUDART_INF_F; }
      // ---- second sweep: the sums under the slice's own shifts (the partial's definition: no factor to apply)
      float2 Ss = splat(0.f), St = splat(0.f), Td = splat(0.f), M1 = splat(0.f), M2 = splat(0.f), M3 = splat(0.f), M4 = splat(0.f);
      const float msc = fminf(fmaxf(ms, -1e30f), 1e30f), mtc = fminf(fmaxf(mt, -1e30f), 1e30f);
      const float2 nms = splat(-msc), nmt = splat(-mtc);
#pragma unroll 2
      for (int c = tid; c < n_chunks; c += FT) {
        const uint4 s4 = vf_ld(s + (size_t)c * 8), t4 = vf_ld(t + (size_t)c * 8);
        const uint32_t sw[4] = {s4.x, s4.y, s4.z, s4.w}, tw[4] = {t4.x, t4.y, t4.z, t4.w};
        float2 cs = splat(0.f), ct = splat(0.f);     // per chunk first: a running sum takes one addition per chunk
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float2 sf = fadd2(unpack_bf16x2(sw[i]), nms), tf = fadd2(unpack_bf16x2(tw[i]), nmt);
          const float2 d = ffma2(sf, neg1, tf);
          const float2 es = ex2f2(fmul2(sf, cc));
          const float2 et = ex2f2(fmul2(tf, cc));
          cs = i == 0 ? es : fadd2(cs, es);
          ct = i == 0 ? et : fadd2(ct, et);
          Td = ffma2(et, d, Td);
          const float2 d2 = fmul2(d, d);
          M1 = ffma2(es, d, M1);
          const float2 u = fmul2(es, d2);
          M2 = fadd2(M2, u);
          M3 = ffma2(u, d, M3);
          M4 = ffma2(u, d2, M4);
        }
        Ss = fadd2(Ss, cs);
        St = fadd2(St, ct);
      }
      double a[7] = {vf_tot(Ss), vf_tot(St), vf_tot(Td), vf_tot(M1), vf_tot(M2), vf_tot(M3), vf_tot(M4)};
      vf_block_sum<7>(a, red);
      if (tid == 0) {
        int am = 0x7fffffff;                       // lowest index of the teacher's maximum inside its first chunk
        if (n_chunks > 0 && ac != 0x7fffffff) {
          for (int i = 7; i >= 0; --i) if (__bfloat162float(t[(size_t)ac * 8 + i]) == mt) am = ac * 8 + i;
        }
        bool finite = true;
#pragma unroll
        for (int k = 0; k < 7; ++k) finite = finite && isfinite(a[k]);
        finite = finite && (n_chunks == 0 || (ms > -1e30f && mt > -1e30f && ms < 1e30f && mt < 1e30f));
        const int x = S.proposal[row] - S.v0;
        const bool own = x >= 0 && x < Vl;
        for (int k = 0; k < SAKI_VSHARD_PARTIALS; ++k) out[k] = 0.0;
        out[0] = (double)ms; out[1] = (double)mt; out[2] = am == 0x7fffffff ? 2147483647.0 : (double)(S.v0 + am);
        out[3] = finite ? 1.0 : 0.0;
        if (finite && n_chunks > 0) {
          const double r2 = rtau * rtau, D = (double)mtc - (double)msc;
          a[2] += D * a[1];
          vf_uncentre(D, a[0], a[3], a[4], a[5], a[6]);
          out[4] = a[0]; out[5] = a[1]; out[6] = a[2] * rtau;
          out[7] = a[3] * rtau; out[8] = a[4] * r2; out[12] = a[5] * r2 * rtau; out[13] = a[6] * r2 * r2;
        }
        out[9] = own ? (double)__bfloat162float(s[x]) : 0.0; out[10] = own ? (double)__bfloat162float(t[x]) : 0.0;
        out[11] = own ? 1.0 : 0.0;
      }
    } else if (STAGE == 1) {
      // ---- stage B: one evaluation at the row's current beta, under the row's shift (its maxima: no factor)
      if ((int)st[VS_MODE] != VS_SOLVING) {        // (block-uniform)
        if (tid < SAKI_VSHARD_PARTIALS) out[tid] = 0.0;
        continue;
      }
      const double beta = st[VS_BETA];
      float cb = (float)(c64 * beta);
      const float ccb = c32 - cb;                  // the exponent is formed as (c - cb) s' + cb t'
      cb = c32 - ccb;                              // (so that the pair adds up to c exactly)
      const float msf = (float)st[VS_MS], mtf = (float)st[VS_MT];
      const float2 cbb = splat(cb), ccbb = splat(ccb), nms = splat(-msf), nmt = splat(-mtf);
      float2 S0 = splat(0.f), S1 = splat(0.f), S2 = splat(0.f), S3 = splat(0.f), S4 = splat(0.f);
#pragma unroll 2
      for (int c = tid; c < n_chunks; c += FT) {
        const uint4 s4 = vf_ld(s + (size_t)c * 8), t4 = vf_ld(t + (size_t)c * 8);
        const uint32_t sw[4] = {s4.x, s4.y, s4.z, s4.w}, tw[4] = {t4.x, t4.y, t4.z, t4.w};
float2 c0 = splat(0.f), c1 = splat(0.f);      // the chunk's share of S0 and S1
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float2 sf = fadd2(unpack_bf16x2(sw[i]), nms), tf = fadd2(unpack_bf16x2(tw[i]), nmt);
          const float2 d = ffma2(sf, neg1, tf);
          const float2 e = ex2f2(ffma2(tf, cbb, fmul2(sf, ccbb)));
          const float2 d2 = fmul2(d, d);
          c0 = i == 0 ? e : fadd2(c0, e);
          c1 = i == 0 ? fmul2(e, d) : ffma2(e, d, c1);
          const float2 u = fmul2(e, d2);
          S2 = fadd2(S2, u);
          S3 = ffma2(u, d, S3);
          S4 = ffma2(u, d2, S4);
        }
        S0 = fadd2(S0, c0);
        S1 = fadd2(S1, c1);
      }
      double a[5] = {vf_tot(S0), vf_tot(S1), vf_tot(S2), vf_tot(S3), vf_tot(S4)};
      vf_block_sum<5>(a, red);
      if (tid == 0) {
        const double r2 = rtau * rtau;
        vf_uncentre((double)mtf - (double)msf, a[0], a[1], a[2], a[3], a[4]);
        for (int k = 0; k < SAKI_VSHARD_PARTIALS; ++k) out[k] = 0.0;
        out[0] = a[0]; out[1] = a[1] * rtau; out[2] = a[2] * r2; out[3] = a[3] * r2 * rtau; out[4] = a[4] * r2 * r2;
      }
    } else if (STAGE == 2) {
      // ---- stage C: the slice's share of TV and KL(q||p); the student's logit at the teacher's argmax
      const bool live = (int)st[VS_MODE] == VS_SETTLED;
      const double lam = st[VS_LAM];
      double a[3] = {0.0, 0.0, 0.0};
      double fq = 0.0, D = 0.0;
      if (live && lam > 0.0) {
        const double lse_s = st[VS_LSE_S], lse_t = st[VS_LSE_T], logZ = st[VS_LOGZ];
        float cl = (float)(c64 * lam);
        const float ccl = c32 - cl;
        cl = c32 - ccl;
        const float msf = (float)st[VS_MS], mtf = (float)st[VS_MT];
        D = (double)mtf - (double)msf;
        // p = 2^(c s' - kp2), q = 2^((c - cl) s' + cl t' - kq2); whole-number shifts kpi <= kp2, kqi <= kq2 (both
        // arguments stay below 1), the factors between them applied in float64
        // (with the log-sum-exps relative to the maxima: what the sums of 2^(c s'), 2^(c t') came to)
        const double ls = lse_s - st[VS_MS] * rtau, lt = lse_t - st[VS_MT] * rtau;
        const double kp2 = ls * VF_LOG2E, kq2 = ((1.0 - lam) * ls + lam * lt + logZ) * VF_LOG2E;
        const float kpi = floorf((float)kp2 - 1e-3f), kqi = floorf((float)kq2 - 1e-3f);
        const double fp = exp2((double)kpi - kp2);
        fq = exp2((double)kqi - kq2);
        const float2 cll = splat(cl), ccll = splat(ccl), kpp = splat(-kpi), kqq = splat(-kqi), nrho = splat(-(float)(fp / fq));
        const float2 nms = splat(-msf), nmt = splat(-mtf);
        float2 R = splat(0.f), Sq = splat(0.f), Sqd = splat(0.f);
#pragma unroll 2
        for (int c = tid; c < n_chunks; c += FT) {
          const uint4 s4 = vf_ld(s + (size_t)c * 8), t4 = vf_ld(t + (size_t)c * 8);
          const uint32_t sw[4] = {s4.x, s4.y, s4.z, s4.w}, tw[4] = {t4.x, t4.y, t4.z, t4.w};
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            const float2 sf = fadd2(unpack_bf16x2(sw[i]), nms), tf = fadd2(unpack_bf16x2(tw[i]), nmt);
            const float2 d = ffma2(sf, neg1, tf);
            const float2 ep = ex2f2(ffma2(sf, cc, kpp));
            const float2 eq = ex2f2(ffma2(tf, cll, ffma2(sf, ccll, kqq)));
            float2 r = ffma2(ep, nrho, eq);          // (q_i - p_i) / fq
            r.x = fmaxf(r.x, 0.f); r.y = fmaxf(r.y, 0.f);
            R = fadd2(R, r);
            Sq = fadd2(Sq, eq);
            Sqd = ffma2(eq, d, Sqd);
          }
        }
        a[0] = vf_tot(R); a[1] = vf_tot(Sq); a[2] = vf_tot(Sqd);
      }
      vf_block_sum<3>(a, red);
      if (tid == 0) {
        for (int k = 0; k < SAKI_VSHARD_PARTIALS; ++k) out[k] = 0.0;
        if (live && lam > 0.0) {
          const double cc0 = st[VS_LSE_T] - st[VS_LSE_S];      // log q - log p = lam ((t - s)/tau - cc0) - log Z
          out[0] = fq * a[0];
          out[1] = fq * (lam * rtau * (a[2] + D * a[1]) - (lam * cc0 + st[VS_LOGZ]) * a[1]);
        }
        const int vs = (int)st[VS_VSTAR] - S.v0;
        out[2] = (live && vs >= 0 && vs < Vl) ? (double)__bfloat162float(s[vs]) : 0.0;
      }
    } else {
      // ---- stage D: the gradient slice; on the owning rank the residual draw
      const int mode = (int)st[VS_MODE];
      __nv_bfloat16* g = dlogits ? (__nv_bfloat16*)dlogits + row * ld_g : nullptr;
      if (g) {
        const double sc = mode == VS_FLAGGED ? 0.0 : grad_scale * st[VS_COEF] * rtau;
        if (sc == 0.0) {
          for (int c = tid; c < n_chunks; c += FT) *reinterpret_cast<uint4*>(g + (size_t)c * 8) = make_uint4(0, 0, 0, 0);
        } else {
          const float msf = (float)st[VS_MS];
          const double kp2 = (st[VS_LSE_S] - st[VS_MS] * rtau) * VF_LOG2E;
          const float kpi = floorf((float)kp2 - 1e-3f);
          const float kgf = (float)(sc * exp2((double)kpi - kp2)), scf = (float)sc;     // gradient entry = e_p * kgf (- sc at the token)
          const float2 kpp = splat(-kpi), kgg = splat(kgf), nms = splat(-msf);
          const int tok = (int)st[VS_TOK] - S.v0;
          const int tok_c = (tok >= 0 && tok < Vl) ? (tok >> 3) : -1;
          for (int c = tid; c < n_chunks; c += FT) {
            const uint4 s4 = vf_ld(s + (size_t)c * 8);
            const uint32_t sw[4] = {s4.x, s4.y, s4.z, s4.w};
            float gv[8];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
              const float2 ep = ex2f2(ffma2(fadd2(unpack_bf16x2(sw[i]), nms), cc, kpp));
              const float2 v = fmul2(ep, kgg);
              gv[2 * i] = v.x; gv[2 * i + 1] = v.y;
            }
            if (c == tok_c) {
#pragma unroll
              for (int i = 0; i < 8; ++i) if (i == (tok & 7)) gv[i] -= scf;
            }
            *reinterpret_cast<uint4*>(g + (size_t)c * 8) =
                make_uint4(pack_bf16x2(gv[0], gv[1]), pack_bf16x2(gv[2], gv[3]), pack_bf16x2(gv[4], gv[5]), pack_bf16x2(gv[6], gv[7]));
          }
        }
      }
      if (tid == 0) stoken = -1;
      __syncthreads();
      const bool mine = mode == VS_SETTLED && st[VS_CORR] != 0.0 && (int)st[VS_OWNER] == S.rank;
      if (mine) vf_draw(s, t, n_chunks, c32, c64, S.tau, st, red, &stoken);
      __syncthreads();
      if (tid == 0) {
        for (int k = 0; k < SAKI_VSHARD_PARTIALS; ++k) out[k] = 0.0;
        out[0] = -1.0;
        if (mine && stoken >= 0 && stoken < Vl) {
          out[0] = (double)(S.v0 + stoken);
          out[1] = (double)__bfloat162float(s[stoken]); out[2] = (double)__bfloat162float(t[stoken]);
        }
      }
      __syncthreads();
    }
  }
}

__global__ void vs_combine_kernel(const VsConsts C, const int stage, const double* part, double* state, const saki_out o,
                                  unsigned int* n_solving) {
  const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= C.N) return;
  double* st = state + i * SAKI_VSHARD_STATE;
  if (stage == 0) { vs_combine_a(C, i, part, st); if ((int)st[VS_MODE] == VS_SOLVING && n_solving) atomicAdd(n_solving, 1u); }
  else if (stage == 1) { if (vs_combine_b(C, i, part, st) && n_solving) atomicAdd(n_solving, 1u); }
  else if (stage == 2) vs_combine_c(C, i, part, st);
  else vs_combine_d(C, i, part, st, o);
}

// the call may use the float32 slice kernels: a property of the call's arguments alone, so that every rank's
// combine takes the same decisions (a rank whose own slice is not aligned for them simply computes in float64)
static bool vshard_fast_call(const saki_vshard_in& in, bool allow_fast) {
  return allow_fast && in.dtype == SAKI_BF16 && in.eps >= 0.02f;   // below, KL needs the float64 sums (or a quadrature)
}

cudaError_t launch_vshard_partial(const saki_vshard_in& in, int stage, const double* state, double* partial, void* dlogits,
                                  int64_t ld_g, float grad_scale, bool allow_fast, cudaStream_t st) {
  VsSlice S;
  S.s = in.student_logits; S.t = in.teacher_logits; S.ld_s = in.ld_s; S.ld_t = in.ld_t; S.N = in.N;
  S.V_local = in.V_local; S.v0 = in.v0; S.rank = in.rank; S.tau = (double)in.temperature; S.proposal = in.proposal;
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  auto al16 = [](const void* q) { return ((uintptr_t)q & 15) == 0; };
  const bool fast = vshard_fast_call(in, allow_fast) && in.V_local % 8 == 0 && in.ld_s % 8 == 0 && in.ld_t % 8 == 0 &&
                    al16(in.student_logits) && al16(in.teacher_logits) && (!dlogits || (al16(dlogits) && ld_g % 8 == 0));
  if (fast) {
    const int fgrid = (int)(in.N < 8LL * sms ? in.N : 8LL * sms);
    const double gs = (double)grad_scale;
    if (stage == 0) vs_fast_kernel<0><<<fgrid, FT, 0, st>>>(S, state, partial, dlogits, ld_g, gs);
    else if (stage == 1) vs_fast_kernel<1><<<fgrid, FT, 0, st>>>(S, state, partial, dlogits, ld_g, gs);
    else if (stage == 2) vs_fast_kernel<2><<<fgrid, FT, 0, st>>>(S, state, partial, dlogits, ld_g, gs);
    else vs_fast_kernel<3><<<fgrid, FT, 0, st>>>(S, state, partial, dlogits, ld_g, gs);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess || stage == 0) return e;          // no row is marked for float64 before the first combine
  }
  const int grid = (int)(in.N < 3LL * sms ? in.N : 3LL * sms);
  if (in.dtype == SAKI_BF16)
    vs_partial_kernel<__nv_bfloat16><<<dim3(grid, 1, 1), VT, 0, st>>>(S, stage, state, partial, dlogits, ld_g, (double)grad_scale, fast);
  else
    vs_partial_kernel<float><<<dim3(grid, 1, 1), VT, 0, st>>>(S, stage, state, partial, dlogits, ld_g, (double)grad_scale, false);
  return cudaGetLastError();
}

static VsConsts consts_of(const saki_vshard_in& in, bool allow_fast) {
  VsConsts c;
  c.N = in.N; c.V = in.V; c.world = in.world; c.eps = (double)in.eps; c.tau = (double)in.temperature;
  c.seed = in.seed; c.row_offset = in.row_offset; c.proposal = in.proposal; c.mask = in.mask;
  c.fast = vshard_fast_call(in, allow_fast) ? 1 : 0;
  return c;
}

cudaError_t launch_vshard_combine(const saki_vshard_in& in, int stage, const double* gathered, double* state, const saki_out& out,
                                  unsigned int* n_solving, bool allow_fast, cudaStream_t st) {
  const VsConsts c = consts_of(in, allow_fast);
  const int th = 128;
  vs_combine_kernel<<<(unsigned)((in.N + th - 1) / th), th, 0, st>>>(c, stage, gathered, state, out, n_solving);
  return cudaGetLastError();
}

// the same combine on HOST buffers (a caller without a GPU at hand, and the multi-process tests of the exchange)
int vshard_combine_host(const saki_vshard_in& in, int stage, const double* gathered, double* state, const saki_out& out,
                        bool allow_fast) {
  const VsConsts c = consts_of(in, allow_fast);
  int solving = 0;
  for (int64_t i = 0; i < in.N; ++i) {
    double* st = state + i * SAKI_VSHARD_STATE;
    if (stage == 0) { vs_combine_a(c, i, gathered, st); solving += (int)st[VS_MODE] == VS_SOLVING; }
    else if (stage == 1) solving += vs_combine_b(c, i, gathered, st);
    else if (stage == 2) vs_combine_c(c, i, gathered, st);
    else vs_combine_d(c, i, gathered, st, out);
  }
  return solving;
}

}  // namespace saki
