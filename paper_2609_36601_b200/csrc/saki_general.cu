// General row kernel: one thread block per position, any V, dtype and strides.
// All arithmetic is float64 and every pass re-reads the row from global
// memory (L2 after the first pass).  It is the library's fallback for layouts
// the bf16 streaming kernels do not serve (fp32 logits, odd strides, ragged V), their second tier
// (rows they hand over through the row list), and the slow, careful path.  Steps follow the method's definition:
//   log-softmax x2 -> lambda (Eqs. "bridge", "trust_region") -> TV and the
//   maximal coupling (Eqs. "accept", "residual") -> routed loss (Eqs.
//   "k1_loss_token", "teacher_mode_loss") -> gradient (Eq. "general_objective").
#include "saki_common.cuh"
#include <math_constants.h>

namespace saki {

constexpr int GT = 512;        // threads per block
constexpr int GW = GT / 32;    // warps per block

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Sum NV doubles over the block; every thread gets the same totals (summed in
// a fixed order, so results are reproducible).
template <int NV>
__device__ __forceinline__ void block_sum(double (&v)[NV], double* sh) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int k = 0; k < NV; ++k) v[k] = warp_sum(v[k]);
  if (lane == 0) {
#pragma unroll
    for (int k = 0; k < NV; ++k) sh[k * GW + warp] = v[k];
  }
  __syncthreads();
#pragma unroll
  for (int k = 0; k < NV; ++k) {
    double a = 0.0;
#pragma unroll
    for (int w = 0; w < GW; ++w) a += sh[k * GW + w];
    v[k] = a;
  }
  __syncthreads();
}

struct Shared {
  double red[4 * GW];
  double warp_tot[GW];
  float fmax_s[GW], fmax_t[GW];
  int arg_t[GW];
  int token;
};

template <typename T>
__global__ void __launch_bounds__(GT) general_kernel(const RowParams P) {
  __shared__ Shared sh;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int V = P.V;
  const double tau = (double)P.temperature;
  const double eps = (double)P.eps;

  const int64_t n_work = P.from_list ? (int64_t)*P.redo_count : P.n_rows;
  for (int64_t item = blockIdx.x; item < n_work; item += gridDim.x) {
    const int64_t row = P.from_list ? (int64_t)P.redo_list[item] : item;   // list mode: rows handed over by the float32 kernels
    const int64_t b = row / P.K1;
    const int j = (int)(row - b * P.K1);
    const T* s = (const T*)P.s + b * P.s_seq + (int64_t)j * P.s_pos;
    const T* t = (const T*)P.t + b * P.t_seq + (int64_t)j * P.t_pos;
    const bool bonus = P.spec && (j == P.K1 - 1);
    int x = 0;
    if (!bonus) x = P.spec ? P.proposal[b * P.prop_ld + j] : P.proposal[row];
    const uint64_t rid = P.row_offset + (uint64_t)row;
    const bool masked = (P.mask != nullptr) && (P.mask[row] == 0);
    T* g = P.dlogits ? (T*)P.dlogits + row * P.ld_g : nullptr;

    // ---- pass 0: maxima, teacher argmax (lowest index among ties), finiteness
    float ms = -CUDART_INF_F, mt = -CUDART_INF_F;
    int am = 0x7fffffff;
    int finite = 1;
    for (int v = tid; v < V; v += GT) {
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
    if (lane == 0) { sh.fmax_s[warp] = ms; sh.fmax_t[warp] = mt; sh.arg_t[warp] = am; }
    finite = __syncthreads_and(finite);
    ms = sh.fmax_s[0]; mt = sh.fmax_t[0]; am = sh.arg_t[0];
#pragma unroll
    for (int w = 1; w < GW; ++w) {
      ms = fmaxf(ms, sh.fmax_s[w]);
      if (sh.fmax_t[w] > mt || (sh.fmax_t[w] == mt && sh.arg_t[w] < am)) { mt = sh.fmax_t[w]; am = sh.arg_t[w]; }
    }
    __syncthreads();

    uint32_t status = 0;
    if (!finite) status = SAKI_ROW_NONFINITE;
    else if (!bonus && (x < 0 || x >= V)) status = SAKI_ROW_BAD_ID;
    if (status) {   // flagged row: zero outputs, zero gradient row
      if (tid == 0) {
        write_row(P.out, row, zero_row(status), !P.spec);
        atomicAdd(P.flagged, 1ull);
      }
      if (g) for (int v = tid; v < V; v += GT) st_from_float(g, v, 0.f);
      continue;
    }

    // ---- pass 1: log-sum-exp of both rows
    const double zms = (double)ms / tau, zmt = (double)mt / tau;
    double acc2[2] = {0.0, 0.0};
    for (int v = tid; v < V; v += GT) {
      acc2[0] += exp((double)ld_as_float(s, v) / tau - zms);
      acc2[1] += exp((double)ld_as_float(t, v) / tau - zmt);
    }
    block_sum<2>(acc2, sh.red);
    const double lse_s = zms + log(acc2[0]), lse_t = zmt + log(acc2[1]);

    // ---- lambda
    double lam = 0.0, Lam = 0.0;   // Lam = log Z(lambda) = log sum p exp(lambda d)
    if (!(eps > 0.0)) {
      status |= SAKI_ROW_EPS_ZERO;
    } else {
      // pass 2: KL(T||p) and the variance of d under p (initial guess)
      double a3[3] = {0.0, 0.0, 0.0};
      for (int v = tid; v < V; v += GT) {
        const double lp = (double)ld_as_float(s, v) / tau - lse_s;
        const double lT = (double)ld_as_float(t, v) / tau - lse_t;
        const double d = lT - lp, p = exp(lp);
        a3[0] += exp(lT) * d;
        a3[1] += p * d;
        a3[2] += p * d * d;
      }
      block_sum<3>(a3, sh.red);
      if (a3[0] <= eps) {
        lam = 1.0;
        status |= SAKI_ROW_SATURATED;
      } else {
        // KL(q_beta||p) is increasing in beta with slope beta Var_q(d):
        // Newton on KL(beta) = eps, kept inside a bisection bracket.
        const double varp = a3[2] - a3[1] * a3[1];
        double lo = 0.0, hi = 1.0;
        double beta = sqrt(2.0 * eps / fmax(varp, 1e-300));
        if (!(beta > 0.0 && beta < 1.0)) beta = 0.5;
        for (int it = 0; it < 100; ++it) {
          double a[3] = {0.0, 0.0, 0.0};
          for (int v = tid; v < V; v += GT) {
            const double lp = (double)ld_as_float(s, v) / tau - lse_s;
            const double lT = (double)ld_as_float(t, v) / tau - lse_t;
            const double d = lT - lp, e = exp(lp + beta * d);
            a[0] += e;
            a[1] += e * d;
            a[2] += e * d * d;
          }
          block_sum<3>(a, sh.red);
          const double E = a[1] / a[0], var = a[2] / a[0] - E * E;
          const double kl = beta * E - log(a[0]);
          if (kl <= eps) lo = beta; else hi = beta;
          if (hi - lo < 1e-15) break;
          const double step = (eps - kl) / (beta * var);
          // at the root to rounding: stop here (a step that small can fall outside the bracket, and the
          // bisection that would follow costs some thirty more passes for nothing)
          if (fabs(step) < 1e-13) { beta = fmin(fmax(beta + step, lo), hi); break; }
          double nb = beta + step;
          if (!(nb > lo && nb < hi)) nb = 0.5 * (lo + hi);
          beta = nb;
        }
        lam = beta;
      }
      // log Z at the final coefficient
      double z1[1] = {0.0};
      for (int v = tid; v < V; v += GT) {
        const double lp = (double)ld_as_float(s, v) / tau - lse_s;
        const double lT = (double)ld_as_float(t, v) / tau - lse_t;
        z1[0] += exp(lp + lam * (lT - lp));
      }
      block_sum<1>(z1, sh.red);
      Lam = log(z1[0]);
    }

    // ---- TV, KL at lambda; partial sums kept per warp segment in index order
    const int seg = (V + GW - 1) / GW;
    const int seg0 = warp * seg, seg1 = min(V, seg0 + seg);
    double tv = 0.0, kl = 0.0, tv_true = 0.0;
    if (lam > 0.0 || bonus) {
      double part = 0.0, klp[2] = {0.0, 0.0};   // klp[1]: TV of a bonus row (its draw weights are q)
      for (int v = seg0 + lane; v < seg1; v += 32) {
        const double lp = (double)ld_as_float(s, v) / tau - lse_s;
        const double lT = (double)ld_as_float(t, v) / tau - lse_t;
        const double lq = lp + lam * (lT - lp) - Lam;
        const double q = exp(lq);
        const double r = fmax(q - exp(lp), 0.0);
        part += bonus ? q : r;
        klp[0] += q * (lq - lp);
        klp[1] += r;
      }
      part = warp_sum(part);
      if (lane == 0) sh.warp_tot[warp] = part;
      block_sum<2>(klp, sh.red);   // contains the __syncthreads that publishes warp_tot
      kl = klp[0];
      tv_true = klp[1];
      for (int w = 0; w < GW; ++w) tv += sh.warp_tot[w];
    }

    // ---- the coupling decision (every thread computes the same scalars)
    double lp_x = 0.0, lT_x = 0.0, acc_p = 1.0;
    int corrected = 0;
    if (!bonus) {
      lp_x = (double)ld_as_float(s, x) / tau - lse_s;
      lT_x = (double)ld_as_float(t, x) / tau - lse_t;
      if (lam > 0.0) {
        acc_p = exp(fmin(0.0, lam * (lT_x - lp_x) - Lam));
        const double u = scalar_uniform(P.seed, rid, STAGE_ACCEPT);
        corrected = (u < acc_p) ? 0 : 1;
      }
    }
    int y = x;
    if (corrected || bonus) {
      // inverse CDF in index order: smallest index whose running sum exceeds u * total
      const double u = scalar_uniform(P.seed, rid, bonus ? STAGE_BONUS : STAGE_RESIDUAL);
      const double target = u * tv;
      int owner = -1;
      double before = 0.0;
      for (int w = 0; w < GW; ++w) {
        if (before + sh.warp_tot[w] > target) { owner = w; break; }
        before += sh.warp_tot[w];
      }
      bool take_last = false;
      if (owner < 0) {   // rounding left no crossing: last index with positive weight
        take_last = true;
        before = 0.0;
        for (int w = GW - 1; w >= 0; --w) if (sh.warp_tot[w] > 0.0) { owner = w; break; }
        if (owner < 0) owner = 0;
      }
      if (tid == 0) sh.token = -1;
      __syncthreads();
      if (warp == owner) {
        double running = before;
        int last_pos = -1, found = -1;
        for (int v0 = owner * seg; v0 < V && found < 0; v0 += 32) {
          const int v = v0 + lane;
          double r = 0.0;
          if (v < V) {
            const double lp = (double)ld_as_float(s, v) / tau - lse_s;
            const double lT = (double)ld_as_float(t, v) / tau - lse_t;
            const double q = exp(lp + lam * (lT - lp) - Lam);
            r = bonus ? q : fmax(q - exp(lp), 0.0);
          }
          double inc = r;
#pragma unroll
          for (int o = 1; o < 32; o <<= 1) {
            const double up = __shfl_up_sync(0xffffffffu, inc, o);
            if (lane >= o) inc += up;
          }
          const unsigned pos = __ballot_sync(0xffffffffu, r > 0.0);
          const unsigned hit = take_last ? 0u : __ballot_sync(0xffffffffu, (running + inc > target) && v < V);
          if (pos) last_pos = v0 + 31 - __clz(pos);
          if (hit) found = v0 + __ffs(hit) - 1;
          running += __shfl_sync(0xffffffffu, inc, 31);
        }
        if (found < 0) found = (last_pos >= 0) ? last_pos : (V - 1);
        if (lane == 0) sh.token = found;
      }
      __syncthreads();
      y = sh.token;
      __syncthreads();
    }

    // ---- routed loss and gradient coefficients
    const double lp_v = (double)ld_as_float(s, am) / tau - lse_s;   // log p(v*)
    double loss = 0.0, coef = 0.0;   // gradient = coef * (p - onehot(tok)) / tau
    int tok = 0;
    if (masked) {
      status |= SAKI_ROW_MASKED;
    } else if (!bonus) {
      if (!corrected) { loss = (lp_x - lT_x) * lp_x; coef = -(lp_x - lT_x); tok = x; }
      else { loss = -lp_v; coef = 1.0; tok = am; }
    }
    if (tid == 0) {
      RowResult r;
      r.corrected = corrected; r.token = y; r.vstar = am;
      r.lambda = (float)lam; r.kl = (float)(lam > 0.0 ? kl : 0.0);
      r.tv = (float)((lam > 0.0) ? (bonus ? tv_true : tv) : 0.0);
      r.accept = bonus ? 0.f : (float)acc_p;
      r.logp_x = (float)lp_x; r.logT_x = (float)lT_x;
      r.logq_x = bonus ? 0.f : (float)(lp_x + lam * (lT_x - lp_x) - Lam);
      const double lp_y = (double)ld_as_float(s, y) / tau - lse_s;
      const double lT_y = (double)ld_as_float(t, y) / tau - lse_t;
      r.logp_y = (float)lp_y;
      r.logq_y = (float)(lp_y + lam * (lT_y - lp_y) - Lam);
      r.logT_y = (float)lT_y;
      r.loss = (float)loss;
      r.status = status;
      write_row(P.out, row, r, !P.spec);
    }
    if (g) {
      const double sc = (double)P.grad_scale * coef / tau;
      for (int v = tid; v < V; v += GT) {
        const double p = exp((double)ld_as_float(s, v) / tau - lse_s);
        const double gv = sc * (p - (v == tok ? 1.0 : 0.0));
        if constexpr (sizeof(T) == 2) g[v] = __double2bfloat16(gv);
        else g[v] = (float)gv;
      }
    }
  }
}

cudaError_t launch_general(const RowParams& p, int dtype, cudaStream_t st, int* n_launches) {
  if (p.n_rows <= 0) return cudaSuccess;
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  const int64_t cap = (int64_t)sms * (p.from_list ? 1 : 3);
  const int grid = (int)(p.n_rows < cap ? p.n_rows : cap);
  if (dtype == SAKI_BF16) general_kernel<__nv_bfloat16><<<grid, GT, 0, st>>>(p);
  else general_kernel<float><<<grid, GT, 0, st>>>(p);
  if (n_launches) *n_launches += 1;
  return cudaGetLastError();
}

}  // namespace saki
