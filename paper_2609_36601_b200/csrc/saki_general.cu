// General row kernel: one thread block per position, any V, dtype and strides.
// All arithmetic is float64 and every pass re-reads the row from global
// memory (L2 after the first pass).  It is the library's fallback for layouts
// the bf16 streaming kernels do not serve (fp32 logits, odd strides, ragged V), their second tier
// (rows they hand over through the row list), and the slow, careful path.  Steps follow the method's definition:
//   log-softmax x2 -> lambda (Eqs. "bridge", "trust_region") -> TV and the
//   maximal coupling (Eqs. "accept", "residual") -> routed loss (Eqs.
//   "k1_loss_token", "teacher_mode_loss") -> gradient (Eq. "general_objective").
// In list mode (the second tier of the bf16 kernels: usually a handful of rows) a short list is routed with a
// row spread over a cluster of 8 thread blocks, which add up their block totals through distributed shared
// memory: one block per row leaves a row of 151,936 elements 1.3 ms on a single SM, a cluster 0.47 ms.  A
// long list keeps one block per row (18 clusters are fewer than 148 blocks).  The host does not know the
// list's length when it launches, so both forms are launched and each returns at once unless the length
// is in its range.
#include "saki_common.cuh"
#include <cooperative_groups.h>
#include <math_constants.h>

namespace cg = cooperative_groups;

namespace saki {

constexpr int GT = 512;        // threads per block
constexpr int GW = GT / 32;    // warps per block

__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}

// Sum NV doubles over the block (CS == 1) or over the cluster's CS blocks; every thread gets the same totals
// (summed in a fixed order: by block rank, then by warp, so results are reproducible).  `sh` is the same
// shared-memory array in every block of the cluster.
template <int NV, int CS>
__device__ __forceinline__ void block_sum(double (&v)[NV], double* sh) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
#pragma unroll
  for (int k = 0; k < NV; ++k) v[k] = warp_sum(v[k]);
  if (lane == 0) {
#pragma unroll
    for (int k = 0; k < NV; ++k) sh[k * GW + warp] = v[k];
  }
  if constexpr (CS == 1) {
    __syncthreads();
#pragma unroll
    for (int k = 0; k < NV; ++k) {
      double a = 0.0;
#pragma unroll
      for (int w = 0; w < GW; ++w) a += sh[k * GW + w];
      v[k] = a;
    }
    __syncthreads();
  } else {
    cg::cluster_group cl = cg::this_cluster();
    cl.sync();
#pragma unroll
    for (int k = 0; k < NV; ++k) v[k] = 0.0;
    for (int r = 0; r < CS; ++r) {
      const double* rs = cl.map_shared_rank(sh, r);
#pragma unroll
      for (int k = 0; k < NV; ++k) {
        double a = 0.0;
#pragma unroll
        for (int w = 0; w < GW; ++w) a += rs[k * GW + w];
        v[k] += a;
      }
    }
    cl.sync();
  }
}

struct Shared {
  double red[4 * GW];
  double warp_tot[GW];
  float fmax_s[GW], fmax_t[GW];
  int arg_t[GW];
  int token;
  int finite;
  double wt_all[GW * 8];   // every warp's draw weight of the cluster, in segment order
};

// CS: blocks per row (1, or a cluster of CS blocks that share the row element by element)
template <typename T, int CS>
__global__ void __launch_bounds__(GT) general_kernel(const RowParams P) {
  __shared__ Shared sh;
  const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
  const int V = P.V;
  const double tau = (double)P.temperature;
  const double eps = (double)P.eps;
  int crank = 0;
  if constexpr (CS > 1) crank = (int)cg::this_cluster().block_rank();
  const int ET = GT * CS, e0 = crank * GT + tid;     // the cluster's threads take the elements e0, e0 + ET, ...

  const int64_t n_work = P.from_list ? (int64_t)*P.redo_count : P.n_rows;
  // list mode is launched twice: a cluster per row for a short list, a block per row for a long one
  if (P.from_list && P.list_max > 0 && (n_work < P.list_min || n_work > P.list_max)) return;
  for (int64_t item = blockIdx.x / CS; item < n_work; item += gridDim.x / CS) {
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
    for (int v = e0; v < V; v += ET) {
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
    if constexpr (CS == 1) {
      ms = sh.fmax_s[0]; mt = sh.fmax_t[0]; am = sh.arg_t[0];
#pragma unroll
      for (int w = 1; w < GW; ++w) {
        ms = fmaxf(ms, sh.fmax_s[w]);
        if (sh.fmax_t[w] > mt || (sh.fmax_t[w] == mt && sh.arg_t[w] < am)) { mt = sh.fmax_t[w]; am = sh.arg_t[w]; }
      }
      __syncthreads();
    } else {
      cg::cluster_group cl = cg::this_cluster();
      if (tid == 0) sh.finite = finite;
      cl.sync();
      ms = -CUDART_INF_F; mt = -CUDART_INF_F; am = 0x7fffffff; finite = 1;
      for (int r = 0; r < CS; ++r) {
        const Shared* rs = cl.map_shared_rank(&sh, r);
        finite &= rs->finite;
        for (int w = 0; w < GW; ++w) {
          ms = fmaxf(ms, rs->fmax_s[w]);
          const float omt = rs->fmax_t[w];
          const int oam = rs->arg_t[w];
          if (omt > mt || (omt == mt && oam < am)) { mt = omt; am = oam; }
        }
      }
      cl.sync();
    }

    uint32_t status = 0;
    if (!finite) status = SAKI_ROW_NONFINITE;
    else if (!bonus && (x < 0 || x >= V)) status = SAKI_ROW_BAD_ID;
    if (status) {   // flagged row: zero outputs, zero gradient row
      if (tid == 0 && crank == 0) {
        write_row(P.out, row, zero_row(status), !P.spec);
        atomicAdd(P.flagged, 1ull);
      }
      if (g) for (int v = e0; v < V; v += ET) st_from_float(g, v, 0.f);
      continue;
    }

    // ---- pass 1: log-sum-exp of both rows
    const double zms = (double)ms / tau, zmt = (double)mt / tau;
    double acc2[2] = {0.0, 0.0};
    for (int v = e0; v < V; v += ET) {
      acc2[0] += exp((double)ld_as_float(s, v) / tau - zms);
      acc2[1] += exp((double)ld_as_float(t, v) / tau - zmt);
    }
    block_sum<2, CS>(acc2, sh.red);
    const double lse_s = zms + log(acc2[0]), lse_t = zmt + log(acc2[1]);

    // ---- lambda
    double lam = 0.0, Lam = 0.0;   // Lam = log Z(lambda) = log sum p exp(lambda d)
    if (!(eps > 0.0)) {
      status |= SAKI_ROW_EPS_ZERO;
    } else {
      // pass 2: KL(T||p) and the variance of d under p (initial guess)
      double a3[3] = {0.0, 0.0, 0.0};
      for (int v = e0; v < V; v += ET) {
        const double lp = (double)ld_as_float(s, v) / tau - lse_s;
        const double lT = (double)ld_as_float(t, v) / tau - lse_t;
        const double d = lT - lp, p = exp(lp);
        a3[0] += exp(lT) * d;
        a3[1] += p * d;
        a3[2] += p * d * d;
      }
      block_sum<3, CS>(a3, sh.red);
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
        if (P.from_list && P.redo_guess) {       // the float32 kernel's value of lambda, good to ~1e-5: two steps from here
          const double g0 = (double)P.redo_guess[item];
          if (g0 > 0.0 && g0 < 1.0) beta = g0;
        }
        for (int it = 0; it < 100; ++it) {
          double a[3] = {0.0, 0.0, 0.0};
          for (int v = e0; v < V; v += ET) {
            const double lp = (double)ld_as_float(s, v) / tau - lse_s;
            const double lT = (double)ld_as_float(t, v) / tau - lse_t;
            const double d = lT - lp, e = exp(lp + beta * d);
            a[0] += e;
            a[1] += e * d;
            a[2] += e * d * d;
          }
          block_sum<3, CS>(a, sh.red);
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
      for (int v = e0; v < V; v += ET) {
        const double lp = (double)ld_as_float(s, v) / tau - lse_s;
        const double lT = (double)ld_as_float(t, v) / tau - lse_t;
        z1[0] += exp(lp + lam * (lT - lp));
      }
      block_sum<1, CS>(z1, sh.red);
      Lam = log(z1[0]);
    }

    // ---- TV, KL at lambda; partial sums kept per warp segment in index order
    const int NWC = GW * CS;                              // warps of the cluster, in index order of their segments
    const int seg = (V + NWC - 1) / NWC;
    const int gw = crank * GW + warp;
    const int seg0 = min(V, gw * seg), seg1 = min(V, seg0 + seg);
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
      block_sum<2, CS>(klp, sh.red);   // its first barrier publishes warp_tot (to the cluster)
      kl = klp[0];
      tv_true = klp[1];
      if (tid < NWC) {                 // every warp's weight of the cluster, in segment order, into this block's copy
        if constexpr (CS == 1) sh.wt_all[tid] = sh.warp_tot[tid];
        else sh.wt_all[tid] = cg::this_cluster().map_shared_rank(&sh, tid / GW)->warp_tot[tid % GW];
      }
      __syncthreads();
      for (int w = 0; w < NWC; ++w) tv += sh.wt_all[w];
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
      for (int w = 0; w < NWC; ++w) {
        if (before + sh.wt_all[w] > target) { owner = w; break; }
        before += sh.wt_all[w];
      }
      bool take_last = false;
      if (owner < 0) {   // rounding left no crossing: last index with positive weight
        take_last = true;
        before = 0.0;
        for (int w = NWC - 1; w >= 0; --w) if (sh.wt_all[w] > 0.0) { owner = w; break; }
        if (owner < 0) owner = 0;
      }
      if (tid == 0) sh.token = -1;
      __syncthreads();
      if (gw == owner) {
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
      if constexpr (CS == 1) {
        __syncthreads();
        y = sh.token;
        __syncthreads();
      } else {             // the owning warp's block holds the token
        cg::cluster_group cl = cg::this_cluster();
        cl.sync();
        y = cl.map_shared_rank(&sh, owner / GW)->token;
        cl.sync();
      }
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
    if (tid == 0 && crank == 0) {
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
      for (int v = e0; v < V; v += ET) {
        const double p = exp((double)ld_as_float(s, v) / tau - lse_s);
        const double gv = sc * (p - (v == tok ? 1.0 : 0.0));
        if constexpr (sizeof(T) == 2) g[v] = __double2bfloat16(gv);
        else g[v] = (float)gv;
      }
    }
  }
  if constexpr (CS > 1) cg::this_cluster().sync();   // no block leaves while a peer may still read its shared memory
}

constexpr int LIST_CS = 8;   // blocks per row in list mode

template <typename T>
static cudaError_t launch_list(const RowParams& p, int sms, cudaStream_t st) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)((sms / LIST_CS) * LIST_CS), 1, 1);
  cfg.blockDim = dim3(GT, 1, 1);
  cfg.dynamicSmemBytes = 0;
  cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeClusterDimension;
  at[0].val.clusterDim.x = LIST_CS; at[0].val.clusterDim.y = 1; at[0].val.clusterDim.z = 1;
  cfg.attrs = at; cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, general_kernel<T, LIST_CS>, p);
}

cudaError_t launch_general(const RowParams& p, int dtype, cudaStream_t st, int* n_launches) {
  if (p.n_rows <= 0) return cudaSuccess;
  int dev = 0, sms = 148;
  cudaGetDevice(&dev);
  cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
  if (n_launches) *n_launches += 1;
  RowParams q = p;
  q.list_min = 0; q.list_max = 0;
  if (p.from_list && sms >= LIST_CS) {   // the rows the bf16 kernels handed over: a cluster per row while they are few
    q.list_min = 0; q.list_max = 3 * (sms / LIST_CS);
    cudaError_t e = dtype == SAKI_BF16 ? launch_list<__nv_bfloat16>(q, sms, st) : launch_list<float>(q, sms, st);
    if (e != cudaSuccess) return e;
    if (n_launches) *n_launches += 1;
    q.list_min = q.list_max + 1; q.list_max = 0x7fffffff;
  }
  const int64_t cap = (int64_t)sms * (p.from_list ? 1 : 3);
  const int grid = (int)(p.n_rows < cap ? p.n_rows : cap);
  if (dtype == SAKI_BF16) general_kernel<__nv_bfloat16, 1><<<grid, GT, 0, st>>>(q);
  else general_kernel<float, 1><<<grid, GT, 0, st>>>(q);
  return cudaGetLastError();
}

}  // namespace saki
