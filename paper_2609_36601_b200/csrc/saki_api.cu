// C ABI of the SAKI routing library: host-side validation, kernel selection,
// the proposal-sampling utility, the block-verification resolve and the
// host-buffer convenience entry.  See include/saki.h for the contract.
#include "saki_common.cuh"
#include <atomic>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <iterator>
#include <map>
#include <mutex>
#include <utility>
#include <vector>
#include <algorithm>

namespace saki {

static thread_local char g_err[512] = "";
static std::atomic<uint64_t> g_launches{0};
static std::atomic<int> g_kernel{0};
static std::atomic<int> g_spec_early_out{1};
static std::atomic<int> g_phase_clock{0};
static std::atomic<long long> g_wait_limit{0};
static thread_local int g_last_kernel = 0;

static int fail(int code, const char* fmt, ...) {
  va_list ap;
  va_start(ap, fmt);
  vsnprintf(g_err, sizeof(g_err), fmt, ap);
  va_end(ap);
  return code;
}
static int cuda_fail(cudaError_t e, const char* what) {
  return fail(SAKI_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

// device-resident count of flagged rows (one per device that loads the library)
__device__ unsigned long long g_flagged_rows = 0ull;

static int device_ready(unsigned long long** flagged) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return fail(SAKI_ERR_UNSUPPORTED, "no CUDA device: %s", cudaGetErrorString(e));
  int major = 0;
  e = cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev);
  if (e != cudaSuccess) return cuda_fail(e, "cudaDeviceGetAttribute");
  if (major != 10) return fail(SAKI_ERR_UNSUPPORTED, "device compute capability %d.x: this library is built for sm_100a only", major);
  e = cudaGetSymbolAddress((void**)flagged, g_flagged_rows);
  if (e != cudaSuccess) return cuda_fail(e, "cudaGetSymbolAddress");
  return SAKI_OK;
}

// Scratch of the two-tier routing: the float32 kernels append the rows they cannot resolve to a list
// that the float64 kernel then routes.  One buffer per (device, stream), so that calls on different
// streams do not share a list; grown on demand, kept until exit.  (Calls on one stream are ordered by the
// stream, so they may share.)  A caller holds g_redo_mu from the hand-out until its kernels are launched,
// and nothing is freed while work that may use it is in flight: a buffer that was outgrown is retired,
// not freed, and the sweep that follows many short-lived streams first waits for the device.  Every
// free bumps g_redo_generation, which the counter readers check before they follow g_last_redo_count.
struct RedoBuf {
  int32_t* list = nullptr;       // [cap] rows, followed by the counter
  int64_t cap = 0;
};
static std::mutex g_redo_mu;
static std::map<std::pair<int, cudaStream_t>, RedoBuf> g_redo;
static std::vector<std::pair<int, int32_t*>> g_retired;          // (device, buffer) outgrown, still possibly in use
static std::atomic<uint64_t> g_redo_generation{0};
static thread_local unsigned int* g_last_redo_count = nullptr;
static thread_local uint64_t g_last_redo_generation = 0;

// g_redo_mu held by the caller
static int redo_scratch(int64_t n_rows, cudaStream_t st, int32_t** list, unsigned int** count) {
  int dev = 0;
  cudaGetDevice(&dev);
  if (g_redo.size() > 256) {   // many short-lived streams: start over, once nothing on the device can still use a list
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return cuda_fail(e, "cudaDeviceSynchronize (scratch sweep)");
    for (auto& kv : g_redo)
      if (kv.first.first == dev && kv.second.list) { cudaFree(kv.second.list); kv.second = RedoBuf(); }
    for (auto it = g_redo.begin(); it != g_redo.end();) it = it->second.list ? std::next(it) : g_redo.erase(it);
    for (auto& r : g_retired)
      if (r.first == dev && r.second) { cudaFree(r.second); r.second = nullptr; }
    g_retired.erase(std::remove_if(g_retired.begin(), g_retired.end(), [](const std::pair<int, int32_t*>& r) { return !r.second; }),
                    g_retired.end());
    g_redo_generation.fetch_add(1);
  }
  RedoBuf& b = g_redo[std::make_pair(dev, st)];
  if (b.cap < n_rows) {
    if (b.list) g_retired.emplace_back(dev, b.list);   // an earlier call on this stream may still be running on it
    b = RedoBuf();
    const int64_t cap = std::max<int64_t>(n_rows, 1 << 16);
    // row ids, 64 words of counters, and as many words again (block verification: one per sequence)
    cudaError_t e = cudaMalloc((void**)&b.list, (size_t)(2 * cap + 64) * sizeof(int32_t));
    if (e != cudaSuccess) { b = RedoBuf(); return cuda_fail(e, "cudaMalloc (redo list)"); }
    b.cap = cap;
  }
  *list = b.list;
  *count = (unsigned int*)(b.list + b.cap);
  return SAKI_OK;
}
// the calling thread's last routing call's counters, or NULL if there are none (any more)
static unsigned int* last_counters() {
  return g_last_redo_generation == g_redo_generation.load() ? g_last_redo_count : nullptr;
}

// Fixed scratch of saki_route_fwd_bwd_noalloc: the redo list of the two-tier routing for callers that must
// not allocate.  SAKI_NOALLOC_MAX_ROWS row ids plus the counter; every device that loads the library holds
// these 4 MB until the process exits.
#define SAKI_NOALLOC_MAX_ROWS (1 << 20)
static __device__ __align__(256) int32_t g_noalloc_scratch[SAKI_NOALLOC_MAX_ROWS + 64];
static std::mutex g_noalloc_mu;
static int32_t* g_noalloc_ptr[64] = {nullptr};   // device address of the array, per device ordinal

// In host code the array's name is only a handle; the kernels need its device address, looked up once per
// device with that device current.
static int noalloc_scratch(int32_t** list, unsigned int** count) {
  int dev = -1;
  cudaError_t e = cudaGetDevice(&dev);
  if (e != cudaSuccess) return cuda_fail(e, "cudaGetDevice");
  if (dev < 0 || dev >= 64) return fail(SAKI_ERR_UNSUPPORTED, "device ordinal %d outside the table", dev);
  std::lock_guard<std::mutex> lock(g_noalloc_mu);
  if (!g_noalloc_ptr[dev]) {
    int32_t* ptr = nullptr;
    e = cudaGetSymbolAddress((void**)&ptr, g_noalloc_scratch);
    if (e != cudaSuccess) return cuda_fail(e, "cudaGetSymbolAddress (fixed scratch)");
    g_noalloc_ptr[dev] = ptr;
  }
  *list = g_noalloc_ptr[dev];
  *count = (unsigned int*)(g_noalloc_ptr[dev] + SAKI_NOALLOC_MAX_ROWS);
  return SAKI_OK;
}

static int check_common(const void* s, const void* t, int64_t n, int32_t V, int32_t dtype, float eps, float tau) {
  if (n < 0) return fail(SAKI_ERR_INVALID_ARG, "negative row count");
  if (V < 2) return fail(SAKI_ERR_INVALID_ARG, "V must be >= 2 (got %d)", V);
  if (dtype != SAKI_F32 && dtype != SAKI_BF16) return fail(SAKI_ERR_INVALID_ARG, "unknown dtype %d", dtype);
  if (!(eps >= 0.f)) return fail(SAKI_ERR_INVALID_ARG, "eps must be >= 0 and not NaN");
  if (!(tau > 0.f) || std::isinf(tau)) return fail(SAKI_ERR_INVALID_ARG, "temperature must be finite and > 0");
  if (n > 0 && (!s || !t)) return fail(SAKI_ERR_INVALID_ARG, "NULL logits pointer");
  return SAKI_OK;
}

// `scratch_list` / `scratch_count`: where the two-tier routing keeps its redo list (NULL: the library's
// own per-device buffer, allocated on demand).
static int dispatch_rows(RowParams p, int dtype, cudaStream_t st, int32_t* scratch_list = nullptr,
                         unsigned int* scratch_count = nullptr) {
  int launches = 0;
  cudaError_t e;
  bool served = false;
  const int which = g_kernel.load();
  int used = 1;
  // Directly, float32 sums resolve KL(q||p) to a few 1e-7 absolute: enough for |d lambda| <= 1e-5 when
  // eps >= 5e-3 (measured), not below: for the cluster kernel smaller positive radii run on the float64
  // kernel.  The row-per-SM kernel gets KL for small radii from a quadrature of its slope instead
  // (relative, not absolute, accuracy) and takes every radius.
  const bool eps_ok = !(p.eps > 0.f) || p.eps >= 5e-3f;
  const bool rowsm_ok = (which == 0 || which == 3) && rowsm_can_serve(p, dtype);
  const bool fast = (which != 1) && (rowsm_ok || (eps_ok && cluster_can_serve(p, dtype)));
  p.redo_list = nullptr; p.redo_count = nullptr; p.redo_guess = nullptr; p.from_list = 0;
  p.wait_limit = g_wait_limit.load();
  g_last_redo_count = nullptr;          // the counters below describe this call only
  std::unique_lock<std::mutex> scratch_lock(g_redo_mu, std::defer_lock);
  if (fast) {
    if (scratch_list) { p.redo_list = scratch_list; p.redo_count = scratch_count; }
    else {
      scratch_lock.lock();       // until the kernels that use the list are launched
      const int rc = redo_scratch(p.n_rows, st, &p.redo_list, &p.redo_count);
      if (rc) return rc;
      // the words behind the counters (one per row; block verification keeps its sequences' stops there) take
      // what the float32 kernel made of lambda for the rows it hands over
      if (!p.spec) p.redo_guess = (float*)(p.redo_count + 64);
    }
    // the counter, the three statistics words after it, and the phase clock's sums
    e = cudaMemsetAsync(p.redo_count, 0, (8 + 2 * SAKI_PHASE_COUNTERS) * sizeof(unsigned int), st);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMemsetAsync");
    p.phase_cycles = g_phase_clock.load() ? (unsigned long long*)(p.redo_count + 8) : nullptr;
    g_last_redo_count = p.redo_count;
    g_last_redo_generation = g_redo_generation.load();
  }
  // A handful of long rows (a decoding step of a small batch) finish sooner spread over the whole GPU, one
  // row per cluster of 8 blocks, than on one SM each: 32 clusters fit at once, and at V = 151936 a call of
  // up to 32 rows takes 32 to 40 us there against 62 us (V = 65536: 28 to 34 against 33 to 39; at V = 32000
  // the row-per-SM kernel is the faster one at every size).
  if (fast && which == 0 && p.n_rows <= 32 && p.V >= 65536 && eps_ok && cluster_can_serve(p, dtype)) {
    e = launch_cluster(p, st, &launches, &served);
    if (e != cudaSuccess) return cuda_fail(e, "cluster kernel launch");
    if (served) used = 2;
  }
  if (fast && !served && (which == 0 || which == 3) && rowsm_can_serve(p, dtype)) {
    // Block verification with early out: positions handed out as tickets, sequences record their first stop.
    // Only with two or more sequences per SM: with fewer, most positions are handed out before their
    // predecessor's decision is known, and the bookkeeping costs more than the few skipped rows save.
    int sms = 0, dev_now = 0;
    if (p.spec && (cudaGetDevice(&dev_now) != cudaSuccess ||
                   cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev_now) != cudaSuccess)) sms = 0;
    if (p.spec && g_spec_early_out.load() && !scratch_list && sms > 0 && p.n_rows / p.K1 >= 2 * (int64_t)sms) {
      p.seq_next = p.redo_count + 1;
      p.seq_stop = (int*)(p.redo_count + 64);
      e = cudaMemsetAsync(p.seq_stop, 0x7f, (size_t)(p.n_rows / p.K1) * sizeof(int), st);   // "no stop yet": above any position
      if (e != cudaSuccess) return cuda_fail(e, "cudaMemsetAsync");
    }
    e = launch_rowsm(p, st, &launches, &served);
    p.seq_next = nullptr; p.seq_stop = nullptr;
    if (e != cudaSuccess) return cuda_fail(e, "row-per-SM kernel launch");
    if (served) used = 3;
  }
  if (fast && !served && which == 2 && cluster_can_serve(p, dtype)) {
    e = launch_cluster(p, st, &launches, &served);
    if (e != cudaSuccess) return cuda_fail(e, "cluster kernel launch");
    if (served) used = 2;
  }
  if (served) {   // second tier: the rows the float32 kernel handed over
    p.from_list = 1;
    e = launch_general(p, dtype, st, &launches);
    if (e != cudaSuccess) return cuda_fail(e, "general kernel launch (redo list)");
  } else {
    e = launch_general(p, dtype, st, &launches);
    if (e != cudaSuccess) return cuda_fail(e, "general kernel launch");
  }
  g_launches += (uint64_t)launches;
  g_last_kernel = used;
  return SAKI_OK;
}

static int route_impl(const saki_in* in, const saki_out* out, void* dlogits, int64_t ld_g, float grad_scale,
                      bool bwd, void* stream, bool fixed_scratch = false) {
  g_err[0] = 0;
  if (!in || !out) return fail(SAKI_ERR_INVALID_ARG, "NULL argument struct");
  if (fixed_scratch && in->N > SAKI_NOALLOC_MAX_ROWS)
    return fail(SAKI_ERR_INVALID_ARG, "N = %lld exceeds the fixed scratch of this entry point (%d rows): split the batch",
                (long long)in->N, SAKI_NOALLOC_MAX_ROWS);
  int rc = check_common(in->student_logits, in->teacher_logits, in->N, in->V, in->dtype, in->eps, in->temperature);
  if (rc) return rc;
  if (in->ld_s < in->V || in->ld_t < in->V) return fail(SAKI_ERR_INVALID_ARG, "row stride smaller than V");
  if (in->N > 0 && !in->proposal) return fail(SAKI_ERR_INVALID_ARG, "NULL proposal pointer");
  if (in->N > 0 && (!out->corrected || !out->token)) return fail(SAKI_ERR_INVALID_ARG, "out.corrected and out.token are required");
  if (bwd) {
    if (in->N > 0 && !dlogits) return fail(SAKI_ERR_INVALID_ARG, "NULL dlogits pointer");
    if (ld_g < in->V) return fail(SAKI_ERR_INVALID_ARG, "gradient row stride smaller than V");
    if (!std::isfinite(grad_scale)) return fail(SAKI_ERR_INVALID_ARG, "grad_scale must be finite");
  }
  if (in->N == 0) return SAKI_OK;
  unsigned long long* flagged = nullptr;
  rc = device_ready(&flagged);
  if (rc) return rc;
  RowParams p;
  memset(&p, 0, sizeof(p));
  p.s = in->student_logits; p.t = in->teacher_logits;
  p.s_seq = in->ld_s; p.s_pos = 0; p.t_seq = in->ld_t; p.t_pos = 0;
  p.n_rows = in->N; p.V = in->V; p.K1 = 1; p.spec = 0;
  p.proposal = in->proposal; p.prop_ld = 0; p.mask = in->mask;
  p.eps = in->eps; p.temperature = in->temperature; p.seed = in->seed; p.row_offset = in->row_offset;
  p.out = *out;
  p.dlogits = bwd ? dlogits : nullptr; p.ld_g = ld_g; p.grad_scale = grad_scale;
  p.flagged = flagged;
  if (fixed_scratch) {
    int32_t* list = nullptr;
    unsigned int* count = nullptr;
    rc = noalloc_scratch(&list, &count);
    if (rc) return rc;
    return dispatch_rows(p, in->dtype, (cudaStream_t)stream, list, count);
  }
  return dispatch_rows(p, in->dtype, (cudaStream_t)stream);
}

// ---- the trainer's step: loss and gradient from the rollout's metadata (Section 3.5) ----
static int meta_impl(const saki_meta_in* in, const saki_meta_out* out, void* dlogits, int64_t ld_g, float grad_scale,
                     void* stream) {
  g_err[0] = 0;
  if (!in || !out) return fail(SAKI_ERR_INVALID_ARG, "NULL argument struct");
  if (in->N < 0) return fail(SAKI_ERR_INVALID_ARG, "negative row count");
  if (in->V < 2) return fail(SAKI_ERR_INVALID_ARG, "V must be >= 2 (got %d)", in->V);
  if (in->dtype != SAKI_F32 && in->dtype != SAKI_BF16) return fail(SAKI_ERR_INVALID_ARG, "unknown dtype %d", in->dtype);
  if (!(in->temperature > 0.f) || std::isinf(in->temperature))
    return fail(SAKI_ERR_INVALID_ARG, "temperature must be finite and > 0");
  if (in->ld_s < in->V || ld_g < in->V) return fail(SAKI_ERR_INVALID_ARG, "row stride smaller than V");
  if (!std::isfinite(grad_scale)) return fail(SAKI_ERR_INVALID_ARG, "grad_scale must be finite");
  if (in->N == 0) return SAKI_OK;
  if (!in->student_logits || !dlogits) return fail(SAKI_ERR_INVALID_ARG, "NULL logits or dlogits pointer");
  if (!in->corrected || !in->proposal || !in->teacher_top1 || !in->advantage)
    return fail(SAKI_ERR_INVALID_ARG, "corrected, proposal, teacher_top1 and advantage are required");
  unsigned long long* flagged = nullptr;
  int rc = device_ready(&flagged);
  if (rc) return rc;
  MetaParams p;
  memset(&p, 0, sizeof(p));
  p.s = in->student_logits; p.ld_s = in->ld_s; p.n_rows = in->N; p.V = in->V;
  p.corrected = in->corrected; p.proposal = in->proposal; p.teacher_top1 = in->teacher_top1;
  p.advantage = in->advantage; p.mask = in->mask; p.rollout_status = in->rollout_status;
  p.temperature = in->temperature; p.out = *out; p.dlogits = dlogits; p.ld_g = ld_g; p.grad_scale = grad_scale;
  p.flagged = flagged;
  cudaStream_t st = (cudaStream_t)stream;
  int launches = 0;
  cudaError_t e;
  bool served = false;
  int used = 1;
  g_last_redo_count = nullptr;
  std::unique_lock<std::mutex> scratch_lock(g_redo_mu, std::defer_lock);
  if (g_kernel.load() != 1 && meta_stream_can_serve(p, in->dtype)) {
    scratch_lock.lock();         // until the kernels that use the list are launched
    rc = redo_scratch(p.n_rows, st, &p.redo_list, &p.redo_count);
    if (rc) return rc;
    e = cudaMemsetAsync(p.redo_count, 0, (8 + 2 * SAKI_PHASE_COUNTERS) * sizeof(unsigned int), st);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMemsetAsync");
    g_last_redo_count = p.redo_count;
    g_last_redo_generation = g_redo_generation.load();
    e = launch_meta_stream(p, st, &launches, &served);
    if (e != cudaSuccess) return cuda_fail(e, "streaming backward kernel launch");
    if (served) { used = 4; p.from_list = 1; }
  }
  e = launch_meta_general(p, in->dtype, st, &launches);
  if (e != cudaSuccess) return cuda_fail(e, "general backward kernel launch");
  g_launches += (uint64_t)launches;
  g_last_kernel = used;
  return SAKI_OK;
}

// ---- block verification: per-sequence first-rejection resolve (Section 3.5) ----
__global__ void spec_resolve_kernel(int64_t B, int K, saki_out o, int32_t* n_accept, int32_t* next_token,
                                    uint8_t* next_is_corr) {
  const int64_t b = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (b >= B) return;
  const int K1 = K + 1;
  int n = K, stopped = 0, next = -1, isc = 0;
  for (int j = 0; j < K; ++j) {
    const int64_t r = b * K1 + j;
    if (o.token[r] < 0) { n = j; stopped = 1; break; }            // flagged row: cannot verify further
    if (o.corrected[r]) { n = j; stopped = 1; next = o.token[r]; isc = 1; break; }
  }
  if (!stopped) next = o.token[b * K1 + K];                        // bonus draw (or -1 if flagged)
  n_accept[b] = n; next_token[b] = next; next_is_corr[b] = (uint8_t)isc;
  if (stopped) {                                                   // later positions sit on an invalid prefix
    const RowResult z = zero_row(SAKI_ROW_NOT_COMPUTED);
    for (int j = n + 1; j < K1; ++j) write_row(o, b * K1 + j, z, false);
  }
}

// ---- proposal utility: Gumbel-max with per-element Philox noise ----
template <typename T>
__global__ void __launch_bounds__(256) proposal_kernel(const T* logits, int64_t ld, int64_t N, int V, double tau,
                                                        uint64_t seed, uint64_t row_offset, int32_t* out) {
  __shared__ double skey[8];
  __shared__ int sidx[8];
  for (int64_t row = blockIdx.x; row < N; row += gridDim.x) {
    const T* s = logits + row * ld;
    const uint64_t rid = row_offset + (uint64_t)row;
    double best = -INFINITY;
    int bi = 0x7fffffff;
    for (int blk = threadIdx.x; blk * 4 < V; blk += blockDim.x) {
      uint32_t w[4];
      philox4x32_10((uint32_t)rid, (uint32_t)(rid >> 32), STAGE_PROPOSE, (uint32_t)blk, (uint32_t)seed,
                    (uint32_t)(seed >> 32), w);
#pragma unroll
      for (int k = 0; k < 4; ++k) {
        const int v = blk * 4 + k;
        if (v < V) {
          const double u = ((double)w[k] + 0.5) * (1.0 / 4294967296.0);
          const double key = (double)ld_as_float(s, v) / tau - log(-log(u));
          if (key > best) { best = key; bi = v; }
        }
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const double ob = __shfl_xor_sync(0xffffffffu, best, o);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      if (ob > best || (ob == best && oi < bi)) { best = ob; bi = oi; }
    }
    if ((threadIdx.x & 31) == 0) { skey[threadIdx.x >> 5] = best; sidx[threadIdx.x >> 5] = bi; }
    __syncthreads();
    if (threadIdx.x == 0) {
      for (int w = 1; w < 8; ++w)
        if (skey[w] > best || (skey[w] == best && sidx[w] < bi)) { best = skey[w]; bi = sidx[w]; }
      out[row] = bi;
    }
    __syncthreads();
  }
}

// ---- host-buffer entry: staged, double-buffered ----
struct HostStage {
  std::mutex mu;
  int dev = -1;
  cudaStream_t st[2] = {nullptr, nullptr};
  void* buf[2] = {nullptr, nullptr};
  size_t cap[2] = {0, 0};
};
static HostStage g_stage;

static size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

}  // namespace saki

using namespace saki;

extern "C" {

SAKI_API int saki_route_fwd(const saki_in* in, const saki_out* out, void* cuda_stream) {
  return route_impl(in, out, nullptr, 0, 0.f, false, cuda_stream);
}

SAKI_API int saki_route_fwd_bwd(const saki_in* in, const saki_out* out, void* dlogits, int64_t ld_g, float grad_scale,
                       void* cuda_stream) {
  return route_impl(in, out, dlogits, ld_g, grad_scale, true, cuda_stream);
}

SAKI_API int saki_route_fwd_bwd_noalloc(const saki_in* in, const saki_out* out, void* dlogits, int64_t ld_g,
                                        float grad_scale, void* cuda_stream) {
  return route_impl(in, out, dlogits, ld_g, grad_scale, true, cuda_stream, true);
}

SAKI_API int saki_route_bwd_from_meta(const saki_meta_in* in, const saki_meta_out* out, void* dlogits, int64_t ld_g,
                                      float grad_scale, void* cuda_stream) {
  return meta_impl(in, out, dlogits, ld_g, grad_scale, cuda_stream);
}

SAKI_API int saki_select_tm(const saki_select_in* in, uint8_t* selected, int32_t* m, void* cuda_stream) {
  g_err[0] = 0;
  if (!in) return fail(SAKI_ERR_INVALID_ARG, "NULL argument struct");
  if (in->N < 0 || in->B < 0) return fail(SAKI_ERR_INVALID_ARG, "negative size");
  if (in->mode != SAKI_SELECT_RANDOM && in->mode != SAKI_SELECT_TV_WEIGHTED)
    return fail(SAKI_ERR_INVALID_ARG, "unknown selection mode %d", in->mode);
  if (in->B == 0 || in->N == 0) return SAKI_OK;
  if (!in->seq_start || !in->corrected || !selected) return fail(SAKI_ERR_INVALID_ARG, "seq_start, corrected and selected are required");
  if (in->mode == SAKI_SELECT_TV_WEIGHTED && !in->tv) return fail(SAKI_ERR_INVALID_ARG, "tv is required in TV-weighted mode");
  unsigned long long* flagged = nullptr;
  int rc = device_ready(&flagged);
  if (rc) return rc;
  SelectParams p;
  memset(&p, 0, sizeof(p));
  p.N = in->N; p.B = in->B; p.seq_start = in->seq_start; p.corrected = in->corrected; p.tv = in->tv;
  p.mask = in->mask; p.rollout_status = in->rollout_status; p.mode = in->mode; p.seed = in->seed;
  p.row_offset = in->row_offset; p.selected = selected; p.m = m;
  int launches = 0;
  cudaError_t e = launch_select(p, (cudaStream_t)cuda_stream, &launches);
  if (e != cudaSuccess) return cuda_fail(e, "selection kernel launch");
  g_launches += (uint64_t)launches;
  return SAKI_OK;
}

static int vshard_check(const saki_vshard_in* in, int stage) {
  if (!in) return fail(SAKI_ERR_INVALID_ARG, "NULL argument struct");
  if (stage < 0 || stage > 3) return fail(SAKI_ERR_INVALID_ARG, "stage must be 0..3 (got %d)", stage);
  if (in->N < 0) return fail(SAKI_ERR_INVALID_ARG, "negative row count");
  if (in->V < 2) return fail(SAKI_ERR_INVALID_ARG, "V must be >= 2 (got %d)", in->V);
  if (in->world < 1 || in->rank < 0 || in->rank >= in->world) return fail(SAKI_ERR_INVALID_ARG, "rank %d outside [0, %d)", in->rank, in->world);
  if (in->V_local < 0 || in->v0 < 0 || (int64_t)in->v0 + in->V_local > in->V)
    return fail(SAKI_ERR_INVALID_ARG, "slice [%d, %d) outside [0, %d)", in->v0, in->v0 + in->V_local, in->V);
  if (in->dtype != SAKI_F32 && in->dtype != SAKI_BF16) return fail(SAKI_ERR_INVALID_ARG, "unknown dtype %d", in->dtype);
  if (!(in->eps >= 0.f)) return fail(SAKI_ERR_INVALID_ARG, "eps must be >= 0 and not NaN");
  if (!(in->temperature > 0.f) || std::isinf(in->temperature)) return fail(SAKI_ERR_INVALID_ARG, "temperature must be finite and > 0");
  if (in->N > 0 && !in->proposal) return fail(SAKI_ERR_INVALID_ARG, "NULL proposal pointer");
  return SAKI_OK;
}

SAKI_API int saki_vshard_partial(const saki_vshard_in* in, int stage, const double* state, double* partial,
                                 void* dlogits_slice, int64_t ld_g, float grad_scale, void* cuda_stream) {
  g_err[0] = 0;
  int rc = vshard_check(in, stage);
  if (rc) return rc;
  if (in->N == 0) return SAKI_OK;
  if (in->V_local > 0 && (!in->student_logits || !in->teacher_logits)) return fail(SAKI_ERR_INVALID_ARG, "NULL logits pointer");
  if (in->ld_s < in->V_local || in->ld_t < in->V_local) return fail(SAKI_ERR_INVALID_ARG, "row stride smaller than the slice");
  if (!partial || (stage > 0 && !state)) return fail(SAKI_ERR_INVALID_ARG, "NULL partial or state pointer");
  if (dlogits_slice && (ld_g < in->V_local || !std::isfinite(grad_scale))) return fail(SAKI_ERR_INVALID_ARG, "bad gradient stride or scale");
  unsigned long long* flagged = nullptr;
  rc = device_ready(&flagged);
  if (rc) return rc;
  cudaError_t e = launch_vshard_partial(*in, stage, state, partial, stage == 3 ? dlogits_slice : nullptr, ld_g, grad_scale,
                                        g_kernel.load() != 1, (cudaStream_t)cuda_stream);
  if (e != cudaSuccess) return cuda_fail(e, "vocabulary-sharded partial kernel launch");
  g_launches += 1;
  return SAKI_OK;
}

SAKI_API int saki_vshard_combine(const saki_vshard_in* in, int stage, const double* gathered, double* state,
                                 const saki_out* out, uint32_t* n_solving, void* cuda_stream) {
  g_err[0] = 0;
  int rc = vshard_check(in, stage);
  if (rc) return rc;
  if (in->N == 0) return SAKI_OK;
  if (!gathered || !state) return fail(SAKI_ERR_INVALID_ARG, "NULL gathered or state pointer");
  if (stage == 3 && (!out || !out->corrected || !out->token)) return fail(SAKI_ERR_INVALID_ARG, "out.corrected and out.token are required at stage 3");
  unsigned long long* flagged = nullptr;
  rc = device_ready(&flagged);
  if (rc) return rc;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (n_solving) {
    cudaError_t e0 = cudaMemsetAsync(n_solving, 0, sizeof(uint32_t), st);
    if (e0 != cudaSuccess) return cuda_fail(e0, "cudaMemsetAsync");
  }
  saki_out none;
  memset(&none, 0, sizeof(none));
  cudaError_t e = launch_vshard_combine(*in, stage, gathered, state, out ? *out : none, n_solving, g_kernel.load() != 1, st);
  if (e != cudaSuccess) return cuda_fail(e, "vocabulary-sharded combine kernel launch");
  g_launches += 1;
  return SAKI_OK;
}

SAKI_API int saki_vshard_combine_host(const saki_vshard_in* in, int stage, const double* gathered, double* state,
                                      const saki_out* out, int32_t* n_solving) {
  g_err[0] = 0;
  int rc = vshard_check(in, stage);
  if (rc) return rc;
  if (n_solving) *n_solving = 0;
  if (in->N == 0) return SAKI_OK;
  if (!gathered || !state) return fail(SAKI_ERR_INVALID_ARG, "NULL gathered or state pointer");
  if (stage == 3 && (!out || !out->corrected || !out->token)) return fail(SAKI_ERR_INVALID_ARG, "out.corrected and out.token are required at stage 3");
  saki_out none;
  memset(&none, 0, sizeof(none));
  const int solving = vshard_combine_host(*in, stage, gathered, state, out ? *out : none, g_kernel.load() != 1);
  if (n_solving) *n_solving = solving;
  return SAKI_OK;
}

SAKI_API int64_t saki_lmhead_scratch_bytes(int64_t N, int32_t V) {
  if (N < 0 || V < 1) return 0;
  return lmhead_scratch_bytes(N, V);
}

SAKI_API int saki_lmhead_lse(const saki_lmhead_in* in, void* logits, int64_t ld_l, float* row_max, float* lse,
                             void* scratch, int64_t scratch_bytes, void* cuda_stream) {
  g_err[0] = 0;
  if (!in) return fail(SAKI_ERR_INVALID_ARG, "NULL argument struct");
  if (in->N < 0) return fail(SAKI_ERR_INVALID_ARG, "negative row count");
  if (in->V < 8 || in->d < 8) return fail(SAKI_ERR_INVALID_ARG, "V and d must be >= 8 (got %d, %d)", in->V, in->d);
  if (!(in->temperature > 0.f) || std::isinf(in->temperature)) return fail(SAKI_ERR_INVALID_ARG, "temperature must be finite and > 0");
  if (in->ld_h < in->d || in->ld_w < in->d || ld_l < in->V) return fail(SAKI_ERR_INVALID_ARG, "row stride smaller than the row");
  if (in->N == 0) return SAKI_OK;
  if (!in->hidden || !in->weight || !logits || !scratch) return fail(SAKI_ERR_INVALID_ARG, "NULL hidden, weight, logits or scratch pointer");
  if (scratch_bytes < lmhead_scratch_bytes(in->N, in->V)) return fail(SAKI_ERR_INVALID_ARG, "scratch too small: %lld bytes needed", (long long)lmhead_scratch_bytes(in->N, in->V));
  auto al = [](const void* q, uintptr_t a) { return ((uintptr_t)q & (a - 1)) == 0; };
  if (!al(in->hidden, 16) || !al(in->weight, 16) || !al(logits, 16) || !al(scratch, 256) || in->ld_h % 8 || in->ld_w % 8 || ld_l % 8 || in->V % 8)
    return fail(SAKI_ERR_UNSUPPORTED, "pointers must be 16-byte aligned (scratch 256), strides and V multiples of 8");
  unsigned long long* flagged = nullptr;
  int rc = device_ready(&flagged);
  if (rc) return rc;
  const char* why = nullptr;
  cudaError_t e = launch_lmhead(*in, logits, ld_l, row_max, lse, scratch, (cudaStream_t)cuda_stream, &why);
  if (e != cudaSuccess) return why ? fail(SAKI_ERR_CUDA, "%s", why) : cuda_fail(e, "lm-head kernel launch");
  g_launches += 2;
  return SAKI_OK;
}

SAKI_API int saki_spec_verify(const saki_spec_in* in, const saki_spec_out* out, void* cuda_stream) {
  g_err[0] = 0;
  if (!in || !out) return fail(SAKI_ERR_INVALID_ARG, "NULL argument struct");
  int rc = check_common(in->student_logits, in->teacher_logits, in->B, in->V, in->dtype, in->eps, in->temperature);
  if (rc) return rc;
  if (in->K < 1 || in->K > 16) return fail(SAKI_ERR_INVALID_ARG, "K must be in [1,16] (got %d)", in->K);
  if (in->ss_pos < in->V || in->ts_pos < in->V) return fail(SAKI_ERR_INVALID_ARG, "position stride smaller than V");
  if (in->ss_seq < in->ss_pos || in->ts_seq < in->ts_pos) return fail(SAKI_ERR_INVALID_ARG, "sequence stride smaller than position stride");
  if (in->B > 0 && (!in->draft || in->draft_ld < in->K)) return fail(SAKI_ERR_INVALID_ARG, "bad draft pointer or stride");
  if (in->B > 0 && (!out->n_accept || !out->next_token || !out->next_is_correction || !out->per_pos.corrected ||
                    !out->per_pos.token))
    return fail(SAKI_ERR_INVALID_ARG, "n_accept, next_token, next_is_correction, per_pos.corrected and per_pos.token are required");
  if (in->B == 0) return SAKI_OK;
  unsigned long long* flagged = nullptr;
  rc = device_ready(&flagged);
  if (rc) return rc;
  RowParams p;
  memset(&p, 0, sizeof(p));
  p.s = in->student_logits; p.t = in->teacher_logits;
  p.s_seq = in->ss_seq; p.s_pos = in->ss_pos; p.t_seq = in->ts_seq; p.t_pos = in->ts_pos;
  p.K1 = in->K + 1; p.n_rows = in->B * p.K1; p.V = in->V; p.spec = 1;
  p.proposal = in->draft; p.prop_ld = in->draft_ld; p.mask = nullptr;
  p.eps = in->eps; p.temperature = in->temperature; p.seed = in->seed;
  p.row_offset = in->seq_offset * (uint64_t)p.K1;
  p.out = out->per_pos;
  p.out.loss = nullptr;
  p.dlogits = nullptr; p.ld_g = 0; p.grad_scale = 0.f; p.flagged = flagged;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  rc = dispatch_rows(p, in->dtype, st);
  if (rc) return rc;
  const int th = 128;
  spec_resolve_kernel<<<(unsigned)((in->B + th - 1) / th), th, 0, st>>>(in->B, in->K, p.out, out->n_accept,
                                                                        out->next_token, out->next_is_correction);
  g_launches += 1;
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e, "resolve kernel launch");
  return SAKI_OK;
}

SAKI_API int saki_sample_proposal(const void* logits, int64_t ld, int64_t N, int32_t V, int32_t dtype, float temperature,
                         uint64_t seed, uint64_t row_offset, int32_t* out, void* cuda_stream) {
  g_err[0] = 0;
  int rc = check_common(logits, logits, N, V, dtype, 0.f, temperature);
  if (rc) return rc;
  if (ld < V) return fail(SAKI_ERR_INVALID_ARG, "row stride smaller than V");
  if (N > 0 && !out) return fail(SAKI_ERR_INVALID_ARG, "NULL output pointer");
  if (N == 0) return SAKI_OK;
  unsigned long long* flagged = nullptr;
  rc = device_ready(&flagged);
  if (rc) return rc;
  const int grid = (int)std::min<int64_t>(N, 148 * 8);
  cudaStream_t st = (cudaStream_t)cuda_stream;
  if (dtype == SAKI_BF16)
    proposal_kernel<__nv_bfloat16><<<grid, 256, 0, st>>>((const __nv_bfloat16*)logits, ld, N, V, (double)temperature,
                                                         seed, row_offset, out);
  else
    proposal_kernel<float><<<grid, 256, 0, st>>>((const float*)logits, ld, N, V, (double)temperature, seed,
                                                 row_offset, out);
  g_launches += 1;
  cudaError_t e = cudaGetLastError();
  if (e != cudaSuccess) return cuda_fail(e, "proposal kernel launch");
  return SAKI_OK;
}

SAKI_API int saki_check(void* cuda_stream, uint64_t* n_flagged) {
  g_err[0] = 0;
  unsigned long long* flagged = nullptr;
  int rc = device_ready(&flagged);
  if (rc) return rc;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  cudaError_t e = cudaStreamSynchronize(st);
  if (e != cudaSuccess) return cuda_fail(e, "cudaStreamSynchronize");
  unsigned long long h = 0, zero = 0;
  e = cudaMemcpy(&h, flagged, sizeof(h), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return cuda_fail(e, "cudaMemcpy");
  e = cudaMemcpy(flagged, &zero, sizeof(zero), cudaMemcpyHostToDevice);
  if (e != cudaSuccess) return cuda_fail(e, "cudaMemcpy");
  if (n_flagged) *n_flagged = h;
  if (h) return fail(SAKI_ERR_ROW_STATUS, "%llu row(s) flagged (non-finite logits, bad proposal id or timeout)", h);
  return SAKI_OK;
}

SAKI_API int saki_route_host(const saki_in* in, const saki_out* out, void* dlogits, int64_t ld_g, float grad_scale) {
  g_err[0] = 0;
  if (!in || !out) return fail(SAKI_ERR_INVALID_ARG, "NULL argument struct");
  int rc = check_common(in->student_logits, in->teacher_logits, in->N, in->V, in->dtype, in->eps, in->temperature);
  if (rc) return rc;
  if (in->ld_s < in->V || in->ld_t < in->V) return fail(SAKI_ERR_INVALID_ARG, "row stride smaller than V");
  if (dlogits && ld_g < in->V) return fail(SAKI_ERR_INVALID_ARG, "gradient row stride smaller than V");
  if (in->N > 0 && (!in->proposal || !out->corrected || !out->token))
    return fail(SAKI_ERR_INVALID_ARG, "proposal, out.corrected and out.token are required");
  if (in->N == 0) return SAKI_OK;
  unsigned long long* flagged = nullptr;
  rc = device_ready(&flagged);
  if (rc) return rc;

  std::lock_guard<std::mutex> lock(g_stage.mu);
  int dev = 0;
  cudaGetDevice(&dev);
  cudaError_t e;
  if (g_stage.dev != dev) {   // (re)create the staging streams on this device
    for (int k = 0; k < 2; ++k) {
      if (g_stage.buf[k]) { cudaFree(g_stage.buf[k]); g_stage.buf[k] = nullptr; g_stage.cap[k] = 0; }
      if (g_stage.st[k]) { cudaStreamDestroy(g_stage.st[k]); g_stage.st[k] = nullptr; }
      e = cudaStreamCreateWithFlags(&g_stage.st[k], cudaStreamNonBlocking);
      if (e != cudaSuccess) return cuda_fail(e, "cudaStreamCreate");
    }
    g_stage.dev = dev;
  }
  const size_t es = in->dtype == SAKI_BF16 ? 2 : 4;
  const size_t Vp = align_up((size_t)in->V, 16);   // padded device row stride: rows stay 16-byte aligned
  // rows per chunk: about 192 MB of logits per buffer
  int64_t chunk = (int64_t)std::max<size_t>(1, (size_t)192 << 20) / (int64_t)(2 * Vp * es);
  chunk = std::max<int64_t>(1, std::min<int64_t>(chunk, in->N));
  const size_t row_bytes = Vp * es;
  // device layout of one chunk
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
  const size_t o_s = take(chunk * row_bytes), o_t = take(chunk * row_bytes);
  const size_t o_g = dlogits ? take(chunk * row_bytes) : 0;
  const size_t o_prop = take(chunk * 4), o_mask = take(chunk);
  const size_t o_corr = take(chunk), o_tok = take(chunk * 4), o_top = take(chunk * 4), o_stat = take(chunk * 4);
  size_t o_f[11];
  for (int k = 0; k < 11; ++k) o_f[k] = take(chunk * 4);
  const size_t total = off;
  for (int k = 0; k < 2; ++k) {
    if (g_stage.cap[k] < total) {
      if (g_stage.buf[k]) cudaFree(g_stage.buf[k]);
      g_stage.buf[k] = nullptr; g_stage.cap[k] = 0;
      e = cudaMalloc(&g_stage.buf[k], total);
      if (e != cudaSuccess) return cuda_fail(e, "cudaMalloc (staging)");
      g_stage.cap[k] = total;
    }
  }
  float* const host_f[11] = {out->lambda, out->kl, out->tv, out->accept_prob, out->logp_x,
                             out->logq_x, out->logT_x, out->logp_y, out->logq_y, out->logT_y, out->loss};
  int result = SAKI_OK;
  int k = 0;
  for (int64_t r0 = 0; r0 < in->N && result == SAKI_OK; r0 += chunk, k ^= 1) {
    const int64_t n = std::min<int64_t>(chunk, in->N - r0);
    char* base = (char*)g_stage.buf[k];
    cudaStream_t st = g_stage.st[k];
    const char* hs = (const char*)in->student_logits + (size_t)r0 * in->ld_s * es;
    const char* ht = (const char*)in->teacher_logits + (size_t)r0 * in->ld_t * es;
    e = cudaMemcpy2DAsync(base + o_s, row_bytes, hs, in->ld_s * es, in->V * es, n, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess)
      e = cudaMemcpy2DAsync(base + o_t, row_bytes, ht, in->ld_t * es, in->V * es, n, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess)
      e = cudaMemcpyAsync(base + o_prop, in->proposal + r0, n * 4, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess && in->mask) e = cudaMemcpyAsync(base + o_mask, in->mask + r0, n, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) { result = cuda_fail(e, "host-to-device copy"); break; }
    saki_in din = *in;
    din.student_logits = base + o_s; din.teacher_logits = base + o_t; din.ld_s = din.ld_t = (int64_t)Vp;
    din.N = n; din.proposal = (const int32_t*)(base + o_prop);
    din.mask = in->mask ? (const uint8_t*)(base + o_mask) : nullptr;
    din.row_offset = in->row_offset + (uint64_t)r0;
    saki_out dout;
    dout.corrected = (uint8_t*)(base + o_corr); dout.token = (int32_t*)(base + o_tok);
    dout.teacher_top1 = (int32_t*)(base + o_top); dout.row_status = (uint32_t*)(base + o_stat);
    float** df[11] = {&dout.lambda, &dout.kl, &dout.tv, &dout.accept_prob, &dout.logp_x,
                      &dout.logq_x, &dout.logT_x, &dout.logp_y, &dout.logq_y, &dout.logT_y, &dout.loss};
    for (int q = 0; q < 11; ++q) *df[q] = (float*)(base + o_f[q]);
    result = route_impl(&din, &dout, dlogits ? base + o_g : nullptr, (int64_t)Vp, grad_scale, dlogits != nullptr, st);
    if (result != SAKI_OK) break;
    e = cudaMemcpyAsync(out->corrected + r0, dout.corrected, n, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(out->token + r0, dout.token, n * 4, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess && out->teacher_top1)
      e = cudaMemcpyAsync(out->teacher_top1 + r0, dout.teacher_top1, n * 4, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess && out->row_status)
      e = cudaMemcpyAsync(out->row_status + r0, dout.row_status, n * 4, cudaMemcpyDeviceToHost, st);
    for (int q = 0; q < 11 && e == cudaSuccess; ++q)
      if (host_f[q]) e = cudaMemcpyAsync(host_f[q] + r0, *df[q], n * 4, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess && dlogits)
      e = cudaMemcpy2DAsync((char*)dlogits + (size_t)r0 * ld_g * es, ld_g * es, base + o_g, row_bytes, in->V * es, n,
                            cudaMemcpyDeviceToHost, st);
    if (e != cudaSuccess) { result = cuda_fail(e, "device-to-host copy"); break; }
    // the other buffer is reused two chunks later: its stream must have drained by then
    if (r0 + chunk < in->N) {
      e = cudaStreamSynchronize(g_stage.st[k ^ 1]);
      if (e != cudaSuccess) { result = cuda_fail(e, "cudaStreamSynchronize"); break; }
    }
  }
  for (int q = 0; q < 2; ++q) {
    e = cudaStreamSynchronize(g_stage.st[q]);
    if (e != cudaSuccess && result == SAKI_OK) result = cuda_fail(e, "cudaStreamSynchronize");
  }
  return result;
}

SAKI_API int saki_set_kernel(int which) {
  if (which < 0 || which > 3) which = 0;
  return g_kernel.exchange(which);
}

SAKI_API int saki_last_kernel(void) { return g_last_kernel; }

SAKI_API int saki_redo_count(void* cuda_stream, uint64_t* n_rows) {
  g_err[0] = 0;
  if (!n_rows) return fail(SAKI_ERR_INVALID_ARG, "NULL output pointer");
  *n_rows = 0;
  unsigned int* const counters = last_counters();
  if (!counters) return SAKI_OK;
  cudaError_t e = cudaStreamSynchronize((cudaStream_t)cuda_stream);
  if (e != cudaSuccess) return cuda_fail(e, "cudaStreamSynchronize");
  unsigned int h = 0;
  e = cudaMemcpy(&h, counters, sizeof(h), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return cuda_fail(e, "cudaMemcpy");
  *n_rows = h;
  return SAKI_OK;
}

SAKI_API int saki_solve_evaluations(void* cuda_stream, uint64_t* n_passes) {
  g_err[0] = 0;
  if (!n_passes) return fail(SAKI_ERR_INVALID_ARG, "NULL output pointer");
  *n_passes = 0;
  unsigned int* const counters = last_counters();
  if (!counters) return SAKI_OK;
  cudaError_t e = cudaStreamSynchronize((cudaStream_t)cuda_stream);
  if (e != cudaSuccess) return cuda_fail(e, "cudaStreamSynchronize");
  unsigned int h = 0;
  e = cudaMemcpy(&h, counters + 3, sizeof(h), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return cuda_fail(e, "cudaMemcpy");
  *n_passes = h;
  return SAKI_OK;
}

SAKI_API int64_t saki_set_wait_limit(int64_t cycles) { return (int64_t)g_wait_limit.exchange(cycles > 0 ? (long long)cycles : 0); }

SAKI_API int saki_set_phase_clock(int on) { return g_phase_clock.exchange(on ? 1 : 0); }

SAKI_API int saki_phase_cycles(void* cuda_stream, uint64_t* cycles) {
  g_err[0] = 0;
  if (!cycles) return fail(SAKI_ERR_INVALID_ARG, "NULL output pointer");
  memset(cycles, 0, SAKI_PHASE_COUNTERS * sizeof(uint64_t));
  unsigned int* const counters = last_counters();
  if (!counters) return SAKI_OK;
  cudaError_t e = cudaStreamSynchronize((cudaStream_t)cuda_stream);
  if (e != cudaSuccess) return cuda_fail(e, "cudaStreamSynchronize");
  e = cudaMemcpy(cycles, counters + 8, SAKI_PHASE_COUNTERS * sizeof(uint64_t), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return cuda_fail(e, "cudaMemcpy");
  return SAKI_OK;
}

SAKI_API int saki_set_spec_early_out(int on) { return g_spec_early_out.exchange(on ? 1 : 0); }

SAKI_API int saki_spec_positions_routed(void* cuda_stream, uint64_t* n_positions) {
  g_err[0] = 0;
  if (!n_positions) return fail(SAKI_ERR_INVALID_ARG, "NULL output pointer");
  *n_positions = 0;
  unsigned int* const counters = last_counters();
  if (!counters) return SAKI_OK;
  cudaError_t e = cudaStreamSynchronize((cudaStream_t)cuda_stream);
  if (e != cudaSuccess) return cuda_fail(e, "cudaStreamSynchronize");
  unsigned int h = 0;
  e = cudaMemcpy(&h, counters + 2, sizeof(h), cudaMemcpyDeviceToHost);
  if (e != cudaSuccess) return cuda_fail(e, "cudaMemcpy");
  *n_positions = h;
  return SAKI_OK;
}

SAKI_API uint64_t saki_launch_count(void) { return g_launches.load(); }

SAKI_API const char* saki_last_error(void) { return g_err; }

SAKI_API int saki_version(void) { return 100; }

}  // extern "C"
