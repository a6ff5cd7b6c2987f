// Shared declarations of the SAKI routing library (device + host side).
#pragma once
#include <cuda_runtime.h>
#include <cuda_bf16.h>
#include <stdint.h>
#include "../../include/saki.h"

namespace saki {

// Phases of the row-per-SM kernel's row loop, as timed by thread 0 of every CTA (saki_phase_cycles):
// the three passes, the waits and block reductions around them, the float64 scalar steps between them.
enum { PH_ROW_TOP = 0, PH_COPY_WAIT, PH_LSE, PH_LSE_REDUCE, PH_LSE_GATHER, PH_LSE_SCALAR, PH_SOLVE_TOP, PH_SOLVE,
       PH_SOLVE_COMBINE, PH_SOLVE_SCALAR, PH_FINAL_TOP, PH_FINAL, PH_ROW_END, PH_TAIL, PH_SPARE, PH_ROWS,
       PH_LAST /* shared memory only: the last mark */, PH_WORDS };
static_assert(PH_LAST == SAKI_PHASE_COUNTERS, "saki.h publishes the number of phase counters");

enum { STAGE_PROPOSE = 0, STAGE_ACCEPT = 1, STAGE_RESIDUAL = 2, STAGE_BONUS = 3, STAGE_SELECT = 4 };

// Everything a row kernel needs; passed by value as the kernel parameter.
// Plain routing and block verification share it: row i is position
// j = i % K1 of sequence b = i / K1 (K1 = 1 for plain routing).
struct RowParams {
  const void* s;
  const void* t;
  int64_t s_seq, s_pos, t_seq, t_pos;  // element strides (plain: s_seq = ld_s, s_pos = 0)
  int64_t n_rows;
  int32_t V;
  int32_t K1;                          // positions per sequence; the last one is the bonus row if spec
  int32_t spec;                        // 1: block verification (proposal from draft, bonus row)
  const int32_t* proposal;             // plain: [N]; spec: draft [B,K] with row stride prop_ld
  int64_t prop_ld;
  const uint8_t* mask;
  float eps;
  float temperature;
  uint64_t seed;
  uint64_t row_offset;
  saki_out out;
  void* dlogits;                       // NULL: forward only
  int64_t ld_g;
  float grad_scale;
  unsigned long long* flagged;         // device counter of flagged rows
  int32_t* redo_list;                  // scratch: rows the float32 kernels hand to the float64 kernel
  unsigned int* redo_count;            // scratch: their number (zeroed before the launch, with the three words
                                       // after it: [1], [2] see seq_next; [3] evaluation passes of the row-per-SM kernel)
  float* redo_guess;                   // scratch or NULL: what the float32 kernel made of lambda for each row of redo_list (< 0: nothing)
  int32_t from_list;                   // general kernel only: route the rows of redo_list
  int32_t list_min, list_max;          // ... and only if their number lies in [list_min, list_max] (0, 0: any number)
  long long wait_limit;                // row-per-SM kernel: SM cycles a block waits for a row's bulk copy (<= 0: ~2 s)
  unsigned long long* phase_cycles;    // row-per-SM kernel: [SAKI_PHASE_COUNTERS] cycle sums per phase (zeroed before
                                       // the launch); NULL: not wanted
  unsigned int* seq_next;              // row-per-SM kernel, block verification with early out: [0] ticket counter,
                                       // [1] positions routed (both zeroed before the launch); NULL: rows in static order
  int* seq_stop;                       // [n_rows / K1] position of each sequence's first stop (>= K1 before the launch)
};

// Parameters of the metadata-driven backward kernels (saki_route_bwd_from_meta).
struct MetaParams {
  const void* s;                       // current student logits [n_rows, V]
  int64_t ld_s;
  int64_t n_rows;
  int32_t V;
  const uint8_t* corrected;
  const int32_t* proposal;
  const int32_t* teacher_top1;
  const float* advantage;
  const uint8_t* mask;                 // may be NULL
  const uint32_t* rollout_status;      // may be NULL
  float temperature;
  saki_meta_out out;
  void* dlogits;
  int64_t ld_g;
  float grad_scale;
  unsigned long long* flagged;         // device counter of flagged rows
  int32_t* redo_list;                  // rows the streaming kernel hands to the float64 kernel
  unsigned int* redo_count;
  int32_t from_list;                   // general kernel only: take the rows of redo_list
};

// Parameters of the placement-control kernel (saki_select_tm).
struct SelectParams {
  int64_t N, B;
  const int64_t* seq_start;
  const uint8_t* corrected;
  const float* tv;
  const uint8_t* mask;
  const uint32_t* rollout_status;
  int32_t mode;
  uint64_t seed, row_offset;
  uint8_t* selected;
  int32_t* m;
};

// ---- Philox4x32-10 (Salmon et al., SC'11), written from the published round function ----
__host__ __device__ inline void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                              uint32_t k0, uint32_t k1, uint32_t out[4]) {
  const uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
#pragma unroll
  for (int r = 0; r < 10; ++r) {
    uint64_t p0 = (uint64_t)M0 * c0;
    uint64_t p1 = (uint64_t)M1 * c2;
    uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
    uint32_t n1 = (uint32_t)p1;
    uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
    uint32_t n3 = (uint32_t)p0;
    c0 = n0; c1 = n1; c2 = n2; c3 = n3;
    k0 += W0; k1 += W1;
  }
  out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

// the one uniform a (row, stage) pair owns: an odd multiple of 2^-24 in (0,1)
__host__ __device__ inline double scalar_uniform(uint64_t seed, uint64_t row, uint32_t stage) {
  uint32_t w[4];
  philox4x32_10((uint32_t)row, (uint32_t)(row >> 32), stage, 0u, (uint32_t)seed, (uint32_t)(seed >> 32), w);
  return ((double)(w[0] >> 9) + 0.5) * (1.0 / 8388608.0);
}

template <typename T> __device__ __forceinline__ float ld_as_float(const T* p, int64_t i);
template <> __device__ __forceinline__ float ld_as_float<float>(const float* p, int64_t i) { return p[i]; }
template <> __device__ __forceinline__ float ld_as_float<__nv_bfloat16>(const __nv_bfloat16* p, int64_t i) {
  return __bfloat162float(p[i]);
}
template <typename T> __device__ __forceinline__ void st_from_float(T* p, int64_t i, float v);
template <> __device__ __forceinline__ void st_from_float<float>(float* p, int64_t i, float v) { p[i] = v; }
template <> __device__ __forceinline__ void st_from_float<__nv_bfloat16>(__nv_bfloat16* p, int64_t i, float v) {
  p[i] = __float2bfloat16_rn(v);
}

// Per-row scalar results, written by one thread.
struct RowResult {
  int corrected, token, vstar;
  float lambda, kl, tv, accept, logp_x, logq_x, logT_x, logp_y, logq_y, logT_y, loss;
  uint32_t status;
};

__host__ __device__ inline void write_row(const saki_out& o, int64_t i, const RowResult& r, bool write_loss) {
  o.corrected[i] = (uint8_t)r.corrected;
  o.token[i] = r.token;
  if (o.teacher_top1) o.teacher_top1[i] = r.vstar;
  if (o.lambda) o.lambda[i] = r.lambda;
  if (o.kl) o.kl[i] = r.kl;
  if (o.tv) o.tv[i] = r.tv;
  if (o.accept_prob) o.accept_prob[i] = r.accept;
  if (o.logp_x) o.logp_x[i] = r.logp_x;
  if (o.logq_x) o.logq_x[i] = r.logq_x;
  if (o.logT_x) o.logT_x[i] = r.logT_x;
  if (o.logp_y) o.logp_y[i] = r.logp_y;
  if (o.logq_y) o.logq_y[i] = r.logq_y;
  if (o.logT_y) o.logT_y[i] = r.logT_y;
  if (o.loss && write_loss) o.loss[i] = r.loss;
  if (o.row_status) o.row_status[i] = r.status;
}

__host__ __device__ inline RowResult zero_row(uint32_t status) {
  RowResult r;
  r.corrected = 0; r.token = -1; r.vstar = -1;
  r.lambda = r.kl = r.tv = r.accept = r.logp_x = r.logq_x = r.logT_x = r.logp_y = r.logq_y = r.logT_y = r.loss = 0.f;
  r.status = status;
  return r;
}

// host-side launchers (defined in the kernel translation units)
cudaError_t launch_general(const RowParams& p, int dtype, cudaStream_t st, int* n_launches);
cudaError_t launch_cluster(const RowParams& p, cudaStream_t st, int* n_launches, bool* served);
bool cluster_can_serve(const RowParams& p, int dtype);
cudaError_t launch_rowsm(const RowParams& p, cudaStream_t st, int* n_launches, bool* served);
namespace full_sm { cudaError_t launch(const RowParams& p, cudaStream_t st, int* n_launches, bool* served); int max_v(); }
namespace half_sm { cudaError_t launch(const RowParams& p, cudaStream_t st, int* n_launches, bool* served); int max_v(); }
namespace quarter_sm { cudaError_t launch(const RowParams& p, cudaStream_t st, int* n_launches, bool* served); int max_v(); }
bool rowsm_can_serve(const RowParams& p, int dtype);
cudaError_t launch_meta_general(const MetaParams& p, int dtype, cudaStream_t st, int* n_launches);
cudaError_t launch_meta_stream(const MetaParams& p, cudaStream_t st, int* n_launches, bool* served);
bool meta_stream_can_serve(const MetaParams& p, int dtype);
cudaError_t launch_select(const SelectParams& p, cudaStream_t st, int* n_launches);
cudaError_t launch_vshard_partial(const saki_vshard_in& in, int stage, const double* state, double* partial, void* dlogits,
                                  int64_t ld_g, float grad_scale, bool allow_fast, cudaStream_t st);
cudaError_t launch_vshard_combine(const saki_vshard_in& in, int stage, const double* gathered, double* state, const saki_out& out,
                                  unsigned int* n_solving, bool allow_fast, cudaStream_t st);
int64_t lmhead_scratch_bytes(int64_t N, int32_t V);
cudaError_t launch_lmhead(const saki_lmhead_in& in, void* logits, int64_t ld_l, float* row_max, float* lse, void* scratch,
                          cudaStream_t st, const char** why);
int vshard_combine_host(const saki_vshard_in& in, int stage, const double* gathered, double* state, const saki_out& out,
                        bool allow_fast);

}  // namespace saki
