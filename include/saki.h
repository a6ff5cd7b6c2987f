/*
 * saki.h - C ABI of the B200-native SAKI per-position routing library.
 *
 * For every generated position the library takes the full-vocabulary row of
 * student logits s and teacher logits t and computes, on the GPU:
 *   1. p = softmax(s/temperature), T = softmax(t/temperature)  (Section 3.1)
 *   2. the geometric bridge q = p^(1-lambda) T^lambda / Z with the largest
 *      lambda in [0,1] such that KL(q || p) <= eps              (Eqs. "bridge",
 *      "trust_region"; endpoints: Appendix J)
 *   3. the maximal coupling of the student's proposal x with q: accept with
 *      probability min(1, q(x)/p(x)), otherwise draw the committed token from
 *      [q-p]_+ / TV(p,q); TV(p,q) is the correction probability (Eqs.
 *      "accept", "residual", Proposition 1)
 *   4. the routed loss: -A log pi(x), A = -(log p(x) - log T(x)), at accepted
 *      positions (Eqs. "k1_loss_token", "k1_advantage_token"); -log pi(v*),
 *      v* = argmax T, at corrected positions (Eq. "teacher_mode_loss")
 *   5. the gradient of that loss with respect to the student logits
 *      (Eq. "general_objective"; lambda, q, the coupling outcome and A are
 *      constants of differentiation)
 *   6. for drafted blocks, the left-to-right first-rejection resolve of
 *      Section 3.5 / Appendix I;
 *   7. for the training loop, which sees metadata instead of logits, the
 *      same loss and gradient recomputed from freshly evaluated student
 *      logits (saki_route_bwd_from_meta).
 *
 * Conventions
 *   - Every pointer in the structs below is a DEVICE pointer owned by the
 *     caller unless a comment says HOST.  The library never frees or keeps
 *     them.  Input and output buffers must not overlap.
 *   - Calls are asynchronous on the given CUDA stream (a cudaStream_t passed
 *     as void*; NULL = the legacy default stream) and return after host-side
 *     validation and launch.  Outputs are valid once the stream has run.
 *   - No exception, abort or device trap crosses this boundary.  Bad
 *     arguments return an error code with nothing launched; bad DATA (a
 *     non-finite logit, a proposal id outside [0,V)) flags the row in
 *     `row_status`, zeroes its float outputs and gradient row and sets its
 *     ids to -1.
 *   - Random numbers: Philox4x32-10, key = (seed lo, seed hi), counter =
 *     (row lo, row hi, stage, block); stage 0 proposal Gumbel noise (word
 *     v%4 of block v/4), 1 acceptance uniform, 2 residual draw, 3 bonus draw,
 *     4 placement-control key (word 0 of block 0).  A word w gives the uniform ((w>>9)+0.5) 2^-23.
 *     `row` is the GLOBAL row id row_offset + i, so the random numbers a position
 *     sees do not depend on how a batch is chunked or sharded.
 *   - Results are deterministic: same call (inputs, sizes), same GPU model, same bits.  Chunking or
 *     sharding a batch leaves every output bit-identical as long as each piece is served by the same
 *     kernel as the whole; the library picks the kernel from the call's size (calls of at most 32 rows
 *     with V >= 65536 run one row per thread-block cluster, larger ones one row per SM), so a tail piece
 *     of 32 long rows or fewer agrees with the same rows inside a large call to the tolerances of the
 *     arithmetic (float outputs to ~1e-6, flags and ids wherever the decision is not within 1e-6 of
 *     its threshold), not to the bit.  saki_set_kernel pins the choice where bit-identity across pieces
 *     matters.
 */
#ifndef SAKI_H_
#define SAKI_H_

#include <stdint.h>

#if defined(__GNUC__)
#define SAKI_API __attribute__((visibility("default")))
#else
#define SAKI_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  SAKI_OK = 0,
  SAKI_ERR_INVALID_ARG = 1, /* NULL required pointer, N < 0, V < 2, ld < V, eps NaN or < 0,
                               temperature <= 0 or NaN, K outside [1,16], bad dtype */
  SAKI_ERR_UNSUPPORTED = 2, /* no CUDA device of compute capability 10.x, or a layout the
                               kernels do not serve */
  SAKI_ERR_CUDA = 3,        /* a CUDA runtime call failed; text via saki_last_error() */
  SAKI_ERR_ROW_STATUS = 4   /* returned only by saki_check(): some row was flagged */
} saki_status;

typedef enum { SAKI_F32 = 0, SAKI_BF16 = 1 } saki_dtype;

/* row_status bits */
#define SAKI_ROW_SATURATED    1u  /* lambda = 1: KL(T||p) <= eps (Appendix J, teacher endpoint) */
#define SAKI_ROW_EPS_ZERO     2u  /* eps <= 0: lambda = 0, q = p, never corrected (Appendix J) */
#define SAKI_ROW_MASKED       4u  /* mask[i] = 0: loss 0, gradient row 0 (M_t of Eq. "general_objective") */
#define SAKI_ROW_NONFINITE    8u  /* a logit of the row is NaN or +-Inf */
#define SAKI_ROW_BAD_ID      16u  /* proposal id outside [0,V) */
#define SAKI_ROW_TIMEOUT     32u  /* a bounded on-device wait expired; the row's outputs are void */
#define SAKI_ROW_NOT_COMPUTED 64u /* block verification: position after the first rejection */

/* Inputs of one routing call over N positions. */
typedef struct {
  const void* student_logits; /* [N,V] stored logits s, unit stride along V, row stride ld_s ELEMENTS */
  const void* teacher_logits; /* [N,V] stored logits t, row stride ld_t elements */
  int64_t ld_s, ld_t;         /* >= V */
  int64_t N;                  /* >= 0; 0 is a no-op */
  int32_t V;                  /* >= 2 */
  int32_t dtype;              /* saki_dtype of both logit arrays (and of dlogits) */
  const int32_t* proposal;    /* [N] the student's sampled token z_t ~ p_t (Section 3.3). Required */
  const uint8_t* mask;        /* [N] valid-response mask M_t, or NULL = all valid */
  float eps;                  /* trust-region radius of Eq. "trust_region", >= 0 */
  float temperature;          /* > 0; divides both logit rows */
  uint64_t seed;              /* Philox key */
  uint64_t row_offset;        /* global id of row 0 */
} saki_in;

/* Per-position outputs (the token-aligned metadata of Appendix K).  Any pointer
 * may be NULL (= not wanted) except `corrected` and `token`. Arrays of length N. */
typedef struct {
  uint8_t* corrected;    /* C_t: 1 = proposal rejected, token drawn from the residual */
  int32_t* token;        /* committed token y_t (= proposal when accepted) */
  int32_t* teacher_top1; /* v*_t = argmax_v t[v], lowest index among exact ties */
  float* lambda;         /* solved coefficient */
  float* kl;             /* KL(q||p) at lambda, nats */
  float* tv;             /* TV(p,q) = residual mass = correction probability */
  float* accept_prob;    /* min(1, q(x)/p(x)) */
  float* logp_x;         /* log p(x), log q(x), log T(x) at the proposal */
  float* logq_x;
  float* logT_x;
  float* logp_y;         /* log p(y), log q(y) at the committed token */
  float* logq_y;
  float* logT_y;         /* log T(y): with logp_y, the advantage at the committed token */
  float* loss;           /* routed loss of the position, NOT scaled by grad_scale; 0 where masked */
  uint32_t* row_status;  /* SAKI_ROW_* bits */
} saki_out;

/* Steps 1-4 above for N positions (no gradient).  `in`/`out` are HOST structs
 * read during the call.  Returns SAKI_OK after the kernels are enqueued. */
SAKI_API int saki_route_fwd(const saki_in* in, const saki_out* out, void* cuda_stream);

/* Steps 1-5: as saki_route_fwd, plus dlogits[i,:] = grad_scale * d loss_i / d s[i,:]
 * in the logits' dtype (round to nearest even), row stride ld_g >= V elements.
 * grad_scale is the caller's 1/N_valid (Appendix L, "Normalization"). */
SAKI_API int saki_route_fwd_bwd(const saki_in* in, const saki_out* out, void* dlogits,
                       int64_t ld_g, float grad_scale, void* cuda_stream);

/* saki_route_fwd_bwd for callers that must not allocate device memory: code that runs while an
 * allocator is locked or memory is fully committed (inside another framework's allocator callback, a
 * real-time serving loop with a frozen memory plan, a process whose device memory is entirely handed to
 * a pool it may not touch).  The paper has no counterpart; this is a property of the library only.
 * Same arguments, outputs and results as saki_route_fwd_bwd.  The one piece of scratch the routing needs
 * (the list of rows that the float32 kernel passes on to the float64 kernel) lives in a fixed device
 * array inside the library (4 MB per device, held from library load to process exit) instead of a buffer
 * allocated on first use, so the call makes no cudaMalloc / cudaFree and calls no allocating routine.
 *   - N may not exceed 1,048,576 rows: larger batches return SAKI_ERR_INVALID_ARG; split them.
 *   - The first call on a device looks up the array's device address (once, with that device current);
 *     make that first call before any stream capture.
 *   - All calls on a device share the array.  The library clears what must start at zero at the start of
 *     every call, but two calls whose kernels overlap on the GPU (different streams, no ordering between
 *     them) race on it: order them, or use saki_route_fwd_bwd for one of them. */
SAKI_API int saki_route_fwd_bwd_noalloc(const saki_in* in, const saki_out* out, void* dlogits,
                                        int64_t ld_g, float grad_scale, void* cuda_stream);

/* The same computation with every array in HOST memory (pageable or pinned):
 * the library stages rows through device buffers it allocates and caches,
 * overlapping the copies with the kernels on its own streams, and returns
 * when all outputs are in host memory.  `dlogits` may be NULL (forward only). */
SAKI_API int saki_route_host(const saki_in* in_host, const saki_out* out_host,
                    void* dlogits_host, int64_t ld_g, float grad_scale);

/* The trainer's step (Section 3.5, Appendix K): the rollout keeps the full-vocabulary rows on its own
 * GPUs and hands the training loop token-aligned metadata only.  The trainer recomputes the CURRENT
 * student's logits and needs, per position, the loss of Eq. "general_objective" and its gradient with
 * respect to those logits:
 *     C = 0:  L = -A log pi(x),   A = log T(x) - log p_rollout(x)  (Eqs. "k1_loss_token", "k1_advantage_token")
 *     C = 1:  L = -log pi(v*)                                      (Eq. "teacher_mode_loss")
 *     dlogits[i,:] = grad_scale * coef * (pi - onehot(tok)) / temperature,  (coef, tok) = (A, x) or (1, v*)
 * with pi = softmax(student_logits[i,:] / temperature) of the logits passed HERE.  On the rollout's own
 * logits and metadata this reproduces saki_route_fwd_bwd's loss and gradient. */
typedef struct {
  const void* student_logits;   /* [N,V] current student logits, unit stride along V, row stride ld_s elements */
  int64_t ld_s;                 /* >= V */
  int64_t N;                    /* >= 0 */
  int32_t V;                    /* >= 2 */
  int32_t dtype;                /* saki_dtype of the logits and of dlogits */
  const uint8_t* corrected;     /* [N] C_t as returned by the routing call. Required */
  const int32_t* proposal;      /* [N] x_t, the supervised token where C_t = 0. Required */
  const int32_t* teacher_top1;  /* [N] v*_t, the supervised token where C_t = 1. Required */
  const float* advantage;       /* [N] A_t = logT_x - logp_x of the routing call (a constant of
                                   differentiation); read where C_t = 0. Required */
  const uint8_t* mask;          /* [N] M_t or NULL = all valid */
  const uint32_t* rollout_status; /* [N] row_status of the routing call, or NULL: rows it flagged NONFINITE,
                                   BAD_ID, TIMEOUT or NOT_COMPUTED contribute nothing here */
  float temperature;            /* > 0 */
} saki_meta_in;

typedef struct {
  float* loss;          /* [N] un-normalised loss of the position; 0 where it contributes nothing. May be NULL */
  float* logp_tok;      /* [N] log pi(tok) under the current logits. May be NULL */
  uint32_t* row_status; /* [N] 0, or SAKI_ROW_MASKED / NOT_COMPUTED (nothing to do), or NONFINITE (a logit or
                           the advantage is not finite) / BAD_ID (supervised token outside [0,V)): loss 0 and
                           gradient row 0 in all four cases. May be NULL */
} saki_meta_out;

/* `in`/`out` are HOST structs read during the call; dlogits [N,V] (required), row stride ld_g >= V
 * elements, in the logits' dtype (round to nearest even).  Asynchronous on the stream.  bf16 rows with
 * 16-byte aligned rows, strides and V multiples of 8 and V >= 2048 run on a streaming kernel that reads
 * each row from HBM once and writes the gradient row once; everything else, and rows whose float32
 * sums overflow, on a float64 kernel.  Flagged rows count towards saki_check(). */
SAKI_API int saki_route_bwd_from_meta(const saki_meta_in* in, const saki_meta_out* out, void* dlogits,
                                      int64_t ld_g, float grad_scale, void* cuda_stream);

/* Placement controls of the paper's ablation (Appendix "placement_control"): for every trajectory b
 * (positions seq_start[b] .. seq_start[b+1]-1) choose m_b = number of its corrected valid positions,
 * valid positions that receive the teacher-mode loss INSTEAD of the coupling's own corrections:
 *   SAKI_SELECT_RANDOM       m_b valid positions uniformly at random;
 *   SAKI_SELECT_TV_WEIGHTED  m_b valid positions without replacement with weights tv[t], by
 *                            exponential-race keys -log(U_t)/tv[t], the m_b smallest; if fewer than m_b
 *                            valid positions have positive TV, the rest is filled uniformly (smallest U_t).
 * U_t is the uniform of (seed, row_offset + t, stage 4); a position is valid if mask[t] != 0 and the
 * rollout routed it; ties go to the lower index.  Keys are formed in float64.  Feed `selected` to
 * saki_route_bwd_from_meta as its `corrected`.  (Teacher-sampled supervision, the other ablation,
 * needs no call of its own: draw the target with saki_sample_proposal on the teacher's logits under
 * another seed and pass it as `teacher_top1`.) */
typedef enum { SAKI_SELECT_RANDOM = 0, SAKI_SELECT_TV_WEIGHTED = 1 } saki_select_mode;
typedef struct {
  int64_t N;                      /* positions, = seq_start[B] */
  int64_t B;                      /* trajectories */
  const int64_t* seq_start;       /* [B+1] DEVICE, non-decreasing, seq_start[0] = 0 */
  const uint8_t* corrected;       /* [N] C_t of the routing call. Required */
  const float* tv;                /* [N] TV(p_t, q_t) of the routing call. Required in TV-weighted mode */
  const uint8_t* mask;            /* [N] or NULL */
  const uint32_t* rollout_status; /* [N] or NULL */
  int32_t mode;                   /* saki_select_mode */
  uint64_t seed;
  uint64_t row_offset;            /* global id of position 0 */
} saki_select_in;

/* selected: [N] uint8 (required); m: [B] int32 or NULL.  Asynchronous on the stream. */
SAKI_API int saki_select_tm(const saki_select_in* in, uint8_t* selected, int32_t* m, void* cuda_stream);

/* Vocabulary-sharded rows (the paper fixes only the [B,K,V] -> [BK,V] shape of the engine's logits,
 * Appendix K "Engine-Resident q Backend"; with a tensor-parallel lm-head each GPU holds a slice of every
 * row).  Rank r of `world` holds columns [v0, v0 + V_local) of both logit tensors; the slices of the ranks,
 * taken in rank order, tile [0, V) without gaps.  A row is routed without gathering it, in stages; in each
 * stage every rank reduces its slice to SAKI_VSHARD_PARTIALS doubles per row (saki_vshard_partial), the
 * ranks exchange them (the caller's all-gather into [world][N][SAKI_VSHARD_PARTIALS], rank-major) and
 * every rank folds the gathered partials, in rank order, into the same per-row state of
 * SAKI_VSHARD_STATE doubles (saki_vshard_combine).  Stages, run in this order:
 *   0  maxima, teacher argmax, sums of exponentials and moments of the logit difference (Section 3.1)
 *   1  one evaluation of KL(q_beta || p) and of the cumulants of the logit difference at every unsettled
 *      row's current beta (Eqs. "bridge", "trust_region"); repeat stage 1 until the combine reports no row
 *      still solving (each wave moves to the root of a fourth-order model: two waves as a rule)
 *   2  shares of TV(p, q) and KL(q || p); the combine decides acceptance (Eq. "accept"), the routed loss
 *      (Eqs. "k1_loss_token", "teacher_mode_loss") and which rank owns the residual draw (Eq. "residual")
 *   3  the gradient slice (Eq. "general_objective": dlogits_slice [N, V_local], same dtype, may be NULL) and,
 *      on the owning rank, the drawn token; the combine writes the per-position outputs
 * Arithmetic: bf16 slices that start on 16-byte boundaries (V_local, v0 and the strides multiples of 8) with
 * eps >= 0.02 are reduced with the per-element arithmetic of the unsharded bf16 kernels (float32 elements,
 * float64 sums and scalars; a row that float32 cannot resolve goes on in float64, decided in the combine);
 * everything else, and every call under saki_set_kernel(1), is float64 throughout.  Results equal the
 * unsharded call's within the tolerances of that arithmetic (float64: ~1e-12 before the cast to float32;
 * flags and ids wherever the decision is not within rounding of its threshold) and do not depend on the
 * number of ranks beyond that.  saki_set_kernel must be the same on every rank of a call.  Arguments: `proposal` holds GLOBAL token ids; `state` and
 * `partial` are caller-owned buffers ([N][SAKI_VSHARD_STATE], [N][SAKI_VSHARD_PARTIALS] doubles); `state`
 * may be NULL at stage 0 of saki_vshard_partial.  saki_vshard_partial and saki_vshard_combine take DEVICE
 * pointers and run asynchronously on the stream; `n_solving` (device, may be NULL) receives the number of
 * rows that need another stage-1 wave (meaningful after stages 0 and 1).  saki_vshard_combine_host is the
 * same combine for HOST buffers (every pointer, `proposal` and `mask` of `in` and the arrays of `out`
 * included, is a host pointer; the logits pointers of `in` are not read): for callers that exchange
 * through host memory.  Errors: SAKI_ERR_INVALID_ARG for NULL required pointers, a stage outside 0..3,
 * sizes or strides that do not fit; SAKI_ERR_CUDA for a failed launch. */
#define SAKI_VSHARD_PARTIALS 16
#define SAKI_VSHARD_STATE 32
typedef struct {
  const void* student_logits;  /* DEVICE [N, V_local]: this rank's columns, unit column stride, row stride ld_s elements */
  const void* teacher_logits;  /* DEVICE [N, V_local], row stride ld_t */
  int64_t ld_s, ld_t, N;
  int32_t V;                   /* the whole vocabulary */
  int32_t V_local, v0;         /* this rank's columns are [v0, v0 + V_local) */
  int32_t dtype;               /* SAKI_F32 or SAKI_BF16 */
  const int32_t* proposal;     /* [N] global ids of the student's sampled tokens */
  const uint8_t* mask;         /* [N] or NULL */
  float eps, temperature;
  uint64_t seed, row_offset;
  int32_t rank, world;
} saki_vshard_in;
SAKI_API int saki_vshard_partial(const saki_vshard_in* in, int stage, const double* state, double* partial,
                                 void* dlogits_slice, int64_t ld_g, float grad_scale, void* cuda_stream);
SAKI_API int saki_vshard_combine(const saki_vshard_in* in, int stage, const double* gathered, double* state,
                                 const saki_out* out, uint32_t* n_solving, void* cuda_stream);
SAKI_API int saki_vshard_combine_host(const saki_vshard_in* in, int stage, const double* gathered, double* state,
                                      const saki_out* out, int32_t* n_solving);

/* The step in front of the path (Section 3.5, Appendix K: drafting and verification leave full-vocabulary
 * logits): logits = hidden x weight^T in bf16 on the tensor cores, fp32 accumulation, with the row
 * statistics of the first pass of routing (Section 3.1: p = softmax(logits / tau)) taken in the GEMM's
 * epilogue from the ROUNDED bf16 values that are stored: row_max[i] = max_v logits[i, v] and
 * lse[i] = log sum_v exp(logits[i, v] / temperature).  All pointers are DEVICE pointers owned by the caller:
 *   hidden  [N, d] bf16, unit stride along d, row stride ld_h elements
 *   weight  [V, d] bf16 (one row per vocabulary entry), row stride ld_w
 *   logits  [N, V] bf16 out, row stride ld_l; row_max, lse: [N] float out (either may be NULL)
 *   scratch saki_lmhead_scratch_bytes(N, V) bytes, 256-byte aligned (per-tile partial statistics)
 * Requirements: 16-byte aligned hidden / weight / logits, ld_h, ld_w, ld_l and V multiples of 8, d >= 8.
 * Asynchronous on the stream.  Errors: SAKI_ERR_INVALID_ARG (NULL pointers, sizes, strides, scratch too
 * small), SAKI_ERR_UNSUPPORTED (alignment), SAKI_ERR_CUDA.  Every wait inside the kernel is bounded; should
 * one run out (a fault of the machine, not of the data) the kernel still returns and row_max and lse are NaN. */
typedef struct {
  const void* hidden; int64_t ld_h;
  const void* weight; int64_t ld_w;
  int64_t N; int32_t d; int32_t V;
  float temperature;
} saki_lmhead_in;
SAKI_API int64_t saki_lmhead_scratch_bytes(int64_t N, int32_t V);
SAKI_API int saki_lmhead_lse(const saki_lmhead_in* in, void* logits, int64_t ld_l, float* row_max, float* lse,
                             void* scratch, int64_t scratch_bytes, void* cuda_stream);

/* Block verification (Section 3.5, Appendix I) of B drafted blocks of K tokens. */
typedef struct {
  const void* student_logits; /* [B,K+1,V]: position j of sequence b at element offset
                                 b*ss_seq + j*ss_pos; unit stride along V */
  const void* teacher_logits; /* [B,K+1,V], strides ts_seq, ts_pos (elements) */
  int64_t ss_seq, ss_pos, ts_seq, ts_pos;
  int64_t B;                  /* >= 0 */
  int32_t K;                  /* 1..16 drafted tokens per block */
  int32_t V;
  int32_t dtype;
  const int32_t* draft;       /* [B,K] drafted ids, row stride draft_ld */
  int64_t draft_ld;
  float eps, temperature;
  uint64_t seed;
  uint64_t seq_offset;        /* global id of sequence 0; position j of sequence b uses the
                                 random stream of row (seq_offset+b)*(K+1)+j */
} saki_spec_in;

typedef struct {
  int32_t* n_accept;           /* [B] length of the accepted prefix, 0..K */
  int32_t* next_token;         /* [B] residual draw at the first rejection, else a draw from q
                                  at the bonus position K; -1 if that row was flagged */
  uint8_t* next_is_correction; /* [B] 1 if next_token is a correction */
  saki_out per_pos;            /* arrays of length B*(K+1), row b*(K+1)+j; `corrected` and
                                  `token` required; rows after the first rejection are zeroed
                                  and carry SAKI_ROW_NOT_COMPUTED; `loss` is not written */
} saki_spec_out;

SAKI_API int saki_spec_verify(const saki_spec_in* in, const saki_spec_out* out, void* cuda_stream);

/* Harness utility (the proposal is an input of the method: z_t ~ p_t, Section
 * 3.3): out[i] = argmax_v (logits[i,v]/temperature + G_v) with Gumbel noise
 * G_v = -log(-log((w_v+0.5) 2^-32)) from stage 0 of row row_offset+i; lowest
 * index on ties.  Keys are formed in float64. */
SAKI_API int saki_sample_proposal(const void* logits, int64_t ld, int64_t N, int32_t V,
                         int32_t dtype, float temperature, uint64_t seed,
                         uint64_t row_offset, int32_t* out, void* cuda_stream);

/* Synchronises the stream, then reports and clears the number of rows flagged
 * NONFINITE, BAD_ID or TIMEOUT by calls on this device since the last check.
 * Returns SAKI_ERR_ROW_STATUS if that number is non-zero.  n_flagged may be NULL. */
SAKI_API int saki_check(void* cuda_stream, uint64_t* n_flagged);

/* Selects the row kernel: 0 = automatic, 1 = the general kernel (one block per
 * row, float64, any V, dtype and layout), 2 = the register-resident cluster
 * kernel (one row per cluster of up to 8 blocks), 3 = the row-per-SM kernel
 * (one row per block; shared memory plus L2; one block of 512 threads per SM for
 * V > 98304, two of 256 for shorter rows).  2 and 3 serve bf16 rows with
 * 16-byte aligned rows and V a multiple of 8, V >= 2048 (2: V <= 163840; and
 * eps = 0 or eps >= 5e-3: its float32 sums cannot resolve smaller radii to the
 * tolerance, whereas 3 takes every radius); other inputs fall back to 1.  Automatic prefers 3,
 * except for calls of at most 32 rows with V >= 65536 that 2 can serve: a few long rows finish sooner
 * spread over the whole GPU.  Process-wide; meant for
 * tests and benchmarks.  Returns the previous value. */
SAKI_API int saki_set_kernel(int which);

/* Which row kernel the calling thread's last routing call used: 1 general, 2 cluster,
 * 3 row-per-SM, 4 the streaming kernel of saki_route_bwd_from_meta (which saki_set_kernel(1) also
 * turns off), 0 if none yet. */
SAKI_API int saki_last_kernel(void);

/* Two-tier routing: the float32 kernels (2, 3) hand rows whose KL they cannot resolve to the
 * tolerance (very small eps, nearly one-hot rows) to the float64 kernel, through a row list in device
 * memory that the library allocates once per device and stream and keeps (calls on different streams
 * may overlap; calls on one stream are ordered by it).  Synchronises the stream and returns
 * how many rows of the calling thread's last routing call took that second tier. */
SAKI_API int saki_redo_count(void* cuda_stream, uint64_t* n_rows);

/* Synchronises the stream and returns how many evaluation passes (one pass over a row at a trial
 * beta, Section 3.2's boundary search) the row-per-SM kernel ran in the calling thread's last routing
 * call, summed over its rows; 0 if another kernel served the call.  Every row also takes the two fixed
 * passes (log-sum-exp with moments, final). */
SAKI_API int saki_solve_evaluations(void* cuda_stream, uint64_t* n_passes);

/* Failure behaviour of the row-per-SM kernel (no counterpart in the paper).  A thread block waits for a
 * row's bulk copy from global memory for a bounded number of SM cycles (about two seconds' worth by
 * default).  If the wait runs out the block stops fetching, flags that row and every row it still owns
 * SAKI_ROW_TIMEOUT with zero outputs, waits (full limit) for the copy it has in flight, and returns: the
 * kernel always terminates, saki_check() counts the flagged rows and later calls are unaffected.  This
 * call sets the limit for the routing calls that follow, from any thread (0: the default), and returns
 * the previous value; tests use a limit of a few cycles to exercise that path without withholding
 * anything. */
SAKI_API int64_t saki_set_wait_limit(int64_t cycles);

/* Where the row-per-SM kernel's time goes (no counterpart in the paper: a measurement aid, off by
 * default; it costs the kernel about 1.5 %).  saki_set_phase_clock(1) makes the routing calls that follow,
 * from any thread, carry the clock (returns the previous setting).  With it, thread 0 of
 * every thread block reads the SM's cycle counter at fixed marks of its row loop and adds the differences
 * up per phase; saki_phase_cycles synchronises the stream and copies the SAKI_PHASE_COUNTERS sums (over all thread
 * blocks) of the calling thread's last routing call into cycles[] (HOST memory, caller-owned): in order,
 * the top of the row loop, the wait for the row's bulk copy, pass "lse", its warp reductions up to the
 * first block barrier, the block-level gather, the float64 scalar step, the top of an evaluation, pass
 * "solve", its block combine, its scalar step, the top of pass "final", pass "final", the end of the row
 * loop, the kernel's tail, one spare word, and last the number of rows behind the sums.  Divide by that
 * number for cycles per row.  All zero if the clock was off or another kernel served the call. */
#define SAKI_PHASE_COUNTERS 16
SAKI_API int saki_set_phase_clock(int on);
SAKI_API int saki_phase_cycles(void* cuda_stream, uint64_t* cycles);

/* Block verification, early out (Section 3.5: what follows a sequence's first rejected position is
 * discarded).  When on (the default) and the call has at least two sequences per SM, the row-per-SM
 * kernel hands out positions from a device counter in position-major order and passes over a position
 * once an earlier position of its sequence is known to be rejected or flagged, so most discarded
 * positions are never read; nothing waits, a position whose predecessor is still undecided is routed.
 * Which block routes which position varies from run to run; the outputs do not (every random number is
 * keyed by the position).  Off, or with fewer sequences: every position of every sequence is routed,
 * then resolved (what the other kernels always do).  Process-wide; returns the previous value. */
SAKI_API int saki_set_spec_early_out(int on);

/* Synchronises the stream and returns how many positions the calling thread's last saki_spec_verify
 * actually routed when it ran with early out (0 otherwise); B * (K + 1) minus this were skipped. */
SAKI_API int saki_spec_positions_routed(void* cuda_stream, uint64_t* n_positions);

/* Number of kernels this library has launched in this process (all threads). */
SAKI_API uint64_t saki_launch_count(void);

/* Text of the last error on the calling thread ("" if none). Never NULL. */
SAKI_API const char* saki_last_error(void);

/* Library version, major*10000 + minor*100 + patch. */
SAKI_API int saki_version(void);

#ifdef __cplusplus
}
#endif
#endif /* SAKI_H_ */
