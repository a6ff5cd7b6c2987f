// One-row-per-SM kernel for bf16 rows: the implementation, compiled twice.
//   saki_rowsm.cu       one persistent CTA of 512 threads per SM (namespace full_sm)
//   saki_rowsm_half.cu  two persistent CTAs of 256 threads per SM (namespace half_sm, SAKI_ROWSM_HALF):
//                       for short rows, whose passes are short against the serial phases between them,
//                       so that one CTA's scalar phases run under the other CTA's passes
//   saki_rowsm_quarter.cu  four of 128 threads (namespace quarter_sm, SAKI_ROWSM_QUARTER): shorter rows still
//
// A persistent CTA routes whole rows, one after the
// other.  A row pair (student + teacher, e.g. 608 KB at V = 151936) does not
// fit on one SM.  Every warp owns a contiguous segment of the row and visits
// it in steps of 32 chunks of 8 elements; it keeps
//   - the leading steps of its segment resident in shared memory, filled by
//     per-warp 1-D bulk async copies on an mbarrier, issued for the NEXT row
//     as soon as the warp has read its resident part for the last time;
//   - the rest in global memory, streamed in every pass through a small ring
//     of per-lane cp.async slots.  Each row is touched by one SM only, so
//     after the first pass these reads are L2 hits.
// HBM therefore sees each logit row once and the gradient row once.  All
// reductions stay inside the CTA (warp shuffles + shared memory), so a pass of
// ~150 k elements per SM amortises them.  Passes:
//   lse      2 exponentials/element under shifts fixed before the pass:
//            log-sum-exps, moments of the logit difference under p (initial
//            guess of lambda), KL(T||p), maxima, teacher argmax
//   solve    1 exponential/element per evaluation of KL(q_beta||p) and the
//            first four cumulants of the logit difference under q_beta;
//            lambda = root of the fourth-order Taylor model in a bisection
//            bracket (Eqs. "bridge", "trust_region")
//   final    2 exponentials/element: TV = sum [q-p]_+ with per-step ordered
//            partial sums for the inverse-CDF residual draw (Eqs. "accept",
//            "residual"), gradient row streamed out (Eq. "general_objective")
// Per-element work is float32 (packed f32x2 FMAs, ex2.approx); cross-thread
// combinations and per-row scalars are float64.
#include "saki_device.cuh"
#include <mutex>

#if defined(SAKI_ROWSM_QUARTER)
#define SAKI_ROWSM_NS quarter_sm
#define SAKI_ROWSM_THREADS 128
#define SAKI_ROWSM_CTAS 4
#elif defined(SAKI_ROWSM_HALF)
#define SAKI_ROWSM_NS half_sm
#define SAKI_ROWSM_THREADS 256
#define SAKI_ROWSM_CTAS 2
#else
#define SAKI_ROWSM_NS full_sm
#define SAKI_ROWSM_THREADS 512
#define SAKI_ROWSM_CTAS 1
#endif

namespace saki {
namespace SAKI_ROWSM_NS {

constexpr int RT = SAKI_ROWSM_THREADS;  // threads per CTA
constexpr int RW = RT / 32;             // warps per CTA
constexpr int CTAS_PER_SM = SAKI_ROWSM_CTAS;
constexpr int KS_MAX = 208 / (RW * CTAS_PER_SM);   // steps per warp that fit in shared memory (a step = 32 chunks of 8 elements = 1 KB of logit pairs)
constexpr int MAX_STEPS = 64;            // steps per warp the draw bookkeeping can hold (V <= 64*32*8*RW)
constexpr int RES_CHUNKS = KS_MAX * 32; // resident chunks per warp and row
constexpr int RNV = 9;                  // doubles per partial vector
static_assert(RW >= 14 || RW == 8 || RW == 4, "the eight gather roles go round the first eight warps; the side work has warps of its own, or is shared out");
// Who does what beside the passes.  With 14 warps or more the row scalars that do not depend on the
// passes (uniforms, the logits at the proposal) are fetched by warps 8-10 while warps 0-7 gather; with
// eight warps, by warps 1-3 before the block barrier that ends pass "lse".  After the gather, while
// thread 0 does the scalars: FIN_WARP finishes the previous row, RES_WARP reserves the next row of a
// block verification, lane 0 of SV_WARP fetches the student's logit at the teacher's argmax.
constexpr bool SIDE_WARPS = RW >= 14;
constexpr int UACC_WARP = SIDE_WARPS ? 8 : 1, UDRAW_WARP = SIDE_WARPS ? 9 : 2, SX_WARP = SIDE_WARPS ? 10 : 3;
constexpr int RES_WARP = SIDE_WARPS ? 11 : (RW == 8 ? 5 : 2), SV_WARP = SIDE_WARPS ? 13 : (RW == 8 ? 6 : 3);
static_assert(KS_MAX - 4 >= 1, "every warp keeps at least its first step resident");

constexpr int ROFF_S = 0;                                        // [RW][RES_CHUNKS] uint4
constexpr int ROFF_T = RW * RES_CHUNKS * 16;
constexpr int ROFF_RED = 2 * RW * RES_CHUNKS * 16;               // [RNV][RW] doubles
constexpr int ROFF_GAT = ROFF_RED + RNV * RW * 8;                // [16] doubles: block totals
constexpr int ROFF_BC = ROFF_GAT + 16 * 8;                       // [2][BC_DOUBLES] doubles, alternating by row
constexpr int ROFF_WMAX = ROFF_BC + 2 * BC_DOUBLES * 8;          // [3][RW]: teacher maximum, its index, student maximum per warp
constexpr int ROFF_STEP = ROFF_WMAX + 4 * RW * 4;                // [RW][MAX_STEPS] floats: draw weight of each step
constexpr int ROFF_FIN = ROFF_STEP + RW * MAX_STEPS * 4;          // [2][2][RW] doubles: what pass "final" leaves per warp, by row parity
constexpr int ROFF_MBAR = ROFF_FIN + 2 * 2 * RW * 8;
constexpr int FIN_WARP = SIDE_WARPS ? 12 : (RW == 8 ? 4 : 1);   // the warp that finishes the previous row
constexpr int ROFF_SEQ = ROFF_MBAR + 16;   // [4] ints: block verification, the CTA's reservation state
constexpr int ROFF_PH = ROFF_SEQ + 16;     // [PH_WORDS] 64-bit words: the phase clock of thread 0
constexpr int RSMEM_BYTES = ROFF_PH + PH_WORDS * 8;

// L2 residency hints: the part of a row that is re-read from L2 in every pass is marked
// evict-last; everything that passes through L2 once (the shared-memory resident part, the
// gradient row) is marked evict-first so that it does not push the re-read part out.
__device__ __forceinline__ uint64_t policy_evict_last() {
  uint64_t p;
  asm("createpolicy.fractional.L2::evict_last.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ uint64_t policy_evict_first() {
  uint64_t p;
  asm("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(p));
  return p;
}
__device__ __forceinline__ void bulk_load_hint(void* dst_smem, const void* src, uint32_t bytes, uint64_t* bar, uint64_t pol) {
  asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;"
               ::"r"(smem_addr(dst_smem)), "l"(src), "r"(bytes), "r"(smem_addr(bar)), "l"(pol) : "memory");
}
__device__ __forceinline__ uint4 ld_l2(const __nv_bfloat16* p, uint64_t pol) {
  uint4 v;
  asm volatile("ld.global.nc.L1::no_allocate.L2::cache_hint.v4.u32 {%0, %1, %2, %3}, [%4], %5;"
               : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "l"(p), "l"(pol));
  return v;
}
__device__ __forceinline__ void st_stream(__nv_bfloat16* p, uint4 v, uint64_t pol) {
  asm volatile("st.global.L2::cache_hint.v4.b32 [%0], {%1, %2, %3, %4}, %5;"
               ::"l"(p), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w), "l"(pol) : "memory");
}

__device__ __forceinline__ double warp_sum_d(double a) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) a += __shfl_xor_sync(0xffffffffu, a, o);
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

__device__ __forceinline__ float pow2f_exact(float n) {   // 2^n for whole n, clamped to the normal float range
  const int i = (int)fminf(fmaxf(n, -126.f), 127.f);
  return __uint_as_float((uint32_t)(127 + i) << 23);
}

constexpr int NST = 4;                  // ring stages: steps of the streamed part in flight per warp
constexpr int KS_RES = KS_MAX - NST;    // resident steps of a warp whose segment does not fit entirely

// 16-byte asynchronous copy global -> shared (through L2 only), grouped per thread
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src, uint64_t pol) {
  asm volatile("cp.async.cg.shared.global.L2::cache_hint [%0], [%1], 16, %2;"
               ::"r"(dst), "l"(__cvta_generic_to_global(src)), "l"(pol) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ uint4 lds128(uint32_t addr) {
  uint4 v;
  asm volatile("ld.shared.v4.u32 {%0, %1, %2, %3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr) : "memory");
  return v;
}

__device__ __forceinline__ void sts128(uint32_t addr, uint32_t w) {
  asm volatile("st.shared.v4.u32 [%0], {%1, %1, %1, %1};" ::"r"(addr), "r"(w) : "memory");
}
constexpr uint32_t FILLER = 0xFF7FFF7Fu;          // two bf16 of the most negative finite value: exp -> 0, difference 0
constexpr uint32_t T_OFF = RW * RES_CHUNKS * 16;  // a teacher slot lies this far behind its student slot

// The streamed part of a warp's segment passes through a ring in shared memory, two steps (a "double
// step": 64 chunks, two per lane) at a time: NSD double steps fill the NST steps of the ring.  Every lane
// owns two 16-byte slots per double stage and array and fills them itself (cp.async, or the filler where
// the row has no chunk for it), so no lane ever reads what another lane wrote: a thread's own wait_group is
// all the synchronisation there is, and the bookkeeping of a ring step (wait, commit, offsets, wrap) is
// paid once per two chunks.  A streamed part is a whole number of double steps (the resident part gives up
// a step where it would not be).  Invariant between passes: the first NSD double steps of the coming
// pass are in flight or landed, one committed group per double step.
constexpr int NSD = NST / 2;
static_assert(NST == 2 * NSD && NSD >= 2, "the ring holds whole double steps");
struct Ring {
  uint32_t base;   // shared-memory address of this lane's first student slot of double stage 0 (a double stage is 1024 bytes on)
  uint32_t slot;   // slot of the next double step to consume
};

// request the first NSD double steps of a row (g_s == nullptr: no row) once everything in flight has landed
__device__ __forceinline__ void ring_prime(Ring& rg, const Seg& sg, int lane, const __nv_bfloat16* g_s,
                                           const __nv_bfloat16* g_t, uint64_t pol) {
  cp_async_wait<0>();
  if (sg.res == sg.steps) return;          // nothing is streamed
  uint32_t slot = rg.slot;
#pragma unroll
  for (int j = 0; j < NSD; ++j) {
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      const int c = sg.c0 + (sg.res + 2 * j + h) * 32 + lane;
      if (g_s != nullptr && c < sg.c1) {
        cp_async16(slot + h * 512, g_s + (size_t)c * 8, pol);
        cp_async16(slot + h * 512 + T_OFF, g_t + (size_t)c * 8, pol);
      } else {
        sts128(slot + h * 512, FILLER);
        sts128(slot + h * 512 + T_OFF, FILLER);
      }
    }
    cp_async_commit();
    slot += 1024;
    if (slot == rg.base + NSD * 1024) slot = rg.base;
  }
}

// Visits this thread's chunks in step order: body(a, b, chunk, valid) with the packed student /
// teacher words of the chunk (the filler where valid is false).  Resident steps are read from shared
// memory; streamed steps come out of the ring, and each double step consumed requests the one NSD further
// on: of this pass, or, past its end, of the next pass, whose rows are wrap_s / wrap_t (the same row
// again, the next row after the last pass, nullptr if nothing follows).
// after_resident() runs once the resident steps are done.
template <typename Body, typename Mid>
__device__ __forceinline__ void for_each_chunk(const Seg& sg, int lane, const uint4* res_s, const uint4* res_t,
                                               const __nv_bfloat16* g_s, const __nv_bfloat16* g_t,
                                               const __nv_bfloat16* wrap_s, const __nv_bfloat16* wrap_t,
                                               uint64_t pol, Ring& rg, Body&& body, Mid&& after_resident) {
  // resident part (slots past the end of the segment hold the filler); kept rolled: the pass bodies
  // are large and must stay in the instruction cache
  int c = sg.c0 + lane;
#pragma unroll 1
  for (int k = 0; k < sg.res; ++k, c += 32) body(res_s[k * 32 + lane], res_t[k * 32 + lane], c, c < sg.c1);
  after_resident();
  const int TD = (sg.steps - sg.res) >> 1;          // streamed double steps: 0 or more than NSD
  if (TD <= 0) return;
  const uint32_t first_off = (uint32_t)c * 16u;
  uint32_t off = first_off + 1024u * NSD;           // byte offset, in either row, of the first chunk of the double step requested next
  uint32_t lim = (uint32_t)sg.c1 * 16u;
  const char* bs = reinterpret_cast<const char*>(g_s);   // (warp-uniform) rows the requests read
  const char* bt = reinterpret_cast<const char*>(g_t);
  uint32_t slot = rg.slot;
  const uint32_t slot_end = rg.base + NSD * 1024;
  int i = 0;
  // all but the last NSD + 1 double steps: the chunks consumed and the chunks requested exist for every lane,
  // and the requests stay inside this pass, so this copy of the loop carries none of the checks below
#pragma unroll 1
  for (; i < TD - NSD - 1; ++i, c += 64) {
    cp_async_wait<NSD - 1>();
    const uint4 a0 = lds128(slot), b0 = lds128(slot + T_OFF);
    const uint4 a1 = lds128(slot + 512), b1 = lds128(slot + 512 + T_OFF);
    cp_async16(slot, bs + off, pol);
    cp_async16(slot + T_OFF, bt + off, pol);
    cp_async16(slot + 512, bs + off + 512, pol);
    cp_async16(slot + 512 + T_OFF, bt + off + 512, pol);
    cp_async_commit();
    off += 1024;
    slot += 1024;
    if (slot == slot_end) slot = rg.base;
    body(a0, b0, c, true);
    body(a1, b1, c + 32, true);
  }
#pragma unroll 1
  for (; i < TD; ++i, c += 64) {
    if (i == TD - NSD) {   // from here on the requests belong to the pass that follows
      off = first_off;
      if (wrap_s != nullptr) { bs = reinterpret_cast<const char*>(wrap_s); bt = reinterpret_cast<const char*>(wrap_t); }
      else lim = 0;
    }
    cp_async_wait<NSD - 1>();
    const uint4 a0 = lds128(slot), b0 = lds128(slot + T_OFF);
    const uint4 a1 = lds128(slot + 512), b1 = lds128(slot + 512 + T_OFF);
#pragma unroll
    for (int h = 0; h < 2; ++h) {
      if (off + h * 512 < lim) {
        cp_async16(slot + h * 512, bs + off + h * 512, pol);
        cp_async16(slot + h * 512 + T_OFF, bt + off + h * 512, pol);
      } else {
        sts128(slot + h * 512, FILLER);
        sts128(slot + h * 512 + T_OFF, FILLER);
      }
    }
    cp_async_commit();
    off += 1024;
    slot += 1024;
    if (slot == slot_end) slot = rg.base;
    body(a0, b0, c, c < sg.c1);
    body(a1, b1, c + 32, c + 32 < sg.c1);
  }
  rg.slot = slot;
}

// Phase clock (only when the call asks for it): thread 0 of every CTA adds the cycles between two marks
// to phase i of a small table in shared memory; at the end of the kernel the table goes to the device
// counters that saki_phase_cycles() reads (sums over CTAs; PH_ROWS counts the rows behind them).
#define RTS(i) do { if (timing && tid == 0) { const long long _n = clock64(); ph[i] += _n - ph[PH_LAST]; ph[PH_LAST] = _n; } } while (0)

// SPEC: the instance that serves block verification (bonus rows, positions handed out as tickets); plain
// routing runs an instance without that code.
template <bool SPEC>
__global__ void __launch_bounds__(RT, CTAS_PER_SM) rowsm_kernel(const RowParams P) {
  extern __shared__ __align__(128) unsigned char smem[];
  const int tid = threadIdx.x, lane = tid & 31;
  const bool spec = SPEC && P.spec != 0;
  const int K1c = SPEC ? P.K1 : 1;             // positions per sequence
  const bool timing = P.phase_cycles != nullptr;
  // how long a thread waits for a row's bulk copy before the block gives up on its rows (the drain at
  // the end of the kernel always takes the full limit: no copy is in flight when a block leaves)
  const long long wait_limit = P.wait_limit > 0 ? P.wait_limit : WAIT_LIMIT_CYCLES;
  long long* ph = (long long*)(smem + ROFF_PH);
  if (timing && tid == 0) {
#pragma unroll 1
    for (int i = 0; i < PH_WORDS; ++i) ph[i] = 0;
    ph[PH_LAST] = clock64();
  }
  const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);   // broadcast: lets the compiler treat it as warp-uniform
  const uint4* res_s = reinterpret_cast<const uint4*>(smem + ROFF_S) + warp * RES_CHUNKS;
  const uint4* res_t = reinterpret_cast<const uint4*>(smem + ROFF_T) + warp * RES_CHUNKS;
  double* red = (double*)(smem + ROFF_RED);
  double* gat = (double*)(smem + ROFF_GAT);
  uint64_t* mbar = (uint64_t*)(smem + ROFF_MBAR);

  const int V = P.V;
  const int n_chunks = V / 8;
  // A row is cut into steps of 32 chunks (256 elements) and the steps are dealt out in order: every warp
  // gets steps_q of them, the first steps_r warps one more.  Whole steps: a segment that ended inside a
  // step would cost its warp a nearly empty step in every pass.
  const int steps_all = (n_chunks + 31) / 32, steps_q = steps_all / RW, steps_r = steps_all - steps_q * RW;
  auto seg_of = [&](int w, Seg& g) {
    g.steps = steps_q + (w < steps_r ? 1 : 0);
    g.c0 = min(n_chunks, 32 * (w * steps_q + min(w, steps_r)));
    g.c1 = min(n_chunks, g.c0 + 32 * g.steps);
  };
  Seg sg;
  seg_of(warp, sg);
  // a segment that does not fit leaves NST steps to the ring, and one more where the streamed part would not be
  // a whole number of double steps
  sg.res = sg.steps <= KS_MAX ? sg.steps : KS_RES - ((sg.steps - KS_RES) & 1);
  const int res_chunks = min(sg.c1 - sg.c0, sg.res * 32);          // resident chunks of this warp
  const uint32_t res_bytes = (uint32_t)res_chunks * 16u;
  Ring rg;
  rg.base = smem_addr(res_s + KS_RES * 32 + lane);
  rg.slot = rg.base;
  // slots of the resident area that no copy ever writes (a segment that ends inside its last step) hold the filler
#pragma unroll 1
  for (int k = res_chunks + lane; k < RES_CHUNKS; k += 32) {
    sts128(smem_addr(res_s + k), FILLER);
    sts128(smem_addr(res_t + k), FILLER);
  }

  const float c32 = (float)(1.4426950408889634 / (double)P.temperature);     // log2(e)/temperature
  Consts K;
  K.tau = (double)P.temperature; K.rtau = 1.0 / K.tau; K.eps = (double)P.eps; K.c64 = (double)c32;
  K.rc64 = 1.0 / K.c64; K.grad_scale = (double)P.grad_scale; K.sqrt_eps = sqrtf(P.eps); K.V = V;
  const uint64_t pol_last = policy_evict_last(), pol_first = policy_evict_first();

  // rows fit 31 bits (see rowsm_can_serve): 32-bit divisions
  auto row_ptrs = [&](int64_t row, const __nv_bfloat16*& s, const __nv_bfloat16*& t) {
    const int64_t b = K1c == 1 ? row : (int64_t)((uint32_t)row / (uint32_t)K1c);
    const int j = (int)(row - b * K1c);
    s = (const __nv_bfloat16*)P.s + b * P.s_seq + (int64_t)j * P.s_pos;
    t = (const __nv_bfloat16*)P.t + b * P.t_seq + (int64_t)j * P.t_pos;
  };
  // lane 0 of each warp: fetch the warp's resident part of `row` into shared memory
  auto issue = [&](const __nv_bfloat16* s, const __nv_bfloat16* t) {
    mbar_expect_tx(mbar, 2u * res_bytes);
    if (res_bytes) {
      bulk_load_hint((void*)res_s, s + (size_t)sg.c0 * 8, res_bytes, mbar, pol_first);
      bulk_load_hint((void*)res_t, t + (size_t)sg.c0 * 8, res_bytes, mbar, pol_first);
    }
  };
  // n per-warp vectors -> gat[k] = sum over warps of component k; warp k adds up component k, so the
  // serial part after the barrier is one shuffle tree deep
  auto combine = [&](const double* v, int n) {
    if (lane == 0) {
#pragma unroll
      for (int k = 0; k < RNV; ++k) if (k < n) red[k * RW + warp] = v[k];
    }
    __syncthreads();
#pragma unroll 1
    for (int k = warp; k < n; k += RW) {
      const double a = warp_sum_d(lane < RW ? red[k * RW + lane] : 0.0);
      if (lane == 0) gat[k] = a;
    }
    __syncthreads();
  };

  // Block verification with early out (Section 3.5 discards what lies behind a sequence's first
  // rejection).  Positions are handed out as tickets from a device counter in position-major order
  // (ticket = position * n_seq + sequence: all first positions, then all second ones, ...).  A row whose
  // draft token is rejected, or that is flagged, records its position in seq_stop[sequence] (atomicMin)
  // as soon as its decision is known; a ticket whose sequence has stopped before its position is passed
  // over.  Nothing waits: a ticket whose predecessor is still undecided is routed anyway (the resolve
  // step discards it if it was not needed).  `seqres`: [0] the row reserved for this CTA's next turn
  // (n_rows: none left), [1], [2] the rest of a ticket range this CTA holds, [3] how many tickets it takes
  // at a time: it aims at one live ticket per range (doubles after a range without one, halves after a
  // range with several), so late positions, where most sequences have stopped, cost few round trips.
  const bool dyn = SPEC && P.seq_next != nullptr;
  const int n_seq = dyn ? (int)(P.n_rows / K1c) : 1;
  const int n_tickets = (int)P.n_rows;
  int* seqres = (int*)(smem + ROFF_SEQ);
  auto ticket_row = [&](int tk) { const int j = tk / n_seq; return (int64_t)(tk - j * n_seq) * K1c + j; };
  auto ticket_live = [&](int tk, int hi) {   // not known to lie behind its sequence's first stop
    if (tk >= hi) return false;
    const int j = tk / n_seq;
    return *(volatile const int*)(P.seq_stop + (tk - j * n_seq)) >= j;
  };
  // warp-wide, all 32 lanes: find this CTA's next row.  Each turn of the loop takes tickets from the
  // device counter or uses up tickets the CTA holds, so it ends without depending on any other CTA.
  auto reserve_next = [&] {
    int blo = seqres[1], bhi = seqres[2], n = seqres[3], res = n_tickets;
    while (res == n_tickets) {
      bool fresh = false;
      if (blo >= bhi) {
        int old = 0;
        if (lane == 0) old = (int)min((unsigned int)n_tickets, gridDim.x + atomicAdd(P.seq_next, (unsigned int)n));
        old = __shfl_sync(0xffffffffu, old, 0);
        blo = old; bhi = min(old + n, n_tickets);
        if (blo >= bhi) break;
        fresh = true;
      }
      const unsigned m = __ballot_sync(0xffffffffu, ticket_live(blo + lane, bhi));   // a range is at most 32 tickets
      if (fresh) n = m == 0 ? min(32, 2 * n) : (__popc(m) > 1 ? max(1, n / 2) : n);
      if (m) { res = blo + __ffs(m) - 1; blo = res + 1; }
      else blo = bhi;
    }
    if (lane == 0) {
      seqres[0] = res < n_tickets ? (int)ticket_row(res) : n_tickets;
      seqres[1] = blo; seqres[2] = bhi; seqres[3] = n;
    }
  };
  if (tid == 0) {
    mbar_init(mbar, RW);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    seqres[0] = n_tickets; seqres[1] = 0; seqres[2] = 0; seqres[3] = 1;
  }
  __syncthreads();
  const __nv_bfloat16 *n_s = nullptr, *n_t = nullptr;   // the rows of the CTA's next position, if any
  const int64_t first_row = dyn ? ticket_row((int)blockIdx.x) : (int64_t)blockIdx.x;   // grid <= n_rows
  if (first_row < P.n_rows) {
    row_ptrs(first_row, n_s, n_t);
    if (lane == 0) issue(n_s, n_t);
    ring_prime(rg, sg, lane, n_s, n_t, pol_last);
  }
  uint32_t phase = 0;
  bool dead = false;
  bool undrained = false;   // this thread gave up on a copy that may still be in flight
  int rb = 0;
  // Pass "final" ends without a barrier.  What is left of a row after it (the total variation, the
  // one-hot entry of the gradient, the residual draw, the outputs) is done one row later by warp
  // FIN_WARP while thread 0 does the next row's scalars: the row's broadcast buffer, the per-warp sums
  // of its last pass and the step weights of the draw stay intact until then.  The last row of the
  // CTA is finished after the loop.  `pb`: the row's buffer parity; all 32 lanes call.
  int64_t pending_row = -1;
  auto finish_row = [&](int64_t prow, int pb) {
    const double* bcp = (const double*)(smem + ROFF_BC) + pb * BC_DOUBLES;
    const double* fin = (const double*)(smem + ROFF_FIN) + pb * 2 * RW;
    const __nv_bfloat16 *ps, *pt;
    row_ptrs(prow, ps, pt);
    const int64_t pseq = K1c == 1 ? prow : (int64_t)((uint32_t)prow / (uint32_t)K1c);
    const int ppos = (int)(prow - pseq * K1c);
    const bool pbonus = spec && (ppos == K1c - 1);
    const int xp = pbonus ? 0 : (spec ? P.proposal[pseq * P.prop_ld + ppos] : P.proposal[prow]);
    const double tv_sum = warp_sum_d(lane < RW ? fin[lane] : 0.0);
    const double tv = (bcp[BC_LAMBDA] > 0.0) ? tv_sum : 0.0;
    const float k0p = (float)bcp[BC_K0];
    const int tok = (int)bcp[BC_TOK];
    if (lane == 0 && P.dlogits && tok >= 0) {   // the supervised token: gradient KG * (p - 1), over the entry its chunk's owner stored
      const float ipf = (float)bcp[BC_IP];
      const float kgf = (float)(bcp[BC_KG] * (double)ipf);
      const float s_tok = (float)(tok == xp ? bcp[BC_SX] : bcp[BC_SV]);
      const float ep = ex2f(fmaf(s_tok, c32, k0p));
      ((__nv_bfloat16*)P.dlogits + prow * P.ld_g)[tok] = __float2bfloat16_rn(fmaf(ep, kgf, -(float)bcp[BC_KG]));
    }
    if (!(pbonus || bcp[BC_CORR] != 0.0)) {
      if (lane == 0) write_result_tv(bcp, P.out, !spec, prow, 0, xp, false, K.c64, ps, pt, tv);
      return;
    }
    // ---- the draw (corrected and bonus rows): the warp that owns the inverse-CDF target, by an
    // ordered scan of the per-warp weights
    const double mine_w = lane < RW ? fin[RW + lane] : 0.0;
    double inc_w = mine_w;
#pragma unroll
    for (int o = 1; o < RW; o <<= 1) {
      const double up = __shfl_up_sync(0xffffffffu, inc_w, o);
      if (lane >= o) inc_w += up;
    }
    const double target = bcp[BC_UDRAW] * __shfl_sync(0xffffffffu, inc_w, RW - 1);
    const unsigned cross = __ballot_sync(0xffffffffu, lane < RW && inc_w > target);
    const unsigned posw = __ballot_sync(0xffffffffu, mine_w > 0.0);
    int owner;
    double running = 0.0;
    bool last_mode = false;
    if (cross) {
      owner = __ffs(cross) - 1;
      running = __shfl_sync(0xffffffffu, inc_w - mine_w, owner);
    } else {       // rounding left no crossing: the last warp with positive weight, its last position
      owner = posw ? 31 - __clz(posw) : 0;
      last_mode = true;
    }
    Seg so;          // the owner's segment
    seg_of(owner, so);
    const float* step_w = (const float*)(smem + ROFF_STEP) + owner * MAX_STEPS;
    const int ns = min(so.steps, MAX_STEPS);
    // the step that holds the target (every lane walks the same few numbers)
    int ks = -1, kpos = -1;
#pragma unroll 1
    for (int k = 0; k < ns; ++k) {
      const double w = (double)step_w[k];
      if (w > 0.0) kpos = k;
      if (!last_mode && running + w > target) { ks = k; break; }
      running += w;
    }
    if (ks < 0) { last_mode = true; ks = max(kpos, 0); }   // rounding: last step with positive weight
    const int c = so.c0 + ks * 32 + lane;
    const bool valid = c < so.c1;
    uint4 s4 = make_uint4(FILLER, FILLER, FILLER, FILLER), t4 = s4;
    if (valid) { s4 = ld_l2(ps + (size_t)c * 8, pol_last); t4 = ld_l2(pt + (size_t)c * 8, pol_last); }
    const uint32_t sw[4] = {s4.x, s4.y, s4.z, s4.w}, tw[4] = {t4.x, t4.y, t4.z, t4.w};
    const float clp = (float)bcp[BC_CL], kqp = (float)bcp[BC_KQ];
    const float rhop = (float)bcp[BC_IP] / (float)bcp[BC_IQ];     // as in pass "final": weights in units of iq
    float w[8];
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      const float2 sf = unpack_bf16x2(sw[i]), tf = unpack_bf16x2(tw[i]);
      const float2 ep = i == 0 ? ex2_fma2(ffma2(sf, splat(c32), splat(k0p))) : ex2f2(ffma2(sf, splat(c32), splat(k0p)));   // as in pass "final"
      const float2 eq = ex2f2(ffma2(tf, splat(clp), ffma2(sf, splat(c32 - clp), splat(kqp))));
      w[2 * i] = pbonus ? eq.x : fmaxf(fmaf(ep.x, -rhop, eq.x), 0.f);
      w[2 * i + 1] = pbonus ? eq.y : fmaxf(fmaf(ep.y, -rhop, eq.y), 0.f);
    }
    double mine = 0.0;
#pragma unroll
    for (int i = 0; i < 8; ++i) mine += (double)w[i];
    double inc = mine;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
      const double up = __shfl_up_sync(0xffffffffu, inc, o);
      if (lane >= o) inc += up;
    }
    const unsigned posm = __ballot_sync(0xffffffffu, mine > 0.0);
    const unsigned hit = last_mode ? 0u : __ballot_sync(0xffffffffu, running + inc > target);
    int y = -1;
    if (hit) {
      int found = -1;
      if (lane == __ffs(hit) - 1) {                   // walk the 8 elements of the crossing chunk
        double run = running + inc - mine;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
          run += (double)w[i];
          if (found < 0 && run > target) found = c * 8 + i;
        }
        if (found < 0) {
#pragma unroll
          for (int i = 0; i < 8; ++i) if (w[i] > 0.f) found = c * 8 + i;
        }
      }
      y = __shfl_sync(0xffffffffu, found, __ffs(hit) - 1);
    } else if (posm) {                                // rounding: last positive element of the step
      int lastp = -1;
      if (lane == 31 - __clz(posm)) {
#pragma unroll
        for (int i = 0; i < 8; ++i) if (w[i] > 0.f) lastp = c * 8 + i;
      }
      y = __shfl_sync(0xffffffffu, lastp, 31 - __clz(posm));
    }
    if (y < 0) y = min(V - 1, max(so.c0 * 8, so.c1 * 8 - 1));
    if (lane == 0) write_result_tv(bcp, P.out, !spec, prow, pbonus ? 0 : 1, y, pbonus, K.c64, ps, pt, tv);
  };

  int64_t next_row_c = P.n_rows;
  for (int64_t row = first_row; row < P.n_rows; row = next_row_c, rb ^= 1) {
    double* bc = (double*)(smem + ROFF_BC) + rb * BC_DOUBLES;   // this row's broadcast scalars
    const uint64_t rid = P.row_offset + (uint64_t)row;
    const int64_t seq = K1c == 1 ? row : (int64_t)((uint32_t)row / (uint32_t)K1c);
    const int pos = (int)(row - seq * K1c);
    const bool bonus = spec && (pos == K1c - 1);
    const int x = bonus ? 0 : (spec ? P.proposal[seq * P.prop_ld + pos] : P.proposal[row]);
    const bool masked = (P.mask != nullptr) && (P.mask[row] == 0);
    const __nv_bfloat16 *g_s = n_s, *g_t = n_t;
    __nv_bfloat16* g_out = P.dlogits ? (__nv_bfloat16*)P.dlogits + row * P.ld_g : nullptr;
    // thread 0, once the row's decision is known: where the CTA goes next when sequences are handed out
    auto plan_next = [&] {
      const int mode = (int)bc[BC_MODE];
      if (!dyn || mode == MODE_SOLVE) return;
      if (!bonus && (mode == MODE_FLAGGED || (mode == MODE_FINAL && bc[BC_CORR] != 0.0)))
        atomicMin(P.seq_stop + seq, pos);        // verification of this sequence ends here
      atomicAdd(P.seq_next + 1, 1u);             // statistic: positions routed
    };
    if (timing && tid == 0) ph[PH_ROWS] += 1;
    RTS(PH_ROW_TOP);
    if (!dead) {
      if (!mbar_wait_bounded(mbar, phase, wait_limit)) { dead = true; undrained = true; }
      else phase ^= 1u;
    }
    RTS(PH_COPY_WAIT);

    // ------------------------------------------------ pass "lse" (no separate maximum pass)
    // The exponent shifts of this pass are fixed before it starts: -ceil(c * m) with m the largest
    // logit among the first 256 of the warp's segment.  m is an element of the row, so no term that
    // matters can underflow; a row whose maximum lies more than ~88 nats above m overflows, shows as
    // a non-finite sum and goes to the float64 kernel.  Shifts are whole numbers, so bringing the
    // warps onto the row's common shifts multiplies their sums by exact powers of two.  The true
    // maxima are tracked on the side (packed bf16 for the student, value + chunk for the teacher).
    {
      float ksw = 1e30f, ktw = 1e30f;            // this warp's shifts (1e30: the warp has no element)
      {
        uint4 fs = make_uint4(FILLER, FILLER, FILLER, FILLER), ft = fs;
        if (sg.c0 + lane < sg.c1) { fs = res_s[lane]; ft = res_t[lane]; }
        const float2 a = unpack_bf16x2(max_bf16x2(max_bf16x2(fs.x, fs.y), max_bf16x2(fs.z, fs.w)));
        const float2 b = unpack_bf16x2(max_bf16x2(max_bf16x2(ft.x, ft.y), max_bf16x2(ft.z, ft.w)));
        const float ms0 = warp_max_f(fmaxf(a.x, a.y)), mt0 = warp_max_f(fmaxf(b.x, b.y));
        if (sg.c0 < sg.c1) {
          ksw = -ceilf(c32 * fmaxf(ms0, -1e30f));
          ktw = -ceilf(c32 * fmaxf(mt0, -1e30f));
        }
      }
      float2 Ss = splat(0.f), St = splat(0.f), M1 = splat(0.f), M2 = splat(0.f), M3 = splat(0.f), M4 = splat(0.f), N1 = splat(0.f);
      uint32_t run_s = FILLER;                   // packed running maxima of the student's even / odd elements
      float mt_run = -CUDART_INF_F;              // running maximum of the teacher, and the first chunk that reached it
      int arg_c = -1;
      const float2 cc = splat(c32), neg1 = splat(-1.f), kk0 = splat(ksw), kk1 = splat(ktw);
      for_each_chunk(sg, lane, res_s, res_t, g_s, g_t, g_s, g_t, pol_last, rg, [&](const uint4& s4, const uint4& t4, int c, bool valid) {
        const uint32_t sw[4] = {s4.x, s4.y, s4.z, s4.w}, tw[4] = {t4.x, t4.y, t4.z, t4.w};
        run_s = max_bf16x2(run_s, max_bf16x2(max_bf16x2(sw[0], sw[1]), max_bf16x2(sw[2], sw[3])));
        const float2 cmt = unpack_bf16x2(max_bf16x2(max_bf16x2(tw[0], tw[1]), max_bf16x2(tw[2], tw[3])));
        const float cm_t = fmaxf(cmt.x, cmt.y);
        if (valid && cm_t > mt_run) { mt_run = cm_t; arg_c = c; }
        // the two sums of exponentials are formed per chunk first and then added to the running sums: a thread's
        // running sum takes one addition per chunk, so a dominant element swamps four times fewer small ones
        float2 cs = splat(0.f), ct = splat(0.f);
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float2 sf = unpack_bf16x2(sw[i]), tf = unpack_bf16x2(tw[i]);
          const float2 d = ffma2(sf, neg1, tf);
          const float2 es = ex2f2(ffma2(sf, cc, kk0));
          const float2 et = ex2f2(ffma2(tf, cc, kk1));
          cs = i == 0 ? es : fadd2(cs, es);
          ct = i == 0 ? et : fadd2(ct, et);
          const float2 d2 = fmul2(d, d);
          M1 = ffma2(es, d, M1);
          const float2 u = fmul2(es, d2);
          M2 = fadd2(M2, u);
          M3 = ffma2(u, d, M3);
          M4 = ffma2(u, d2, M4);
          N1 = ffma2(et, d, N1);
        }
        Ss = fadd2(Ss, cs);
        St = fadd2(St, ct);
      }, [] {});
      RTS(PH_LSE);
      // warp: teacher maximum with the lowest chunk that holds it (a chunk belongs to one thread, so
      // chunk order is index order; the element is found once, by the block's winner), student
      // maximum, sums
      const float2 rs2 = unpack_bf16x2(run_s);
      const float wms = warp_max_f(fmaxf(rs2.x, rs2.y));
      float wmt = mt_run;
      int warg = arg_c >= 0 ? arg_c : 0x7fffffff;
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float om = __shfl_xor_sync(0xffffffffu, wmt, o);
        const int oa = __shfl_xor_sync(0xffffffffu, warg, o);
        if (om > wmt || (om == wmt && oa < warg)) { wmt = om; warg = oa; }
      }
      const float kws = ksw, kwt = ktw;
      auto tot = [](const float2 a) { return (double)a.x + (double)a.y; };
      double v[7] = {tot(Ss), tot(St), tot(M1), tot(M2), tot(M3), tot(N1), tot(M4)};
#pragma unroll
      for (int k = 0; k < 7; ++k) v[k] = warp_sum_d(v[k]);
      if (lane == 0) {
#pragma unroll
        for (int k = 0; k < 7; ++k) red[k * RW + warp] = v[k];
        red[7 * RW + warp] = (double)kws; red[8 * RW + warp] = (double)kwt;
        float* wm = (float*)(smem + ROFF_WMAX);
        wm[warp] = wmt; ((int*)wm)[RW + warp] = warg; wm[2 * RW + warp] = wms;
      }
      // the row scalars that do not depend on the passes
      auto side_work = [&] {
        if (warp == UACC_WARP) bc[BC_UACC] = scalar_uniform(P.seed, rid, STAGE_ACCEPT);
        if (warp == UDRAW_WARP) bc[BC_UDRAW] = scalar_uniform(P.seed, rid, bonus ? STAGE_BONUS : STAGE_RESIDUAL);
        if (warp == SX_WARP) {
          const bool ok = (x >= 0 && x < V);
          bc[BC_SX] = ok ? (double)__bfloat162float(g_s[x]) : 0.0;
          bc[BC_TX] = ok ? (double)__bfloat162float(g_t[x]) : 0.0;
        }
      };
      if (!SIDE_WARPS && lane == 0) side_work();
      const int any_dead = __syncthreads_or(dead ? 1 : 0);
      RTS(PH_LSE_REDUCE);
      if (warp < 8) {   // block level, eight roles dealt round the first eight warps: 0-6 add up one sum each on the row's shifts, 7 finds the argmax
#pragma unroll 1
       for (int role = warp; role < 8; role += RW) {
        const int wl = lane < RW ? lane : 0;       // lanes beyond the warp count carry zero weight
        const float* wm = (const float*)(smem + ROFF_WMAX);
        if (role < 7) {
          // From here on the row's shifts are those of its true maxima (the largest term of each sum has
          // its exponent argument in (-1, 0], where float32 resolves it best); a warp's shift came from an
          // element of the row, so it is never below the row's, and the factor is an exact power of two <= 1.
          const bool teacher = (role == 1 || role == 5);
          const float mx = warp_max_f(lane < RW ? wm[teacher ? wl : 2 * RW + wl] : -CUDART_INF_F);
          const double kr = (double)-ceilf(c32 * fmaxf(mx, -1e30f));
          const double kw = lane < RW ? red[(teacher ? 8 : 7) * RW + wl] : 1e30;
          const double f = kw < 1e29 ? (double)pow2f_exact((float)(kr - kw)) : 0.0;
          const double a = warp_sum_d(f * red[role * RW + wl]);
          if (lane == 0) { gat[role < 6 ? role : 9] = a; if (role < 2) gat[7 + role] = kr; }   // gat[9]: the fourth moment
        } else {
          float gmt = lane < RW ? wm[wl] : -CUDART_INF_F;
          int garg = ((const int*)wm)[RW + wl];
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) {
            const float om = __shfl_xor_sync(0xffffffffu, gmt, o);
            const int oa = __shfl_xor_sync(0xffffffffu, garg, o);
            if (om > gmt || (om == gmt && oa < garg)) { gmt = om; garg = oa; }
          }
          if (lane == 0) {
            int best = -1;                       // lowest index of the maximum inside the winning chunk
            if (garg != 0x7fffffff) {
              const uint4 t4 = ld_l2(g_t + (size_t)garg * 8, pol_last);
              const uint32_t tw[4] = {t4.x, t4.y, t4.z, t4.w};
#pragma unroll
              for (int i = 3; i >= 0; --i) {
                const float2 f2 = unpack_bf16x2(tw[i]);
                if (f2.y == gmt) best = garg * 8 + 2 * i + 1;
                if (f2.x == gmt) best = garg * 8 + 2 * i;
              }
            }
            gat[6] = (double)best;
          }
        }
       }
      } else if (SIDE_WARPS && lane == 0) {
        side_work();                             // meanwhile, on warps that would only wait
      }
      if (any_dead) dead = true;
      __syncthreads();
      RTS(PH_LSE_GATHER);
      if (warp == FIN_WARP && pending_row >= 0) finish_row(pending_row, rb ^ 1);   // meanwhile: the previous row's draw and outputs
      if (dyn && warp == RES_WARP) reserve_next();     // and the CTA's next row (block verification), while thread 0 does the scalars
      pending_row = -1;
      if (tid == SV_WARP * 32) {   // and the student's logit at the teacher's argmax (the supervised token of a corrected row)
        const int vs = (gat[6] >= 0.0 && gat[6] < (double)V) ? (int)gat[6] : 0;
        bc[BC_SV] = (double)__bfloat162float(g_s[vs]);
      }
      if (tid < 2) {   // lane 0: the student's sum, lane 1: the teacher's; then lane 0 alone
        double rS, G;
        lse_of_sum(gat[lane], gat[7 + lane], rS, G);
        const double rSt = __shfl_sync(0x3u, rS, 1), G1 = __shfl_sync(0x3u, G, 1);
        if (tid == 0) {
          bc[BC_K0] = gat[7]; bc[BC_K1] = gat[8];
          scalar_after_lse_tail(bc, gat, K, (float)gat[7], (float)gat[8], x, bonus, masked, any_dead != 0, 1.f, true,
                                rS, rSt, G, G1, gat + 9);
          plan_next();
        }
      }
      RTS(PH_LSE_SCALAR);
      __syncthreads();
    }
    const float k0 = (float)bc[BC_K0], k1 = (float)bc[BC_K1];   // the row's shifts: exponent arguments <= 0

    // ------------------------------------------------ pass "solve" (repeated)
    while ((int)bc[BC_MODE] == MODE_SOLVE) {
      RTS(PH_SOLVE_TOP);
      const float cb = (float)bc[BC_CB], kb = (float)bc[BC_KB];
      float2 S0 = splat(0.f), S1 = splat(0.f), S2 = splat(0.f), S3 = splat(0.f), S4 = splat(0.f);
      const float2 cc = splat(c32), cbb = splat(cb), kbb = splat(kb), neg1 = splat(-1.f);
      for_each_chunk(sg, lane, res_s, res_t, g_s, g_t, g_s, g_t, pol_last, rg, [&](const uint4& s4, const uint4& t4, int, bool) {
        const uint32_t sw[4] = {s4.x, s4.y, s4.z, s4.w}, tw[4] = {t4.x, t4.y, t4.z, t4.w};
        float2 c0 = splat(0.f), c1 = splat(0.f);       // the chunk's share of S0 and S1 (see pass "lse")
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float2 sf = unpack_bf16x2(sw[i]), tf = unpack_bf16x2(tw[i]);
          const float2 d = ffma2(sf, neg1, tf);
          const float2 e = ex2f2(ffma2(d, cbb, ffma2(sf, cc, kbb)));
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
      }, [] {});
      RTS(PH_SOLVE);
      auto tot = [](const float2 a) { return (double)a.x + (double)a.y; };
      const double v[5] = {warp_sum_d(tot(S0)), warp_sum_d(tot(S1)), warp_sum_d(tot(S2)), warp_sum_d(tot(S3)),
                           warp_sum_d(tot(S4))};
      combine(v, 5);
      RTS(PH_SOLVE_COMBINE);
      if (tid == 0) {
        scalar_after_solve4(bc, gat, K, k0, k1, x, bonus, masked);
        plan_next();
        atomicAdd(P.redo_count + 3, 1u);         // statistic: evaluation passes
      }
      RTS(PH_SOLVE_SCALAR);
      __syncthreads();
    }
    const int64_t next_row = dyn ? (int64_t)seqres[0] : row + gridDim.x;
    next_row_c = next_row;
    n_s = nullptr; n_t = nullptr;
    if (next_row < P.n_rows) row_ptrs(next_row, n_s, n_t);

    // ------------------------------------------------ flagged row: zero outputs, zero gradient
    if ((int)bc[BC_MODE] == MODE_FLAGGED || (int)bc[BC_MODE] == MODE_REDO) {
      const bool redo = (int)bc[BC_MODE] == MODE_REDO;   // ill-conditioned for float32: the float64 kernel routes it
      if (tid == 0) {
        if (redo) {
          const unsigned int slot = atomicAdd(P.redo_count, 1u);
          P.redo_list[slot] = (int32_t)row;
          if (P.redo_guess) P.redo_guess[slot] = (float)bc[BC_BETA];     // where the float64 kernel starts its iteration
        }
        else {
          write_row(P.out, row, zero_row((uint32_t)bc[BC_STATUS]), !spec);
          atomicAdd(P.flagged, 1ull);
        }
      }
      if (g_out && !redo) {
#pragma unroll 1
        for (int k = 0; k < sg.steps; ++k) {
          const int c = sg.c0 + k * 32 + lane;
          if (c < sg.c1) st_stream(g_out + (size_t)c * 8, make_uint4(0, 0, 0, 0), pol_first);
        }
      }
      __syncwarp();
      if (lane == 0 && !dead && next_row < P.n_rows) {
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        issue(n_s, n_t);
      }
      ring_prime(rg, sg, lane, n_s, n_t, pol_last);   // the ring holds steps of this row: refill it for the next
      continue;
    }

    // ------------------------------------------------ pass "final"
    RTS(PH_FINAL_TOP);
    const bool need_draw = bonus || bc[BC_CORR] != 0.0;
    const float cl = (float)bc[BC_CL], kq = (float)bc[BC_KQ];
    const float iq = (float)bc[BC_IQ], ip = (float)bc[BC_IP];
    const float kg = (float)(bc[BC_KG] * (double)ip);     // gradient entry = e_p * kg
    const float rho = ip / iq;                            // q_i - p_i = iq * (e_q - rho * e_p)
    {
      const bool want_g = (g_out != nullptr);
      float2 R = splat(0.f);
      const float2 cc = splat(c32), cll = splat(cl), kqq = splat(kq), kk0 = splat(k0);
      const float2 nrho = splat(-rho), kgg = splat(kg);
      const float2 ccl = splat(c32 - cl);               // exact: the scalar step rounds cl so that (c - cl) + cl = c in float32
      float* step_w = (float*)(smem + ROFF_STEP) + warp * MAX_STEPS;   // draw weight of each of this warp's steps
      for_each_chunk(sg, lane, res_s, res_t, g_s, g_t, n_s, n_t, pol_last, rg, [&](const uint4& s4, const uint4& t4, int c, bool valid) {
        const uint32_t sw[4] = {s4.x, s4.y, s4.z, s4.w}, tw[4] = {t4.x, t4.y, t4.z, t4.w};
        uint32_t gp[4];
        float2 sqc = splat(0.f), rc = splat(0.f);       // this chunk's share of Sq and R
#pragma unroll
        for (int i = 0; i < 4; ++i) {
          const float2 sf = unpack_bf16x2(sw[i]), tf = unpack_bf16x2(tw[i]);
          // (one of the chunk's eight exponential pairs goes to the FMA pipe: this pass is bound by the
          // special-function pipe, and one pair is what the issue slots have room for)
          const float2 ep = i == 0 ? ex2_fma2(ffma2(sf, cc, kk0)) : ex2f2(ffma2(sf, cc, kk0));
          const float2 eq = ex2f2(ffma2(tf, cll, ffma2(sf, ccl, kqq)));     // c s + cl (t - s) as (c - cl) s + cl t: no difference to form

          sqc = fadd2(sqc, eq);
          float2 r = ffma2(ep, nrho, eq);                // (q_i - p_i) / iq
          r.x = fmaxf(r.x, 0.f); r.y = fmaxf(r.y, 0.f);
          rc = fadd2(rc, r);
          const float2 gv = fmul2(ep, kgg);
          gp[i] = pack_bf16x2(gv.x, gv.y);
        }
        R = fadd2(R, rc);
        if (need_draw) {   // ordered bookkeeping for the inverse-CDF draw: the weight of this step of the warp
          float wsum = bonus ? (sqc.x + sqc.y) : (rc.x + rc.y);   // in units of iq, like every draw weight
#pragma unroll
          for (int o = 16; o > 0; o >>= 1) wsum += __shfl_xor_sync(0xffffffffu, wsum, o);
          const int k = (c - sg.c0) >> 5;
          if (lane == 0 && k < MAX_STEPS) step_w[k] = wsum;
        }
        if (want_g && valid) st_stream(g_out + (size_t)c * 8, make_uint4(gp[0], gp[1], gp[2], gp[3]), pol_first);
      }, [&] {
        // the warp has read its resident part for the last time: the next row's may land there
        __syncwarp();
        if (lane == 0 && !dead && next_row < P.n_rows) {
          asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
          issue(n_s, n_t);
        }
      });
      RTS(PH_FINAL);
      // no barrier: each warp leaves its share of the total variation and its draw weight (its step
      // weights, in order) for finish_row
      double part = 0.0;
      if (need_draw) {
        __syncwarp();
        const int ns = min(sg.steps, MAX_STEPS);
        static_assert(MAX_STEPS <= 64, "two step weights per lane");
        part = warp_sum_d((lane < ns ? (double)step_w[lane] : 0.0) + (lane + 32 < ns ? (double)step_w[lane + 32] : 0.0));
      }
      const double v1 = warp_sum_d((double)(R.x + R.y) * (double)iq);
      if (lane == 0) {
        double* fin = (double*)(smem + ROFF_FIN) + rb * 2 * RW;
        fin[warp] = v1; fin[RW + warp] = part;
      }
      pending_row = row;
    }
    RTS(PH_ROW_END);
    // no barrier here: the next row uses the other broadcast buffer, and every other shared area is
    // rewritten only after the next row's first block barrier
  }

  cp_async_wait<0>();
  __syncthreads();
  if (warp == FIN_WARP && pending_row >= 0) finish_row(pending_row, rb ^ 1);
  // a CTA that gave up on a copy still waits (bounded) for what it has in flight before leaving
  if (undrained && tid == 0) (void)mbar_wait_bounded(mbar, phase);
  if (timing && tid == 0) {
    RTS(PH_TAIL);
#pragma unroll 1
    for (int i = 0; i < PH_LAST; ++i) atomicAdd(P.phase_cycles + i, (unsigned long long)ph[i]);
  }
}

// ---------------------------------------------------------------- host side
cudaError_t launch(const RowParams& p, cudaStream_t st, int* n_launches, bool* served) {
  *served = false;
  if (p.n_rows <= 0) { *served = true; return cudaSuccess; }
  static std::mutex mu;
  static int cached_dev = -1, cached_sms = 0;
  int dev = 0;
  cudaGetDevice(&dev);
  {
    std::lock_guard<std::mutex> lock(mu);
    if (cached_dev != dev) {
      cudaError_t e = cudaFuncSetAttribute(rowsm_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, RSMEM_BYTES);
      if (e != cudaSuccess) return e;
      e = cudaFuncSetAttribute(rowsm_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, RSMEM_BYTES);
      if (e != cudaSuccess) return e;
      e = cudaDeviceGetAttribute(&cached_sms, cudaDevAttrMultiProcessorCount, dev);
      if (e != cudaSuccess) return e;
      cached_dev = dev;
    }
  }
  const int64_t ctas = (int64_t)cached_sms * CTAS_PER_SM;
  const int grid = (int)(p.n_rows < ctas ? p.n_rows : ctas);
  if (p.spec) rowsm_kernel<true><<<grid, RT, RSMEM_BYTES, st>>>(p);
  else rowsm_kernel<false><<<grid, RT, RSMEM_BYTES, st>>>(p);
  cudaError_t e = cudaGetLastError();
  if (e == cudaSuccess) { *served = true; if (n_launches) *n_launches += 1; }
  return e;
}

// largest V the variant takes (its draw bookkeeping holds MAX_STEPS steps per warp)
int max_v() { return MAX_STEPS * 32 * 8 * RW; }

}  // namespace SAKI_ROWSM_NS
}  // namespace saki
