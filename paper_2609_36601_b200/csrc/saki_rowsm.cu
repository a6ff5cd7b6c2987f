// Row-per-SM kernel, the variant with one CTA of 512 threads per SM, and the choice between the three
// variants (the implementation is saki_rowsm_impl.cuh).
#include "saki_rowsm_impl.cuh"

namespace saki {

// Rows up to this length go to the variant with two CTAs of 256 threads per SM: their passes are short
// against the serial phases between them (block reductions, float64 scalars), and a second CTA on the
// SM runs its passes meanwhile.  Longer rows stay with one CTA per SM: with two rows in flight per SM
// the streamed parts of all rows no longer stay in L2 between the passes.  Measured (fwd+bwd, M rows/s,
// one / two CTAs per SM): V = 8192 15.9 / 25.3, 32000 9.9 / 12.7, 65536 6.5 / 7.5, 81920 5.6 / 6.3,
// 100000 4.85 / 5.06, 131072 3.95 / 3.76.
constexpr int HALF_MAX_V = 98304;
// Shorter rows still go to the variant with four CTAs of 128 threads per SM: more of the SM's rows are in a
// pass at any time.  Measured (M rows/s, two / four CTAs per SM): V = 4096 29.7 / 44.4, 8192 26.0 / 35.0,
// 16384 19.6 / 21.7, 32000 13.1 / 14.3, 49152 9.8 / 10.0, 65536 7.8 / 7.5.
constexpr int QUARTER_MAX_V = 49152;

bool rowsm_can_serve(const RowParams& p, int dtype) {
  if (dtype != SAKI_BF16) return false;
  if (p.V < 2048 || p.V % 8 != 0 || p.V > full_sm::max_v()) return false;
  if (p.n_rows > 0x7fffffffLL) return false;     // row numbers are kept in 32 bits (redo list, divisions)
  auto al16 = [](const void* q) { return ((uintptr_t)q & 15) == 0; };
  if (!al16(p.s) || !al16(p.t)) return false;
  if (p.s_seq % 8 || p.s_pos % 8 || p.t_seq % 8 || p.t_pos % 8) return false;
  if (p.dlogits && (!al16(p.dlogits) || p.ld_g % 8)) return false;
  return true;
}

cudaError_t launch_rowsm(const RowParams& p, cudaStream_t st, int* n_launches, bool* served) {
  if (p.V <= QUARTER_MAX_V && p.V <= quarter_sm::max_v()) return quarter_sm::launch(p, st, n_launches, served);
  if (p.V <= HALF_MAX_V && p.V <= half_sm::max_v()) return half_sm::launch(p, st, n_launches, served);
  return full_sm::launch(p, st, n_launches, served);
}

}  // namespace saki
