// Row-per-SM kernel, the variant with two CTAs of 256 threads per SM (the implementation is
// saki_rowsm_impl.cuh).
#define SAKI_ROWSM_HALF 1
#include "saki_rowsm_impl.cuh"
