// Row-per-SM kernel, the variant with four CTAs of 128 threads per SM (the implementation is
// saki_rowsm_impl.cuh).
#define SAKI_ROWSM_QUARTER 1
#include "saki_rowsm_impl.cuh"
