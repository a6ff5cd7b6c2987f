// Register-resident cluster kernel (placeholder until the kernel lands).
#include "saki_common.cuh"
namespace saki {
bool cluster_can_serve(const RowParams&, int) { return false; }
cudaError_t launch_cluster(const RowParams&, cudaStream_t, int*, bool* served) { *served = false; return cudaSuccess; }
}
