// Tensor-core (tcgen05 / TMEM / TMA) chunkwise path.  Placeholder until the kernel lands.
#include "common.cuh"
namespace gdn {
cudaError_t launch_tcgen05(const Problem&, const Sched&, cudaStream_t, int*) { return cudaErrorNotSupported; }
}
