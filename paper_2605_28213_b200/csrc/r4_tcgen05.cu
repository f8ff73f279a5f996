#include "common.cuh"
namespace klin {
cudaError_t launch_r4_tcgen05(const GemmArgs&, RunContext&, cudaStream_t, int*) { return cudaErrorNotSupported; }
}
