// placeholder until the tensor-core GEMM lands
#include "dm_internal.h"
namespace dm {
bool gemm_tcgen05_supports(const GemmArgs &) { return false; }
cudaError_t gemm_tcgen05(const GemmArgs &, cudaStream_t) { return cudaErrorNotSupported; }
}
