// placeholder until the tensor-core path lands
#include "pbt_common.cuh"
namespace pbt {
bool gemm_tc_supported(const GemmArgs&) { return false; }
cudaError_t launch_gemm_tc(const GemmArgs&, Counters*, cudaStream_t) { return cudaErrorNotSupported; }
}
