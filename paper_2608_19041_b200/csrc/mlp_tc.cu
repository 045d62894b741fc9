// Tensor-core GEMM for the MLP layers (tcgen05 / TMEM / TMA, 3xTF32 split).
#include "mlp_gemm.h"

namespace umd {

bool gemm_tc_supported(const GemmArgs&) { return false; }
cudaError_t launch_gemm_tc(const GemmArgs&, cudaStream_t) { return cudaErrorNotSupported; }

}  // namespace umd
