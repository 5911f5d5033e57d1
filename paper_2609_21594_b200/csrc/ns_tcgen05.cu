// Tensor-core Newton-Schulz engine (placeholder translation unit: filled in by the tcgen05 kernels).
#include "internal.h"

namespace muon {
bool tc_supported(const GemmArgs&) { return false; }
int launch_gemm_tc(muon_ctx*, const GemmArgs&, cudaStream_t) { return MUON_ERR_UNSUPPORTED; }
}  // namespace muon
