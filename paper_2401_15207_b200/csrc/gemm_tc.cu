#include "gemm_tc.h"

namespace hift {
int gemm_tc_init() { return 1; }
bool gemm_tc_eligible(const GemmArgs&) { return false; }
cudaError_t gemm_tc_launch(cudaStream_t, const GemmArgs&) { return cudaErrorNotSupported; }
}  // namespace hift
