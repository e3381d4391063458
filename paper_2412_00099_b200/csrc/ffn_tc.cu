#include "ffn_tc.cuh"

namespace mcce {
bool tc_applicable(const mcce_config&) { return false; }
int tc_plan(const mcce_config&, const void*, const void*, const void*, const void*, const void*, const void*, void*,
            void*, TcPlan*) { return MCCE_EINVAL; }
cudaError_t tc_launch_up(TcPlan&, const FfnParams&, uint32_t*, cudaStream_t) { return cudaErrorNotSupported; }
cudaError_t tc_launch_down(TcPlan&, const FfnParams&, uint32_t*, cudaStream_t) { return cudaErrorNotSupported; }
}  // namespace mcce
