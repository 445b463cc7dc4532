// bf16 tensor-core rollout (tcgen05 / TMEM).  Placeholder until the kernel lands: reports the
// path as not compiled so that create() answers MAVA_ERR_UNSUPPORTED for MAVA_PRECISION_BF16.
#include "common.cuh"

namespace mava {
bool tc_supported(const mava_config_t &) { return false; }
size_t tc_weight_bytes(const mava_config_t &, int) { return 16; }
cudaError_t launch_prep_tc(mava_rollout *, const float *) { return cudaErrorNotSupported; }
cudaError_t launch_rollout_tc(mava_rollout *, const RolloutArgs &) { return cudaErrorNotSupported; }
}  // namespace mava
