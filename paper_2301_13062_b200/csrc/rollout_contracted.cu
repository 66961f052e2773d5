// The rollout kernels in the contracted arithmetic (fused multiply-adds, reciprocal constants;
// see euler_step_contracted): an optional variant, selected per call, never the default.
#include "rollout_kernel.cuh"

namespace cp {

cudaError_t launch_rollout_contracted(RolloutParams &p, int policy, bool streams, cudaStream_t s) {
    return launch_rollout_arith<true>(p, policy, streams, s);
}

}  // namespace cp
