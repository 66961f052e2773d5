// The rollout kernels of the MLP policies (16 / 32 / 64 hidden units, two hidden layers) in the
// canonical arithmetic. A translation unit of its own so that the kernel families compile in
// parallel.
#include "rollout_kernel.cuh"

namespace cp {

cudaError_t launch_rollout_networks(RolloutParams &p, int policy, int mode, int shape, cudaStream_t s) {
    return launch_networks_arith<false>(p, policy, mode, shape, s);
}

}  // namespace cp
