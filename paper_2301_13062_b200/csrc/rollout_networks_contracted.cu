// The rollout kernels of the MLP policies in the contracted arithmetic (fused multiply-adds in
// the dynamics, five-instruction tanh): an optional variant, selected per call.
#include "rollout_kernel.cuh"

namespace cp {

cudaError_t launch_rollout_networks_contracted(RolloutParams &p, int policy, int mode, int shape, cudaStream_t s) {
    return launch_networks_arith<true>(p, policy, mode, shape, s);
}

}  // namespace cp
