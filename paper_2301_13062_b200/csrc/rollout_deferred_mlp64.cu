// The deferred-restart rollout kernel (rollout_deferred.cuh) for the 4-64-2 network.
#include "rollout_deferred.cuh"

namespace cp {

cudaError_t launch_rollout_deferred_mlp64(RolloutParams &p, bool contracted, cudaStream_t s) {
    return launch_limit<5, false>(p, 3, contracted, s);
}

}  // namespace cp
