// The deferred-restart rollout kernel (rollout_deferred.cuh) for the 4-32-2 and the 4-16-16-2
// network (the 4-64-2 one is in a file of its own: build time).
#include "rollout_deferred.cuh"

namespace cp {

cudaError_t launch_rollout_deferred_mlp64(RolloutParams &p, bool contracted, cudaStream_t s);

// p.w holds every weight twice (launch_rollout_deferred has paired them).
cudaError_t launch_rollout_deferred_wide(RolloutParams &p, int policy, bool contracted, cudaStream_t s) {
    switch (policy) {
        case 4: return launch_limit<4, false>(p, 3, contracted, s);
        case 7: return launch_limit<7, false>(p, 3, contracted, s);
        default: return launch_rollout_deferred_mlp64(p, contracted, s);
    }
}

}  // namespace cp
