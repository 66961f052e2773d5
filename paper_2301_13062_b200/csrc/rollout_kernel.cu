// The rollout kernels in the canonical arithmetic (every operation rounded once, in the order
// of the per-op ladder), and the entry the C ABI calls.
#include "rollout_kernel.cuh"

namespace cp {

cudaError_t launch_rollout(RolloutParams &p, int policy, bool streams, bool contracted, cudaStream_t s) {
    // very small batches with hashed actions: a helper warp per stepping warp (rollout_assisted.cu)
    if (rollout_assisted_applies(p, policy, streams)) return launch_rollout_assisted(p, contracted, s);
    if (contracted) return launch_rollout_contracted(p, policy, streams, s);
    return launch_rollout_arith<false>(p, policy, streams, s);
}

}  // namespace cp
