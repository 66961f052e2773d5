// The rollout kernels in the canonical arithmetic (every operation rounded once, in the order
// of the per-op ladder), and the entry the C ABI calls.
#include "rollout_kernel.cuh"

namespace cp {

cudaError_t launch_rollout(RolloutParams &p, int policy, bool streams, bool contracted, cudaStream_t s) {
    // very small batches with hashed actions: a helper warp per stepping warp (rollout_assisted.cu)
    if (rollout_assisted_applies(p, policy, streams)) return launch_rollout_assisted(p, contracted, s);
    // batches that fill the chip, at least a dozen steps; hashed actions, a linear policy or the 4-16-2
    // network; per-step outputs none or reward plane + done bits:
    // restarts deferred to every few trips (rollout_deferred.cu); rollout_coop = 5 forces it
    // wherever it applies, any other forced shape keeps the general kernel
    const bool fills_chip = (p.n + 63) / 64 >= (int64_t)sm_count() * 16;
    const bool by_default = g_tuning.rollout_coop == 0 && g_tuning.rollout_ept == 0 && fills_chip && p.T >= 12u &&
                            (policy == 0 || policy == 1 || policy == 2 || policy == 6);
    if ((by_default || g_tuning.rollout_coop == 5) && rollout_deferred_applies(p, policy, streams))
        return launch_rollout_deferred(p, policy, contracted, s);
    if (contracted) return launch_rollout_contracted(p, policy, streams, s);
    return launch_rollout_arith<false>(p, policy, streams, s);
}

}  // namespace cp
