// The rollout kernels in the canonical arithmetic (every operation rounded once, in the order
// of the per-op ladder), and the entry the C ABI calls.
#include "rollout_kernel.cuh"

namespace cp {

cudaError_t launch_rollout(RolloutParams &p, int policy, bool streams, bool contracted, cudaStream_t s) {
    // The deferred-restart kernel (rollout_deferred.cu) by default: from one 64-env warp per
    // scheduler on (37,888 envs on 148 SMs) for hashed actions and the linear policies, from seven
    // warps per SM on (66,304 envs) for the tanh networks, launches of at least a dozen steps,
    // per-step outputs none or reward plane + done bits. Measured at T = 500, this kernel against
    // the kernels below: hashed actions 37,888 envs 0.093 / 0.096 ms, 65,536 0.098 / 0.142,
    // 131,072 0.163 / 0.251; linear policy 47,360 0.088 / 0.100, 131,072 0.154 / 0.212; network
    // 56,832 0.483 / 0.427, 75,776 0.483 / 0.545. rollout_coop = 5 forces it wherever it
    // applies, any other forced shape keeps the other kernels.
    const int64_t warps64 = (p.n + 63) / 64;
    const bool network = policy == 2 || policy == 4 || policy == 5 || policy == 7;
    const bool enough = network ? warps64 >= (int64_t)sm_count() * 7 : warps64 >= (int64_t)sm_count() * 4;
    const bool by_default = g_tuning.rollout_coop == 0 && g_tuning.rollout_ept == 0 && enough && p.T >= 12u &&
                            (policy == 0 || policy == 1 || policy == 6 || network);
    if ((by_default || g_tuning.rollout_coop == 5) && rollout_deferred_applies(p, policy, streams))
        return launch_rollout_deferred(p, policy, contracted, s);
    // very small batches with hashed actions: a helper warp per stepping warp (rollout_assisted.cu)
    if (rollout_assisted_applies(p, policy, streams)) return launch_rollout_assisted(p, contracted, s);
    if (contracted) return launch_rollout_contracted(p, policy, streams, s);
    return launch_rollout_arith<false>(p, policy, streams, s);
}

}  // namespace cp
