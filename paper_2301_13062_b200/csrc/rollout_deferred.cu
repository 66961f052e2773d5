// The deferred-restart rollout kernel (rollout_deferred.cuh) for hashed actions, the linear
// policies and the 4-16-2 network, and the entry that picks the instance for a call; the wider
// and deeper networks are instantiated in rollout_deferred_networks.cu and
// rollout_deferred_mlp64.cu (build time).
#include "rollout_deferred.cuh"

namespace cp {

bool rollout_deferred_applies(const RolloutParams &p, int policy, bool streams) {
    // per-step outputs: none, or exactly the reward plane + done bitmask
    const bool outputs_ok = !streams || (p.reward_stream && p.done_bits && !p.action_bits && !p.trajectory);
    if (!outputs_ok || p.action_bits_in || p.start_in) return false;
    if (is_wide_network(policy)) return !streams && !p.max_steps;
    return policy == 0 || policy == 1 || policy == 2 || policy == 6;
}

cudaError_t launch_rollout_deferred(RolloutParams &p, int policy, bool contracted, cudaStream_t s) {
    // measured on 1,048,576 x 500 at K = 3 / 4 / 6 / 8: hashed actions (22-step episodes) 0.996 /
    // 0.987 / 0.965 / 0.987 ms, the linear policy (80-step episodes) 0.945 / 0.924 / 0.907 / 0.908 ms
    // The 4-16-2 network of config 5 ends its episodes after 9-10 steps, so waiting costs more and
    // a restart pass less (next to a 600-instruction trip): 16,777,216 x 200 takes 38.4 / 38.0 /
    // 41.5 ms at K = 2 / 3 / 4 (the general kernel: 43.2 ms).
    // Short launches (chunked rollouts of a batch in place) pay the ragged end on every call, so
    // the passes come closer together (us per step of 1,048,576 envs at K = 2 / 4 / 6, hashed
    // actions: T = 16: 3.39 / 3.65 / 4.03, T = 64: 2.41 / 2.38 / 2.45, T = 256: 2.17 / 2.02 / 2.00;
    // below 12 steps the general kernel is as fast or faster and keeps the call).
    // The shared linear policy's 80-step episodes leave a pass little to do, so long launches
    // space them further (with the reward plane and done bits, K = 4 / 6 / 8: 1,048,576 x 500
    // 1.076 / 1.041 / 1.027 ms, 4,194,304 x 1,000 8.45 / 8.12 / 7.97 ms; without them 4,194,304 x
    // 1,000 7.05 / 7.01 ms at K = 6 / 8; at 200 steps K = 6 is ahead, and so it is at every length
    // with hashed actions: 4,194,304 x 1,000 with streams 9.11 / 8.57 / 8.90 ms).
    const int by_length = p.T < 48u ? 2 : p.T < 192u ? 4 : (policy == 1 && p.T >= 384u) ? 8 : 6;
    const int k = g_tuning.rollout_defer > 0 ? g_tuning.rollout_defer : (is_network(policy) ? 3 : by_length);
    // the action hash folds the time's upper half into the lower one: nothing to do below 2^16
    const bool short_times = (uint64_t)p.t0 + p.T <= 65536u;
    if (policy == 1 || is_network(policy)) {  // every shared weight twice: one packed operand for both slots
        const int count = policy == 1 ? 10 : policy == 2 ? 114 : policy == 4 ? 226 : policy == 5 ? 450 : 386;
        static_assert(sizeof(p.w) >= 2 * 450 * sizeof(float), "the launch parameters hold the largest policy twice");
        for (int i = count - 1; i >= 0; --i) p.w[2 * i] = p.w[2 * i + 1] = p.w[i];
    }
    switch (policy) {
        case 0: return short_times ? launch_limit<0, true>(p, k, contracted, s) : launch_limit<0, false>(p, k, contracted, s);
        case 1: return launch_limit<1, false>(p, k, contracted, s);
        case 2: return launch_limit<2, false>(p, k, contracted, s);
        case 6: return launch_limit<6, false>(p, k, contracted, s);
        default: return launch_rollout_deferred_wide(p, policy, contracted, s);  // 4, 5, 7: weights already paired
    }
}

}  // namespace cp
