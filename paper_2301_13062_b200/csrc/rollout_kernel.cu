// Fused multi-step rollout: one launch runs all T steps (paper Sec. V-D, loop
// unrolling, taken to its limit, and the single-kernel CUDA comparison of
// Sec. V-G). Each environment's state, hash keys and episode counters stay in
// registers for the whole time loop; HBM sees 8 bytes per environment in total
// unless per-step streams are requested.
//
// Work decomposition: a "warp task" is 32*EPT consecutive environments; lane l
// owns environments base + j*32 + l (j < EPT), so that per-step stream stores
// are one contiguous 128-byte line per j and a done/action bitmask word is one
// warp ballot. Tasks are dealt round-robin to the resident warps (persistent
// grid, sized from the occupancy calculator times the SM count).
//
// The kernel has no shared memory, no inter-warp synchronisation and no waits.
#include "cartpole_device.cuh"
#include "cartpole_internal.h"

namespace cp {

template <int POLICY>
__device__ __forceinline__ uint32_t policy_signbit(const RolloutParams &p, const Keys &ka, uint32_t t,
                                                   const State &z) {
    if (POLICY == 0) {
        return action_signbit(ka, t);
    } else if (POLICY == 1) {
        return linear_action(*reinterpret_cast<const LinearW *>(p.w), z);
    } else {
        return mlp_action(*reinterpret_cast<const MlpW *>(p.w), z);
    }
}

#ifndef CP_ROLLOUT_MIN_CTAS
#define CP_ROLLOUT_MIN_CTAS 1
#endif

template <int POLICY, int EPT, int STREAMS>
__global__ void __launch_bounds__(256, CP_ROLLOUT_MIN_CTAS) rollout_kernel(const __grid_constant__ RolloutParams p) {
    const uint32_t lane = threadIdx.x & 31u;
    const int64_t warps_total = (int64_t)gridDim.x * (blockDim.x >> 5);
    const int64_t words = (p.n + 31) >> 5;
    unsigned long long tot_ret = 0, tot_cnt = 0;

    for (int64_t task = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); task < p.n_tasks;
         task += warps_total) {
        const int64_t base = task * (32 * EPT);
        State z[EPT];
        Keys ka[EPT], kr[EPT];
        // Episode bookkeeping: every step earns reward 1, so the returns of the episodes completed
        // in this launch add up to (steps carried in) + (time of the last termination), and only
        // the count and the time of the last termination need to live in the loop.
        uint32_t cnt[EPT], last[EPT];  // last: global time just after the last done (t0 = none yet)
        int64_t idx[EPT];
        bool valid[EPT];
#pragma unroll
        for (int j = 0; j < EPT; ++j) {
            idx[j] = base + j * 32 + lane;
            valid[j] = idx[j] < p.n;
            if (!valid[j]) idx[j] = p.n - 1;  // idle lanes shadow the last environment and store nothing
            const uint32_t env = p.env_offset + (uint32_t)idx[j];
            if (POLICY == 0) ka[j] = make_keys(p.salt_a, env);
            kr[j] = make_keys(p.salt_r, env);
            if (p.init_planes) {
                z[j].x = p.init_planes[idx[j]];
                z[j].xd = p.init_planes[p.init_stride + idx[j]];
                z[j].th = p.init_planes[2 * p.init_stride + idx[j]];
                z[j].thd = p.init_planes[3 * p.init_stride + idx[j]];
            } else {
                z[j] = start_state(kr[j], p.t0);
            }
            cnt[j] = 0u;
            last[j] = p.t0;
        }

        // Per-step stream outputs advance by one row per step: keep running pointers / offsets
        // instead of recomputing row * width + column with 64-bit multiplies every step.
        // STREAMS == 1: exactly the reward plane and the done bitmask are written (no run-time
        // tests in the loop); STREAMS == 2: any combination, tested per step.
        float *rew_ptr[EPT];
        uint32_t *done_ptr[EPT];
        int64_t env_off[EPT], word_off[EPT];  // into [T][n] planes and [T][words] bit planes
        bool word_ok[EPT];
#pragma unroll
        for (int j = 0; j < EPT; ++j) {
            env_off[j] = idx[j];
            word_off[j] = task * EPT + j;
            word_ok[j] = lane == 0 && word_off[j] < words;
            rew_ptr[j] = STREAMS == 1 ? p.reward_stream + idx[j] : nullptr;
            done_ptr[j] = STREAMS == 1 ? p.done_bits + (word_ok[j] ? word_off[j] : 0) : nullptr;
        }
        const bool want_done = STREAMS == 2 && p.done_bits, want_act = STREAMS == 2 && p.action_bits;
        const bool want_rew = STREAMS == 2 && p.reward_stream, want_traj = STREAMS == 2 && p.trajectory;

        const uint32_t t_end = p.t0 + p.T;
        for (uint32_t t = p.t0; t != t_end; ++t) {
#pragma unroll
            for (int j = 0; j < EPT; ++j) {
                const uint32_t sb = policy_signbit<POLICY>(p, ka[j], t, z[j]);
                const bool done = euler_step(z[j], force_from_signbit(sb));
                if (done) {
                    cnt[j] += 1u;
                    last[j] = t + 1u;
                    z[j] = start_state(kr[j], t + 1u);
                }
                if (STREAMS == 1) {
                    const uint32_t m = __ballot_sync(0xffffffffu, done && valid[j]);
                    if (word_ok[j]) *done_ptr[j] = m;
                    if (valid[j]) *rew_ptr[j] = 1.0f;
                    done_ptr[j] += words;
                    rew_ptr[j] += p.n;
                }
                if (STREAMS == 2) {
                    if (want_done) {
                        const uint32_t m = __ballot_sync(0xffffffffu, done && valid[j]);
                        if (word_ok[j]) p.done_bits[word_off[j]] = m;
                    }
                    if (want_act) {
                        const uint32_t m = __ballot_sync(0xffffffffu, (sb != 0u) && valid[j]);
                        if (word_ok[j]) p.action_bits[word_off[j]] = m;
                    }
                    if (valid[j]) {
                        if (want_rew) p.reward_stream[env_off[j]] = 1.0f;
                        if (want_traj) {
                            float *tr = p.trajectory + 4 * env_off[j] - 3 * idx[j];  // row 4k, column idx
                            tr[0] = z[j].x;
                            tr[p.n] = z[j].xd;
                            tr[2 * p.n] = z[j].th;
                            tr[3 * p.n] = z[j].thd;
                        }
                    }
                    env_off[j] += p.n;
                    word_off[j] += words;
                }
            }
        }

#pragma unroll
        for (int j = 0; j < EPT; ++j) {
            if (!valid[j]) continue;
            const uint32_t carried = p.ep_len_io ? p.ep_len_io[idx[j]] : 0u;
            const bool any = last[j] != p.t0;
            const uint32_t ret = any ? carried + (last[j] - p.t0) : 0u;
            if (p.ep_return_sum) p.ep_return_sum[idx[j]] = (float)ret;
            if (p.ep_count) p.ep_count[idx[j]] = cnt[j];
            if (p.ep_len_io) p.ep_len_io[idx[j]] = any ? t_end - last[j] : carried + p.T;
            if (p.out_planes) {
                p.out_planes[idx[j]] = z[j].x;
                p.out_planes[p.out_stride + idx[j]] = z[j].xd;
                p.out_planes[2 * p.out_stride + idx[j]] = z[j].th;
                p.out_planes[3 * p.out_stride + idx[j]] = z[j].thd;
            }
            tot_ret += ret;
            tot_cnt += cnt[j];
        }
    }

    if (p.totals) {
        for (int o = 16; o > 0; o >>= 1) {
            tot_ret += __shfl_down_sync(0xffffffffu, tot_ret, o);
            tot_cnt += __shfl_down_sync(0xffffffffu, tot_cnt, o);
        }
        if (lane == 0 && (tot_ret | tot_cnt)) {
            atomicAdd(p.totals, tot_ret);
            atomicAdd(p.totals + 1, tot_cnt);
        }
    }
}

namespace {

template <int POLICY, int EPT, int STREAMS>
cudaError_t launch_one(RolloutParams &p, cudaStream_t s) {
    const int block = g_tuning.rollout_block;
    p.n_tasks = (p.n + 32 * EPT - 1) / (32 * EPT);
    // Default: one task per warp, CTAs handed out by the hardware scheduler as others retire.
    // All tasks take the same time, so a persistent grid would run ceil(tasks / resident warps)
    // full rounds, whereas here the last, partly filled round runs with fewer warps per SM
    // and therefore faster (the kernel is issue-bound, not latency-bound): measured 7-10 %
    // quicker at 1,048,576 envs. A positive rollout_ctas_per_sm selects the persistent form.
    const int per_sm = g_tuning.rollout_ctas_per_sm;
    const int wpb = block / 32;
    int64_t grid = (p.n_tasks + wpb - 1) / wpb;
    if (per_sm > 0) {
        const int64_t resident = (int64_t)per_sm * sm_count();
        if (grid > resident) grid = resident;
    }
    if (grid > 0x7fffffffLL) grid = 0x7fffffffLL;
    rollout_kernel<POLICY, EPT, STREAMS><<<(unsigned)grid, block, 0, s>>>(p);
    count_launch();
    return cudaGetLastError();
}

template <int POLICY, int STREAMS>
cudaError_t launch_ept(RolloutParams &p, int ept, cudaStream_t s) {
    switch (ept) {
        case 1: return launch_one<POLICY, 1, STREAMS>(p, s);
        case 2: return launch_one<POLICY, 2, STREAMS>(p, s);
        default: return launch_one<POLICY, 4, STREAMS>(p, s);
    }
}

}  // namespace

cudaError_t launch_rollout(RolloutParams &p, int policy, bool streams, cudaStream_t s) {
    int ept = g_tuning.rollout_ept;
    if (ept == 0) ept = 2;
    // Small batches: spread environments over as many warps as possible.
    while (ept > 1 && (p.n + 32 * ept - 1) / (32 * ept) < (int64_t)sm_count() * 16) ept >>= 1;
    // 0: no per-step output; 1: reward plane + done bitmask only; 2: any other combination
    const int mode = !streams ? 0 : (p.reward_stream && p.done_bits && !p.action_bits && !p.trajectory) ? 1 : 2;
    switch (policy * 3 + mode) {
        case 0: return launch_ept<0, 0>(p, ept, s);
        case 1: return launch_ept<0, 1>(p, ept, s);
        case 2: return launch_ept<0, 2>(p, ept, s);
        case 3: return launch_ept<1, 0>(p, ept, s);
        case 4: return launch_ept<1, 1>(p, ept, s);
        case 5: return launch_ept<1, 2>(p, ept, s);
        case 6: return launch_ept<2, 0>(p, ept, s);
        case 7: return launch_ept<2, 1>(p, ept, s);
        default: return launch_ept<2, 2>(p, ept, s);
    }
}

}  // namespace cp
