// Fused multi-step rollout: one launch runs all T steps (paper Sec. V-D, loop
// unrolling, taken to its limit, and the single-kernel CUDA comparison of
// Sec. V-G). Each environment's state, hash keys and episode counters stay in
// registers for the whole time loop; HBM sees 8 bytes per environment in total
// unless per-step streams are requested.
//
// Work decomposition: a "warp task" is 32*EPT consecutive environments; lane l
// owns environments base + j*32 + l (j < EPT), so that per-step stream stores
// are one contiguous 128-byte line per j and a done/action bitmask word is one
// warp ballot. By default every warp gets exactly one task and the hardware
// hands out CTAs as others retire; a persistent grid looping over tasks is
// available for tuning.
//
// The kernel has no shared memory, no inter-warp synchronisation and no waits.
//
// This header holds the kernel template and its dispatch; rollout_kernel.cu instantiates it
// for the canonical (one rounding per op) arithmetic, rollout_contracted.cu for the
// contracted arithmetic, so that the two sets of kernels compile side by side.
#pragma once
#include "cartpole_device.cuh"
#include "cartpole_internal.h"

namespace cp {

// POLICY: 0 hashed random action, 1 linear, 2 MLP with 16 hidden units, 3 action bits supplied by
// the caller, 4 / 5 MLP with 32 / 64 hidden units, 6 one linear policy per environment (its ten
// parameters are loaded into registers before the time loop; handled in the kernel body).
template <int POLICY>
__device__ __forceinline__ uint32_t policy_signbit(const RolloutParams &p, const Keys &ka, uint32_t t,
                                                   const State &z) {
    if (POLICY == 0) {
        return action_signbit(ka, t);
    } else if (POLICY == 1) {
        return linear_action(*reinterpret_cast<const LinearW *>(p.w), z);
    } else if (POLICY == 2) {
        return mlp_action<16>(*reinterpret_cast<const MlpWT<16> *>(p.w), z);
    } else if (POLICY == 4) {
        return mlp_action<32>(*reinterpret_cast<const MlpWT<32> *>(p.w), z);
    } else {
        return mlp_action<64>(*reinterpret_cast<const MlpWT<64> *>(p.w), z);
    }
}

#ifndef CP_ROLLOUT_MIN_CTAS
#define CP_ROLLOUT_MIN_CTAS 1
#endif
#ifndef CP_CONTRACT_MIN_CTAS
#define CP_CONTRACT_MIN_CTAS 1
#endif

// STREAMS: 0 no per-step output; 1 exactly the reward plane and the done bitmask (no run-time
// tests in the loop); 2 any combination, tested per step.
// LIMIT: episodes are cut off after p.max_steps steps.
// CONTRACT: the contracted arithmetic of euler_step_contracted instead of the canonical order.
template <int POLICY, int EPT, int STREAMS, bool LIMIT, bool CONTRACT>
__global__ void __launch_bounds__(256, CONTRACT ? CP_CONTRACT_MIN_CTAS : CP_ROLLOUT_MIN_CTAS)
    rollout_kernel(const __grid_constant__ RolloutParams p) {
    const uint32_t lane = threadIdx.x & 31u;
    const int64_t warps_total = (int64_t)gridDim.x * (blockDim.x >> 5);
    const int64_t words = (p.n + 31) >> 5;
    unsigned long long tot_ret = 0, tot_cnt = 0;

    for (int64_t task = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); task < p.n_tasks;
         task += warps_total) {
        const int64_t base = task * (32 * EPT);
        State z[EPT];
        Keys ka[EPT], kr[EPT];
        LinearW own[POLICY == 6 ? EPT : 1];  // per-environment policies live in registers
        // Episode bookkeeping: every step earns reward 1, so the returns of the episodes completed
        // in this launch add up to (time of the last termination) - (time the first of them began),
        // and only the count and the start time of the running episode need to live in the loop.
        // begin[j]: global time at which env j's running episode began (before t0 if steps were
        // carried in; unsigned wrap-around is harmless, only differences are used).
        uint32_t cnt[EPT], begin[EPT];
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
            if (POLICY == 6) {  // parameter q of env i at env_weights[q*n + i]: coalesced per plane
                LinearW &o = own[POLICY == 6 ? j : 0];
#pragma unroll
                for (int q = 0; q < 8; ++q) o.w[q / 4][q % 4] = p.env_weights[(int64_t)q * p.n + idx[j]];
                o.b[0] = p.env_weights[8 * p.n + idx[j]];
                o.b[1] = p.env_weights[9 * p.n + idx[j]];
            }
            cnt[j] = 0u;
            // Only the step limit needs the carried-in length inside the loop; without it the
            // counter is read once, at the end (loading it here costs four registers in the loop
            // and 6 % of the stream variant's speed).
            begin[j] = p.t0 - ((LIMIT && p.ep_len_io) ? p.ep_len_io[idx[j]] : 0u);
        }

        // Per-step stream outputs advance by one row per step: keep running pointers / offsets
        // instead of recomputing row * width + column with 64-bit multiplies every step.
        float *rew_ptr[EPT];
        uint32_t *done_ptr[EPT];
        const uint32_t *act_ptr[EPT];
        int64_t env_off[EPT], word_off[EPT];  // into [T][n] planes and [T][words] bit planes
        bool word_ok[EPT];
#pragma unroll
        for (int j = 0; j < EPT; ++j) {
            env_off[j] = idx[j];
            word_off[j] = task * EPT + j;
            const bool in_range = word_off[j] < words;
            word_ok[j] = lane == 0 && in_range;
            rew_ptr[j] = STREAMS == 1 ? p.reward_stream + idx[j] : nullptr;
            done_ptr[j] = STREAMS == 1 ? p.done_bits + (word_ok[j] ? word_off[j] : 0) : nullptr;
            act_ptr[j] = POLICY == 3 ? p.action_bits_in + (in_range ? word_off[j] : 0) : nullptr;
        }
        const bool want_done = STREAMS == 2 && p.done_bits, want_act = STREAMS == 2 && p.action_bits;
        const bool want_rew = STREAMS == 2 && p.reward_stream, want_traj = STREAMS == 2 && p.trajectory;

        const uint32_t t_end = p.t0 + p.T;
        for (uint32_t t = p.t0; t != t_end; ++t) {
#pragma unroll
            for (int j = 0; j < EPT; ++j) {
                uint32_t sb;
                if (POLICY == 3) {
                    sb = (__ldg(act_ptr[j]) << (31u - lane)) & 0x80000000u;  // one word per warp, broadcast
                    act_ptr[j] += words;
                } else if (POLICY == 6) {
                    sb = linear_action(own[POLICY == 6 ? j : 0], z[j]);
                } else {
                    sb = policy_signbit<POLICY>(p, ka[j], t, z[j]);
                }
                bool done = CONTRACT ? euler_step_contracted(z[j], force_from_signbit(sb))
                                     : euler_step(z[j], force_from_signbit(sb));
                if (LIMIT) done |= (t + 1u - begin[j]) >= p.max_steps;
                if (done) {
                    cnt[j] += 1u;
                    begin[j] = t + 1u;
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
            // sum of the returns of the completed episodes = last termination time - time the first began
            const uint32_t carried = p.ep_len_io ? p.ep_len_io[idx[j]] : 0u;
            const uint32_t first_begin = p.t0 - carried;
            const uint32_t ret = cnt[j] ? begin[j] - first_begin : 0u;
            // begin[j] still holds t0 (LIMIT: t0 - carried) if no episode ended in this launch
            const uint32_t running = t_end - begin[j] + ((!LIMIT && cnt[j] == 0u) ? carried : 0u);
            if (p.ep_return_sum) p.ep_return_sum[idx[j]] = (float)ret;
            if (p.ep_count) p.ep_count[idx[j]] = cnt[j];
            if (p.ep_len_io) p.ep_len_io[idx[j]] = running;
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

template <int POLICY, int EPT, int STREAMS, bool LIMIT, bool CONTRACT>
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
    rollout_kernel<POLICY, EPT, STREAMS, LIMIT, CONTRACT><<<(unsigned)grid, block, 0, s>>>(p);
    count_launch();
    return cudaGetLastError();
}

template <int POLICY, int STREAMS, bool LIMIT, bool CONTRACT>
cudaError_t launch_ept(RolloutParams &p, int ept, cudaStream_t s) {
    return ept == 1 ? launch_one<POLICY, 1, STREAMS, LIMIT, CONTRACT>(p, s)
                    : launch_one<POLICY, 2, STREAMS, LIMIT, CONTRACT>(p, s);
}

template <int POLICY, int STREAMS, bool CONTRACT>
cudaError_t launch_limit(RolloutParams &p, int ept, cudaStream_t s) {
    return p.max_steps ? launch_ept<POLICY, STREAMS, true, CONTRACT>(p, ept, s)
                       : launch_ept<POLICY, STREAMS, false, CONTRACT>(p, ept, s);
}

template <int POLICY, bool CONTRACT>
cudaError_t launch_mode(RolloutParams &p, int mode, int ept, cudaStream_t s) {
    switch (mode) {
        case 0: return launch_limit<POLICY, 0, CONTRACT>(p, ept, s);
        case 1: return launch_limit<POLICY, 1, CONTRACT>(p, ept, s);
        default: return launch_limit<POLICY, 2, CONTRACT>(p, ept, s);
    }
}

template <bool CONTRACT>
cudaError_t launch_rollout_arith(RolloutParams &p, int policy, bool streams, cudaStream_t s) {
    int ept = g_tuning.rollout_ept;
    if (ept == 0) {
        // Two envs per thread (two independent dependency chains) unless the batch is so small
        // that spreading it over twice as many warps matters more. The MLP policies carry enough
        // independent work per env (H hidden units) to fill the pipes with one env per thread,
        // and a second one only costs registers: measured 1.5 % (canonical) and 20 % (contracted,
        // where the compiler interleaves the two networks at 180+ registers) slower with two.
        const bool mlp = policy == 2 || policy == 4 || policy == 5;
        ept = (mlp && !p.action_bits_in) || (p.n + 63) / 64 < (int64_t)sm_count() * 16 ? 1 : 2;
    }
    // 0: no per-step output; 1: reward plane + done bitmask only; 2: any other combination
    const int mode = !streams ? 0 : (p.reward_stream && p.done_bits && !p.action_bits && !p.trajectory) ? 1 : 2;
    if (p.action_bits_in) policy = 3;
    switch (policy) {
        case 0: return launch_mode<0, CONTRACT>(p, mode, ept, s);
        case 1: return launch_mode<1, CONTRACT>(p, mode, ept, s);
        case 2: return launch_mode<2, CONTRACT>(p, mode, ept, s);
        case 3: return launch_mode<3, CONTRACT>(p, mode, ept, s);
        case 4: return launch_mode<4, CONTRACT>(p, mode, ept, s);
        case 5: return launch_mode<5, CONTRACT>(p, mode, ept, s);
        default: return launch_mode<6, CONTRACT>(p, mode, ept, s);
    }
}

}  // namespace

}  // namespace cp
