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
// Warps never talk to each other and nothing waits on memory written by another warp; the
// only synchronisation is __syncwarp() around a warp's own 192 bytes of shared memory in the
// cooperative restart.
//
// Where a thread owns two environments (SHAPE 2) and the arithmetic is the canonical one, both
// are stepped by the packed float32 instructions of sm_100a (euler_step_pair). Batches that fill
// the chip mostly go to the deferred-restart kernel of rollout_deferred.cu instead; this
// kernel keeps every call that one does not cover (action bit stream or trajectory written,
// supplied actions or start states, the wider and deeper networks, very short launches, batches
// too small to fill the chip) and is the form the others are compared with bit for bit.
//
// This header holds the kernel template and its dispatch; rollout_kernel.cu and
// rollout_networks.cu instantiate it for the canonical (one rounding per op) arithmetic,
// rollout_contracted.cu and rollout_networks_contracted.cu for the contracted arithmetic (the
// *_networks files hold the MLP policies), so that the kernel families compile side by side.
#pragma once
#include "cartpole_device.cuh"
#include "cartpole_internal.h"

namespace cp {

// POLICY: 0 hashed random action, 1 linear, 2 MLP with 16 hidden units, 3 action bits supplied by
// the caller, 4 / 5 MLP with 32 / 64 hidden units, 6 one linear policy per environment (its ten
// parameters are loaded into registers before the time loop; handled in the kernel body), 7 MLP
// with two hidden layers of 16 units.
template <int POLICY, bool CONTRACT>
__device__ __forceinline__ uint32_t policy_signbit(const RolloutParams &p, const FoldedKeys &ka,
                                                   uint32_t folded_t, const State &z) {
    if (POLICY == 0) {
        return action_signbit_folded(ka, folded_t);
    } else if (POLICY == 1) {
        return linear_action(*reinterpret_cast<const LinearW *>(p.w), z);
    } else if (POLICY == 2) {
        return mlp_action<16, CONTRACT>(*reinterpret_cast<const MlpWT<16> *>(p.w), z);
    } else if (POLICY == 4) {
        return mlp_action<32, CONTRACT>(*reinterpret_cast<const MlpWT<32> *>(p.w), z);
    } else if (POLICY == 7) {
        return mlp_deep_action<CONTRACT>(*reinterpret_cast<const MlpDeepW *>(p.w), z);
    } else {
        return mlp_action<64, CONTRACT>(*reinterpret_cast<const MlpWT<64> *>(p.w), z);
    }
}

constexpr int kMaxWarpsPerCta = 8;  // __launch_bounds__(256)

// SHAPE: how a warp holds and restarts its environments.
//   0: one env per thread, each lane restarts its own env (shortest dependency chain per step:
//      for batches too small to fill the chip, where a step's latency is what is paid);
//   1: one env per thread, restarts done by the whole warp (see below);
//   2: two envs per thread (two independent dependency chains), restarts by the whole warp;
//   3: as 0, but every lane computes the next start state every step, ahead of the dynamics,
//      and a finished env just takes it (instantiated for the hashed and the supplied actions,
//      whose episodes are short: for at most two warps per scheduler the four hashes fill
//      issue slots the dynamics' dependency chain leaves empty, which is quicker than a restart
//      branch on 77 % of the steps; with more warps, or rare restarts, it is wasted issue);
//   4: as 0, with the start states read from the caller's array instead of hashed (a shape of
//      its own because even a never-taken run-time test in the restart path cost shape 0
//      4-6 %).
// STREAMS: 0 no per-step output; 1 exactly the reward plane and the done bitmask (no run-time
// tests in the loop); 2 any combination, tested per step.
// LIMIT: episodes are cut off after p.max_steps steps.
// CONTRACT: the contracted arithmetic of euler_step_contracted instead of the canonical order.
template <int POLICY, int SHAPE, int STREAMS, bool LIMIT, bool CONTRACT>
__global__ void __launch_bounds__(256, 1) rollout_kernel(const __grid_constant__ RolloutParams p) {
    constexpr int EPT = SHAPE == 2 ? 2 : 1;
    constexpr bool COOP = SHAPE == 1 || SHAPE == 2;
    constexpr bool AHEAD = SHAPE == 3;
    constexpr bool START_IN = SHAPE == 4;
    constexpr bool PAIR = SHAPE == 2 && !CONTRACT;  // packed two-env arithmetic
    const uint32_t lane = threadIdx.x & 31u;
    // Per warp: key pairs of up to 8 finished envs, and their 8 x 4 start-state components.
    __shared__ uint2 s_keys[COOP ? kMaxWarpsPerCta : 1][8];
    __shared__ __align__(16) float s_out[COOP ? kMaxWarpsPerCta : 1][32];
    uint2 *const keys_w = s_keys[COOP ? threadIdx.x >> 5 : 0];
    float *const out_w = s_out[COOP ? threadIdx.x >> 5 : 0];
    const uint32_t lane_lt = (1u << lane) - 1u;
    if (COOP) {
        if (lane < 8u) keys_w[lane] = make_uint2(0u, 0u);
        __syncwarp();
    }
    const int64_t warps_total = (int64_t)gridDim.x * (blockDim.x >> 5);
    const int64_t words = (p.n + 31) >> 5;
    unsigned long long tot_ret = 0, tot_cnt = 0;

    for (int64_t task = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); task < p.n_tasks;
         task += warps_total) {
        const int64_t base = task * (32 * EPT);
        State z[EPT];
        FoldedKeys ka[EPT], kr[EPT];  // action and restart streams (see fold16)
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
            if (POLICY == 0) ka[j] = fold_keys(make_keys(p.salt_a, env));
            kr[j] = fold_keys(make_keys(p.salt_r, env));
            if (p.init_planes) {
                z[j].x = p.init_planes[idx[j]];
                z[j].xd = p.init_planes[p.init_stride + idx[j]];
                z[j].th = p.init_planes[2 * p.init_stride + idx[j]];
                z[j].thd = p.init_planes[3 * p.init_stride + idx[j]];
            } else {
                z[j] = start_state_folded(kr[j], fold16(4u * p.t0));
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
        uint32_t vmask[EPT];  // lanes of slot j that own a real environment
#pragma unroll
        for (int j = 0; j < EPT; ++j) {
            env_off[j] = idx[j];
            word_off[j] = task * EPT + j;
            const bool in_range = word_off[j] < words;
            word_ok[j] = lane == 0 && in_range;
            // STREAMS == 1 keeps ONE running pointer per stream: slot j's element lies a constant
            // 32 floats / 1 word behind slot 0's (never dereferenced where the slot has no env)
            rew_ptr[j] = STREAMS == 1 ? p.reward_stream + (base + lane) : nullptr;
            done_ptr[j] = STREAMS == 1 ? p.done_bits + task * EPT : nullptr;
            act_ptr[j] = POLICY == 3 ? p.action_bits_in + (in_range ? word_off[j] : 0) : nullptr;
            vmask[j] = __ballot_sync(0xffffffffu, valid[j]);
        }
        const bool want_done = STREAMS == 2 && p.done_bits, want_act = STREAMS == 2 && p.action_bits;
        const bool want_rew = STREAMS == 2 && p.reward_stream, want_traj = STREAMS == 2 && p.trajectory;

        uint32_t act_word[EPT] = {};
        if (POLICY == 3) {
#pragma unroll
            for (int j = 0; j < EPT; ++j) act_word[j] = __ldg(act_ptr[j]);
        }
        const uint32_t t_end = p.t0 + p.T;
        // Is every angle of this warp within the polynomial range of sine and cosine? After the
        // first step it is: a survivor has |theta| <= 0.2095 and a restarted env |theta| <= 0.05
        // (unless the start states are the caller's data). A warp-uniform flag instead of a
        // per-lane angle test every step: no divergent branch in the loop.
        bool small_mine = true;
#pragma unroll
        for (int j = 0; j < EPT; ++j) small_mine = small_mine && fabsf(z[j].th) <= kSmallAngle;
        bool small_all = __all_sync(0xffffffffu, small_mine);
        // SHAPE 3 runs where only latency is paid: two steps per loop trip give the scheduler a
        // little more to overlap (2,048 x 10,000: 1.30 -> 1.22 ms). The other shapes gain nothing
        // from it or lose (SHAPE 0 at 65,536 envs: 4 % slower; four steps per trip: slower everywhere).
        constexpr int kTimeUnroll = AHEAD ? 2 : 1;
#pragma unroll kTimeUnroll
        for (uint32_t t = p.t0; t < t_end; ++t) {
            const uint32_t t1 = t + 1u;
            const uint32_t folded_t = fold16(t), folded_4t1 = fold16(4u * t1);  // warp-uniform
            bool done[EPT];
            uint32_t sb[EPT];
#pragma unroll
            for (int j = 0; j < EPT; ++j) {
                if (POLICY == 3) {
                    // One word per warp, broadcast; the next step's word is requested now, a whole
                    // step ahead of its use (the warp barriers of the restart keep the compiler
                    // from hoisting the load by itself).
                    sb[j] = (act_word[j] << (31u - lane)) & 0x80000000u;
                    act_ptr[j] += words;
                    if (t1 != t_end) act_word[j] = __ldg(act_ptr[j]);
                } else if (POLICY == 6) {
                    sb[j] = linear_action(own[POLICY == 6 ? j : 0], z[j]);
                } else {
                    sb[j] = policy_signbit<POLICY, CONTRACT>(p, ka[j], folded_t, z[j]);
                }
                // SHAPE 3: the start state of time t+1 depends on the key and the time only, so it
                // is computed here, ahead of the step and whether or not the env finishes. (The
                // empty asm keeps the compiler from sinking the hashes back into the branch.)
                State fresh;
                if (AHEAD) {
                    fresh = start_state_folded(kr[j], folded_4t1);
                    asm volatile("" : "+f"(fresh.x), "+f"(fresh.xd), "+f"(fresh.th), "+f"(fresh.thd));
                }
                if (PAIR && small_all) continue;  // both envs step together below
                const float force = force_from_signbit(sb[j]);
                // warp-uniform; the per-lane shapes and the contracted arithmetic keep the per-lane
                // test (measured faster there: 2,048 x 10,000 loses 6 % with the flag)
                if (COOP && !CONTRACT && small_all)
                    done[j] = CONTRACT ? euler_step_contracted<true>(z[j], force) : euler_step<true>(z[j], force);
                else
                    done[j] = CONTRACT ? euler_step_contracted<false>(z[j], force) : euler_step<false>(z[j], force);
                if (LIMIT) done[j] |= (t1 - begin[j]) >= p.max_steps;
                if (!COOP && done[j]) {
                    cnt[j] += 1u;
                    begin[j] = t1;
                    if (AHEAD) {
                        z[j] = fresh;
                    } else if (START_IN) {  // start states supplied as data: row (t - t0) of [T][4][n]
                        const float *row = p.start_in + (int64_t)(t - p.t0) * 4 * p.n + idx[j];
                        z[j].x = __ldg(row);
                        z[j].xd = __ldg(row + p.n);
                        z[j].th = __ldg(row + 2 * p.n);
                        z[j].thd = __ldg(row + 3 * p.n);
                    } else {
                        z[j] = start_state_folded(kr[j], folded_4t1);
                    }
                }
            }

            if (PAIR && small_all) {
                // Two envs per thread, canonical arithmetic, every angle in the polynomial range:
                // one packed instruction steps both envs (same operations, same bits).
                StatePair zz = pack_states(z[0], z[EPT - 1]);
                euler_step_pair(zz, pack2(force_from_signbit(sb[0]), force_from_signbit(sb[EPT - 1])), done[0],
                                done[EPT - 1]);
                unpack_states(zz, z[0], z[EPT - 1]);
                if (LIMIT) {
#pragma unroll
                    for (int j = 0; j < EPT; ++j) done[j] |= (t1 - begin[j]) >= p.max_steps;
                }
            }

            // Restart by the whole warp. A start state is four independent hashes of the env's key
            // pair, and with the random policy 1.4 of a warp's 32 envs finish per step: restarting
            // lane by lane issues all four hashes (45 instructions) for the whole warp on 77 % of
            // the steps of each j — a third of all issue slots. Instead the finished lanes post
            // their key pairs to a per-warp list in shared memory (slot j owns entries
            // [j*CAP, (j+1)*CAP), position = rank among the finished lanes of that slot), lane L
            // computes component L%4 of entry L/4 — eight restarts in one pass, one hash per lane —
            // and each finished lane reads its four components back. Same hash, same bits; about
            // 51 instead of 2 x 35 warp instructions per warp-step (measured: 105 -> 94 issue
            // slots per env-step, 1.61 -> 1.45 ms on 1,048,576 x 500).
            uint32_t dmask[EPT] = {};
            if (COOP) {
                uint32_t any = 0u;
#pragma unroll
                for (int j = 0; j < EPT; ++j) {
                    dmask[j] = __ballot_sync(0xffffffffu, done[j]);
                    any |= dmask[j];
                }
                if (any) {  // warp-uniform
                    constexpr uint32_t CAP = 8u / EPT;
                    uint32_t slot[EPT];
                    bool listed[EPT];
#pragma unroll
                    for (int j = 0; j < EPT; ++j) {
                        const uint32_t r = __popc(dmask[j] & lane_lt);
                        slot[j] = j * CAP + r;
                        listed[j] = done[j] && r < CAP;
                        if (done[j]) {
                            cnt[j] += 1u;
                            begin[j] = t1;
                        }
                        if (listed[j]) keys_w[slot[j]] = make_uint2(kr[j].f0, kr[j].k1);
                    }
                    __syncwarp();
                    const uint2 kq = keys_w[lane >> 2];  // unused entries hold stale keys: harmless
                    FoldedKeys k;
                    k.f0 = kq.x;
                    k.k1 = kq.y;
                    out_w[lane] = start_component_folded(k, folded_4t1, lane & 3u);
                    __syncwarp();
#pragma unroll
                    for (int j = 0; j < EPT; ++j) {
                        if (STREAMS == 0) {
                            // A listed lane takes its four components with one predicated 16-byte
                            // load straight into the state registers, written as such: the
                            // compiler's form loads into temporaries and moves them (1,048,576 x
                            // 500: 1.320 -> 1.302 ms; with the reward and done streams this form
                            // costs six registers and 1.4 %, so those instances keep the other).
                            const uint32_t out_addr = (uint32_t)__cvta_generic_to_shared(out_w) + slot[j] * 16u;
                            asm volatile(
                                "{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %4, 0;\n\t"
                                "@p ld.shared.v4.f32 {%0, %1, %2, %3}, [%5];\n\t}"
                                : "+f"(z[j].x), "+f"(z[j].xd), "+f"(z[j].th), "+f"(z[j].thd)
                                : "r"((uint32_t)listed[j]), "r"(out_addr)
                                : "memory");
                        } else if (listed[j]) {
                            const float4 s = reinterpret_cast<const float4 *>(out_w)[slot[j]];
                            z[j].x = s.x;
                            z[j].xd = s.y;
                            z[j].th = s.z;
                            z[j].thd = s.w;
                        }
                    }
                    // More than CAP envs of one slot finished at once (rare): the surplus lanes hash
                    // their own start states. Found by one warp-uniform test of the two masks; a
                    // per-lane test costs a divergent branch per env slot on every pass through
                    // the block (1.301 -> 1.287 ms on 1,048,576 x 500).
                    bool surplus = false;
#pragma unroll
                    for (int j = 0; j < EPT; ++j) surplus = surplus || __popc(dmask[j]) > (int)CAP;
                    if (surplus) {
#pragma unroll
                        for (int j = 0; j < EPT; ++j)
                            if (done[j] && !listed[j]) z[j] = start_state_folded(kr[j], folded_4t1);
                    }
                    // No third barrier: the next write to keys_w follows this step's reads of it by
                    // the second barrier, and the next write to out_w follows the next first barrier.
                }
            }

#pragma unroll
            for (int j = 0; j < EPT; ++j) {
                if (STREAMS == 1) {
                    const uint32_t m = COOP ? (dmask[j] & vmask[j]) : __ballot_sync(0xffffffffu, done[j] && valid[j]);
                    if (word_ok[j]) done_ptr[0][j] = m;
                    if (valid[j]) rew_ptr[0][32 * j] = 1.0f;
                    if (j == EPT - 1) {
                        done_ptr[0] += words;
                        rew_ptr[0] += p.n;
                    }
                }
                if (STREAMS == 2) {
                    if (want_done) {
                        const uint32_t m =
                            COOP ? (dmask[j] & vmask[j]) : __ballot_sync(0xffffffffu, done[j] && valid[j]);
                        if (word_ok[j]) p.done_bits[word_off[j]] = m;
                    }
                    if (want_act) {
                        const uint32_t m = __ballot_sync(0xffffffffu, (sb[j] != 0u) && valid[j]);
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
            small_all = true;  // only read by the warp-restart shapes, which always restart from the hash
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

template <int POLICY, int SHAPE, int STREAMS, bool LIMIT, bool CONTRACT>
cudaError_t launch_one(RolloutParams &p, cudaStream_t s) {
    constexpr int EPT = SHAPE == 2 ? 2 : 1;
    p.n_tasks = (p.n + 32 * EPT - 1) / (32 * EPT);
    // CTA size: 256 threads, except that up to three warps per scheduler are spread in CTAs of
    // four warps, one per scheduler, so that no SM holds two warps on one scheduler while other
    // schedulers idle (2,048 x 10,000: 1.30 ms against 1.49 ms with eight-warp CTAs).
    int block = g_tuning.rollout_block;
    if (block == 0) block = p.n_tasks <= (int64_t)sm_count() * 4 * 3 ? 128 : 256;
    if (block > 32 * kMaxWarpsPerCta) block = 32 * kMaxWarpsPerCta;
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
    rollout_kernel<POLICY, SHAPE, STREAMS, LIMIT, CONTRACT><<<(unsigned)grid, block, 0, s>>>(p);
    count_launch();
    return cudaGetLastError();
}

template <int POLICY, int STREAMS, bool LIMIT, bool CONTRACT>
cudaError_t launch_shape(RolloutParams &p, int shape, cudaStream_t s) {
    if constexpr (POLICY == 0 || POLICY == 3) {
        if (shape == 3) return launch_one<POLICY, 3, STREAMS, LIMIT, CONTRACT>(p, s);
    }
    switch (shape) {
        case 0:
        case 3: return launch_one<POLICY, 0, STREAMS, LIMIT, CONTRACT>(p, s);
        case 1: return launch_one<POLICY, 1, STREAMS, LIMIT, CONTRACT>(p, s);
        case 4: return launch_one<POLICY, 4, STREAMS, LIMIT, CONTRACT>(p, s);
        default: return launch_one<POLICY, 2, STREAMS, LIMIT, CONTRACT>(p, s);
    }
}

template <int POLICY, int STREAMS, bool CONTRACT>
cudaError_t launch_limit(RolloutParams &p, int shape, cudaStream_t s) {
    return p.max_steps ? launch_shape<POLICY, STREAMS, true, CONTRACT>(p, shape, s)
                       : launch_shape<POLICY, STREAMS, false, CONTRACT>(p, shape, s);
}

template <int POLICY, bool CONTRACT>
cudaError_t launch_mode(RolloutParams &p, int mode, int shape, cudaStream_t s) {
    switch (mode) {
        case 0: return launch_limit<POLICY, 0, CONTRACT>(p, shape, s);
        case 1: return launch_limit<POLICY, 1, CONTRACT>(p, shape, s);
        default: return launch_limit<POLICY, 2, CONTRACT>(p, shape, s);
    }
}

template <bool CONTRACT>
cudaError_t launch_rollout_arith(RolloutParams &p, int policy, bool streams, cudaStream_t s) {
    if (p.action_bits_in) policy = 3;
    // A batch too small to give every SM sixteen two-env warps is latency-bound: one env per
    // thread over twice as many warps, and per-lane restarts (the cooperative restart adds two
    // shared-memory round trips to every step's dependency chain: 2,048 envs x 10,000 steps
    // take 1.85 ms with per-lane restarts, 2.14 ms with cooperative ones). Otherwise the kernel
    // is issue-bound and the cooperative restart's fewer instructions win. The MLP policies
    // carry enough independent work per env (H hidden units) to fill the pipes with one env
    // per thread, and a second one only costs registers: measured 1.5 % (canonical) and 20 %
    // (contracted, where the compiler interleaves the two networks at 180+ registers) slower.
    // Per-environment linear policies keep ten weights per env in registers: 89 registers with
    // two envs per thread, 63 with one, which is 8 % faster.
    const bool small = (p.n + 63) / 64 < (int64_t)sm_count() * 16;
    const bool heavy = policy == 2 || policy == 4 || policy == 5 || policy == 6 || policy == 7;
    int ept = g_tuning.rollout_ept;      // 0 auto, 1, 2
    int coop = g_tuning.rollout_coop;    // 0 auto, 1 cooperative, 2 per lane, 3 per lane and ahead
    if (coop == 5) coop = 0;  // the deferred-restart kernel does not cover this call: default shape
    if (ept == 0) ept = (small || heavy || coop >= 2) ? 1 : 2;
    // at most two warps per scheduler and short episodes: start states computed ahead (measured:
    // 2,048 x 10,000 1.49 vs 1.65 ms, 32,768 x 5,000 0.75 vs 0.83 ms; slower from 65,536 envs on,
    // and with the linear policy, whose episodes are long)
    const bool tiny = (p.n + 31) / 32 <= (int64_t)sm_count() * 4 * 2;
    if (coop == 0) coop = (small && ept == 1) ? ((tiny && (policy == 0 || policy == 3)) ? 3 : 2) : 1;
    // two envs per thread are always cooperative; supplied start states are read by the lane that
    // needs them, so they always take the per-lane shape that reads them (4)
    // (coop 4 asks for the producer-assisted kernel of rollout_assisted.cu; a call it does not
    // cover lands here and takes the plain per-lane shape)
    const int shape = p.start_in ? 4 : ept == 2 ? 2 : ((coop == 2 || coop == 4) ? 0 : coop == 3 ? 3 : 1);
    // 0: no per-step output; 1: reward plane + done bitmask only; 2: any other combination
    const int mode = !streams ? 0 : (p.reward_stream && p.done_bits && !p.action_bits && !p.trajectory) ? 1 : 2;
    // the network policies are instantiated in translation units of their own (build time)
    if (policy == 2 || policy == 4 || policy == 5 || policy == 7)
        return CONTRACT ? launch_rollout_networks_contracted(p, policy, mode, shape, s)
                        : launch_rollout_networks(p, policy, mode, shape, s);
    switch (policy) {
        case 0: return launch_mode<0, CONTRACT>(p, mode, shape, s);
        case 1: return launch_mode<1, CONTRACT>(p, mode, shape, s);
        case 3: return launch_mode<3, CONTRACT>(p, mode, shape, s);
        default: return launch_mode<6, CONTRACT>(p, mode, shape, s);
    }
}

template <bool CONTRACT>
cudaError_t launch_networks_arith(RolloutParams &p, int policy, int mode, int shape, cudaStream_t s) {
    switch (policy) {
        case 2: return launch_mode<2, CONTRACT>(p, mode, shape, s);
        case 4: return launch_mode<4, CONTRACT>(p, mode, shape, s);
        case 5: return launch_mode<5, CONTRACT>(p, mode, shape, s);
        default: return launch_mode<7, CONTRACT>(p, mode, shape, s);
    }
}

}  // namespace

}  // namespace cp
