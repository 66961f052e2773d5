// Rollout for batches far too small to fill the chip (the paper's own shape, 2,048 environments
// x 10,000 steps, Sec. V-A, is 64 warps on 592 warp schedulers): there a step's LATENCY is what
// is paid, and every instruction the stepping warp does not have to issue shortens it.
//
// Everything random in a rollout depends on (seed, env, time) only, never on the trajectory. So
// each stepping warp ("consumer") gets a helper warp ("producer") on another scheduler of the
// same SM that hashes, a chunk of steps ahead, the action force and the start state of every
// step for the consumer's 32 environments into shared memory. The consumer's step is then two
// shared-memory loads, the dynamics, the termination test and four selects: about 60 instead
// of 110 instructions, with no integer hashing in its dependency chain. Same hashes, same
// dynamics function, same bits as the general kernel.
//
// Synchronisation: one hardware barrier per consumer/producer pair (bar.sync with the pair's own
// id, 64 threads), once per chunk, double-buffered. Both warps of a pair execute exactly
// 1 + ceil(T / kChunk) barriers, a number fixed by the launch parameters alone; there is no flag,
// no spin and no dependence on data, so neither warp can wait for an arrival that does not come.
//
// Scope: hashed or supplied actions (the producer turns the caller's action words into forces),
// hashed start states, either arithmetic, with or without an episode step limit and per-step
// output streams. Calls with a feedback policy or supplied start states take the general kernel.
#include "cartpole_device.cuh"
#include "cartpole_internal.h"

namespace cp {

namespace {

// Steps per hand-over: 40 KB of static shared memory per CTA either way (640 bytes per step, two
// buffers). Measured on 2,048 x 10,000: 8 steps 0.543 ms, 16 steps 0.512 ms.
template <int PAIRS>
constexpr int kChunkOf = PAIRS == 1 ? 32 : 16;

// Steps per trip of the consumer's loop over a chunk. Measured on 2,048 x 10,000 (ms per launch):
// 1: 0.666, 2: 0.481, 3: 0.487, 4: 0.503, 8: 0.504, 16: 0.506, whole chunk: 0.506.
constexpr int kStepUnroll = 2;

template <int CHUNK>
struct PairBuffers {
    float4 start[2][CHUNK][32];  // start state of time t + 1, for the env of each lane
    float force[2][CHUNK][32];   // +-F of the action at time t
};

// Barrier 1 for pair 0, barrier 2 for pair 1 (immediates: a register id makes the kernel claim
// all sixteen barriers).
template <int PAIRS>
__device__ __forceinline__ void pair_barrier(uint32_t pair) {
    __syncwarp();
    if (PAIRS == 1 || pair == 0u)
        asm volatile("bar.sync 1, 64;" ::: "memory");
    else
        asm volatile("bar.sync 2, 64;" ::: "memory");
}

// Where the consumer's per-step outputs go (only read when STREAMS): offsets into the [T][n]
// planes and the [T][words] bit planes advance by one row per step.
struct StreamCursor {
    int64_t env_off, word_off, idx, words;
    bool valid, want_done, want_act, want_rew, want_traj;
};

template <bool KNOWN_SMALL, bool LIMIT, bool CONTRACT, int STREAMS, int CHUNK>
__device__ __forceinline__ void consume_step(const RolloutParams &p, const PairBuffers<CHUNK> &buf, uint32_t b,
                                             int s, uint32_t lane, uint32_t t1, StreamCursor &sc, State &z,
                                             uint32_t &cnt, uint32_t &begin) {
    const float4 fresh = buf.start[b][s][lane];
    const float force = buf.force[b][s][lane];
    bool done = CONTRACT ? euler_step_contracted<KNOWN_SMALL>(z, force) : euler_step<KNOWN_SMALL>(z, force);
    if (LIMIT) done |= (t1 - begin) >= p.max_steps;
    // selects, not a branch: nothing diverges in the stepping warp (measured equal or up to 4 % faster)
    cnt += done ? 1u : 0u;
    begin = done ? t1 : begin;
    z.x = done ? fresh.x : z.x;
    z.xd = done ? fresh.y : z.xd;
    z.th = done ? fresh.z : z.th;
    z.thd = done ? fresh.w : z.thd;
    // Same layout and meaning as the general kernel's streams. STREAMS 1: exactly the reward plane
    // and the done bits, no tests (each run-time test is a branch in the one warp whose latency
    // is the launch's time); 2: any combination.
    if (STREAMS == 1) {
        const uint32_t m = __ballot_sync(0xffffffffu, done && sc.valid);
        if (lane == 0u) p.done_bits[sc.word_off] = m;
        if (sc.valid) p.reward_stream[sc.env_off] = 1.0f;
        sc.env_off += p.n;
        sc.word_off += sc.words;
    }
    if (STREAMS == 2) {
        if (sc.want_done) {
            const uint32_t m = __ballot_sync(0xffffffffu, done && sc.valid);
            if (lane == 0u) p.done_bits[sc.word_off] = m;
        }
        if (sc.want_act) {
            const uint32_t m = __ballot_sync(0xffffffffu, force > 0.0f && sc.valid);
            if (lane == 0u) p.action_bits[sc.word_off] = m;
        }
        if (sc.valid) {
            if (sc.want_rew) p.reward_stream[sc.env_off] = 1.0f;
            if (sc.want_traj) {
                float *tr = p.trajectory + 4 * sc.env_off - 3 * sc.idx;  // row 4k, column idx
                tr[0] = z.x;
                tr[p.n] = z.xd;
                tr[2 * p.n] = z.th;
                tr[3 * p.n] = z.thd;
            }
        }
        sc.env_off += p.n;
        sc.word_off += sc.words;
    }
}

template <int PAIRS, bool LIMIT, bool CONTRACT, int STREAMS>
__global__ void __launch_bounds__(64 * PAIRS) rollout_assisted_kernel(const __grid_constant__ RolloutParams p) {
    constexpr int kChunk = kChunkOf<PAIRS>;
    __shared__ PairBuffers<kChunk> s_buf[PAIRS];
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    const bool producer = warp >= (uint32_t)PAIRS;
    const uint32_t pair = producer ? warp - PAIRS : warp;
    const int64_t task = (int64_t)blockIdx.x * PAIRS + pair;
    // Both warps of a pair leave here together, before their first barrier; no other pair uses
    // their barrier. Nothing that differs between the two warps of a pair (or between lanes) may
    // decide an exit or a barrier from here on: each warp must execute exactly 1 + n_chunks
    // barriers, a count fixed by the launch parameters, or its partner waits for ever.
    if (task >= p.n_tasks) return;
    PairBuffers<kChunk> &buf = s_buf[pair];
    const uint32_t n_chunks = (p.T + kChunk - 1) / kChunk;

    int64_t idx = task * 32 + lane;
    const bool valid = idx < p.n;
    if (!valid) idx = p.n - 1;  // idle lanes shadow the last environment and store nothing
    const uint32_t env = p.env_offset + (uint32_t)idx;
    const FoldedKeys kr = fold_keys(make_keys(p.salt_r, env));

    if (producer) {
        const FoldedKeys ka = fold_keys(make_keys(p.salt_a, env));
        const int64_t words = (p.n + 31) >> 5;
        for (uint32_t c = 0; c <= n_chunks; ++c) {
            // chunk c is written while the consumer works on chunk c - 1 (other buffer); the
            // buffer written here was last read in chunk c - 2, which the barrier before closed
            if (c < n_chunks) {
                const uint32_t b = c & 1u, tc = p.t0 + c * kChunk;
                // The caller's actions: row (t - t0) of [T][words], one word per warp task. Lane s
                // fetches the word of the chunk's step s, all in one load issued before the
                // hashing below and used after it, when it has long arrived.
                uint32_t my_word = 0u;
                if (p.action_bits_in) {
                    const uint32_t row = c * kChunk + lane;
                    if (lane < (uint32_t)kChunk && row < p.T)
                        my_word = __ldg(p.action_bits_in + (int64_t)row * words + task);
                }
#pragma unroll 4
                for (int s = 0; s < kChunk; ++s) {
                    const uint32_t t = tc + s;
                    const State f = start_state_folded(kr, fold16(4u * (t + 1u)));
                    buf.start[b][s][lane] = make_float4(f.x, f.xd, f.th, f.thd);
                    if (!p.action_bits_in)
                        buf.force[b][s][lane] = force_from_signbit(action_signbit_folded(ka, fold16(t)));
                }
                if (p.action_bits_in) {
#pragma unroll 4
                    for (int s = 0; s < kChunk; ++s) {
                        const uint32_t word = __shfl_sync(0xffffffffu, my_word, s);
                        buf.force[b][s][lane] = force_from_signbit((word << (31u - lane)) & 0x80000000u);
                    }
                }
            }
            pair_barrier<PAIRS>(pair);
        }
        return;
    }

    State z;
    if (p.init_planes) {
        z.x = p.init_planes[idx];
        z.xd = p.init_planes[p.init_stride + idx];
        z.th = p.init_planes[2 * p.init_stride + idx];
        z.thd = p.init_planes[3 * p.init_stride + idx];
    } else {
        z = start_state_folded(kr, fold16(4u * p.t0));
    }
    // as in the general kernel: the returns follow from the time of the last termination, and
    // only the step limit needs the carried-in episode length inside the loop
    uint32_t cnt = 0u, begin = p.t0 - ((LIMIT && p.ep_len_io) ? p.ep_len_io[idx] : 0u);
    const uint32_t t_end = p.t0 + p.T;
    StreamCursor sc;
    sc.env_off = sc.idx = idx;
    sc.word_off = task;  // one 32-env word per warp task
    sc.words = (p.n + 31) >> 5;
    sc.valid = valid;
    sc.want_done = STREAMS == 2 && p.done_bits;
    sc.want_act = STREAMS == 2 && p.action_bits;
    sc.want_rew = STREAMS == 2 && p.reward_stream;
    sc.want_traj = STREAMS == 2 && p.trajectory;
    pair_barrier<PAIRS>(pair);  // chunk 0 is there
    for (uint32_t c = 0; c < n_chunks; ++c) {
        const uint32_t b = c & 1u, tc = p.t0 + c * kChunk;
        const int steps = (int)min((uint32_t)kChunk, t_end - tc);
        if (c != 0u && steps == kChunk) {
#pragma unroll kStepUnroll
            for (int s = 0; s < kChunk; ++s)
                consume_step<true, LIMIT, CONTRACT, STREAMS>(p, buf, b, s, lane, tc + s + 1u, sc, z, cnt, begin);
        } else {
            // The caller's initial state may hold any angle: the very first step tests it per
            // lane. From the second step on every angle is a survivor's (<= 0.2095) or a start
            // state's (<= 0.05).
            int s = 0;
            if (c == 0u) {
                consume_step<false, LIMIT, CONTRACT, STREAMS>(p, buf, b, 0, lane, tc + 1u, sc, z, cnt, begin);
                s = 1;
            }
#pragma unroll kStepUnroll
            for (; s < steps; ++s)
                consume_step<true, LIMIT, CONTRACT, STREAMS>(p, buf, b, s, lane, tc + s + 1u, sc, z, cnt, begin);
        }
        pair_barrier<PAIRS>(pair);
    }

    unsigned long long tot_ret = 0, tot_cnt = 0;
    if (valid) {
        const uint32_t carried = p.ep_len_io ? p.ep_len_io[idx] : 0u;
        const uint32_t first_begin = p.t0 - carried;
        const uint32_t ret = cnt ? begin - first_begin : 0u;
        const uint32_t running = t_end - begin + ((!LIMIT && cnt == 0u) ? carried : 0u);
        if (p.ep_return_sum) p.ep_return_sum[idx] = (float)ret;
        if (p.ep_count) p.ep_count[idx] = cnt;
        if (p.ep_len_io) p.ep_len_io[idx] = running;
        if (p.out_planes) {
            p.out_planes[idx] = z.x;
            p.out_planes[p.out_stride + idx] = z.xd;
            p.out_planes[2 * p.out_stride + idx] = z.th;
            p.out_planes[3 * p.out_stride + idx] = z.thd;
        }
        tot_ret = ret;
        tot_cnt = cnt;
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

}  // namespace

bool rollout_assisted_applies(const RolloutParams &p, int policy, bool streams) {
    (void)streams;
    // supplied actions replace whatever policy was named
    if ((policy != 0 && !p.action_bits_in) || p.start_in) return false;
    if (g_tuning.rollout_coop == 4) return true;
    if (g_tuning.rollout_coop != 0 || g_tuning.rollout_ept != 0) return false;
    // up to ten pairs per SM (five CTAs of two pairs: 200 KB of shared memory; a sixth CTA would
    // wait for a second wave). Measured against the general kernel's best shape, ms per launch:
    // x 5,000 steps 9,472 envs 0.25 / 0.61, 18,944 envs 0.45 / 0.61, 28,416 envs 0.57 / 0.74,
    // 37,888 envs 0.70 / 0.74; x 4,000 steps 47,360 envs (ten pairs per SM) 0.72 / 0.83,
    // 56,832 envs (twelve) 0.88 / 0.82.
    return (p.n + 31) / 32 <= (int64_t)sm_count() * 10;
}

namespace {
template <int PAIRS, bool CONTRACT, int STREAMS>
void launch_limit(const RolloutParams &p, unsigned grid, cudaStream_t s) {
    if (p.max_steps)
        rollout_assisted_kernel<PAIRS, true, CONTRACT, STREAMS><<<grid, 64 * PAIRS, 0, s>>>(p);
    else
        rollout_assisted_kernel<PAIRS, false, CONTRACT, STREAMS><<<grid, 64 * PAIRS, 0, s>>>(p);
}
template <int PAIRS, bool CONTRACT>
void launch_pairs(const RolloutParams &p, unsigned grid, cudaStream_t s) {
    if (p.reward_stream && p.done_bits && !p.action_bits && !p.trajectory)
        launch_limit<PAIRS, CONTRACT, 1>(p, grid, s);
    else if (p.reward_stream || p.done_bits || p.action_bits || p.trajectory)
        launch_limit<PAIRS, CONTRACT, 2>(p, grid, s);
    else
        launch_limit<PAIRS, CONTRACT, 0>(p, grid, s);
}
}  // namespace

cudaError_t launch_rollout_assisted(RolloutParams &p, bool contracted, cudaStream_t s) {
    p.n_tasks = (p.n + 31) / 32;
    // one pair per CTA spreads the pairs over the SMs; beyond one pair per SM, two pairs per CTA
    // put the four warps of a CTA on the four schedulers of one SM
    const bool two = g_tuning.rollout_block ? g_tuning.rollout_block >= 128 : p.n_tasks > sm_count();
    const unsigned grid = (unsigned)(two ? (p.n_tasks + 1) / 2 : p.n_tasks);
    if (two)
        contracted ? launch_pairs<2, true>(p, grid, s) : launch_pairs<2, false>(p, grid, s);
    else
        contracted ? launch_pairs<1, true>(p, grid, s) : launch_pairs<1, false>(p, grid, s);
    count_launch();
    return cudaGetLastError();
}

}  // namespace cp
