// Fused rollout with deferred restarts (paper Sec. V-D / V-G: all steps in one launch; Sec. V-A:
// the random values must not stand in the step's way).
//
// The general rollout kernel restarts finished environments after every step, and with the
// random policy some environment of a warp finishes on 95 % of the steps, so the restart
// machinery (ballots, ranks, shared-memory exchange, or four hashes issued for the whole warp) is
// paid on practically every step although 4.5 % of the environments need it. Nothing forces an
// environment to restart in the same loop trip it finished in: every random value is a function
// of (seed, env, global time), so an environment that waits keeps its own clock and simply
// continues later from the start state of the time it finished at. Here
//
//   * a thread owns two environments ("slots"), stepped together by the packed float32
//     instructions of sm_100a (euler_step_pair: one instruction, two independent roundings);
//   * every slot has its own global time t; a slot whose episode ended stops counting and idles
//     (its half of the packed arithmetic computes values nobody reads);
//   * every K trips the idle slots hash their start state of time t and go on. A slot therefore
//     lags behind the trip counter by the trips it idled (about (K-1)/2 per episode), and the
//     loop runs until the slowest slot of the warp has done its T steps.
//
// Every environment still takes exactly the steps t0 .. t0+T-1 with the actions and start states
// of those times: the results are bit for bit those of the other work shapes (the tests compare
// them). What changes is the issue count: restart work drops from every trip to every K-th, and
// the price is idle slots (about 7 % at K = 4 with the random policy's 22-step episodes) and a
// ragged end.
//
// Scope: hashed actions, the shared linear policy, the shared 4-16-2 tanh network or one linear
// policy per environment; either arithmetic; with or without the episode step limit; per-step
// outputs either none or exactly the reward plane + done bitmask (the action bitmask and the
// trajectory are rows of global time that half the lanes would have to touch every step). The
// wider and deeper networks (4-32-2, 4-64-2, 4-16-16-2) too, for the plain call: no step limit,
// no per-step outputs. Everything else takes the general kernel.
//
// No warp waits for another one and nothing spins: the loop's trip count is bounded by the
// launch parameters (every trip block advances every unfinished slot by at least one step).
#pragma once
#include <type_traits>

#include "cartpole_device.cuh"
#include "cartpole_internal.h"

namespace cp {

namespace {

// Shared policies read their weights as (w, w) pairs: the launcher duplicates every weight in the
// launch parameters, so that one packed fused multiply-add applies it to both environments of a
// thread. Each half is the scalar chain of linear_action / mlp_action (same order, one rounding per
// fused operation), hence the same logits bit for bit.
__device__ __forceinline__ void argmax_pair(f32x2 l0, f32x2 l1, uint32_t &sb0, uint32_t &sb1) {
    float a0, a1, b0, b1;
    unpack2(l0, a0, a1);
    unpack2(l1, b0, b1);
    sb0 = (b0 > a0) ? 0x80000000u : 0u;
    sb1 = (b1 > a1) ? 0x80000000u : 0u;
}
__device__ __forceinline__ void linear_action_pair(const f32x2 *w, const StatePair &z, uint32_t &sb0, uint32_t &sb1) {
    // w: W[2][4] then b[2], as pairs
    f32x2 l0 = w[8], l1 = w[9];
    l0 = fma2(w[0], z.x, l0);
    l1 = fma2(w[4], z.x, l1);
    l0 = fma2(w[1], z.xd, l0);
    l1 = fma2(w[5], z.xd, l1);
    l0 = fma2(w[2], z.th, l0);
    l1 = fma2(w[6], z.th, l1);
    l0 = fma2(w[3], z.thd, l0);
    l1 = fma2(w[7], z.thd, l1);
    argmax_pair(l0, l1, sb0, sb1);
}
template <int H, bool CONTRACT>
__device__ __forceinline__ void mlp_action_pair(const f32x2 *w, const StatePair &z, uint32_t &sb0, uint32_t &sb1) {
    // w: W1[H][4], b1[H], W2[2][H], b2[2], as pairs
    const f32x2 *w1 = w, *b1 = w + 4 * H, *w2 = w + 5 * H, *b2 = w + 7 * H;
    f32x2 l0 = b2[0], l1 = b2[1];
#pragma unroll
    for (int j = 0; j < H; ++j) {
        f32x2 acc = b1[j];
        acc = fma2(w1[4 * j + 0], z.x, acc);
        acc = fma2(w1[4 * j + 1], z.xd, acc);
        acc = fma2(w1[4 * j + 2], z.th, acc);
        acc = fma2(w1[4 * j + 3], z.thd, acc);
        const f32x2 h = CONTRACT ? tanh_contracted_pair(acc) : tanh_pair(acc);
        l0 = fma2(w2[j], h, l0);
        l1 = fma2(w2[H + j], h, l1);
    }
    argmax_pair(l0, l1, sb0, sb1);
}

// 4-16-16-2 (MlpDeepW as pairs: W1[16][4], b1[16], W2[16][16], b2[16], W3[2][16], b3[2]): the
// sixteen first-layer activations of both slots stay in registers, second-layer units feed the
// logit chains as they are produced — mlp_deep_action's order, half by half.
template <bool CONTRACT>
__device__ __forceinline__ void mlp_deep_action_pair(const f32x2 *w, const StatePair &z, uint32_t &sb0, uint32_t &sb1) {
    const f32x2 *w1 = w, *b1 = w + 64, *w2 = w + 80, *b2 = w + 336, *w3 = w + 352, *b3 = w + 384;
    f32x2 h1[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        f32x2 acc = b1[j];
        acc = fma2(w1[4 * j + 0], z.x, acc);
        acc = fma2(w1[4 * j + 1], z.xd, acc);
        acc = fma2(w1[4 * j + 2], z.th, acc);
        acc = fma2(w1[4 * j + 3], z.thd, acc);
        h1[j] = CONTRACT ? tanh_contracted_pair(acc) : tanh_pair(acc);
    }
    f32x2 l0 = b3[0], l1 = b3[1];
#pragma unroll
    for (int k = 0; k < 16; ++k) {
        f32x2 acc = b2[k];
#pragma unroll
        for (int j = 0; j < 16; ++j) acc = fma2(w2[16 * k + j], h1[j], acc);
        const f32x2 h2 = CONTRACT ? tanh_contracted_pair(acc) : tanh_pair(acc);
        l0 = fma2(w3[k], h2, l0);
        l1 = fma2(w3[16 + k], h2, l1);
    }
    argmax_pair(l0, l1, sb0, sb1);
}

// The shared tanh networks: 2 (4-16-2), 4 (4-32-2), 5 (4-64-2), 7 (4-16-16-2).
__host__ __device__ constexpr bool is_network(int policy) { return policy == 2 || policy == 4 || policy == 5 || policy == 7; }
// The networks wider or deeper than 4-16-2 (4, 5, 7): built for the plain call only — no step limit,
// no per-step outputs, default trip spacing (a kernel of theirs takes up to a minute to compile).
// Against the general kernel with one environment per thread, 16,777,216 x 200: 4-32-2 77.3 ->
// 70.0 ms, 4-64-2 145.1 -> 135.3 ms, 4-16-16-2 94.9 -> 88.7 ms (contracted arithmetic 54.4 ->
// 51.0, 103.8 -> 98.5, 72.4 -> 59.0 ms).
__host__ __device__ constexpr bool is_wide_network(int policy) { return is_network(policy) && policy != 2; }

// The done bit plane of a launch that sets its bits by atomic OR has to be zeroed first.
// A warp that clears its own words inside the rollout writes 4 bytes into each of T separate
// sectors; contiguous stores (clear_words_kernel) are far cheaper per byte but cost a launch. With
// the reward plane and done bits, in-kernel against separate clearing (us per launch): 65,536 envs
// x 64 steps 20.7 / 24.9, 1,048,576 x 64 168.8 / 173.2, x 192 455.1 / 454.9, linear policy x 384
// 831.0 / 795.1, 4,194,304 x 1,000 8.45 / 8.12 ms.
constexpr uint32_t kClearApartFrom = 192u;

// Actions of both slots, in sign-bit form. SHORT: every time of the launch is below 2^16, where
// fold16(t) == t.
template <int POLICY, bool SHORT, bool CONTRACT>
__device__ __forceinline__ void deferred_actions(const RolloutParams &p, const FoldedKeys (&ka)[2],
                                                 const LinearW *own, const uint32_t (&t)[2], const StatePair &zz,
                                                 uint32_t &sb0, uint32_t &sb1) {
    const f32x2 *pairs = reinterpret_cast<const f32x2 *>(p.w);
    if (POLICY == 0) {
        sb0 = action_signbit_folded(ka[0], SHORT ? t[0] : fold16(t[0]));
        sb1 = action_signbit_folded(ka[1], SHORT ? t[1] : fold16(t[1]));
    } else if (POLICY == 1) {
        linear_action_pair(pairs, zz, sb0, sb1);
    } else if (POLICY == 2) {
        mlp_action_pair<16, CONTRACT>(pairs, zz, sb0, sb1);
    } else if (POLICY == 4) {
        mlp_action_pair<32, CONTRACT>(pairs, zz, sb0, sb1);
    } else if (POLICY == 5) {
        mlp_action_pair<64, CONTRACT>(pairs, zz, sb0, sb1);
    } else if (POLICY == 7) {
        mlp_deep_action_pair<CONTRACT>(pairs, zz, sb0, sb1);
    } else {
        State a, b;
        unpack_states(zz, a, b);
        sb0 = linear_action(own[0], a);
        sb1 = linear_action(own[POLICY == 6 ? 1 : 0], b);
    }
}

// POLICY: 0 hashed actions, 1 shared linear policy, 2 / 4 / 5 / 7 a shared tanh network (is_network),
// 6 one linear policy per environment.
// K: trips between restart passes. LIMIT: episodes are cut off after p.max_steps steps.
// RD: the reward plane and the done bitmask are written (see the comment at reward_row).
// CONTRACT: the contracted arithmetic (euler_step_contracted_pair, tanh_contracted_pair).
// One CTA per SM is all the launch bounds ask for, which lets the assembler take the registers it
// wants (77-96 instead of the 58-64 it settles for when left to aim at occupancy): the kernel is
// bound by the float32 pipe, not by latency, and the extra registers hold the packed constants
// that are otherwise re-materialised every trip (1,048,576 x 500: 1.032 -> 0.988 ms; with the
// reward plane and done bits, 4,194,304 x 100: 0.936 -> 0.828 ms; forcing 3 or 4 CTAs per SM
// measured 1.04 / 1.01 and 0.87 / 0.93 ms).
// (The network policies are the exception: their hidden units are latency — exp2 and
// reciprocal on the special-function pipe — that only more resident warps hide: 16,777,216 x
// 200 takes 53.1 / 41.1 / 39.9 / 39.4 / 40.8 ms at 1 / 2 / 3 / 4 / 5 CTAs per SM.)
template <int POLICY, int K, bool SHORT, bool LIMIT, bool RD, bool CONTRACT>
__global__ void __launch_bounds__(256, is_network(POLICY) ? 4 : 1) rollout_deferred_kernel(const __grid_constant__ RolloutParams p) {
    const uint32_t lane = threadIdx.x & 31u;
    const int64_t task = (int64_t)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5);
    unsigned long long tot_ret = 0, tot_cnt = 0;
    if (task < p.n_tasks) {  // warp-uniform
        const int64_t base = task * 64;
        const uint32_t t_end = p.t0 + p.T;
        FoldedKeys ka[2], kr[2];
        LinearW own[POLICY == 6 ? 2 : 1];
        uint32_t t[2], cnt[2], begin[2];
        bool act[2];
        State z0[2];
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            int64_t idx = base + j * 32 + lane;
            if (idx >= p.n) idx = p.n - 1;  // idle lanes shadow the last environment and store nothing
            const uint32_t env = p.env_offset + (uint32_t)idx;
            if (POLICY == 0) ka[j] = fold_keys(make_keys(p.salt_a, env));
            else ka[j] = FoldedKeys{0u, 0u};
            kr[j] = fold_keys(make_keys(p.salt_r, env));
            if (p.init_planes) {
                z0[j].x = p.init_planes[idx];
                z0[j].xd = p.init_planes[p.init_stride + idx];
                z0[j].th = p.init_planes[2 * p.init_stride + idx];
                z0[j].thd = p.init_planes[3 * p.init_stride + idx];
            } else {
                z0[j] = start_state_folded(kr[j], fold16(4u * p.t0));
            }
            if (POLICY == 6) {
                LinearW &o = own[POLICY == 6 ? j : 0];
#pragma unroll
                for (int q = 0; q < 8; ++q) o.w[q / 4][q % 4] = p.env_weights[(int64_t)q * p.n + idx];
                o.b[0] = p.env_weights[8 * p.n + idx];
                o.b[1] = p.env_weights[9 * p.n + idx];
            }
            t[j] = p.t0;
            cnt[j] = 0u;
            begin[j] = p.t0 - ((LIMIT && p.ep_len_io) ? p.ep_len_io[idx] : 0u);
            act[j] = true;
        }
        StatePair zz = pack_states(z0[0], z0[1]);

        // Per-step outputs although the environments run on clocks of their own (RD):
        //  * every step of every environment earns reward 1, so row r of the reward plane does not
        //    depend on any clock: the warp writes it for its 64 environments in trip r, as full lines;
        //  * a done bit is rare. The bit plane is zeroed first — for launches of kClearApartFrom
        //    steps or more by a launch of its own before this one (clear_words_kernel: contiguous
        //    16-byte stores), for shorter ones here, every warp its own two words of every row — and
        //    an environment whose episode ended at step t sets its bit in row t - t0 with one
        //    atomic OR — in the restart pass, where its stopped clock still tells that time.
        const int64_t words = (p.n + 31) >> 5;
        const int64_t word0 = task * 2;
        float *rew_row = RD ? p.reward_stream + base + lane : nullptr;
        if (RD && p.T < kClearApartFrom) {
            for (uint32_t r = lane; r < p.T; r += 32u) {
                if (word0 < words) p.done_bits[(int64_t)r * words + word0] = 0u;
                if (word0 + 1 < words) p.done_bits[(int64_t)r * words + word0 + 1] = 0u;
            }
            __syncwarp();  // orders the clearing stores before any lane's later atomic on the same word
        }
        const bool has0 = base + lane < p.n, has1 = base + 32 + lane < p.n;
        // CHECK: the row may lie beyond the last one (only the tail's trips can)
        auto reward_row = [&](auto check, uint32_t row) {
            if (RD && (!decltype(check)::value || row < p.T)) {
                if (has0) rew_row[0] = 1.0f;
                if (has1) rew_row[32] = 1.0f;
                rew_row += p.n;
            }
        };
        // the done bit of slot j's episode that ended with the step of time t_done
        auto set_done_bit = [&](int j, uint32_t t_done) {
            if (RD && base + j * 32 + lane < p.n)
                atomicOr(p.done_bits + (int64_t)(t_done - p.t0) * words + word0 + j, 1u << lane);
        };

        uint32_t trips = 0;  // trips made; no slot's clock is more than one step ahead of t0 + trips

        // Slot j has done its last step (its clock reached t_end) and retires. cnt / begin are
        // brought up to date by the restart pass, so an episode that ended on this very step
        // (done_now) is added here; it also hands over the start state of t_end. The final state is
        // stored now (the slot's half of the packed arithmetic goes on computing values nobody
        // reads); the per-env results wait in cnt / begin and are stored by the whole warp after
        // the loop, as full lines (a caller may have pointed them at pinned host memory).
        auto finalize = [&](int j, bool done_now) {
            if (done_now) {
                cnt[j] += 1u;
                begin[j] = t_end;
                set_done_bit(j, t_end - 1u);
            }
            if (p.out_planes) {
                State a, b;
                unpack_states(zz, a, b);
                State mine = j ? b : a;
                if (done_now) mine = start_state_folded(kr[j], fold16(4u * t_end));
                const int64_t idx = base + j * 32 + lane;
                if (idx < p.n) {
                    p.out_planes[idx] = mine.x;
                    p.out_planes[p.out_stride + idx] = mine.xd;
                    p.out_planes[2 * p.out_stride + idx] = mine.th;
                    p.out_planes[3 * p.out_stride + idx] = mine.thd;
                }
            }
        };

        // Slot j after a trip: a stepping slot's clock advances, and it goes idle if its episode
        // ended (done_now). TAIL: the slot may have done its last step.
        auto after_step = [&](auto tail, int j, bool done_now) {
            constexpr bool TAIL = decltype(tail)::value;
            const bool live = act[j];
            if (live) t[j] += 1u;
            // begin[j] is the time the running episode began (set by the restart pass; before t0 by
            // the steps carried in): an episode that has lasted max_steps steps ends like a fall
            if (LIMIT) done_now = done_now || (t[j] - begin[j]) >= p.max_steps;
            act[j] = live && !done_now;
            if (TAIL) {
                if (live && t[j] == t_end) {
                    finalize(j, done_now);
                    act[j] = false;
                }
            }
        };

        // Idle slots that still have steps to do: their episode ended at their (stopped) clock,
        // which is also the time the next one begins; they take that time's start state, each
        // lane hashing its own. (Handing the hashes to the whole warp through shared memory, as
        // the general kernel does after every step, was measured here too: with a dozen restarts
        // per pass its ballots, ranks, barriers and rounds cost more instructions than the
        // divergent per-lane hashes, 1.29 against 1.14 ms on 1,048,576 x 500.)
        //
        // One step of foresight shortens the waiting: whether an episode ends with its NEXT step is
        // decided by x + tau*x_dot and theta + tau*theta_dot of the state it has now (the step's
        // accelerations only reach the velocities), and the state a terminal step produces is
        // discarded anyway. So a stepping slot whose next step is terminal takes that step here, on
        // the books only — clock + 1 — and restarts in this pass instead of ending in the next trip
        // and idling until the pass after. Same comparison on the same roundings as the step
        // itself, hence the same decision. To keep the bound on the clocks (with foresight no clock
        // more than one step ahead of the trip counter, without it none ahead at all: the main part
        // of the loop relies on that) a slot that is already ahead does not look ahead, and neither
        // does one whose next step is its last.
        // (Only for the network policies — config 5's episodes last 9 steps: 39.4 -> 38.0 ms.
        // With hashed actions (22-step episodes) the saved waiting and the cost of the test in
        // every pass cancel — 1,048,576 x 500: 0.947 ms without, 0.956 ms with it — and with the
        // linear policies' 80-step episodes the test only costs: 4,194,304 x 100 with streams
        // 0.828 -> 0.878 ms.)
        constexpr bool FORESIGHT = is_network(POLICY);
        auto restart_pass = [&](auto tail) {
            constexpr bool TAIL = decltype(tail)::value;
            if (FORESIGHT) {
                const f32x2 tau = splat2(kTau), ntau = splat2(-kTau);
                const f32x2 nx = CONTRACT ? fma2(tau, zz.xd, zz.x) : add_product2(zz.x, mul2(ntau, zz.xd));
                const f32x2 nth = CONTRACT ? fma2(tau, zz.thd, zz.th) : add_product2(zz.th, mul2(ntau, zz.thd));
                float x0, x1, a0, a1;
                unpack2(nx, x0, x1);
                unpack2(nth, a0, a1);
                bool ends[2] = {fabsf(x0) > kXT || fabsf(a0) > kTT, fabsf(x1) > kXT || fabsf(a1) > kTT};
#pragma unroll
                for (int j = 0; j < 2; ++j) {
                    if (LIMIT) ends[j] = ends[j] || (t[j] + 1u - begin[j]) >= p.max_steps;
                    if (act[j] && ends[j] && t[j] <= p.t0 + trips && t[j] + 1u != t_end) {
                        t[j] += 1u;
                        act[j] = false;
                    }
                }
            }
#pragma unroll
            for (int j = 0; j < 2; ++j) {
                if (!act[j] && (!TAIL || t[j] != t_end)) {
                    cnt[j] += 1u;
                    begin[j] = t[j];
                    set_done_bit(j, t[j] - 1u);
                    State a, b;
                    unpack_states(zz, a, b);
                    (j ? b : a) = start_state_folded(kr[j], fold16(4u * t[j]));
                    zz = pack_states(a, b);
                    act[j] = true;
                }
            }
        };

        uint32_t row = 0;  // trips made so far = the row of the reward plane the next trip writes
        auto trip = [&](auto tail) {
            if (RD) reward_row(tail, row++);
            uint32_t sb0, sb1;
            deferred_actions<POLICY, SHORT, CONTRACT>(p, ka, own, t, zz, sb0, sb1);
            bool d0, d1;
            const f32x2 force = pack2(force_from_signbit(sb0), force_from_signbit(sb1));
            if (CONTRACT) euler_step_contracted_pair(zz, force, d0, d1);
            else euler_step_pair(zz, force, d0, d1);
            after_step(tail, 0, d0);
            after_step(tail, 1, d1);
        };

        if (p.init_planes) {
            // A caller's states may hold any angle: the first trip uses the general scalar step.
            // From then on every stepping slot is a survivor (|theta| <= 0.2095) or a fresh
            // start state (|theta| <= 0.05), which is the packed step's domain.
            if (RD) reward_row(std::false_type{}, row++);
            uint32_t sb0, sb1;
            deferred_actions<POLICY, SHORT, CONTRACT>(p, ka, own, t, zz, sb0, sb1);
            State a, b;
            unpack_states(zz, a, b);
            const bool d0 = CONTRACT ? euler_step_contracted<false>(a, force_from_signbit(sb0))
                                     : euler_step<false>(a, force_from_signbit(sb0));
            const bool d1 = CONTRACT ? euler_step_contracted<false>(b, force_from_signbit(sb1))
                                     : euler_step<false>(b, force_from_signbit(sb1));
            zz = pack_states(a, b);
            after_step(std::true_type{}, 0, d0);
            after_step(std::true_type{}, 1, d1);
            trips = 1;
            restart_pass(std::true_type{});
        }
        // Main part: after these trips no clock can have reached t_end yet (clocks run at most one
        // step ahead of the trips), so no slot can retire.
        // (a network policy's trip is 600 instructions or more: its K trips stay a loop)
        constexpr int kUnroll = is_network(POLICY) ? 1 : K;
        while (trips + K + (FORESIGHT ? 1u : 0u) <= p.T - 1u) {
#pragma unroll kUnroll
            for (int k = 0; k < K; ++k) trip(std::false_type{});
            trips += K;
            restart_pass(std::false_type{});
        }
        // Tail: slots retire as their clocks reach t_end. Every block of K trips advances every
        // unretired slot by at least one step, so p.T blocks always suffice.
        for (uint32_t block = 0; block <= p.T; ++block) {
            if (__all_sync(0xffffffffu, t[0] == t_end && t[1] == t_end)) break;
#pragma unroll kUnroll
            for (int k = 0; k < K; ++k) trip(std::true_type{});
            if (FORESIGHT) trips += K;
            restart_pass(std::true_type{});
        }
#pragma unroll
        for (int j = 0; j < 2; ++j) {
            const int64_t idx = base + j * 32 + lane;
            if (idx >= p.n) continue;
            // sum of the returns of the completed episodes = last termination time - time the first
            // of them began (every step earns reward 1); begin[j] still holds its initial value if
            // no episode ended in this launch
            const uint32_t carried = p.ep_len_io ? p.ep_len_io[idx] : 0u;
            const uint32_t ret = cnt[j] ? begin[j] - (p.t0 - carried) : 0u;
            const uint32_t running = t_end - begin[j] + ((!LIMIT && cnt[j] == 0u) ? carried : 0u);
            if (p.ep_return_sum) p.ep_return_sum[idx] = (float)ret;
            if (p.ep_count) p.ep_count[idx] = cnt[j];
            if (p.ep_len_io) p.ep_len_io[idx] = running;
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

// Zeroes n 32-bit words (see kClearApartFrom).
__global__ void __launch_bounds__(256) clear_words_kernel(uint32_t *w, int64_t n) {
    const int64_t i = ((int64_t)blockIdx.x * 256 + threadIdx.x) * 4;
    if (i + 4 <= n && (reinterpret_cast<uintptr_t>(w) & 15u) == 0u) {
        *reinterpret_cast<uint4 *>(w + i) = make_uint4(0u, 0u, 0u, 0u);
    } else {
        for (int k = 0; k < 4; ++k)
            if (i + k < n) w[i + k] = 0u;
    }
}

template <int POLICY, bool SHORT, bool LIMIT, bool RD>
cudaError_t launch_k(RolloutParams &p, int k, bool contracted, cudaStream_t s) {
    p.n_tasks = (p.n + 63) / 64;
    int64_t grid = (p.n_tasks + 7) / 8;
    if (grid > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
    if (RD && p.T >= kClearApartFrom) {
        const int64_t n_words = (int64_t)p.T * ((p.n + 31) >> 5);
        const int64_t clear_grid = (n_words + 1023) / 1024;
        if (clear_grid > 0x7fffffffLL) return cudaErrorInvalidConfiguration;
        clear_words_kernel<<<(unsigned)clear_grid, 256, 0, s>>>(p.done_bits, n_words);
        count_launch();
    }
    if (contracted) {  // the optional arithmetic comes at the default trip spacing only
        constexpr int kC = is_network(POLICY) ? 2 : 6;
        rollout_deferred_kernel<POLICY, kC, SHORT, LIMIT, RD, true><<<(unsigned)grid, 256, 0, s>>>(p);
    } else if constexpr (is_wide_network(POLICY)) {  // and so do the wider and deeper networks
        rollout_deferred_kernel<POLICY, 3, SHORT, LIMIT, RD, false><<<(unsigned)grid, 256, 0, s>>>(p);
    } else {
        switch (k) {
            case 2: rollout_deferred_kernel<POLICY, 2, SHORT, LIMIT, RD, false><<<(unsigned)grid, 256, 0, s>>>(p); break;
            case 3: rollout_deferred_kernel<POLICY, 3, SHORT, LIMIT, RD, false><<<(unsigned)grid, 256, 0, s>>>(p); break;
            case 6: rollout_deferred_kernel<POLICY, 6, SHORT, LIMIT, RD, false><<<(unsigned)grid, 256, 0, s>>>(p); break;
            case 8: rollout_deferred_kernel<POLICY, 8, SHORT, LIMIT, RD, false><<<(unsigned)grid, 256, 0, s>>>(p); break;
            default: rollout_deferred_kernel<POLICY, 4, SHORT, LIMIT, RD, false><<<(unsigned)grid, 256, 0, s>>>(p); break;
        }
    }
    count_launch();
    return cudaGetLastError();
}

template <int POLICY, bool SHORT>
cudaError_t launch_limit(RolloutParams &p, int k, bool contracted, cudaStream_t s) {
    if constexpr (is_wide_network(POLICY)) {
        return launch_k<POLICY, SHORT, false, false>(p, k, contracted, s);  // rollout_deferred_applies: nothing else gets here
    } else {
        const bool rd = p.reward_stream != nullptr;  // rollout_deferred_applies: then done_bits too, nothing else
        if (p.max_steps)
            return rd ? launch_k<POLICY, SHORT, true, true>(p, k, contracted, s)
                      : launch_k<POLICY, SHORT, true, false>(p, k, contracted, s);
        return rd ? launch_k<POLICY, SHORT, false, true>(p, k, contracted, s)
                  : launch_k<POLICY, SHORT, false, false>(p, k, contracted, s);
    }
}

}  // namespace

}  // namespace cp
