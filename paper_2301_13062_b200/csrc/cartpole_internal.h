// Host-side declarations shared by the .cu files of libcartpole (not installed).
#pragma once
#include <cstddef>
#include <cstdint>
#include <cuda_runtime.h>

struct cp_state;

namespace cp {

// Parameters of one fused step launch.
struct StepParams {
    const float *in;
    int64_t in_stride;
    float *out;
    int64_t out_stride;
    int64_t n;
    uint32_t t, env_offset, salt_a, salt_r;
    const uint8_t *action;  // or nullptr: hashed
    float *reward;          // or nullptr
    uint8_t *done;          // or nullptr
    uint32_t *ep_len;       // or nullptr: steps taken in each running episode, in/out
    uint32_t max_steps;     // episode step limit (needs ep_len), 0 = none
};

// Parameters of one rollout launch. Weights travel in the launch parameters
// (constant bank), so every policy FMA reads its weight as an immediate operand.
struct RolloutParams {
    int64_t n;
    int64_t n_tasks;  // warp tasks of 32*EPT envs
    uint32_t T, t0, env_offset, salt_a, salt_r;
    const float *init_planes;  // nullptr: start states of time t0
    int64_t init_stride;
    float *out_planes;  // nullptr: final state not stored
    int64_t out_stride;
    uint32_t *ep_len_io;
    float *ep_return_sum;
    uint32_t *ep_count;
    unsigned long long *totals;
    float *reward_stream;
    uint32_t *done_bits;
    uint32_t *action_bits;
    float *trajectory;
    uint32_t max_steps;              // episode step limit, 0 = none
    const uint32_t *action_bits_in;  // [T][words] supplied actions or nullptr
    const float *start_in;           // [T][4][n] supplied start states or nullptr
    const float *env_weights;        // [10][n] one linear policy per env (policy kind 6) or nullptr
    // largest policy: the network with 64 hidden units, 7*64 + 2 floats; twice the room, because the
    // deferred-restart kernel reads every shared weight as a (w, w) pair
    float w[900];
};

struct LaunchTuning {
    int rollout_block = 0;        // 0: 128 for very small batches, 256 otherwise
    int rollout_ept = 0;          // 0: chosen per policy and batch size
    int rollout_coop = 0;         // 0: chosen per batch size; 1 restarts by the warp; 2 per lane (ept 1);
                                  // 3 per lane, computed ahead; 4 handed over by a producer warp;
                                  // 5 deferred (two envs per thread, own clock per env, restarts every few trips)
    int rollout_ctas_per_sm = 0;  // 0: one task per warp (non-persistent grid)
    int rollout_defer = 0;        // deferred-restart kernel: trips between restart passes (0: by horizon and policy)
    int step_block = 64;
    // Below this many envs the one-env-per-thread kernel is used: a small batch is latency-bound,
    // and four envs in sequence per thread take longer than four times as many threads
    // (65,536 envs, graph replay: 1.9 us vs 2.5 us per launch; equal at 262,144; slower above).
    int step_vec_min_envs = 262144;
    // 1: launch the step kernel with programmatic stream serialization, so that a launch's
    // memory-independent preamble overlaps the tail of the launch before it (same stream).
    // Measured per launch, 65,536 envs: 4.10 -> 2.38 us issued eagerly, 2.01 -> 1.46 us from a graph.
    // The ladder's 46 one-op kernels are launched the same way (each waits for its predecessor
    // before its first access): 16,777,216 envs 1.209 -> 1.106 ms per step, 4,194,304 envs 0.386 -> 0.295 ms.
    int step_pdl = 1;
};
extern LaunchTuning g_tuning;

void count_launch(int n = 1);
int sm_count();

cudaError_t launch_step(const StepParams &p, bool vec, cudaStream_t s);
cudaError_t launch_fill_start(float *planes, int64_t stride, int64_t n, uint32_t env_offset, uint32_t salt_r,
                              uint32_t t, cudaStream_t s);
cudaError_t launch_actions(uint8_t *out, int64_t n, uint32_t env_offset, uint32_t salt_a, uint32_t t,
                           cudaStream_t s);
cudaError_t launch_rollout(RolloutParams &p, int policy, bool streams, bool contracted, cudaStream_t s);
cudaError_t launch_rollout_contracted(RolloutParams &p, int policy, bool streams, cudaStream_t s);
// the producer-assisted kernel for very small batches, and whether a call is one it covers
bool rollout_assisted_applies(const RolloutParams &p, int policy, bool streams);
cudaError_t launch_rollout_assisted(RolloutParams &p, bool contracted, cudaStream_t s);
// the deferred-restart kernel (large batches, no per-step streams), and whether a call is one it covers
bool rollout_deferred_applies(const RolloutParams &p, int policy, bool streams);
cudaError_t launch_rollout_deferred(RolloutParams &p, int policy, bool contracted, cudaStream_t s);
cudaError_t launch_rollout_deferred_wide(RolloutParams &p, int policy, bool contracted, cudaStream_t s);  // policies 4, 5, 7
// the MLP policies (kinds 2, 4, 5, 7), canonical and contracted arithmetic; mode and shape as
// chosen by launch_rollout_arith
cudaError_t launch_rollout_networks(RolloutParams &p, int policy, int mode, int shape, cudaStream_t s);
cudaError_t launch_rollout_networks_contracted(RolloutParams &p, int policy, int mode, int shape, cudaStream_t s);
cudaError_t launch_sincos_selftest(uint32_t lo_bits, uint32_t hi_bits, unsigned long long *mismatches,
                                   cudaStream_t s);

cudaError_t launch_sincos_accuracy(uint32_t lo_bits, uint32_t hi_bits, unsigned long long *out, cudaStream_t s);
cudaError_t launch_tanh_accuracy(uint32_t lo_bits, uint32_t hi_bits, unsigned long long *out, cudaStream_t s);
cudaError_t launch_pipe_rate(int kind, const float *seed, float *sink, int iters, int *threads, cudaStream_t s);
cudaError_t launch_arith_selftest(unsigned long long *out, cudaStream_t s);
cudaError_t launch_pair_selftest(unsigned long long count, uint32_t seed, unsigned long long *out, cudaStream_t s);
cudaError_t launch_tame_div_selftest(uint32_t den_step, unsigned long long *out, cudaStream_t s);

// The per-op ladder. Workspace layout is private to ladder_kernels.cu.
size_t ladder_workspace_bytes(int64_t n);
int ladder_launch_count(bool hashed_action);
cudaError_t launch_ladder(const StepParams &p, void *workspace, cudaStream_t s);

// Defined in capi.cu, for entry points that live in other translation units.
cudaStream_t thread_stream();                    // stream chosen by cp_set_stream on this thread
int set_error(int code, const char *text);       // records the text for cp_last_error, returns code
void adopt_step(cp_state *state, cp_state *out_state, uint32_t steps);  // out takes seed/offset, t + steps

}  // namespace cp
