// extern "C" boundary of libcartpole: argument checking, handle bookkeeping,
// stream selection and launch of the kernels. No arithmetic of the method lives
// here except the two per-launch salts of the counter hash.
#include <atomic>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>

#include "../../include/cartpole.h"
#include "cartpole_device.cuh"
#include "cartpole_internal.h"

struct cp_state {
    int64_t n;
    int64_t stride;
    uint32_t seed, t, env_offset;
    float *planes;
    bool owns;
    void (*release)(void *);  // how owned planes go back: the allocator's release, or NULL = cudaFree
};

namespace cp {

LaunchTuning g_tuning;
static std::atomic<uint64_t> g_launches{0};
void count_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }

int sm_count() {
    static int cached = 0;
    if (cached == 0) {
        int dev = 0, sms = 0;
        if (cudaGetDevice(&dev) == cudaSuccess &&
            cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && sms > 0)
            cached = sms;
        else
            return 148;
    }
    return cached;
}

}  // namespace cp

namespace {

thread_local cudaStream_t tl_stream = nullptr;
thread_local char tl_error[512] = "";

// Device allocator of cp_reset (cp_set_allocator); both NULL = cudaMalloc / cudaFree.
std::mutex g_alloc_mu;
void *(*g_alloc)(size_t) = nullptr;
void (*g_release)(void *) = nullptr;

int fail(int code, const char *fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(tl_error, sizeof tl_error, fmt, ap);
    va_end(ap);
    return code;
}

int cuda_fail(cudaError_t e, const char *what) {
    return fail(CP_ECUDA, "%s: %s", what, cudaGetErrorString(e));
}

inline bool is_aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

bool state_vec_ok(const cp_state *s) { return is_aligned(s->planes, 16) && (s->stride % 4) == 0; }

int check_state(const cp_state *s, const char *name) {
    if (!s) return fail(CP_EINVAL, "%s is NULL", name);
    if (!s->planes || s->n <= 0 || s->stride < s->n) return fail(CP_EINVAL, "%s is not a valid batch", name);
    return CP_OK;
}

int check_policy(const cp_policy *policy, int *kind) {
    *kind = policy ? policy->kind : CP_POLICY_RANDOM;
    if (*kind != CP_POLICY_RANDOM && *kind != CP_POLICY_LINEAR && *kind != CP_POLICY_MLP &&
        *kind != CP_POLICY_MLP32 && *kind != CP_POLICY_MLP64 && *kind != CP_POLICY_LINEAR_PER_ENV &&
        *kind != CP_POLICY_MLP_DEEP)
        return fail(CP_EINVAL, "unknown policy kind %d", *kind);
    if (*kind != CP_POLICY_RANDOM && !policy->weights) return fail(CP_EINVAL, "policy weights are NULL");
    if (*kind == CP_POLICY_LINEAR_PER_ENV && !is_aligned(policy->weights, 4))
        return fail(CP_EINVAL, "per-environment weights are not float-aligned");
    return CP_OK;
}

int check_range(int64_t n_envs, uint32_t env_offset) {
    if (n_envs <= 0) return fail(CP_EINVAL, "n_envs must be positive (got %lld)", (long long)n_envs);
    if ((uint64_t)n_envs + env_offset > (1ull << 32))
        return fail(CP_EINVAL, "env_offset + n_envs exceeds 2^32 environment ids");
    return CP_OK;
}

void fill_step_params(cp::StepParams &p, const cp_state *in, cp_state *out, const uint8_t *action, float *reward,
                      uint8_t *done) {
    p.in = in->planes;
    p.in_stride = in->stride;
    p.out = out->planes;
    p.out_stride = out->stride;
    p.n = in->n;
    p.t = in->t;
    p.env_offset = in->env_offset;
    p.salt_a = cp::salt(in->seed, 0u);
    p.salt_r = cp::salt(in->seed, 1u);
    p.action = action;
    p.reward = reward;
    p.done = done;
    p.ep_len = nullptr;
    p.max_steps = 0;
}

int check_step_args(cp_state *state, cp_state *out_state) {
    int rc;
    if ((rc = check_state(state, "state")) != CP_OK) return rc;
    if ((rc = check_state(out_state, "out_state")) != CP_OK) return rc;
    if (out_state->n != state->n) return fail(CP_EINVAL, "out_state has %lld envs, state has %lld",
                                              (long long)out_state->n, (long long)state->n);
    if (state->t >= (1u << 30)) return fail(CP_EINVAL, "global step out of range");
    return CP_OK;
}

void advance(cp_state *state, cp_state *out_state, uint32_t steps) {
    out_state->seed = state->seed;
    out_state->env_offset = state->env_offset;
    out_state->t = state->t + steps;
}

// Rollout shared by cp_rollout / cp_rollout_shard / cp_rollout_from / cp_rollout_host.
int rollout_impl(uint32_t env_offset, int64_t n_envs, int64_t T, uint32_t seed, uint32_t t0, const cp_policy *policy,
                 const cp_returns *ret, const float *init_planes, int64_t init_stride, float *out_planes,
                 int64_t out_stride, uint32_t *ep_len, uint32_t max_steps = 0,
                 const uint32_t *action_bits_in = nullptr, uint32_t arithmetic = CP_ARITH_EXACT,
                 const float *start_states_in = nullptr) {
    int kind, rc;
    if (start_states_in && !is_aligned(start_states_in, 4)) return fail(CP_EINVAL, "start_states_in is misaligned");
    if (arithmetic != CP_ARITH_EXACT && arithmetic != CP_ARITH_CONTRACTED)
        return fail(CP_EINVAL, "arithmetic must be CP_ARITH_EXACT or CP_ARITH_CONTRACTED (got %u)", arithmetic);
    if ((rc = check_range(n_envs, env_offset)) != CP_OK) return rc;
    if (T <= 0 || T > CP_MAX_T || (int64_t)t0 + T > CP_MAX_T)
        return fail(CP_EINVAL, "T must be in [1, 2^30] and t0 + T <= 2^30 (got T=%lld, t0=%u)", (long long)T, t0);
    if ((rc = check_policy(policy, &kind)) != CP_OK) return rc;
    if (!ret) return fail(CP_EINVAL, "returns is NULL");
    if (ret->totals && !is_aligned(ret->totals, 8)) return fail(CP_EINVAL, "totals must be 8-byte aligned");
    // every other output is stored in 4-byte units: a misaligned pointer would fault on the device
    const struct { const void *p; const char *name; } four_byte[] = {
        {ret->ep_return_sum, "ep_return_sum"}, {ret->ep_count, "ep_count"}, {ret->reward_stream, "reward_stream"},
        {ret->done_bits, "done_bits"}, {ret->action_bits, "action_bits"}, {ret->trajectory, "trajectory"},
        {out_planes, "final_state"}, {init_planes, "state planes"}, {ep_len, "ep_len"}, {action_bits_in, "action_bits_in"}};
    for (const auto &q : four_byte)
        if (q.p && !is_aligned(q.p, 4)) return fail(CP_EINVAL, "%s is not 4-byte aligned", q.name);
    cp::RolloutParams p;
    memset(&p, 0, sizeof p);
    p.n = n_envs;
    p.T = (uint32_t)T;
    p.t0 = t0;
    p.env_offset = env_offset;
    p.salt_a = cp::salt(seed, 0u);
    p.salt_r = cp::salt(seed, 1u);
    p.init_planes = init_planes;
    p.init_stride = init_stride;
    p.out_planes = out_planes;
    p.out_stride = out_stride;
    p.ep_len_io = ep_len;
    p.ep_return_sum = ret->ep_return_sum;
    p.ep_count = ret->ep_count;
    p.totals = reinterpret_cast<unsigned long long *>(ret->totals);
    p.reward_stream = ret->reward_stream;
    p.done_bits = ret->done_bits;
    p.action_bits = ret->action_bits;
    p.trajectory = ret->trajectory;
    p.max_steps = max_steps;
    p.action_bits_in = action_bits_in;
    p.start_in = start_states_in;
    if (kind == CP_POLICY_LINEAR) memcpy(p.w, policy->weights, 10 * sizeof(float));
    if (kind == CP_POLICY_MLP) memcpy(p.w, policy->weights, 114 * sizeof(float));
    if (kind == CP_POLICY_MLP32) memcpy(p.w, policy->weights, 226 * sizeof(float));
    if (kind == CP_POLICY_MLP64) memcpy(p.w, policy->weights, 450 * sizeof(float));
    if (kind == CP_POLICY_MLP_DEEP) memcpy(p.w, policy->weights, 386 * sizeof(float));
    if (kind == CP_POLICY_LINEAR_PER_ENV) p.env_weights = policy->weights;  // DEVICE [10][n_envs]
    const bool streams = p.reward_stream || p.done_bits || p.action_bits || p.trajectory;
    cudaError_t e = cp::launch_rollout(p, kind, streams, arithmetic == CP_ARITH_CONTRACTED, tl_stream);
    if (e != cudaSuccess) return cuda_fail(e, "rollout launch");
    return CP_OK;
}

// Library-owned device staging for the HOST-buffer entry points.
struct Staging {
    std::mutex mu;
    void *buf = nullptr;
    size_t bytes = 0;
} g_staging;

int staging_reserve(size_t bytes, void **out) {
    if (g_staging.bytes < bytes) {
        if (g_staging.buf) {
            cudaError_t e = cudaFree(g_staging.buf);
            g_staging.buf = nullptr;
            g_staging.bytes = 0;
            if (e != cudaSuccess) return cuda_fail(e, "cudaFree(staging)");
        }
        cudaError_t e = cudaMalloc(&g_staging.buf, bytes);
        if (e != cudaSuccess) {
            g_staging.buf = nullptr;
            (void)cudaGetLastError();
            return fail(CP_ENOMEM, "cudaMalloc(%zu) for staging failed: %s", bytes, cudaGetErrorString(e));
        }
        g_staging.bytes = bytes;
    }
    *out = g_staging.buf;
    return CP_OK;
}

inline size_t round_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// Device-side address of a page-locked host range [p, p + bytes), or nullptr if the range is
// pageable (or not wholly inside one registered allocation).
void *device_view_of_pinned(void *p, size_t bytes) {
    cudaPointerAttributes a0, a1;
    if (cudaPointerGetAttributes(&a0, p) != cudaSuccess || a0.type != cudaMemoryTypeHost || !a0.devicePointer) {
        (void)cudaGetLastError();
        return nullptr;
    }
    if (cudaPointerGetAttributes(&a1, static_cast<char *>(p) + bytes - 1) != cudaSuccess ||
        a1.type != cudaMemoryTypeHost || !a1.devicePointer ||
        static_cast<char *>(a1.devicePointer) - static_cast<char *>(a0.devicePointer) != (ptrdiff_t)(bytes - 1)) {
        (void)cudaGetLastError();
        return nullptr;
    }
    return a0.devicePointer;
}

}  // namespace

// Accessors for entry points that live in other translation units.
namespace cp {
cudaStream_t thread_stream() { return tl_stream; }
int set_error(int code, const char *text) { return fail(code, "%s", text); }
void adopt_step(cp_state *state, cp_state *out_state, uint32_t steps) { advance(state, out_state, steps); }
}  // namespace cp

extern "C" {

cp_state *cp_reset(int64_t n_envs, uint32_t seed) {
    if (check_range(n_envs, 0) != CP_OK) return nullptr;
    cp_state *s = new (std::nothrow) cp_state;
    if (!s) {
        fail(CP_ENOMEM, "out of host memory");
        return nullptr;
    }
    s->n = n_envs;
    s->stride = (n_envs + 3) / 4 * 4;
    s->seed = seed;
    s->t = 0;
    s->env_offset = 0;
    s->owns = true;
    s->planes = nullptr;
    s->release = nullptr;
    const size_t bytes = (size_t)s->stride * 4 * sizeof(float);
    void *(*alloc)(size_t);
    {
        std::lock_guard<std::mutex> lock(g_alloc_mu);
        alloc = g_alloc;
        s->release = g_release;
    }
    cudaError_t e;
    if (alloc) {
        s->planes = static_cast<float *>(alloc(bytes));
        if (!s->planes || !is_aligned(s->planes, 16)) {
            fail(CP_ENOMEM, "the allocator returned %s for %zu bytes", s->planes ? "a pointer not 16-byte aligned" : "NULL",
                 bytes);
            if (s->planes && s->release) s->release(s->planes);
            delete s;
            return nullptr;
        }
    } else {
        e = cudaMalloc(reinterpret_cast<void **>(&s->planes), bytes);
        if (e != cudaSuccess) {
            (void)cudaGetLastError();
            fail(CP_ENOMEM, "cudaMalloc of %lld envs failed: %s", (long long)n_envs, cudaGetErrorString(e));
            delete s;
            return nullptr;
        }
    }
    // pad lanes hold start states too, so vector loads never see uninitialised memory
    e = cp::launch_fill_start(s->planes, s->stride, s->stride, 0, cp::salt(seed, 1u), 0, tl_stream);
    if (e != cudaSuccess) {
        cuda_fail(e, "start-state launch");
        if (s->release) s->release(s->planes); else cudaFree(s->planes);
        delete s;
        return nullptr;
    }
    return s;
}

int cp_set_allocator(void *(*alloc)(size_t), void (*release)(void *)) {
    if ((alloc == nullptr) != (release == nullptr))
        return fail(CP_EINVAL, "alloc and release must be given together (or both NULL for cudaMalloc / cudaFree)");
    std::lock_guard<std::mutex> lock(g_alloc_mu);
    g_alloc = alloc;
    g_release = release;
    return CP_OK;
}

cp_state *cp_wrap(float *planes, int64_t n_envs, int64_t plane_stride, uint32_t seed, uint32_t t,
                  uint32_t env_offset) {
    if (!planes || !is_aligned(planes, 4)) {
        fail(CP_EINVAL, "planes is NULL or not float-aligned");
        return nullptr;
    }
    if (check_range(n_envs, env_offset) != CP_OK) return nullptr;
    if (plane_stride < n_envs) {
        fail(CP_EINVAL, "plane_stride %lld < n_envs %lld", (long long)plane_stride, (long long)n_envs);
        return nullptr;
    }
    if (t > (1u << 30)) {
        fail(CP_EINVAL, "global step out of range");
        return nullptr;
    }
    cp_state *s = new (std::nothrow) cp_state;
    if (!s) {
        fail(CP_ENOMEM, "out of host memory");
        return nullptr;
    }
    *s = cp_state{n_envs, plane_stride, seed, t, env_offset, planes, false, nullptr};
    return s;
}

int cp_fill_start(cp_state *state) {
    int rc = check_state(state, "state");
    if (rc != CP_OK) return rc;
    cudaError_t e = cp::launch_fill_start(state->planes, state->stride, state->n, state->env_offset,
                                          cp::salt(state->seed, 1u), state->t, tl_stream);
    return e == cudaSuccess ? CP_OK : cuda_fail(e, "start-state launch");
}

int cp_set_time(cp_state *state, uint32_t t) {
    if (!state) return fail(CP_EINVAL, "state is NULL");
    if (t > (1u << 30)) return fail(CP_EINVAL, "global step out of range");
    state->t = t;
    return CP_OK;
}

void cp_free(cp_state *state) {
    if (!state) return;
    if (state->owns && state->planes) {
        if (state->release) state->release(state->planes); else cudaFree(state->planes);
    }
    delete state;
}

int cp_state_info(const cp_state *state, int64_t *n_envs, int64_t *plane_stride, uint32_t *seed, uint32_t *t,
                  uint32_t *env_offset, float **planes) {
    if (!state) return fail(CP_EINVAL, "state is NULL");
    if (n_envs) *n_envs = state->n;
    if (plane_stride) *plane_stride = state->stride;
    if (seed) *seed = state->seed;
    if (t) *t = state->t;
    if (env_offset) *env_offset = state->env_offset;
    if (planes) *planes = state->planes;
    return CP_OK;
}

static int step_impl(cp_state *state, const uint8_t *action, cp_state *out_state, float *reward, uint8_t *done,
                     uint32_t *ep_len, uint32_t max_steps) {
    int rc = check_step_args(state, out_state);
    if (rc != CP_OK) return rc;
    if (reward && !is_aligned(reward, 4)) return fail(CP_EINVAL, "reward is not float-aligned");
    if (ep_len && !is_aligned(ep_len, 4)) return fail(CP_EINVAL, "ep_len is not 4-byte aligned");
    if (max_steps && !ep_len) return fail(CP_EINVAL, "an episode step limit needs the ep_len counters");
    cp::StepParams p;
    fill_step_params(p, state, out_state, action, reward, done);
    p.ep_len = ep_len;
    p.max_steps = max_steps;
    const bool vec = state->n >= cp::g_tuning.step_vec_min_envs && state_vec_ok(state) && state_vec_ok(out_state) &&
                     (!reward || is_aligned(reward, 16)) && (!done || is_aligned(done, 4)) &&
                     (!action || is_aligned(action, 4)) && (!ep_len || is_aligned(ep_len, 16));
    cudaError_t e = cp::launch_step(p, vec, tl_stream);
    if (e != cudaSuccess) return cuda_fail(e, "step launch");
    advance(state, out_state, 1);
    return CP_OK;
}

int cp_step(cp_state *state, const uint8_t *action, cp_state *out_state, float *reward, uint8_t *done) {
    return step_impl(state, action, out_state, reward, done, nullptr, 0);
}

int cp_step_ex(cp_state *state, const uint8_t *action, cp_state *out_state, float *reward, uint8_t *done,
               uint32_t *ep_len, uint32_t max_episode_steps) {
    return step_impl(state, action, out_state, reward, done, ep_len, max_episode_steps);
}

int cp_step_repeat(cp_state *state, int64_t k, float *reward, uint8_t *done) {
    if (k < 0 || k > CP_MAX_T) return fail(CP_EINVAL, "k must be in [0, 2^30]");
    for (int64_t i = 0; i < k; ++i) {
        int rc = cp_step(state, nullptr, state, reward, done);
        if (rc != CP_OK) return rc;
    }
    return CP_OK;
}

size_t cp_unfused_workspace_bytes(int64_t n_envs) {
    return n_envs > 0 ? cp::ladder_workspace_bytes(n_envs) : 0;
}

int cp_step_unfused(cp_state *state, const uint8_t *action, cp_state *out_state, float *reward, uint8_t *done,
                    void *workspace, size_t workspace_bytes) {
    int rc = check_step_args(state, out_state);
    if (rc != CP_OK) return rc;
    if (!reward || !done) return fail(CP_EINVAL, "reward and done must not be NULL for the unfused step");
    if (!is_aligned(reward, 4)) return fail(CP_EINVAL, "reward is not float-aligned");
    if (!state_vec_ok(state) || !state_vec_ok(out_state))
        return fail(CP_EINVAL, "the unfused step needs 16-byte aligned planes with plane_stride %% 4 == 0");
    if (state->planes == out_state->planes) return fail(CP_EINVAL, "the unfused step cannot run in place");
    if (!workspace || !is_aligned(workspace, 256)) return fail(CP_EINVAL, "workspace is NULL or not 256-byte aligned");
    if (workspace_bytes < cp::ladder_workspace_bytes(state->n))
        return fail(CP_ENOMEM, "workspace has %zu bytes, %zu needed", workspace_bytes,
                    cp::ladder_workspace_bytes(state->n));
    cp::StepParams p;
    fill_step_params(p, state, out_state, action, reward, done);
    cudaError_t e = cp::launch_ladder(p, workspace, tl_stream);
    if (e != cudaSuccess) return cuda_fail(e, "ladder launch");
    advance(state, out_state, 1);
    return CP_OK;
}

int cp_actions(int64_t n_envs, uint32_t seed, uint32_t t, uint32_t env_offset, uint8_t *out) {
    int rc = check_range(n_envs, env_offset);
    if (rc != CP_OK) return rc;
    if (!out) return fail(CP_EINVAL, "out is NULL");
    cudaError_t e = cp::launch_actions(out, n_envs, env_offset, cp::salt(seed, 0u), t, tl_stream);
    return e == cudaSuccess ? CP_OK : cuda_fail(e, "actions launch");
}

int cp_rollout(int64_t n_envs, int64_t T, uint32_t seed, const cp_policy *policy, const cp_returns *returns) {
    return cp_rollout_shard(0, n_envs, T, seed, policy, returns);
}

int cp_rollout_shard(uint32_t env_offset, int64_t n_envs, int64_t T, uint32_t seed, const cp_policy *policy,
                     const cp_returns *returns) {
    if (!returns) return fail(CP_EINVAL, "returns is NULL");
    return rollout_impl(env_offset, n_envs, T, seed, 0, policy, returns, nullptr, 0, returns->final_state, n_envs,
                        nullptr);
}

int cp_rollout_from(cp_state *state, int64_t T, uint32_t *ep_len, const cp_policy *policy,
                    const cp_returns *returns) {
    int rc = check_state(state, "state");
    if (rc != CP_OK) return rc;
    rc = rollout_impl(state->env_offset, state->n, T, state->seed, state->t, policy, returns, state->planes,
                      state->stride, state->planes, state->stride, ep_len);
    if (rc != CP_OK) return rc;
    state->t += (uint32_t)T;
    return CP_OK;
}

int cp_rollout_ex(const cp_rollout_args *a) {
    if (!a) return fail(CP_EINVAL, "args is NULL");
    if (a->struct_size != sizeof(cp_rollout_args))
        return fail(CP_EINVAL, "struct_size is %u, this library expects %zu", a->struct_size, sizeof(cp_rollout_args));
    if (!a->returns) return fail(CP_EINVAL, "returns is NULL");
    if (a->action_bits_in && !is_aligned(a->action_bits_in, 4)) return fail(CP_EINVAL, "action_bits_in is misaligned");
    if (a->state) {
        int rc = check_state(a->state, "state");
        if (rc != CP_OK) return rc;
        cp_state *st = a->state;
        rc = rollout_impl(st->env_offset, st->n, a->T, st->seed, st->t, a->policy, a->returns, st->planes, st->stride,
                          st->planes, st->stride, a->ep_len, a->max_episode_steps, a->action_bits_in, a->arithmetic,
                          a->start_states_in);
        if (rc != CP_OK) return rc;
        st->t += (uint32_t)a->T;
        return CP_OK;
    }
    return rollout_impl(a->env_offset, a->n_envs, a->T, a->seed, a->t0, a->policy, a->returns, nullptr, 0,
                        a->returns->final_state, a->n_envs, a->ep_len, a->max_episode_steps, a->action_bits_in,
                        a->arithmetic, a->start_states_in);
}

int cp_rollout_host(int64_t n_envs, int64_t T, uint32_t seed, const cp_policy *policy, float *h_ep_return_sum,
                    uint32_t *h_ep_count, uint64_t *h_totals) {
    return cp_rollout_host_shard(0, n_envs, T, seed, policy, h_ep_return_sum, h_ep_count, h_totals);
}

int cp_rollout_host_shard(uint32_t env_offset, int64_t n_envs, int64_t T, uint32_t seed, const cp_policy *policy,
                          float *h_ep_return_sum, uint32_t *h_ep_count, uint64_t *h_totals) {
    int rc = check_range(n_envs, env_offset);
    if (rc != CP_OK) return rc;
    if (!h_ep_return_sum || !h_ep_count || !h_totals) return fail(CP_EINVAL, "a host output pointer is NULL");
    std::lock_guard<std::mutex> lock(g_staging.mu);
    // Page-locked host buffers are addressable from the device: the kernel then stores each env's
    // two results straight into host memory as its warp finishes (8 B/env spread over the whole
    // launch), instead of a device buffer plus a copy after the kernel. Pageable buffers take the
    // staged route.
    float *d_ret = static_cast<float *>(device_view_of_pinned(h_ep_return_sum, (size_t)n_envs * 4));
    uint32_t *d_cnt = static_cast<uint32_t *>(device_view_of_pinned(h_ep_count, (size_t)n_envs * 4));
    const bool direct = d_ret && d_cnt;
    const size_t per = direct ? 0 : round_up((size_t)n_envs * 4, 256);
    void *buf;
    if ((rc = staging_reserve(2 * per + 256, &buf)) != CP_OK) return rc;
    char *base = static_cast<char *>(buf);
    cp_returns r;
    memset(&r, 0, sizeof r);
    r.ep_return_sum = direct ? d_ret : reinterpret_cast<float *>(base);
    r.ep_count = direct ? d_cnt : reinterpret_cast<uint32_t *>(base + per);
    r.totals = reinterpret_cast<uint64_t *>(base + 2 * per);
    cudaError_t e = cudaMemsetAsync(r.totals, 0, 16, tl_stream);
    if (e != cudaSuccess) return cuda_fail(e, "cudaMemsetAsync");
    if ((rc = rollout_impl(env_offset, n_envs, T, seed, 0, policy, &r, nullptr, 0, nullptr, 0, nullptr)) != CP_OK)
        return rc;
    if (!direct) {
        e = cudaMemcpyAsync(h_ep_return_sum, r.ep_return_sum, (size_t)n_envs * 4, cudaMemcpyDeviceToHost, tl_stream);
        if (e == cudaSuccess)
            e = cudaMemcpyAsync(h_ep_count, r.ep_count, (size_t)n_envs * 4, cudaMemcpyDeviceToHost, tl_stream);
    }
    if (e == cudaSuccess) e = cudaMemcpyAsync(h_totals, r.totals, 16, cudaMemcpyDeviceToHost, tl_stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(tl_stream);
    return e == cudaSuccess ? CP_OK : cuda_fail(e, "rollout copy-out");
}

int cp_step_host(int64_t n_envs, uint32_t seed, uint32_t t, const float *h_planes_in, const uint8_t *h_action,
                 float *h_planes_out, float *h_reward, uint8_t *h_done) {
    int rc = check_range(n_envs, 0);
    if (rc != CP_OK) return rc;
    if (!h_planes_in || !h_planes_out || !h_reward || !h_done) return fail(CP_EINVAL, "a host pointer is NULL");
    if (t >= (1u << 30)) return fail(CP_EINVAL, "global step out of range");
    std::lock_guard<std::mutex> lock(g_staging.mu);
    const int64_t stride = (n_envs + 63) / 64 * 64;
    const size_t plane_bytes = (size_t)stride * 4;
    const size_t byte_plane = round_up((size_t)n_envs, 256);
    void *buf;
    if ((rc = staging_reserve(5 * plane_bytes + 2 * byte_plane, &buf)) != CP_OK) return rc;
    char *base = static_cast<char *>(buf);
    float *d_planes = reinterpret_cast<float *>(base);
    float *d_reward = reinterpret_cast<float *>(base + 4 * plane_bytes);
    uint8_t *d_done = reinterpret_cast<uint8_t *>(base + 5 * plane_bytes);
    uint8_t *d_action = d_done + byte_plane;
    cudaError_t e = cudaMemcpy2DAsync(d_planes, plane_bytes, h_planes_in, (size_t)n_envs * 4, (size_t)n_envs * 4, 4,
                                      cudaMemcpyHostToDevice, tl_stream);
    if (e == cudaSuccess && h_action)
        e = cudaMemcpyAsync(d_action, h_action, (size_t)n_envs, cudaMemcpyHostToDevice, tl_stream);
    if (e != cudaSuccess) return cuda_fail(e, "step copy-in");
    cp_state s{n_envs, stride, seed, t, 0, d_planes, false};
    if ((rc = cp_step(&s, h_action ? d_action : nullptr, &s, d_reward, d_done)) != CP_OK) return rc;
    e = cudaMemcpy2DAsync(h_planes_out, (size_t)n_envs * 4, d_planes, plane_bytes, (size_t)n_envs * 4, 4,
                          cudaMemcpyDeviceToHost, tl_stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(h_reward, d_reward, (size_t)n_envs * 4, cudaMemcpyDeviceToHost, tl_stream);
    if (e == cudaSuccess) e = cudaMemcpyAsync(h_done, d_done, (size_t)n_envs, cudaMemcpyDeviceToHost, tl_stream);
    if (e == cudaSuccess) e = cudaStreamSynchronize(tl_stream);
    return e == cudaSuccess ? CP_OK : cuda_fail(e, "step copy-out");
}

void cp_shutdown(void) {
    std::lock_guard<std::mutex> lock(g_staging.mu);
    if (g_staging.buf) {
        cudaDeviceSynchronize();
        cudaFree(g_staging.buf);
        g_staging.buf = nullptr;
        g_staging.bytes = 0;
    }
}

void cp_set_stream(void *cuda_stream) { tl_stream = static_cast<cudaStream_t>(cuda_stream); }

int cp_tune(const char *key, int value) {
    if (!key) return fail(CP_EINVAL, "key is NULL");
    if (!strcmp(key, "rollout_block")) {
        if (value != 0 && (value < 32 || value > 256 || value % 32))
            return fail(CP_EINVAL, "rollout_block must be 0 or 32..256, multiple of 32");
        cp::g_tuning.rollout_block = value;
    } else if (!strcmp(key, "rollout_ept")) {
        if (value != 0 && value != 1 && value != 2) return fail(CP_EINVAL, "rollout_ept must be 0, 1 or 2");
        cp::g_tuning.rollout_ept = value;
    } else if (!strcmp(key, "rollout_coop")) {
        if (value < 0 || value > 5) return fail(CP_EINVAL, "rollout_coop must be 0..5");
        cp::g_tuning.rollout_coop = value;
    } else if (!strcmp(key, "rollout_defer")) {
        if (value != 0 && value != 2 && value != 3 && value != 4 && value != 6 && value != 8)
            return fail(CP_EINVAL, "rollout_defer must be 0, 2, 3, 4, 6 or 8");
        cp::g_tuning.rollout_defer = value;
    } else if (!strcmp(key, "rollout_ctas_per_sm")) {
        if (value < 0 || value > 1024) return fail(CP_EINVAL, "rollout_ctas_per_sm must be 0..1024");
        cp::g_tuning.rollout_ctas_per_sm = value;
    } else if (!strcmp(key, "step_block")) {
        if (value < 32 || value > 256 || value % 32) return fail(CP_EINVAL, "step_block must be 32..256, multiple of 32");
        cp::g_tuning.step_block = value;
    } else if (!strcmp(key, "step_pdl")) {
        if (value != 0 && value != 1) return fail(CP_EINVAL, "step_pdl must be 0 or 1");
        cp::g_tuning.step_pdl = value;
    } else if (!strcmp(key, "step_vec_min_envs")) {
        if (value < 0) return fail(CP_EINVAL, "step_vec_min_envs must be >= 0");
        cp::g_tuning.step_vec_min_envs = value;
    } else {
        return fail(CP_EINVAL, "unknown tuning key '%s'", key);
    }
    return CP_OK;
}

uint64_t cp_launch_count(void) { return cp::g_launches.load(std::memory_order_relaxed); }

int cp_selftest_sincos(uint32_t lo_bits, uint32_t hi_bits, uint64_t *mismatches) {
    if (!mismatches || !is_aligned(mismatches, 8)) return fail(CP_EINVAL, "mismatches is NULL or misaligned");
    if (lo_bits > hi_bits || hi_bits >= 0x7F800000u) return fail(CP_EINVAL, "need lo <= hi, both finite and non-negative");
    cudaError_t e = cp::launch_sincos_selftest(lo_bits, hi_bits, reinterpret_cast<unsigned long long *>(mismatches),
                                               tl_stream);
    return e == cudaSuccess ? CP_OK : cuda_fail(e, "self-test launch");
}

int cp_selftest_sincos_accuracy(uint32_t lo_bits, uint32_t hi_bits, uint64_t *out) {
    if (!out || !is_aligned(out, 8)) return fail(CP_EINVAL, "out is NULL or misaligned");
    if (lo_bits > hi_bits || hi_bits >= 0x7F800000u) return fail(CP_EINVAL, "need lo <= hi, both finite and non-negative");
    cudaError_t e = cp::launch_sincos_accuracy(lo_bits, hi_bits, reinterpret_cast<unsigned long long *>(out), tl_stream);
    return e == cudaSuccess ? CP_OK : cuda_fail(e, "self-test launch");
}

int cp_selftest_tanh(uint32_t lo_bits, uint32_t hi_bits, uint64_t *out) {
    if (!out || !is_aligned(out, 8)) return fail(CP_EINVAL, "out is NULL or misaligned");
    if (lo_bits > hi_bits || hi_bits >= 0x7F800000u) return fail(CP_EINVAL, "need lo <= hi, both finite and non-negative");
    cudaError_t e = cp::launch_tanh_accuracy(lo_bits, hi_bits, reinterpret_cast<unsigned long long *>(out), tl_stream);
    return e == cudaSuccess ? CP_OK : cuda_fail(e, "self-test launch");
}

int cp_selftest_arith(uint64_t *out) {
    if (!out || !is_aligned(out, 8)) return fail(CP_EINVAL, "out is NULL or misaligned");
    cudaError_t e = cp::launch_arith_selftest(reinterpret_cast<unsigned long long *>(out), tl_stream);
    return e == cudaSuccess ? CP_OK : cuda_fail(e, "self-test launch");
}

int cp_selftest_pair(uint64_t count, uint32_t seed, uint64_t *out) {
    if (!out || !is_aligned(out, 8)) return fail(CP_EINVAL, "out is NULL or misaligned");
    if (count == 0) return fail(CP_EINVAL, "count must be >= 1");
    cudaError_t e = cp::launch_pair_selftest(count, seed, reinterpret_cast<unsigned long long *>(out), tl_stream);
    return e == cudaSuccess ? CP_OK : cuda_fail(e, "self-test launch");
}

int cp_selftest_tame_div(uint32_t den_step, uint64_t *out) {
    if (!out || !is_aligned(out, 8)) return fail(CP_EINVAL, "out is NULL or misaligned");
    if (den_step == 0) return fail(CP_EINVAL, "den_step must be >= 1");
    cudaError_t e = cp::launch_tame_div_selftest(den_step, reinterpret_cast<unsigned long long *>(out), tl_stream);
    return e == cudaSuccess ? CP_OK : cuda_fail(e, "self-test launch");
}

int64_t cp_calibrate_pipe(int kind, const float *seed, float *sink, int iters) {
    if (kind < 0 || kind > 7) return fail(CP_EINVAL, "kind must be 0..7 (FFMA, IMAD, MUFU, FFMA2, and four mixes)");
    if (!seed || !sink || !is_aligned(seed, 4) || !is_aligned(sink, 4)) return fail(CP_EINVAL, "seed or sink is NULL or misaligned");
    if (iters < 1 || iters > (1 << 24)) return fail(CP_EINVAL, "iters must be in [1, 2^24]");
    int threads = 0;
    cudaError_t e = cp::launch_pipe_rate(kind, seed, sink, iters, &threads, tl_stream);
    if (e != cudaSuccess) return cuda_fail(e, "calibration launch");
    return (int64_t)threads * iters * 8;
}

const char *cp_last_error(void) { return tl_error; }
const char *cp_version(void) { return "cartpole-b200 0.1 (sm_100a)"; }

}  // extern "C"
