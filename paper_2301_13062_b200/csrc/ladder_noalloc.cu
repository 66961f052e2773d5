// cp_step_unfused_noalloc: the per-op ladder with its intermediates in a scratch
// array that is part of the library image, for callers that may not allocate.
//
// Who cannot allocate: code running where cudaMalloc is forbidden or unwanted —
// a host thread inside a latency-critical loop (cudaMalloc may synchronise the
// whole device), a plugin whose memory budget is fixed by its host application,
// or a process whose device memory is fully handed to another allocator. Such a
// caller still owns the input and output buffers; only the ladder's intermediate
// planes come from here.
//
// The scratch is one file-scope __device__ array of fixed size. Every GPU whose
// context loads this library holds those bytes until the process exits. In host
// code the array's name is only a handle for the runtime, not a device address,
// so the address is looked up once per device with cudaGetSymbolAddress and that
// pointer is what the kernels receive.
#include <mutex>

#include "../../include/cartpole.h"
#include "cartpole_device.cuh"
#include "cartpole_internal.h"

namespace {

// Bytes the ladder needs for CP_NOALLOC_MAX_ENVS environments: 33 float planes and
// 7 byte planes, each padded to 256 bytes (same layout rule as the caller-supplied
// workspace; checked against cp_unfused_workspace_bytes at set-up).
constexpr size_t kMaxEnvs = CP_NOALLOC_MAX_ENVS;
constexpr size_t kPaddedEnvs = (kMaxEnvs + 63) / 64 * 64;
constexpr size_t kScratchBytes = kPaddedEnvs * 33 * sizeof(float) + ((kPaddedEnvs + 3) / 4 + 63) / 64 * 64 * 4 * 7;

static __device__ __align__(256) unsigned char g_ladder_scratch[kScratchBytes];

constexpr int kMaxDevices = 64;
std::mutex g_mu;
void *g_scratch_ptr[kMaxDevices] = {};  // device address of g_ladder_scratch, per device ordinal

// Look up (once per device, with that device current) where the scratch array lives.
int scratch_for_current_device(void **out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return cp::set_error(CP_ECUDA, cudaGetErrorString(e));
    if (dev < 0 || dev >= kMaxDevices) return cp::set_error(CP_EINVAL, "device ordinal out of range for the no-alloc step");
    std::lock_guard<std::mutex> lock(g_mu);
    if (!g_scratch_ptr[dev]) {
        void *ptr = nullptr;
        e = cudaGetSymbolAddress(&ptr, g_ladder_scratch);
        if (e != cudaSuccess || !ptr) {
            (void)cudaGetLastError();
            return cp::set_error(CP_ECUDA, e != cudaSuccess ? cudaGetErrorString(e) : "scratch symbol has no address");
        }
        if (cp::ladder_workspace_bytes((int64_t)kMaxEnvs) > kScratchBytes)
            return cp::set_error(CP_ENOMEM, "built-in scratch is smaller than the ladder's workspace layout");
        g_scratch_ptr[dev] = ptr;
    }
    *out = g_scratch_ptr[dev];
    return CP_OK;
}

}  // namespace

extern "C" int cp_step_unfused_noalloc(cp_state *state, const uint8_t *action, cp_state *out_state, float *reward,
                                       uint8_t *done) {
    int64_t n = 0, stride = 0, n_out = 0, stride_out = 0;
    uint32_t seed = 0, t = 0, env_offset = 0;
    float *planes = nullptr, *planes_out = nullptr;
    if (cp_state_info(state, &n, &stride, &seed, &t, &env_offset, &planes) != CP_OK) return CP_EINVAL;
    if (cp_state_info(out_state, &n_out, &stride_out, nullptr, nullptr, nullptr, &planes_out) != CP_OK) return CP_EINVAL;
    if (n > (int64_t)kMaxEnvs)
        return cp::set_error(CP_EINVAL, "the no-alloc step handles at most CP_NOALLOC_MAX_ENVS (65536) environments; "
                                        "use cp_step_unfused with your own workspace for more");
    if (n <= 0 || n_out != n || !planes || !planes_out || stride < n || stride_out < n)
        return cp::set_error(CP_EINVAL, "state and out_state must be valid batches of the same size");
    if (!reward || !done) return cp::set_error(CP_EINVAL, "reward and done must not be NULL for the unfused step");
    if (reinterpret_cast<uintptr_t>(reward) % 4) return cp::set_error(CP_EINVAL, "reward is not float-aligned");
    if (reinterpret_cast<uintptr_t>(planes) % 16 || reinterpret_cast<uintptr_t>(planes_out) % 16 || stride % 4 ||
        stride_out % 4)
        return cp::set_error(CP_EINVAL, "the unfused step needs 16-byte aligned planes with plane_stride % 4 == 0");
    if (planes == planes_out) return cp::set_error(CP_EINVAL, "the unfused step cannot run in place");
    if (t >= (1u << 30)) return cp::set_error(CP_EINVAL, "global step out of range");

    void *scratch = nullptr;
    int rc = scratch_for_current_device(&scratch);
    if (rc != CP_OK) return rc;

    cp::StepParams p;
    p.in = planes;
    p.in_stride = stride;
    p.out = planes_out;
    p.out_stride = stride_out;
    p.n = n;
    p.t = t;
    p.env_offset = env_offset;
    p.salt_a = cp::salt(seed, 0u);
    p.salt_r = cp::salt(seed, 1u);
    p.action = action;
    p.reward = reward;
    p.done = done;
    p.ep_len = nullptr;
    p.max_steps = 0;
    // Every intermediate plane is fully written by the kernel that produces it before any
    // kernel reads it, so nothing in the scratch needs clearing between calls.
    cudaError_t e = cp::launch_ladder(p, scratch, cp::thread_stream());
    if (e != cudaSuccess) return cp::set_error(CP_ECUDA, cudaGetErrorString(e));
    cp::adopt_step(state, out_state, 1);
    return CP_OK;
}
