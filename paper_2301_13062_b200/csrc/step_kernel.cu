// Fused single-step kernel (paper Sec. V-C: the four state values travel as
// separate planes and the whole update is one kernel with the state in
// registers), plus the small generator kernels (start states, hashed actions)
// and the sine/cosine self-test.
//
// HBM traffic per env-step: 16 B state in + 16 B state out + 4 B reward + 1 B
// done (+ 1 B action when supplied). Vector form: each thread owns 4 consecutive
// environments, i.e. one float4 per plane, so a warp moves 512 B per plane per
// access and keeps 4 x 16 B loads in flight per thread.
#include <cstring>

#include "cartpole_device.cuh"
#include "cartpole_internal.h"

namespace cp {

// Action of one environment in sign-bit form: hashed (independent of any memory) or supplied.
__device__ __forceinline__ uint32_t hashed_signbit(const StepParams &p, uint32_t env) {
    return action_signbit(make_keys(p.salt_a, env), p.t);
}

// The kernel is written for programmatic dependent launch: everything that does not depend on
// what the previous launch wrote (the action hashes, about a quarter of the instructions) comes
// first; then the kernel waits for the previous launch's memory to be visible and immediately
// lets the next launch begin its own preamble. Launched without that attribute the two
// grid-dependency instructions do nothing.
template <bool VEC>
__global__ void __launch_bounds__(256, 1) step_kernel(const __grid_constant__ StepParams p) {
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    const bool has_action = p.action != nullptr;
    if (VEC) {
        const int64_t i0 = tid * 4;
        if (i0 >= p.n) return;
        const uint32_t env0 = p.env_offset + (uint32_t)i0;
        const bool full = i0 + 3 < p.n;
        uint32_t sb[4] = {0u, 0u, 0u, 0u};
        if (!has_action) {
#pragma unroll
            for (int j = 0; j < 4; ++j) sb[j] = hashed_signbit(p, env0 + j);
        }
        cudaGridDependencySynchronize();
        cudaTriggerProgrammaticLaunchCompletion();
        const float4 vx = *reinterpret_cast<const float4 *>(p.in + i0);
        const float4 vxd = *reinterpret_cast<const float4 *>(p.in + p.in_stride + i0);
        const float4 vth = *reinterpret_cast<const float4 *>(p.in + 2 * p.in_stride + i0);
        const float4 vthd = *reinterpret_cast<const float4 *>(p.in + 3 * p.in_stride + i0);
        State z[4] = {{vx.x, vxd.x, vth.x, vthd.x},
                      {vx.y, vxd.y, vth.y, vthd.y},
                      {vx.z, vxd.z, vth.z, vthd.z},
                      {vx.w, vxd.w, vth.w, vthd.w}};
        if (has_action) {
            if (full) {
                uchar4 av = *reinterpret_cast<const uchar4 *>(p.action + i0);
                sb[0] = av.x ? 0x80000000u : 0u;
                sb[1] = av.y ? 0x80000000u : 0u;
                sb[2] = av.z ? 0x80000000u : 0u;
                sb[3] = av.w ? 0x80000000u : 0u;
            } else {
                for (int j = 0; j < 4; ++j)
                    if (i0 + j < p.n) sb[j] = p.action[i0 + j] ? 0x80000000u : 0u;
            }
        }
        uint32_t dmask = 0;
#pragma unroll
        for (int j = 0; j < 4; ++j) dmask |= (euler_step(z[j], force_from_signbit(sb[j])) ? 1u : 0u) << j;
        if (p.ep_len) {  // optional episode-length counters and step limit
            uint32_t len[4] = {0u, 0u, 0u, 0u};
            if (full) {
                const uint4 v = *reinterpret_cast<const uint4 *>(p.ep_len + i0);
                len[0] = v.x; len[1] = v.y; len[2] = v.z; len[3] = v.w;
            } else {
                for (int j = 0; j < 4; ++j)
                    if (i0 + j < p.n) len[j] = p.ep_len[i0 + j];
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                len[j] += 1u;
                if (p.max_steps && len[j] >= p.max_steps) dmask |= 1u << j;
                if ((dmask >> j) & 1u) len[j] = 0u;
            }
            if (full) {
                *reinterpret_cast<uint4 *>(p.ep_len + i0) = make_uint4(len[0], len[1], len[2], len[3]);
            } else {
                for (int j = 0; j < 4; ++j)
                    if (i0 + j < p.n) p.ep_len[i0 + j] = len[j];
            }
        }
        // Restart finished environments one per pass: almost always at most one of a
        // thread's four environments finishes in a step, so the start-state hashes are
        // issued once per warp instead of once per environment slot.
        uint32_t pending = dmask;
        while (pending) {
            const int j = __ffs(pending) - 1;
            pending &= pending - 1;
            const State r = start_state(make_keys(p.salt_r, env0 + j), p.t + 1u);
#pragma unroll
            for (int q = 0; q < 4; ++q)
                if (q == j) z[q] = r;
        }
        *reinterpret_cast<float4 *>(p.out + i0) = make_float4(z[0].x, z[1].x, z[2].x, z[3].x);
        *reinterpret_cast<float4 *>(p.out + p.out_stride + i0) = make_float4(z[0].xd, z[1].xd, z[2].xd, z[3].xd);
        *reinterpret_cast<float4 *>(p.out + 2 * p.out_stride + i0) = make_float4(z[0].th, z[1].th, z[2].th, z[3].th);
        *reinterpret_cast<float4 *>(p.out + 3 * p.out_stride + i0) = make_float4(z[0].thd, z[1].thd, z[2].thd, z[3].thd);
        if (full) {
            if (p.reward) *reinterpret_cast<float4 *>(p.reward + i0) = make_float4(1.0f, 1.0f, 1.0f, 1.0f);
            if (p.done)
                *reinterpret_cast<uchar4 *>(p.done + i0) =
                    make_uchar4(dmask & 1u, (dmask >> 1) & 1u, (dmask >> 2) & 1u, (dmask >> 3) & 1u);
        } else {
            for (int j = 0; j < 4; ++j)
                if (i0 + j < p.n) {
                    if (p.reward) p.reward[i0 + j] = 1.0f;
                    if (p.done) p.done[i0 + j] = (dmask >> j) & 1u;
                }
        }
    } else {
        const int64_t i = tid;
        if (i >= p.n) return;
        const uint32_t env = p.env_offset + (uint32_t)i;
        uint32_t sb = has_action ? 0u : hashed_signbit(p, env);
        cudaGridDependencySynchronize();
        cudaTriggerProgrammaticLaunchCompletion();
        State z = {p.in[i], p.in[p.in_stride + i], p.in[2 * p.in_stride + i], p.in[3 * p.in_stride + i]};
        if (has_action) sb = p.action[i] ? 0x80000000u : 0u;
        bool d = euler_step(z, force_from_signbit(sb));
        if (p.ep_len) {
            uint32_t len = p.ep_len[i] + 1u;
            if (p.max_steps && len >= p.max_steps) d = true;
            p.ep_len[i] = d ? 0u : len;
        }
        if (d) z = start_state(make_keys(p.salt_r, env), p.t + 1u);
        p.out[i] = z.x;
        p.out[p.out_stride + i] = z.xd;
        p.out[2 * p.out_stride + i] = z.th;
        p.out[3 * p.out_stride + i] = z.thd;
        if (p.reward) p.reward[i] = 1.0f;
        if (p.done) p.done[i] = d ? 1 : 0;
    }
}

template <bool VEC>
static cudaError_t launch_step_kernel(const StepParams &p, unsigned grid, int block, cudaStream_t s) {
    if (!g_tuning.step_pdl) {
        step_kernel<VEC><<<grid, block, 0, s>>>(p);
        return cudaGetLastError();
    }
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(grid);
    cfg.blockDim = dim3(block);
    cfg.stream = s;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, step_kernel<VEC>, p);
}

cudaError_t launch_step(const StepParams &p, bool vec, cudaStream_t s) {
    const int block = g_tuning.step_block;
    cudaError_t e;
    if (vec) {
        const int64_t threads = (p.n + 3) / 4;
        e = launch_step_kernel<true>(p, (unsigned)((threads + block - 1) / block), block, s);
    } else {
        e = launch_step_kernel<false>(p, (unsigned)((p.n + block - 1) / block), block, s);
    }
    count_launch();
    return e;
}

// ---- generators ----
__global__ void fill_start_kernel(float *planes, int64_t stride, int64_t n, uint32_t env_offset, uint32_t salt_r,
                                  uint32_t t) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    const State z = start_state(make_keys(salt_r, env_offset + (uint32_t)i), t);
    planes[i] = z.x;
    planes[stride + i] = z.xd;
    planes[2 * stride + i] = z.th;
    planes[3 * stride + i] = z.thd;
}

cudaError_t launch_fill_start(float *planes, int64_t stride, int64_t n, uint32_t env_offset, uint32_t salt_r,
                              uint32_t t, cudaStream_t s) {
    const int block = 256;
    fill_start_kernel<<<(unsigned)((n + block - 1) / block), block, 0, s>>>(planes, stride, n, env_offset, salt_r, t);
    count_launch();
    return cudaGetLastError();
}

__global__ void actions_kernel(uint8_t *out, int64_t n, uint32_t env_offset, uint32_t salt_a, uint32_t t) {
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
    out[i] = (uint8_t)(step_hash(make_keys(salt_a, env_offset + (uint32_t)i), t) >> 31);
}

cudaError_t launch_actions(uint8_t *out, int64_t n, uint32_t env_offset, uint32_t salt_a, uint32_t t,
                           cudaStream_t s) {
    const int block = 256;
    actions_kernel<<<(unsigned)((n + block - 1) / block), block, 0, s>>>(out, n, env_offset, salt_a, t);
    count_launch();
    return cudaGetLastError();
}

// ---- self-test: fused sine/cosine vs separate sinf and cosf ----
__global__ void sincos_selftest_kernel(uint32_t lo, uint32_t hi, unsigned long long *mismatches) {
    unsigned long long bad = 0;
    const uint64_t span = (uint64_t)hi - lo + 1;
    for (uint64_t k = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; k < span; k += (uint64_t)gridDim.x * blockDim.x) {
        const float v = __uint_as_float(lo + (uint32_t)k);
        float s, c;
        sin_cos(v, s, c);
        bad += (__float_as_uint(s) != __float_as_uint(sin_op(v))) | (__float_as_uint(c) != __float_as_uint(cos_op(v)));
        sin_cos(-v, s, c);
        bad += (__float_as_uint(s) != __float_as_uint(sin_op(-v))) | (__float_as_uint(c) != __float_as_uint(cos_op(-v)));
    }
    for (int o = 16; o > 0; o >>= 1) bad += __shfl_down_sync(0xffffffffu, bad, o);
    if ((threadIdx.x & 31) == 0 && bad) atomicAdd(mismatches, bad);
}

cudaError_t launch_sincos_selftest(uint32_t lo_bits, uint32_t hi_bits, unsigned long long *mismatches,
                                   cudaStream_t s) {
    sincos_selftest_kernel<<<sm_count() * 8, 256, 0, s>>>(lo_bits, hi_bits, mismatches);
    count_launch();
    return cudaGetLastError();
}

// ---- self-test: error of the kernels' sine/cosine against float64, in millionths of an ulp ----
// out[0], out[1] = max error of sin, cos; out[2], out[3] = how many results are not the
// correctly rounded float32 value.
__device__ __forceinline__ unsigned long long micro_ulps(float got, double exact) {
    const float near = (float)exact;
    // ulp of the exact value's binade
    const float up = __uint_as_float(__float_as_uint(fabsf(near)) + 1u);
    const double ulp = (double)up - (double)fabsf(near);
    const double e = fabs((double)got - exact) / ulp;
    return (unsigned long long)(e * 1e6);
}

__global__ void sincos_accuracy_kernel(uint32_t lo, uint32_t hi, unsigned long long *out) {
    unsigned long long ms = 0, mc = 0, ns = 0, nc = 0;
    const uint64_t span = (uint64_t)hi - lo + 1;
    for (uint64_t k = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; k < span; k += (uint64_t)gridDim.x * blockDim.x) {
        const float v = __uint_as_float(lo + (uint32_t)k);
        float s, c;
        sin_cos(v, s, c);
        const double es = sin((double)v), ec = cos((double)v);
        const unsigned long long a = micro_ulps(s, es), b = micro_ulps(c, ec);
        ms = a > ms ? a : ms;
        mc = b > mc ? b : mc;
        ns += __float_as_uint(s) != __float_as_uint((float)es);
        nc += __float_as_uint(c) != __float_as_uint((float)ec);
    }
    for (int o = 16; o > 0; o >>= 1) {
        const unsigned long long a = __shfl_down_sync(0xffffffffu, ms, o), b = __shfl_down_sync(0xffffffffu, mc, o);
        ms = a > ms ? a : ms;
        mc = b > mc ? b : mc;
        ns += __shfl_down_sync(0xffffffffu, ns, o);
        nc += __shfl_down_sync(0xffffffffu, nc, o);
    }
    if ((threadIdx.x & 31) == 0) {
        atomicMax(out, ms);
        atomicMax(out + 1, mc);
        if (ns) atomicAdd(out + 2, ns);
        if (nc) atomicAdd(out + 3, nc);
    }
}

cudaError_t launch_sincos_accuracy(uint32_t lo_bits, uint32_t hi_bits, unsigned long long *out, cudaStream_t s) {
    sincos_accuracy_kernel<<<sm_count() * 8, 256, 0, s>>>(lo_bits, hi_bits, out);
    count_launch();
    return cudaGetLastError();
}

// ---- self-test: error of the hyperbolic tangents against float64 ----
// Over the float32 values with bit patterns in [lo, hi] and their negatives. Largest absolute
// error in units of 1e-12: out[0] tanh_contracted, out[1] the library's tanhf, out[2]
// tanh_canonical; largest error in millionths of an ulp: out[3] tanh_canonical, out[4] the
// library's; out[5] += values for which tanh_pair differs from tanh_canonical in any bit.
__global__ void tanh_accuracy_kernel(uint32_t lo, uint32_t hi, unsigned long long *out) {
    double worst_fast = 0.0, worst_lib = 0.0, worst_own = 0.0, worst_own_ulp = 0.0, worst_lib_ulp = 0.0;
    unsigned long long pair_mismatch = 0;
    const uint64_t span = (uint64_t)hi - lo + 1;
    for (uint64_t k = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; k < span; k += (uint64_t)gridDim.x * blockDim.x) {
        float own[2];
        for (int sign = 0; sign < 2; ++sign) {
            const float v = __uint_as_float((lo + (uint32_t)k) | (sign ? 0x80000000u : 0u));
            const double exact = tanh((double)v);
            // one unit in the last place of the correctly rounded result
            const float w = fabsf((float)exact);
            double ulp = (double)__uint_as_float(__float_as_uint(w) + 1u) - (double)w;
            if (!(ulp > 0.0)) ulp = 1.4e-45;
            own[sign] = tanh_canonical(v);
            const float lib = tanhf(v);
            worst_fast = fmax(worst_fast, fabs((double)tanh_contracted(v) - exact));
            worst_lib = fmax(worst_lib, fabs((double)lib - exact));
            worst_own = fmax(worst_own, fabs((double)own[sign] - exact));
            worst_own_ulp = fmax(worst_own_ulp, fabs((double)own[sign] - exact) / ulp);
            worst_lib_ulp = fmax(worst_lib_ulp, fabs((double)lib - exact) / ulp);
        }
        // the packed form on (v, -v) and on (-v, v): the same bits as the scalar form, either half
        const float v = __uint_as_float(lo + (uint32_t)k);
        float p0, p1, q0, q1;
        unpack2(tanh_pair(pack2(v, -v)), p0, p1);
        unpack2(tanh_pair(pack2(-v, v)), q0, q1);
        pair_mismatch += __float_as_uint(p0) != __float_as_uint(own[0]) || __float_as_uint(p1) != __float_as_uint(own[1]) ||
                         __float_as_uint(q0) != __float_as_uint(own[1]) || __float_as_uint(q1) != __float_as_uint(own[0]);
    }
    unsigned long long m[5] = {(unsigned long long)(worst_fast * 1e12), (unsigned long long)(worst_lib * 1e12),
                               (unsigned long long)(worst_own * 1e12), (unsigned long long)(worst_own_ulp * 1e6),
                               (unsigned long long)(worst_lib_ulp * 1e6)};
    for (int o = 16; o > 0; o >>= 1) {
        for (int i = 0; i < 5; ++i) {
            const unsigned long long other = __shfl_down_sync(0xffffffffu, m[i], o);
            m[i] = other > m[i] ? other : m[i];
        }
        pair_mismatch += __shfl_down_sync(0xffffffffu, pair_mismatch, o);
    }
    if ((threadIdx.x & 31) == 0) {
        for (int i = 0; i < 5; ++i) atomicMax(out + i, m[i]);
        if (pair_mismatch) atomicAdd(out + 5, pair_mismatch);
    }
}

cudaError_t launch_tanh_accuracy(uint32_t lo_bits, uint32_t hi_bits, unsigned long long *out, cudaStream_t s) {
    tanh_accuracy_kernel<<<sm_count() * 8, 256, 0, s>>>(lo_bits, hi_bits, out);
    count_launch();
    return cudaGetLastError();
}

// ---- self-test: the exact shortcuts against the operations they replace ----
// out[0]: bit patterns x (all 2^32) where div_mtot(x) != __fdiv_rn(x, 1.1f)
// out[1]: patterns inside div_mtot_not_tiny's domain (+0, NaN, Inf, |x| >= 2^-100) where it differs
// out[2]: patterns inside div_mtot_normal's domain (+0, NaN, 2^-100 <= |x| <= FLT_MAX) where it differs
// out[3]: 24-bit inputs where start_from_bits differs from the definition's three operations
__global__ void arith_selftest_kernel(unsigned long long *out) {
    unsigned long long b0 = 0, b1 = 0, b2 = 0, b3 = 0;
    for (uint64_t k = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; k < (1ull << 32);
         k += (uint64_t)gridDim.x * blockDim.x) {
        const uint32_t bits = (uint32_t)k;
        const float x = __uint_as_float(bits);
        const uint32_t want = __float_as_uint(__fdiv_rn(x, kMTot));
        const float ax = fabsf(x);
        const bool is_nan = x != x;
        const bool pos_zero = bits == 0u;
        b0 += __float_as_uint(div_mtot(x)) != want;
        if (pos_zero || is_nan || ax >= 7.888609052e-31f) b1 += __float_as_uint(div_mtot_not_tiny(x)) != want;
        if (pos_zero || is_nan || (ax >= 7.888609052e-31f && ax <= 3.402823466e+38f))
            b2 += __float_as_uint(div_mtot_normal(x)) != want;
        if (bits < (1u << 24))
            b3 += __float_as_uint(start_from_bits(bits)) != __float_as_uint(start_from_bits_reference(bits));
    }
    for (int o = 16; o > 0; o >>= 1) {
        b0 += __shfl_down_sync(0xffffffffu, b0, o);
        b1 += __shfl_down_sync(0xffffffffu, b1, o);
        b2 += __shfl_down_sync(0xffffffffu, b2, o);
        b3 += __shfl_down_sync(0xffffffffu, b3, o);
    }
    if ((threadIdx.x & 31) == 0 && (b0 | b1 | b2 | b3)) {
        atomicAdd(out, b0);
        atomicAdd(out + 1, b1);
        atomicAdd(out + 2, b2);
        atomicAdd(out + 3, b3);
    }
}

// ---- self-test: the tame-state division against IEEE division over its whole operand domain ----
// den: every den_step-th float in [kTameDenLo, kTameDenHi]; num: every float in [2, 32) (the
// sequence is odd in num, so negative numerators need no separate pass).
// out[0] += mismatches, out[1] += pairs tested.
__global__ void tame_div_selftest_kernel(uint32_t den_lo, uint32_t den_hi, uint32_t den_step,
                                         unsigned long long *out) {
    unsigned long long bad = 0, pairs = 0;
    for (uint64_t db = (uint64_t)den_lo + (uint64_t)blockIdx.y * den_step; db <= den_hi;
         db += (uint64_t)gridDim.y * den_step) {
        const float den = __uint_as_float((uint32_t)db);
        for (uint32_t nb = 0x40000000u + blockIdx.x * blockDim.x + threadIdx.x; nb < 0x42000000u;
             nb += gridDim.x * blockDim.x) {
            const float num = __uint_as_float(nb);
            bad += __float_as_uint(div_tame(num, den)) != __float_as_uint(__fdiv_rn(num, den));
            bad += __float_as_uint(div_tame(-num, den)) != (__float_as_uint(__fdiv_rn(num, den)) ^ 0x80000000u);
            pairs += 1;
        }
    }
    for (int o = 16; o > 0; o >>= 1) {
        bad += __shfl_down_sync(0xffffffffu, bad, o);
        pairs += __shfl_down_sync(0xffffffffu, pairs, o);
    }
    if ((threadIdx.x & 31) == 0) {
        if (bad) atomicAdd(out, bad);
        atomicAdd(out + 1, pairs);
    }
}

cudaError_t launch_tame_div_selftest(uint32_t den_step, unsigned long long *out, cudaStream_t s) {
    uint32_t lo, hi;
    memcpy(&lo, &kTameDenLo, 4);
    memcpy(&hi, &kTameDenHi, 4);
    tame_div_selftest_kernel<<<dim3(sm_count() * 2, 64), 256, 0, s>>>(lo, hi, den_step, out);
    count_launch();
    return cudaGetLastError();
}

// ---- calibration: what one pipe sustains, for the roofline denominators ----
// Every thread runs `iters` rounds of eight independent chains, sixteen resident warps per
// scheduler. KIND 0: FFMA, 1: IMAD, 2: MUFU reciprocal, 3: packed FFMA2 (two float32 FMAs per
// instruction); mixes of four chains each: 4: FFMA2 + FFMA, 5: FFMA2 + IMAD, 6: FFMA2 + integer
// logic (the ALU pipe), 7: FFMA + IMAD. The host times the launch; instructions = threads *
// iters * 8. The seeds come from memory so that nothing folds at compile time, and the results
// are stored so that nothing is dead.
template <int KIND>
__global__ void __launch_bounds__(256) pipe_rate_kernel(const float *seed, float *sink, int iters) {
    float a[8];
    uint32_t u[8];
    f32x2 q[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        a[k] = seed[k] + (float)threadIdx.x * 1e-3f;
        u[k] = __float_as_uint(a[k]) | 1u;
        q[k] = pack2(a[k], a[k] + 0.5f);
    }
    const float m = seed[8], c = seed[9];
    const uint32_t um = __float_as_uint(m) | 1u, uc = __float_as_uint(c);
    const f32x2 qm = pack2(m, m), qc = pack2(c, c);
    for (int i = 0; i < iters; ++i) {
#pragma unroll
        for (int k = 0; k < 8; ++k) {
            const bool second = k >= 4;  // the mixes: chains 0-3 packed (7: scalar float), 4-7 the partner
            if (KIND == 0 || (KIND == 4 && second) || (KIND == 7 && !second)) a[k] = __fmaf_rn(a[k], m, c);
            if (KIND == 1 || ((KIND == 5 || KIND == 7) && second)) u[k] = u[k] * um + uc;
            if (KIND == 2) {  // the add keeps the assembler from cancelling a reciprocal of a reciprocal
                asm volatile("rcp.approx.ftz.f32 %0, %0;" : "+f"(a[k]));
                a[k] = __fadd_rn(a[k], c);
            }
            if (KIND == 3 || ((KIND == 4 || KIND == 5 || KIND == 6) && !second)) q[k] = fma2(q[k], qm, qc);
            if (KIND == 6 && second) u[k] = (u[k] ^ um) + (u[k] >> 7);  // two ALU instructions per round
        }
    }
    float acc = 0.0f;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        float lo, hi;
        unpack2(q[k], lo, hi);
        acc += __uint_as_float(u[k] & 0x3fffffffu) + a[k] + lo + hi;
    }
    sink[(size_t)blockIdx.x * blockDim.x + threadIdx.x] = acc;
}

cudaError_t launch_pipe_rate(int kind, const float *seed, float *sink, int iters, int *threads, cudaStream_t s) {
    const int grid = sm_count() * 8, block = 256;  // 64 warps per SM = 16 per scheduler
    *threads = grid * block;
    switch (kind) {
        case 0: pipe_rate_kernel<0><<<grid, block, 0, s>>>(seed, sink, iters); break;
        case 1: pipe_rate_kernel<1><<<grid, block, 0, s>>>(seed, sink, iters); break;
        case 2: pipe_rate_kernel<2><<<grid, block, 0, s>>>(seed, sink, iters); break;
        case 3: pipe_rate_kernel<3><<<grid, block, 0, s>>>(seed, sink, iters); break;
        case 4: pipe_rate_kernel<4><<<grid, block, 0, s>>>(seed, sink, iters); break;
        case 5: pipe_rate_kernel<5><<<grid, block, 0, s>>>(seed, sink, iters); break;
        case 6: pipe_rate_kernel<6><<<grid, block, 0, s>>>(seed, sink, iters); break;
        default: pipe_rate_kernel<7><<<grid, block, 0, s>>>(seed, sink, iters); break;
    }
    count_launch();
    return cudaGetLastError();
}

// ---- self-test: the packed two-environment step against the scalar step ----
// count pseudo-random pairs of states from the domain the packed step is used on (|theta| <= 0.22)
// and a little beyond what an episode visits in the other components; every pair is stepped by
// euler_step_pair and, half by half, by euler_step<true>. out[0] += pairs whose eight new state
// components or two termination flags differ in any bit, out[1] += pairs tested, out[2] += pairs
// for which the contracted arithmetic's packed and scalar steps differ.
__global__ void pair_selftest_kernel(unsigned long long count, uint32_t seed, unsigned long long *out) {
    unsigned long long bad = 0, bad_c = 0, seen = 0;
    const uint32_t s0 = salt(seed, 7u);
    for (unsigned long long k = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x; k < count;
         k += (unsigned long long)gridDim.x * blockDim.x) {
        const Keys key = make_keys(s0 ^ (uint32_t)(k >> 32), (uint32_t)k);
        float u[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) u[i] = (float)(step_hash(key, (uint32_t)i) >> 8) * 1.1920929e-07f - 1.0f;  // [-1, 1)
        const uint32_t bits = step_hash(key, 8u);
        // every fourth pair at the scale of start states, the others across the whole live range
        const float scale = (bits & 3u) ? 1.0f : 0.25f;
        State a, b;
        a.x = u[0] * 2.5f * scale;
        a.xd = u[1] * 4.0f * scale;
        a.th = u[2] * kSmallAngle * scale;
        a.thd = u[3] * 22.0f * scale;
        b.x = u[4] * 2.5f * scale;
        b.xd = u[5] * 4.0f * scale;
        b.th = u[6] * kSmallAngle * scale;
        b.thd = u[7] * 22.0f * scale;
        const float fa = force_from_signbit((bits << 8) & 0x80000000u), fb = force_from_signbit((bits << 9) & 0x80000000u);
        StatePair zz = pack_states(a, b);
        bool pd0, pd1;
        euler_step_pair(zz, pack2(fa, fb), pd0, pd1);
        State pa, pb;
        unpack_states(zz, pa, pb);
        const bool d0 = euler_step<true>(a, fa), d1 = euler_step<true>(b, fb);
        const bool same = __float_as_uint(pa.x) == __float_as_uint(a.x) && __float_as_uint(pa.xd) == __float_as_uint(a.xd) &&
                          __float_as_uint(pa.th) == __float_as_uint(a.th) && __float_as_uint(pa.thd) == __float_as_uint(a.thd) &&
                          __float_as_uint(pb.x) == __float_as_uint(b.x) && __float_as_uint(pb.xd) == __float_as_uint(b.xd) &&
                          __float_as_uint(pb.th) == __float_as_uint(b.th) && __float_as_uint(pb.thd) == __float_as_uint(b.thd) &&
                          pd0 == d0 && pd1 == d1;
        bad += !same;
        seen += 1;
        // the same for the contracted arithmetic (a and b now hold the stepped states: step them again)
        State ca = a, cb = b;
        StatePair cz = pack_states(a, b);
        bool qd0, qd1;
        euler_step_contracted_pair(cz, pack2(fa, fb), qd0, qd1);
        State qa, qb;
        unpack_states(cz, qa, qb);
        const bool e0 = euler_step_contracted<true>(ca, fa), e1 = euler_step_contracted<true>(cb, fb);
        bad_c += !(__float_as_uint(qa.x) == __float_as_uint(ca.x) && __float_as_uint(qa.xd) == __float_as_uint(ca.xd) &&
                   __float_as_uint(qa.th) == __float_as_uint(ca.th) && __float_as_uint(qa.thd) == __float_as_uint(ca.thd) &&
                   __float_as_uint(qb.x) == __float_as_uint(cb.x) && __float_as_uint(qb.xd) == __float_as_uint(cb.xd) &&
                   __float_as_uint(qb.th) == __float_as_uint(cb.th) && __float_as_uint(qb.thd) == __float_as_uint(cb.thd) &&
                   qd0 == e0 && qd1 == e1);
    }
    for (int o = 16; o > 0; o >>= 1) {
        bad += __shfl_down_sync(0xffffffffu, bad, o);
        bad_c += __shfl_down_sync(0xffffffffu, bad_c, o);
        seen += __shfl_down_sync(0xffffffffu, seen, o);
    }
    if ((threadIdx.x & 31) == 0) {
        if (bad) atomicAdd(out, bad);
        atomicAdd(out + 1, seen);
        if (bad_c) atomicAdd(out + 2, bad_c);
    }
}

cudaError_t launch_pair_selftest(unsigned long long count, uint32_t seed, unsigned long long *out, cudaStream_t s) {
    pair_selftest_kernel<<<sm_count() * 8, 256, 0, s>>>(count, seed, out);
    count_launch();
    return cudaGetLastError();
}

cudaError_t launch_arith_selftest(unsigned long long *out, cudaStream_t s) {
    arith_selftest_kernel<<<sm_count() * 8, 256, 0, s>>>(out);
    count_launch();
    return cudaGetLastError();
}

}  // namespace cp
