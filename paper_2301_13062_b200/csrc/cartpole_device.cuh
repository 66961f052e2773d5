// Device-side building blocks shared by the three execution strategies
// (per-op ladder, fused step, fused rollout): counter hash, start states,
// the float32 dynamics in their canonical operation order, policies.
//
// Every float operation of the dynamics goes through a round-to-nearest
// intrinsic (__fmul_rn / __fadd_rn / __fsub_rn / __fdiv_rn), which the compiler
// never contracts into a fused multiply-add, so the ladder's one-op kernels and
// the fused kernels produce the same bits (paper Sec. V-C: fusion changes where
// values live, not what is computed).
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace cp {

// ---- constants (float32 roundings of the CartPole-v1 parameters) ----
constexpr float kG = 9.8f;
constexpr float kMPole = 0.1f;
constexpr float kMTot = 1.1f;   // m_cart + m_pole
constexpr float kL = 0.5f;      // half pole length
constexpr float kPML = 0.05f;   // m_pole * l
constexpr float kF = 10.0f;
constexpr float kTau = 0.02f;
constexpr float kFT = 1.33333337306976318359375f;  // (float)(4/3)
constexpr float kXT = 2.4f;
constexpr float kTT = 0.2094395160675048828125f;   // (float)(12 * 2*pi / 360)

constexpr uint32_t kMA = 0x6A09E667u;
constexpr uint32_t kMB = 0xBB67AE85u;
constexpr uint32_t kMG = 0x9E3779B1u;

// ---- counter hash ----
__host__ __device__ __forceinline__ uint32_t mix32(uint32_t h) {
    h ^= h >> 16;
    h *= kMA;
    h ^= h >> 15;
    h *= kMB;
    h ^= h >> 16;
    return h;
}

// Per-(seed, stream) salt; computed once on the host and passed to kernels.
__host__ __device__ __forceinline__ uint32_t salt(uint32_t seed, uint32_t stream) {
    return mix32(mix32(seed ^ kMG) + stream);
}

struct Keys {
    uint32_t k0, k1;
};

__device__ __forceinline__ Keys make_keys(uint32_t salt_, uint32_t env) {
    Keys k;
    k.k0 = mix32(env ^ salt_);
    k.k1 = mix32(k.k0 + kMG);
    return k;
}

__device__ __forceinline__ uint32_t step_hash(Keys k, uint32_t c) {
    uint32_t h = k.k0 ^ c;
    h = (h ^ (h >> 16)) * kMA + k.k1;
    h = (h ^ (h >> 15)) * kMB;
    h ^= h >> 16;
    return h;
}

// Top bit of step_hash: the final xorshift cannot change bit 31, so it is skipped.
__device__ __forceinline__ uint32_t action_signbit(Keys k, uint32_t t) {
    uint32_t h = k.k0 ^ t;
    h = (h ^ (h >> 16)) * kMA + k.k1;
    h = (h ^ (h >> 15)) * kMB;
    return h & 0x80000000u;
}

// force = a ? +F : -F, from the action's sign-bit form (0x80000000 = push right).
__device__ __forceinline__ float force_from_signbit(uint32_t sb) {
    return __uint_as_float(sb ^ 0xC1200000u);  // -10.0f with the sign flipped when a = 1
}

// Component j of the start state of an episode beginning at global time t.
__device__ __forceinline__ float start_value(Keys kr, uint32_t t, uint32_t j) {
    uint32_t bits = step_hash(kr, 4u * t + j) >> 8;
    float u = __fmul_rn(__uint2float_rn(bits), 5.9604644775390625e-08f);  // * 2^-24, exact
    return __fmul_rn(__fsub_rn(u, 0.5f), 0.1f);
}

struct State {
    float x, xd, th, thd;
};

__device__ __forceinline__ State start_state(Keys kr, uint32_t t) {
    State z;
    z.x = start_value(kr, t, 0);
    z.xd = start_value(kr, t, 1);
    z.th = start_value(kr, t, 2);
    z.thd = start_value(kr, t, 3);
    return z;
}

// ---- dynamics ----
// Sine and cosine used by the fused kernels. The ladder calls sinf and cosf in
// two separate kernels; cp_selftest_sincos checks both give the same bits.
__device__ __forceinline__ void sin_cos(float th, float &s, float &c) {
    sincosf(th, &s, &c);
}

// Accelerations (canonical op order; one rounding per op).
__device__ __forceinline__ void accel(float th, float thd, float force, float s, float c,
                                      float &xacc, float &thacc) {
    float t0 = __fmul_rn(thd, thd);
    float t1 = __fmul_rn(kPML, t0);
    float t2 = __fmul_rn(t1, s);
    float t3 = __fadd_rn(force, t2);
    float temp = __fdiv_rn(t3, kMTot);
    float n0 = __fmul_rn(kG, s);
    float n1 = __fmul_rn(c, temp);
    float num = __fsub_rn(n0, n1);
    float d0 = __fmul_rn(c, c);
    float d1 = __fmul_rn(kMPole, d0);
    float d2 = __fdiv_rn(d1, kMTot);
    float d3 = __fsub_rn(kFT, d2);
    float den = __fmul_rn(kL, d3);
    thacc = __fdiv_rn(num, den);
    float p0 = __fmul_rn(kPML, thacc);
    float p1 = __fmul_rn(p0, c);
    float p2 = __fdiv_rn(p1, kMTot);
    xacc = __fsub_rn(temp, p2);
    (void)th;
}

// One explicit-Euler step, no reset. Returns done evaluated on the new state.
__device__ __forceinline__ bool euler_step(State &z, float force) {
    float s, c, xacc, thacc;
    sin_cos(z.th, s, c);
    accel(z.th, z.thd, force, s, c, xacc, thacc);
    float nx = __fadd_rn(z.x, __fmul_rn(kTau, z.xd));
    float nxd = __fadd_rn(z.xd, __fmul_rn(kTau, xacc));
    float nth = __fadd_rn(z.th, __fmul_rn(kTau, z.thd));
    float nthd = __fadd_rn(z.thd, __fmul_rn(kTau, thacc));
    z.x = nx;
    z.xd = nxd;
    z.th = nth;
    z.thd = nthd;
    // x' < -XT | x' > XT  ==  |x'| > XT (false for NaN either way)
    return (fabsf(nx) > kXT) | (fabsf(nth) > kTT);
}

// ---- policies (observation = state before the step) ----
struct LinearW {
    float w[2][4];
    float b[2];
};
struct MlpW {
    float w1[16][4];
    float b1[16];
    float w2[2][16];
    float b2[2];
};

// Returns the action in sign-bit form (0x80000000 = push right).
__device__ __forceinline__ uint32_t linear_action(const LinearW &p, const State &z) {
    float l0 = p.b[0], l1 = p.b[1];
    l0 = __fmaf_rn(p.w[0][0], z.x, l0);
    l1 = __fmaf_rn(p.w[1][0], z.x, l1);
    l0 = __fmaf_rn(p.w[0][1], z.xd, l0);
    l1 = __fmaf_rn(p.w[1][1], z.xd, l1);
    l0 = __fmaf_rn(p.w[0][2], z.th, l0);
    l1 = __fmaf_rn(p.w[1][2], z.th, l1);
    l0 = __fmaf_rn(p.w[0][3], z.thd, l0);
    l1 = __fmaf_rn(p.w[1][3], z.thd, l1);
    return (l1 > l0) ? 0x80000000u : 0u;
}

__device__ __forceinline__ uint32_t mlp_action(const MlpW &p, const State &z) {
    float l0 = p.b2[0], l1 = p.b2[1];
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        float acc = p.b1[j];
        acc = __fmaf_rn(p.w1[j][0], z.x, acc);
        acc = __fmaf_rn(p.w1[j][1], z.xd, acc);
        acc = __fmaf_rn(p.w1[j][2], z.th, acc);
        acc = __fmaf_rn(p.w1[j][3], z.thd, acc);
        float h = tanhf(acc);
        l0 = __fmaf_rn(p.w2[0][j], h, l0);
        l1 = __fmaf_rn(p.w2[1][j], h, l1);
    }
    return (l1 > l0) ? 0x80000000u : 0u;
}

}  // namespace cp
