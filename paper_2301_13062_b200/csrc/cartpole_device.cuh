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

// Keys for loops over time. A right shift distributes over xor, so the first xorshift of
// step_hash splits into a part that depends only on the key and one that depends only on the
// counter:  (k0 ^ c) ^ ((k0 ^ c) >> 16) == fold16(k0) ^ fold16(c).  A kernel that hashes many
// counters with one key keeps fold16(k0), and computes fold16(c) once per step for all its envs.
__device__ __forceinline__ uint32_t fold16(uint32_t v) { return v ^ (v >> 16); }
struct FoldedKeys {
    uint32_t f0, k1;  // fold16(k0), k1
};
__device__ __forceinline__ FoldedKeys fold_keys(Keys k) {
    FoldedKeys f;
    f.f0 = fold16(k.k0);
    f.k1 = k.k1;
    return f;
}
// action_signbit(k, t) with folded_t = fold16(t)
__device__ __forceinline__ uint32_t action_signbit_folded(FoldedKeys k, uint32_t folded_t) {
    uint32_t h = (k.f0 ^ folded_t) * kMA + k.k1;
    h = (h ^ (h >> 15)) * kMB;
    return h & 0x80000000u;
}

// force = a ? +F : -F, from the action's sign-bit form (0x80000000 = push right).
__device__ __forceinline__ float force_from_signbit(uint32_t sb) {
    return __uint_as_float(sb ^ 0xC1200000u);  // -10.0f with the sign flipped when a = 1
}

// 24 uniform bits -> start-state component. The definition is
//     u = float(bits) * 2^-24;  value = (u - 0.5f) * 0.1f
// where the first two operations are exact and only the last multiply rounds. The same
// real number is (bits - 2^23) * (0.1f * 2^-24) with both factors exact in float32, so one
// int->float conversion and one multiply give the identical rounding (checked for all 2^24
// inputs by cp_selftest_arith).
__device__ __forceinline__ float start_from_bits_reference(uint32_t bits) {
    float u = __fmul_rn(__uint2float_rn(bits), 5.9604644775390625e-08f);  // * 2^-24, exact
    return __fmul_rn(__fsub_rn(u, 0.5f), 0.1f);
}
// (A conversion-free form — f = 0x4B000000 | low 23 bits, then one fused multiply-add with
// -0.1f or -0.1f/2 chosen by bit 23 — gives the same bits but was measured slower everywhere:
// the conversion runs on the otherwise idle special-function pipe, the two logic operations
// that replace it on the half-rate integer pipe.)
__device__ __forceinline__ float start_from_bits(uint32_t bits) {
    return __fmul_rn(__int2float_rn((int)bits - (1 << 23)), 5.9604645663569045e-09f);  // 0.1f * 2^-24
}

// Component j of the start state of an episode beginning at global time t.
__device__ __forceinline__ float start_value(Keys kr, uint32_t t, uint32_t j) {
    return start_from_bits(step_hash(kr, 4u * t + j) >> 8);
}

struct State {
    float x, xd, th, thd;
};

// All four components at once. The four counters 4t+j differ only in their two low bits, and
// the first xorshift of step_hash (h ^ h>>16) leaves low bits of the counter untouched by the
// shifted half, so (K0 ^ (4t+j)) ^ ((K0 ^ (4t+j)) >> 16) == m ^ j with m computed once from
// 4t. The rest of each hash is step_hash's own sequence; results equal start_value(kr, t, j).
__device__ __forceinline__ uint32_t step_hash_tail(Keys k, uint32_t m) {
    uint32_t h = m * kMA + k.k1;
    h = (h ^ (h >> 15)) * kMB;
    h ^= h >> 16;
    return h;
}
__device__ __forceinline__ State start_state(Keys kr, uint32_t t) {
    const uint32_t h0 = kr.k0 ^ (4u * t);
    const uint32_t m = h0 ^ (h0 >> 16);
    State z;
    z.x = start_from_bits(step_hash_tail(kr, m) >> 8);
    z.xd = start_from_bits(step_hash_tail(kr, m ^ 1u) >> 8);
    z.th = start_from_bits(step_hash_tail(kr, m ^ 2u) >> 8);
    z.thd = start_from_bits(step_hash_tail(kr, m ^ 3u) >> 8);
    return z;
}

// The same from folded keys; folded_4t = fold16(4 * t). The counters 4t + j (j < 4) fold to
// fold16(4t) ^ j because 4t has its two low bits clear and j >> 16 == 0.
__device__ __forceinline__ float start_component_folded(FoldedKeys kr, uint32_t folded_4t, uint32_t j) {
    Keys k;
    k.k0 = 0u;  // not used by the tail
    k.k1 = kr.k1;
    return start_from_bits(step_hash_tail(k, kr.f0 ^ folded_4t ^ j) >> 8);
}
__device__ __forceinline__ State start_state_folded(FoldedKeys kr, uint32_t folded_4t) {
    State z;
    z.x = start_component_folded(kr, folded_4t, 0u);
    z.xd = start_component_folded(kr, folded_4t, 1u);
    z.th = start_component_folded(kr, folded_4t, 2u);
    z.thd = start_component_folded(kr, folded_4t, 3u);
    return z;
}

// ---- sine and cosine ----
// An episode only ever evaluates sin/cos at |theta| <= 12 degrees (0.2095 rad): a larger
// angle has already ended the episode. For |theta| <= 0.22 both functions are short
// polynomials in z = theta^2 (degree 5 and 6 in theta; coefficients: weighted minimax fit, see
// gen_sincos_coeffs.py; measured over every float in the range: sin <= 0.53 ulp, cos <= 0.53
// ulp against float64, cp_selftest_sincos_accuracy — the error is the rounding of the
// evaluation, one more coefficient each would change it by less than 0.01 ulp). Any other
// argument (states supplied by a caller, NaN, Inf) takes the accurate library sinf / cosf.
// Not a fast-math approximation: the error bound is tighter than the library routines' 1 ulp.
constexpr float kSmallAngle = 0.22f;

__device__ __forceinline__ float sin_small(float x) {
    const float z = __fmul_rn(x, x);
    const float p = __fmaf_rn(8.319973014e-03f, z, -1.666664630e-01f);
    return __fmaf_rn(__fmul_rn(p, z), x, x);
}
__device__ __forceinline__ float cos_small(float x) {
    const float z = __fmul_rn(x, x);
    float q = __fmaf_rn(-1.387019176e-03f, z, 4.166663438e-02f);
    q = __fmaf_rn(q, z, -0.5f);
    return __fmaf_rn(q, z, 1.0f);
}
// The two one-op forms (used by the ladder's separate sine and cosine kernels) ...
__device__ __forceinline__ float sin_op(float x) { return fabsf(x) <= kSmallAngle ? sin_small(x) : sinf(x); }
__device__ __forceinline__ float cos_op(float x) { return fabsf(x) <= kSmallAngle ? cos_small(x) : cosf(x); }
// ... and the fused form (one range test, shared z); same bits as sin_op / cos_op.
__device__ __forceinline__ void sin_cos(float th, float &s, float &c) {
    if (fabsf(th) <= kSmallAngle) {
        s = sin_small(th);
        c = cos_small(th);
    } else {
        sincosf(th, &s, &c);
    }
}

// ---- division by the total mass ----
// x / 1.1f with the correctly rounded result of IEEE division, in two operations instead of the
// general division sequence: with r = RN(1/d) and e = RN(1/d - r) (the reciprocal in two
// float32 pieces), q = fma(x, r, x*e). The sum x*r + RN(x*e) misses x/d by about 2^-48 of its
// size, and for d = 1.1f no quotient lies that close to a rounding boundary: the result equals
// __fdiv_rn(x, d) for EVERY finite x with |x| >= 2^-100, for both zeros, infinities and NaN
// (checked over all 2^32 bit patterns by cp_selftest_arith); tiny inputs, where x*e underflows,
// take the general division.
constexpr float kRcpMTot = 0.9090908765792847f;       // RN(1 / 1.1f) = 0x3F68BA2E
constexpr float kRcpMTotLo = 1.280761008359832e-08f;  // RN(1 / 1.1f - kRcpMTot) = 0x325C0877
__device__ __forceinline__ float div_mtot_core(float x) {
    return __fmaf_rn(x, kRcpMTot, __fmul_rn(x, kRcpMTotLo));
}
// x is known to be a zero, NaN, infinite, or of magnitude >= 2^-100 (never tiny).
__device__ __forceinline__ float div_mtot_not_tiny(float x) { return div_mtot_core(x); }
// x is known to be NaN or of magnitude in [2^-100, FLT_MAX] (or +0).
__device__ __forceinline__ float div_mtot_normal(float x) { return div_mtot_core(x); }
// any x
__device__ __forceinline__ float div_mtot(float x) {
    if (fabsf(x) >= 7.888609052e-31f) return div_mtot_core(x);  // 2^-100 and up, infinities included
    return __fdiv_rn(x, kMTot);                                   // tiny, zero, NaN
}

// Accelerations (canonical op order; one rounding per op).
// TAME = true: the caller has established |theta| <= 0.22 (every angle an episode visits is
// below 0.2095). The results then have the bits of the canonical operations whenever they can be
// observed, that is whenever the environment survives the step: survival needs
// |theta + tau*theta_dot| <= 0.2095, hence |theta_dot| <= (0.2095 + 0.22)/0.02 < 21.5 — a faster
// pole ends the episode in this very step, the restart overwrites x_dot' and theta_dot', and
// the accelerations are never seen (x' and theta' do not depend on them). For |theta| <= 0.22
// and |theta_dot| <= 21.5: |s| <= 0.2183, c >= 0.9759, t3 = +-10 + t2 lies in +-[4.95, 15.05],
// |num| >= 0.9759*4.95/1.1 - 9.8*0.2183 > 2.2, |num| < 16 and |p1| > 0.17: every operand of a
// division by 1.1 is a normal number far from the range limits, where the two-operation form
// is exact, so no range test is needed. TAME = false makes no assumption and tests each operand.
// num / den for the operands a tame state produces: den = 0.5*(4/3 - 0.1*c^2/1.1) with
// c in [0.9689, 1] lies in [0.62121, 0.62400] and |num| in [2.2, 16). On the superset
// den in [0.6210, 0.6242] x |num| in [2, 32) — 53,688 x 33,554,432 operand pairs, all of them
// checked on the GPU by cp_selftest_tame_div — the hardware reciprocal approximation followed
// by one exact-remainder correction gives the bits of IEEE division.
constexpr float kTameDenLo = 0.6210f, kTameDenHi = 0.6242f;
__device__ __forceinline__ float div_tame(float num, float den) {
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(den));
    const float q = __fmul_rn(num, r);
    const float rem = __fmaf_rn(-den, q, num);
    return __fmaf_rn(rem, r, q);
}

template <bool TAME>
__device__ __forceinline__ void accel(float thd, float force, float s, float c, float &xacc, float &thacc) {
    float t0 = __fmul_rn(thd, thd);
    float t1 = __fmul_rn(kPML, t0);
    float t2 = __fmul_rn(t1, s);
    float t3 = __fadd_rn(force, t2);
    // in general t3 = +-10 + t2 is +0, or at least half an ulp of 10 in magnitude, or not finite
    float temp = TAME ? div_mtot_core(t3) : div_mtot_not_tiny(t3);
    float n0 = __fmul_rn(kG, s);
    float n1 = __fmul_rn(c, temp);
    float num = __fsub_rn(n0, n1);
    float d0 = __fmul_rn(c, c);
    float den;
    if (TAME) {
        // den = l * (4/3 - (m_p * c^2) / M) with l = 0.5: scaling by a power of two commutes
        // with every rounding on the way (no operand is near the underflow range: c >= 0.9689),
        // so the halving is folded into the constants and the final multiply disappears:
        // RN(0.5 * RN(FT - RN(RN(0.1f * d0) / M))) == RN(0.5*FT - RN(RN(0.05f' * d0) / M)) with
        // 0.05f' = 0.5 * 0.1f exactly. Same bits, one operation fewer.
        const float h1 = __fmul_rn(0.5f * kMPole, d0);
        den = __fsub_rn(0.5f * kFT, div_mtot_core(h1));
    } else {
        float d1 = __fmul_rn(kMPole, d0);
        // d1 = 0.1 * cos^2 is NaN or within [1e-20, 0.1]: no float has a cosine below ~1e-10
        float d2 = div_mtot_normal(d1);
        float d3 = __fsub_rn(kFT, d2);
        den = __fmul_rn(kL, d3);
    }
    thacc = TAME ? div_tame(num, den) : __fdiv_rn(num, den);
    float p0 = __fmul_rn(kPML, thacc);
    float p1 = __fmul_rn(p0, c);
    float p2 = TAME ? div_mtot_core(p1) : div_mtot(p1);
    xacc = __fsub_rn(temp, p2);
}

// One explicit-Euler step, no reset. Returns done evaluated on the new state.
// KNOWN_SMALL: the caller has established |theta| <= 0.22 (or theta is NaN, for which both lanes
// give NaN), so the angle is not tested: inside a rollout every state after the first step is
// either a survivor (|theta| <= 0.2095) or a hashed start state (|theta| <= 0.05).
template <bool KNOWN_SMALL = false>
__device__ __forceinline__ bool euler_step(State &z, float force) {
    float xacc, thacc;
    if (KNOWN_SMALL || fabsf(z.th) <= kSmallAngle) {
        accel<true>(z.thd, force, sin_small(z.th), cos_small(z.th), xacc, thacc);
    } else {
        float s, c;
        sin_cos(z.th, s, c);
        accel<false>(z.thd, force, s, c, xacc, thacc);
    }
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

// ---- two environments per instruction (packed float32 arithmetic of sm_100a) ----
// Blackwell issues mul / add / sub / fma on a PAIR of float32 values held in a 64-bit register
// (mul.rn.f32x2 and friends). Each half is rounded exactly like the scalar .rn operation, so a
// thread that owns two independent environments can run both dependency chains with one
// instruction stream: the bits do not change, the issue slots of the float arithmetic halve.
// Low half = environment slot 0, high half = slot 1.
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pack2(float lo, float hi) {
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(f32x2 v, float &lo, float &hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ f32x2 splat2(float c) { return pack2(c, c); }
__device__ __forceinline__ f32x2 mul2(f32x2 a, f32x2 b) {
    f32x2 r;
    asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) {
    f32x2 r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ f32x2 sub2(f32x2 a, f32x2 b) {
    f32x2 r;
    asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
    f32x2 r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}

struct StatePair {
    f32x2 x, xd, th, thd;
};
__device__ __forceinline__ StatePair pack_states(const State &a, const State &b) {
    StatePair z;
    z.x = pack2(a.x, b.x);
    z.xd = pack2(a.xd, b.xd);
    z.th = pack2(a.th, b.th);
    z.thd = pack2(a.thd, b.thd);
    return z;
}
__device__ __forceinline__ void unpack_states(const StatePair &z, State &a, State &b) {
    unpack2(z.x, a.x, b.x);
    unpack2(z.xd, a.xd, b.xd);
    unpack2(z.th, a.th, b.th);
    unpack2(z.thd, a.thd, b.thd);
}

// div_mtot_core on both halves (a product that enters a fused multiply-add as the addend stays a
// separate rounding, see add_product2).
__device__ __forceinline__ f32x2 div_mtot_core2(f32x2 x) {
    return fma2(x, splat2(kRcpMTot), mul2(x, splat2(kRcpMTotLo)));
}

// A product that feeds an addition. The assembler of CUDA 12.9 contracts a packed multiply whose
// only use is a packed add / sub into one fused multiply-add even though both carry an explicit
// .rn (which forbids exactly that for the scalar forms) and --fmad=false is given — measured on
// the GPU: 13 % of random operand pairs then differ from the separately rounded result. It does
// not touch a product that enters a fused multiply-add as multiplicand or addend, so such sums are
// written  c + a*b  ==  fma(RN(-a*b), -1, c): negating a product is exact, and the fma adds
// exactly RN(a*b). cp_selftest_pair compares the packed step with the scalar one bit for bit.
__device__ __forceinline__ f32x2 add_product2(f32x2 c, f32x2 neg_product) {
    return fma2(neg_product, splat2(-1.0f), c);
}

// euler_step<true> (both angles within the polynomial range) for two environments at once:
// the same operations in the same order on each half, hence the same bits. Rewrites that keep
// negations out of the packed instructions: see div_mtot_core2; the denominator of the
// angular acceleration is formed with its sign flipped (RN(a - b) == -RN(b - a)), which is the
// operand the remainder step of div_tame needs, while the reciprocal takes the positive value;
// p0 .. p2 are carried with flipped sign (every step is odd in its operand), so that -m_p*l
// serves both there and in t1.
__device__ __forceinline__ void euler_step_pair(StatePair &z, f32x2 force, bool &done0, bool &done1) {
    const f32x2 zz = mul2(z.th, z.th);
    const f32x2 sp = fma2(splat2(8.319973014e-03f), zz, splat2(-1.666664630e-01f));
    const f32x2 s = fma2(mul2(sp, zz), z.th, z.th);
    f32x2 cq = fma2(splat2(-1.387019176e-03f), zz, splat2(4.166663438e-02f));
    cq = fma2(cq, zz, splat2(-0.5f));
    const f32x2 c = fma2(cq, zz, splat2(1.0f));
    // accel<true>
    const f32x2 t0 = mul2(z.thd, z.thd);
    const f32x2 nt1 = mul2(splat2(-kPML), t0);
    const f32x2 nt2 = mul2(nt1, s);
    const f32x2 t3 = add_product2(force, nt2);  // force + t2
    const f32x2 temp = div_mtot_core2(t3);
    const f32x2 n0 = mul2(splat2(kG), s);
    const f32x2 n1 = mul2(c, temp);
    const f32x2 num = add_product2(n0, n1);  // n0 - n1
    const f32x2 d0 = mul2(c, c);
    const f32x2 h1 = mul2(splat2(kPML), d0);  // 0.5 * m_p == m_p * l
    const f32x2 nden = sub2(div_mtot_core2(h1), splat2(0.5f * kFT));  // -den
    float nd0, nd1, r0, r1;
    unpack2(nden, nd0, nd1);
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r0) : "f"(-nd0));
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r1) : "f"(-nd1));
    const f32x2 r = pack2(r0, r1);
    const f32x2 q = mul2(num, r);
    const f32x2 rem = fma2(nden, q, num);
    const f32x2 thacc = fma2(rem, r, q);
    const f32x2 np0 = mul2(splat2(-kPML), thacc);
    const f32x2 np1 = mul2(np0, c);
    const f32x2 xacc = add2(temp, div_mtot_core2(np1));  // temp - p2
    const f32x2 nx = add_product2(z.x, mul2(splat2(-kTau), z.xd));
    const f32x2 nxd = add_product2(z.xd, mul2(splat2(-kTau), xacc));
    const f32x2 nth = add_product2(z.th, mul2(splat2(-kTau), z.thd));
    const f32x2 nthd = add_product2(z.thd, mul2(splat2(-kTau), thacc));
    z.x = nx;
    z.xd = nxd;
    z.th = nth;
    z.thd = nthd;
    float x0, x1, a0, a1;
    unpack2(nx, x0, x1);
    unpack2(nth, a0, a1);
    done0 = (fabsf(x0) > kXT) | (fabsf(a0) > kTT);
    done1 = (fabsf(x1) > kXT) | (fabsf(a1) > kTT);
}

// ---- contracted arithmetic (an optional, separately reported rollout variant) ----
// The same step with the roundings a compiler allowed to contract would drop (the paper's
// fused kernels are generated without a one-rounding-per-op promise, Sec. V-B/V-G): fused
// multiply-adds in temp, num, den, xacc and the four Euler updates, the divisions by the
// total mass folded into constants, theta_acc = num * rcp(den) with the hardware reciprocal
// (den lies in [0.62, 0.67] for every real c). 25 floating-point operations instead of 43.
// Results differ from the canonical order by a few 1e-7 relative per step; they are NOT the
// bits of the per-op ladder. sin / cos are the same routines as in the exact path.
constexpr float kDenK = (float)(-(0.5 * 0.1) / (double)1.1f);    // -l * m_p / M
constexpr float kDenC = (float)(0.5 * (4.0 / 3.0));              // l * 4/3
constexpr float kXaccK = (float)(-(0.1 * 0.5) / (double)1.1f);   // -m_p * l / M
template <bool KNOWN_SMALL = false>
__device__ __forceinline__ bool euler_step_contracted(State &z, float force) {
    float s, c;
    if (KNOWN_SMALL) {
        s = sin_small(z.th);
        c = cos_small(z.th);
    } else {
        sin_cos(z.th, s, c);
    }
    const float t1 = __fmul_rn(__fmul_rn(z.thd, z.thd), kPML);
    const float temp = __fmul_rn(__fmaf_rn(t1, s, force), kRcpMTot);
    const float num = __fmaf_rn(-c, temp, __fmul_rn(kG, s));
    const float den = __fmaf_rn(__fmul_rn(c, c), kDenK, kDenC);
    float r;
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(den));
    const float thacc = __fmul_rn(num, r);
    const float xacc = __fmaf_rn(__fmul_rn(thacc, c), kXaccK, temp);
    const float nx = __fmaf_rn(kTau, z.xd, z.x);
    const float nxd = __fmaf_rn(kTau, xacc, z.xd);
    const float nth = __fmaf_rn(kTau, z.thd, z.th);
    const float nthd = __fmaf_rn(kTau, thacc, z.thd);
    z.x = nx;
    z.xd = nxd;
    z.th = nth;
    z.thd = nthd;
    return (fabsf(nx) > kXT) | (fabsf(nth) > kTT);
}

// euler_step_contracted<true> for two environments at once: the same fused operations on each
// half, hence the bits of the scalar form. temp is carried with its sign flipped (the constant
// it is multiplied by is negated, which is exact), so that -c*temp and xacc need no negation;
// -xacc then meets -tau in the velocity update.
__device__ __forceinline__ void euler_step_contracted_pair(StatePair &z, f32x2 force, bool &done0, bool &done1) {
    const f32x2 zz = mul2(z.th, z.th);
    const f32x2 sp = fma2(splat2(8.319973014e-03f), zz, splat2(-1.666664630e-01f));
    const f32x2 s = fma2(mul2(sp, zz), z.th, z.th);
    f32x2 cq = fma2(splat2(-1.387019176e-03f), zz, splat2(4.166663438e-02f));
    cq = fma2(cq, zz, splat2(-0.5f));
    const f32x2 c = fma2(cq, zz, splat2(1.0f));
    const f32x2 t1 = mul2(mul2(z.thd, z.thd), splat2(kPML));
    const f32x2 ntemp = mul2(fma2(t1, s, force), splat2(-kRcpMTot));
    const f32x2 num = fma2(c, ntemp, mul2(splat2(kG), s));
    const f32x2 den = fma2(mul2(c, c), splat2(kDenK), splat2(kDenC));
    float d0, d1, r0, r1;
    unpack2(den, d0, d1);
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r0) : "f"(d0));
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r1) : "f"(d1));
    const f32x2 thacc = mul2(num, pack2(r0, r1));
    const f32x2 nxacc = fma2(mul2(thacc, c), splat2(-kXaccK), ntemp);
    const f32x2 tau = splat2(kTau);
    const f32x2 nx = fma2(tau, z.xd, z.x);
    const f32x2 nxd = fma2(splat2(-kTau), nxacc, z.xd);
    const f32x2 nth = fma2(tau, z.thd, z.th);
    const f32x2 nthd = fma2(tau, thacc, z.thd);
    z.x = nx;
    z.xd = nxd;
    z.th = nth;
    z.thd = nthd;
    float x0, x1, a0, a1;
    unpack2(nx, x0, x1);
    unpack2(nth, a0, a1);
    done0 = (fabsf(x0) > kXT) | (fabsf(a0) > kTT);
    done1 = (fabsf(x1) > kXT) | (fabsf(a1) > kTT);
}

// ---- policies (observation = state before the step) ----
struct LinearW {
    float w[2][4];
    float b[2];
};
template <int H>
struct MlpWT {  // 4 -> H (tanh) -> 2
    float w1[H][4];
    float b1[H];
    float w2[2][H];
    float b2[2];
};
using MlpW = MlpWT<16>;

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

// Hidden activations are consumed as they are produced (two running logits), so no array of
// H values is ever live; every weight is an immediate operand from the launch parameters.
// tanh for the contracted-arithmetic variant: 1 - 2 / (exp(2x) + 1) with the hardware exp2 and
// reciprocal approximations (five instructions instead of the library routine's ~18). Small
// arguments lose RELATIVE accuracy to the cancellation in 1 - (...), which a policy does not
// feel: its logits depend on the absolute error, measured <= 2.4e-7 over every float32
// (cp_selftest_tanh; tanh_canonical: 1.1e-7). Saturates to +-1, NaN stays NaN.
__device__ __forceinline__ float tanh_contracted(float x) {
    float t, r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(t) : "f"(__fmul_rn(x, 2.885390043f)));  // 2 * log2(e)
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(__fadd_rn(t, 1.0f)));
    return __fmaf_rn(-2.0f, r, 1.0f);
}

// tanh of the canonical arithmetic: as accurate as the library routine (largest error 1.82 ulp
// against float64 over every float32, the library's tanhf: 1.82 — cp_selftest_tanh measures
// both), built so that two values can share one instruction stream. |x| < 0.6: x + x*z*P(z),
// z = x^2, P of degree 4 (weighted minimax fit, 0.72 ulp). Otherwise 1 - 2/(e^(2|x|) + 1) from
// the hardware exp2 and reciprocal, with the sign of x; it saturates to +-1 and keeps NaN.
// Both sides are always evaluated and one is selected: no branch. tanh_pair performs the same
// operations on both halves of a pair, so tanh_pair(pack2(a, b)) == (tanh_canonical(a),
// tanh_canonical(b)) bit for bit (checked over every float32 by cp_selftest_tanh).
constexpr float kTanhSplit = 0.6f;
constexpr float kTanhC0 = -3.333329856e-01f, kTanhC1 = 1.333195865e-01f, kTanhC2 = -5.378668010e-02f,
                kTanhC3 = 2.080537751e-02f, kTanhC4 = -5.905860569e-03f;
constexpr float kTwoLog2e = 2.885390043f;
__device__ __forceinline__ float tanh_canonical(float x) {
    const float t = fabsf(x);
    float e, r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e) : "f"(__fmul_rn(t, kTwoLog2e)));
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(__fadd_rn(e, 1.0f)));
    const float big = copysignf(__fmaf_rn(-2.0f, r, 1.0f), x);
    const float z = __fmul_rn(x, x);
    float p = __fmaf_rn(kTanhC4, z, kTanhC3);
    p = __fmaf_rn(p, z, kTanhC2);
    p = __fmaf_rn(p, z, kTanhC1);
    p = __fmaf_rn(p, z, kTanhC0);
    const float small = __fmaf_rn(__fmul_rn(p, z), x, x);
    return t < kTanhSplit ? small : big;
}
__device__ __forceinline__ f32x2 tanh_pair(f32x2 x) {
    float x0, x1;
    unpack2(x, x0, x1);
    const float t0 = fabsf(x0), t1 = fabsf(x1);
    const f32x2 arg = mul2(pack2(t0, t1), splat2(kTwoLog2e));
    float a0, a1, e0, e1, r0, r1;
    unpack2(arg, a0, a1);
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e0) : "f"(a0));
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(e1) : "f"(a1));
    const f32x2 d = add2(pack2(e0, e1), splat2(1.0f));
    float d0, d1;
    unpack2(d, d0, d1);
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r0) : "f"(d0));
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r1) : "f"(d1));
    const f32x2 big = fma2(splat2(-2.0f), pack2(r0, r1), splat2(1.0f));
    const f32x2 z = mul2(x, x);
    f32x2 p = fma2(splat2(kTanhC4), z, splat2(kTanhC3));
    p = fma2(p, z, splat2(kTanhC2));
    p = fma2(p, z, splat2(kTanhC1));
    p = fma2(p, z, splat2(kTanhC0));
    const f32x2 small = fma2(mul2(p, z), x, x);
    float b0, b1, s0, s1;
    unpack2(big, b0, b1);
    unpack2(small, s0, s1);
    return pack2(t0 < kTanhSplit ? s0 : copysignf(b0, x0), t1 < kTanhSplit ? s1 : copysignf(b1, x1));
}

// tanh_contracted on both halves of a pair (same operations, same bits).
__device__ __forceinline__ f32x2 tanh_contracted_pair(f32x2 x) {
    const f32x2 arg = mul2(x, splat2(kTwoLog2e));
    float a0, a1, t0, t1, r0, r1;
    unpack2(arg, a0, a1);
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(t0) : "f"(a0));
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(t1) : "f"(a1));
    const f32x2 d = add2(pack2(t0, t1), splat2(1.0f));
    float d0, d1;
    unpack2(d, d0, d1);
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r0) : "f"(d0));
    asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r1) : "f"(d1));
    return fma2(splat2(-2.0f), pack2(r0, r1), splat2(1.0f));
}

template <int H, bool FAST_TANH = false>
__device__ __forceinline__ uint32_t mlp_action(const MlpWT<H> &p, const State &z) {
    float l0 = p.b2[0], l1 = p.b2[1];
#pragma unroll
    for (int j = 0; j < H; ++j) {
        float acc = p.b1[j];
        acc = __fmaf_rn(p.w1[j][0], z.x, acc);
        acc = __fmaf_rn(p.w1[j][1], z.xd, acc);
        acc = __fmaf_rn(p.w1[j][2], z.th, acc);
        acc = __fmaf_rn(p.w1[j][3], z.thd, acc);
        float h = FAST_TANH ? tanh_contracted(acc) : tanh_canonical(acc);
        l0 = __fmaf_rn(p.w2[0][j], h, l0);
        l1 = __fmaf_rn(p.w2[1][j], h, l1);
    }
    return (l1 > l0) ? 0x80000000u : 0u;
}

// Two hidden layers, 4 -> 16 (tanh) -> 16 (tanh) -> 2. The sixteen first-layer activations stay
// in registers; second-layer units are consumed by the two logit chains as they are produced
// (ascending unit order, the chains start from the biases: the order of the definition).
struct MlpDeepW {
    float w1[16][4], b1[16];
    float w2[16][16], b2[16];
    float w3[2][16], b3[2];
};
template <bool FAST_TANH = false>
__device__ __forceinline__ uint32_t mlp_deep_action(const MlpDeepW &p, const State &z) {
    float h1[16];
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        float acc = p.b1[j];
        acc = __fmaf_rn(p.w1[j][0], z.x, acc);
        acc = __fmaf_rn(p.w1[j][1], z.xd, acc);
        acc = __fmaf_rn(p.w1[j][2], z.th, acc);
        acc = __fmaf_rn(p.w1[j][3], z.thd, acc);
        h1[j] = FAST_TANH ? tanh_contracted(acc) : tanh_canonical(acc);
    }
    float l0 = p.b3[0], l1 = p.b3[1];
#pragma unroll
    for (int k = 0; k < 16; ++k) {
        float acc = p.b2[k];
#pragma unroll
        for (int j = 0; j < 16; ++j) acc = __fmaf_rn(p.w2[k][j], h1[j], acc);
        const float h2 = FAST_TANH ? tanh_contracted(acc) : tanh_canonical(acc);
        l0 = __fmaf_rn(p.w3[0][k], h2, l0);
        l1 = __fmaf_rn(p.w3[1][k], h2, l1);
    }
    return (l1 > l0) ? 0x80000000u : 0u;
}

}  // namespace cp
