// The unfused ladder: the same step as the fused kernel, executed as one kernel
// per elementwise operation with every intermediate written to and re-read from
// an HBM plane. It stands in for eager per-op execution (paper Sec. V-F: dozens
// more kernels than the fused baseline, 0.13x) and is the bottom rung of the
// fusion comparison. It uses the very same rounded operations, so its results
// equal the fused step bit for bit.
//
// 45 launches per step (46 when the action is hashed):
//   K00 action hash (only if no action is supplied)
//   K01 force | K02 sin | K03 cos | K04-K08 temp chain | K09-K17 theta_acc chain
//   K18-K21 x_acc chain | K22-K29 Euler (mul, add) x 4 | K30-K33 four compares
//   K34-K36 three ORs | K37 reward fill | K38-K41 start-state values | K42-K45 selects
// Each kernel is vectorised (4 elements per thread) like a tuned eager kernel would be.
#include "cartpole_device.cuh"
#include "cartpole_internal.h"

namespace cp {

namespace {

template <typename T>
struct Vec4;
template <>
struct Vec4<float> {
    using type = float4;
};
template <>
struct Vec4<uint8_t> {
    using type = uchar4;
};

template <typename T>
__device__ __forceinline__ void load4(const T *p, int64_t i, int cnt, bool vec, T (&r)[4]) {
    if (vec && cnt == 4) {
        typename Vec4<T>::type v = *reinterpret_cast<const typename Vec4<T>::type *>(p + i);
        r[0] = v.x; r[1] = v.y; r[2] = v.z; r[3] = v.w;
    } else {
#pragma unroll
        for (int j = 0; j < 4; ++j) r[j] = j < cnt ? p[i + j] : T(0);
    }
}

template <typename T>
__device__ __forceinline__ void store4(T *p, int64_t i, int cnt, bool vec, const T (&r)[4]) {
    if (vec && cnt == 4) {
        typename Vec4<T>::type v;
        v.x = r[0]; v.y = r[1]; v.z = r[2]; v.w = r[3];
        *reinterpret_cast<typename Vec4<T>::type *>(p + i) = v;
    } else {
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if (j < cnt) p[i + j] = r[j];
    }
}

// Every kernel may be launched with programmatic stream serialization (Launcher::go): it waits
// for the launch before it — whose plane it reads — ahead of its first memory access, and lets the
// launch after it be set up at once; that one waits the same way. (Without the launch attribute
// both calls return immediately.)
#define CP_EW_PROLOGUE                                                          \
    cudaGridDependencySynchronize();                                            \
    cudaTriggerProgrammaticLaunchCompletion();                                  \
    const int64_t i = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;     \
    if (i >= n) return;                                                         \
    const int cnt = (n - i) < 4 ? (int)(n - i) : 4;

// out[i] = op(global index)
template <class Op, typename TO>
__global__ void __launch_bounds__(256) ew0(int64_t n, bool vec, TO *out, Op op) {
    CP_EW_PROLOGUE
    TO r[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) r[j] = op(i + j);
    store4(out, i, cnt, vec, r);
}

template <class Op, typename TO, typename TA>
__global__ void __launch_bounds__(256) ew1(int64_t n, bool vec, TO *out, const TA *a, Op op) {
    CP_EW_PROLOGUE
    TA ra[4];
    TO r[4];
    load4(a, i, cnt, vec, ra);
#pragma unroll
    for (int j = 0; j < 4; ++j) r[j] = op(ra[j]);
    store4(out, i, cnt, vec, r);
}

template <class Op, typename TO, typename TA, typename TB>
__global__ void __launch_bounds__(256) ew2(int64_t n, bool vec, TO *out, const TA *a, const TB *b, Op op) {
    CP_EW_PROLOGUE
    TA ra[4];
    TB rb[4];
    TO r[4];
    load4(a, i, cnt, vec, ra);
    load4(b, i, cnt, vec, rb);
#pragma unroll
    for (int j = 0; j < 4; ++j) r[j] = op(ra[j], rb[j]);
    store4(out, i, cnt, vec, r);
}

template <class Op, typename TO, typename TA, typename TB, typename TC>
__global__ void __launch_bounds__(256) ew3(int64_t n, bool vec, TO *out, const TA *a, const TB *b, const TC *c,
                                           Op op) {
    CP_EW_PROLOGUE
    TA ra[4];
    TB rb[4];
    TC rc[4];
    TO r[4];
    load4(a, i, cnt, vec, ra);
    load4(b, i, cnt, vec, rb);
    load4(c, i, cnt, vec, rc);
#pragma unroll
    for (int j = 0; j < 4; ++j) r[j] = op(ra[j], rb[j], rc[j]);
    store4(out, i, cnt, vec, r);
}

// ---- the elementwise operations ----
struct OpActionHash {
    uint32_t salt_a, env_offset, t;
    __device__ uint8_t operator()(int64_t i) const {
        return (uint8_t)(step_hash(make_keys(salt_a, env_offset + (uint32_t)i), t) >> 31);
    }
};
struct OpStartValue {
    uint32_t salt_r, env_offset, t, j;
    __device__ float operator()(int64_t i) const {
        return start_value(make_keys(salt_r, env_offset + (uint32_t)i), t, j);
    }
};
struct OpFill {
    float v;
    __device__ float operator()(int64_t) const { return v; }
};
struct OpForce {
    __device__ float operator()(uint8_t a) const { return a ? kF : -kF; }
};
struct OpSin {
    __device__ float operator()(float x) const { return sin_op(x); }
};
struct OpCos {
    __device__ float operator()(float x) const { return cos_op(x); }
};
struct OpMulC {
    float c;
    __device__ float operator()(float x) const { return __fmul_rn(c, x); }
};
struct OpDivC {
    float c;
    __device__ float operator()(float x) const { return __fdiv_rn(x, c); }
};
struct OpRSubC {
    float c;
    __device__ float operator()(float x) const { return __fsub_rn(c, x); }
};
struct OpLtC {
    float c;
    __device__ uint8_t operator()(float x) const { return x < c; }
};
struct OpGtC {
    float c;
    __device__ uint8_t operator()(float x) const { return x > c; }
};
struct OpMul {
    __device__ float operator()(float a, float b) const { return __fmul_rn(a, b); }
};
struct OpAdd {
    __device__ float operator()(float a, float b) const { return __fadd_rn(a, b); }
};
struct OpSub {
    __device__ float operator()(float a, float b) const { return __fsub_rn(a, b); }
};
struct OpDiv {
    __device__ float operator()(float a, float b) const { return __fdiv_rn(a, b); }
};
struct OpOr {
    __device__ uint8_t operator()(uint8_t a, uint8_t b) const { return a | b; }
};
struct OpSelect {
    __device__ float operator()(uint8_t m, float a, float b) const { return m ? a : b; }
};

inline bool aligned(const void *p, size_t a) { return (reinterpret_cast<uintptr_t>(p) % a) == 0; }

constexpr int kFloatPlanes = 33;
constexpr int kBytePlanes = 7;

inline int64_t padded(int64_t n) { return (n + 63) / 64 * 64; }  // 256-byte float planes

struct Launcher {
    int64_t n;
    cudaStream_t s;
    unsigned grid() const { return (unsigned)(((n + 3) / 4 + 255) / 256); }
    // One launch of the ladder. With g_tuning.step_pdl the launch may be set up while the one
    // before it in the stream still runs (the kernels wait for it themselves): what an eager
    // executor that issues one kernel per operation can do about launch latency without fusing.
    template <typename... P, typename... A>
    void go(void (*kernel)(P...), A... args) const {
        if (!g_tuning.step_pdl) {
            kernel<<<grid(), 256, 0, s>>>(args...);
        } else {
            cudaLaunchConfig_t cfg = {};
            cfg.gridDim = dim3(grid());
            cfg.blockDim = dim3(256);
            cfg.stream = s;
            cudaLaunchAttribute attr[1];
            attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            attr[0].val.programmaticStreamSerializationAllowed = 1;
            cfg.attrs = attr;
            cfg.numAttrs = 1;
            cudaLaunchKernelEx(&cfg, kernel, P(args)...);
        }
        count_launch();
    }
    template <class Op, typename TO>
    void gen(TO *out, Op op) const {
        go(ew0<Op, TO>, n, aligned(out, 4 * sizeof(TO)), out, op);
    }
    template <class Op, typename TO, typename TA>
    void un(TO *out, const TA *a, Op op) const {
        const bool v = aligned(out, 4 * sizeof(TO)) && aligned(a, 4 * sizeof(TA));
        go(ew1<Op, TO, TA>, n, v, out, a, op);
    }
    template <class Op, typename TO, typename TA, typename TB>
    void bin(TO *out, const TA *a, const TB *b, Op op) const {
        const bool v = aligned(out, 4 * sizeof(TO)) && aligned(a, 4 * sizeof(TA)) && aligned(b, 4 * sizeof(TB));
        go(ew2<Op, TO, TA, TB>, n, v, out, a, b, op);
    }
    template <class Op, typename TO, typename TA, typename TB, typename TC>
    void tri(TO *out, const TA *a, const TB *b, const TC *c, Op op) const {
        const bool v = aligned(out, 4 * sizeof(TO)) && aligned(a, 4 * sizeof(TA)) && aligned(b, 4 * sizeof(TB)) &&
                       aligned(c, 4 * sizeof(TC));
        go(ew3<Op, TO, TA, TB, TC>, n, v, out, a, b, c, op);
    }
};

}  // namespace

size_t ladder_workspace_bytes(int64_t n) {
    const int64_t np = padded(n);
    return (size_t)np * (kFloatPlanes * sizeof(float)) + (size_t)padded((np + 3) / 4) * 4 * kBytePlanes;
}

int ladder_launch_count(bool hashed_action) { return hashed_action ? 46 : 45; }

cudaError_t launch_ladder(const StepParams &p, void *workspace, cudaStream_t s) {
    const int64_t n = p.n;
    const int64_t np = padded(n);
    float *fbase = static_cast<float *>(workspace);
    uint8_t *bbase = reinterpret_cast<uint8_t *>(fbase + (size_t)np * kFloatPlanes);
    const int64_t bp = padded((np + 3) / 4) * 4;
    int fi = 0, bi = 0;
    auto F = [&]() { return fbase + (size_t)np * (fi++); };
    auto B = [&]() { return bbase + (size_t)bp * (bi++); };

    const float *x = p.in, *xd = p.in + p.in_stride, *th = p.in + 2 * p.in_stride, *thd = p.in + 3 * p.in_stride;
    float *ox = p.out, *oxd = p.out + p.out_stride, *oth = p.out + 2 * p.out_stride, *othd = p.out + 3 * p.out_stride;
    Launcher L{n, s};

    const uint8_t *a = p.action;
    if (!a) {
        uint8_t *ah = B();
        L.gen(ah, OpActionHash{p.salt_a, p.env_offset, p.t});  // K00
        a = ah;
    } else {
        B();
    }
    float *force = F(), *sn = F(), *cs = F();
    L.un(force, a, OpForce{});  // K01
    L.un(sn, th, OpSin{});      // K02
    L.un(cs, th, OpCos{});      // K03
    float *t0 = F(), *t1 = F(), *t2 = F(), *t3 = F(), *temp = F();
    L.bin(t0, thd, thd, OpMul{});      // K04
    L.un(t1, t0, OpMulC{kPML});        // K05
    L.bin(t2, t1, sn, OpMul{});        // K06
    L.bin(t3, force, t2, OpAdd{});     // K07
    L.un(temp, t3, OpDivC{kMTot});     // K08
    float *n0 = F(), *n1 = F(), *num = F(), *d0 = F(), *d1 = F(), *d2 = F(), *d3 = F(), *den = F(), *thacc = F();
    L.un(n0, sn, OpMulC{kG});          // K09
    L.bin(n1, cs, temp, OpMul{});      // K10
    L.bin(num, n0, n1, OpSub{});       // K11
    L.bin(d0, cs, cs, OpMul{});        // K12
    L.un(d1, d0, OpMulC{kMPole});      // K13
    L.un(d2, d1, OpDivC{kMTot});       // K14
    L.un(d3, d2, OpRSubC{kFT});        // K15
    L.un(den, d3, OpMulC{kL});         // K16
    L.bin(thacc, num, den, OpDiv{});   // K17
    float *p0 = F(), *p1 = F(), *p2 = F(), *xacc = F();
    L.un(p0, thacc, OpMulC{kPML});     // K18
    L.bin(p1, p0, cs, OpMul{});        // K19
    L.un(p2, p1, OpDivC{kMTot});       // K20
    L.bin(xacc, temp, p2, OpSub{});    // K21
    float *e0 = F(), *nx = F(), *e1 = F(), *nxd = F(), *e2 = F(), *nth = F(), *e3 = F(), *nthd = F();
    L.un(e0, xd, OpMulC{kTau});        // K22
    L.bin(nx, x, e0, OpAdd{});         // K23
    L.un(e1, xacc, OpMulC{kTau});      // K24
    L.bin(nxd, xd, e1, OpAdd{});       // K25
    L.un(e2, thd, OpMulC{kTau});       // K26
    L.bin(nth, th, e2, OpAdd{});       // K27
    L.un(e3, thacc, OpMulC{kTau});     // K28
    L.bin(nthd, thd, e3, OpAdd{});     // K29
    uint8_t *c0 = B(), *c1 = B(), *c2 = B(), *c3 = B(), *o0 = B(), *o1 = B();
    L.un(c0, nx, OpLtC{-kXT});         // K30
    L.un(c1, nx, OpGtC{kXT});          // K31
    L.un(c2, nth, OpLtC{-kTT});        // K32
    L.un(c3, nth, OpGtC{kTT});         // K33
    L.bin(o0, c0, c1, OpOr{});         // K34
    L.bin(o1, c2, c3, OpOr{});         // K35
    L.bin(p.done, o0, o1, OpOr{});     // K36
    L.gen(p.reward, OpFill{1.0f});     // K37
    float *r0 = F(), *r1 = F(), *r2 = F(), *r3 = F();
    L.gen(r0, OpStartValue{p.salt_r, p.env_offset, p.t + 1u, 0});  // K38
    L.gen(r1, OpStartValue{p.salt_r, p.env_offset, p.t + 1u, 1});  // K39
    L.gen(r2, OpStartValue{p.salt_r, p.env_offset, p.t + 1u, 2});  // K40
    L.gen(r3, OpStartValue{p.salt_r, p.env_offset, p.t + 1u, 3});  // K41
    L.tri(ox, (const uint8_t *)p.done, (const float *)r0, (const float *)nx, OpSelect{});      // K42
    L.tri(oxd, (const uint8_t *)p.done, (const float *)r1, (const float *)nxd, OpSelect{});    // K43
    L.tri(oth, (const uint8_t *)p.done, (const float *)r2, (const float *)nth, OpSelect{});    // K44
    L.tri(othd, (const uint8_t *)p.done, (const float *)r3, (const float *)nthd, OpSelect{});  // K45
    (void)fi;
    (void)bi;
    return cudaGetLastError();
}

}  // namespace cp
