/*
 * cartpole_oracle.c — plain scalar CPU oracle for the batched CartPole step.
 *
 * TEST INFRASTRUCTURE ONLY. This file is the slow, obviously-correct statement
 * of what the CUDA library must compute. It shares no code, header, table or
 * constant generator with the CUDA path; only the tests, the smoke check and
 * the benchmark's CPU-baseline leg may build, load or call it.
 *
 * What it follows (paper: "Operator Fusion in XLA: Analysis and Evaluation"):
 *   - Sec. IV "Case Study on Cart-pole": the environment update function is a
 *     chain of elementwise float32 ops over N independent environments
 *     (force from the action, sin/cos of the pole angle, the shared `temp`
 *     term, angular and linear acceleration, four explicit-Euler updates,
 *     termination test, reward, reset of finished environments).
 *   - Sec. V (Evaluations): N parallel environments are stepped T times with
 *     random actions and random start states; Sec. V-A replaces the library
 *     RNG kernel by values that need no separate kernel — here a stateless
 *     counter hash of (seed, env, step).
 *   - Sec. V-C "no concat": the state is four separate per-environment values
 *     (x, x_dot, theta, theta_dot); the batch layout is four planes.
 *   The equations of motion are the classical cart-pole ones the paper cites
 *   (uniform pole of half-length l on a cart, force +-F), constants
 *   g=9.8, m_cart=1.0, m_pole=0.1, l=0.5, F=10, tau=0.02, terminate when
 *   |x|>2.4 or |theta|>12 degrees.
 *
 * Arithmetic: float32, one rounding per written operation, no contraction
 * (build with -ffp-contract=off -fno-fast-math), glibc sinf/cosf/tanhf. The
 * policy dot products are the one place where a fused multiply-add is
 * specified (fmaf). A float64 copy of the dynamics exists for the pins.
 *
 * Parity pins: every function here is pinned by tests/test_oracle_*.py
 * (Lagrangian 2x2 solve, exact rational first step, mirror antisymmetry,
 * linearised closed form, hash bijection/inverse, constant derivations,
 * brute-force tiny batches). sinf/cosf/tanhf last-bit behaviour is glibc's
 * and is "parity unpinned" beyond the stated float tolerances.
 */
#include <math.h>
#include <pthread.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------ */
/* Counter hash (definition H). All arithmetic is mod 2^32.            */
/* ------------------------------------------------------------------ */

#define CO_MA 0x6A09E667u /* floor(frac(sqrt 2) * 2^32) */
#define CO_MB 0xBB67AE85u /* floor(frac(sqrt 3) * 2^32) */
#define CO_MG 0x9E3779B1u /* 2654435761: the prime next below 2^32 / golden ratio */

uint32_t co_mix32(uint32_t h)
{
    h ^= h >> 16;
    h *= CO_MA;
    h ^= h >> 15;
    h *= CO_MB;
    h ^= h >> 16;
    return h;
}

/* Per-(seed, stream) salt. stream 0 = actions, 1 = reset states. */
uint32_t co_salt(uint32_t seed, uint32_t stream)
{
    return co_mix32(co_mix32(seed ^ CO_MG) + stream);
}

/* Per-environment key pair, invariant over time. */
void co_keys(uint32_t seed, uint32_t env, uint32_t stream, uint32_t *k0, uint32_t *k1)
{
    uint32_t s0 = co_salt(seed, stream);
    *k0 = co_mix32(env ^ s0);
    *k1 = co_mix32(*k0 + CO_MG);
}

uint32_t co_step_hash(uint32_t k0, uint32_t k1, uint32_t c)
{
    uint32_t h = k0 ^ c;
    h = (h ^ (h >> 16)) * CO_MA + k1;
    h = (h ^ (h >> 15)) * CO_MB;
    h ^= h >> 16;
    return h;
}

/* Bernoulli(1/2) action of environment `env` at global step t. */
uint32_t co_action(uint32_t seed, uint32_t env, uint32_t t)
{
    uint32_t k0, k1;
    co_keys(seed, env, 0u, &k0, &k1);
    return co_step_hash(k0, k1, t) >> 31;
}

/* Start state of an episode of `env` that begins at global time t:
 * four 24-bit uniforms mapped to [-0.05, 0.05). u - 0.5f is exact, so each
 * component is rounded exactly once (the final multiply). */
void co_reset_state(uint32_t seed, uint32_t env, uint32_t t, float out[4])
{
    uint32_t k0, k1;
    co_keys(seed, env, 1u, &k0, &k1);
    for (uint32_t j = 0; j < 4; ++j) {
        uint32_t bits = co_step_hash(k0, k1, 4u * t + j) >> 8;
        float u = (float)bits * 0x1p-24f;
        out[j] = (u - 0.5f) * 0.1f;
    }
}

/* ------------------------------------------------------------------ */
/* Dynamics: one explicit-Euler step, float32, canonical op order.     */
/* ------------------------------------------------------------------ */

static const float CO_G = 9.8f;
static const float CO_MPOLE = 0.1f;
static const float CO_MTOT = 1.1f;  /* m_cart + m_pole */
static const float CO_L = 0.5f;     /* half pole length */
static const float CO_PML = 0.05f;  /* m_pole * l */
static const float CO_F = 10.0f;
static const float CO_TAU = 0.02f;
static const float CO_FT = (float)(4.0 / 3.0);
static const float CO_XT = 2.4f;
static const float CO_TT = (float)(12.0 * 2.0 * 3.14159265358979323846 / 360.0);

/* Accelerations for state z = (x, x_dot, theta, theta_dot) and action a. */
void co_accel_f32(const float z[4], int a, float *xacc_out, float *thacc_out)
{
    float th = z[2], thd = z[3];
    float force = a ? CO_F : -CO_F;
    float s = sinf(th);
    float c = cosf(th);
    float t0 = thd * thd;
    float t1 = CO_PML * t0;
    float t2 = t1 * s;
    float t3 = force + t2;
    float temp = t3 / CO_MTOT;
    float n0 = CO_G * s;
    float n1 = c * temp;
    float num = n0 - n1;
    float d0 = c * c;
    float d1 = CO_MPOLE * d0;
    float d2 = d1 / CO_MTOT;
    float d3 = CO_FT - d2;
    float den = CO_L * d3;
    float thacc = num / den;
    float p0 = CO_PML * thacc;
    float p1 = p0 * c;
    float p2 = p1 / CO_MTOT;
    float xacc = temp - p2;
    *xacc_out = xacc;
    *thacc_out = thacc;
}

/* One step without reset: out = state after the Euler update; returns the
 * termination flag evaluated on that post-update state (strict compares). */
int co_dynamics_f32(const float z[4], int a, float out[4])
{
    float xacc, thacc;
    co_accel_f32(z, a, &xacc, &thacc);
    float e0 = CO_TAU * z[1];
    float e1 = CO_TAU * xacc;
    float e2 = CO_TAU * z[3];
    float e3 = CO_TAU * thacc;
    out[0] = z[0] + e0;
    out[1] = z[1] + e1;
    out[2] = z[2] + e2;
    out[3] = z[3] + e3;
    return (out[0] < -CO_XT) | (out[0] > CO_XT) | (out[2] < -CO_TT) | (out[2] > CO_TT);
}

/* float64 copy (decimal constants, not the float32 roundings), for pins. */
void co_accel_f64(const double z[4], int a, double *xacc_out, double *thacc_out)
{
    const double g = 9.8, mp = 0.1, mt = 1.1, l = 0.5, pml = 0.05, F = 10.0;
    double th = z[2], thd = z[3];
    double force = a ? F : -F;
    double s = sin(th), c = cos(th);
    double temp = (force + pml * (thd * thd) * s) / mt;
    double thacc = (g * s - c * temp) / (l * (4.0 / 3.0 - mp * (c * c) / mt));
    double xacc = temp - pml * thacc * c / mt;
    *xacc_out = xacc;
    *thacc_out = thacc;
}

int co_dynamics_f64(const double z[4], int a, double out[4])
{
    const double tau = 0.02, xt = 2.4, tt = 12.0 * 2.0 * 3.14159265358979323846 / 360.0;
    double xacc, thacc;
    co_accel_f64(z, a, &xacc, &thacc);
    out[0] = z[0] + tau * z[1];
    out[1] = z[1] + tau * xacc;
    out[2] = z[2] + tau * z[3];
    out[3] = z[3] + tau * thacc;
    return (out[0] < -xt) | (out[0] > xt) | (out[2] < -tt) | (out[2] > tt);
}

/* ------------------------------------------------------------------ */
/* Policies: observation is the state before the step.                 */
/* kind 0: hashed random action. kind 1: linear 4->2. kind 2: MLP      */
/* 4->16 (tanh)->2. argmax with index 0 winning ties.                  */
/* ------------------------------------------------------------------ */

#define CO_POLICY_RANDOM 0
#define CO_POLICY_LINEAR 1
#define CO_POLICY_MLP 2
#define CO_MLP_HIDDEN 16

/* Linear weights: W[2][4] row-major, then b[2] (10 floats). */
void co_linear_logits(const float *w, const float z[4], float logits[2])
{
    const float *b = w + 8;
    for (int k = 0; k < 2; ++k) {
        float acc = b[k];
        for (int i = 0; i < 4; ++i)
            acc = fmaf(w[4 * k + i], z[i], acc);
        logits[k] = acc;
    }
}

/* MLP weights: W1[16][4], b1[16], W2[2][16], b2[2] (114 floats). */
void co_mlp_logits(const float *w, const float z[4], float logits[2])
{
    const float *w1 = w;
    const float *b1 = w + 64;
    const float *w2 = w + 80;
    const float *b2 = w + 112;
    float h[CO_MLP_HIDDEN];
    for (int j = 0; j < CO_MLP_HIDDEN; ++j) {
        float acc = b1[j];
        for (int i = 0; i < 4; ++i)
            acc = fmaf(w1[4 * j + i], z[i], acc);
        h[j] = tanhf(acc);
    }
    for (int k = 0; k < 2; ++k) {
        float acc = b2[k];
        for (int j = 0; j < CO_MLP_HIDDEN; ++j)
            acc = fmaf(w2[CO_MLP_HIDDEN * k + j], h[j], acc);
        logits[k] = acc;
    }
}

/* The same network with H hidden units (kinds 4 and 5: H = 32 and 64):
 * W1[H][4], b1[H], W2[2][H], b2[2] (7H + 2 floats), same chain order. */
#define CO_POLICY_MLP32 4
#define CO_POLICY_MLP64 5
#define CO_POLICY_LINEAR_PER_ENV 6 /* one linear policy per environment (rollouts only) */
void co_mlp_logits_wide(const float *w, int H, const float z[4], float logits[2])
{
    const float *w1 = w;
    const float *b1 = w + 4 * H;
    const float *w2 = w + 5 * H;
    const float *b2 = w + 7 * H;
    float acc0 = b2[0], acc1 = b2[1];
    for (int j = 0; j < H; ++j) {
        float acc = b1[j];
        for (int i = 0; i < 4; ++i)
            acc = fmaf(w1[4 * j + i], z[i], acc);
        float h = tanhf(acc);
        acc0 = fmaf(w2[j], h, acc0);
        acc1 = fmaf(w2[H + j], h, acc1);
    }
    logits[0] = acc0;
    logits[1] = acc1;
}

/* A deeper network (kind 7): 4 -> 16 (tanh) -> 16 (tanh) -> 2, the paper's
 * future work "fusing simulation with neural network inference" (Sec. VI)
 * one layer further. W1[16][4], b1[16], W2[16][16], b2[16], W3[2][16],
 * b3[2] (386 floats); every unit is the left-to-right fmaf chain that
 * starts from its bias. */
#define CO_POLICY_MLP_DEEP 7
void co_mlp_deep_logits(const float *w, const float z[4], float logits[2])
{
    const float *w1 = w;
    const float *b1 = w + 64;
    const float *w2 = w + 80;
    const float *b2 = w + 336;
    const float *w3 = w + 352;
    const float *b3 = w + 384;
    float h1[16], h2[16];
    for (int j = 0; j < 16; ++j) {
        float acc = b1[j];
        for (int i = 0; i < 4; ++i)
            acc = fmaf(w1[4 * j + i], z[i], acc);
        h1[j] = tanhf(acc);
    }
    for (int k = 0; k < 16; ++k) {
        float acc = b2[k];
        for (int j = 0; j < 16; ++j)
            acc = fmaf(w2[16 * k + j], h1[j], acc);
        h2[k] = tanhf(acc);
    }
    for (int m = 0; m < 2; ++m) {
        float acc = b3[m];
        for (int k = 0; k < 16; ++k)
            acc = fmaf(w3[16 * m + k], h2[k], acc);
        logits[m] = acc;
    }
}

/* Action for one environment; *gap (optional) receives |logit1 - logit0|
 * (infinity for the random policy) so tests can excuse argmax near-ties. */
static int co_policy_action(int kind, const float *w, uint32_t ka0, uint32_t ka1, uint32_t t,
                            const float z[4], float *gap)
{
    float logits[2];
    if (kind == CO_POLICY_RANDOM) {
        if (gap) *gap = INFINITY;
        return (int)(co_step_hash(ka0, ka1, t) >> 31);
    }
    if (kind == CO_POLICY_LINEAR)
        co_linear_logits(w, z, logits);
    else if (kind == CO_POLICY_MLP)
        co_mlp_logits(w, z, logits);
    else if (kind == CO_POLICY_MLP_DEEP)
        co_mlp_deep_logits(w, z, logits);
    else
        co_mlp_logits_wide(w, kind == CO_POLICY_MLP32 ? 32 : 64, z, logits);
    if (gap) *gap = fabsf(logits[1] - logits[0]);
    return logits[1] > logits[0];
}

/* ------------------------------------------------------------------ */
/* Batched single step (the cp_step contract).                         */
/*                                                                     */
/* planes_in / planes_out: four planes x|x_dot|theta|theta_dot, plane  */
/* p of env i at [p*stride + i]. action: n bytes or NULL (hash at      */
/* global step t). Environment i has global id env_offset + i.         */
/* reward is 1.0f for every step (each step starts from a live state,  */
/* the terminating step included). A finished environment's output     */
/* state is the start state of the episode beginning at time t+1.      */
/* Optional outputs (may be NULL): action_out[n], pre_reset[4][n]      */
/* (the post-Euler state before any reset, plane stride n).            */
/* ------------------------------------------------------------------ */
void co_step(uint32_t env_offset, int64_t n, int64_t stride_in, int64_t stride_out, uint32_t seed,
             uint32_t t, const float *planes_in, const uint8_t *action, float *planes_out,
             float *reward, uint8_t *done, uint8_t *action_out, float *pre_reset)
{
    for (int64_t i = 0; i < n; ++i) {
        uint32_t env = env_offset + (uint32_t)i;
        float z[4], zn[4];
        for (int p = 0; p < 4; ++p)
            z[p] = planes_in[p * stride_in + i];
        int a = action ? (action[i] != 0) : (int)co_action(seed, env, t);
        int d = co_dynamics_f32(z, a, zn);
        if (action_out) action_out[i] = (uint8_t)a;
        if (pre_reset)
            for (int p = 0; p < 4; ++p)
                pre_reset[p * n + i] = zn[p];
        if (d) co_reset_state(seed, env, t + 1u, zn);
        for (int p = 0; p < 4; ++p)
            planes_out[p * stride_out + i] = zn[p];
        if (reward) reward[i] = 1.0f;
        if (done) done[i] = (uint8_t)d;
    }
}

/* ------------------------------------------------------------------ */
/* Rollout (the cp_rollout contract): env loop outside, time inside.   */
/* ------------------------------------------------------------------ */
typedef struct {
    uint32_t env_offset;
    int64_t n, T;
    uint32_t seed, t0;
    int kind;
    const float *w;
    const float *init_state; /* [4][n] or NULL -> R(seed, env, t0) */
    uint32_t *ep_len_io;     /* [n] or NULL: steps already taken in the running episode (in/out) */
    float *ep_return_sum;    /* [n] or NULL */
    uint32_t *ep_count;      /* [n] or NULL */
    float *reward_stream;    /* [T][n] or NULL */
    uint32_t *done_bits;     /* [T][ceil(n/32)] or NULL (caller zeroes) */
    uint32_t *action_bits;   /* [T][ceil(n/32)] or NULL (caller zeroes) */
    float *final_state;      /* [4][n] or NULL */
    float *trajectory;       /* [T][4][n] or NULL: state after step t (after any reset) */
    float *min_gap;          /* [n] or NULL: smallest |logit1-logit0| seen */
    float *min_margin;       /* [n] or NULL: smallest distance of an updated |x| or |theta| from its
                                termination threshold seen (a diagnostic for the comparison rules:
                                "bit-exact wherever no state is within 1e-5 of a threshold") */
    uint32_t max_steps;      /* episode step limit (CartPole-v1 uses 500); 0 = none */
    const uint32_t *action_bits_in; /* [T][ceil(n/32)] supplied actions (bit i%32 of word i/32) or NULL */
    const float *start_states_in;   /* [T][4][n] supplied start states or NULL: an env that finishes at
                                       the k-th step of this call continues from row k (the paper's
                                       baseline feeds all its random values as data, Sec. V-A) */
    int64_t lo, hi;          /* env sub-range handled by this worker */
    uint64_t tot_ret, tot_cnt;
} co_rollout_job;

static void co_rollout_range(co_rollout_job *J)
{
    const int64_t n = J->n, T = J->T;
    const int64_t words = (n + 31) / 32;
    uint64_t tot_ret = 0, tot_cnt = 0;
    for (int64_t i = J->lo; i < J->hi; ++i) {
        uint32_t env = J->env_offset + (uint32_t)i;
        uint32_t ka0, ka1;
        co_keys(J->seed, env, 0u, &ka0, &ka1);
        float z[4], zn[4];
        if (J->init_state)
            for (int p = 0; p < 4; ++p)
                z[p] = J->init_state[p * n + i];
        else
            co_reset_state(J->seed, env, J->t0, z);
        uint32_t ep_len = J->ep_len_io ? J->ep_len_io[i] : 0u;
        uint32_t ret_sum = 0, ep_cnt = 0;
        float min_gap = INFINITY;
        double min_margin = INFINITY;
        for (int64_t k = 0; k < T; ++k) {
            uint32_t t = J->t0 + (uint32_t)k;
            float gap;
            int a;
            if (J->action_bits_in) {
                a = (int)((J->action_bits_in[k * words + i / 32] >> (i % 32)) & 1u);
                gap = INFINITY;
            } else if (J->kind == CO_POLICY_LINEAR_PER_ENV) {
                /* every environment has its own linear policy: parameter q of env i at w[q*n + i]
                 * (q = 0..7 the 2x4 matrix row-major, 8..9 the biases) */
                float wi[10];
                for (int q = 0; q < 10; ++q)
                    wi[q] = J->w[q * n + i];
                a = co_policy_action(CO_POLICY_LINEAR, wi, ka0, ka1, t, z, &gap);
            } else {
                a = co_policy_action(J->kind, J->w, ka0, ka1, t, z, &gap);
            }
            if (gap < min_gap) min_gap = gap;
            int d = co_dynamics_f32(z, a, zn);
            if (J->min_margin) {
                double mx = fabs(fabs((double)zn[0]) - (double)CO_XT), mt = fabs(fabs((double)zn[2]) - (double)CO_TT);
                if (mx < min_margin) min_margin = mx;
                if (mt < min_margin) min_margin = mt;
            }
            ep_len += 1u; /* reward 1 per step, terminating step included */
            /* an episode that has lasted max_steps steps is cut off: it counts as finished
             * (done = 1, its return is its length) and the env restarts like after a fall */
            if (J->max_steps && ep_len >= J->max_steps) d = 1;
            if (d) {
                ret_sum += ep_len;
                ep_cnt += 1u;
                ep_len = 0u;
                if (J->start_states_in)
                    for (int p = 0; p < 4; ++p)
                        zn[p] = J->start_states_in[(k * 4 + p) * n + i];
                else
                    co_reset_state(J->seed, env, t + 1u, zn);
            }
            memcpy(z, zn, sizeof z);
            if (J->reward_stream) J->reward_stream[k * n + i] = 1.0f;
            if (J->done_bits && d) J->done_bits[k * words + i / 32] |= 1u << (i % 32);
            if (J->action_bits && a) J->action_bits[k * words + i / 32] |= 1u << (i % 32);
            if (J->trajectory)
                for (int p = 0; p < 4; ++p)
                    J->trajectory[(k * 4 + p) * n + i] = z[p];
        }
        if (J->ep_len_io) J->ep_len_io[i] = ep_len;
        if (J->ep_return_sum) J->ep_return_sum[i] = (float)ret_sum;
        if (J->ep_count) J->ep_count[i] = ep_cnt;
        if (J->final_state)
            for (int p = 0; p < 4; ++p)
                J->final_state[p * n + i] = z[p];
        if (J->min_gap) J->min_gap[i] = min_gap;
        if (J->min_margin) J->min_margin[i] = (float)min_margin;
        tot_ret += ret_sum;
        tot_cnt += ep_cnt;
    }
    J->tot_ret = tot_ret;
    J->tot_cnt = tot_cnt;
}

static void *co_rollout_thread(void *arg)
{
    co_rollout_range((co_rollout_job *)arg);
    return NULL;
}

/* totals[0] += sum over envs of ep_return_sum (as integer), totals[1] +=
 * sum of ep_count. nthreads > 1 splits the env range statically; worker
 * ranges are multiples of 32 envs so bit-stream words are never shared. */
void co_rollout_ex(uint32_t env_offset, int64_t n, int64_t T, uint32_t seed, uint32_t t0, int kind,
                   const float *weights, const float *init_state, uint32_t *ep_len_io,
                   float *ep_return_sum, uint32_t *ep_count, uint64_t *totals, float *reward_stream,
                   uint32_t *done_bits, uint32_t *action_bits, float *final_state, float *trajectory,
                   float *min_gap, int nthreads, uint32_t max_steps, const uint32_t *action_bits_in,
                   const float *start_states_in, float *min_margin)
{
    if (nthreads < 1) nthreads = 1;
    if (nthreads > 256) nthreads = 256;
    co_rollout_job jobs[256];
    pthread_t tid[256];
    int64_t chunks = (n + 31) / 32;
    int64_t per = (chunks + nthreads - 1) / nthreads;
    int used = 0;
    for (int w = 0; w < nthreads; ++w) {
        int64_t lo = (int64_t)w * per * 32, hi = lo + per * 32;
        if (lo >= n) break;
        if (hi > n) hi = n;
        co_rollout_job J = {env_offset, n, T, seed, t0, kind, weights, init_state, ep_len_io,
                            ep_return_sum, ep_count, reward_stream, done_bits, action_bits,
                            final_state, trajectory, min_gap, min_margin, max_steps, action_bits_in,
                            start_states_in, lo, hi, 0, 0};
        jobs[used++] = J;
    }
    if (used == 1) {
        co_rollout_range(&jobs[0]);
    } else {
        for (int w = 0; w < used; ++w)
            pthread_create(&tid[w], NULL, co_rollout_thread, &jobs[w]);
        for (int w = 0; w < used; ++w)
            pthread_join(tid[w], NULL);
    }
    if (totals)
        for (int w = 0; w < used; ++w) {
            totals[0] += jobs[w].tot_ret;
            totals[1] += jobs[w].tot_cnt;
        }
}

/* The basic contract: no episode step limit, actions from the policy. */
void co_rollout(uint32_t env_offset, int64_t n, int64_t T, uint32_t seed, uint32_t t0, int kind,
                const float *weights, const float *init_state, uint32_t *ep_len_io,
                float *ep_return_sum, uint32_t *ep_count, uint64_t *totals, float *reward_stream,
                uint32_t *done_bits, uint32_t *action_bits, float *final_state, float *trajectory,
                float *min_gap, int nthreads)
{
    co_rollout_ex(env_offset, n, T, seed, t0, kind, weights, init_state, ep_len_io, ep_return_sum, ep_count,
                  totals, reward_stream, done_bits, action_bits, final_state, trajectory, min_gap, nthreads,
                  0u, NULL, NULL, NULL);
}

/* co_step with an episode step limit: ep_len [n] holds the steps already taken in each
 * running episode, in and out (0 after a restart). max_steps = 0 means no limit. */
void co_step_limited(uint32_t env_offset, int64_t n, int64_t stride_in, int64_t stride_out, uint32_t seed,
                     uint32_t t, const float *planes_in, const uint8_t *action, float *planes_out,
                     float *reward, uint8_t *done, uint32_t *ep_len, uint32_t max_steps)
{
    for (int64_t i = 0; i < n; ++i) {
        uint32_t env = env_offset + (uint32_t)i;
        float z[4], zn[4];
        for (int p = 0; p < 4; ++p)
            z[p] = planes_in[p * stride_in + i];
        int a = action ? (action[i] != 0) : (int)co_action(seed, env, t);
        int d = co_dynamics_f32(z, a, zn);
        uint32_t len = ep_len[i] + 1u;
        if (max_steps && len >= max_steps) d = 1;
        if (d) {
            co_reset_state(seed, env, t + 1u, zn);
            len = 0u;
        }
        ep_len[i] = len;
        for (int p = 0; p < 4; ++p)
            planes_out[p * stride_out + i] = zn[p];
        if (reward) reward[i] = 1.0f;
        if (done) done[i] = (uint8_t)d;
    }
}
