/*
 * cartpole.h — C ABI of libcartpole.so: the batched CartPole environment step on
 * one NVIDIA B200 (sm_100a), in three execution strategies.
 *
 * The computation is the "environment update function" of the paper "Operator
 * Fusion in XLA: Analysis and Evaluation" (Sec. IV, Case Study on Cart-pole):
 * a chain of elementwise float32 operations over N independent environments —
 * force from the action, sin/cos of the pole angle, the shared `temp` term,
 * angular and linear acceleration, four explicit-Euler updates, termination
 * test, reward, and reset of finished environments — repeated for T steps with
 * random actions and random start states (Sec. V, 2,048 envs x 10,000 steps).
 * The three strategies are the rungs of the paper's fusion ladder:
 *   cp_step_unfused  one kernel per elementwise op, every intermediate in HBM
 *                    (the eager per-op execution of Sec. V-F);
 *   cp_step          one fused kernel per step, state passed as four separate
 *                    planes and kept in registers (Sec. V-C, "no concat");
 *   cp_rollout       one kernel for all T steps, state in registers across
 *                    steps (Sec. V-D loop unrolling taken to its limit, and the
 *                    single-kernel CUDA comparison of Sec. V-G).
 * Random numbers never need a kernel of their own (Sec. V-A): actions and start
 * states are a stateless counter hash of (seed, env, step), defined below.
 *
 * Conventions
 *   - Every pointer is marked DEVICE or HOST. Device buffers belong to the caller
 *     unless stated; the library never frees or reallocates them.
 *   - Calls enqueue work on the stream set with cp_set_stream (default: the legacy
 *     default stream) and return without synchronising, unless stated.
 *   - int functions return CP_OK or a negative code; cp_last_error() gives the text
 *     for the calling thread. Nothing aborts, traps or throws.
 *   - State layout: four float32 planes x | x_dot | theta | theta_dot; element i of
 *     plane p is planes[p * plane_stride + i]. Vector (16-byte) access is used when
 *     planes is 16-byte aligned and plane_stride is a multiple of 4; any other
 *     layout takes a scalar path with identical results.
 *   - Environment i of a batch has global id env_offset + i; all hashing uses the
 *     global id, so results do not depend on how environments are sharded.
 *
 * Arithmetic (identical in all three strategies, bit for bit)
 *   constants  g=9.8f m_pole=0.1f m_total=1.1f l=0.5f pml=0.05f F=10.0f tau=0.02f
 *              ft=(float)(4/3) x_max=2.4f theta_max=(float)(12*2*pi/360)
 *   force = a ? +F : -F;  s = sinf(theta); c = cosf(theta)
 *   temp  = (force + (pml*(thd*thd))*s) / m_total
 *   thacc = (g*s - c*temp) / (l*(ft - (m_pole*(c*c))/m_total))
 *   xacc  = temp - ((pml*thacc)*c)/m_total
 *   x' = x + tau*xd; xd' = xd + tau*xacc; th' = th + tau*thd; thd' = thd + tau*thacc
 *   every operation rounded once to float32 (no fused multiply-add, IEEE division; no
 *   fast-math). sinf/cosf: for |theta| <= 0.22 (every angle an episode can hold; the
 *   termination threshold is 0.2095) a polynomial with measured error <= 0.53 ulp, for any
 *   other argument the CUDA library's accurate sinf/cosf;
 *   done = x'<-x_max | x'>x_max | th'<-theta_max | th'>theta_max  (strict, on the
 *   updated state); reward = 1.0f for every step (each step starts from a live
 *   state; the terminating step counts); a finished environment continues from a
 *   fresh start state and reports done=1 for that step.
 *
 * Counter hash (uint32 arithmetic mod 2^32)
 *   MA=0x6A09E667 MB=0xBB67AE85 MG=0x9E3779B1
 *   mix32(h): h^=h>>16; h*=MA; h^=h>>15; h*=MB; h^=h>>16
 *   salt(seed,stream) = mix32(mix32(seed^MG)+stream)         stream 0 actions, 1 starts
 *   K0 = mix32(env ^ salt); K1 = mix32(K0+MG)
 *   H(K,c): h=K0^c; h=(h^(h>>16))*MA+K1; h=(h^(h>>15))*MB; h^=h>>16
 *   action(seed,env,t)   = H(K(stream 0), t) >> 31
 *   start_j(seed,env,t)  = ((float)(H(K(stream 1), 4t+j)>>8) * 2^-24 - 0.5f) * 0.1f,
 *                          j=0..3 -> x, x_dot, theta, theta_dot of an episode that
 *                          begins at global time t (initial state: t of the reset;
 *                          after done at step t: t+1). Steps exist for t < 2^30, so every
 *                          start state an episode RUNS from has 4t+j < 2^32. The one start
 *                          state of time 2^30 (handed over, never stepped from, when an episode
 *                          ends on the very last permitted step) takes its counters mod 2^32,
 *                          i.e. 0..3 — defined, shared with the reference implementation the
 *                          tests use, and pinned by the end-of-time tests.
 */
#ifndef CARTPOLE_H_
#define CARTPOLE_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define CP_OK 0
#define CP_EINVAL (-1) /* bad argument: null/misaligned pointer, size out of range, unknown kind */
#define CP_ECUDA (-2)  /* a CUDA runtime call failed; text in cp_last_error() */
#define CP_ENOMEM (-3) /* allocation failed, or a caller-supplied workspace is too small */

#define CP_POLICY_RANDOM 0 /* hashed Bernoulli(1/2) action */
#define CP_POLICY_LINEAR 1 /* argmax(W obs + b), W 2x4 */
#define CP_POLICY_MLP 2    /* argmax(W2 tanh(W1 obs + b1) + b2), 4 -> 16 -> 2 */
#define CP_MLP_HIDDEN 16
#define CP_POLICY_MLP32 4  /* the same network with 32 hidden units (226 floats) */
#define CP_POLICY_MLP64 5  /* ... with 64 hidden units (450 floats); kind 3 is not a policy */
#define CP_POLICY_LINEAR_PER_ENV 6 /* a different linear policy for every environment (population
                                      search): `weights` is then a DEVICE pointer to [10][n_envs]
                                      floats, parameter q of env i at weights[q * n_envs + i], rows
                                      0-7 the 2x4 matrix row-major, rows 8-9 the biases; loaded into
                                      registers once per launch */
#define CP_POLICY_MLP_DEEP 7 /* two hidden layers, 4 -> 16 (tanh) -> 16 (tanh) -> 2 (386 floats) */
#define CP_MAX_T (1LL << 30)

/* Opaque HOST handle of a batch: n_envs, plane_stride, seed, global step t,
 * env_offset and the DEVICE address of the four state planes. */
typedef struct cp_state cp_state;

/* Policy evaluated inside the rollout kernel on the state BEFORE the step ("fusing
 * simulation with neural network inference", the paper's future work, Sec. VI).
 * weights is a HOST pointer, copied into the launch parameters by the call:
 *   linear: W[2][4] row-major, b[2]                         (10 floats)
 *   MLP:    W1[H][4], b1[H], W2[2][H], b2[2], H = 16 / 32 / 64   (7H + 2 = 114 / 226 / 450 floats)
 *   deep:   W1[16][4], b1[16], W2[16][16], b2[16], W3[2][16], b3[2]   (386 floats)
 * Each logit is a left-to-right chain acc = fmaf(w_i, v_i, acc) starting from the
 * bias; hidden units use an accurate tanh (largest error 1.82 units in the last place, the
 * same as the CUDA library's tanhf; see cp_selftest_tanh); action = (logit[1] > logit[0]),
 * so a tie pushes left. */
typedef struct cp_policy {
    int32_t kind;
    const float *weights; /* HOST (DEVICE for CP_POLICY_LINEAR_PER_ENV); NULL for CP_POLICY_RANDOM */
} cp_policy;

/* Outputs of a rollout; every pointer is DEVICE memory of the caller and may be
 * NULL (not produced). Per-step planes are time-major so that a warp writes one
 * contiguous 128-byte line per step. */
typedef struct cp_returns {
    float *ep_return_sum;  /* [n_envs] sum of the returns (= lengths) of episodes completed in the T steps;
                              a whole number, exact in float32 up to 2^24 = 16,777,216 (any T below that;
                              beyond it the value is rounded to float32 while `totals` stays exact) */
    uint32_t *ep_count;    /* [n_envs] number of completed episodes */
    uint64_t *totals;      /* [2] += {sum of ep_return_sum, sum of ep_count}; caller zeroes before the call */
    float *reward_stream;  /* [T][n_envs] reward of every step (1.0f) */
    uint32_t *done_bits;   /* [T][ceil(n_envs/32)] bit (i%32) of word (i/32) = done of env i at that step; every
                              word is written, the caller need not clear it (long launches of batches that fill
                              the GPU zero the plane with a small launch before the rollout kernel sets its bits) */
    uint32_t *action_bits; /* [T][ceil(n_envs/32)] same packing, the action taken */
    float *final_state;    /* [4][n_envs] state after the last step */
    float *trajectory;     /* [T][4][n_envs] state after every step, after any reset (validation aid) */
} cp_returns;

/* ---- the three calls of the hot path ------------------------------------------------ */

/* Sec. V (random start states): allocate a batch of n_envs environments (cudaMalloc,
 * planes padded to a multiple of 4 floats) and fill it with start states of global time 0.
 * 1 <= n_envs, n_envs + env_offset(=0) <= 2^32. Returns NULL on error. Free with cp_free. */
cp_state *cp_reset(int64_t n_envs, uint32_t seed);

/* Sec. IV / Sec. V-C: one fused step of every environment, one kernel launch.
 *   state      in: batch at global step t.
 *   action     DEVICE [n_envs] bytes (non-zero = push right), or NULL = hashed action of step t.
 *   out_state  out: same n_envs; may be `state` itself (in place). Receives t+1 (host side),
 *              and seed / env_offset of `state`.
 *   reward     DEVICE [n_envs] float32 or NULL.   done  DEVICE [n_envs] bytes (0/1) or NULL.
 * Algorithmic HBM traffic: 16 B read + 16 B written per env, + 4 (reward) + 1 (done) [+ 1 action]. */
int cp_step(cp_state *state, const uint8_t *action, cp_state *out_state, float *reward, uint8_t *done);

/* Sec. V-D / V-G: T steps of n_envs environments in ONE kernel, state in registers for
 * all T steps; starts from the start states of global time 0 (equal to cp_reset followed by
 * T cp_step calls with action == NULL, bit for bit). 1 <= T <= CP_MAX_T.
 * policy NULL or kind CP_POLICY_RANDOM = hashed actions. */
int cp_rollout(int64_t n_envs, int64_t T, uint32_t seed, const cp_policy *policy, const cp_returns *returns);

/* ---- helpers ------------------------------------------------------------------------- */

/* Sec. V (the host loop over steps): k consecutive cp_step launches in place with hashed
 * actions, issued from one call so that the host cost per step is one kernel launch. reward and
 * done (each may be NULL) are overwritten by every step and end up holding the last step's. */
int cp_step_repeat(cp_state *state, int64_t k, float *reward, uint8_t *done);

/* Sec. V-F (eager per-op execution): the same step as cp_step computed by one kernel per
 * elementwise operation (45 launches, 46 when the action is hashed), every intermediate a
 * plane in `workspace` (DEVICE, 256-byte aligned, >= cp_unfused_workspace_bytes(n_envs)).
 * Results equal cp_step bit for bit. Needs 16-byte aligned planes with plane_stride % 4 == 0.
 * Unlike cp_step, out_state must not alias state. reward / done as in cp_step (non-NULL). */
int cp_step_unfused(cp_state *state, const uint8_t *action, cp_state *out_state, float *reward,
                    uint8_t *done, void *workspace, size_t workspace_bytes);
size_t cp_unfused_workspace_bytes(int64_t n_envs);

/* The paper has no counterpart to this call; it exists for callers that cannot allocate device
 * memory themselves or let a library do it on their behalf: a control loop that must not hit
 * the device-wide synchronisation an allocation can cause, a plugin living inside another
 * application's fixed memory budget, a process whose free device memory already belongs to
 * some other allocator. It is cp_step_unfused with the workspace taken from an array built
 * into the library instead of from the caller: same arguments otherwise, same results bit for
 * bit, and it calls no cudaMalloc / cudaFree or any other allocating routine.
 *   - At most CP_NOALLOC_MAX_ENVS environments; a larger batch is refused with CP_EINVAL
 *     (cp_last_error says so). The array (about 8.7 MiB) is resident on every GPU that loads
 *     this library until the process exits.
 *   - The first call on each device looks up the array's device address (with that device
 *     current) and keeps it. Where the CUDA runtime loads device code lazily, that first call
 *     is also what brings the module holding the array onto the device, so only from then on
 *     is the array resident and do calls leave the device's free memory untouched: make the
 *     first call a warm-up, outside latency-critical code and before any stream capture.
 *   - All calls share the one array, which still holds the previous call's intermediates.
 *     Nothing in it needs to start at zero (each plane is fully rewritten before it is read),
 *     but two calls whose kernels overlap on the GPU (different streams, or different threads
 *     without ordering between them) race on it: order such calls yourself. */
#define CP_NOALLOC_MAX_ENVS 65536
int cp_step_unfused_noalloc(cp_state *state, const uint8_t *action, cp_state *out_state, float *reward,
                            uint8_t *done);

/* Wrap caller-owned DEVICE planes (for example a torch tensor) as a batch at global step t.
 * plane_stride >= n_envs. The handle does not own the planes. NULL on error. */
cp_state *cp_wrap(float *planes, int64_t n_envs, int64_t plane_stride, uint32_t seed, uint32_t t,
                  uint32_t env_offset);
/* Overwrite the planes with the start states of the batch's current global step t. */
int cp_fill_start(cp_state *state);
/* Set the batch's global step (host side only). */
int cp_set_time(cp_state *state, uint32_t t);
/* Release the handle (and the planes if cp_reset allocated them). NULL is allowed. */
void cp_free(cp_state *state);
/* Read the handle's fields; any out pointer may be NULL. planes is a DEVICE address. */
int cp_state_info(const cp_state *state, int64_t *n_envs, int64_t *plane_stride, uint32_t *seed,
                  uint32_t *t, uint32_t *env_offset, float **planes);

/* Sec. V-A (the random actions, drawn without a random-number kernel of their own): hashed actions
 * of global step t for envs env_offset .. env_offset+n_envs-1 -> out DEVICE [n_envs]. */
int cp_actions(int64_t n_envs, uint32_t seed, uint32_t t, uint32_t env_offset, uint8_t *out);

/* Sec. V (N independent environments): cp_rollout for the env range [env_offset, env_offset +
 * n_envs) of a larger job (one range per GPU; no exchange is needed besides adding the ranks'
 * `totals`). The paper runs one GPU; the sharding itself has no counterpart there. */
int cp_rollout_shard(uint32_t env_offset, int64_t n_envs, int64_t T, uint32_t seed,
                     const cp_policy *policy, const cp_returns *returns);

/* Sec. V-D (k steps per kernel, the knob between cp_step and cp_rollout): advance an existing
 * batch by T steps in one launch, in place, from its current global step. ep_len DEVICE [n_envs]
 * (or NULL = all episodes start now) carries the steps already taken in each running episode in
 * and out, so that consecutive chunks give the same returns as one long rollout.
 * returns->final_state is ignored (the batch itself is updated); state->t advances by T. */
int cp_rollout_from(cp_state *state, int64_t T, uint32_t *ep_len, const cp_policy *policy,
                    const cp_returns *returns);

/* The general rollout call: everything cp_rollout / cp_rollout_shard / cp_rollout_from do, plus
 *   - an episode step limit (CartPole-v1 cuts an episode off after 500 steps): an episode that has
 *     lasted max_episode_steps steps ends on that step exactly like a fall — done = 1, reward 1, its
 *     length added to ep_return_sum, counted in ep_count — and the environment restarts;
 *   - actions given as data instead of drawn by a policy (the paper's baseline, Sec. V-A, feeds
 *     precomputed random values): action_bits_in DEVICE [T][ceil(n_envs/32)], bit (i%32) of word
 *     (i/32) of row k = action of env i at the k-th step of this call; overrides `policy`;
 *   - start states given as data too (the other half of that baseline's randomness; also the way
 *     to evaluate a policy from chosen start states): start_states_in DEVICE [T][4][n_envs], an
 *     environment that finishes at the k-th step of this call continues from row k (planes x,
 *     x_dot, theta, theta_dot) instead of the hashed start state. The first states still come
 *     from `state`, or from the hash of time t0;
 *   - a choice of arithmetic. CP_ARITH_EXACT (0, what every other entry point uses): each operation
 *     of the step rounded once, in the order of the per-op ladder, so that ladder, fused step and
 *     rollout give the same bits. CP_ARITH_CONTRACTED: the step as a contracting compiler would
 *     emit it for a fused kernel (Sec. V-B, V-G: generated fused code carries no such promise) —
 *     fused multiply-adds, divisions by the total mass folded into constants, theta_acc by
 *     reciprocal; 25 instead of 43 floating-point operations per step; the MLP policies' tanh
 *     from the hardware exp2 and reciprocal (absolute error <= 2.4e-7). One step from the same
 *     state differs by at most 2e-6 relative (on the scale of value and update) and a done flag
 *     only where x' or theta' lies within 1e-5 of its threshold. Start states, actions of the
 *     hashed policy and the bookkeeping are the same bits in both. Free-running returns stay
 *     identical on more than 99.9 % of environments when the actions do not depend on the state
 *     (hashed or supplied actions: every restart re-synchronises the two arithmetics); under a
 *     state-feedback policy the per-step differences are amplified through the action choice and
 *     only the statistics (mean return, episode count) agree: measured on 40,000 environments,
 *     identical returns on 96.3 % after 300 steps with a linear policy whose episodes last about
 *     80 steps, on 100 % with a 4-16-2 network whose episodes last 9. What does hold under any
 *     policy is the per-step contract: from the same state, the same action wherever the two
 *     logits are 1e-5 apart, and then the tolerances above. Use CP_ARITH_EXACT where
 *     reproducibility against the per-op order matters.
 * struct_size must be sizeof(cp_rollout_args) (guards against a caller built for another layout).
 * state == NULL: start states of global time t0, env range [env_offset, env_offset + n_envs);
 * state != NULL: that batch is advanced in place from its own time (n_envs, seed, env_offset, t0 of
 * the struct are ignored, returns->final_state too) and state->t grows by T.
 * ep_len: DEVICE [n_envs] steps already taken in each running episode, read and rewritten, or NULL
 * (all episodes start at this call; nothing written). t0 + T <= CP_MAX_T. */
#define CP_ARITH_EXACT 0u
#define CP_ARITH_CONTRACTED 1u
typedef struct cp_rollout_args {
    uint32_t struct_size;
    uint32_t env_offset;
    int64_t n_envs, T;
    uint32_t seed, t0;
    const cp_policy *policy;       /* HOST, or NULL = hashed random actions */
    const cp_returns *returns;     /* HOST struct of DEVICE pointers, not NULL */
    cp_state *state;               /* or NULL */
    uint32_t *ep_len;              /* DEVICE or NULL */
    uint32_t max_episode_steps;    /* 0 = no limit */
    uint32_t arithmetic;           /* CP_ARITH_EXACT or CP_ARITH_CONTRACTED */
    const uint32_t *action_bits_in; /* DEVICE or NULL */
    const float *start_states_in;   /* DEVICE or NULL */
} cp_rollout_args;
int cp_rollout_ex(const cp_rollout_args *args);

/* Sec. V-C's step with CartPole-v1's episode limit (the paper names no limit; an option of this
 * build): cp_step with per-environment episode-length counters and the same optional step limit:
 * ep_len DEVICE [n_envs] (16-byte aligned for the vector kernel) is incremented, compared with
 * max_episode_steps (0 = no limit; an env reaching it reports done = 1 and restarts) and reset to
 * 0 for finished environments. ep_len == NULL makes this cp_step (and then the limit must be 0). */
int cp_step_ex(cp_state *state, const uint8_t *action, cp_state *out_state, float *reward, uint8_t *done,
               uint32_t *ep_len, uint32_t max_episode_steps);

/* Plumbing, no counterpart in the paper (it times device-resident runs): end-to-end forms with
 * HOST buffers (pinned memory recommended): device staging buffers
 * are owned by the library (grown on demand, released by cp_shutdown); the calls copy in,
 * launch, copy out and SYNCHRONISE the stream before returning.
 * cp_rollout_host: h_ep_return_sum [n_envs], h_ep_count [n_envs], h_totals [2] (overwritten).
 * When the two per-env buffers are page-locked (cudaHostAlloc / cudaHostRegister, e.g. torch
 * pinned tensors) the kernel stores into them directly over PCIe while it runs, so the transfer
 * overlaps the computation; pageable buffers are filled by copies after the kernel. */
int cp_rollout_host(int64_t n_envs, int64_t T, uint32_t seed, const cp_policy *policy,
                    float *h_ep_return_sum, uint32_t *h_ep_count, uint64_t *h_totals);
/* The same for the env range [env_offset, env_offset + n_envs) of a larger job (one range per GPU). */
int cp_rollout_host_shard(uint32_t env_offset, int64_t n_envs, int64_t T, uint32_t seed, const cp_policy *policy,
                          float *h_ep_return_sum, uint32_t *h_ep_count, uint64_t *h_totals);
/* cp_step_host: h_planes_in/out [4][n_envs] (stride n_envs), h_action [n_envs] or NULL,
 * h_reward [n_envs], h_done [n_envs]; the step at global time t of envs 0..n_envs-1. */
int cp_step_host(int64_t n_envs, uint32_t seed, uint32_t t, const float *h_planes_in,
                 const uint8_t *h_action, float *h_planes_out, float *h_reward, uint8_t *h_done);
/* Free the library-owned staging buffers (synchronises the device). */
void cp_shutdown(void);

/* Stream used by this thread's later calls (a cudaStream_t; NULL = legacy default stream). */
void cp_set_stream(void *cuda_stream);

/* Device allocator used by cp_reset for the batches it owns, process-wide (plumbing; the paper
 * has no counterpart): alloc(bytes) returns a
 * DEVICE pointer aligned to at least 16 bytes or NULL, release(ptr) takes it back (a handle keeps
 * the release function it was created under, so the allocator may change while handles live).
 * Both NULL (the default) = cudaMalloc / cudaFree. A host program that runs its own caching
 * allocator (torch's, for instance) passes that, so that cp_reset neither synchronises the device
 * nor takes memory the host program cannot see. Everything else the library touches is
 * caller-provided, except the staging buffer of the HOST-buffer calls (always cudaMalloc). */
int cp_set_allocator(void *(*alloc)(size_t), void (*release)(void *));

/* Launch tuning, process-wide (no counterpart in the paper; its analogue is XLA's flag for
 * switching passes off, Sec. III). key: "rollout_block" (threads per CTA, 32..256, multiple of 32;
 * 0 = default: 128 for very small batches, else 256), "rollout_ept" (environments per thread: 1 or 2; 0 = default, 2 for large
 * batches except with the MLP policies), "rollout_coop" (how finished environments get their
 * start state: 1 = by the whole warp through shared memory, 2 = each lane its own when its env
 * finishes, 3 = each lane computes it every step ahead of the dynamics (hashed or supplied
 * actions only, otherwise as 2), 4 = a helper warp per stepping warp hashes every step's action
 * and start state ahead into shared memory (hashed or supplied actions and hashed start
 * states; otherwise as 2), 2, 3 and 4 only with one environment per
 * thread; 0 = default: helper warps for up to ten warps of environments per SM, per lane for
 * other batches too small to fill the GPU (ahead for the smaller ones), deferred (5) from one
 * 64-environment warp per scheduler on (37,888 environments on 148 SMs) where that form applies,
 * by the warp otherwise;
 * 5 = two environments per thread with a clock per environment and restarts deferred to every
 * few loop trips (per-step outputs none or reward plane + done bits; hashed actions, a linear
 * policy or the 4-16-2 network; the wider and deeper networks without step limit and per-step
 * outputs; otherwise the default); every choice gives the same bits), "rollout_defer" (loop
 * trips between the restart passes of that deferred form: 2, 3, 4, 6 or 8; 0 = default: 2, 4 or
 * 6 by the number of steps (8 for the shared linear policy from 384 steps on), 3 with a network policy; the wider and deeper networks always use 3),
 * "rollout_ctas_per_sm" (0 = default: one 32*ept-environment task per warp and as many
 * CTAs as that takes; k > 0 = persistent grid of k CTAs per SM looping over tasks), "step_block"
 * (32..256, default 64), "step_vec_min_envs" (batches smaller than this use the one-env-per-thread
 * step kernel even when the four-envs-per-thread vector form is possible; default 262144),
 * "step_pdl" (1 = default: the step kernels and the ladder's one-op kernels are launched with
 * programmatic stream serialization, so that a launch is set up — and, in the fused step, the
 * actions hashed — while the launch before it still runs; 0 = plain launches).
 * Returns CP_EINVAL for an unknown key or value. */
int cp_tune(const char *key, int value);

/* Number of kernels this library has launched in this process (all threads). A measurement aid
 * (the paper counts launches with a profiler, Sec. V-G); no counterpart as a call. */
uint64_t cp_launch_count(void);

/* The cp_selftest_* calls below are diagnostics of this build's arithmetic shortcuts; the paper
 * has no counterpart to any of them.
 * Diagnostics: count float32 values v in [lo, hi] (bit patterns, both >= 0, lo <= hi, and their
 * negatives) for which the fused kernels' combined sine/cosine differs in any bit from the
 * ladder's separate sine and cosine kernels. mismatches DEVICE [1] uint64, caller zeroes. */
int cp_selftest_sincos(uint32_t lo_bits, uint32_t hi_bits, uint64_t *mismatches);

/* Diagnostics: error of the kernels' sine and cosine against float64 over the float32 values in
 * [lo, hi] (bit patterns as above). out DEVICE [4] uint64, caller zeroes: out[0] / out[1] = largest
 * error of sin / cos in millionths of a float32 ulp; out[2] / out[3] = number of results that are
 * not the correctly rounded value. */
int cp_selftest_sincos_accuracy(uint32_t lo_bits, uint32_t hi_bits, uint64_t *out);

/* Diagnostics: error against float64 of the hyperbolic tangents the MLP policies use, over the
 * float32 values in [lo, hi] (bit patterns as above) and their negatives, largest value seen.
 * out DEVICE [6] uint64, caller zeroes. Absolute error in units of 1e-12: out[0] the
 * five-instruction form of CP_ARITH_CONTRACTED, out[1] the CUDA library's tanhf (for comparison),
 * out[2] the tanh of CP_ARITH_EXACT (polynomial below 0.6, hardware exp2 / reciprocal above,
 * branch-free). In millionths of a unit in the last place: out[3] that tanh, out[4] the library's.
 * out[5] += values for which the packed two-environment form of that tanh differs in any bit
 * from the scalar form (must stay 0). */
int cp_selftest_tanh(uint32_t lo_bits, uint32_t hi_bits, uint64_t *out);

/* Diagnostics: the kernels replace x / 1.1f by a two-operation exact sequence and the start-state
 * mapping by an equivalent two-operation one. This checks, over all 2^32 float bit patterns (2^24
 * for the mapping), that the replacements give the bits of the operations they stand for wherever
 * they are used. out DEVICE [4] uint64, caller zeroes; every count must come back 0. */
int cp_selftest_arith(uint64_t *out);

/* Diagnostics: for states with |theta| <= 0.22 (every angle an episode visits; such a state only
 * survives its step if |theta_dot| < 21.5, and the accelerations of a state that does not survive
 * are never observed) the
 * kernels compute the angular acceleration's quotient with the hardware reciprocal plus one exact
 * correction instead of the general division. This compares the two over the whole operand domain
 * of such states: every den_step-th float32 denominator in [0.6210, 0.6242] (53,688 values at
 * den_step = 1) times every float32 numerator of magnitude in [2, 32), both signs (about two
 * seconds of GPU time at den_step = 1). out DEVICE [2] uint64, caller zeroes:
 * out[0] += mismatching quotients (must stay 0), out[1] += (denominator, |numerator|) pairs tested. */
int cp_selftest_tame_div(uint32_t den_step, uint64_t *out);

/* Diagnostics (no counterpart in the paper): where a thread owns two environments the rollout
 * kernels step both with sm_100a's packed float32 instructions (one instruction, two
 * independent roundings). This steps `count` pseudo-random pairs of states (|theta| <= 0.22, the
 * other components across and beyond the live range; drawn from `seed`) both ways and compares
 * all eight new components and both termination flags bit for bit. out DEVICE [3] uint64, caller
 * zeroes: out[0] += pairs that differ (must stay 0), out[1] += pairs tested, out[2] += pairs for
 * which the packed and scalar steps of CP_ARITH_CONTRACTED differ (must stay 0). */
int cp_selftest_pair(uint64_t count, uint32_t seed, uint64_t *out);

/* Calibration of the roofline denominators (a measurement aid; the paper has no counterpart):
 * enqueue one launch in which every thread executes
 * iters rounds of eight independent chains of one instruction kind — 0: float32 fused
 * multiply-add, 1: 32-bit integer multiply-add, 2: the special-function reciprocal, 3: the packed
 * float32 fused multiply-add of sm_100a (two results per instruction) — or of a half-and-half mix:
 * 4: packed + scalar float, 5: packed float + integer multiply-add, 6: packed float + integer
 * logic, 7: scalar float + integer multiply-add (which pipes share hardware) — on a grid of
 * 8 CTAs x 256 threads per SM. seed DEVICE [10] floats (ordinary magnitudes, e.g. 0.5 .. 1.5),
 * sink DEVICE [CP_CALIBRATE_THREADS_PER_SM x SM count] floats, overwritten. Returns the number of
 * thread-instructions the chains execute (a packed instruction counts once; kind 6 issues two
 * logic instructions per counted one; the caller times the launch), or a negative error code. */
#define CP_CALIBRATE_THREADS_PER_SM 2048
int64_t cp_calibrate_pipe(int kind, const float *seed, float *sink, int iters);

const char *cp_last_error(void);
const char *cp_version(void);

#ifdef __cplusplus
}
#endif
#endif /* CARTPOLE_H_ */
