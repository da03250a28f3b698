/*
 * sim.h -- C ABI of the batched environment-stepping library (CUDA, sm_100a).
 *
 * The problem, as the paper states it: N simulator instances advance in parallel on the
 * GPU ("GPU vectorization", Section 3) and K simulator steps run inside one kernel launch
 * with the simulator state cached on chip ("simulator kernel fusion", Section 4).  Each
 * step here is: pick an action (uniform random, a small MLP, or given by the caller),
 * advance the physics, compute reward and done, auto-reset finished envs, and append to a
 * trajectory buffer.  N envs never interact.
 *
 * Conventions for every call
 *   - Return value: 0 (SIM_OK) or a negative SIM_E* code.  Nothing throws or aborts.
 *     Argument errors are detected on the host before any work is enqueued.
 *   - Pointers named d_* / out_* are DEVICE pointers owned by the caller; they must stay
 *     valid until the work enqueued by the call has finished.  Pointers named h_* are
 *     HOST pointers.  The library never frees or keeps a caller pointer.
 *   - The handle and its internal buffers (state [N,S] fp32 row-major, ep_len [N] u32,
 *     reset_count [N] u32) are owned by the library: sim_create allocates, sim_destroy frees.
 *   - Except sim_create / sim_destroy / sim_rollout_host, calls only enqueue work on the
 *     handle's stream and return; the caller synchronises the stream.
 *   - Because those calls only enqueue kernels (no allocation, no synchronisation, no host-side read of device
 *     data), a caller may record them into a CUDA graph by stream capture and replay it, e.g. sim_reset followed by
 *     a sim_rollout with K_fused = 1, whose launches are then replayed without per-launch host cost.  The launch
 *     arguments carry the handle's step counter t as it was at capture time, so a replay repeats exactly the
 *     captured steps; the host-side t does not advance on replay (set it with sim_set_counters if needed).
 *   - A handle belongs to the CUDA device that was current in sim_create; a call made while
 *     another device is current returns SIM_ESTATE and enqueues nothing.
 *   - All floating point is IEEE binary32 with a fixed operation order, so results are
 *     reproducible bit for bit for a given (seed, env index, step index), whatever K is.
 *   - Random numbers: Philox4x32-10 keyed by the seed.  Action word of (env, t) = word
 *     (t mod 4) of the block with counter (env, t div 4, 0, 0).  State draw r of an env
 *     (r = 0 at reset, r = reset_count after the r-th auto-reset) uses counters
 *     (env, r, 1, j) for elements 4j..4j+3.
 *   - Action encoding: CartPole 0 = push left (-10 N), 1 = push right; Acrobot 0,1,2 =
 *     torque -1,0,+1; synthetic 0,1 = a = -1,+1.  Out-of-range bytes: CartPole and
 *     synthetic use (a != 0); Acrobot clamps to [0,2].
 */
#ifndef PAPER_2207_07736_SIM_H
#define PAPER_2207_07736_SIM_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct sim sim_t;   /* opaque */

enum { SIM_CARTPOLE = 0, SIM_ACROBOT = 1, SIM_SYNTH = 2 };
enum { SIM_OK = 0, SIM_EINVAL = -1, SIM_ENOMEM = -2, SIM_ECUDA = -3, SIM_ESTATE = -4, SIM_ECAPACITY = -5 };

#define SIM_POLICY_PARAM_COUNT 4610   /* W1[64][4] b1[64] W2[64][64] b2[64] W3[2][64] b3[2], rows = output units */

/*
 * sim_create -- make N simulator instances on the current CUDA device (Section 3: the N
 * parallel simulator instances of GPU vectorization; Section 2.2: the CartPole state of S = 4
 * floats; Section 4.2: the state-size factor S of the synthetic simulator).
 *   out       receives the handle.
 *   env_kind  SIM_CARTPOLE | SIM_ACROBOT | SIM_SYNTH.
 *   n_envs    1 .. 2^32-1.
 *   state_dim 4 for CartPole/Acrobot; a power of two in [4, 4096] for SIM_SYNTH.
 *   seed      Philox key.
 * Allocates device memory, then enqueues the initial-state draw (like sim_reset) on the
 * default stream and waits for it.  Errors: SIM_EINVAL, SIM_ENOMEM, SIM_ECUDA.
 */
int sim_create(sim_t **out, int env_kind, int64_t n_envs, int state_dim, uint64_t seed);

/* sim_destroy -- wait for the handle's stream, free everything.  NULL is SIM_EINVAL.
 * (No passage of the paper: lifetime hook.) */
int sim_destroy(sim_t *s);

/* sim_set_stream -- use this cudaStream_t (passed as void*) for all later work; NULL = default stream.
 * (No passage of the paper: plumbing hook; the stream belongs to the caller.) */
int sim_set_stream(sim_t *s, void *cuda_stream);

/* sim_set_env_offset -- global index of this handle's env 0 (default 0).  Random draws are keyed by
 * offset + local index, so handles that own disjoint ranges of one global population reproduce the
 * single-handle result exactly (sharding across GPUs needs no exchange: envs never interact).
 * offset + n_envs must not exceed 2^32.  Action draws use the new offset from the next call on, reset
 * draws from the next reset on; the states a handle already holds were drawn with the old offset, so call
 * sim_reset after changing it.  (No passage of the paper: Section 3 only says the instances are independent,
 * which is what makes this sharding exact.) */
int sim_set_env_offset(sim_t *s, uint64_t env_offset);

/* sim_set_compute_factor -- the paper's compute-factor knob C (Section 4.2: C multiplies the number of
 * simulation iterations per step, and with it the compute per step): one recorded step becomes C
 * iterations of the env's dynamics update under the step's one action (for Acrobot each iteration is a
 * full RK4 step with wrap and clip); reward, the done test and ep_len refer to the state after the last
 * iteration, and the trajectory still has one row per recorded step.  1 <= C <= 65536, default 1 (the
 * plain simulator).  Applies to every later sim_step / sim_rollout of the handle. */
int sim_set_compute_factor(sim_t *s, int compute_factor);

/* sim_set_action_stream -- how the uniform random policy turns Philox output into actions.
 *   SIM_ACTIONS_WORD (default): one 32-bit word per (env, step), as described at the top of this file.
 *   SIM_ACTIONS_BITS (CartPole only, an optional cheaper variant): one bit per (env, step): bit (t mod 128)
 *     of the 128-bit block with counter (env, c, 2, 0), c = (low 32 bits of t div 4) div 32; bit b is bit
 *     (b mod 32) of word (b div 32).  One Philox evaluation then serves 128 steps of an env instead of 4.
 * The MLP policy and caller-given actions are not affected.  SIM_EINVAL for other env kinds.  (The paper
 * names no generator; both streams are deterministic functions of (seed, env, step).) */
enum { SIM_ACTIONS_WORD = 0, SIM_ACTIONS_BITS = 1 };
int sim_set_action_stream(sim_t *s, int mode);

/* sim_set_policy_mode -- how the MLP policy is evaluated inside sim_rollout / sim_rollout_host /
 * sim_policy_logits (CartPole only; SIM_EINVAL for other env kinds or an unknown mode).  The two tensor modes are
 * the fusion of simulation and inference that Section 7 of the paper leaves as future work, with all three layers
 * on the tensor cores; the arithmetic is this library's.  Which mode meets which tolerance:
 *   SIM_POLICY_EXACT (default): the fp32 definition at the top of this file.  Logits, actions and everything
 *     else are bit-reproducible (tolerance: none).
 *   SIM_POLICY_TENSOR_PRECISE: logits within 1e-5 (absolute) of the fp32 definition for weights and observations
 *     of ordinary size (checked up to logits of magnitude 7); a sampled action can differ from exact mode only where
 *     the uniform draw lies within the resulting change of the action probability (below 1e-5 of the env-steps).
 *       z1 = W1 obs + b1      observation, W1 and b1 each split into THREE FP16 parts (x = x1 + x2 + x3); the six
 *                             leading products of parts are exact and summed in fp32 by the tensor core
 *       h1 = tanh'(z1)        tanh'(z) = 1 - 2 / (2^(2 log2(e) z) + 1) in fp32 with the GPU's base-2 exponential
 *                             and reciprocal approximations (one reciprocal shared by four evaluations): absolute
 *                             error below 4e-7
 *       z2 = b2 + W2 h1       h1 = hi + lo (hi = h1 cut to 11 significant bits, lo = f16(h1 - hi)), W2 = f16(W2) +
 *                             f16(W2 - f16(W2)); hi*hi + hi*lo + lo*hi summed in fp32 by the tensor core, b2 added in fp32
 *       h2 = tanh'(z2);       logits = b3 + W3 h2 in fp32 on the ordinary pipes (two partial sums per logit, over the
 *                             hidden units 4g, 4g+2 and 4g+1, 4g+3, added at the end).
 *   SIM_POLICY_TENSOR: the fast mode; it does NOT meet the 1e-5 logit tolerance (typical logit error 2e-3, bound
 *     below); use it where throughput matters more than the third digit of the action probabilities.
 *       z1 = W1 obs + b1      observation, W1 and b1 each split into two FP16 parts (x = hi + lo); the
 *                             products hi*hi, lo*hi, hi*lo are exact and summed in fp32: about 21 bits
 *       h1 = tanh~(f16(z1))   tanh~ = the GPU's packed half-precision tanh approximation (absolute error
 *                             about 2^-11), result in FP16
 *       z2 = b2 + sum_k f16(W2[j][k]) * h1[k]   FP16 operands (b2 split in two parts), products exact,
 *                             fp32 accumulation in the order the tensor core chooses
 *       h2 = tanh~(f16(z2));  logits = b3 + W3 h2 with W3 and b3 split in two FP16 parts, fp32 accumulation.
 *     The logit error is bounded by
 *       sum_j |W3[i][j]| (e + sum_k |W2[j][k]| (e + 2^-11 |h1[k]|)),  e = 2^-10.987 + 0.448 * 2^-11,
 *     and is far smaller for typical weights.
 * In both tensor modes parameters beyond the FP16 range (|x| > 65504) saturate; sampling, physics, reset and
 * outputs are unchanged, so a trajectory stays an exact CartPole trajectory under the actions it records; only the
 * action probabilities differ from exact mode, by the logit error.  Not bit-reproducible across GPU generations.
 * The first call that selects a tensor mode allocates a 4-byte device status word (see
 * sim_get_device_status). */
enum { SIM_POLICY_EXACT = 0, SIM_POLICY_TENSOR = 1, SIM_POLICY_TENSOR_PRECISE = 2 };
int sim_set_policy_mode(sim_t *s, int mode);

/* sim_get_device_status -- flags raised by kernels of this handle since it was created; synchronises the
 * handle's stream.  h_flags is a HOST pointer.  Bit 0 (SIM_STATUS_TENSOR_WAIT): a tensor-mode kernel gave
 * up waiting for the tensor core (every such wait is bounded, about a second); the rollout that hit it
 * left states and outputs of the affected envs unspecified.  0 when tensor mode was never selected. */
enum { SIM_STATUS_TENSOR_WAIT = 1 };
int sim_get_device_status(sim_t *s, uint32_t *h_flags);

/* sim_selfcheck_tensor_wait -- exercises the bounded wait of the tensor-mode kernels without a fault: one CTA
 * runs the policy with its tensor-core contractions left out, so every wait must give up (after about a
 * millisecond here), raise the status bit, skip the rest and free its tensor memory.  Synchronises the stream.
 *   h_status            HOST: the status word of that launch (expected SIM_STATUS_TENSOR_WAIT)
 *   h_threads_completed HOST: threads whose policy evaluation reported success (expected 0)
 * Uses a status word of its own: the handle's status (sim_get_device_status) is not touched. */
int sim_selfcheck_tensor_wait(sim_t *s, uint32_t *h_status, uint32_t *h_threads_completed);

/* sim_reset -- t = 0, ep_len = 0, reset_count = 0, state = draw #0 for every env: the initial state that the
 * step() transition of Section 3.2 starts from. */
int sim_reset(sim_t *s);

/*
 * sim_step -- one step of every env with caller-given actions: the step() state
 * transition of Section 3.2, vectorised over N (one kernel launch).
 *   d_actions  [N] int8 action indices.
 *   d_next_obs [N,S] fp32, state after the step and after auto-reset (may be NULL).
 *   d_rew      [N] fp32 (may be NULL).      d_done [N] u8 (may be NULL).
 * Advances t by one.
 */
int sim_step(sim_t *s, const int8_t *d_actions, float *d_next_obs, float *d_rew, uint8_t *d_done);

/*
 * sim_rollout -- T steps of every env in ceil(T / K_fused) kernel launches; inside one
 * launch the state lives in registers / shared memory (Section 4: simulator kernel fusion runs
 * K simulator steps in one kernel launch).  K_fused = 1 is plain GPU vectorization (Section 3).
 *   T >= 1, K_fused >= 1 (values above T are clamped to T).
 *   d_policy_params  NULL = uniform random actions; else SIM_POLICY_PARAM_COUNT floats of
 *                    the 4-64-64-2 tanh MLP whose softmax is sampled with the action word
 *                    (CartPole only; SIM_EINVAL for the other kinds).
 *   out_obs  [T,N,S] fp32: state each env's policy saw at step t (before the step).
 *   out_act  [T,N] int8.   out_rew [T,N] fp32.   out_done [T,N] u8.
 *   Any of the four may be NULL and is then not written.
 * Results do not depend on K_fused.  Advances t by T.
 */
int sim_rollout(sim_t *s, int T, int K_fused, const float *d_policy_params,
                float *out_obs, int8_t *out_act, float *out_rew, uint8_t *out_done);

/*
 * sim_rollout_host -- the same rollout with HOST buffers, for callers that consume the
 * trajectory on the CPU.  h_policy_params (NULL or SIM_POLICY_PARAM_COUNT floats) is
 * copied to the device; the trajectory is produced in chunks of K_fused steps into
 * library-owned device staging buffers and copied to the h_* arrays (same shapes as in
 * sim_rollout, each may be NULL) while the next chunk is being computed.  Pinned host
 * memory gives the best copy rate; pageable memory works.  Blocks until all copies are
 * done.  Staging buffers (two chunks) are allocated on first use and kept by the handle;
 * SIM_ENOMEM if they do not fit.
 */
int sim_rollout_host(sim_t *s, int T, int K_fused, const float *h_policy_params,
                     float *h_obs, int8_t *h_act, float *h_rew, uint8_t *h_done);

/* Inspection and checkpoint hooks: copy state / counters out of or into the handle
 * (device pointers; d_* may be NULL to skip one).  h_t is a host pointer.  (No passage of the paper:
 * together with t and the seed these are the complete state of a rollout, so saving and restoring them
 * resumes it exactly.) */
int sim_get_state(sim_t *s, float *d_state /* [N,S] */);
int sim_set_state(sim_t *s, const float *d_state /* [N,S] */);
int sim_get_counters(sim_t *s, uint32_t *d_ep_len, uint32_t *d_reset_count, uint64_t *h_t);
int sim_set_counters(sim_t *s, const uint32_t *d_ep_len, const uint32_t *d_reset_count, uint64_t t);

/* sim_policy_logits -- logits of the MLP for M observations (no sampling, no stepping): the inference half of
 * the data-collection loop of Section 2.1 on its own, as a test and inspection hook.
 *   d_obs [M,4] fp32, d_params SIM_POLICY_PARAM_COUNT fp32, d_logits [M,2] fp32.  s may be
 *   any live handle (it provides the stream and the policy mode). */
int sim_policy_logits(sim_t *s, const float *d_obs, int64_t M, const float *d_params, float *d_logits);

/* sim_acrobot_observation -- the six-value observation an RL consumer of Acrobot usually wants,
 * (cos theta1, sin theta1, cos theta2, sin theta2, omega1, omega2), from raw 4-float states (the
 * trajectory's out_obs rows, or sim_get_state): d_state [M,4] fp32 -> d_obs6 [M,6] fp32, both device
 * pointers, 16- and 8-byte aligned.  Uses the library's specified sin/cos, so it is reproducible bit for
 * bit.  (The paper's simulators expose raw state only; this is a convenience on top of the path.) */
int sim_acrobot_observation(sim_t *s, const float *d_state, int64_t M, float *d_obs6);

/* sim_episode_returns -- running return of every episode of a trajectory, for consumers that label the
 * collected samples with returns (Section 2.1: the rewards become the labels of the collected data).  d_rew [T,n] fp32 and d_done [T,n] u8 as written by sim_rollout; d_ret [T,n] fp32 receives
 * ret[t,e] = rew[t,e] + (done[t-1,e] ? 0 : ret[t-1,e]), added in time order in fp32.  d_carry [n] fp32
 * (nullable) carries the return accumulated so far across calls: read before row 0, written after the last
 * row (0 where the episode just ended).  All device pointers. */
int sim_episode_returns(sim_t *s, const float *d_rew, const uint8_t *d_done, int T, int64_t n, float *d_carry, float *d_ret);

/* sim_selfcheck_division -- numerical self-check of the divisions inside the fused kernels (the paper
 * has no counterpart; it exists so a test can prove the kernels' arithmetic on the device they run
 * on).  The fused CartPole and Acrobot kernels divide by well-conditioned denominators with a refined
 * hardware reciprocal instead of the general division sequence, and the MLP's tanh uses the refined
 * reciprocal of exp(2|x|)+1.  For EVERY binary32 value of each denominator range (CartPole [0.62, 0.67];
 * Acrobot [2.4, 4.6] and [0.5, 1.1]; tanh [2, 2^27]) the refined reciprocal is compared with the correctly
 * rounded one, and for the division ranges the kernels' quotient is compared with the IEEE quotient for
 * nums_per_den (CartPole) or nums_per_den/16 (Acrobot) pseudo-random numerators per denominator inside the
 * guarded exponent range.  *h_mismatches (host) = reciprocal mismatches * 2^32 + quotient mismatches; 0
 * means the kernels' divisions are the IEEE divisions on this device.  Synchronises. */
int sim_selfcheck_division(sim_t *s, int nums_per_den, uint64_t *h_mismatches);

/*
 * sim_rollout_noalloc -- reset N envs and roll them out for T steps without allocating anything
 * (the paper has no counterpart: it is an addition for callers that cannot allocate).
 *
 * Who needs it: a latency-critical loop that must not call cudaMalloc / cudaFree because both
 * stall every stream of the device; a process whose device memory has been handed out in full to
 * another allocator; a component that may only touch the buffers it is given.  Instead of the
 * buffers sim_create would allocate, the per-env working memory (state matrix, episode lengths,
 * reset counts) sits in a fixed array of SIM_NOALLOC_SCRATCH_BYTES inside the library's device
 * image; every GPU that loads the library holds that array until the process exits.
 *
 *   env_kind, n_envs, state_dim, seed   as in sim_create; env offset 0.
 *   T, K_fused, d_policy_params, out_*  as in sim_rollout (device pointers, outputs nullable);
 *                                       the rollout starts from the freshly drawn state at t = 0,
 *                                       so the outputs equal sim_create + sim_rollout bit for bit.
 *   cuda_stream                         cudaStream_t as void*, NULL = default stream.  Work is
 *                                       only enqueued; the caller synchronises.
 * Limit: 256-aligned(4*state_dim*n_envs) + 2 * 256-aligned(4*n_envs) bytes must not exceed
 * SIM_NOALLOC_SCRATCH_BYTES (at most 349 504 four-float envs); larger problems return
 * SIM_ECAPACITY and enqueue nothing.  Other errors: SIM_EINVAL, SIM_ECUDA.
 * The call makes no cudaMalloc, cudaFree or other allocating call, on the host or the device.
 * First use on a device looks up the array's device address (once per device, with that device
 * current): make that first call outside any stream capture.  With CUDA's lazy module loading that
 * first lookup is also the moment the driver loads the library's device image, array included, and
 * reserves its 8 MiB, which can fail if the device is full: callers that must not allocate later
 * should make one small warm-up call at start-up.  From the second call on a device nothing is
 * allocated by anyone (the test suite checks the device's free memory across such calls).
 * The launches are planned exactly as in sim_rollout (same kernels for the same env kind, policy and
 * launch length); the policy is evaluated in exact mode.
 * All calls share the one array.  It keeps the previous call's contents; each call rewrites every
 * word it later reads before reading it, so nothing needs clearing by the caller -- but two
 * calls whose work overlaps on the GPU (different streams, or one process-wide device shared by
 * threads) race on it and corrupt each other.  Serialise them.
 */
#define SIM_NOALLOC_SCRATCH_BYTES (8u << 20)
int sim_rollout_noalloc(int env_kind, int64_t n_envs, int state_dim, uint64_t seed, int T, int K_fused,
                        const float *d_policy_params, float *out_obs, int8_t *out_act, float *out_rew, uint8_t *out_done,
                        void *cuda_stream);

/* sim_launch_count -- kernels launched by this handle since creation (the launch accounting of Section 3.3:
 * one launch per K_fused steps). */
int64_t sim_launch_count(sim_t *s);

/* sim_strerror -- static string for a SIM_* code.  sim_last_cuda_error -- the cudaError_t
 * behind the most recent SIM_ECUDA of this handle (0 if none).  (No passage of the paper: error reporting.) */
const char *sim_strerror(int code);
int sim_last_cuda_error(sim_t *s);

#ifdef __cplusplus
}
#endif
#endif
