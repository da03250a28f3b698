// Host-side declarations shared by the translation units of the library (not part of the ABI).
#pragma once
#include <cstdint>
#include <cuda_runtime.h>
#include "sim_math.cuh"

namespace simk {

enum : int { POLICY_RANDOM = 0, POLICY_GIVEN = 1, POLICY_MLP = 2 };

// Arguments of one launch over envs with a 4-float state (CartPole, Acrobot).
// Output pointers are already advanced to the row of the launch's first step.
struct S4Args {
    float4 *state;            // [n]
    uint32_t *ep_len;         // [n]
    uint32_t *reset_count;    // [n]
    uint32_t n;               // envs in this handle
    uint32_t env_offset;      // global index of env 0
    uint32_t tb0;             // (t0 >> 2) truncated to 32 bits: Philox counter word of the first action block
    int phase;                // t0 & 3
    int K;                    // steps in this launch
    int C;                    // compute factor: dynamics iterations per recorded step (>= 1)
    int action_bits;          // 1: bit-sliced action stream (CartPole, random policy)
    float4 *out_obs;          // [K, n] or nullptr
    int8_t *out_act;          // [K, n] or nullptr
    float *out_rew;           // [K, n] or nullptr
    uint8_t *out_done;        // [K, n] or nullptr
    const int8_t *actions;    // [n], POLICY_GIVEN only
    float4 *next_obs;         // [n] post-step state, POLICY_GIVEN only (nullable)
    const float *params;      // MLP parameters, POLICY_MLP only
    uint32_t *status;         // device status word (tensor-mode policy: bit 0 = a bounded wait ran out), nullable
    RoundKeys rk;
};

// Arguments of one launch of the synthetic S-float simulator.
struct SynthArgs {
    float *state;             // [n, S]
    uint32_t *ep_len;
    uint32_t *reset_count;
    uint32_t n;
    uint32_t env_offset;
    uint32_t tb0;
    int phase;
    int K;
    int C;                    // compute factor
    float *out_obs;           // [K, n, S] or nullptr
    int8_t *out_act;
    float *out_rew;
    uint8_t *out_done;
    const int8_t *actions;    // [n] or nullptr (given-action step, K == 1)
    float *next_obs;          // [n, S] or nullptr
    RoundKeys rk;
};

// One population of envs as the launch planner sees it: kind, sizes, where its buffers live, keys, the step counter
// and the per-handle options.  A handle of the C ABI is one of these plus host-side bookkeeping.
struct SimCore {
    int env_kind;
    int S;
    uint32_t n;
    uint64_t env_offset;
    uint64_t t;               // global step index of the next step
    int compute_factor;
    int action_stream;
    int policy_mode;
    uint32_t *d_status;       // device status word (tensor policy modes), nullable
    float *state;             // [n, S]
    uint32_t *ep_len;         // [n]
    uint32_t *reset_count;    // [n]
    RoundKeys rk;
};

// Programmatic dependent launch: consecutive rollout launches of one stream overlap their launch
// latency.  A kernel calls pdl_wait() before its first global-memory access (it returns once every
// earlier grid of the stream has completed and its writes are visible; a no-op when the launch did not
// ask for overlap) and pdl_release() right after, which lets the next launch start its own prologue.
// Overlap is requested for short launches only (K <= kOverlapMaxK): there the launch latency is the
// cost; for long launches, CTAs of the next grid placed while the current one still fills the SMs end up
// unevenly spread and the next grid runs slower (measured: +40 % at K = 1000).
constexpr int kOverlapMaxK = 4;
#ifdef __CUDACC__
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_release() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

template <typename... KArgs, typename... Args>
static inline cudaError_t launch_overlapped(bool overlap, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args &&...args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr; cfg.numAttrs = overlap ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}
#endif

void expand_round_keys(uint64_t seed, RoundKeys &rk);
// The launch planner: one launch of K steps of population `c` from step c.t (it advances nothing itself).
cudaError_t launch_planned(const SimCore &c, int K, int policy, const float *d_params, const int8_t *d_actions, float *next_obs,
                           float *obs, int8_t *act, float *rew, uint8_t *done, cudaStream_t st);

// Launchers (each returns the launch error, enqueues on `st`, never synchronises).
cudaError_t launch_reset(int env_kind, int S, float *state, uint32_t *ep_len, uint32_t *reset_count,
                         uint32_t n, uint32_t env_offset, const RoundKeys &rk, cudaStream_t st);
cudaError_t launch_s4(int env_kind, int policy, const S4Args &a, cudaStream_t st);
cudaError_t launch_cartpole_random(const S4Args &a, cudaStream_t st);   // CartPole, uniform random policy, packed two-env kernel
cudaError_t launch_acrobot_random(const S4Args &a, cudaStream_t st);    // Acrobot, uniform random torque, packed two-env kernel
cudaError_t launch_cartpole_mlp(const S4Args &a, cudaStream_t st);      // CartPole, MLP policy, packed two-env kernel
cudaError_t launch_cartpole_mlp_tc(const S4Args &a, cudaStream_t st);   // CartPole, MLP policy in tensor mode (tcgen05 hidden layer)
cudaError_t launch_cartpole_mlp_tcp(const S4Args &a, cudaStream_t st);  // the same with split operands and fp32 tanh (precise tensor mode)
cudaError_t launch_policy_logits_tcp(const float *obs, int64_t M, const float *params, float *logits, uint32_t *status, cudaStream_t st);
cudaError_t launch_policy_logits_tc(const float *obs, int64_t M, const float *params, float *logits, uint32_t *status, cudaStream_t st);
cudaError_t launch_tensor_wait_selfcheck(const float *params, long long wait_cycles, uint32_t *status, uint32_t *completed, cudaStream_t st);   // 256 words
cudaError_t launch_division_selfcheck(int nums_per_den, unsigned long long *d_bad, cudaStream_t st);
cudaError_t launch_synth(int S, const SynthArgs &a, cudaStream_t st);
cudaError_t launch_acrobot_observation(const float *state, int64_t M, float *obs6, cudaStream_t st);
cudaError_t launch_episode_returns(const float *rew, const uint8_t *done, int T, int64_t n, float *carry, float *ret, cudaStream_t st);
cudaError_t launch_policy_logits(const float *obs, int64_t M, const float *params, float *logits, cudaStream_t st);

}  // namespace simk
