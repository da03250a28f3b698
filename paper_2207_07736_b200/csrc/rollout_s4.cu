// Generic fused multi-step rollout for envs with a 4-float state (Acrobot; CartPole with caller-given
// actions): one thread owns
// one env, keeps its state and counters in registers for the K steps of the launch, and streams
// the per-step trajectory rows to global memory with coalesced stores (obs as one float4 per
// env, so a warp writes 512 contiguous bytes).
#include "sim_internal.h"
#include "sim_envs.cuh"

namespace simk {

// ---------------------------------------------------------------------------------------------
// The rollout kernel.
// ---------------------------------------------------------------------------------------------
template <int ENV>
__device__ __forceinline__ int random_action(uint32_t w)
{
    return ENV == ENV_ACROBOT ? (int)__umulhi(w, 3u) : (int)(w >> 31);
}

// One recorded step: C iterations of the dynamics under one action (C = 1: the plain simulator);
// reward, done and ep_len refer to the state after the last iteration.
template <int ENV>
__device__ __forceinline__ bool env_step(float4 &s, int &act, uint32_t &len, float &rew, int C)
{
    if (ENV == ENV_CARTPOLE) {
        act = act ? 1 : 0;
        bool done = cartpole_step(s, act != 0);
        for (int c = 1; c < C; ++c) done = cartpole_step(s, act != 0);
        len += 1u;
        rew = 1.0f;
        return done;
    } else {
        act = min(max(act, 0), 2);
        bool goal = acrobot_step(s, act);
        for (int c = 1; c < C; ++c) goal = acrobot_step(s, act);
        len += 1u;
        rew = goal ? 0.0f : -1.0f;
        return goal | (len >= 500u);
    }
}

constexpr int kS4Threads = 64;      // small CTAs spread the envs evenly over 148 SMs

template <int ENV, int POLICY>
__global__ void __launch_bounds__(kS4Threads)
rollout_s4_kernel(const __grid_constant__ S4Args a)
{
    const uint64_t i64 = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i64 >= a.n) return;
    const uint32_t i = (uint32_t)i64;
    const uint32_t env = a.env_offset + i;
    pdl_wait();
    pdl_release();

    float4 s = a.state[i];
    uint32_t len = a.ep_len[i];
    uint32_t rc = a.reset_count[i];
    size_t row = i;                                    // element index into the [K, n] outputs

    const int nblk = (a.phase + a.K + 3) >> 2;         // Philox action blocks touched by this launch
    uint4 bits_blk = make_uint4(0u, 0u, 0u, 0u);       // bit-sliced action stream: current 128-bit block
    uint32_t bits_idx = 0u;
    bool bits_have = false;
    for (int b = 0; b < nblk; ++b) {
        uint4 blk = make_uint4(0u, 0u, 0u, 0u);
        if (POLICY != POLICY_GIVEN && !a.action_bits) blk = philox(env, a.tb0 + (uint32_t)b, 0u, 0u, a.rk);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int k = 4 * b + j - a.phase;         // step index inside the launch (warp-uniform)
            if (k < 0 || k >= a.K) continue;
            uint32_t w = j == 0 ? blk.x : j == 1 ? blk.y : j == 2 ? blk.z : blk.w;
            if (POLICY == POLICY_RANDOM && ENV == ENV_CARTPOLE && a.action_bits) {
                // bit-sliced stream: bit (t mod 128) of the block with counter (env, (t >> 2) >> 5, 2, 0)
                const uint32_t tb = a.tb0 + (uint32_t)b;
                if (!bits_have || (tb >> 5) != bits_idx) { bits_blk = philox(env, tb >> 5, 2u, 0u, a.rk); bits_idx = tb >> 5; bits_have = true; }
                const uint32_t bi = ((tb & 31u) << 2) | (uint32_t)j;
                const uint32_t word = (bi >> 5) == 0 ? bits_blk.x : (bi >> 5) == 1 ? bits_blk.y : (bi >> 5) == 2 ? bits_blk.z : bits_blk.w;
                w = (word >> (bi & 31u)) << 31;
            }

            if (a.out_obs) __stcs(&a.out_obs[row], s);

            int act;
            if (POLICY == POLICY_GIVEN) {
                act = a.actions[i];
            } else {
                act = random_action<ENV>(w);
            }

            float rew;
            const bool done = env_step<ENV>(s, act, len, rew, a.C);

            if (a.out_act) __stcs(&a.out_act[row], (int8_t)act);
            if (a.out_rew) __stcs(&a.out_rew[row], rew);
            if (a.out_done) __stcs(&a.out_done[row], (uint8_t)done);

            if (done) {
                rc += 1u;
                s = draw_state4<ENV>(env, rc, 0u, a.rk);
                len = 0u;
            }
            row += a.n;
        }
    }

    a.state[i] = s;
    a.ep_len[i] = len;
    a.reset_count[i] = rc;
    if (POLICY == POLICY_GIVEN && a.next_obs) a.next_obs[i] = s;
}

template <int ENV>
__global__ void __launch_bounds__(256)
reset_s4_kernel(float4 *state, uint32_t *ep_len, uint32_t *reset_count, uint32_t n, uint32_t env_offset, const __grid_constant__ RoundKeys rk)
{
    const uint64_t i64 = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i64 >= n) return;
    const uint32_t i = (uint32_t)i64;
    state[i] = draw_state4<ENV>(env_offset + i, 0u, 0u, rk);
    ep_len[i] = 0u;
    reset_count[i] = 0u;
}

// One thread per group of four consecutive elements of the [n, S] synthetic state matrix.
__global__ void __launch_bounds__(256)
reset_synth_kernel(float4 *state, uint32_t *ep_len, uint32_t *reset_count, uint32_t n, int log2_groups, uint32_t env_offset,
                   const __grid_constant__ RoundKeys rk)
{
    const size_t g = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    const size_t total = (size_t)n << log2_groups;
    if (g >= total) return;
    const uint32_t i = (uint32_t)(g >> log2_groups);
    const uint32_t j = (uint32_t)(g & ((1u << log2_groups) - 1u));
    state[g] = draw_state4<ENV_SYNTH>(env_offset + i, 0u, j, rk);
    if (j == 0) { ep_len[i] = 0u; reset_count[i] = 0u; }
}

// Gym-style six-value Acrobot observation (cos t1, sin t1, cos t2, sin t2, w1, w2) of M states.
__global__ void __launch_bounds__(256)
acrobot_observation_kernel(const float4 *__restrict__ state, int64_t M, float *__restrict__ obs6)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= M) return;
    const float4 s = state[i];
    float s1, c1, s2, c2;
    sincos_s(s.x, s1, c1);
    sincos_s(s.y, s2, c2);
    float2 *o = reinterpret_cast<float2 *>(obs6 + i * 6);       // rows of 24 bytes: 8-byte aligned
    o[0] = make_float2(c1, s1);
    o[1] = make_float2(c2, s2);
    o[2] = make_float2(s.z, s.w);
}

cudaError_t launch_acrobot_observation(const float *state, int64_t M, float *obs6, cudaStream_t st)
{
    if (M <= 0) return cudaSuccess;
    const int64_t blocks = (M + 255) / 256;
    if (blocks > 0x7FFFFFFFll) return cudaErrorInvalidConfiguration;
    acrobot_observation_kernel<<<(unsigned)blocks, 256, 0, st>>>(reinterpret_cast<const float4 *>(state), M, obs6);
    return cudaGetLastError();
}

// Running episode return over a trajectory: one thread per env walks the T rows (each row access of a
// warp is contiguous), adding in time order, restarting after a done.
__global__ void __launch_bounds__(256)
episode_returns_kernel(const float *__restrict__ rew, const uint8_t *__restrict__ done, int T, int64_t n, float *carry, float *__restrict__ ret)
{
    const int64_t e = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (e >= n) return;
    float acc = carry ? carry[e] : 0.0f;
    for (int t = 0; t < T; ++t) {
        const size_t at = (size_t)t * (size_t)n + (size_t)e;
        acc = __fadd_rn(acc, rew[at]);
        ret[at] = acc;
        if (done[at]) acc = 0.0f;
    }
    if (carry) carry[e] = acc;
}

cudaError_t launch_episode_returns(const float *rew, const uint8_t *done, int T, int64_t n, float *carry, float *ret, cudaStream_t st)
{
    if (n <= 0 || T <= 0) return cudaSuccess;
    const int64_t blocks = (n + 255) / 256;
    if (blocks > 0x7FFFFFFFll) return cudaErrorInvalidConfiguration;
    episode_returns_kernel<<<(unsigned)blocks, 256, 0, st>>>(rew, done, T, n, carry, ret);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------
// Launchers
// ---------------------------------------------------------------------------------------------
cudaError_t launch_reset(int env_kind, int S, float *state, uint32_t *ep_len, uint32_t *reset_count,
                         uint32_t n, uint32_t env_offset, const RoundKeys &rk, cudaStream_t st)
{
    if (env_kind == ENV_SYNTH) {
        int lg = 0;
        while ((4 << lg) < S) ++lg;
        const size_t total = (size_t)n << lg;
        const size_t blocks = (total + 255) / 256;
        if (blocks > 0x7FFFFFFFull) return cudaErrorInvalidConfiguration;
        reset_synth_kernel<<<(unsigned)blocks, 256, 0, st>>>(reinterpret_cast<float4 *>(state), ep_len, reset_count, n, lg, env_offset, rk);
    } else {
        const unsigned blocks = (n + 255u) / 256u;
        if (env_kind == ENV_CARTPOLE)
            reset_s4_kernel<ENV_CARTPOLE><<<blocks, 256, 0, st>>>(reinterpret_cast<float4 *>(state), ep_len, reset_count, n, env_offset, rk);
        else
            reset_s4_kernel<ENV_ACROBOT><<<blocks, 256, 0, st>>>(reinterpret_cast<float4 *>(state), ep_len, reset_count, n, env_offset, rk);
    }
    return cudaGetLastError();
}

template <int ENV, int POLICY>
static cudaError_t launch_s4_t(const S4Args &a, cudaStream_t st)
{
    const unsigned blocks = (a.n + kS4Threads - 1u) / kS4Threads;
    return launch_overlapped(a.K <= kOverlapMaxK, rollout_s4_kernel<ENV, POLICY>, dim3(blocks), dim3(kS4Threads), 0, st, a);
}

cudaError_t launch_s4(int env_kind, int policy, const S4Args &a, cudaStream_t st)
{
    if (env_kind == ENV_CARTPOLE) {
        if (policy == POLICY_RANDOM) return launch_s4_t<ENV_CARTPOLE, POLICY_RANDOM>(a, st);
        if (policy == POLICY_GIVEN) return launch_s4_t<ENV_CARTPOLE, POLICY_GIVEN>(a, st);
    } else if (env_kind == ENV_ACROBOT) {
        if (policy == POLICY_RANDOM) return launch_s4_t<ENV_ACROBOT, POLICY_RANDOM>(a, st);
        if (policy == POLICY_GIVEN) return launch_s4_t<ENV_ACROBOT, POLICY_GIVEN>(a, st);
    }
    return cudaErrorInvalidValue;
}

}  // namespace simk
