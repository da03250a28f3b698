// Fused multi-step rollout for envs with a 4-float state (CartPole, Acrobot): one thread owns
// one env, keeps its state and counters in registers for the K steps of the launch, and streams
// the per-step trajectory rows to global memory with coalesced stores (obs as one float4 per
// env, so a warp writes 512 contiguous bytes).
#include "sim_internal.h"
#include "sim_envs.cuh"

namespace simk {

// ---------------------------------------------------------------------------------------------
// MLP policy 4 -> 64 -> 64 -> 2 (tanh).  The parameters are staged once per CTA into shared
// memory, layer 2 transposed so that the weights of consecutive output units for one input are
// contiguous (one 128-bit broadcast load feeds four accumulators).  Every output unit is one
// sequential fma chain over its inputs in ascending order, starting from the bias.
// ---------------------------------------------------------------------------------------------
struct MlpSmem {
    float4 w1[64];        // w1[j] = W1[j][0..3]
    float b1[64];
    float w2t[64 * 64];   // w2t[k*64 + j] = W2[j][k]
    float b2[64];
    float2 w3[64];        // w3[j] = (W3[0][j], W3[1][j])
    float b3[2];
};

__device__ __forceinline__ void stage_mlp(const float *__restrict__ p, MlpSmem &s)
{
    const int tid = threadIdx.x, nt = blockDim.x;
    for (int i = tid; i < 64; i += nt) {
        s.w1[i] = make_float4(p[i * 4 + 0], p[i * 4 + 1], p[i * 4 + 2], p[i * 4 + 3]);
        s.b1[i] = p[256 + i];
        s.b2[i] = p[4416 + i];
        s.w3[i] = make_float2(p[4480 + i], p[4544 + i]);
    }
    for (int i = tid; i < 4096; i += nt) {
        const int j = i >> 6, k = i & 63;              // coalesced read of W2[j][k]
        s.w2t[k * 64 + j] = p[320 + i];
    }
    if (tid < 2) s.b3[tid] = p[4608 + tid];
    __syncthreads();
}

__device__ __forceinline__ void mlp_logits(const float4 obs, const MlpSmem &s, float &l0, float &l1)
{
    float h1[64];
#pragma unroll
    for (int j = 0; j < 64; ++j) {
        const float4 w = s.w1[j];
        float acc = s.b1[j];
        acc = __fmaf_rn(w.x, obs.x, acc);
        acc = __fmaf_rn(w.y, obs.y, acc);
        acc = __fmaf_rn(w.z, obs.z, acc);
        acc = __fmaf_rn(w.w, obs.w, acc);
        h1[j] = tanh_s(acc);
    }
    l0 = s.b3[0];
    l1 = s.b3[1];
#pragma unroll 1
    for (int jb = 0; jb < 64; jb += 8) {
        float acc[8];
        {
            const float4 ba = *reinterpret_cast<const float4 *>(&s.b2[jb]);
            const float4 bb = *reinterpret_cast<const float4 *>(&s.b2[jb + 4]);
            acc[0] = ba.x; acc[1] = ba.y; acc[2] = ba.z; acc[3] = ba.w;
            acc[4] = bb.x; acc[5] = bb.y; acc[6] = bb.z; acc[7] = bb.w;
        }
#pragma unroll
        for (int k = 0; k < 64; ++k) {
            const float4 wa = *reinterpret_cast<const float4 *>(&s.w2t[k * 64 + jb]);
            const float4 wb = *reinterpret_cast<const float4 *>(&s.w2t[k * 64 + jb + 4]);
            const float h = h1[k];
            acc[0] = __fmaf_rn(wa.x, h, acc[0]); acc[1] = __fmaf_rn(wa.y, h, acc[1]);
            acc[2] = __fmaf_rn(wa.z, h, acc[2]); acc[3] = __fmaf_rn(wa.w, h, acc[3]);
            acc[4] = __fmaf_rn(wb.x, h, acc[4]); acc[5] = __fmaf_rn(wb.y, h, acc[5]);
            acc[6] = __fmaf_rn(wb.z, h, acc[6]); acc[7] = __fmaf_rn(wb.w, h, acc[7]);
        }
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float h2 = tanh_s(acc[i]);
            const float2 w3 = s.w3[jb + i];
            l0 = __fmaf_rn(w3.x, h2, l0);
            l1 = __fmaf_rn(w3.y, h2, l1);
        }
    }
}

// Inverse-CDF sample over the two unnormalised softmax weights: action 0 iff u*(e0+e1) < e0.
__device__ __forceinline__ int sample2(float l0, float l1, uint32_t w)
{
    const float m = fmaxf(l0, l1);
    const float e0 = exp_s(__fsub_rn(l0, m));
    const float e1 = exp_s(__fsub_rn(l1, m));
    const float thr = __fmul_rn(uniform01(w), __fadd_rn(e0, e1));
    return (thr < e0) ? 0 : 1;
}

// ---------------------------------------------------------------------------------------------
// The rollout kernel.
// ---------------------------------------------------------------------------------------------
template <int ENV>
__device__ __forceinline__ int random_action(uint32_t w)
{
    return ENV == ENV_ACROBOT ? (int)__umulhi(w, 3u) : (int)(w >> 31);
}

template <int ENV>
__device__ __forceinline__ bool env_step(float4 &s, int &act, uint32_t &len, float &rew)
{
    if (ENV == ENV_CARTPOLE) {
        act = act ? 1 : 0;
        const bool done = cartpole_step(s, act != 0);
        len += 1u;
        rew = 1.0f;
        return done;
    } else {
        act = min(max(act, 0), 2);
        const bool goal = acrobot_step(s, act);
        len += 1u;
        rew = goal ? 0.0f : -1.0f;
        return goal | (len >= 500u);
    }
}

constexpr int kS4Threads = 64;      // small CTAs spread 65 536 envs evenly over 148 SMs
constexpr int kMlpThreads = 128;

template <int ENV, int POLICY>
__global__ void __launch_bounds__(POLICY == POLICY_MLP ? kMlpThreads : kS4Threads)
rollout_s4_kernel(const __grid_constant__ S4Args a)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    MlpSmem &ms = *reinterpret_cast<MlpSmem *>(smem_raw);
    if (POLICY == POLICY_MLP) stage_mlp(a.params, ms);

    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= a.n) return;
    const uint32_t env = a.env_offset + i;

    float4 s = a.state[i];
    uint32_t len = a.ep_len[i];
    uint32_t rc = a.reset_count[i];
    size_t row = i;                                    // element index into the [K, n] outputs

    const int nblk = (a.phase + a.K + 3) >> 2;         // Philox action blocks touched by this launch
    for (int b = 0; b < nblk; ++b) {
        uint4 blk = make_uint4(0u, 0u, 0u, 0u);
        if (POLICY != POLICY_GIVEN) blk = philox(env, a.tb0 + (uint32_t)b, 0u, 0u, a.rk);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int k = 4 * b + j - a.phase;         // step index inside the launch (warp-uniform)
            if (k < 0 || k >= a.K) continue;
            const uint32_t w = j == 0 ? blk.x : j == 1 ? blk.y : j == 2 ? blk.z : blk.w;

            if (a.out_obs) __stcs(&a.out_obs[row], s);

            int act;
            if (POLICY == POLICY_GIVEN) {
                act = a.actions[i];
            } else if (POLICY == POLICY_MLP) {
                float l0, l1;
                mlp_logits(s, ms, l0, l1);
                act = sample2(l0, l1, w);
            } else {
                act = random_action<ENV>(w);
            }

            float rew;
            const bool done = env_step<ENV>(s, act, len, rew);

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
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n) return;
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

__global__ void __launch_bounds__(kMlpThreads)
policy_logits_kernel(const float4 *__restrict__ obs, int64_t M, const float *__restrict__ params, float2 *__restrict__ logits)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    MlpSmem &ms = *reinterpret_cast<MlpSmem *>(smem_raw);
    stage_mlp(params, ms);
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= M) return;
    float l0, l1;
    mlp_logits(obs[i], ms, l0, l1);
    logits[i] = make_float2(l0, l1);
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
    constexpr int threads = POLICY == POLICY_MLP ? kMlpThreads : kS4Threads;
    const size_t smem = POLICY == POLICY_MLP ? sizeof(MlpSmem) : 0;
    const unsigned blocks = (a.n + threads - 1u) / threads;
    rollout_s4_kernel<ENV, POLICY><<<blocks, threads, smem, st>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_s4(int env_kind, int policy, const S4Args &a, cudaStream_t st)
{
    if (env_kind == ENV_CARTPOLE) {
        if (policy == POLICY_RANDOM) return launch_s4_t<ENV_CARTPOLE, POLICY_RANDOM>(a, st);
        if (policy == POLICY_GIVEN) return launch_s4_t<ENV_CARTPOLE, POLICY_GIVEN>(a, st);
        if (policy == POLICY_MLP) return launch_s4_t<ENV_CARTPOLE, POLICY_MLP>(a, st);
    } else if (env_kind == ENV_ACROBOT) {
        if (policy == POLICY_RANDOM) return launch_s4_t<ENV_ACROBOT, POLICY_RANDOM>(a, st);
        if (policy == POLICY_GIVEN) return launch_s4_t<ENV_ACROBOT, POLICY_GIVEN>(a, st);
    }
    return cudaErrorInvalidValue;
}

cudaError_t launch_policy_logits(const float *obs, int64_t M, const float *params, float *logits, cudaStream_t st)
{
    if (M <= 0) return cudaSuccess;
    const int64_t blocks = (M + kMlpThreads - 1) / kMlpThreads;
    if (blocks > 0x7FFFFFFFll) return cudaErrorInvalidConfiguration;
    policy_logits_kernel<<<(unsigned)blocks, kMlpThreads, sizeof(MlpSmem), st>>>(reinterpret_cast<const float4 *>(obs), M, params,
                                                                                reinterpret_cast<float2 *>(logits));
    return cudaGetLastError();
}

}  // namespace simk
