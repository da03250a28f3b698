// Fused multi-step rollout of the synthetic S-float simulator (the "state factor" experiment:
// S times the state, S times the global loads and stores per unfused step).
//
// Mapping: an env's S floats are split into L = S/E contiguous chunks of E floats, one chunk
// per thread, held in registers for all K steps of the launch.  L <= 32: the L threads of an env
// are adjacent lanes of one warp (several envs per warp when L < 32) and exchange the one halo
// element and the partial sums with shuffles.  L > 32: one CTA per env, the warps exchange
// through shared memory.  The sum of squares follows an adjacent-pairs-first binary tree over
// the element index: inside a chunk, then across lanes by xor-shuffles, then across warps.
#include "sim_internal.h"
#include "sim_envs.cuh"

namespace simk {

template <int S> struct SynthShape {
    static constexpr int E = S <= 128 ? 4 : (S <= 512 ? S / 32 : 16);   // floats per thread
    static constexpr int L = S / E;                                     // threads per env
    static constexpr int WARPS = L > 32 ? L / 32 : 1;                   // warps per env when L > 32
    static constexpr int THREADS = L > 32 ? L : 256;
    static constexpr int ENVS_PER_CTA = THREADS / L;
};

template <int S>
__global__ void __launch_bounds__(SynthShape<S>::THREADS)
rollout_synth_kernel(const __grid_constant__ SynthArgs a)
{
    using Sh = SynthShape<S>;
    constexpr int E = Sh::E, L = Sh::L, W = Sh::WARPS;
    constexpr int LS = L < 32 ? L : 32;                 // lanes of one env inside a warp
    __shared__ float sm_halo[W];
    __shared__ float sm_sum[W];

    const uint32_t tid = threadIdx.x;
    const uint32_t lane = tid & 31u;
    const uint32_t warp = tid >> 5;
    const uint32_t sub = tid % L;                       // this thread's chunk index inside its env
    uint32_t i = blockIdx.x * (uint32_t)Sh::ENVS_PER_CTA + tid / L;
    const bool valid = i < a.n;                         // tail threads compute on env n-1 and store nothing
    if (!valid) i = a.n - 1u;
    const uint32_t env = a.env_offset + i;
    const bool leader = valid && sub == 0;

    float x[E];
    const float *src = a.state + (size_t)i * S + (size_t)sub * E;
#pragma unroll
    for (int v = 0; v < E / 4; ++v) {
        const float4 f = *reinterpret_cast<const float4 *>(src + 4 * v);
        x[4 * v + 0] = f.x; x[4 * v + 1] = f.y; x[4 * v + 2] = f.z; x[4 * v + 3] = f.w;
    }
    uint32_t len = a.ep_len[i];
    uint32_t rc = a.reset_count[i];
    size_t row = i;

    const int nblk = (a.phase + a.K + 3) >> 2;
    for (int b = 0; b < nblk; ++b) {
        uint4 blk = make_uint4(0u, 0u, 0u, 0u);
        if (!a.actions) blk = philox(env, a.tb0 + (uint32_t)b, 0u, 0u, a.rk);
#pragma unroll 1
        for (int j = 0; j < 4; ++j) {
            const int k = 4 * b + j - a.phase;
            if (k < 0 || k >= a.K) continue;
            const uint32_t w = j == 0 ? blk.x : j == 1 ? blk.y : j == 2 ? blk.z : blk.w;

            if (a.out_obs && valid) {
                float *dst = a.out_obs + row * S + (size_t)sub * E;
#pragma unroll
                for (int v = 0; v < E / 4; ++v)
                    __stcs(reinterpret_cast<float4 *>(dst + 4 * v), make_float4(x[4 * v], x[4 * v + 1], x[4 * v + 2], x[4 * v + 3]));
            }

            const int act = a.actions ? (a.actions[i] != 0) : (int)(w >> 31);
            const float c = __fmul_rn(fbits(0x3A83126Fu), act ? 1.0f : -1.0f);

            // halo: first element of the next chunk of the same env (wrapping around)
            float halo;
            if (L == 1) {
                halo = x[0];
            } else {
                halo = __shfl_sync(0xFFFFFFFFu, x[0], (lane & ~(uint32_t)(LS - 1)) | ((lane + 1u) & (uint32_t)(LS - 1)));
                if (W > 1) {
                    if (lane == 0) sm_halo[warp] = x[0];
                    __syncthreads();
                    if (lane == 31) halo = sm_halo[(warp + 1u) % W];
                }
            }

            // Jacobi update: every right-hand side reads pre-step values
            float q[E];
#pragma unroll
            for (int e = 0; e < E; ++e) {
                const float right = e + 1 < E ? x[e + 1] : halo;
                const float z = sin_s(__fadd_rn(x[e], right));
                q[e] = __fadd_rn(__fmaf_rn(fbits(0x3C23D70Au), z, x[e]), c);
            }
#pragma unroll
            for (int e = 0; e < E; ++e) {
                x[e] = q[e];
                q[e] = __fmul_rn(q[e], q[e]);
            }
#pragma unroll
            for (int wdt = 1; wdt < E; wdt <<= 1)
#pragma unroll
                for (int e = 0; e < E; e += 2 * wdt) q[e] = __fadd_rn(q[e], q[e + wdt]);
            float sum = q[0];
#pragma unroll
            for (int m = 1; m < LS; m <<= 1) sum = __fadd_rn(sum, __shfl_xor_sync(0xFFFFFFFFu, sum, m));
            if (W > 1) {
                if (lane == 0) sm_sum[warp] = sum;
                __syncthreads();
                float part[W];
#pragma unroll
                for (int v = 0; v < W; ++v) part[v] = sm_sum[v];
#pragma unroll
                for (int wdt = 1; wdt < W; wdt <<= 1)
#pragma unroll
                    for (int v = 0; v < W; v += 2 * wdt) part[v] = __fadd_rn(part[v], part[v + wdt]);
                sum = part[0];
            }
            const bool done = __fmul_rn(sum, 1.0f / (float)S) > 4.0f;
            len += 1u;

            if (leader) {
                if (a.out_act) __stcs(&a.out_act[row], (int8_t)act);
                if (a.out_rew) __stcs(&a.out_rew[row], 1.0f);
                if (a.out_done) __stcs(&a.out_done[row], (uint8_t)done);
            }

            if (done) {                                     // uniform over the threads of one env
                rc += 1u;
#pragma unroll
                for (int v = 0; v < E / 4; ++v) {
                    const float4 f = draw_state4<ENV_SYNTH>(env, rc, sub * (uint32_t)(E / 4) + (uint32_t)v, a.rk);
                    x[4 * v + 0] = f.x; x[4 * v + 1] = f.y; x[4 * v + 2] = f.z; x[4 * v + 3] = f.w;
                }
                len = 0u;
            }
            row += a.n;
        }
    }

    if (valid) {
        float *dst = a.state + (size_t)i * S + (size_t)sub * E;
#pragma unroll
        for (int v = 0; v < E / 4; ++v)
            *reinterpret_cast<float4 *>(dst + 4 * v) = make_float4(x[4 * v], x[4 * v + 1], x[4 * v + 2], x[4 * v + 3]);
        if (a.next_obs) {
            float *nd = a.next_obs + (size_t)i * S + (size_t)sub * E;
#pragma unroll
            for (int v = 0; v < E / 4; ++v)
                *reinterpret_cast<float4 *>(nd + 4 * v) = make_float4(x[4 * v], x[4 * v + 1], x[4 * v + 2], x[4 * v + 3]);
        }
        if (sub == 0) { a.ep_len[i] = len; a.reset_count[i] = rc; }
    }
}

template <int S>
static cudaError_t launch_synth_t(const SynthArgs &a, cudaStream_t st)
{
    using Sh = SynthShape<S>;
    const uint32_t blocks = (a.n + Sh::ENVS_PER_CTA - 1u) / Sh::ENVS_PER_CTA;
    rollout_synth_kernel<S><<<blocks, Sh::THREADS, 0, st>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_synth(int S, const SynthArgs &a, cudaStream_t st)
{
    switch (S) {
    case 4: return launch_synth_t<4>(a, st);
    case 8: return launch_synth_t<8>(a, st);
    case 16: return launch_synth_t<16>(a, st);
    case 32: return launch_synth_t<32>(a, st);
    case 64: return launch_synth_t<64>(a, st);
    case 128: return launch_synth_t<128>(a, st);
    case 256: return launch_synth_t<256>(a, st);
    case 512: return launch_synth_t<512>(a, st);
    case 1024: return launch_synth_t<1024>(a, st);
    case 2048: return launch_synth_t<2048>(a, st);
    case 4096: return launch_synth_t<4096>(a, st);
    default: return cudaErrorInvalidValue;
    }
}

}  // namespace simk
