// Fused CartPole rollout with the 4-64-64-2 tanh MLP policy evaluated inside the kernel, two envs
// per thread.
//
// The policy dominates (4480 fused multiply-adds and 128 tanh per env-step against ~50 flops of
// physics), so the kernel is organised around the FMA pipe:
//   * parameters are staged once per CTA into shared memory, each layer transposed so that the
//     weights of consecutive OUTPUT units for one input are adjacent: a 128-bit broadcast load
//     yields two (W[j][k], W[j+1][k]) pairs, and one packed fma advances two output units;
//   * the loaded weights are used for both envs of the thread (half the shared-memory traffic);
//   * every output unit is still one sequential fma chain over its inputs in ascending order,
//     starting from the bias, so the sums are bit-identical to the plain definition;
//   * tanh runs on packed pairs of adjacent units.
// Layer 3 is folded into the layer-2 loop: as soon as a block of eight hidden units is finished
// its tanh values are accumulated into the two logits, in ascending unit order.
#include "sim_internal.h"
#include "sim_envs.cuh"

namespace simk {

struct MlpSmem2 {
    float w1t[4 * 64];    // w1t[k*64 + j] = W1[j][k]
    float b1[64];
    float w2t[64 * 64];   // w2t[k*64 + j] = W2[j][k]
    float b2[64];
    float2 w3[64];        // w3[j] = (W3[0][j], W3[1][j])
    float2 b3;
};

__device__ __forceinline__ void stage_mlp2(const float *__restrict__ p, MlpSmem2 &s)
{
    const int tid = threadIdx.x, nt = blockDim.x;
    for (int i = tid; i < 256; i += nt) s.w1t[(i & 3) * 64 + (i >> 2)] = p[i];
    for (int i = tid; i < 64; i += nt) {
        s.b1[i] = p[256 + i];
        s.b2[i] = p[4416 + i];
        s.w3[i] = make_float2(p[4480 + i], p[4544 + i]);
    }
    for (int i = tid; i < 4096; i += nt) s.w2t[(i & 63) * 64 + (i >> 6)] = p[320 + i];
    if (tid == 0) s.b3 = make_float2(p[4608], p[4609]);
    __syncthreads();
}

#ifndef MLP_JB
#define MLP_JB 8
#endif
#ifndef MLP_MINBLOCKS
#define MLP_MINBLOCKS 2
#endif
constexpr int kJB = MLP_JB;        // hidden units of layer 2 advanced together (accumulators live in registers)

__device__ __forceinline__ const float4 &ld4(const float *p) { return *reinterpret_cast<const float4 *>(p); }

// Logits of two observations: la = (logit0, logit1) of obs A, lb of obs B.
__device__ __forceinline__ void mlp_logits2(const float4 oa, const float4 ob, const MlpSmem2 &s, f2 &la, f2 &lb)
{
    float ha[64], hb[64];
    {
        const f2 a0 = splat(oa.x), a1 = splat(oa.y), a2 = splat(oa.z), a3 = splat(oa.w);
        const f2 b0 = splat(ob.x), b1 = splat(ob.y), b2 = splat(ob.z), b3 = splat(ob.w);
#pragma unroll
        for (int j = 0; j < 64; j += 4) {
            const float4 bias = ld4(&s.b1[j]);
            const float4 w0 = ld4(&s.w1t[0 * 64 + j]), w1 = ld4(&s.w1t[1 * 64 + j]);
            const float4 w2 = ld4(&s.w1t[2 * 64 + j]), w3 = ld4(&s.w1t[3 * 64 + j]);
            f2 pa = pk(bias.x, bias.y), qa = pk(bias.z, bias.w), pb = pa, qb = qa;
            pa = fma2(pk(w0.x, w0.y), a0, pa); qa = fma2(pk(w0.z, w0.w), a0, qa);
            pb = fma2(pk(w0.x, w0.y), b0, pb); qb = fma2(pk(w0.z, w0.w), b0, qb);
            pa = fma2(pk(w1.x, w1.y), a1, pa); qa = fma2(pk(w1.z, w1.w), a1, qa);
            pb = fma2(pk(w1.x, w1.y), b1, pb); qb = fma2(pk(w1.z, w1.w), b1, qb);
            pa = fma2(pk(w2.x, w2.y), a2, pa); qa = fma2(pk(w2.z, w2.w), a2, qa);
            pb = fma2(pk(w2.x, w2.y), b2, pb); qb = fma2(pk(w2.z, w2.w), b2, qb);
            pa = fma2(pk(w3.x, w3.y), a3, pa); qa = fma2(pk(w3.z, w3.w), a3, qa);
            pb = fma2(pk(w3.x, w3.y), b3, pb); qb = fma2(pk(w3.z, w3.w), b3, qb);
            pa = tanh2(pa); qa = tanh2(qa); pb = tanh2(pb); qb = tanh2(qb);
            ha[j] = lo(pa); ha[j + 1] = hi(pa); ha[j + 2] = lo(qa); ha[j + 3] = hi(qa);
            hb[j] = lo(pb); hb[j + 1] = hi(pb); hb[j + 2] = lo(qb); hb[j + 3] = hi(qb);
        }
    }
    la = pk(s.b3.x, s.b3.y);
    lb = la;
#pragma unroll 1
    for (int jb = 0; jb < 64; jb += kJB) {
        f2 ca[kJB / 2], cb[kJB / 2];
#pragma unroll
        for (int v = 0; v < kJB / 4; ++v) {
            const float4 u = ld4(&s.b2[jb + 4 * v]);
            ca[2 * v] = pk(u.x, u.y); ca[2 * v + 1] = pk(u.z, u.w);
            cb[2 * v] = ca[2 * v]; cb[2 * v + 1] = ca[2 * v + 1];
        }
#pragma unroll
        for (int k = 0; k < 64; ++k) {
            const f2 da = splat(ha[k]), db = splat(hb[k]);
#pragma unroll
            for (int v = 0; v < kJB / 4; ++v) {
                const float4 u = ld4(&s.w2t[k * 64 + jb + 4 * v]);
                const f2 w0 = pk(u.x, u.y), w1 = pk(u.z, u.w);
                ca[2 * v] = fma2(w0, da, ca[2 * v]); ca[2 * v + 1] = fma2(w1, da, ca[2 * v + 1]);
                cb[2 * v] = fma2(w0, db, cb[2 * v]); cb[2 * v + 1] = fma2(w1, db, cb[2 * v + 1]);
            }
        }
#pragma unroll
        for (int i = 0; i < kJB / 2; ++i) {
            const f2 ta = tanh2(ca[i]), tb = tanh2(cb[i]);
            const float2 wl = s.w3[jb + 2 * i], wh = s.w3[jb + 2 * i + 1];
            la = fma2(pk(wl.x, wl.y), splat(lo(ta)), la);
            lb = fma2(pk(wl.x, wl.y), splat(lo(tb)), lb);
            la = fma2(pk(wh.x, wh.y), splat(hi(ta)), la);
            lb = fma2(pk(wh.x, wh.y), splat(hi(tb)), lb);
        }
    }
}

#ifndef MLP_THREADS
#define MLP_THREADS 128
#endif
constexpr int kMlp2Threads = MLP_THREADS;  // warps of 64 envs each

__global__ void __launch_bounds__(kMlp2Threads, MLP_MINBLOCKS)
rollout_cartpole_mlp_kernel(const __grid_constant__ S4Args a)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    MlpSmem2 &ms = *reinterpret_cast<MlpSmem2 *>(smem_raw);
    pdl_wait();                                          // parameters and state may come from the previous launch
    pdl_release();
    stage_mlp2(a.params, ms);

    const uint32_t lane = threadIdx.x & 31u;
    const uint64_t base64 = ((uint64_t)blockIdx.x * (kMlp2Threads / 32) + (threadIdx.x >> 5)) * 64u;  // may exceed 2^32 near the largest N
    if (base64 >= a.n) return;                           // whole warp beyond the batch
    const uint32_t base = (uint32_t)base64;
    uint32_t ia = base + lane, ib = base + 32u + lane;
    const bool va = base64 + lane < a.n, vb = base64 + 32u + lane < a.n;
    if (!va) ia = a.n - 1u;
    if (!vb) ib = a.n - 1u;
    const uint32_t env_a = a.env_offset + ia, env_b = a.env_offset + ib;

    float4 A = a.state[ia], B = a.state[ib];
    uint32_t len_a = a.ep_len[ia], len_b = a.ep_len[ib];
    uint32_t rc_a = a.reset_count[ia], rc_b = a.reset_count[ib];
    const bool sa_obs = a.out_obs && va, sb_obs = a.out_obs && vb, sa_act = a.out_act && va, sb_act = a.out_act && vb;
    const bool sa_rew = a.out_rew && va, sb_rew = a.out_rew && vb, sa_done = a.out_done && va, sb_done = a.out_done && vb;
    const size_t n = a.n;
    size_t row = (size_t)base + lane;

    const int nblk = (a.phase + a.K + 3) >> 2;
    for (int b = 0; b < nblk; ++b) {
        const uint4 ba = philox(env_a, a.tb0 + (uint32_t)b, 0u, 0u, a.rk);
        const uint4 bb = philox(env_b, a.tb0 + (uint32_t)b, 0u, 0u, a.rk);
#pragma unroll 1
        for (int j = 0; j < 4; ++j) {                    // not unrolled: one copy of the policy code
            const int k = 4 * b + j - a.phase;
            if (k < 0 || k >= a.K) continue;
            const uint32_t wa = j == 0 ? ba.x : j == 1 ? ba.y : j == 2 ? ba.z : ba.w;
            const uint32_t wb = j == 0 ? bb.x : j == 1 ? bb.y : j == 2 ? bb.z : bb.w;
            if (sa_obs) __stcs(a.out_obs + row, A);
            if (sb_obs) __stcs(a.out_obs + row + 32, B);
            f2 la, lb;
            mlp_logits2(A, B, ms, la, lb);
            const int act_a = sample_pair(la, wa), act_b = sample_pair(lb, wb);
            bool da = cartpole_step(A, act_a != 0);
            bool db = cartpole_step(B, act_b != 0);
            for (int c = 1; c < a.C; ++c) { da = cartpole_step(A, act_a != 0); db = cartpole_step(B, act_b != 0); }   // compute factor
            len_a += 1u; len_b += 1u;
            if (sa_act) __stcs(a.out_act + row, (int8_t)act_a);
            if (sb_act) __stcs(a.out_act + row + 32, (int8_t)act_b);
            if (sa_rew) __stcs(a.out_rew + row, 1.0f);
            if (sb_rew) __stcs(a.out_rew + row + 32, 1.0f);
            if (sa_done) __stcs(a.out_done + row, (uint8_t)da);
            if (sb_done) __stcs(a.out_done + row + 32, (uint8_t)db);
            if (da) { rc_a += 1u; A = draw_state4<ENV_CARTPOLE>(env_a, rc_a, 0u, a.rk); len_a = 0u; }
            if (db) { rc_b += 1u; B = draw_state4<ENV_CARTPOLE>(env_b, rc_b, 0u, a.rk); len_b = 0u; }
            row += n;
        }
    }
    if (va) { a.state[ia] = A; a.ep_len[ia] = len_a; a.reset_count[ia] = rc_a; }
    if (vb) { a.state[ib] = B; a.ep_len[ib] = len_b; a.reset_count[ib] = rc_b; }
}

__global__ void __launch_bounds__(kMlp2Threads, 2)
policy_logits2_kernel(const float4 *__restrict__ obs, int64_t M, const float *__restrict__ params, float2 *__restrict__ logits)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    MlpSmem2 &ms = *reinterpret_cast<MlpSmem2 *>(smem_raw);
    stage_mlp2(params, ms);
    const int64_t ia = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 2;
    if (ia >= M) return;
    const int64_t ib = ia + 1 < M ? ia + 1 : ia;
    f2 la, lb;
    mlp_logits2(obs[ia], obs[ib], ms, la, lb);
    logits[ia] = make_float2(lo(la), hi(la));
    if (ib != ia) logits[ib] = make_float2(lo(lb), hi(lb));
}

cudaError_t launch_cartpole_mlp(const S4Args &a, cudaStream_t st)
{
    const unsigned envs_per_cta = kMlp2Threads * 2;
    const unsigned blocks = (a.n + envs_per_cta - 1u) / envs_per_cta;
    return launch_overlapped(a.K <= kOverlapMaxK, rollout_cartpole_mlp_kernel, dim3(blocks), dim3(kMlp2Threads), sizeof(MlpSmem2), st, a);
}

cudaError_t launch_policy_logits(const float *obs, int64_t M, const float *params, float *logits, cudaStream_t st)
{
    if (M <= 0) return cudaSuccess;
    const int64_t per_cta = kMlp2Threads * 2;
    const int64_t blocks = (M + per_cta - 1) / per_cta;
    if (blocks > 0x7FFFFFFFll) return cudaErrorInvalidConfiguration;
    policy_logits2_kernel<<<(unsigned)blocks, kMlp2Threads, sizeof(MlpSmem2), st>>>(reinterpret_cast<const float4 *>(obs), M, params,
                                                                                   reinterpret_cast<float2 *>(logits));
    return cudaGetLastError();
}

}  // namespace simk
