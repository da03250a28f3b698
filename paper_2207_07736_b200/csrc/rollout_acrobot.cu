// Fused Acrobot rollout under the uniform random torque policy, two envs per thread.
//
// One RK4 step evaluates the two-link dynamics four times: 14 sin/cos evaluations and 12 divisions per
// env-step.  The two envs of a thread (lanes l and l+32 of a 64-env group, so that stores stay
// contiguous) run through all of it as the halves of packed fp32 pairs.  The divisions have
// well-conditioned denominators (d1 = 3.5 + cos in [2.5, 4.5], the reduced inertia in [0.56, 1.03]):
// a reciprocal refined by one Newton step is the correctly rounded one there (checked value by value
// on the device by the library's self-check), and quotient estimate + exact residual correction gives
// the IEEE quotient whenever the numerator's exponent is ordinary.  That condition, and whether any
// angle needs wrapping or any velocity clipping, is checked once per step by one warp vote; a step that
// fails it is redone by the plain scalar step, which assumes nothing.
#include "sim_internal.h"
#include "sim_envs.cuh"

namespace simk {

struct Y4 { f2 t1, t2, w1, w2; };      // (theta1, theta2, omega1, omega2) of two envs

__device__ __forceinline__ Y4 acrobot_dsdt2(const Y4 &y, f2 a, uint32_t &guard)
{
    f2 s2, ns2, c2;
    sincos2_full(y.t2, s2, ns2, c2);
    const f2 s1 = sin2(y.t1);
    const f2 s12 = sin2(add2(y.t1, y.t2));
    const f2 d1 = add2(c2, splat(3.5f));
    const f2 nd1 = fma2(c2, splat(-1.0f), splat(-3.5f));            // -d1, exactly
    const f2 d2 = fma2(splat(0.5f), c2, splat(1.25f));
    const f2 nd2 = fma2(splat(-0.5f), c2, splat(-1.25f));           // -d2, exactly
    const f2 phi2 = mul2(splat(4.9f), s12);
    const f2 nh = mul2(splat(-0.5f), s2);                           // -(0.5 sin theta2), exactly
    const f2 t1 = mul2(y.w2, y.w2);
    const f2 t2 = mul2(y.w2, y.w1);
    f2 phi1 = fma2(splat(14.7f), s1, phi2);
    phi1 = fma2(nh, t1, phi1);
    phi1 = fma2(ns2, t2, phi1);
    const f2 y1 = rcp2_refined(d1, nd1);
    const f2 r = div2_refined(d2, y1, nd1);                         // d2 in [0.75, 1.75]: always an ordinary numerator
    f2 num = fma2(r, phi1, a);
    num = fma2(nh, mul2(y.w1, y.w1), num);
    num = sub2(num, phi2);
    const f2 den = fma2(nd2, r, splat(1.25f));
    const f2 nden = fma2(d2, r, splat(-1.25f));                     // -den, exactly
    exponent_guard(num, guard);
    const f2 dd2 = div2_refined(num, rcp2_refined(den, nden), nden);
    const f2 X = fma2(d2, dd2, phi1);
    exponent_guard(X, guard);
    // dd1 = (-X)/d1 = X/(-d1): reciprocal of -d1 is -y1, and minus the divisor is d1
    const f2 ny1 = neg2(y1);
    const f2 q0 = mul2(X, ny1);
    const f2 dd1 = fma2(fma2(d1, q0, X), ny1, q0);
    Y4 k;
    k.t1 = y.w1; k.t2 = y.w2; k.w1 = dd1; k.w2 = dd2;
    return k;
}

__device__ __forceinline__ Y4 axpy(f2 h, const Y4 &k, const Y4 &y)
{
    Y4 o;
    o.t1 = fma2(h, k.t1, y.t1); o.t2 = fma2(h, k.t2, y.t2); o.w1 = fma2(h, k.w1, y.w1); o.w2 = fma2(h, k.w2, y.w2);
    return o;
}

__device__ __forceinline__ f2 rk4_combine2(f2 y, f2 k1, f2 k2, f2 k3, f2 k4)
{
    const f2 sm = fma2(splat(2.0f), add2(k2, k3), add2(k1, k4));
    return fma2(splat(fbits(0x3D088889u)), sm, y);
}

// The plain scalar step (general division, wrap, clip), kept out of line: it runs only when a step fails the vote.
__device__ __noinline__ bool acrobot_step_plain(float4 &s, int act, int C)
{
    bool goal = acrobot_step(s, act);
    for (int c = 1; c < C; ++c) goal = acrobot_step(s, act);
    return goal;
}

constexpr int kAcroThreads = 64;   // two warps = 128 envs per CTA

__global__ void __launch_bounds__(kAcroThreads)
rollout_acrobot_x2_kernel(const __grid_constant__ S4Args a)
{
    const uint32_t lane = threadIdx.x & 31u;
    const uint64_t base64 = ((uint64_t)blockIdx.x * (kAcroThreads / 32) + (threadIdx.x >> 5)) * 64u;   // may exceed 2^32 near the largest N
    if (base64 >= a.n) return;
    const uint32_t base = (uint32_t)base64;
    uint32_t ia = base + lane, ib = base + 32u + lane;
    const bool va = base64 + lane < a.n, vb = base64 + 32u + lane < a.n;   // tail envs: computed on a clamped index, never stored
    if (!va) ia = a.n - 1u;
    if (!vb) ib = a.n - 1u;
    const uint32_t env_a = a.env_offset + ia, env_b = a.env_offset + ib;
    pdl_wait();
    pdl_release();

    Y4 s;
    {
        const float4 A = a.state[ia], B = a.state[ib];
        s.t1 = pk(A.x, B.x); s.t2 = pk(A.y, B.y); s.w1 = pk(A.z, B.z); s.w2 = pk(A.w, B.w);
    }
    uint32_t len_a = a.ep_len[ia], len_b = a.ep_len[ib];
    uint32_t rc_a = a.reset_count[ia], rc_b = a.reset_count[ib];
    const bool sa_obs = a.out_obs && va, sb_obs = a.out_obs && vb, sa_act = a.out_act && va, sb_act = a.out_act && vb;
    const bool sa_rew = a.out_rew && va, sb_rew = a.out_rew && vb, sa_done = a.out_done && va, sb_done = a.out_done && vb;
    const size_t n = a.n;
    size_t row = (size_t)base + lane;

    const f2 H = splat(fbits(0x3E4CCCCDu)), H2 = splat(fbits(0x3DCCCCCDu));
    const float PI = fbits(0x40490FDBu), W1M = fbits(0x41490FDBu), W2M = fbits(0x41E231D6u);

    const int nblk = (a.phase + a.K + 3) >> 2;
    const PhiloxEnv pe_a = philox_prepare(env_a, a.rk), pe_b = philox_prepare(env_b, a.rk);
    for (int b = 0; b < nblk; ++b) {
        const uint4 ba = philox_action_block(pe_a, a.tb0 + (uint32_t)b, a.rk);
        const uint4 bb = philox_action_block(pe_b, a.tb0 + (uint32_t)b, a.rk);
#pragma unroll 1
        for (int j = 0; j < 4; ++j) {
            const int k = 4 * b + j - a.phase;
            if (k < 0 || k >= a.K) continue;
            const uint32_t wa = j == 0 ? ba.x : j == 1 ? ba.y : j == 2 ? ba.z : ba.w;
            const uint32_t wb = j == 0 ? bb.x : j == 1 ? bb.y : j == 2 ? bb.z : bb.w;
            const int act_a = (int)__umulhi(wa, 3u), act_b = (int)__umulhi(wb, 3u);

            float4 A = make_float4(lo(s.t1), lo(s.t2), lo(s.w1), lo(s.w2));
            float4 B = make_float4(hi(s.t1), hi(s.t2), hi(s.w1), hi(s.w2));
            if (sa_obs) __stcs(a.out_obs + row, A);
            if (sb_obs) __stcs(a.out_obs + row + 32, B);

            bool goal_a, goal_b;
            {
                const f2 tq = pk((float)(act_a - 1), (float)(act_b - 1));
                uint32_t guard = 0u;
                Y4 y = s;
                for (int c = 0; c < a.C; ++c) {                       // compute factor: C full RK4 steps
                    const Y4 k1 = acrobot_dsdt2(y, tq, guard);
                    const Y4 k2 = acrobot_dsdt2(axpy(H2, k1, y), tq, guard);
                    const Y4 k3 = acrobot_dsdt2(axpy(H2, k2, y), tq, guard);
                    const Y4 k4 = acrobot_dsdt2(axpy(H, k3, y), tq, guard);
                    Y4 o;
                    o.t1 = rk4_combine2(y.t1, k1.t1, k2.t1, k3.t1, k4.t1);
                    o.t2 = rk4_combine2(y.t2, k1.t2, k2.t2, k3.t2, k4.t2);
                    o.w1 = rk4_combine2(y.w1, k1.w1, k2.w1, k3.w1, k4.w1);
                    o.w2 = rk4_combine2(y.w2, k1.w2, k2.w2, k3.w2, k4.w2);
                    // does anything need the wrap or the clip?  (!(x <= m) also catches NaN)
                    const bool odd = !(fabsf(lo(o.t1)) <= PI) | !(fabsf(hi(o.t1)) <= PI) | !(fabsf(lo(o.t2)) <= PI) | !(fabsf(hi(o.t2)) <= PI) |
                                     !(fabsf(lo(o.w1)) <= W1M) | !(fabsf(hi(o.w1)) <= W1M) | !(fabsf(lo(o.w2)) <= W2M) | !(fabsf(hi(o.w2)) <= W2M);
                    if (odd) guard |= 0x40000000u;
                    y = o;
                    if (a.C > 1 && __any_sync(0xFFFFFFFFu, (guard >> 30) & 1u)) break;   // the plain path redoes the whole recorded step
                }
                if (__any_sync(0xFFFFFFFFu, (guard >> 30) & 1u)) {
                    // plain scalar path from the state before the step (general division, wrap, clip)
                    goal_a = acrobot_step_plain(A, act_a, a.C);
                    goal_b = acrobot_step_plain(B, act_b, a.C);
                    s.t1 = pk(A.x, B.x); s.t2 = pk(A.y, B.y); s.w1 = pk(A.z, B.z); s.w2 = pk(A.w, B.w);
                } else {
                    s = y;
                    const f2 c1 = cos2(s.t1);
                    const f2 c12 = cos2(add2(s.t1, s.t2));
                    const f2 g = sub2(neg2(c1), c12);
                    goal_a = lo(g) > 1.0f;
                    goal_b = hi(g) > 1.0f;
                }
            }
            len_a += 1u; len_b += 1u;
            const bool da = goal_a | (len_a >= 500u), db = goal_b | (len_b >= 500u);

            if (sa_act) __stcs(a.out_act + row, (int8_t)act_a);
            if (sb_act) __stcs(a.out_act + row + 32, (int8_t)act_b);
            if (sa_rew) __stcs(a.out_rew + row, goal_a ? 0.0f : -1.0f);
            if (sb_rew) __stcs(a.out_rew + row + 32, goal_b ? 0.0f : -1.0f);
            if (sa_done) __stcs(a.out_done + row, (uint8_t)da);
            if (sb_done) __stcs(a.out_done + row + 32, (uint8_t)db);

            if (__any_sync(0xFFFFFFFFu, da | db)) {
                if (da) { rc_a += 1u; const float4 r = draw_state4<ENV_ACROBOT>(env_a, rc_a, 0u, a.rk); s.t1 = pk(r.x, hi(s.t1)); s.t2 = pk(r.y, hi(s.t2)); s.w1 = pk(r.z, hi(s.w1)); s.w2 = pk(r.w, hi(s.w2)); len_a = 0u; }
                if (db) { rc_b += 1u; const float4 r = draw_state4<ENV_ACROBOT>(env_b, rc_b, 0u, a.rk); s.t1 = pk(lo(s.t1), r.x); s.t2 = pk(lo(s.t2), r.y); s.w1 = pk(lo(s.w1), r.z); s.w2 = pk(lo(s.w2), r.w); len_b = 0u; }
            }
            row += n;
        }
    }

    if (va) { a.state[ia] = make_float4(lo(s.t1), lo(s.t2), lo(s.w1), lo(s.w2)); a.ep_len[ia] = len_a; a.reset_count[ia] = rc_a; }
    if (vb) { a.state[ib] = make_float4(hi(s.t1), hi(s.t2), hi(s.w1), hi(s.w2)); a.ep_len[ib] = len_b; a.reset_count[ib] = rc_b; }
}

cudaError_t launch_acrobot_random(const S4Args &a, cudaStream_t st)
{
    const unsigned envs_per_cta = kAcroThreads * 2;
    const unsigned blocks = (a.n + envs_per_cta - 1u) / envs_per_cta;
    return launch_overlapped(a.K <= kOverlapMaxK, rollout_acrobot_x2_kernel, dim3(blocks), dim3(kAcroThreads), 0, st, a);
}

}  // namespace simk
