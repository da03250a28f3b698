// Per-environment dynamics, one env per call, state in registers (scalar reference forms;
// the packed two-env forms live beside the kernels that use them).
#pragma once
#include "sim_math.cuh"

namespace simk {

enum : int { ENV_CARTPOLE = 0, ENV_ACROBOT = 1, ENV_SYNTH = 2 };

// Reset distribution lo + width*u of each env kind.
template <int ENV> struct ResetRange;
template <> struct ResetRange<ENV_CARTPOLE> { static __device__ __forceinline__ float width() { return 0.1f; } static __device__ __forceinline__ float lo() { return -0.05f; } };
template <> struct ResetRange<ENV_ACROBOT>  { static __device__ __forceinline__ float width() { return 0.2f; } static __device__ __forceinline__ float lo() { return -0.1f; } };
template <> struct ResetRange<ENV_SYNTH>    { static __device__ __forceinline__ float width() { return 2.0f; } static __device__ __forceinline__ float lo() { return -1.0f; } };

// Four state elements 4j..4j+3 of draw number r of env `env`.
template <int ENV>
__device__ __forceinline__ float4 draw_state4(uint32_t env, uint32_t r, uint32_t j, const RoundKeys &rk)
{
    const uint4 b = philox(env, r, 1u, j, rk);
    const float w = ResetRange<ENV>::width(), lo = ResetRange<ENV>::lo();
    return make_float4(uniform_range(b.x, w, lo), uniform_range(b.y, w, lo), uniform_range(b.z, w, lo), uniform_range(b.w, w, lo));
}

// Categorical sample of the two-action policy from its logits l = (logit0, logit1) and one Philox word:
// inverse CDF over the two unnormalised softmax weights: action 0 iff u*(e0+e1) < e0.
__device__ __forceinline__ int sample_pair(f2 l, uint32_t w)
{
    const float m = fmaxf(lo(l), hi(l));
    const float y0 = fminf(fmaxf(__fsub_rn(lo(l), m), -87.0f), 88.0f);
    const float y1 = fminf(fmaxf(__fsub_rn(hi(l), m), -87.0f), 88.0f);
    const f2 e = exp2_core(pk(y0, y1));
    const float thr = __fmul_rn(uniform01(w), __fadd_rn(lo(e), hi(e)));
    return (thr < lo(e)) ? 0 : 1;
}

// CartPole: explicit Euler with tau = 0.02; state (x, x_dot, theta, theta_dot).
// Returns done; reward is 1 on every step.
__device__ __forceinline__ bool cartpole_step(float4 &s, bool push_right)
{
    float sn, cs;
    sincos_s(s.z, sn, cs);
    const float F = push_right ? 10.0f : -10.0f;
    const float w2 = __fmul_rn(s.w, s.w);
    const float u = __fmul_rn(fbits(0x3D4CCCCDu), w2);                     // m_p l theta_dot^2
    const float v = __fmaf_rn(u, sn, F);
    const float temp = __fmul_rn(v, fbits(0x3F68BA2Fu));                   // / (m_c + m_p)
    const float m = __fmul_rn(cs, temp);
    const float num = __fmaf_rn(fbits(0x411CCCCDu), sn, -m);               // g sin - cos*temp
    const float cc = __fmul_rn(cs, cs);
    const float e = __fmaf_rn(-fbits(0x3DBA2E8Cu), cc, fbits(0x3FAAAAABu)); // 4/3 - m_p cos^2/(m_c+m_p)
    const float den = __fmul_rn(0.5f, e);
    const float thacc = __fdiv_rn(num, den);
    const float g = __fmul_rn(fbits(0x3D3A2E8Cu), thacc);
    const float xacc = __fmaf_rn(-g, cs, temp);
    const float TAU = fbits(0x3CA3D70Au);
    const float nx = __fmaf_rn(TAU, s.y, s.x);
    const float nxd = __fmaf_rn(TAU, xacc, s.y);
    const float nth = __fmaf_rn(TAU, s.w, s.z);
    const float nthd = __fmaf_rn(TAU, thacc, s.w);
    s = make_float4(nx, nxd, nth, nthd);
    return (fabsf(nx) > fbits(0x4019999Au)) | (fabsf(nth) > fbits(0x3E567750u));
}

// Acrobot derivative (theta1, theta2, omega1, omega2) -> (omega1, omega2, acc1, acc2), torque a.
__device__ __forceinline__ float4 acrobot_dsdt(const float4 y, float a)
{
    float s2, c2;
    sincos_s(y.y, s2, c2);
    const float s1 = sin_s(y.x);
    const float s12 = sin_s(__fadd_rn(y.x, y.y));
    const float w1 = y.z, w2 = y.w;
    const float d1 = __fadd_rn(c2, 3.5f);
    const float d2 = __fmaf_rn(0.5f, c2, 1.25f);
    const float phi2 = __fmul_rn(4.9f, s12);
    const float h = __fmul_rn(0.5f, s2);
    const float t1 = __fmul_rn(w2, w2);
    const float t2 = __fmul_rn(w2, w1);
    float phi1 = __fmaf_rn(14.7f, s1, phi2);
    phi1 = __fmaf_rn(-h, t1, phi1);
    phi1 = __fmaf_rn(-s2, t2, phi1);
    const float r = __fdiv_rn(d2, d1);
    float num = __fmaf_rn(r, phi1, a);
    num = __fmaf_rn(-h, __fmul_rn(w1, w1), num);
    num = __fsub_rn(num, phi2);
    const float den = __fmaf_rn(-d2, r, 1.25f);
    const float dd2 = __fdiv_rn(num, den);
    const float dd1 = __fdiv_rn(-__fmaf_rn(d2, dd2, phi1), d1);
    return make_float4(w1, w2, dd1, dd2);
}

__device__ __forceinline__ float4 axpy4(float h, const float4 k, const float4 y)
{
    return make_float4(__fmaf_rn(h, k.x, y.x), __fmaf_rn(h, k.y, y.y), __fmaf_rn(h, k.z, y.z), __fmaf_rn(h, k.w, y.w));
}

__device__ __forceinline__ float rk4_combine(float y, float k1, float k2, float k3, float k4)
{
    float sm = __fadd_rn(k1, k4);
    const float m = __fadd_rn(k2, k3);
    sm = __fmaf_rn(2.0f, m, sm);
    return __fmaf_rn(fbits(0x3D088889u), sm, y);                            // dt/6
}

// Angle wrap into [-pi, pi] by repeated +-2pi.  One pass suffices for every state a step can
// produce; the pass count is bounded so that no input can spin the kernel.
__device__ __forceinline__ float wrap_pi(float th)
{
    const float PI = fbits(0x40490FDBu), TWO_PI = fbits(0x40C90FDBu);
    for (int it = 0; it < 8 && th > PI; ++it) th = __fsub_rn(th, TWO_PI);
    for (int it = 0; it < 8 && th < -PI; ++it) th = __fadd_rn(th, TWO_PI);
    return th;
}

// Acrobot: one RK4 step of 0.2 s, wrap, clip.  act in {0,1,2} -> torque act-1.  Returns the goal test.
__device__ __forceinline__ bool acrobot_step(float4 &s, int act)
{
    const float a = (float)(act - 1);
    const float H = fbits(0x3E4CCCCDu), H2 = fbits(0x3DCCCCCDu);
    const float4 k1 = acrobot_dsdt(s, a);
    const float4 k2 = acrobot_dsdt(axpy4(H2, k1, s), a);
    const float4 k3 = acrobot_dsdt(axpy4(H2, k2, s), a);
    const float4 k4 = acrobot_dsdt(axpy4(H, k3, s), a);
    float th1 = rk4_combine(s.x, k1.x, k2.x, k3.x, k4.x);
    float th2 = rk4_combine(s.y, k1.y, k2.y, k3.y, k4.y);
    float w1 = rk4_combine(s.z, k1.z, k2.z, k3.z, k4.z);
    float w2 = rk4_combine(s.w, k1.w, k2.w, k3.w, k4.w);
    th1 = wrap_pi(th1);
    th2 = wrap_pi(th2);
    const float W1M = fbits(0x41490FDBu), W2M = fbits(0x41E231D6u);
    w1 = fminf(fmaxf(w1, -W1M), W1M);
    w2 = fminf(fmaxf(w2, -W2M), W2M);
    s = make_float4(th1, th2, w1, w2);
    const float g = __fsub_rn(-cos_s(th1), cos_s(__fadd_rn(th1, th2)));
    return g > 1.0f;
}

}  // namespace simk
