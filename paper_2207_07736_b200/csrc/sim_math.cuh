// Device arithmetic of the environment-stepping kernels (sm_100a).
//
// Every floating-point operation is written with an explicit round-to-nearest intrinsic
// (__fadd_rn, __fmul_rn, __fmaf_rn, __fdiv_rn, __frcp_rn) so that the compiler can neither
// contract nor reorder it: results are identical bit for bit on every launch shape and do
// not depend on compiler flags.  Elementary functions are fixed polynomial evaluations
// (no libm, no fast-math approximations).
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace simk {

__device__ __forceinline__ float fbits(uint32_t b) { return __uint_as_float(b); }

// ---------------------------------------------------------------------------------------------
// Philox4x32-10.  The ten round keys depend only on the seed, so the host expands them once and
// they arrive as kernel parameters (constant-bank operands of the xor instructions).
// ---------------------------------------------------------------------------------------------
struct RoundKeys { uint32_t k[10][2]; };

__device__ __forceinline__ uint4 philox(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, const RoundKeys &rk)
{
    constexpr uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        uint32_t hi0 = __umulhi(M0, c0), lo0 = M0 * c0;
        uint32_t hi1 = __umulhi(M1, c2), lo1 = M1 * c2;
        uint32_t n0 = hi1 ^ c1 ^ rk.k[r][0];
        uint32_t n2 = hi0 ^ c3 ^ rk.k[r][1];
        c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    }
    return make_uint4(c0, c1, c2, c3);
}

// The action blocks of one env have the counter (env, tb, 0, 0) with only tb changing, so everything in the
// first three rounds that depends on the env and the keys alone is computed once per env (three of the six
// multiplications of those rounds); philox_action_block(prepared, tb) == philox(env, tb, 0, 0).
struct PhiloxEnv { uint32_t a, b, c, g; };

__device__ __forceinline__ PhiloxEnv philox_prepare(uint32_t env, const RoundKeys &rk)
{
    constexpr uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
    const uint32_t e2 = __umulhi(M0, env) ^ rk.k[0][1], e3 = M0 * env;      // state after round 0: (tb ^ k00, 0, e2, e3)
    const uint32_t f0 = __umulhi(M1, e2) ^ rk.k[1][0], f1 = M1 * e2;        // after round 1: (f0, f1, hi(M0 x) ^ e3 ^ k11, lo(M0 x))
    PhiloxEnv p;
    p.a = e3 ^ rk.k[1][1];
    p.b = f1 ^ rk.k[2][0];
    p.c = __umulhi(M0, f0) ^ rk.k[2][1];
    p.g = M0 * f0;
    return p;
}

__device__ __forceinline__ uint4 philox_action_block(const PhiloxEnv &p, uint32_t tb, const RoundKeys &rk)
{
    constexpr uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
    const uint32_t x = tb ^ rk.k[0][0];
    uint32_t c2 = __umulhi(M0, x) ^ p.a, c3 = M0 * x;                        // round 1
    uint32_t c0 = __umulhi(M1, c2) ^ p.b, c1 = M1 * c2;                      // round 2
    c2 = c3 ^ p.c; c3 = p.g;
#pragma unroll
    for (int r = 3; r < 10; ++r) {
        uint32_t hi0 = __umulhi(M0, c0), lo0 = M0 * c0;
        uint32_t hi1 = __umulhi(M1, c2), lo1 = M1 * c2;
        uint32_t n0 = hi1 ^ c1 ^ rk.k[r][0];
        uint32_t n2 = hi0 ^ c3 ^ rk.k[r][1];
        c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    }
    return make_uint4(c0, c1, c2, c3);
}

// u in [0, 1 - 2^-24]: top 24 bits, exact.
__device__ __forceinline__ float uniform01(uint32_t w) { return __fmul_rn(__uint2float_rn(w >> 8), fbits(0x33800000u)); }

// lo + width*u with a single rounding.
__device__ __forceinline__ float uniform_range(uint32_t w, float width, float lo) { return __fmaf_rn(uniform01(w), width, lo); }

// ---------------------------------------------------------------------------------------------
// Round-to-nearest-even to an integer by adding 1.5*2^23: valid for |t| < 2^22.  `neg_k` is the
// negated integer (exact, and +0 when the integer is 0), `bits` carries the integer in its low
// mantissa bits (two's complement), so no float->int conversion instruction is needed.
// ---------------------------------------------------------------------------------------------
constexpr float kRoundMagic = 12582912.0f;

// sin and cos of x (|x| < 1e6): three-term Cody-Waite reduction by pi/2, degree-9 / degree-10
// Taylor polynomials with fused multiply-adds, quadrant fix-up by sign-bit arithmetic.
__device__ __forceinline__ void sincos_s(float x, float &sn, float &cs)
{
    const float t = __fmul_rn(x, fbits(0x3F22F983u));           // x * 2/pi
    const float nb = __fadd_rn(t, kRoundMagic);
    const float nk = __fsub_rn(kRoundMagic, nb);                 // -k
    const uint32_t q = __float_as_uint(nb);
    float r = __fmaf_rn(nk, fbits(0x3FC90FDBu), x);
    r = __fmaf_rn(nk, fbits(0xB33BBD2Eu), r);
    r = __fmaf_rn(nk, fbits(0xA6F72CEDu), r);
    const float r2 = __fmul_rn(r, r);
    float p = __fmaf_rn(fbits(0x3638EF1Du), r2, fbits(0xB9500D01u));
    p = __fmaf_rn(p, r2, fbits(0x3C088889u));
    p = __fmaf_rn(p, r2, fbits(0xBE2AAAABu));
    const float S = __fmaf_rn(p, __fmul_rn(r2, r), r);
    float c = __fmaf_rn(fbits(0xB493F27Eu), r2, fbits(0x37D00D01u));
    c = __fmaf_rn(c, r2, fbits(0xBAB60B61u));
    c = __fmaf_rn(c, r2, fbits(0x3D2AAAABu));
    c = __fmaf_rn(c, r2, -0.5f);
    const float C = __fmaf_rn(c, r2, 1.0f);
    const bool odd = q & 1u;
    const float a = odd ? C : S;
    const float b = odd ? S : C;
    sn = __uint_as_float(__float_as_uint(a) ^ ((q & 2u) << 30));
    cs = __uint_as_float(__float_as_uint(b) ^ (((q + 1u) & 2u) << 30));
}

__device__ __forceinline__ float sin_s(float x) { float s, c; sincos_s(x, s, c); return s; }
__device__ __forceinline__ float cos_s(float x) { float s, c; sincos_s(x, s, c); return c; }

// exp(y) for y already inside [-87, 88].
__device__ __forceinline__ float exp_core(float y)
{
    const float t = __fmul_rn(y, fbits(0x3FB8AA3Bu));           // y * log2(e)
    const float nb = __fadd_rn(t, kRoundMagic);
    const float nn = __fsub_rn(kRoundMagic, nb);                 // -n
    float r = __fmaf_rn(nn, fbits(0x3F317218u), y);
    r = __fmaf_rn(nn, fbits(0xB102E308u), r);
    float p = __fmaf_rn(fbits(0x39500D01u), r, fbits(0x3AB60B61u));
    p = __fmaf_rn(p, r, fbits(0x3C088889u));
    p = __fmaf_rn(p, r, fbits(0x3D2AAAABu));
    p = __fmaf_rn(p, r, fbits(0x3E2AAAABu));
    p = __fmaf_rn(p, r, 0.5f);
    p = __fmaf_rn(p, r, 1.0f);
    p = __fmaf_rn(p, r, 1.0f);
    const float scale = __uint_as_float((__float_as_uint(nb) << 23) + 0x3F800000u);   // 2^n
    return __fmul_rn(p, scale);
}

__device__ __forceinline__ float exp_s(float y) { return exp_core(fminf(fmaxf(y, -87.0f), 88.0f)); }

// tanh(x) = sign(x) * (1 - 2/(exp(2|x|)+1)), saturating to 1 above |x| = 9 (whatever exp_core
// returns for larger arguments is discarded by the select).
// 2/d is twice the correctly rounded reciprocal (scaling by two is exact), so the final
// subtraction is one fused multiply-add.
__device__ __forceinline__ float tanh_s(float x)
{
    const float a = fabsf(x);
    const float e = exp_core(__fadd_rn(a, a));                  // the clamp of exp is inactive for a <= 9
    const float d = __fadd_rn(e, 1.0f);
    float t = __fmaf_rn(-2.0f, __frcp_rn(d), 1.0f);
    t = (a > 9.0f) ? 1.0f : t;
    return copysignf(t, x);
}

// ---------------------------------------------------------------------------------------------
// Packed pairs of fp32 (Blackwell add/mul/fma.rn.f32x2): one instruction issues two IEEE
// operations, so two envs (or two state elements) advance per issue slot.  Each half is rounded
// exactly like the scalar intrinsic, so packed and scalar code give identical bits.
// ---------------------------------------------------------------------------------------------
struct f2 { unsigned long long v; };

__device__ __forceinline__ f2 pk(float a, float b) { f2 r; asm("mov.b64 %0, {%1, %2};" : "=l"(r.v) : "f"(a), "f"(b)); return r; }
__device__ __forceinline__ float lo(f2 a) { float x; [[maybe_unused]] float y; asm("mov.b64 {%0, %1}, %2;" : "=f"(x), "=f"(y) : "l"(a.v)); return x; }
__device__ __forceinline__ float hi(f2 a) { [[maybe_unused]] float x; float y; asm("mov.b64 {%0, %1}, %2;" : "=f"(x), "=f"(y) : "l"(a.v)); return y; }
__device__ __forceinline__ f2 splat(float c) { return pk(c, c); }
__device__ __forceinline__ f2 fma2(f2 a, f2 b, f2 c) { f2 r; asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r.v) : "l"(a.v), "l"(b.v), "l"(c.v)); return r; }
__device__ __forceinline__ f2 add2(f2 a, f2 b) { f2 r; asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r.v) : "l"(a.v), "l"(b.v)); return r; }
__device__ __forceinline__ f2 sub2(f2 a, f2 b) { f2 r; asm("sub.rn.f32x2 %0, %1, %2;" : "=l"(r.v) : "l"(a.v), "l"(b.v)); return r; }
__device__ __forceinline__ f2 mul2(f2 a, f2 b) { f2 r; asm("mul.rn.f32x2 %0, %1, %2;" : "=l"(r.v) : "l"(a.v), "l"(b.v)); return r; }


// Polynomial halves of sin/cos for two arguments at once (general quadrant): returns the two
// polynomial values and the quadrant words; the callers below pick what they need.
__device__ __forceinline__ void sincos_poly2(f2 x, f2 &S, f2 &C, uint32_t &qa, uint32_t &qb)
{
    const f2 magic = splat(kRoundMagic);
    const f2 t = mul2(x, splat(fbits(0x3F22F983u)));
    const f2 nb = add2(t, magic);
    const f2 nk = sub2(magic, nb);
    f2 r = fma2(nk, splat(fbits(0x3FC90FDBu)), x);
    r = fma2(nk, splat(fbits(0xB33BBD2Eu)), r);
    r = fma2(nk, splat(fbits(0xA6F72CEDu)), r);
    const f2 r2 = mul2(r, r);
    f2 p = fma2(splat(fbits(0x3638EF1Du)), r2, splat(fbits(0xB9500D01u)));
    p = fma2(p, r2, splat(fbits(0x3C088889u)));
    p = fma2(p, r2, splat(fbits(0xBE2AAAABu)));
    S = fma2(p, mul2(r2, r), r);
    f2 c = fma2(splat(fbits(0xB493F27Eu)), r2, splat(fbits(0x37D00D01u)));
    c = fma2(c, r2, splat(fbits(0xBAB60B61u)));
    c = fma2(c, r2, splat(fbits(0x3D2AAAABu)));
    c = fma2(c, r2, splat(-0.5f));
    C = fma2(c, r2, splat(1.0f));
    qa = __float_as_uint(lo(nb));
    qb = __float_as_uint(hi(nb));
}

// sin of two arguments: one select and one sign flip per element.
__device__ __forceinline__ f2 sin2(f2 x)
{
    f2 S, C; uint32_t qa, qb;
    sincos_poly2(x, S, C, qa, qb);
    const float sa = (qa & 1u) ? lo(C) : lo(S);
    const float sb = (qb & 1u) ? hi(C) : hi(S);
    return pk(__uint_as_float(__float_as_uint(sa) ^ ((qa << 30) & 0x80000000u)),
              __uint_as_float(__float_as_uint(sb) ^ ((qb << 30) & 0x80000000u)));
}

// cos of two arguments.
__device__ __forceinline__ f2 cos2(f2 x)
{
    f2 S, C; uint32_t qa, qb;
    sincos_poly2(x, S, C, qa, qb);
    const float ca = (qa & 1u) ? lo(S) : lo(C);
    const float cb = (qb & 1u) ? hi(S) : hi(C);
    return pk(__uint_as_float(__float_as_uint(ca) ^ (((qa + 1u) << 30) & 0x80000000u)),
              __uint_as_float(__float_as_uint(cb) ^ (((qb + 1u) << 30) & 0x80000000u)));
}

// sin and cos of two arguments, and the negated sin (one more xor per element).
__device__ __forceinline__ void sincos2_full(f2 x, f2 &sn, f2 &nsn, f2 &cs)
{
    f2 S, C; uint32_t qa, qb;
    sincos_poly2(x, S, C, qa, qb);
    const bool oa = qa & 1u, ob = qb & 1u;
    const uint32_t sa = __float_as_uint(oa ? lo(C) : lo(S)) ^ ((qa << 30) & 0x80000000u);
    const uint32_t sb = __float_as_uint(ob ? hi(C) : hi(S)) ^ ((qb << 30) & 0x80000000u);
    const float ca = oa ? lo(S) : lo(C), cb = ob ? hi(S) : hi(C);
    sn = pk(__uint_as_float(sa), __uint_as_float(sb));
    nsn = pk(__uint_as_float(sa ^ 0x80000000u), __uint_as_float(sb ^ 0x80000000u));
    cs = pk(__uint_as_float(__float_as_uint(ca) ^ (((qa + 1u) << 30) & 0x80000000u)),
            __uint_as_float(__float_as_uint(cb) ^ (((qb + 1u) << 30) & 0x80000000u)));
}

__device__ __forceinline__ f2 neg2(f2 a) { return pk(-lo(a), -hi(a)); }

__device__ __forceinline__ float rcp_approx(float x) { float r; asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x)); return r; }

// Correctly rounded reciprocals of two denominators that lie in a range for which the library's
// arithmetic self-check has verified, value by value, that one Newton step from the hardware
// approximation equals the IEEE reciprocal.  nd = -d.
__device__ __forceinline__ f2 rcp2_refined(f2 d, f2 nd)
{
    const f2 y0 = pk(rcp_approx(lo(d)), rcp_approx(hi(d)));
    return fma2(y0, fma2(nd, y0, splat(1.0f)), y0);
}

// IEEE quotients num/d given y = RN(1/d) and nd = -d: estimate, exact residual, correction.  Exact when the
// numerator's exponent lies in [2^-63, 2^65) (see exponent_guard) or the numerator needs no guard.
__device__ __forceinline__ f2 div2_refined(f2 num, f2 y, f2 nd)
{
    const f2 q0 = mul2(num, y);
    return fma2(fma2(nd, q0, num), y, q0);
}

// Accumulates into bit 30 of `acc` whether either half of v has its two top exponent bits equal, i.e.
// lies outside [2^-63, 2^65) (zero, tiny, huge, infinite or NaN).
__device__ __forceinline__ void exponent_guard(f2 v, uint32_t &acc)
{
    const uint32_t a = __float_as_uint(lo(v)), b = __float_as_uint(hi(v));
    acc |= ~(a ^ (a << 1)) | ~(b ^ (b << 1));
}

// exp of two arguments already inside [-87, 88] (same operations as exp_core, two at a time).
__device__ __forceinline__ f2 exp2_core(f2 y)
{
    const f2 magic = splat(kRoundMagic);
    const f2 t = mul2(y, splat(fbits(0x3FB8AA3Bu)));
    const f2 nb = add2(t, magic);
    const f2 nn = sub2(magic, nb);
    f2 r = fma2(nn, splat(fbits(0x3F317218u)), y);
    r = fma2(nn, splat(fbits(0xB102E308u)), r);
    f2 p = fma2(splat(fbits(0x39500D01u)), r, splat(fbits(0x3AB60B61u)));
    p = fma2(p, r, splat(fbits(0x3C088889u)));
    p = fma2(p, r, splat(fbits(0x3D2AAAABu)));
    p = fma2(p, r, splat(fbits(0x3E2AAAABu)));
    p = fma2(p, r, splat(0.5f));
    p = fma2(p, r, splat(1.0f));
    p = fma2(p, r, splat(1.0f));
    const f2 scale = pk(__uint_as_float((__float_as_uint(lo(nb)) << 23) + 0x3F800000u),
                        __uint_as_float((__float_as_uint(hi(nb)) << 23) + 0x3F800000u));
    return mul2(p, scale);
}

// exp of two arguments in [0, 88] whose reduced exponent n is >= 0: p * 2^n is formed by adding n to the
// exponent field of p (p lies in [0.7, 1.42], so the sum stays a normal number and equals the product
// exactly); this frees one FMA-pipe slot per pair.
__device__ __forceinline__ f2 exp2_nonneg(f2 y)
{
    const f2 magic = splat(kRoundMagic);
    const f2 t = mul2(y, splat(fbits(0x3FB8AA3Bu)));
    const f2 nb = add2(t, magic);
    const f2 nn = sub2(magic, nb);
    f2 r = fma2(nn, splat(fbits(0x3F317218u)), y);
    r = fma2(nn, splat(fbits(0xB102E308u)), r);
    f2 p = fma2(splat(fbits(0x39500D01u)), r, splat(fbits(0x3AB60B61u)));
    p = fma2(p, r, splat(fbits(0x3C088889u)));
    p = fma2(p, r, splat(fbits(0x3D2AAAABu)));
    p = fma2(p, r, splat(fbits(0x3E2AAAABu)));
    p = fma2(p, r, splat(0.5f));
    p = fma2(p, r, splat(1.0f));
    p = fma2(p, r, splat(1.0f));
    return pk(__uint_as_float(__float_as_uint(lo(p)) + (__float_as_uint(lo(nb)) << 23)),
              __uint_as_float(__float_as_uint(hi(p)) + (__float_as_uint(hi(nb)) << 23)));
}

// tanh of two arguments.  d = exp(2|x|) + 1 lies in [2, 2^27) whenever the result is used, where one
// Newton step from the hardware reciprocal is the correctly rounded reciprocal (checked exhaustively
// on the device by the library's arithmetic self-check), so 1 - 2/d is one more fused multiply-add.
// Sign flips and the 2^n scaling run on the integer pipe; the FMA pipe is the one this kernel fills.
__device__ __forceinline__ f2 tanh2(f2 x)
{
    const float xa = lo(x), xb = hi(x);
    const float aa = fabsf(xa), ab = fabsf(xb);
    const f2 a = pk(aa, ab);                                        // above 9 whatever comes out is replaced below
    const f2 e = exp2_nonneg(add2(a, a));
    const f2 d = add2(e, splat(1.0f));
    const f2 nd = pk(-lo(d), -hi(d));
    const f2 y0 = pk(rcp_approx(lo(d)), rcp_approx(hi(d)));
    const f2 y1 = fma2(y0, fma2(nd, y0, splat(1.0f)), y0);
    const f2 t = fma2(splat(-2.0f), y1, splat(1.0f));
    const float ta = aa > 9.0f ? 1.0f : lo(t);
    const float tb = ab > 9.0f ? 1.0f : hi(t);
    return pk(copysignf(ta, xa), copysignf(tb, xb));
}

}  // namespace simk
