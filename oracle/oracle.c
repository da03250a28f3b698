/*
 * CPU oracle for batched environment stepping (test infrastructure, NOT product code).
 *
 * Only the tests, the smoke check and the bench's CPU-baseline / reference legs may call
 * this file.  It shares no code, header, table or constant generator with the CUDA path;
 * both were written independently from the same mathematical statement of the method.
 *
 * What it computes: N independent environments advanced T steps, one after the other, on
 * host arrays, single-threaded, with no notion of K (kernel fusion changes where the
 * simulator state lives, never what is computed -- paper Section 4.1, "Simulator kernel
 * fusion throughput"; the N x S state matrix and the step() transition are Section 3.2).
 *
 * Arithmetic: IEEE-754 binary32, round-to-nearest-even, no flush-to-zero, no contraction
 * except where fmaf() is written, '/' correctly rounded, evaluation order as written.
 * Compile with  gcc -O2 -ffp-contract=off  (never -ffast-math).
 *
 * Parity pins (tests/test_oracle_*.py): Philox known-answer vectors; sin/cos/exp/tanh
 * against double libm; CartPole and Acrobot accelerations against an independent
 * mass-matrix linear solve, closed forms at rest, mirror symmetry and the energy
 * balance; Acrobot RK4 against a tight-tolerance adaptive integrator; the synthetic
 * update against hand cases and rotation equivariance; the MLP against a float64
 * matmul and the zero-parameter reduction to the random policy; whole-pipeline
 * bookkeeping invariants.  No function here is "parity unpinned".
 */
#include <math.h>
#include <stdint.h>
#include <stddef.h>
#include <string.h>

#define ORACLE_API __attribute__((visibility("default")))

enum { ENV_CARTPOLE = 0, ENV_ACROBOT = 1, ENV_SYNTH = 2 };

static float f32_from_bits(uint32_t b) { float f; memcpy(&f, &b, 4); return f; }

/* ------------------------------------------------------------------------------------
 * Philox4x32-10 (Salmon, Moraes, Dror, Shaw 2011).  The paper names no generator; the
 * task statement fixes a counter-based Philox keyed per (seed, env, step).
 * ---------------------------------------------------------------------------------- */
ORACLE_API void oracle_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    const uint64_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u;
    const uint32_t W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        if (round > 0) { k0 += W0; k1 += W1; }          /* nine key bumps in total */
        uint64_t p0 = M0 * (uint64_t)c0;
        uint64_t p1 = M1 * (uint64_t)c2;
        uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
        uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

static void seed_key(uint64_t seed, uint32_t key[2])
{
    key[0] = (uint32_t)(seed & 0xFFFFFFFFu);
    key[1] = (uint32_t)(seed >> 32);
}

/* Action word for (env, t): word (t mod 4) of the block with counter (env, t div 4, 0, 0). */
ORACLE_API uint32_t oracle_action_word(uint64_t seed, uint32_t env, uint64_t t)
{
    uint32_t key[2], ctr[4], blk[4];
    seed_key(seed, key);
    ctr[0] = env; ctr[1] = (uint32_t)(t >> 2); ctr[2] = 0; ctr[3] = 0;
    oracle_philox4x32_10(ctr, key, blk);
    return blk[t & 3];
}

/* Bit-sliced action stream (an optional variant for two-action envs): the action of (env, t) is bit
 * (t mod 128) of the 128-bit block with counter (env, c, 2, 0), c = (low 32 bits of t div 4) div 32;
 * bit b lives in word b div 32 at position b mod 32 (least significant first). */
ORACLE_API int oracle_action_bit(uint64_t seed, uint32_t env, uint64_t t)
{
    uint32_t key[2], ctr[4], blk[4];
    seed_key(seed, key);
    uint32_t tb = (uint32_t)(t >> 2);
    ctr[0] = env; ctr[1] = tb >> 5; ctr[2] = 2; ctr[3] = 0;
    oracle_philox4x32_10(ctr, key, blk);
    uint32_t b = (uint32_t)(t & 127);
    return (int)((blk[b >> 5] >> (b & 31)) & 1u);
}

/* u = (top 24 bits of w) * 2^-24, exact in binary32, in [0, 1 - 2^-24]. */
ORACLE_API float oracle_uniform01(uint32_t w)
{
    return (float)(w >> 8) * f32_from_bits(0x33800000u);
}

/* Random action index: top bit (two actions) or multiply-shift by 3 (three actions). */
ORACLE_API int oracle_random_action(int env_kind, uint32_t w)
{
    if (env_kind == ENV_ACROBOT) return (int)(((uint64_t)w * 3u) >> 32);
    return (int)(w >> 31);
}

/* State draw number r of one env: element 4j+i is word i of the block with counter
 * (env, r, 1, j), mapped to lo + width*u with one fused multiply-add. */
ORACLE_API void oracle_draw_state(int env_kind, int S, uint64_t seed, uint32_t env, uint32_t r, float *out)
{
    float width, lo;
    if (env_kind == ENV_CARTPOLE)      { width = 0.1f; lo = -0.05f; }
    else if (env_kind == ENV_ACROBOT)  { width = 0.2f; lo = -0.1f; }
    else                               { width = 2.0f; lo = -1.0f; }
    uint32_t key[2];
    seed_key(seed, key);
    for (int j = 0; j < S / 4; ++j) {
        uint32_t ctr[4] = { env, r, 1u, (uint32_t)j }, blk[4];
        oracle_philox4x32_10(ctr, key, blk);
        for (int i = 0; i < 4; ++i)
            out[4 * j + i] = fmaf(oracle_uniform01(blk[i]), width, lo);
    }
}

/* ------------------------------------------------------------------------------------
 * Elementary functions fixed by the build's reading of the method, so that two
 * independent implementations can agree bit for bit (libm is not used).
 * ---------------------------------------------------------------------------------- */
ORACLE_API void oracle_sincos_s(float x, float *sn, float *cs)
{
    const float TWO_OVER_PI = f32_from_bits(0x3F22F983u);
    const float P1 = f32_from_bits(0x3FC90FDBu);   /*  1.5707964     */
    const float P2 = f32_from_bits(0xB33BBD2Eu);   /* -4.371139e-8   */
    const float P3 = f32_from_bits(0xA6F72CEDu);   /* -1.7151245e-15 */
    const float s1 = f32_from_bits(0xBE2AAAABu), s2 = f32_from_bits(0x3C088889u);
    const float s3 = f32_from_bits(0xB9500D01u), s4 = f32_from_bits(0x3638EF1Du);
    const float c2 = f32_from_bits(0x3D2AAAABu), c3 = f32_from_bits(0xBAB60B61u);
    const float c4 = f32_from_bits(0x37D00D01u), c5 = f32_from_bits(0xB493F27Eu);

    float t = x * TWO_OVER_PI;
    float k = rintf(t);                            /* round-half-even under the default mode */
    float r = fmaf(-k, P1, x);
    r = fmaf(-k, P2, r);
    r = fmaf(-k, P3, r);
    float r2 = r * r;

    float p = fmaf(s4, r2, s3);
    p = fmaf(p, r2, s2);
    p = fmaf(p, r2, s1);
    float r3 = r2 * r;
    float S = fmaf(p, r3, r);

    float q = fmaf(c5, r2, c4);
    q = fmaf(q, r2, c3);
    q = fmaf(q, r2, c2);
    q = fmaf(q, r2, -0.5f);
    float C = fmaf(q, r2, 1.0f);

    switch (((int)k) & 3) {
    case 0:  *sn = S;  *cs = C;  break;
    case 1:  *sn = C;  *cs = -S; break;
    case 2:  *sn = -S; *cs = -C; break;
    default: *sn = -C; *cs = S;  break;
    }
}

ORACLE_API float oracle_sin_s(float x) { float s, c; oracle_sincos_s(x, &s, &c); return s; }
ORACLE_API float oracle_cos_s(float x) { float s, c; oracle_sincos_s(x, &s, &c); return c; }

ORACLE_API float oracle_exp_s(float y)
{
    const float LOG2E  = f32_from_bits(0x3FB8AA3Bu);
    const float LN2_HI = f32_from_bits(0x3F317218u);
    const float LN2_LO = f32_from_bits(0xB102E308u);
    y = fminf(fmaxf(y, -87.0f), 88.0f);
    float n = rintf(y * LOG2E);
    float r = fmaf(-n, LN2_HI, y);
    r = fmaf(-n, LN2_LO, r);
    float p = f32_from_bits(0x39500D01u);          /* 1/5040 */
    p = fmaf(p, r, f32_from_bits(0x3AB60B61u));    /* 1/720  */
    p = fmaf(p, r, f32_from_bits(0x3C088889u));    /* 1/120  */
    p = fmaf(p, r, f32_from_bits(0x3D2AAAABu));    /* 1/24   */
    p = fmaf(p, r, f32_from_bits(0x3E2AAAABu));    /* 1/6    */
    p = fmaf(p, r, 0.5f);
    p = fmaf(p, r, 1.0f);
    p = fmaf(p, r, 1.0f);
    uint32_t sb = (uint32_t)((int)n + 127) << 23;
    return p * f32_from_bits(sb);
}

ORACLE_API float oracle_tanh_s(float x)
{
    float a = fabsf(x);
    float t;
    if (a > 9.0f) {
        t = 1.0f;
    } else {
        float e = oracle_exp_s(a + a);
        t = 1.0f - 2.0f / (e + 1.0f);
    }
    return copysignf(t, x);
}

/* Elementwise maps for the accuracy tests: which = 0 sin, 1 cos, 2 exp, 3 tanh. */
ORACLE_API void oracle_map_f32(int which, const float *x, int64_t n, float *out)
{
    for (int64_t i = 0; i < n; ++i) {
        switch (which) {
        case 0:  out[i] = oracle_sin_s(x[i]);  break;
        case 1:  out[i] = oracle_cos_s(x[i]);  break;
        case 2:  out[i] = oracle_exp_s(x[i]);  break;
        default: out[i] = oracle_tanh_s(x[i]); break;
        }
    }
}

/* ------------------------------------------------------------------------------------
 * CartPole, explicit Euler, tau = 0.02 (the paper's S = 4 simulator, Section 2.2;
 * equations of motion are the textbook cart-pole the benchmark spec names).
 * State order (x, x_dot, theta, theta_dot); act 0 pushes with -10 N, anything else +10 N.
 * ---------------------------------------------------------------------------------- */
ORACLE_API void oracle_cartpole_accel(const float s[4], int act, float *temp_out, float *thacc_out, float *xacc_out)
{
    const float GRAV = f32_from_bits(0x411CCCCDu);         /* 9.8        */
    const float INV_TOTAL = f32_from_bits(0x3F68BA2Fu);    /* 1/1.1      */
    const float MPT = f32_from_bits(0x3DBA2E8Cu);          /* 0.1/1.1    */
    const float PML = f32_from_bits(0x3D4CCCCDu);          /* 0.05       */
    const float PMLT = f32_from_bits(0x3D3A2E8Cu);         /* 0.05/1.1   */
    const float FOUR_THIRDS = f32_from_bits(0x3FAAAAABu);
    float th = s[2], thd = s[3];
    float sn, cs;
    oracle_sincos_s(th, &sn, &cs);
    float F = act ? 10.0f : -10.0f;
    float w2 = thd * thd;
    float u = PML * w2;
    float v = fmaf(u, sn, F);
    float temp = v * INV_TOTAL;
    float m = cs * temp;
    float num = fmaf(GRAV, sn, -m);
    float cc = cs * cs;
    float e = fmaf(-MPT, cc, FOUR_THIRDS);
    float den = 0.5f * e;
    float thacc = num / den;
    float g = PMLT * thacc;
    float xacc = fmaf(-g, cs, temp);
    *temp_out = temp; *thacc_out = thacc; *xacc_out = xacc;
}

/* Returns done (0/1); reward is 1.0f on every executed step. */
ORACLE_API int oracle_cartpole_step(const float s[4], int act, float out[4])
{
    const float TAU = f32_from_bits(0x3CA3D70Au);          /* 0.02 */
    const float X_TH = f32_from_bits(0x4019999Au);         /* 2.4 */
    const float TH_TH = f32_from_bits(0x3E567750u);        /* 12 degrees in radians */
    float temp, thacc, xacc;
    oracle_cartpole_accel(s, act, &temp, &thacc, &xacc);
    float x = s[0], xd = s[1], th = s[2], thd = s[3];
    float nx  = fmaf(TAU, xd, x);
    float nxd = fmaf(TAU, xacc, xd);
    float nth = fmaf(TAU, thd, th);
    float nthd = fmaf(TAU, thacc, thd);
    out[0] = nx; out[1] = nxd; out[2] = nth; out[3] = nthd;
    return (nx < -X_TH) | (nx > X_TH) | (nth < -TH_TH) | (nth > TH_TH);
}

/* ------------------------------------------------------------------------------------
 * Acrobot, RK4 with dt = 0.2 (task statement, config 4; the energy-conserving "book"
 * Lagrangian of the two-link pendulum).  State (theta1, theta2, omega1, omega2).
 * ---------------------------------------------------------------------------------- */
ORACLE_API void oracle_acrobot_dsdt(const float y[4], float a, float out[4])
{
    float th1 = y[0], th2 = y[1], w1 = y[2], w2 = y[3];
    float s2, c2, s1, s12, dummy;
    oracle_sincos_s(th2, &s2, &c2);
    oracle_sincos_s(th1, &s1, &dummy);
    oracle_sincos_s(th1 + th2, &s12, &dummy);
    float d1 = c2 + 3.5f;
    float d2 = fmaf(0.5f, c2, 1.25f);
    float phi2 = 4.9f * s12;
    float h = 0.5f * s2;
    float t1 = w2 * w2;
    float t2 = w2 * w1;
    float phi1 = fmaf(14.7f, s1, phi2);
    phi1 = fmaf(-h, t1, phi1);
    phi1 = fmaf(-s2, t2, phi1);
    float r = d2 / d1;
    float num = fmaf(r, phi1, a);
    num = fmaf(-h, w1 * w1, num);
    num = num - phi2;
    float den = fmaf(-d2, r, 1.25f);
    float dd2 = num / den;
    float dd1 = -(fmaf(d2, dd2, phi1)) / d1;
    out[0] = w1; out[1] = w2; out[2] = dd1; out[3] = dd2;
}

/* One RK4 step + wrap + clip.  act in {0,1,2} -> torque act-1 (clamped).  Returns the goal test. */
ORACLE_API int oracle_acrobot_step(const float s[4], int act, float out[4])
{
    const float H  = f32_from_bits(0x3E4CCCCDu);   /* 0.2   */
    const float H2 = f32_from_bits(0x3DCCCCCDu);   /* 0.1   */
    const float H6 = f32_from_bits(0x3D088889u);   /* 0.2/6 */
    const float PI = f32_from_bits(0x40490FDBu), TWO_PI = f32_from_bits(0x40C90FDBu);
    const float W1_MAX = f32_from_bits(0x41490FDBu);   /* 4 pi */
    const float W2_MAX = f32_from_bits(0x41E231D6u);   /* 9 pi */
    if (act < 0) act = 0;
    if (act > 2) act = 2;
    float a = (float)(act - 1);
    float k1[4], k2[4], k3[4], k4[4], y[4];
    oracle_acrobot_dsdt(s, a, k1);
    for (int i = 0; i < 4; ++i) y[i] = fmaf(H2, k1[i], s[i]);
    oracle_acrobot_dsdt(y, a, k2);
    for (int i = 0; i < 4; ++i) y[i] = fmaf(H2, k2[i], s[i]);
    oracle_acrobot_dsdt(y, a, k3);
    for (int i = 0; i < 4; ++i) y[i] = fmaf(H, k3[i], s[i]);
    oracle_acrobot_dsdt(y, a, k4);
    for (int i = 0; i < 4; ++i) {
        float sm = k1[i] + k4[i];
        float m = k2[i] + k3[i];
        sm = fmaf(2.0f, m, sm);
        out[i] = fmaf(H6, sm, s[i]);
    }
    for (int i = 0; i < 2; ++i) {
        while (out[i] > PI) out[i] -= TWO_PI;
        while (out[i] < -PI) out[i] += TWO_PI;
    }
    out[2] = fminf(fmaxf(out[2], -W1_MAX), W1_MAX);
    out[3] = fminf(fmaxf(out[3], -W2_MAX), W2_MAX);
    float g = (-oracle_cos_s(out[0])) - oracle_cos_s(out[0] + out[1]);
    return g > 1.0f;
}

/* Gym-style six-value observation of an Acrobot state: (cos t1, sin t1, cos t2, sin t2, w1, w2). */
ORACLE_API void oracle_acrobot_observation(const float s[4], float out[6])
{
    oracle_sincos_s(s[0], &out[1], &out[0]);
    oracle_sincos_s(s[1], &out[3], &out[2]);
    out[4] = s[2];
    out[5] = s[3];
}

/* ------------------------------------------------------------------------------------
 * Synthetic S-float simulator (the paper's "state factor" knob of Section 4.2, with the
 * per-element update the benchmark spec gives).  Jacobi update: every right-hand side
 * uses pre-step values.  act 0 -> a = -1, anything else -> a = +1.
 * ---------------------------------------------------------------------------------- */
static float pairwise_sum(const float *q, int lo, int hi)
{
    if (hi - lo == 1) return q[lo];
    int mid = lo + (hi - lo) / 2;
    return pairwise_sum(q, lo, mid) + pairwise_sum(q, mid, hi);
}

/* The reduction order on its own (adjacent pairs first), exported so a test can pin it. */
ORACLE_API float oracle_pairwise_sum(const float *q, int S) { return pairwise_sum(q, 0, S); }

/* `scratch` holds S floats.  Returns done. */
ORACLE_API int oracle_synth_step(const float *x, int S, int act, float *out, float *scratch)
{
    const float C001 = f32_from_bits(0x3A83126Fu);   /* 0.001 */
    const float C01  = f32_from_bits(0x3C23D70Au);   /* 0.01  */
    float a = act ? 1.0f : -1.0f;
    float c = C001 * a;
    for (int i = 0; i < S; ++i) {
        float y = x[i] + x[(i + 1) % S];
        float z = oracle_sin_s(y);
        float w = fmaf(C01, z, x[i]);
        out[i] = w + c;
    }
    for (int i = 0; i < S; ++i) scratch[i] = out[i] * out[i];
    float sum = pairwise_sum(scratch, 0, S);
    float mean = sum * (1.0f / (float)S);            /* S is a power of two: exact scaling */
    return mean > 4.0f;
}

/* ------------------------------------------------------------------------------------
 * MLP policy 4 -> 64 -> 64 -> 2 with tanh hidden layers (task statement, config 3; the
 * paper leaves inference/simulation fusion as future work, Section 7).
 * params = W1[64][4], b1[64], W2[64][64], b2[64], W3[2][64], b3[2]  ([out][in] rows).
 * ---------------------------------------------------------------------------------- */
ORACLE_API void oracle_mlp_logits(const float *params, const float obs[4], float logits[2])
{
    const float *W1 = params, *b1 = W1 + 256, *W2 = b1 + 64, *b2 = W2 + 4096, *W3 = b2 + 64, *b3 = W3 + 128;
    float h1[64], h2[64];
    for (int j = 0; j < 64; ++j) {
        float acc = b1[j];
        for (int k = 0; k < 4; ++k) acc = fmaf(W1[j * 4 + k], obs[k], acc);
        h1[j] = oracle_tanh_s(acc);
    }
    for (int j = 0; j < 64; ++j) {
        float acc = b2[j];
        for (int k = 0; k < 64; ++k) acc = fmaf(W2[j * 64 + k], h1[k], acc);
        h2[j] = oracle_tanh_s(acc);
    }
    for (int i = 0; i < 2; ++i) {
        float acc = b3[i];
        for (int j = 0; j < 64; ++j) acc = fmaf(W3[i * 64 + j], h2[j], acc);
        logits[i] = acc;
    }
}

/* Inverse-CDF categorical sample over two unnormalised softmax weights. */
ORACLE_API int oracle_sample_action(const float logits[2], uint32_t w)
{
    float m = fmaxf(logits[0], logits[1]);
    float e0 = oracle_exp_s(logits[0] - m);
    float e1 = oracle_exp_s(logits[1] - m);
    float Z = e0 + e1;
    float thr = oracle_uniform01(w) * Z;
    return (thr < e0) ? 0 : 1;
}

/* ------------------------------------------------------------------------------------
 * Whole pipeline for an arbitrary list of global env indices.
 *
 * For each listed env, for t = t0 .. t0+T-1:
 *   record obs[t] = state;  pick the action (given / MLP / random);  step;  record
 *   act, rew, done;  on done: reset_count += 1, state = draw #reset_count, ep_len = 0.
 *
 * state [n_sel,S], ep_len [n_sel], reset_count [n_sel] are read and updated in place.
 * given_actions, if not NULL, is [T,n_sel] and overrides the policy.
 * Outputs are [T,n_sel,S], [T,n_sel], [T,n_sel], [T,n_sel]; each may be NULL.
 * next_obs, if not NULL, is [T,n_sel,S]: the state after step t and after auto-reset.
 * Returns 0, or -1 on bad arguments.
 * ---------------------------------------------------------------------------------- */
ORACLE_API int oracle_rollout_x(int env_kind, int S, uint64_t seed, int compute_factor, int action_stream,
                              int64_t n_sel, const uint32_t *env_ids,
                              float *state, uint32_t *ep_len, uint32_t *reset_count,
                              uint64_t t0, int T,
                              const float *policy_params, const int8_t *given_actions,
                              float *out_obs, int8_t *out_act, float *out_rew, uint8_t *out_done,
                              float *next_obs)
{
    if (env_kind < 0 || env_kind > 2 || S < 4 || S > 4096 || (S & (S - 1)) || T < 0 || n_sel < 0) return -1;
    if (env_kind != ENV_SYNTH && S != 4) return -1;
    if (policy_params && env_kind != ENV_CARTPOLE) return -1;
    if (compute_factor < 1) return -1;
    if (action_stream != 0 && (action_stream != 1 || env_kind != ENV_CARTPOLE || policy_params)) return -1;
    float cur[4096], nxt[4096], scratch[4096];
    for (int64_t e = 0; e < n_sel; ++e) {
        uint32_t env = env_ids[e];
        memcpy(cur, state + (size_t)e * S, sizeof(float) * (size_t)S);
        uint32_t len = ep_len[e], rc = reset_count[e];
        for (int k = 0; k < T; ++k) {
            uint64_t t = t0 + (uint64_t)k;
            size_t row = (size_t)k * (size_t)n_sel + (size_t)e;
            if (out_obs) memcpy(out_obs + row * S, cur, sizeof(float) * (size_t)S);

            int act;
            uint32_t w = oracle_action_word(seed, env, t);
            if (given_actions) {
                act = given_actions[row];
            } else if (policy_params) {
                float logits[2];
                oracle_mlp_logits(policy_params, cur, logits);
                act = oracle_sample_action(logits, w);
            } else {
                act = action_stream ? oracle_action_bit(seed, env, t) : oracle_random_action(env_kind, w);
            }

            /* compute factor C (paper Section 4.2): the dynamics update is iterated C times with the
             * action held; reward, done and ep_len refer to the state after the last iteration */
            int done = 0; float rew;
            if (env_kind == ENV_CARTPOLE) act = act ? 1 : 0;
            else if (env_kind == ENV_ACROBOT) act = act < 0 ? 0 : (act > 2 ? 2 : act);
            else act = act ? 1 : 0;
            for (int c = 0; c < compute_factor; ++c) {
                if (c > 0) memcpy(cur, nxt, sizeof(float) * (size_t)S);
                if (env_kind == ENV_CARTPOLE) done = oracle_cartpole_step(cur, act, nxt);
                else if (env_kind == ENV_ACROBOT) done = oracle_acrobot_step(cur, act, nxt);
                else done = oracle_synth_step(cur, S, act, nxt, scratch);
            }
            len += 1;
            if (env_kind == ENV_ACROBOT) {
                int goal = done;
                done = goal | (len >= 500u);
                rew = goal ? 0.0f : -1.0f;
            } else {
                rew = 1.0f;
            }
            if (out_act) out_act[row] = (int8_t)act;
            if (out_rew) out_rew[row] = rew;
            if (out_done) out_done[row] = (uint8_t)done;

            if (done) {
                rc += 1;
                oracle_draw_state(env_kind, S, seed, env, rc, cur);
                len = 0;
            } else {
                memcpy(cur, nxt, sizeof(float) * (size_t)S);
            }
            if (next_obs) memcpy(next_obs + row * S, cur, sizeof(float) * (size_t)S);
        }
        memcpy(state + (size_t)e * S, cur, sizeof(float) * (size_t)S);
        ep_len[e] = len; reset_count[e] = rc;
    }
    return 0;
}

/* Running return of every episode in a trajectory: ret[t,e] = rew[t,e] + (done[t-1,e] ? 0 : ret[t-1,e]),
 * with `carry` [n] (in: return accumulated before row 0; out: after the last row, 0 where it ended). */
ORACLE_API void oracle_episode_returns(const float *rew, const uint8_t *done, int T, int64_t n, float *carry, float *ret)
{
    for (int64_t e = 0; e < n; ++e) {
        float acc = carry[e];
        for (int t = 0; t < T; ++t) {
            acc = acc + rew[(size_t)t * (size_t)n + (size_t)e];
            ret[(size_t)t * (size_t)n + (size_t)e] = acc;
            if (done[(size_t)t * (size_t)n + (size_t)e]) acc = 0.0f;
        }
        carry[e] = acc;
    }
}

/* Initial condition (draw #0, zeroed counters) for a list of env indices. */
ORACLE_API int oracle_reset(int env_kind, int S, uint64_t seed, int64_t n_sel, const uint32_t *env_ids,
                            float *state, uint32_t *ep_len, uint32_t *reset_count)
{
    if (env_kind < 0 || env_kind > 2 || S < 4 || S > 4096 || (S & (S - 1)) || n_sel < 0) return -1;
    for (int64_t e = 0; e < n_sel; ++e) {
        oracle_draw_state(env_kind, S, seed, env_ids[e], 0u, state + (size_t)e * S);
        ep_len[e] = 0; reset_count[e] = 0;
    }
    return 0;
}
