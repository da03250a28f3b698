// Fused multi-step rollout of the synthetic S-float simulator (the "state factor" experiment:
// S times the state, S times the global loads and stores per unfused step).
//
// Mapping: an env's S floats are split into L = S/E contiguous chunks of E floats, one chunk per
// thread, held in registers for all K steps of the launch.  L <= 32: the L threads of an env are
// adjacent lanes of one warp (several envs per warp when L < 32) and exchange the one halo element
// and the partial sums with shuffles.  L > 32: one CTA per env, the warps exchange through shared
// memory.  Inside a chunk, element j travels with element j + E/2 as one packed fp32 pair, so the
// "right neighbour" operand of pair j is simply pair j+1 and one issue slot updates two elements.
// The sum of squares follows an adjacent-pairs-first binary tree over the element index: inside
// each half chunk (both halves at once, packed), the two halves, then lanes by xor-shuffles, then
// warps.
#include "sim_internal.h"
#include "sim_envs.cuh"

#ifndef SYNTH_E_SHORT
#define SYNTH_E_SHORT 16
#endif
#ifndef SYNTH_E_LONG_CAP
#define SYNTH_E_LONG_CAP 64
#endif

namespace simk {

// Floats per thread.  Long launches want long chunks (64): few shuffles, halo exchanges and barriers per
// element and many independent pairs per thread.  Short launches (a stream over the state matrix) want
// more threads in flight and do best with 16 (measured at K = 1: 4 -> 3.3e11, 8 -> 4.9e11, 16 -> 5.7e11
// element-steps/s for S = 16..128; the per-thread overhead of a tile is what a short launch pays for).
constexpr int synth_chunk_short(int S) { return S < SYNTH_E_SHORT ? S : SYNTH_E_SHORT; }
constexpr int synth_chunk_long(int S) { return S < SYNTH_E_LONG_CAP ? S : SYNTH_E_LONG_CAP; }

template <int S, int E_> struct SynthShape {
    static constexpr int E = E_;                                        // floats per thread
    static constexpr int H = E / 2;                                     // packed pairs per thread
    static constexpr int L = S / E;                                     // threads per env
    static constexpr int WARPS = L > 32 ? L / 32 : 1;                   // warps per env when L > 32
    static constexpr int THREADS = L > 32 ? L : 256;
    static constexpr int ENVS_PER_CTA = THREADS / L;                    // envs per tile
};

// Shared memory used for the cross-warp exchange of one env (L > 32).
template <int W> struct SynthExchange { float halo[2][W]; float sum[W]; };   // halo is double-buffered across iterations

// K steps of one chunk held in registers.  P[j] = (x_j, x_{j+H}).  All threads of a CTA call this
// together (it contains CTA barriers when an env spans several warps).
template <int S, int EE, bool LEAN>
__device__ __forceinline__ void synth_steps(const SynthArgs &a, f2 (&P)[EE / 2], uint32_t &len, uint32_t &rc,
                                            uint32_t i, bool valid, uint32_t sub, SynthExchange<SynthShape<S, EE>::WARPS> &xc)
{
    using Sh = SynthShape<S, EE>;
    constexpr int E = Sh::E, H = Sh::H, L = Sh::L, W = Sh::WARPS;
    constexpr int LS = L < 32 ? L : 32;                 // lanes of one env inside a warp
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    const uint32_t env = a.env_offset + i;
    const bool leader = valid && sub == 0;
    size_t row = i;

    const int nblk = (a.phase + a.K + 3) >> 2;
    for (int b = 0; b < nblk; ++b) {
        uint4 blk = make_uint4(0u, 0u, 0u, 0u);
        if (LEAN || !a.actions) blk = philox(env, a.tb0 + (uint32_t)b, 0u, 0u, a.rk);
        // steps of this launch inside block b: words jlo..jhi-1 (short chunks unroll all four words and skip by test;
        // long chunks run a rolled loop over exactly the words in range, which is one iteration for a one-step launch)
        const int jlo = EE <= 8 ? 0 : max(0, a.phase - 4 * b), jhi = EE <= 8 ? 4 : min(4, a.phase + a.K - 4 * b);
#pragma unroll(EE <= 8 ? 4 : 1)
        for (int j4 = jlo; j4 < jhi; ++j4) {
            const int k = 4 * b + j4 - a.phase;
            if (EE <= 8 && (k < 0 || k >= a.K)) continue;
            const uint32_t w = j4 == 0 ? blk.x : j4 == 1 ? blk.y : j4 == 2 ? blk.z : blk.w;

            if (!LEAN && a.out_obs && valid) {
                float *dst = a.out_obs + row * S + (size_t)sub * E;
                float xo[E];
#pragma unroll
                for (int j = 0; j < H; ++j) { xo[j] = lo(P[j]); xo[j + H] = hi(P[j]); }
#pragma unroll
                for (int v = 0; v < E / 4; ++v)
                    __stcs(reinterpret_cast<float4 *>(dst + 4 * v), make_float4(xo[4 * v], xo[4 * v + 1], xo[4 * v + 2], xo[4 * v + 3]));
            }

            const int act = (!LEAN && a.actions) ? (a.actions[i] != 0) : (int)(w >> 31);
            const f2 c = splat(__fmul_rn(fbits(0x3A83126Fu), act ? 1.0f : -1.0f));

            // compute factor: C Jacobi iterations under one action; squares and the done test use the last one
            f2 Q[H];
            for (int cit = 0; cit < a.C; ++cit) {
                // halo: first element of the next chunk of the same env (wrapping around)
                const float x0 = lo(P[0]);
                float halo;
                if (L == 1) {
                    halo = x0;
                } else {
                    halo = __shfl_sync(0xFFFFFFFFu, x0, (lane & ~(uint32_t)(LS - 1)) | ((lane + 1u) & (uint32_t)(LS - 1)));
                    if (W > 1) {
                        if (lane == 0) xc.halo[cit & 1][warp] = x0;
                        __syncthreads();
                        if (lane == 31) halo = xc.halo[cit & 1][(warp + 1u) % W];
                    }
                }
                // Jacobi update: every right-hand side reads pre-iteration values.  The right neighbours of
                // pair j = (x_j, x_{j+H}) are pair j+1; the last pair's are (x_H, halo).
                const f2 wrap = pk(hi(P[0]), halo);
                const f2 c01 = splat(fbits(0x3C23D70Au));
#pragma unroll
                for (int j = 0; j < H; ++j) {
                    const f2 right = j + 1 < H ? P[j + 1] : wrap;
                    const f2 z = sin2(add2(P[j], right));
                    Q[j] = add2(fma2(c01, z, P[j]), c);
                }
#pragma unroll
                for (int j = 0; j < H; ++j) P[j] = Q[j];
            }
#pragma unroll
            for (int j = 0; j < H; ++j) Q[j] = mul2(P[j], P[j]);
#pragma unroll
            for (int wdt = 1; wdt < H; wdt <<= 1)
#pragma unroll
                for (int j = 0; j < H; j += 2 * wdt) Q[j] = add2(Q[j], Q[j + wdt]);
            float sum = __fadd_rn(lo(Q[0]), hi(Q[0]));               // left half + right half of the chunk
#pragma unroll
            for (int m = 1; m < LS; m <<= 1) sum = __fadd_rn(sum, __shfl_xor_sync(0xFFFFFFFFu, sum, m));
            if (W > 1) {
                if (lane == 0) xc.sum[warp] = sum;
                __syncthreads();
                float part[W];
#pragma unroll
                for (int v = 0; v < W; ++v) part[v] = xc.sum[v];
#pragma unroll
                for (int wdt = 1; wdt < W; wdt <<= 1)
#pragma unroll
                    for (int v = 0; v < W; v += 2 * wdt) part[v] = __fadd_rn(part[v], part[v + wdt]);
                sum = part[0];
            }
            const bool done = __fmul_rn(sum, 1.0f / (float)S) > 4.0f;
            len += 1u;

            if (!LEAN && leader) {
                if (a.out_act) __stcs(&a.out_act[row], (int8_t)act);
                if (a.out_rew) __stcs(&a.out_rew[row], 1.0f);
                if (a.out_done) __stcs(&a.out_done[row], (uint8_t)done);
            }

            if (done) {                                     // uniform over the threads of one env
                rc += 1u;
                float xr[E];
#pragma unroll
                for (int v = 0; v < E / 4; ++v) {
                    const float4 f = draw_state4<ENV_SYNTH>(env, rc, sub * (uint32_t)(E / 4) + (uint32_t)v, a.rk);
                    xr[4 * v + 0] = f.x; xr[4 * v + 1] = f.y; xr[4 * v + 2] = f.z; xr[4 * v + 3] = f.w;
                }
#pragma unroll
                for (int j = 0; j < H; ++j) P[j] = pk(xr[j], xr[j + H]);
                len = 0u;
            }
            row += a.n;
        }
    }
}

template <int S, int EE>
__device__ __forceinline__ void synth_store(const SynthArgs &a, const f2 (&P)[EE / 2], uint32_t len, uint32_t rc,
                                            uint32_t i, uint32_t sub)
{
    constexpr int E = EE, H = EE / 2;
    float xo[E];
#pragma unroll
    for (int j = 0; j < H; ++j) { xo[j] = lo(P[j]); xo[j + H] = hi(P[j]); }
    float4 *dst = reinterpret_cast<float4 *>(a.state + (size_t)i * S + (size_t)sub * E);
#pragma unroll
    for (int v = 0; v < E / 4; ++v) dst[v] = make_float4(xo[4 * v], xo[4 * v + 1], xo[4 * v + 2], xo[4 * v + 3]);
    if (a.next_obs) {
        float4 *nd = reinterpret_cast<float4 *>(a.next_obs + (size_t)i * S + (size_t)sub * E);
#pragma unroll
        for (int v = 0; v < E / 4; ++v) nd[v] = make_float4(xo[4 * v], xo[4 * v + 1], xo[4 * v + 2], xo[4 * v + 3]);
    }
    if (sub == 0) { a.ep_len[i] = len; a.reset_count[i] = rc; }
}

// One tile (THREADS chunks) per CTA; each thread loads its chunk straight into registers.  (A persistent
// variant with a cp.async ring of shared-memory stages was measured for K = 1 and was slower: at K = 1
// the launch is bound by instruction issue per tile, not by bytes in flight.)
// LEAN: no trajectory output and random actions (the timed configuration of the synthetic workload); the
// per-step checks for optional outputs and given actions are compiled out.
template <int S, int EE, bool LEAN>
__global__ void __launch_bounds__(SynthShape<S, EE>::THREADS)
rollout_synth_kernel(const __grid_constant__ SynthArgs a)
{
    using Sh = SynthShape<S, EE>;
    constexpr int E = Sh::E, H = Sh::H, L = Sh::L;
    __shared__ SynthExchange<Sh::WARPS> xc;
    const uint32_t tid = threadIdx.x;
    const uint32_t sub = tid % L;
    const uint64_t i64 = (uint64_t)blockIdx.x * Sh::ENVS_PER_CTA + tid / L;
    const bool valid = i64 < a.n;                       // tail threads compute on env n-1 and store nothing
    uint32_t i = valid ? (uint32_t)i64 : a.n - 1u;
    pdl_wait();
    pdl_release();

    f2 P[H];
    {
        float xin[E];
        const float4 *src = reinterpret_cast<const float4 *>(a.state + (size_t)i * S + (size_t)sub * E);
#pragma unroll
        for (int v = 0; v < E / 4; ++v) { const float4 f = src[v]; xin[4 * v] = f.x; xin[4 * v + 1] = f.y; xin[4 * v + 2] = f.z; xin[4 * v + 3] = f.w; }
#pragma unroll
        for (int j = 0; j < H; ++j) P[j] = pk(xin[j], xin[j + H]);
    }
    uint32_t len = a.ep_len[i], rc = a.reset_count[i];
    synth_steps<S, EE, LEAN>(a, P, len, rc, i, valid, sub, xc);
    if (valid) synth_store<S, EE>(a, P, len, rc, i, sub);
}

template <int S, int EE>
static cudaError_t launch_synth_e(const SynthArgs &a, cudaStream_t st)
{
    using Sh = SynthShape<S, EE>;
    const uint32_t ntiles = (a.n + Sh::ENVS_PER_CTA - 1u) / Sh::ENVS_PER_CTA;
    const bool lean = !a.out_obs && !a.out_act && !a.out_rew && !a.out_done && !a.actions;
    if (lean) return launch_overlapped(a.K <= kOverlapMaxK, rollout_synth_kernel<S, EE, true>, dim3(ntiles), dim3(Sh::THREADS), 0, st, a);
    return launch_overlapped(a.K <= kOverlapMaxK, rollout_synth_kernel<S, EE, false>, dim3(ntiles), dim3(Sh::THREADS), 0, st, a);
}

constexpr int kSynthLongK = 3;     // launches of at least this many steps use the long-chunk shape

template <int S>
static cudaError_t launch_synth_t(const SynthArgs &a, cudaStream_t st)
{
    if (a.K >= kSynthLongK) return launch_synth_e<S, synth_chunk_long(S)>(a, st);
    return launch_synth_e<S, synth_chunk_short(S)>(a, st);
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
