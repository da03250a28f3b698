// Fused CartPole rollout with the MLP policy in TENSOR mode (tolerance mode, not bit-exact): all three
// layers of the 4-64-64-2 network run on the 5th-generation tensor cores (tcgen05, accumulators in
// TMEM), tanh is the packed half-precision hardware approximation.  The paper names fusing simulation
// and inference as future work (Section 7); this is that fusion.
//
// One CTA = 128 threads = 128 envs = the 128 rows (TMEM lanes) of every accumulator.  Per step, three
// contractions, each issued by one thread and awaited by all through an mbarrier:
//   1. z1[128x64] = A1[128x16] B1^T    TF32; A1 row = (o_hi, o_lo, o_hi, 1, 1, 0, 0), B1 row j =
//      (w_hi, w_hi, w_lo, b_hi, b_lo, 0, 0): observation and weights split into two TF32 parts, so the
//      layer-1 sums carry about 21 bits, bias included;
//   2. z2[128x64] = A2[128x80] B2^T    FP16 operands, fp32 accumulation; A2 row = (h1[0..63], 1, 1, 0...)
//      with h1 = tanh.approx.f16x2(z1), B2 row j = (f16(W2[j][.]), b2 hi, b2 lo, 0...);
//   3. l[128x16]  = A2'[128x80] B3^T   A2' = the same tile refilled with h2 = tanh.approx.f16x2(z2);
//      B3 rows 0..3 = W3[0] hi, W3[0] lo, W3[1] hi, W3[1] lo (b3 in the bias columns of the hi rows):
//      logit i = l[2i] + l[2i+1].
// Each thread converts its own accumulator row (tcgen05.ld, 32 lanes x 32 bit) to the next operand row,
// then samples, steps the physics, resets and stores exactly like the exact kernel.
// Operand layout in shared memory (all operands K-major, no swizzle): 8-row x 16-byte core matrices;
// the core matrices of one 8-row group along K are contiguous (128 bytes apart = leading byte offset),
// 8-row groups follow each other (stride byte offset = 128 bytes x 16-byte chunks per row).
// Every wait is bounded: when a barrier does not complete in time the CTA records bit 0 in the status
// word, skips the remaining steps, frees its TMEM columns and returns.
#include "sim_internal.h"
#include "sim_envs.cuh"

namespace simk {

constexpr int kTcThreads = 128;
constexpr uint32_t kTcLBO = 128u;                 // bytes between core matrices adjacent along K
constexpr uint32_t kCh1 = 4u, kCh2 = 10u;         // 16-byte chunks per operand row: 16 TF32 values; 80 FP16 values
constexpr uint32_t kTcCols = 64u;                 // TMEM columns (fp32): z1 / z2 use all, the logits the first 16
// Instruction descriptors: D = fp32 (bit 4), A/B format (bits 7, 10: 2 = TF32, 0 = FP16), K-major, N >> 3 (bit 17), M >> 4 (bit 24).
constexpr uint32_t kIdescTf32N64 = (1u << 4) | (2u << 7) | (2u << 10) | ((64u >> 3) << 17) | ((128u >> 4) << 24);
constexpr uint32_t kIdescF16N64 = (1u << 4) | ((64u >> 3) << 17) | ((128u >> 4) << 24);
constexpr uint32_t kIdescF16N16 = (1u << 4) | ((16u >> 3) << 17) | ((128u >> 4) << 24);
constexpr long long kTcWaitCycles = 2000000000ll; // about a second at the SM clock

struct TcSmem {
    uint4 a1[128 * kCh1];   // layer-1 A operand (TF32 bit patterns)
    uint4 a2[128 * kCh2];   // layer-2 / layer-3 A operand (FP16)
    uint4 b1[64 * kCh1];    // layer-1 weights and bias (TF32, split)
    uint4 b2[64 * kCh2];    // layer-2 weights and bias (FP16)
    uint4 b3[16 * kCh2];    // layer-3 weights and bias (FP16, split), rows 4..15 zero
    unsigned long long bar; // mbarrier the tensor core commits to
    uint32_t tmem_slot;     // TMEM base address written by tcgen05.alloc
};

struct TcCtx {
    uint32_t tmem;
    uint32_t parity;
    bool fail;
};

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ uint32_t to_tf32(float x) { uint32_t r; asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x)); return r; }
__device__ __forceinline__ float tf32_as_float(uint32_t u) { return __uint_as_float(u); }
// f16x2 with `first` in the low half (the lower address / lower k).
__device__ __forceinline__ uint32_t pack_f16x2(float first, float second) { uint32_t r; asm("cvt.rn.satfinite.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(second), "f"(first)); return r; }
__device__ __forceinline__ uint32_t tanh_f16x2(uint32_t x) { uint32_t r; asm("tanh.approx.f16x2 %0, %1;" : "=r"(r) : "r"(x)); return r; }
__device__ __forceinline__ uint16_t f16_bits(float x) { uint16_t r; asm("cvt.rn.satfinite.f16.f32 %0, %1;" : "=h"(r) : "f"(x)); return r; }
__device__ __forceinline__ float f16_value(uint16_t h) { float r; asm("cvt.f32.f16 %0, %1;" : "=f"(r) : "h"(h)); return r; }

// Shared-memory matrix descriptor: start address, leading and stride byte offsets (16-byte units),
// descriptor version 1, no swizzle.
__device__ __forceinline__ uint64_t tc_desc(uint32_t saddr, uint32_t chunks_per_row)
{
    return (uint64_t)((saddr >> 4) & 0x3FFFu) | ((uint64_t)(kTcLBO >> 4) << 16) | ((uint64_t)((chunks_per_row * 128u) >> 4) << 32) | (1ull << 46);
}

// Index (in 16-byte chunks) of chunk c of row `row` of an operand tile with `ch` chunks per row.
__device__ __forceinline__ uint32_t tc_chunk(uint32_t row, uint32_t c, uint32_t ch) { return (row >> 3) * ch * 8u + c * 8u + (row & 7u); }

template <typename T>
__device__ __forceinline__ void tc_put(uint4 *tile, uint32_t row, uint32_t k, uint32_t ch, T value)
{
    constexpr uint32_t per = 16u / sizeof(T);
    reinterpret_cast<T *>(tile + tc_chunk(row, k / per, ch))[k % per] = value;
}

// Stage the parameters as operand tiles, allocate the accumulator columns, initialise the barrier and the
// constant columns of this thread's operand rows.  Called by all threads.
__device__ __forceinline__ void tc_setup(const float *__restrict__ p, TcSmem &s, TcCtx &c)
{
    const uint32_t tid = threadIdx.x;
    for (uint32_t i = tid; i < 64u * kCh1 + 64u * kCh2 + 16u * kCh2; i += kTcThreads) s.b1[i] = make_uint4(0u, 0u, 0u, 0u);   // b1, b2, b3 are contiguous
    __syncthreads();
    for (uint32_t i = tid; i < 256u; i += kTcThreads) {               // W1[j][k]
        const uint32_t j = i >> 2, k = i & 3u;
        const uint32_t hi = to_tf32(p[i]), lo = to_tf32(__fsub_rn(p[i], tf32_as_float(hi)));
        tc_put<uint32_t>(s.b1, j, k, kCh1, hi); tc_put<uint32_t>(s.b1, j, 4u + k, kCh1, hi); tc_put<uint32_t>(s.b1, j, 8u + k, kCh1, lo);
    }
    for (uint32_t j = tid; j < 64u; j += kTcThreads) {
        const float b1 = p[256 + j], b2 = p[4416 + j];
        const uint32_t hi = to_tf32(b1);
        tc_put<uint32_t>(s.b1, j, 12u, kCh1, hi); tc_put<uint32_t>(s.b1, j, 13u, kCh1, to_tf32(__fsub_rn(b1, tf32_as_float(hi))));
        const uint16_t h2 = f16_bits(b2);
        tc_put<uint16_t>(s.b2, j, 64u, kCh2, h2); tc_put<uint16_t>(s.b2, j, 65u, kCh2, f16_bits(__fsub_rn(b2, f16_value(h2))));
    }
    for (uint32_t i = tid; i < 4096u; i += kTcThreads) tc_put<uint16_t>(s.b2, i >> 6, i & 63u, kCh2, f16_bits(p[320 + i]));
    for (uint32_t i = tid; i < 128u; i += kTcThreads) {               // W3[a][k] -> rows 2a (hi), 2a+1 (lo)
        const uint32_t a = i >> 6, k = i & 63u;
        const uint16_t hi = f16_bits(p[4480 + i]);
        tc_put<uint16_t>(s.b3, 2u * a, k, kCh2, hi); tc_put<uint16_t>(s.b3, 2u * a + 1u, k, kCh2, f16_bits(__fsub_rn(p[4480 + i], f16_value(hi))));
    }
    if (tid < 2u) {
        const float b3 = p[4608 + tid];
        const uint16_t hi = f16_bits(b3);
        tc_put<uint16_t>(s.b3, 2u * tid, 64u, kCh2, hi); tc_put<uint16_t>(s.b3, 2u * tid, 65u, kCh2, f16_bits(__fsub_rn(b3, f16_value(hi))));
    }
    // constant columns of my rows: the two ones that multiply the bias parts, zero padding
    s.a1[tc_chunk(tid, 3u, kCh1)] = make_uint4(0x3F800000u, 0x3F800000u, 0u, 0u);
    s.a2[tc_chunk(tid, 8u, kCh2)] = make_uint4(0x3C003C00u, 0u, 0u, 0u);
    s.a2[tc_chunk(tid, 9u, kCh2)] = make_uint4(0u, 0u, 0u, 0u);
    if (tid == 0u) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_u32(&s.bar)), "r"(1u) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (tid < 32u) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" :: "r"(smem_u32(&s.tmem_slot)), "r"(kTcCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // the tiles are read by the tensor core (async proxy)
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    c.tmem = s.tmem_slot;
    c.parity = 0u;
    c.fail = false;
}

// Free the accumulator columns.  Called by all threads, after the last tc_policy.
__device__ __forceinline__ void tc_teardown(TcCtx &c)
{
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (threadIdx.x < 32)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(c.tmem), "r"(kTcCols) : "memory");
}

// One contraction D[128 x N] = A[128 x 16 nk bytes...] B^T over `nk` instructions of 32 bytes of K each (8 TF32 or
// 16 FP16 values): publish this thread's operand row, let thread 0 issue, wait (bounded) for completion.
// Returns false for the whole CTA when a wait ran out earlier; a wait that runs out now is reported by the next call.
template <bool TF32>
__device__ __forceinline__ bool tc_contract(uint32_t a_addr, uint32_t a_ch, uint32_t b_addr, uint32_t b_ch, uint32_t nk, uint32_t idesc,
                                            TcSmem &s, TcCtx &c, uint32_t *status)
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // my operand row: generic-proxy stores -> async proxy
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");  // my accumulator reads so far are done
    if (__syncthreads_or(c.fail ? 1 : 0)) { c.fail = true; return false; }
    if (threadIdx.x == 0) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        for (uint32_t k = 0; k < nk; ++k) {
            const uint64_t da = tc_desc(a_addr + k * 2u * kTcLBO, a_ch), db = tc_desc(b_addr + k * 2u * kTcLBO, b_ch);
            const uint32_t accumulate = k ? 1u : 0u;
            if (TF32)
                asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                             "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
                             :: "r"(c.tmem), "l"(da), "l"(db), "r"(idesc), "r"(accumulate) : "memory");
            else
                asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                             "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                             :: "r"(c.tmem), "l"(da), "l"(db), "r"(idesc), "r"(accumulate) : "memory");
        }
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(smem_u32(&s.bar)) : "memory");
    }
    const uint32_t bar = smem_u32(&s.bar);
    const long long t0 = clock64();
    uint32_t done = 0u;
    for (;;) {
        asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.b32 %0, 1, 0, p;\n\t}"
                     : "=r"(done) : "r"(bar), "r"(c.parity) : "memory");
        if (done || clock64() - t0 > kTcWaitCycles) break;
    }
    if (!done) { c.fail = true; if (status) atomicOr(status, 1u); }
    c.parity ^= 1u;
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    return true;
}

// Columns col0 .. col0+15 of this thread's accumulator row.
__device__ __forceinline__ void tc_load16(uint32_t taddr, uint32_t (&v)[16])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                   "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
                 : "r"(taddr));
}

// My accumulator row (64 columns) -> tanh -> FP16 -> my row of the A2 tile.
__device__ __forceinline__ void tc_activate(uint32_t taddr, TcSmem &s)
{
    uint32_t v[4][16];
#pragma unroll
    for (int q = 0; q < 4; ++q) tc_load16(taddr + 16u * (uint32_t)q, v[q]);
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
    uint4 *row = s.a2 + tc_chunk(threadIdx.x, 0u, kCh2);
#pragma unroll
    for (int q = 0; q < 4; ++q)
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            uint4 u;
            u.x = tanh_f16x2(pack_f16x2(__uint_as_float(v[q][8 * h + 0]), __uint_as_float(v[q][8 * h + 1])));
            u.y = tanh_f16x2(pack_f16x2(__uint_as_float(v[q][8 * h + 2]), __uint_as_float(v[q][8 * h + 3])));
            u.z = tanh_f16x2(pack_f16x2(__uint_as_float(v[q][8 * h + 4]), __uint_as_float(v[q][8 * h + 5])));
            u.w = tanh_f16x2(pack_f16x2(__uint_as_float(v[q][8 * h + 6]), __uint_as_float(v[q][8 * h + 7])));
            row[(2 * q + h) * 8] = u;                                  // chunk 2q+h of my row
        }
}

// Logits of this thread's observation; the CTA's 128 threads evaluate their 128 observations together.
// Returns false for the whole CTA when a wait ran out.
__device__ __forceinline__ bool tc_policy(const float4 o, TcSmem &s, TcCtx &c, uint32_t *status, f2 &logits)
{
    const uint32_t r = threadIdx.x;
    const uint32_t taddr = c.tmem + ((r & ~31u) << 16);
    {   // layer-1 operand row: observation split into two TF32 parts
        const uint32_t h0 = to_tf32(o.x), h1 = to_tf32(o.y), h2 = to_tf32(o.z), h3 = to_tf32(o.w);
        const uint4 hi = make_uint4(h0, h1, h2, h3);
        const uint4 lo = make_uint4(to_tf32(__fsub_rn(o.x, tf32_as_float(h0))), to_tf32(__fsub_rn(o.y, tf32_as_float(h1))),
                                    to_tf32(__fsub_rn(o.z, tf32_as_float(h2))), to_tf32(__fsub_rn(o.w, tf32_as_float(h3))));
        uint4 *row = s.a1 + tc_chunk(r, 0u, kCh1);
        row[0] = hi; row[8] = lo; row[16] = hi;
    }
    if (!tc_contract<true>(smem_u32(s.a1), kCh1, smem_u32(s.b1), kCh1, 2u, kIdescTf32N64, s, c, status)) return false;
    tc_activate(taddr, s);
    if (!tc_contract<false>(smem_u32(s.a2), kCh2, smem_u32(s.b2), kCh2, 5u, kIdescF16N64, s, c, status)) return false;
    tc_activate(taddr, s);
    if (!tc_contract<false>(smem_u32(s.a2), kCh2, smem_u32(s.b3), kCh2, 5u, kIdescF16N16, s, c, status)) return false;
    uint32_t l0, l1, l2, l3;
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(l0), "=r"(l1), "=r"(l2), "=r"(l3) : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
    logits = pk(__fadd_rn(__uint_as_float(l0), __uint_as_float(l1)), __fadd_rn(__uint_as_float(l2), __uint_as_float(l3)));
    return true;                        // a wait that ran out just now is reported (CTA-wide) by the next contraction
}

__global__ void __launch_bounds__(kTcThreads, 5)
rollout_cartpole_mlp_tc_kernel(const __grid_constant__ S4Args a)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    TcSmem &ms = *reinterpret_cast<TcSmem *>(smem_raw);
    TcCtx ctx;
    tc_setup(a.params, ms, ctx);

    // Every thread takes part in every barrier: threads past the batch shadow the last env and store nothing.
    const uint64_t i64 = (uint64_t)blockIdx.x * kTcThreads + threadIdx.x;
    const bool valid = i64 < a.n;
    const uint32_t i = valid ? (uint32_t)i64 : a.n - 1u;
    const uint32_t env = a.env_offset + i;

    float4 s = a.state[i];
    uint32_t len = a.ep_len[i], rc = a.reset_count[i];
    const bool st_obs = a.out_obs && valid, st_act = a.out_act && valid, st_rew = a.out_rew && valid, st_done = a.out_done && valid;
    const size_t n = a.n;
    size_t row = i;
    bool ok = true;

    const int nblk = (a.phase + a.K + 3) >> 2;
    for (int b = 0; b < nblk && ok; ++b) {
        const uint4 blk = philox(env, a.tb0 + (uint32_t)b, 0u, 0u, a.rk);
#pragma unroll 1
        for (int j = 0; j < 4; ++j) {
            const int k = 4 * b + j - a.phase;               // CTA-uniform
            if (k < 0 || k >= a.K) continue;
            const uint32_t w = j == 0 ? blk.x : j == 1 ? blk.y : j == 2 ? blk.z : blk.w;
            if (st_obs) __stcs(a.out_obs + row, s);
            f2 l;
            ok = tc_policy(s, ms, ctx, a.status, l);
            if (!ok) break;
            const int act = sample_pair(l, w);
            bool done = cartpole_step(s, act != 0);
            for (int c = 1; c < a.C; ++c) done = cartpole_step(s, act != 0);
            len += 1u;
            if (st_act) __stcs(a.out_act + row, (int8_t)act);
            if (st_rew) __stcs(a.out_rew + row, 1.0f);
            if (st_done) __stcs(a.out_done + row, (uint8_t)done);
            if (done) { rc += 1u; s = draw_state4<ENV_CARTPOLE>(env, rc, 0u, a.rk); len = 0u; }
            row += n;
        }
    }
    if (valid && ok) { a.state[i] = s; a.ep_len[i] = len; a.reset_count[i] = rc; }
    tc_teardown(ctx);
}

__global__ void __launch_bounds__(kTcThreads, 5)
policy_logits_tc_kernel(const float4 *__restrict__ obs, int64_t M, const float *__restrict__ params, float2 *__restrict__ logits, uint32_t *status)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    TcSmem &ms = *reinterpret_cast<TcSmem *>(smem_raw);
    TcCtx ctx;
    tc_setup(params, ms, ctx);
    const int64_t i = (int64_t)blockIdx.x * kTcThreads + threadIdx.x;
    const bool valid = i < M;
    f2 l;
    const bool ok = tc_policy(obs[valid ? i : M - 1], ms, ctx, status, l);
    if (valid && ok) logits[i] = make_float2(lo(l), hi(l));
    tc_teardown(ctx);
}

static cudaError_t tc_opt_in()
{
    static cudaError_t once = [] {
        cudaError_t e = cudaFuncSetAttribute(rollout_cartpole_mlp_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(TcSmem));
        if (e == cudaSuccess) e = cudaFuncSetAttribute(policy_logits_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(TcSmem));
        return e;
    }();
    return once;
}

cudaError_t launch_cartpole_mlp_tc(const S4Args &a, cudaStream_t st)
{
    cudaError_t e = tc_opt_in();
    if (e != cudaSuccess) return e;
    const unsigned blocks = (a.n + kTcThreads - 1u) / kTcThreads;
    rollout_cartpole_mlp_tc_kernel<<<blocks, kTcThreads, sizeof(TcSmem), st>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_policy_logits_tc(const float *obs, int64_t M, const float *params, float *logits, uint32_t *status, cudaStream_t st)
{
    if (M <= 0) return cudaSuccess;
    cudaError_t e = tc_opt_in();
    if (e != cudaSuccess) return e;
    const int64_t blocks = (M + kTcThreads - 1) / kTcThreads;
    if (blocks > 0x7FFFFFFFll) return cudaErrorInvalidConfiguration;
    policy_logits_tc_kernel<<<(unsigned)blocks, kTcThreads, sizeof(TcSmem), st>>>(reinterpret_cast<const float4 *>(obs), M, params,
                                                                                  reinterpret_cast<float2 *>(logits), status);
    return cudaGetLastError();
}

}  // namespace simk
