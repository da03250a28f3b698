// Fused CartPole rollout with the MLP policy in TENSOR mode (tolerance mode, not bit-exact): the
// 64x64 hidden layer of 128 envs is one tcgen05 TF32 contraction per step, both tanh layers use the
// hardware approximation.  The paper names fusing simulation and inference as future work (Section 7);
// this is that fusion with the layer-2 product on the 5th-generation tensor cores.
//
// One CTA = 128 threads = 128 envs = the 128 rows (TMEM lanes) of the accumulator.  Per step:
//   1. every thread evaluates layer 1 for its env (same fp32 chains as the exact kernel), applies
//      tanh.approx, rounds to TF32 and writes its 64-value row of the A operand to shared memory;
//   2. one thread issues 8 tcgen05.mma (M = 128, N = 64, K = 8 each) against the W2 tile staged once
//      per CTA, accumulating in 64 TMEM columns, and commits to an mbarrier;
//   3. every thread waits for the barrier, reads its accumulator row with tcgen05.ld, adds the bias,
//      applies tanh.approx and reduces layer 3 in fp32; sampling, physics, reset and the trajectory
//      stores are those of the exact kernel.
// Operand layout in shared memory (both operands K-major, no swizzle): 8 x 16-byte core matrices;
// the 16 core matrices of one 8-row group along K are contiguous (128 bytes apart = leading byte
// offset), 8-row groups are 2048 bytes apart (stride byte offset).
// Every wait is bounded: when the barrier does not complete in time the CTA records bit 0 in the
// status word, skips the remaining steps, frees its TMEM columns and returns.
#include "sim_internal.h"
#include "sim_envs.cuh"

namespace simk {

constexpr int kTcThreads = 128;
constexpr uint32_t kTcLBO = 128u;       // bytes between core matrices adjacent along K
constexpr uint32_t kTcSBO = 2048u;      // bytes between 8-row groups
constexpr uint32_t kTcCols = 64u;       // TMEM columns: one fp32 accumulator column per hidden unit
// Instruction descriptor: D = fp32, A = B = TF32, both K-major, N = 64, M = 128, dense, no negation.
constexpr uint32_t kTcIdesc = (1u << 4) | (2u << 7) | (2u << 10) | ((64u >> 3) << 17) | ((128u >> 4) << 24);
constexpr long long kTcWaitCycles = 2000000000ll;   // about a second at the SM clock

struct TcSmem {
    uint32_t a[128 * 64];   // layer-2 A operand: tanh(layer 1) of the CTA's 128 envs, TF32 bit patterns
    uint32_t b[64 * 64];    // layer-2 B operand: W2[out][in], TF32 bit patterns
    float w1t[4 * 64];      // w1t[k*64 + j] = W1[j][k]
    float b1[64];
    float b2[64];
    float2 w3[64];          // (W3[0][j], W3[1][j])
    float2 b3;
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
__device__ __forceinline__ float tanh_hw(float x) { float r; asm("tanh.approx.f32 %0, %1;" : "=f"(r) : "f"(x)); return r; }

// Shared-memory matrix descriptor: start address, leading and stride byte offsets (16-byte units),
// descriptor version 1, no swizzle.
__device__ __forceinline__ uint64_t tc_desc(uint32_t saddr)
{
    return (uint64_t)((saddr >> 4) & 0x3FFFu) | ((uint64_t)(kTcLBO >> 4) << 16) | ((uint64_t)(kTcSBO >> 4) << 32) | (1ull << 46);
}

// Byte offset of element (row, k) of an operand tile.
__device__ __forceinline__ uint32_t tc_offset(uint32_t row, uint32_t k)
{
    return (row >> 3) * kTcSBO + (k >> 2) * kTcLBO + (row & 7u) * 16u + (k & 3u) * 4u;
}

// Stage the parameters, allocate the accumulator columns, initialise the barrier.  Called by all threads.
__device__ __forceinline__ void tc_setup(const float *__restrict__ p, TcSmem &s, TcCtx &c)
{
    const int tid = threadIdx.x;
    for (int i = tid; i < 256; i += kTcThreads) s.w1t[(i & 3) * 64 + (i >> 2)] = p[i];
    for (int i = tid; i < 64; i += kTcThreads) {
        s.b1[i] = p[256 + i];
        s.b2[i] = p[4416 + i];
        s.w3[i] = make_float2(p[4480 + i], p[4544 + i]);
    }
    for (int i = tid; i < 4096; i += kTcThreads)
        s.b[tc_offset((uint32_t)i >> 6, (uint32_t)i & 63u) >> 2] = to_tf32(p[320 + i]);
    if (tid == 0) {
        s.b3 = make_float2(p[4608], p[4609]);
        asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_u32(&s.bar)), "r"(1u) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (tid < 32) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" :: "r"(smem_u32(&s.tmem_slot)), "r"(kTcCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // the B tile is read by the tensor core (async proxy)
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

// Logits of this thread's observation; the CTA's 128 threads evaluate their 128 observations together.
// Returns false for the whole CTA when a wait ran out (now or in an earlier call).
__device__ __forceinline__ bool tc_policy(const float4 o, TcSmem &s, TcCtx &c, uint32_t *status, f2 &logits)
{
    const uint32_t r = threadIdx.x;
    // Layer 1: fp32 chains from the bias over inputs 0..3, as in the exact kernel; tanh; TF32; A row.
    {
        unsigned char *arow = reinterpret_cast<unsigned char *>(s.a) + (r >> 3) * kTcSBO + (r & 7u) * 16u;
        const f2 o0 = splat(o.x), o1 = splat(o.y), o2 = splat(o.z), o3 = splat(o.w);
#pragma unroll
        for (int j = 0; j < 64; j += 4) {
            const float4 bias = *reinterpret_cast<const float4 *>(&s.b1[j]);
            const float4 w0 = *reinterpret_cast<const float4 *>(&s.w1t[0 * 64 + j]), w1 = *reinterpret_cast<const float4 *>(&s.w1t[1 * 64 + j]);
            const float4 w2 = *reinterpret_cast<const float4 *>(&s.w1t[2 * 64 + j]), w3 = *reinterpret_cast<const float4 *>(&s.w1t[3 * 64 + j]);
            f2 p = pk(bias.x, bias.y), q = pk(bias.z, bias.w);
            p = fma2(pk(w0.x, w0.y), o0, p); q = fma2(pk(w0.z, w0.w), o0, q);
            p = fma2(pk(w1.x, w1.y), o1, p); q = fma2(pk(w1.z, w1.w), o1, q);
            p = fma2(pk(w2.x, w2.y), o2, p); q = fma2(pk(w2.z, w2.w), o2, q);
            p = fma2(pk(w3.x, w3.y), o3, p); q = fma2(pk(w3.z, w3.w), o3, q);
            const uint4 u = make_uint4(to_tf32(tanh_hw(lo(p))), to_tf32(tanh_hw(hi(p))), to_tf32(tanh_hw(lo(q))), to_tf32(tanh_hw(hi(q))));
            *reinterpret_cast<uint4 *>(arow + (j >> 2) * kTcLBO) = u;
        }
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // my A row: generic-proxy stores -> async proxy
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");  // my accumulator reads of the previous step are done
    if (__syncthreads_or(c.fail ? 1 : 0)) { c.fail = true; return false; }

    if (r == 0) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t a0 = smem_u32(s.a), b0 = smem_u32(s.b);
#pragma unroll
        for (uint32_t k8 = 0; k8 < 8u; ++k8) {                        // K = 8 TF32 values = two core matrices per instruction
            const uint64_t da = tc_desc(a0 + k8 * 2u * kTcLBO), db = tc_desc(b0 + k8 * 2u * kTcLBO);
            const uint32_t accumulate = k8 ? 1u : 0u;
            asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                         "tcgen05.mma.cta_group::1.kind::tf32 [%0], %1, %2, %3, p;\n\t}"
                         :: "r"(c.tmem), "l"(da), "l"(db), "r"(kTcIdesc), "r"(accumulate) : "memory");
        }
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(smem_u32(&s.bar)) : "memory");
    }

    {   // bounded wait for the contraction
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
    }
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");

    // My accumulator row: TMEM lane = thread index, 64 fp32 columns.
    uint32_t v[64];
    const uint32_t taddr = c.tmem + ((r & ~31u) << 16);
#pragma unroll
    for (int q = 0; q < 4; ++q) {
        asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                     : "=r"(v[q * 16 + 0]), "=r"(v[q * 16 + 1]), "=r"(v[q * 16 + 2]), "=r"(v[q * 16 + 3]),
                       "=r"(v[q * 16 + 4]), "=r"(v[q * 16 + 5]), "=r"(v[q * 16 + 6]), "=r"(v[q * 16 + 7]),
                       "=r"(v[q * 16 + 8]), "=r"(v[q * 16 + 9]), "=r"(v[q * 16 + 10]), "=r"(v[q * 16 + 11]),
                       "=r"(v[q * 16 + 12]), "=r"(v[q * 16 + 13]), "=r"(v[q * 16 + 14]), "=r"(v[q * 16 + 15])
                     : "r"(taddr + (uint32_t)q * 16u));
    }
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");

    // Layer-2 bias and tanh, layer 3 in fp32 in ascending unit order from the bias.
    logits = pk(s.b3.x, s.b3.y);
#pragma unroll
    for (int j = 0; j < 64; j += 4) {
        const float4 bias = *reinterpret_cast<const float4 *>(&s.b2[j]);
        const float4 wa = *reinterpret_cast<const float4 *>(&s.w3[j]), wb = *reinterpret_cast<const float4 *>(&s.w3[j + 2]);
        const float h0 = tanh_hw(__fadd_rn(__uint_as_float(v[j + 0]), bias.x));
        const float h1 = tanh_hw(__fadd_rn(__uint_as_float(v[j + 1]), bias.y));
        const float h2 = tanh_hw(__fadd_rn(__uint_as_float(v[j + 2]), bias.z));
        const float h3 = tanh_hw(__fadd_rn(__uint_as_float(v[j + 3]), bias.w));
        logits = fma2(pk(wa.x, wa.y), splat(h0), logits);
        logits = fma2(pk(wa.z, wa.w), splat(h1), logits);
        logits = fma2(pk(wb.x, wb.y), splat(h2), logits);
        logits = fma2(pk(wb.z, wb.w), splat(h3), logits);
    }
    return true;
}

__global__ void __launch_bounds__(kTcThreads, 4)
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

__global__ void __launch_bounds__(kTcThreads, 4)
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
