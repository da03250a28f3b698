// Fused CartPole rollout with the MLP policy in TENSOR mode (tolerance mode, not bit-exact): all three
// layers of the 4-64-64-2 network run on the 5th-generation tensor cores (tcgen05, FP16 operands, fp32
// accumulators in TMEM), tanh is the packed half-precision hardware approximation.  The paper names
// fusing simulation and inference as future work (Section 7); this is that fusion.
//
// One CTA = 256 threads = two groups of 128 threads; a group owns one tile of 128 envs (thread = env =
// row of the operand tile = TMEM lane of the accumulator) and synchronises on its own named barrier and
// its own mbarrier, so the two groups drift apart and one converts while the other's contraction runs.
// The weight tiles are shared by the groups.  Per step and tile, three contractions, each issued by the
// group's first thread and awaited by the group through the mbarrier:
//   1. z1[128x64] = A1[128x16] B1^T   A1 row = (o_hi[4], o_lo[4], o_hi[4], 1, 1, 0, 0), B1 row j =
//      (w_hi[4], w_hi[4], w_lo[4], b_hi, b_lo, 0, 0): observation, weights and bias split into two FP16
//      parts each, so the layer-1 sums carry about 21 bits;
//   2. z2[128x64] = A2[128x80] B2^T   A2 row = (h1[0..63], 1, 1, 0...), h1 = tanh.approx.f16x2(z1);
//      B2 row j = (f16(W2[j][.]), b2 hi, b2 lo, 0...);
//   3. l[128x16]  = A2'[128x80] B3^T  A2' = the same tile refilled with h2 = tanh.approx.f16x2(z2);
//      B3 rows 0..3 = W3[0] hi, W3[0] lo, W3[1] hi, W3[1] lo (b3 in the bias columns of the hi rows):
//      logit i = l[2i] + l[2i+1].
// Each thread converts its own accumulator row (tcgen05.ld, 32 lanes x 32 bit) into the next operand row,
// then samples, steps the physics, resets and stores exactly like the exact kernel.
// Operand layout in shared memory (all operands K-major, no swizzle): 8-row x 16-byte core matrices;
// the core matrices of one 8-row group along K are contiguous (128 bytes apart = leading byte offset),
// 8-row groups follow each other (stride byte offset = 128 bytes x 16-byte chunks per row).  A1 lives in
// the first 4 KB of the tile's A2 buffer (it is dead before h1 is written).
// Every wait is bounded: when a barrier does not complete in time the group records bit 0 in the status
// word and skips its remaining steps; the CTA then frees its TMEM columns and returns.
#include <mutex>

#include "sim_internal.h"
#include "sim_envs.cuh"
#include "tc_common.cuh"

namespace simk {

constexpr int kTcThreads = 256;                   // per CTA
constexpr uint32_t kTile = 128u;                  // envs (rows) per tile = threads per group
constexpr uint32_t kCh1 = 2u, kCh2 = 10u;         // 16-byte chunks per operand row: 16 and 80 FP16 values
constexpr uint32_t kTileCols = 64u;               // TMEM columns (fp32) per tile: z1 / z2 use all, the logits the first 16
constexpr uint32_t kTcCols = 2u * kTileCols;
// Instruction descriptors: D = fp32 (bit 4), A = B = FP16 (0 at bits 7 and 10), K-major, N >> 3 (bit 17), M >> 4 (bit 24).
constexpr uint32_t kIdescN64 = (1u << 4) | ((64u >> 3) << 17) | ((128u >> 4) << 24);
constexpr uint32_t kIdescN16 = (1u << 4) | ((16u >> 3) << 17) | ((128u >> 4) << 24);
constexpr long long kTcWaitCycles = 2000000000ll; // about a second at the SM clock

struct TcSmem {
    uint4 a[2][kTile * kCh2];  // per tile: A2 operand (FP16, 80 values per row); A1 (16 values per row) in its first 4 KB
    uint4 b1[64 * kCh1];       // layer-1 weights and bias (split)
    uint4 b2[64 * kCh2];       // layer-2 weights and bias
    uint4 b3[16 * kCh2];       // layer-3 weights and bias (split), rows 4..15 zero
    unsigned long long bar[2]; // per tile: mbarrier the tensor core commits to
    uint32_t tmem_slot;        // TMEM base address written by tcgen05.alloc
};

struct TcCtx {
    uint32_t tmem;          // this group's accumulator columns, lane 0
    uint32_t parity;        // phase parity of the group's mbarrier
    uint32_t group;         // 0 or 1
    uint32_t row;           // thread index inside the group
    bool fail;
};

// Group barrier (named barrier 1 + group, 128 threads) with an OR reduction of `flag`.
__device__ __forceinline__ bool group_sync_or(uint32_t group, bool flag)
{
    uint32_t out;
    if (group == 0u)
        asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %1, 0;\n\tbar.red.or.pred p, 1, 128, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(out) : "r"(flag ? 1u : 0u) : "memory");
    else
        asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %1, 0;\n\tbar.red.or.pred p, 2, 128, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                     : "=r"(out) : "r"(flag ? 1u : 0u) : "memory");
    return out != 0u;
}

// Stage the parameters as operand tiles, allocate the accumulator columns, initialise the barriers.
// Called by all threads of the CTA.
__device__ __forceinline__ void tc_setup(const float *__restrict__ p, TcSmem &s, TcCtx &c)
{
    const uint32_t tid = threadIdx.x;
    for (uint32_t i = tid; i < 64u * kCh1 + 64u * kCh2 + 16u * kCh2; i += kTcThreads) s.b1[i] = make_uint4(0u, 0u, 0u, 0u);   // b1, b2, b3 are contiguous
    __syncthreads();
    for (uint32_t i = tid; i < 256u; i += kTcThreads) {               // W1[j][k]
        const uint32_t j = i >> 2, k = i & 3u;
        uint16_t hi, lo;
        f16_split(p[i], hi, lo);
        tc_put(s.b1, j, k, kCh1, hi); tc_put(s.b1, j, 4u + k, kCh1, hi); tc_put(s.b1, j, 8u + k, kCh1, lo);
    }
    for (uint32_t j = tid; j < 64u; j += kTcThreads) {
        uint16_t hi, lo;
        f16_split(p[256 + j], hi, lo);
        tc_put(s.b1, j, 12u, kCh1, hi); tc_put(s.b1, j, 13u, kCh1, lo);
        f16_split(p[4416 + j], hi, lo);
        tc_put(s.b2, j, 64u, kCh2, hi); tc_put(s.b2, j, 65u, kCh2, lo);
    }
    for (uint32_t i = tid; i < 4096u; i += kTcThreads) tc_put(s.b2, i >> 6, i & 63u, kCh2, f16_bits(p[320 + i]));
    for (uint32_t i = tid; i < 128u; i += kTcThreads) {               // W3[a][k] -> rows 2a (hi), 2a+1 (lo)
        const uint32_t a = i >> 6, k = i & 63u;
        uint16_t hi, lo;
        f16_split(p[4480 + i], hi, lo);
        tc_put(s.b3, 2u * a, k, kCh2, hi); tc_put(s.b3, 2u * a + 1u, k, kCh2, lo);
    }
    if (tid < 2u) {
        uint16_t hi, lo;
        f16_split(p[4608 + tid], hi, lo);
        tc_put(s.b3, 2u * tid, 64u, kCh2, hi); tc_put(s.b3, 2u * tid, 65u, kCh2, lo);
    }
    if (tid == 0u) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_u32(&s.bar[0])), "r"(1u) : "memory");
        asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_u32(&s.bar[1])), "r"(1u) : "memory");
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
    c.group = tid >> 7;
    c.row = tid & 127u;
    c.tmem = s.tmem_slot + c.group * kTileCols;
    c.parity = 0u;
    c.fail = false;
}

// Free the accumulator columns.  Called by all threads of the CTA, after their last tc_policy.
__device__ __forceinline__ void tc_teardown(TcSmem &s)
{
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (threadIdx.x < 32)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(s.tmem_slot), "r"(kTcCols) : "memory");
}

enum : int { LAYER1 = 0, LAYER2 = 1, LAYER3 = 2 };

// Publish the group's operand rows, let its first thread issue the contraction of `LAYER` and commit it to the
// group's mbarrier, and wait (bounded) for completion.  Returns false for the whole group when a wait ran out
// earlier; a wait that runs out now sets the status bit and is turned into the group-wide exit by the next call.
// ISSUE = false (self-check only) leaves the contraction out, so that the wait must run out.
template <int LAYER, bool ISSUE = true>
__device__ __forceinline__ bool tc_contract(TcSmem &s, TcCtx &c, uint32_t *status, long long wait_cycles = kTcWaitCycles)
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // my operand row: generic-proxy stores -> async proxy
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");  // my accumulator reads so far are done
    if (group_sync_or(c.group, c.fail)) { c.fail = true; return false; }
    const uint32_t bar = smem_u32(&s.bar[c.group]);
    if (ISSUE && c.row == 0u) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t a_addr = smem_u32(s.a[c.group]);
        const uint32_t b_addr = LAYER == LAYER1 ? smem_u32(s.b1) : LAYER == LAYER2 ? smem_u32(s.b2) : smem_u32(s.b3);
        constexpr uint32_t ch = LAYER == LAYER1 ? kCh1 : kCh2;
        constexpr uint32_t nk = LAYER == LAYER1 ? 1u : 5u;           // instructions of K = 16 values (two core matrices) each
        constexpr uint32_t idesc = LAYER == LAYER3 ? kIdescN16 : kIdescN64;
#pragma unroll
        for (uint32_t k = 0; k < nk; ++k) {
            const uint64_t da = tc_desc(a_addr + k * 2u * kTcLBO, ch), db = tc_desc(b_addr + k * 2u * kTcLBO, ch);
            const uint32_t accumulate = k ? 1u : 0u;
            asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                         "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                         :: "r"(c.tmem), "l"(da), "l"(db), "r"(idesc), "r"(accumulate) : "memory");
        }
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(bar) : "memory");
    }
    const bool done = mbarrier_wait_bounded(bar, c.parity, wait_cycles);
    if (!done) { c.fail = true; if (status) atomicOr(status, 1u); }
    c.parity ^= 1u;
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    return true;
}

// My accumulator row (64 columns) -> tanh -> FP16 -> my row of the group's A2 operand.
__device__ __forceinline__ void tc_activate(TcSmem &s, const TcCtx &c)
{
    const uint32_t taddr = c.tmem + ((c.row & ~31u) << 16);
    uint4 *row = s.a[c.group] + tc_chunk(c.row, 0u, kCh2);
#pragma unroll
    for (int half = 0; half < 2; ++half) {
        uint32_t v[2][16];
        tc_load16(taddr + 32u * (uint32_t)half, v[0]);
        tc_load16(taddr + 32u * (uint32_t)half + 16u, v[1]);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
        for (int q = 0; q < 2; ++q)
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                uint4 u;
                u.x = tanh_f16x2(pack_f16x2(__uint_as_float(v[q][8 * h + 0]), __uint_as_float(v[q][8 * h + 1])));
                u.y = tanh_f16x2(pack_f16x2(__uint_as_float(v[q][8 * h + 2]), __uint_as_float(v[q][8 * h + 3])));
                u.z = tanh_f16x2(pack_f16x2(__uint_as_float(v[q][8 * h + 4]), __uint_as_float(v[q][8 * h + 5])));
                u.w = tanh_f16x2(pack_f16x2(__uint_as_float(v[q][8 * h + 6]), __uint_as_float(v[q][8 * h + 7])));
                row[(4 * half + 2 * q + h) * 8] = u;                   // chunk index along K
            }
    }
}

// Logits of this thread's observation; the group's 128 threads evaluate their 128 observations together.
// Returns false for the whole group when a wait ran out.
template <bool ISSUE = true>
__device__ __forceinline__ bool tc_policy(const float4 o, TcSmem &s, TcCtx &c, uint32_t *status, f2 &logits, long long wait_cycles = kTcWaitCycles)
{
    {   // layer-1 operand row: (o_hi[4], o_lo[4]) (o_hi[4], 1, 1, 0, 0)
        const uint32_t h01 = pack_f16x2(o.x, o.y), h23 = pack_f16x2(o.z, o.w);
        const float r0 = __fsub_rn(o.x, f16_value((uint16_t)(h01 & 0xFFFFu))), r1 = __fsub_rn(o.y, f16_value((uint16_t)(h01 >> 16)));
        const float r2 = __fsub_rn(o.z, f16_value((uint16_t)(h23 & 0xFFFFu))), r3 = __fsub_rn(o.w, f16_value((uint16_t)(h23 >> 16)));
        uint4 *row = s.a[c.group] + tc_chunk(c.row, 0u, kCh1);
        row[0] = make_uint4(h01, h23, pack_f16x2(r0, r1), pack_f16x2(r2, r3));
        row[8] = make_uint4(h01, h23, 0x3C003C00u, 0u);
    }
    if (!tc_contract<LAYER1, ISSUE>(s, c, status, wait_cycles)) return false;
    {   // the bias columns of my A2 row (the A1 rows of other threads may have covered them)
        uint4 *row = s.a[c.group] + tc_chunk(c.row, 0u, kCh2);
        row[8 * 8] = make_uint4(0x3C003C00u, 0u, 0u, 0u);
        row[9 * 8] = make_uint4(0u, 0u, 0u, 0u);
    }
    tc_activate(s, c);
    if (!tc_contract<LAYER2, ISSUE>(s, c, status, wait_cycles)) return false;
    tc_activate(s, c);
    if (!tc_contract<LAYER3, ISSUE>(s, c, status, wait_cycles)) return false;
    const uint32_t taddr = c.tmem + ((c.row & ~31u) << 16);
    uint32_t l0, l1, l2, l3;
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(l0), "=r"(l1), "=r"(l2), "=r"(l3) : "r"(taddr));
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
    logits = pk(__fadd_rn(__uint_as_float(l0), __uint_as_float(l1)), __fadd_rn(__uint_as_float(l2), __uint_as_float(l3)));
    return true;
}

__global__ void __launch_bounds__(kTcThreads, 4)
rollout_cartpole_mlp_tc_kernel(const __grid_constant__ S4Args a)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    TcSmem &ms = *reinterpret_cast<TcSmem *>(smem_raw);
    TcCtx ctx;
    tc_setup(a.params, ms, ctx);

    // Every thread takes part in every barrier of its group: threads past the batch shadow the last env and store nothing.
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
    tc_teardown(ms);
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
    tc_teardown(ms);
}

// Self-check of the bounded wait: one CTA runs the policy with the contractions left out, so the first wait of
// either group must run out (after `wait_cycles`), set the status bit and turn the next contraction into the
// group-wide exit.  completed[i] = 1 if thread i's policy call reported success (expected: none).
__global__ void __launch_bounds__(kTcThreads, 4)
tensor_wait_selfcheck_kernel(const float *__restrict__ params, long long wait_cycles, uint32_t *status, uint32_t *completed)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    TcSmem &ms = *reinterpret_cast<TcSmem *>(smem_raw);
    TcCtx ctx;
    tc_setup(params, ms, ctx);
    f2 l;
    const bool ok = tc_policy<false>(make_float4(0.0f, 0.0f, 0.0f, 0.0f), ms, ctx, status, l, wait_cycles);
    completed[threadIdx.x] = ok ? 1u : 0u;
    tc_teardown(ms);
}

// The kernels need more than 48 KB of dynamic shared memory: opt in once per device.
static cudaError_t tc_opt_in()
{
    static std::mutex lock;
    static bool done[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    std::lock_guard<std::mutex> guard(lock);
    if (dev >= 0 && dev < 64 && done[dev]) return cudaSuccess;
    e = cudaFuncSetAttribute(rollout_cartpole_mlp_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(TcSmem));
    if (e == cudaSuccess) e = cudaFuncSetAttribute(policy_logits_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(TcSmem));
    if (e == cudaSuccess) e = cudaFuncSetAttribute(tensor_wait_selfcheck_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(TcSmem));
    if (e == cudaSuccess && dev >= 0 && dev < 64) done[dev] = true;
    return e;
}

cudaError_t launch_cartpole_mlp_tc(const S4Args &a, cudaStream_t st)
{
    cudaError_t e = tc_opt_in();
    if (e != cudaSuccess) return e;
    const unsigned blocks = (unsigned)(((uint64_t)a.n + kTcThreads - 1u) / kTcThreads);
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

cudaError_t launch_tensor_wait_selfcheck(const float *params, long long wait_cycles, uint32_t *status, uint32_t *completed, cudaStream_t st)
{
    cudaError_t e = tc_opt_in();
    if (e != cudaSuccess) return e;
    tensor_wait_selfcheck_kernel<<<1, kTcThreads, sizeof(TcSmem), st>>>(params, wait_cycles, status, completed);
    return cudaGetLastError();
}

}  // namespace simk
