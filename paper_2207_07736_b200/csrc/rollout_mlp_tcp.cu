// Fused CartPole rollout with the MLP policy in PRECISE TENSOR mode: the two hidden layers of the 4-64-64-2 network
// run on the 5th-generation tensor cores (tcgen05, FP16 operands, fp32 accumulators in TMEM), but every operand is
// carried as a sum of FP16 parts whose products are exact, tanh is evaluated in fp32 and the two-unit output layer
// runs on the fp32 pipes, so that the logits stay within 1e-5 of the fp32 definition (the fast tensor mode of
// rollout_mlp_tc.cu trades three more digits for speed).  The paper names fusing simulation and inference as future
// work (Section 7); this is that fusion at fp32-level accuracy.
//
// One CTA = kGroups groups of 128 threads; a group owns one tile of 128 envs (thread = env = row of the operand tile
// = TMEM lane of the accumulator) and synchronises on its own named barrier and its own mbarrier, so the groups
// drift apart and one converts while another's contraction runs.  The weight tiles are shared by the groups.
// Per step and tile, two contractions, each issued by the group's first thread and awaited through the mbarrier:
//   1. z1[128x64] = A1[128x32] B1^T: observation o = o1 + o2 + o3 and W1 = w1 + w2 + w3 (b1 likewise) in three
//      FP16 parts; the columns pair the parts so that o1w1 + o2w1 + o3w1 + o1w2 + o2w2 + o1w3 + b1 is summed (what is
//      dropped is below 2^-33 of a product);
//   2. z2[128x64] = Ahi Bhi^T + Ahi Blo^T + Alo Bhi^T with h1 = hi + lo (hi = h1 cut to 11 bits, lo = f16(h1 - hi)),
//      W2 = f16(W2) + f16(W2 - f16(W2)); twelve instructions of K = 16 into one accumulator; b2 is added in fp32
//      when the accumulator row is read back.
// Each thread turns its accumulator row of layer 1 into its operand row of layer 2 (tcgen05.ld, tanh, hi / lo split,
// sixteen 16-byte shared-memory stores) and its accumulator row of layer 2 straight into the two logits
// (tanh, then logit_i = b3[i] + sum_j W3[i][j] h2[j] in fp32, two packed partial sums per logit); then it samples,
// steps the physics, resets and stores exactly like the exact kernel.  An output layer on the tensor core (a third
// contraction with N = 16) was measured 13 % slower: it needs the split of h2, its stores and a third round trip.
// tanh(z) = 1 - 2 / (2^(2 log2(e) z) + 1) with the hardware's base-2 exponential and reciprocal approximations
// (relative error about 2^-22 each), four evaluations sharing one reciprocal: absolute error below 4e-7.
// A1 lives in the first 8 KB of the tile's operand buffer (it is dead before h1 is written).
// Every wait is bounded: when a barrier does not complete in time the group records bit 0 in the status word and
// skips its remaining steps; the CTA then frees its TMEM columns and returns.
#include <mutex>

#include "sim_internal.h"
#include "sim_envs.cuh"
#include "tc_common.cuh"

#ifndef TCP_GROUPS
#define TCP_GROUPS 2
#endif
#ifndef TCP_MINBLOCKS
#define TCP_MINBLOCKS 2
#endif

namespace simk {
namespace tcp {

constexpr int kGroups = TCP_GROUPS;               // tiles (groups of 128 threads) per CTA
constexpr int kThreads = 128 * kGroups;
constexpr uint32_t kTile = 128u;                  // envs (rows) per tile = threads per group
constexpr uint32_t kChA = 16u;                    // 16-byte chunks per operand row of layer 2: h1 hi[64] | h1 lo[64]
constexpr uint32_t kCh1 = 4u;                     // layer-1 operand row: 32 FP16 values
constexpr uint32_t kTileCols = 64u;               // TMEM columns (fp32) per tile
constexpr uint32_t kCols = kGroups * kTileCols <= 32 ? 32u : kGroups * kTileCols <= 64 ? 64u : kGroups * kTileCols <= 128 ? 128u
                           : kGroups * kTileCols <= 256 ? 256u : 512u;      // allocations are powers of two
static_assert(kGroups >= 1 && kGroups * kTileCols <= 512, "a CTA's tiles must fit the 512 TMEM columns of an SM");
// Instruction descriptors: D = fp32 (bit 4), A = B = FP16 (0 at bits 7 and 10), K-major, N >> 3 (bit 17), M >> 4 (bit 24).
constexpr uint32_t kIdescN64 = (1u << 4) | ((64u >> 3) << 17) | ((128u >> 4) << 24);
constexpr long long kWaitCycles = 2000000000ll;   // about a second at the SM clock
constexpr float kTwoLog2e = 2.8853900817779268f;  // 2 log2(e)

struct Smem {
    uint4 a[kGroups][kTile * kChA];  // per tile: operand rows (h hi | h lo), 32 KB; the layer-1 rows in its first 8 KB
    uint4 b1[64 * kCh1];             // layer-1 weights and bias, three FP16 parts paired with the observation's
    uint4 b2[64 * kChA];             // layer-2 weights: hi[64] | lo[64] per output unit
    float bias2c[64];                // b2 * 2 log2(e): added as the constant term of the tanh argument
    float4 w3p[32];                  // output layer in fp32, in the order the four-way tanh delivers h2: entry 2g + u = (W3[0][c], W3[0][c+2], W3[1][c], W3[1][c+2]), c = 4g + u
    float bias3[2];
    uint32_t tmem_slot;              // TMEM base address written by tcgen05.alloc
    uint32_t pad;
    unsigned long long bar[kGroups]; // per tile: mbarrier the tensor core commits to
};

struct Ctx {
    uint32_t tmem;          // this group's accumulator columns, lane 0
    uint32_t parity;        // phase parity of the group's mbarrier
    uint32_t group;
    uint32_t row;           // thread index inside the group
    bool fail;
};

__device__ __forceinline__ float ex2_approx(float x) { float r; asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"(x)); return r; }

// x = p1 + p2 + p3 in FP16 parts (each residual is exact in fp32).
__device__ __forceinline__ void f16_split3(float x, uint16_t &p1, uint16_t &p2, uint16_t &p3)
{
    p1 = f16_bits(x);
    const float r1 = __fsub_rn(x, f16_value(p1));
    p2 = f16_bits(r1);
    p3 = f16_bits(__fsub_rn(r1, f16_value(p2)));
}

// Group barrier (named barrier 1 + group, 128 threads) with an OR reduction of `flag`.
__device__ __forceinline__ bool group_sync_or(uint32_t group, bool flag)
{
    uint32_t out;
    asm volatile("{\n\t.reg .pred p, q;\n\tsetp.ne.u32 q, %2, 0;\n\tbar.red.or.pred p, %1, 128, q;\n\tselp.u32 %0, 1, 0, p;\n\t}"
                 : "=r"(out) : "r"(group + 1u), "r"(flag ? 1u : 0u) : "memory");
    return out != 0u;
}

// Stage the parameters as operand tiles, allocate the accumulator columns, initialise the barriers.
// Called by all threads of the CTA.
__device__ __forceinline__ void setup(const float *__restrict__ p, Smem &s, Ctx &c)
{
    const uint32_t tid = threadIdx.x;
    constexpr uint32_t weight_chunks = 64u * kCh1 + 64u * kChA;    // b1 and b2 are contiguous
    for (uint32_t i = tid; i < weight_chunks; i += kThreads) s.b1[i] = make_uint4(0u, 0u, 0u, 0u);
    __syncthreads();
    for (uint32_t i = tid; i < 256u; i += kThreads) {               // W1[j][k]: columns (w1 w1 w1 w2 w2 w3) x 4
        const uint32_t j = i >> 2, k = i & 3u;
        uint16_t w1, w2, w3;
        f16_split3(p[i], w1, w2, w3);
        tc_put(s.b1, j, k, kCh1, w1); tc_put(s.b1, j, 4u + k, kCh1, w1); tc_put(s.b1, j, 8u + k, kCh1, w1);
        tc_put(s.b1, j, 12u + k, kCh1, w2); tc_put(s.b1, j, 16u + k, kCh1, w2); tc_put(s.b1, j, 20u + k, kCh1, w3);
    }
    for (uint32_t j = tid; j < 64u; j += kThreads) {
        uint16_t q1, q2, q3;
        f16_split3(p[256 + j], q1, q2, q3);
        tc_put(s.b1, j, 24u, kCh1, q1); tc_put(s.b1, j, 25u, kCh1, q2); tc_put(s.b1, j, 26u, kCh1, q3);
        s.bias2c[j] = __fmul_rn(p[4416 + j], kTwoLog2e);
    }
    for (uint32_t i = tid; i < 4096u; i += kThreads) {              // W2[j][k]: hi at column k, lo at column 64 + k
        uint16_t hi, lo;
        f16_split(p[320 + i], hi, lo);
        tc_put(s.b2, i >> 6, i & 63u, kChA, hi); tc_put(s.b2, i >> 6, 64u + (i & 63u), kChA, lo);
    }
    if (tid < 32u) {
        const uint32_t c0 = 4u * (tid >> 1) + (tid & 1u);
        s.w3p[tid] = make_float4(p[4480 + c0], p[4480 + c0 + 2], p[4544 + c0], p[4544 + c0 + 2]);
    }
    if (tid < 2u) s.bias3[tid] = p[4608 + tid];
    if (tid == 0u) {
        for (int g = 0; g < kGroups; ++g)
            asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" :: "r"(smem_u32(&s.bar[g])), "r"(1u) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (tid < 32u) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" :: "r"(smem_u32(&s.tmem_slot)), "r"(kCols) : "memory");
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

// Free the accumulator columns.  Called by all threads of the CTA, after their last policy evaluation.
__device__ __forceinline__ void teardown(Smem &s)
{
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (threadIdx.x < 32)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" :: "r"(s.tmem_slot), "r"(kCols) : "memory");
}

enum : int { LAYER1 = 0, LAYER2 = 1 };

__device__ __forceinline__ void mma_f16(uint32_t tmem, uint64_t da, uint64_t db, uint32_t idesc, bool accumulate)
{
    asm volatile("{\n\t.reg .pred p;\n\tsetp.ne.b32 p, %4, 0;\n\t"
                 "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
                 :: "r"(tmem), "l"(da), "l"(db), "r"(idesc), "r"(accumulate ? 1u : 0u) : "memory");
}

// Publish the group's operand rows, let its first thread issue the contraction of `LAYER` and commit it to the
// group's mbarrier, and wait (bounded) for completion.  Returns false for the whole group when a wait ran out
// earlier; a wait that runs out now sets the status bit and is turned into the group-wide exit by the next call.
template <int LAYER>
__device__ __forceinline__ bool contract(Smem &s, Ctx &c, uint32_t *status)
{
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // my operand row: generic-proxy stores -> async proxy
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");  // my accumulator reads so far are done
    if (group_sync_or(c.group, c.fail)) { c.fail = true; return false; }
    const uint32_t bar = smem_u32(&s.bar[c.group]);
    if (c.row == 0u) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t a_addr = smem_u32(s.a[c.group]);
        constexpr uint32_t slice = 2u * kTcLBO;                       // one K = 16 slice = two core matrices along K
        if (LAYER == LAYER1) {
            const uint32_t b_addr = smem_u32(s.b1);
#pragma unroll
            for (uint32_t k = 0; k < 2u; ++k)
                mma_f16(c.tmem, tc_desc(a_addr + k * slice, kCh1), tc_desc(b_addr + k * slice, kCh1), kIdescN64, k != 0u);
        } else {
            const uint32_t b_addr = smem_u32(s.b2);
#pragma unroll
            for (uint32_t k = 0; k < 4u; ++k) {                       // the small terms first, the leading one last
                const uint64_t a_hi = tc_desc(a_addr + k * slice, kChA), a_lo = tc_desc(a_addr + (4u + k) * slice, kChA);
                const uint64_t b_hi = tc_desc(b_addr + k * slice, kChA), b_lo = tc_desc(b_addr + (4u + k) * slice, kChA);
                mma_f16(c.tmem, a_lo, b_hi, kIdescN64, k != 0u);
                mma_f16(c.tmem, a_hi, b_lo, kIdescN64, true);
            }
#pragma unroll
            for (uint32_t k = 0; k < 4u; ++k)
                mma_f16(c.tmem, tc_desc(a_addr + k * slice, kChA), tc_desc(b_addr + k * slice, kChA), kIdescN64, true);
        }
        asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" :: "r"(bar) : "memory");
    }
    const bool done = mbarrier_wait_bounded(bar, c.parity, kWaitCycles);
    if (!done) { c.fail = true; if (status) atomicOr(status, 1u); }
    c.parity ^= 1u;
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    return true;
}

// tanh of FOUR values given y = 2 log2(e) z: 1 - 2 / (2^y + 1).  The special-function unit is the busiest pipe of this
// kernel, so the four reciprocals share ONE hardware reciprocal.  yA = (a0, a1), yB = (b0, b1) scaled arguments; returns the
// transposed pairs T1 = (tanh a0, tanh b0), T2 = (tanh a1, tanh b1).  With d = 2^y + 1: P = (da0 da1, db0 db1), r = 1 / (PA PB),
// R = r (PB, PA) = (1 / PA, 1 / PB), 1 / d_x0 = R d_x1, 1 / d_x1 = R d_x0.  Arguments are clamped to 30 (tanh is 1 to the last
// bit from 2^y = 2^26 on), so the product of the four stays finite; 2^y = 0 for very negative y gives d = 1 and tanh = -1.
__device__ __forceinline__ void tanh4_from_scaled(f2 yA, f2 yB, f2 &T1, f2 &T2)
{
    const f2 D1 = add2(pk(ex2_approx(fminf(lo(yA), 30.0f)), ex2_approx(fminf(lo(yB), 30.0f))), splat(1.0f));   // (da0, db0)
    const f2 D2 = add2(pk(ex2_approx(fminf(hi(yA), 30.0f)), ex2_approx(fminf(hi(yB), 30.0f))), splat(1.0f));   // (da1, db1)
    const f2 P = mul2(D1, D2);
    const float r = rcp_approx(__fmul_rn(lo(P), hi(P)));
    const f2 R = mul2(splat(r), pk(hi(P), lo(P)));
    T1 = fma2(splat(-2.0f), mul2(R, D2), splat(1.0f));
    T2 = fma2(splat(-2.0f), mul2(R, D1), splat(1.0f));
}

// My accumulator row of layer 1 (64 columns; b1 is already in it) -> tanh -> hi / lo FP16 parts -> my row of the group's
// operand tile for layer 2.
__device__ __forceinline__ void activate(Smem &s, const Ctx &c)
{
    const uint32_t taddr = c.tmem + ((c.row & ~31u) << 16);
    uint4 *row = s.a[c.group] + tc_chunk(c.row, 0u, kChA);
    const f2 scale = splat(kTwoLog2e);
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
                const int col = 32 * half + 16 * q + 8 * h;           // first of these eight columns
                uint32_t hp[4], lp[4];
#pragma unroll
                for (int i = 0; i < 4; i += 2) {
                    f2 y[2];
#pragma unroll
                    for (int u = 0; u < 2; ++u) {
                        const f2 z = pk(__uint_as_float(v[q][8 * h + 2 * (i + u)]), __uint_as_float(v[q][8 * h + 2 * (i + u) + 1]));
                        y[u] = mul2(z, scale);
                    }
                    f2 T1, T2;                                         // (t[c], t[c+2]), (t[c+1], t[c+3]) for c = col + 2 i
                    tanh4_from_scaled(y[0], y[1], T1, T2);
                    f2 H1, H2;                                         // hi parts: 11 significant bits, exact in FP16
                    H1.v = T1.v & 0xFFFFE000FFFFE000ull; H2.v = T2.v & 0xFFFFE000FFFFE000ull;
                    const f2 L1 = sub2(T1, H1), L2 = sub2(T2, H2);
                    hp[i] = pack_f16x2(lo(H1), lo(H2)); hp[i + 1] = pack_f16x2(hi(H1), hi(H2));
                    lp[i] = pack_f16x2(lo(L1), lo(L2)); lp[i + 1] = pack_f16x2(hi(L1), hi(L2));
                }
                row[(col >> 3) * 8] = make_uint4(hp[0], hp[1], hp[2], hp[3]);            // chunk index along K: hi part
                row[(8 + (col >> 3)) * 8] = make_uint4(lp[0], lp[1], lp[2], lp[3]);      // lo part
            }
    }
}

// Output layer on the fp32 pipes: my accumulator row of layer 2 -> + bias -> tanh -> logits = b3 + W3 h2, accumulated
// in packed form (two partial sums per logit, added at the end).  Compared with a third contraction this saves the hi / lo
// split of h2, its shared-memory stores and one more round trip to the tensor core, and is exact up to fp32 rounding.
__device__ __forceinline__ f2 activate_output(const Smem &s, const Ctx &c)
{
    const uint32_t taddr = c.tmem + ((c.row & ~31u) << 16);
    const f2 scale = splat(kTwoLog2e);
    f2 acc0 = pk(s.bias3[0], 0.0f), acc1 = pk(s.bias3[1], 0.0f);
#pragma unroll
    for (int half = 0; half < 2; ++half) {
        uint32_t v[2][16];
        tc_load16(taddr + 32u * (uint32_t)half, v[0]);
        tc_load16(taddr + 32u * (uint32_t)half + 16u, v[1]);
        asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
        for (int q = 0; q < 2; ++q)
#pragma unroll
            for (int i = 0; i < 8; i += 2) {
                const int col = 32 * half + 16 * q + 2 * i;               // columns col .. col + 3
                f2 y[2];
#pragma unroll
                for (int u = 0; u < 2; ++u) {
                    const f2 z = pk(__uint_as_float(v[q][2 * (i + u)]), __uint_as_float(v[q][2 * (i + u) + 1]));
                    const float2 b = *reinterpret_cast<const float2 *>(&s.bias2c[col + 2 * u]);
                    y[u] = fma2(z, scale, pk(b.x, b.y));
                }
                f2 T1, T2;                                                 // (h[col], h[col+2]), (h[col+1], h[col+3])
                tanh4_from_scaled(y[0], y[1], T1, T2);
                const float4 wa = s.w3p[col >> 1], wb = s.w3p[(col >> 1) + 1];
                acc0 = fma2(pk(wa.x, wa.y), T1, acc0); acc1 = fma2(pk(wa.z, wa.w), T1, acc1);
                acc0 = fma2(pk(wb.x, wb.y), T2, acc0); acc1 = fma2(pk(wb.z, wb.w), T2, acc1);
            }
    }
    return pk(__fadd_rn(lo(acc0), hi(acc0)), __fadd_rn(lo(acc1), hi(acc1)));
}

// Logits of this thread's observation; the group's 128 threads evaluate their 128 observations together.
// Returns false for the whole group when a wait ran out.
__device__ __forceinline__ bool policy(const float4 o, Smem &s, Ctx &c, uint32_t *status, f2 &logits)
{
    {   // layer-1 operand row: (o1[4] o2[4]) (o3[4] o1[4]) (o2[4] o1[4]) (1 1 1 0 0 0 0 0), o = o1 + o2 + o3
        const uint32_t a01 = pack_f16x2(o.x, o.y), a23 = pack_f16x2(o.z, o.w);
        const float r0 = __fsub_rn(o.x, f16_value((uint16_t)(a01 & 0xFFFFu))), r1 = __fsub_rn(o.y, f16_value((uint16_t)(a01 >> 16)));
        const float r2 = __fsub_rn(o.z, f16_value((uint16_t)(a23 & 0xFFFFu))), r3 = __fsub_rn(o.w, f16_value((uint16_t)(a23 >> 16)));
        const uint32_t b01 = pack_f16x2(r0, r1), b23 = pack_f16x2(r2, r3);
        const float q0 = __fsub_rn(r0, f16_value((uint16_t)(b01 & 0xFFFFu))), q1 = __fsub_rn(r1, f16_value((uint16_t)(b01 >> 16)));
        const float q2 = __fsub_rn(r2, f16_value((uint16_t)(b23 & 0xFFFFu))), q3 = __fsub_rn(r3, f16_value((uint16_t)(b23 >> 16)));
        const uint32_t c01 = pack_f16x2(q0, q1), c23 = pack_f16x2(q2, q3);
        uint4 *row = s.a[c.group] + tc_chunk(c.row, 0u, kCh1);
        row[0] = make_uint4(a01, a23, b01, b23);
        row[8] = make_uint4(c01, c23, a01, a23);
        row[16] = make_uint4(b01, b23, a01, a23);
        row[24] = make_uint4(0x3C003C00u, 0x00003C00u, 0u, 0u);
    }
    if (!contract<LAYER1>(s, c, status)) return false;
    activate(s, c);
    if (!contract<LAYER2>(s, c, status)) return false;
    logits = activate_output(s, c);
    return true;
}

__global__ void __launch_bounds__(kThreads, TCP_MINBLOCKS)
rollout_cartpole_mlp_tcp_kernel(const __grid_constant__ S4Args a)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    Smem &ms = *reinterpret_cast<Smem *>(smem_raw);
    Ctx ctx;
    setup(a.params, ms, ctx);

    // Every thread takes part in every barrier of its group: threads past the batch shadow the last env and store nothing.
    const uint64_t i64 = (uint64_t)blockIdx.x * kThreads + threadIdx.x;
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
            ok = policy(s, ms, ctx, a.status, l);
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
    teardown(ms);
}

__global__ void __launch_bounds__(kThreads, TCP_MINBLOCKS)
policy_logits_tcp_kernel(const float4 *__restrict__ obs, int64_t M, const float *__restrict__ params, float2 *__restrict__ logits, uint32_t *status)
{
    extern __shared__ __align__(16) unsigned char smem_raw[];
    Smem &ms = *reinterpret_cast<Smem *>(smem_raw);
    Ctx ctx;
    setup(params, ms, ctx);
    const int64_t i = (int64_t)blockIdx.x * kThreads + threadIdx.x;
    const bool valid = i < M;
    f2 l;
    const bool ok = policy(obs[valid ? i : M - 1], ms, ctx, status, l);
    if (valid && ok) logits[i] = make_float2(lo(l), hi(l));
    teardown(ms);
}

// The kernels need more than 48 KB of dynamic shared memory: opt in once per device.
static cudaError_t opt_in()
{
    static std::mutex lock;
    static bool done[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    std::lock_guard<std::mutex> guard(lock);
    if (dev >= 0 && dev < 64 && done[dev]) return cudaSuccess;
    e = cudaFuncSetAttribute(rollout_cartpole_mlp_tcp_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(Smem));
    if (e == cudaSuccess) e = cudaFuncSetAttribute(policy_logits_tcp_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sizeof(Smem));
    if (e == cudaSuccess && dev >= 0 && dev < 64) done[dev] = true;
    return e;
}

}  // namespace tcp

cudaError_t launch_cartpole_mlp_tcp(const S4Args &a, cudaStream_t st)
{
    cudaError_t e = tcp::opt_in();
    if (e != cudaSuccess) return e;
    const unsigned blocks = (unsigned)(((uint64_t)a.n + tcp::kThreads - 1u) / tcp::kThreads);
    tcp::rollout_cartpole_mlp_tcp_kernel<<<blocks, tcp::kThreads, sizeof(tcp::Smem), st>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_policy_logits_tcp(const float *obs, int64_t M, const float *params, float *logits, uint32_t *status, cudaStream_t st)
{
    if (M <= 0) return cudaSuccess;
    cudaError_t e = tcp::opt_in();
    if (e != cudaSuccess) return e;
    const int64_t blocks = (M + tcp::kThreads - 1) / tcp::kThreads;
    if (blocks > 0x7FFFFFFFll) return cudaErrorInvalidConfiguration;
    tcp::policy_logits_tcp_kernel<<<(unsigned)blocks, tcp::kThreads, sizeof(tcp::Smem), st>>>(reinterpret_cast<const float4 *>(obs), M, params,
                                                                                            reinterpret_cast<float2 *>(logits), status);
    return cudaGetLastError();
}

}  // namespace simk
