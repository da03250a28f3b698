// Pieces shared by the tensor-core policy kernels (tcgen05 on sm_100a): FP16 packing, shared-memory operand
// layout and descriptors, accumulator loads, the bounded mbarrier wait.
//
// Operand layout in shared memory (all operands K-major, no swizzle): 8-row x 16-byte core matrices; the core
// matrices of one 8-row group along K are contiguous (128 bytes apart = leading byte offset), 8-row groups follow
// each other (stride byte offset = 128 bytes x 16-byte chunks per row).
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace simk {

constexpr uint32_t kTcLBO = 128u;                 // bytes between core matrices adjacent along K

__device__ __forceinline__ uint32_t smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
// f16x2 with `first` in the low half (the lower address / lower k).
__device__ __forceinline__ uint32_t pack_f16x2(float first, float second) { uint32_t r; asm("cvt.rn.satfinite.f16x2.f32 %0, %1, %2;" : "=r"(r) : "f"(second), "f"(first)); return r; }
__device__ __forceinline__ uint32_t tanh_f16x2(uint32_t x) { uint32_t r; asm("tanh.approx.f16x2 %0, %1;" : "=r"(r) : "r"(x)); return r; }
__device__ __forceinline__ uint16_t f16_bits(float x) { uint16_t r; asm("cvt.rn.satfinite.f16.f32 %0, %1;" : "=h"(r) : "f"(x)); return r; }
__device__ __forceinline__ float f16_value(uint16_t h) { float r; asm("cvt.f32.f16 %0, %1;" : "=f"(r) : "h"(h)); return r; }
// x = hi + lo with hi = f16(x), lo = f16(x - hi).
__device__ __forceinline__ void f16_split(float x, uint16_t &hi, uint16_t &lo) { hi = f16_bits(x); lo = f16_bits(__fsub_rn(x, f16_value(hi))); }

// Shared-memory matrix descriptor: start address, leading and stride byte offsets (16-byte units),
// descriptor version 1, no swizzle.
__device__ __forceinline__ uint64_t tc_desc(uint32_t saddr, uint32_t chunks_per_row)
{
    return (uint64_t)((saddr >> 4) & 0x3FFFu) | ((uint64_t)(kTcLBO >> 4) << 16) | ((uint64_t)((chunks_per_row * 128u) >> 4) << 32) | (1ull << 46);
}

// Index (in 16-byte chunks) of chunk c of row `row` of an operand tile with `ch` chunks per row.
__device__ __forceinline__ uint32_t tc_chunk(uint32_t row, uint32_t c, uint32_t ch) { return (row >> 3) * ch * 8u + c * 8u + (row & 7u); }

__device__ __forceinline__ void tc_put(uint4 *tile, uint32_t row, uint32_t k, uint32_t ch, uint16_t value)
{
    reinterpret_cast<uint16_t *>(tile + tc_chunk(row, k >> 3, ch))[k & 7u] = value;
}

// Columns 0..15 from `taddr` of this thread's accumulator row.
__device__ __forceinline__ void tc_load16(uint32_t taddr, uint32_t (&v)[16])
{
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                 : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]),
                   "=r"(v[8]), "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
                 : "r"(taddr));
}


// One attempt, then a loop bounded by `wait_cycles` of the SM clock, on the mbarrier at shared address `bar` for the
// phase of parity `parity`.  Returns whether the phase completed.
__device__ __forceinline__ bool mbarrier_wait_bounded(uint32_t bar, uint32_t parity, long long wait_cycles)
{
    uint32_t done = 0u;
    asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.b32 %0, 1, 0, p;\n\t}"
                 : "=r"(done) : "r"(bar), "r"(parity) : "memory");
    if (!done) {                                                       // rare: the first wait timed out inside the hardware
        const long long t0 = clock64();
        do {
            asm volatile("{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\tselp.b32 %0, 1, 0, p;\n\t}"
                         : "=r"(done) : "r"(bar), "r"(parity) : "memory");
        } while (!done && clock64() - t0 <= wait_cycles);
    }
    return done != 0u;
}

}  // namespace simk
