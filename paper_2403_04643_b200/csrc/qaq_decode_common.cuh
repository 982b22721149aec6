// Pieces shared by the decode kernels (not part of the ABI): the integer tensor-core instruction, the loads that
// turn section words into its operand registers, cp.async staging, the fixed-point outlier sums.
#pragma once
#include "qaq_codec.cuh"
#include "qaq_internal.cuh"

namespace qaqd {

// D(16x8, s32) += A(16x32, u8, row) * B(32x8, s8, col).  Lane = 4*g + t holds
//   a0: row g, k 4t..4t+3   a1: row g+8, k 4t..4t+3   a2: row g, k 16+4t..   a3: row g+8, k 16+4t..   (one k per byte)
//   b0: k 4t..4t+3, column g   b1: k 16+4t.., column g
//   d0, d1: row g, columns 2t, 2t+1   d2, d3: row g+8, columns 2t, 2t+1
__device__ __forceinline__ void mma_u8s8(int (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k32.row.col.s32.u8.s8.s32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+r"(d[0]), "+r"(d[1]), "+r"(d[2]), "+r"(d[3])
                 : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

template <int BYTES>
__device__ __forceinline__ void cp_async(void* smem, const void* gmem) {
    const unsigned s = (unsigned)__cvta_generic_to_shared(smem);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;\n" ::"r"(s), "l"(gmem));
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;\n" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;\n" ::"n"(N) : "memory"); }

// NREG operand registers (one W-bit field per byte lane) with register indices R0 .. R0+NREG-1 of a key plane or
// of a value group (staged in shared memory, or in place in global memory): register R sits in word R / (8/W) at bit W * (R % (8/W)) of every byte.  Nothing is read
// when !ok (the registers are zero).
template <int W, int NREG>
__device__ __forceinline__ void fetch_regs(const uint8_t* base, int R0, bool ok, uint32_t (&reg)[NREG]) {
    constexpr int PER = 8 / W;
    constexpr int NW = NREG >= PER ? NREG / PER : 1;
    constexpr uint32_t MASK = 0x01010101u * ((1u << W) - 1u);
    uint32_t w[NW];
#pragma unroll
    for (int i = 0; i < NW; ++i) w[i] = 0;
    if (ok) qaqc::load_words<NW>(base + 4 * (R0 / PER), w);
    const int f0 = NREG >= PER ? 0 : W * (R0 % PER);     // only a word shared by several lanes starts inside it
#pragma unroll
    for (int r = 0; r < NREG; ++r) {
        if (W == 8) reg[r] = w[r];
        else reg[r] = (w[r / PER] >> (W * (r % PER) + f0)) & MASK;
    }
}

// Fixed-point form of an outlier term for integer atomics: a high part in units of 2^-4 and the exact remainder
// in units of 2^-28.  Terms of 2^18 or more (and non-finite ones) are left out, so that 128 of them stay inside
// 32 bits in both parts.
constexpr float OC_LIMIT = 262144.0f;
__device__ __forceinline__ void outlier_add(int* hi_cell, int* lo_cell, float tm) {
    if (fabsf(tm) < OC_LIMIT) {
        const float hi = rintf(tm * 16.0f);
        const float rem = fmaf(hi, -0.0625f, tm);              // exact, |rem| <= 2^-5
        atomicAdd(hi_cell, (int)hi);
        atomicAdd(lo_cell, __float2int_rn(rem * 268435456.0f));
    }
}
__device__ __forceinline__ float outlier_sum(int hi, int lo) { return fmaf((float)lo, 1.0f / 268435456.0f, (float)hi * 0.0625f); }

}  // namespace qaqd
