// Warp-level 16x8x8 tensor-core products in "3xTF32": every fp32 operand is split into a TF32 head and a TF32
// tail, and a.b is accumulated as a_lo.b_hi + a_hi.b_lo + a_hi.b_hi in fp32.  The dropped tail.tail term is
// ~2^-22 relative and the truncated tails ~2^-21, which keeps the contractions inside the 1e-5 tolerance (a single
// TF32 pass misses it ~40x).
//
// Fragment layout of mma.sync.aligned.m16n8k8.row.col (g = lane / 4, t = lane % 4):
//   A (16x8, row-major):  a0 = A[g][t]      a1 = A[g+8][t]    a2 = A[g][t+4]    a3 = A[g+8][t+4]
//   B (8x8,  k x n):      b0 = B[t][g]      b1 = B[t+4][g]
//   C (16x8):             c0 = C[g][2t]     c1 = C[g][2t+1]   c2 = C[g+8][2t]   c3 = C[g+8][2t+1]
#pragma once
#include <stdint.h>

struct Tf32Pair {
    uint32_t hi, lo;
};

// head = x rounded to TF32 (10 explicit mantissa bits) with integer arithmetic on the bit pattern: add half a TF32
// ulp, clear the 13 low bits.  tail = x - head is exact in fp32 and is handed over as it is: the tensor core reads
// only the TF32 part of an operand register, i.e. it truncates the tail to its own top bits (error <= 2^-21 |x|).
// cvt.rna.tf32.f32 would do the same rounding but runs on the quarter-rate conversion pipe, which made the split
// the bottleneck of the row stage.
__device__ __forceinline__ Tf32Pair tt_split_tf32(float x)
{
    Tf32Pair p;
    p.hi = (__float_as_uint(x) + 0x1000u) & 0xffffe000u;
    p.lo = __float_as_uint(x - __uint_as_float(p.hi));
    return p;
}

__device__ __forceinline__ void tt_mma_tf32(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1)
{
    asm volatile(
        "mma.sync.aligned.m16n8k8.row.col.f32.tf32.tf32.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// d += A.B with A and B given as split fragments (small terms first)
__device__ __forceinline__ void tt_mma_3xtf32(float (&d)[4], const Tf32Pair (&a)[4], const Tf32Pair (&b)[2])
{
    tt_mma_tf32(d, a[0].lo, a[1].lo, a[2].lo, a[3].lo, b[0].hi, b[1].hi);
    tt_mma_tf32(d, a[0].hi, a[1].hi, a[2].hi, a[3].hi, b[0].lo, b[1].lo);
    tt_mma_tf32(d, a[0].hi, a[1].hi, a[2].hi, a[3].hi, b[0].hi, b[1].hi);
}
