// Intermediate products (paper Sec. 3.2, "Intermediate Computation") of several prefix groups at once on the
// tensor cores.
//
// Groups are walked in digit-major order, so neighbours share the slice B = G_{K-1}[i_{K-1}] (r_a x cols).  With
// P_{K-2} of MROWS = 4 (or 2, 8) rows per group, NG = 16 / MROWS = 4 (or 8, 2) groups stack into one 16 x r_a operand, and
//     [C_0; ..; C_{NG-1}] = [P_0; ..; P_{NG-1}] . B
// is a 16 x cols product of m16n8k8 tiles in 3xTF32 (see mma.cuh).  The slice then enters the SM once per NG
// groups instead of once per group (the FP32-pipe form of this product was bound by the L1 operand path), and the
// product leaves the FP32 pipe.  Groups of the batch that use another slice (a run boundary) are handled in a
// further pass; rows of groups that are not part of a pass are zero and their result is not stored.
#pragma once
#include "mma.cuh"

// One pass.  Lane (g = lane / 4, t = lane % 4) feeds rows g and g + 8 of the stacked operand: row g belongs to group
// g / MROWS (source srcA, taken when selA), row g + 8 to group (8 + g) / MROWS (srcB, selB); m = g % MROWS is the row
// of P inside the group.  src points at P (MROWS x ra, row-major).  ra <= 8 * KTMAX, any value (the k range is padded
// with zeros).  Results go to Cs4 + q * MROWS * COLS + m * COLS + column for group q (C_q as [MROWS][COLS] =
// [PM][RB] row-major).
//
// Column mapping: a block of 32 columns is one float4 load per lane and k row (8 lanes x 16 bytes = 128 bytes per
// row); tile j of the block takes component j, i.e. tile column n' stands for slice column 32 * block + 4 n' + j, so
// that a lane ends up with 8 consecutive columns of each of its two rows (two float4 stores per row).
// RBP > 0: C tiles are stored as [PM][RBP + 4] (rows of r_{K-1} = RBP values padded by four floats), which makes the
// row stage's fragment loads from shared memory conflict-free; RBP = 0: plain [MROWS][COLS] tiles.
template <int COLS, int MROWS, int KTMAX, int RBP = 0>
__device__ __forceinline__ void tt_quad_mid_mma(const float* __restrict__ B, int ra, const float* __restrict__ srcA,
                                                const float* __restrict__ srcB, bool selA, bool selB, float* Cs4, int lane,
                                                int nb0 = 0, int nb1 = COLS / 32)   // column blocks of 32 this warp computes
{
    static_assert((MROWS == 2 || MROWS == 4 || MROWS == 8) && KTMAX % 2 == 0, "stacking of 8, 4 or 2 groups");
    const int g = lane >> 2, t = lane & 3, m = g & (MROWS - 1);
    const int kta = (ra + 7) >> 3;
    // the stacked operand stays unsplit in registers (KTMAX * 4) and is split where it is used: half the registers of
    // pre-split fragments, which buys a resident CTA more per SM
    float araw[KTMAX][4];
#pragma unroll
    for (int kt = 0; kt < KTMAX; ++kt) {
        const int k0 = 8 * kt + t, k1 = k0 + 4;
        araw[kt][0] = (selA && k0 < ra) ? __ldg(srcA + m * ra + k0) : 0.f;
        araw[kt][1] = (selB && k0 < ra) ? __ldg(srcB + m * ra + k0) : 0.f;
        araw[kt][2] = (selA && k1 < ra) ? __ldg(srcA + m * ra + k1) : 0.f;
        araw[kt][3] = (selB && k1 < ra) ? __ldg(srcB + m * ra + k1) : 0.f;
    }
    const float4* __restrict__ B4 = reinterpret_cast<const float4*>(B);
    constexpr int C4N = COLS / 4;
    constexpr int DSUB = RBP > 0 ? COLS / RBP : 1;              // d_{K-1}: rows of C per row of P
    constexpr int TILE = RBP > 0 ? MROWS * DSUB * (RBP + 4) : MROWS * COLS;
    float* dstA = Cs4 + (size_t)(g / MROWS) * TILE + (RBP > 0 ? 0 : m * COLS + 8 * t);
    float* dstB = Cs4 + (size_t)((8 + g) / MROWS) * TILE + (RBP > 0 ? 0 : m * COLS + 8 * t);
    // offset of columns [32 nb + 8 t, + 8) of row m inside a tile
    auto coff = [&](int nb) {
        if (RBP > 0) {
            const int col = 32 * nb + 8 * t;
            return (m * DSUB + col / RBP) * (RBP + 4) + col % RBP;
        }
        return 32 * nb;
    };
#pragma unroll 1
    for (int nb = nb0; nb < nb1; ++nb) {
        float acc[4][4];
#pragma unroll
        for (int j = 0; j < 4; ++j) { acc[j][0] = 0.f; acc[j][1] = 0.f; acc[j][2] = 0.f; acc[j][3] = 0.f; }
#pragma unroll
        for (int kc = 0; kc < KTMAX; kc += 2) {   // two k steps (16 rows of B) in flight at a time
            float4 f[2][2];
#pragma unroll
            for (int kt = 0; kt < 2; ++kt) {
                const int k0 = 8 * (kc + kt) + t, k1 = k0 + 4;
                f[kt][0] = k0 < ra ? __ldg(B4 + (size_t)k0 * C4N + 8 * nb + g) : make_float4(0.f, 0.f, 0.f, 0.f);
                f[kt][1] = k1 < ra ? __ldg(B4 + (size_t)k1 * C4N + 8 * nb + g) : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int kt = 0; kt < 2; ++kt) {
                if (kc + kt < kta) {
                    Tf32Pair a[4];
#pragma unroll
                    for (int x = 0; x < 4; ++x) a[x] = tt_split_tf32(araw[kc + kt][x]);
                    const float v0[4] = {f[kt][0].x, f[kt][0].y, f[kt][0].z, f[kt][0].w};
                    const float v1[4] = {f[kt][1].x, f[kt][1].y, f[kt][1].z, f[kt][1].w};
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        Tf32Pair b[2];
                        b[0] = tt_split_tf32(v0[j]);
                        b[1] = tt_split_tf32(v1[j]);
                        tt_mma_3xtf32(acc[j], a, b);
                    }
                }
            }
        }
        if (selA) {
            *reinterpret_cast<float4*>(dstA + coff(nb)) = make_float4(acc[0][0], acc[1][0], acc[2][0], acc[3][0]);
            *reinterpret_cast<float4*>(dstA + coff(nb) + 4) = make_float4(acc[0][1], acc[1][1], acc[2][1], acc[3][1]);
        }
        if (selB) {
            *reinterpret_cast<float4*>(dstB + coff(nb)) = make_float4(acc[0][2], acc[1][2], acc[2][2], acc[3][2]);
            *reinterpret_cast<float4*>(dstB + coff(nb) + 4) = make_float4(acc[0][3], acc[1][3], acc[2][3], acc[3][3]);
        }
    }
}

// All passes of one batch of cnt <= 16 / MROWS groups.  Lane q < cnt holds group q's slice index (imq) and operand
// pointer (srcq).
template <int COLS, int MROWS, int KTMAX, int RBP = 0>
__device__ __forceinline__ void tt_quad_mid(const float* __restrict__ core_mid, size_t slice_floats, int ra, int cnt, uint32_t imq,
                                            const float* srcq, float* Cs4, int lane)
{
    const int g = lane >> 2;
    const int qA = g / MROWS, qB = (8 + g) / MROWS;
    const unsigned long long sp = (unsigned long long)reinterpret_cast<uintptr_t>(srcq);
    const float* srcA = reinterpret_cast<const float*>((uintptr_t)__shfl_sync(0xffffffffu, sp, qA));
    const float* srcB = reinterpret_cast<const float*>((uintptr_t)__shfl_sync(0xffffffffu, sp, qB));
    unsigned remaining = (1u << cnt) - 1u;
    while (remaining) {
        const int first = __ffs(remaining) - 1;
        const uint32_t im = __shfl_sync(0xffffffffu, imq, first);
        const unsigned sel = __ballot_sync(0xffffffffu, lane < 16 / MROWS && ((remaining >> lane) & 1u) && imq == im) & ((1u << (16 / MROWS)) - 1u);
        const bool selA = (sel >> qA) & 1u, selB = (sel >> qB) & 1u;
        tt_quad_mid_mma<COLS, MROWS, KTMAX, RBP>(core_mid + (size_t)im * slice_floats, ra, srcA, srcB, selA, selB, Cs4, lane);
        remaining &= ~sel;
    }
}
