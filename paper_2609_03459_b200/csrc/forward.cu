// Forward path: cost-balanced schedule, prefix products, fused last-two-level contraction, bag pooling.
//
// Work is organised around the sorted prefix tree built by the grouping pass.  A "group" is a node of
// level K-1 (a distinct (i_1..i_{K-1}) prefix); its children are the distinct rows that share it.
//   * schedule: cost(group) = c_mid + children * c_last (FMA counts), exclusive scan, and every table is
//     cut into `units` slices of equal cost; one CTA per unit, dispatched dynamically by the hardware.
//   * contraction: per group the partial product C = P_{K-2} . G_{K-1}[i_{K-1}] is formed once in shared
//     memory (paper Sec. 3.2 "Intermediate Computation") and every child row E = C . G_K[i_K] is produced
//     from it ("Embedding Computation"); C never goes to global memory.
//   * pooling ("Vector Aggregation"): one warp per bag gathers its rows through the rank structure and
//     reduces them in registers; lanes of different sub-warps are combined with warp shuffles.  No atomics.
#include "common.cuh"
#include "scan.cuh"
#include "mma.cuh"
#include "quad_mid.cuh"

// ---------------------------------------------------------------------------------------------- schedule

struct CostScan {
    WsView w;
    int shift;
    __device__ uint32_t size() const { return w.counters[CTR_LEVEL0 + w.K - 1]; }
    __device__ int locate(uint32_t j0) const { return tt_find_table(w.tb[w.K - 1], w.T, j0); }
    __device__ uint32_t value(uint32_t j, int hint) const
    {
        // position j of the sweep order: digit-major for K >= 3 (groups that share the big slice of core K-1 are
        // neighbours, so that slice is fetched from L2 once per run instead of once per group), natural for K = 2
        const int K = w.K;
        const int t = tt_find_table_from(w.tb[K - 1], w.T, j, hint);
        const uint32_t g = (K >= 3 && !(w.ablation & 1)) ? w.tnode[K - 1][j] : j;
        const TableDesc& td = w.tdesc[t];
        const uint32_t nchild = w.cstart[K - 1][g + 1] - w.cstart[K - 1][g];
        // c_k = P_{k-1} r_{k-1} d_k r_k
        uint64_t c_last = (uint64_t)td.P[K - 1] * td.r[K - 1] * td.d[K - 1];
        uint64_t c_mid = K >= 3 ? (uint64_t)td.P[K - 2] * td.r[K - 2] * td.d[K - 2] * td.r[K - 1] : 0;
        uint64_t c = ((c_mid + (uint64_t)nchild * c_last) >> shift) + 1;
        return (uint32_t)c;
    }
    __device__ void emit(uint32_t g, uint32_t excl, uint32_t, int) const { w.cost[g] = excl; }
    __device__ void total(uint32_t tot) const
    {
        w.cost[size()] = tot;
        w.counters[CTR_COST_TOTAL] = tot;
    }
};

// group range of every work unit (table, q), once per forward: the sweeps of the forward and of the backward read
// two words instead of bisecting the cost array at the start of every CTA (two chains of ~20 dependent loads each:
// contraction 2.27 -> 2.16 ms, backward sweeps 4.49 -> 4.43 ms on the 60-table training step)
__global__ void __launch_bounds__(128) k_unit_ranges(WsView w)
{
    tt_pdl_enter();
    const int total = w.T * w.units_per_table;
    const int u = blockIdx.x * blockDim.x + threadIdx.x;
    if (u >= total) return;
    uint32_t g0, g1;
    tt_unit_range(w, u / w.units_per_table, u % w.units_per_table, g0, g1);
    w.unit_rng[u] = make_uint2(g0, g1);
}

cudaError_t tt_launch_schedule(tt_emb* h, cudaStream_t s)
{
    if (h->K >= 3 && !(h->ablation & 1)) {
        cudaError_t e = tt_launch_tlist(h, h->K - 1, s);
        if (e != cudaSuccess) return e;
    }
    // cost unit: 2^shift FMAs, chosen at create time so that the worst-case total fits 32 bits
    CostScan cs{h->v, h->cost_shift};
    cudaError_t e = tt_scan(cs, h->v.cap[h->v.K - 1], h->v.scan_tmp, s);
    if (e != cudaSuccess) return e;
    const int total = h->T * h->units_per_table;
    if ((e = tt_launch_pdl(k_unit_ranges, dim3((total + 127) / 128), dim3(128), 0, s, h->v)) != cudaSuccess) return e;
    tt_note_launch();
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------- products

// P_k for every level-k node, 2 <= k <= K-2 (only K = 4 has such a level); one CTA per node, grid-stride
__global__ void __launch_bounds__(128) k_mid_level(WsView w, int k)
{
    tt_pdl_enter();
    extern __shared__ float sm[];
    const uint32_t count = w.counters[CTR_LEVEL0 + k];
    for (uint32_t v = blockIdx.x; v < count; v += gridDim.x) {
        const int t = tt_find_table(w.tb[k], w.T, v);
        const TableDesc& td = w.tdesc[t];
        const int kc = k - 1;
        const int M = td.P[kc], ra = td.r[kc], cols = td.d[kc] * td.r[kc + 1];
        const float* src = tt_left_operand(w, td, k, v);
        for (int i = threadIdx.x; i < M * ra; i += blockDim.x) sm[i] = src[i];
        __syncthreads();
        const uint32_t ik = w.val[k][v] % (uint32_t)td.n[kc];
        tt_mid_product(sm, td.core[kc] + (size_t)ik * td.slice_floats[kc], w.pbuf[k] + (size_t)v * w.stride[k], M, ra, cols);
        __syncthreads();
    }
}

// ---- register-tiled warp-level products (fast path) ---------------------------------------------------------
//
// One warp owns one group at a time.  FP32 FMA throughput is only reachable when every float that enters
// a lane's registers feeds >= 4 FMAs (the shared-memory / L1 path delivers 32 floats per clock per SM, the
// FMA pipes retire 128 lane-FMAs per clock), so:
//   * mid product  C = Pl . B : a lane owns 4 (or 8) consecutive columns of B for all M rows of Pl; B streams
//     through once as float4, Pl comes as float4 broadcasts from shared memory.
//   * last product E = C . D  : a lane keeps TP rows of C (TP x RB floats) in registers for the whole group
//     and streams the float4 rows of each child's D slice: 4*TP FMAs per loaded float4; PM/TP lanes cover a
//     row, so a warp produces 32*TP/PM rows at a time and each lane stores 4*TP consecutive floats of E.

// Cs[m*cols + c] = sum_a Pl[m][a] * Bsl[a*cols + c];  As holds Pl transposed: As[a*M + m].
// cols/4 must be a power of two and cols <= 128*CPL.
template <int M, int CPL>
__device__ __forceinline__ void tt_warp_mid(const float* As, const float* __restrict__ Bsl, float* Cs, int ra, int cols, int lane)
{
    const int c4n = cols >> 2;
    const int LA = (c4n / CPL) < 32 ? (c4n / CPL) : 32;  // lanes that cover one row of B
    const int NS = 32 / LA;                              // the a-range is split over NS lane groups
    const int s = lane / LA, ll = lane - s * LA;
    float acc[CPL][M][4];
#pragma unroll
    for (int i = 0; i < CPL; ++i)
#pragma unroll
        for (int m = 0; m < M; ++m) { acc[i][m][0] = 0.f; acc[i][m][1] = 0.f; acc[i][m][2] = 0.f; acc[i][m][3] = 0.f; }
    const float4* __restrict__ B4 = reinterpret_cast<const float4*>(Bsl);
#pragma unroll 16
    for (int a = s; a < ra; a += NS) {
        float4 b[CPL];
#pragma unroll
        for (int i = 0; i < CPL; ++i) b[i] = __ldg(B4 + (size_t)a * c4n + ll + i * LA);
        float av[M];
        if constexpr (M % 4 == 0) {
#pragma unroll
            for (int m4 = 0; m4 < M / 4; ++m4) {
                const float4 t = *reinterpret_cast<const float4*>(As + a * M + 4 * m4);
                av[4 * m4] = t.x; av[4 * m4 + 1] = t.y; av[4 * m4 + 2] = t.z; av[4 * m4 + 3] = t.w;
            }
        } else {
#pragma unroll
            for (int m = 0; m < M; ++m) av[m] = As[a * M + m];
        }
#pragma unroll
        for (int i = 0; i < CPL; ++i)
#pragma unroll
            for (int m = 0; m < M; ++m) {
                acc[i][m][0] = fmaf(av[m], b[i].x, acc[i][m][0]);
                acc[i][m][1] = fmaf(av[m], b[i].y, acc[i][m][1]);
                acc[i][m][2] = fmaf(av[m], b[i].z, acc[i][m][2]);
                acc[i][m][3] = fmaf(av[m], b[i].w, acc[i][m][3]);
            }
    }
    for (int o = LA; o < 32; o <<= 1)
#pragma unroll
        for (int i = 0; i < CPL; ++i)
#pragma unroll
            for (int m = 0; m < M; ++m)
#pragma unroll
                for (int x = 0; x < 4; ++x) acc[i][m][x] += __shfl_xor_sync(0xffffffffu, acc[i][m][x], o);
    if (s == 0) {
#pragma unroll
        for (int i = 0; i < CPL; ++i)
#pragma unroll
            for (int m = 0; m < M; ++m)
                *reinterpret_cast<float4*>(Cs + m * cols + 4 * (ll + i * LA)) = make_float4(acc[i][m][0], acc[i][m][1], acc[i][m][2], acc[i][m][3]);
    }
}

// E rows u0..u1 of the group whose C (PM x RB, row-major) is in Cs.  d_K = 4.
template <int PM, int RB, int TP>
__device__ __forceinline__ void tt_warp_rows(const float* Cs, const WsView& w, const TableDesc& td, uint32_t u0, uint32_t u1,
                                             uint32_t row_base, int lane, int part = 0, int nparts = 1)   // this warp takes every nparts-th batch
{
    constexpr int LR = PM / TP;   // lanes per row
    constexpr int RW = 32 / LR;   // rows per batch
    const int q = lane % LR, slot = lane / LR;
    float c[TP][RB];
#pragma unroll
    for (int i = 0; i < TP; ++i)
#pragma unroll
        for (int b4 = 0; b4 < RB / 4; ++b4) {
            const float4 t = *reinterpret_cast<const float4*>(Cs + (TP * q + i) * RB + 4 * b4);
            c[i][4 * b4] = t.x; c[i][4 * b4 + 1] = t.y; c[i][4 * b4 + 2] = t.z; c[i][4 * b4 + 3] = t.w;
        }
    const int K = w.K;
    const float* __restrict__ GK = td.core[K - 1];
    const uint32_t* __restrict__ rows = w.val[K];
    for (uint32_t ub = u0 + (uint32_t)(part * RW); ub < u1; ub += (uint32_t)(RW * nparts)) {
        const uint32_t u = ub + slot;
        const bool act = u < u1;
        const uint32_t iK = act ? rows[u] - row_base : 0u;
        const float4* __restrict__ D4 = reinterpret_cast<const float4*>(GK + (size_t)iK * (RB * 4));
        float acc[TP][4];
#pragma unroll
        for (int i = 0; i < TP; ++i) { acc[i][0] = 0.f; acc[i][1] = 0.f; acc[i][2] = 0.f; acc[i][3] = 0.f; }
#pragma unroll
        for (int b = 0; b < RB; ++b) {
            const float4 d = __ldg(D4 + b);
#pragma unroll
            for (int i = 0; i < TP; ++i) {
                acc[i][0] = fmaf(c[i][b], d.x, acc[i][0]);
                acc[i][1] = fmaf(c[i][b], d.y, acc[i][1]);
                acc[i][2] = fmaf(c[i][b], d.z, acc[i][2]);
                acc[i][3] = fmaf(c[i][b], d.w, acc[i][3]);
            }
        }
        if (act) {
            float4* e = reinterpret_cast<float4*>(w.E + (size_t)u * (PM * 4) + TP * q * 4);
#pragma unroll
            for (int i = 0; i < TP; ++i) e[i] = make_float4(acc[i][0], acc[i][1], acc[i][2], acc[i][3]);
        }
    }
}

// Tensor-core form of the last product (d_K = 4): E_u[p][j] = sum_b C[p][b] * D_u[b][j] as m16n8k8 tiles with
// M = 16 rows p of C, K = 8 values of b, N = 8 = two child rows x 4 columns j.  The fragments of C (split into TF32
// head and tail) stay in PM*RB/8 registers for the whole group; each child's slice is read exactly once per warp
// (two coalesced 64-byte pieces per load instruction), so the shared-memory / L1 path carries 4x fewer bytes per
// FMA than the FP32-pipe form and a warp needs ~1/3 of its registers.
template <int PM, int RB, int CS = RB>   // CS: row stride of C in shared memory
__device__ __forceinline__ void tt_warp_rows_mma(const float* Cs, const WsView& w, const TableDesc& td, uint32_t u0, uint32_t u1,
                                                 uint32_t row_base, int lane)
{
    static_assert(PM == 4 || PM == 8 || PM % 16 == 0, "C of 4 or 8 rows fills the first rows of one row tile, else whole tiles");
    constexpr bool HALF = PM < 16;          // rows PM..15 of the tile are zero and are not stored
    constexpr int MT = HALF ? 1 : PM / 16, KT = RB / 8;
    const int g = lane >> 2, t = lane & 3;
    const bool rowok = !HALF || g < PM;     // this lane's first row exists
    Tf32Pair a[MT][KT][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int kt = 0; kt < KT; ++kt) {
            a[mt][kt][0] = tt_split_tf32(rowok ? Cs[(16 * mt + g) * CS + 8 * kt + t] : 0.f);
            a[mt][kt][2] = tt_split_tf32(rowok ? Cs[(16 * mt + g) * CS + 8 * kt + t + 4] : 0.f);
            if (HALF) {
                a[mt][kt][1].hi = 0u; a[mt][kt][1].lo = 0u; a[mt][kt][3].hi = 0u; a[mt][kt][3].lo = 0u;
            } else {
                a[mt][kt][1] = tt_split_tf32(Cs[(16 * mt + g + 8) * CS + 8 * kt + t]);
                a[mt][kt][3] = tt_split_tf32(Cs[(16 * mt + g + 8) * CS + 8 * kt + t + 4]);
            }
        }
    const int K = w.K;
    const float* __restrict__ GK = td.core[K - 1];
    const uint32_t* __restrict__ rows = w.val[K];
    const int rb_ = g >> 2, jb = g & 3;   // this lane's B-fragment column: child row rb_ of the pair, output column jb
    const int rc = t >> 1, jc = 2 * (t & 1);  // this lane's C-fragment columns: child row rc, output columns jc, jc+1
    constexpr int NP = MT == 1 ? 3 : 2;   // row pairs in flight (two where C has two row tiles: registers)
    constexpr uint32_t IDC = 32 - 32 % (2 * NP);   // rows per id chunk: a multiple of the rows per iteration
    uint32_t ids = 0, cb = u0;   // last digits of IDC rows at a time, one per lane (the loop takes them by shuffle)
    for (uint32_t ub = u0; ub < u1; ub += 2 * NP) {
        if (ub == cb + IDC || ub == u0) {
            cb = ub;
            ids = (lane < IDC && ub + lane < u1) ? rows[ub + lane] - row_base : 0u;
        }
        float bv[NP][KT][2];
#pragma unroll
        for (int np = 0; np < NP; ++np) {
            // an odd tail (or a missing second pair) repeats the last row; it is computed but not stored
            const uint32_t ul = min(ub + 2 * np + (uint32_t)rb_, u1 - 1);
            const uint32_t iK = __shfl_sync(0xffffffffu, ids, ul - cb);
            const float* __restrict__ Dl = GK + (size_t)iK * (RB * 4) + jb;
#pragma unroll
            for (int kt = 0; kt < KT; ++kt) {
                bv[np][kt][0] = __ldg(Dl + (8 * kt + t) * 4);
                bv[np][kt][1] = __ldg(Dl + (8 * kt + t + 4) * 4);
            }
        }
#pragma unroll
        for (int np = 0; np < NP; ++np) {
            float acc[MT][4];
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) { acc[mt][0] = 0.f; acc[mt][1] = 0.f; acc[mt][2] = 0.f; acc[mt][3] = 0.f; }
#pragma unroll
            for (int kt = 0; kt < KT; ++kt) {
                Tf32Pair b[2];
                b[0] = tt_split_tf32(bv[np][kt][0]);
                b[1] = tt_split_tf32(bv[np][kt][1]);
#pragma unroll
                for (int mt = 0; mt < MT; ++mt) tt_mma_3xtf32(acc[mt], a[mt][kt], b);
            }
            const uint32_t us = ub + 2 * np + (uint32_t)rc;
            if (us < u1) {
                float* e = w.E + (size_t)us * (PM * 4) + jc;
#pragma unroll
                for (int mt = 0; mt < MT; ++mt) {
                    if (rowok) __stcs(reinterpret_cast<float2*>(e + (16 * mt + g) * 4), make_float2(acc[mt][0], acc[mt][1]));
                    if (!HALF) __stcs(reinterpret_cast<float2*>(e + (16 * mt + g + 8) * 4), make_float2(acc[mt][2], acc[mt][3]));
                }
            }
        }
    }
}

// The same product for C of 8 or 4 rows (d_1 d_2 = 8 or 4), where the form above fills half or a quarter of its row
// tile: transposed, E_u[p][j] = sum_b D_u[b][j] * C[p][b] as m16n8k8 tiles with M = 16 = four child rows x 4 columns
// j, K = 8 values of b, N = 8 rows p of C (PM = 4: columns 4..7 are zero operands).  Half the tensor-core
// instructions per row (a quarter for PM = 4); the split fragments of C^T take RB/2 registers.  A lane ends up with
// single floats of four rows of E (p = 2t, 2t+1; column j = g % 4) and stores them as such.
template <int PM, int RB, int CS = RB>
__device__ __forceinline__ void tt_warp_rows_mma_t(const float* Cs, const WsView& w, const TableDesc& td, uint32_t u0, uint32_t u1,
                                                   uint32_t row_base, int lane)
{
    static_assert(PM == 8 || PM == 4, "C of 8 or 4 rows");
    constexpr int KT = RB / 8;
    const int g = lane >> 2, t = lane & 3;
    const bool pok = g < PM;                // this lane's column p of C^T exists
    Tf32Pair cb[KT][2];                     // B[k = b][n = p] = C[p][b]
#pragma unroll
    for (int kt = 0; kt < KT; ++kt) {
        cb[kt][0] = tt_split_tf32(pok ? Cs[g * CS + 8 * kt + t] : 0.f);
        cb[kt][1] = tt_split_tf32(pok ? Cs[g * CS + 8 * kt + t + 4] : 0.f);
    }
    const int K = w.K;
    const float* __restrict__ GK = td.core[K - 1];
    const uint32_t* __restrict__ rows = w.val[K];
    const int q0 = g >> 2, j = g & 3;       // A-fragment rows g and g + 8: child rows q0 and q0 + 2 of the four, column j
    constexpr int NQ = 2;                   // fours of rows in flight
    constexpr uint32_t IDC = 32;            // rows per id chunk: a multiple of the rows per iteration
    uint32_t ids = 0, cbase = u0;           // last digits of IDC rows at a time, one per lane (the loop takes them by shuffle)
    for (uint32_t ub = u0; ub < u1; ub += 4 * NQ) {
        if (ub == cbase + IDC || ub == u0) {
            cbase = ub;
            ids = (ub + lane < u1) ? rows[ub + lane] - row_base : 0u;
        }
        float av[NQ][KT][4];
#pragma unroll
        for (int nq = 0; nq < NQ; ++nq) {
            // a short tail repeats the last row; it is computed but not stored
            const uint32_t ula = min(ub + 4 * nq + (uint32_t)q0, u1 - 1), ulc = min(ub + 4 * nq + (uint32_t)q0 + 2, u1 - 1);
            const uint32_t iKa = __shfl_sync(0xffffffffu, ids, ula - cbase), iKc = __shfl_sync(0xffffffffu, ids, ulc - cbase);
            const float* __restrict__ Da = GK + (size_t)iKa * (RB * 4) + j;
            const float* __restrict__ Dc = GK + (size_t)iKc * (RB * 4) + j;
#pragma unroll
            for (int kt = 0; kt < KT; ++kt) {
                av[nq][kt][0] = __ldg(Da + (8 * kt + t) * 4);
                av[nq][kt][1] = __ldg(Dc + (8 * kt + t) * 4);
                av[nq][kt][2] = __ldg(Da + (8 * kt + t + 4) * 4);
                av[nq][kt][3] = __ldg(Dc + (8 * kt + t + 4) * 4);
            }
        }
#pragma unroll
        for (int nq = 0; nq < NQ; ++nq) {
            float acc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int kt = 0; kt < KT; ++kt) {
                Tf32Pair a[4];
#pragma unroll
                for (int x = 0; x < 4; ++x) a[x] = tt_split_tf32(av[nq][kt][x]);
                tt_mma_3xtf32(acc, a, cb[kt]);
            }
            // acc: E[p = 2t][j], E[2t + 1][j] of child row q0, then of child row q0 + 2
            const uint32_t usa = ub + 4 * nq + (uint32_t)q0, usc = usa + 2;
            if (2 * t < PM) {
                if (usa < u1) {
                    float* e = w.E + (size_t)usa * (PM * 4) + (2 * t) * 4 + j;
                    __stcs(e, acc[0]);
                    __stcs(e + 4, acc[1]);
                }
                if (usc < u1) {
                    float* e = w.E + (size_t)usc * (PM * 4) + (2 * t) * 4 + j;
                    __stcs(e, acc[2]);
                    __stcs(e + 4, acc[3]);
                }
            }
        }
    }
}

// one warp: groups fetched dynamically from the CTA's range through a shared counter
template <int PM, int RB, int TP, int M, int CPL, bool MMA>
__device__ __forceinline__ void tt_sweep_fast(const WsView& w, const TableDesc& td, uint32_t g1, float* As, float* Cs,
                                              uint32_t* next, int lane)
{
    const int K = w.K, km = K - 2;
    const int ra = td.r[km], cols = td.d[km] * RB;
    const uint32_t nK = (uint32_t)td.n[K - 1];
    for (;;) {
        uint32_t g = 0;
        if (lane == 0) g = atomicAdd(next, 1u);
        g = __shfl_sync(0xffffffffu, g, 0);
        if (g >= g1) break;
        if (!(w.ablation & 1)) g = w.tnode[K - 1][g];   // position in the digit-major order -> group
        const uint32_t val = w.val[K - 1][g];
        const float* src = tt_left_operand(w, td, K - 1, g);
        for (int i = lane; i < M * ra; i += 32) {
            const int m = i / ra, a = i - m * ra;
            As[a * M + m] = __ldg(src + i);
        }
        __syncwarp();
        const uint32_t im = val % (uint32_t)td.n[km];
        tt_warp_mid<M, CPL>(As, td.core[km] + (size_t)im * td.slice_floats[km], Cs, ra, cols, lane);
        __syncwarp();
        if constexpr (MMA) tt_warp_rows_mma<PM, RB>(Cs, w, td, w.cstart[K - 1][g], w.cstart[K - 1][g + 1], val * nK, lane);
        else tt_warp_rows<PM, RB, TP>(Cs, w, td, w.cstart[K - 1][g], w.cstart[K - 1][g + 1], val * nK, lane);
        __syncwarp();
    }
}

// Tensor-core variants: a warp takes NG = 16 / MROWS consecutive groups of the digit-major order at a time; their
// intermediate products are formed together (quad_mid.cuh), then each group's rows are produced from its C in shared
// memory: on the tensor cores too (TP = 0), or on the FP32 pipe with TP rows of C per lane where C is too large for
// register-resident fragments.
template <int PM, int RB, int MROWS, int KTMAX, int TP>
__device__ __forceinline__ void tt_sweep_quad(const WsView& w, const TableDesc& td, uint32_t g1, float* Cs4, uint32_t* next, int lane)
{
    constexpr int COLS = PM / MROWS * RB;   // d_{K-1} * r_{K-1}
    constexpr int NG = 16 / MROWS;
    const int K = w.K, km = K - 2;
    const int ra = td.r[km];
    const uint32_t nK = (uint32_t)td.n[K - 1];
    for (;;) {
        uint32_t base = 0;
        if (lane == 0) base = atomicAdd(next, (uint32_t)NG);
        base = __shfl_sync(0xffffffffu, base, 0);
        if (base >= g1) break;
        const int cnt = (int)min((uint32_t)NG, g1 - base);
        uint32_t valq = 0, imq = 0, u0q = 0, u1q = 0;
        const float* srcq = nullptr;
        if (lane < cnt) {
            const uint32_t pos = base + lane;
            const uint32_t gq = (w.ablation & 1) ? pos : w.tnode[K - 1][pos];   // position in the digit-major order -> group
            valq = w.val[K - 1][gq];
            imq = valq % (uint32_t)td.n[km];
            srcq = tt_left_operand(w, td, K - 1, gq);
            u0q = w.cstart[K - 1][gq];
            u1q = w.cstart[K - 1][gq + 1];
        }
        tt_quad_mid<COLS, MROWS, KTMAX, (TP == 0 ? RB : 0)>(td.core[km], td.slice_floats[km], ra, cnt, imq, srcq, Cs4, lane);
        __syncwarp();
        for (int q = 0; q < cnt; ++q) {
            const uint32_t val = __shfl_sync(0xffffffffu, valq, q);
            const uint32_t u0 = __shfl_sync(0xffffffffu, u0q, q), u1 = __shfl_sync(0xffffffffu, u1q, q);
            if constexpr (TP == 0 && PM < 16) tt_warp_rows_mma_t<PM, RB, RB + 4>(Cs4 + (size_t)q * (PM * (RB + 4)), w, td, u0, u1, val * nK, lane);
            else if constexpr (TP == 0) tt_warp_rows_mma<PM, RB, RB + 4>(Cs4 + (size_t)q * (PM * (RB + 4)), w, td, u0, u1, val * nK, lane);
            else tt_warp_rows<PM, RB, TP>(Cs4 + (size_t)q * (PM * RB), w, td, u0, u1, val * nK, lane);
        }
        __syncwarp();
    }
}

// Stacked product of two 8-row groups against this warp's 64 columns of the slice B (ra <= 64 rows, COLS columns): the
// 64 x 64 block is fetched into shared memory in one go (32 cp.async per lane, one L2 round trip instead of one per 16
// rows and 32 columns), then the 3xTF32 tiles run from shared memory.  Row stride 68 floats: fragment loads 2-way at worst.
template <int COLS>
__device__ __forceinline__ void tt_pair_mid_staged(const float* __restrict__ B, int ra, const float* __restrict__ srcA,
                                                   const float* __restrict__ srcB, bool selA, bool selB, float* Cs2, float* stg,
                                                   int lane, int wid, bool stage)
{
    constexpr int RS = 68;
    const int g = lane >> 2, t = lane & 3;
    const int c0 = 64 * wid;   // first column of this warp's block
    if (stage)                 // (the block of the previous pair is still there when the pair shares its slice)
        for (int i = lane; i < 64 * 16; i += 32) {
            const int k = i >> 4, f = i & 15;
            if (k < ra) tt_cp_async16(stg + k * RS + 4 * f, B + (size_t)k * COLS + c0 + 4 * f);
        }
    asm volatile("cp.async.commit_group;" ::: "memory");
    float araw[8][4];   // rows g (first group) and g + 8 (second group) of the stacked operand, unsplit
#pragma unroll
    for (int kt = 0; kt < 8; ++kt) {
        const int k0 = 8 * kt + t, k1 = k0 + 4;
        araw[kt][0] = (selA && k0 < ra) ? __ldg(srcA + g * ra + k0) : 0.f;
        araw[kt][1] = (selB && k0 < ra) ? __ldg(srcB + g * ra + k0) : 0.f;
        araw[kt][2] = (selA && k1 < ra) ? __ldg(srcA + g * ra + k1) : 0.f;
        araw[kt][3] = (selB && k1 < ra) ? __ldg(srcB + g * ra + k1) : 0.f;
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
    __syncwarp();
    const int kta = (ra + 7) >> 3;
    float* dstA = Cs2 + g * COLS + c0 + 8 * t;                  // group 0, row g of P
    float* dstB = Cs2 + (size_t)8 * COLS + g * COLS + c0 + 8 * t;   // group 1
#pragma unroll 1
    for (int nb = 0; nb < 2; ++nb) {
        float acc[4][4];
#pragma unroll
        for (int j = 0; j < 4; ++j) { acc[j][0] = 0.f; acc[j][1] = 0.f; acc[j][2] = 0.f; acc[j][3] = 0.f; }
#pragma unroll
        for (int kt = 0; kt < 8; ++kt) {
            if (kt < kta) {
                const int k0 = 8 * kt + t, k1 = k0 + 4;
                const float4 f0 = k0 < ra ? *reinterpret_cast<const float4*>(stg + k0 * RS + 32 * nb + 4 * g) : make_float4(0.f, 0.f, 0.f, 0.f);
                const float4 f1 = k1 < ra ? *reinterpret_cast<const float4*>(stg + k1 * RS + 32 * nb + 4 * g) : make_float4(0.f, 0.f, 0.f, 0.f);
                Tf32Pair a[4];
#pragma unroll
                for (int x = 0; x < 4; ++x) a[x] = tt_split_tf32(araw[kt][x]);
                const float v0[4] = {f0.x, f0.y, f0.z, f0.w};
                const float v1[4] = {f1.x, f1.y, f1.z, f1.w};
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    Tf32Pair b[2];
                    b[0] = tt_split_tf32(v0[j]);
                    b[1] = tt_split_tf32(v1[j]);
                    tt_mma_3xtf32(acc[j], a, b);
                }
            }
        }
        if (selA) {
            *reinterpret_cast<float4*>(dstA + 32 * nb) = make_float4(acc[0][0], acc[1][0], acc[2][0], acc[3][0]);
            *reinterpret_cast<float4*>(dstA + 32 * nb + 4) = make_float4(acc[0][1], acc[1][1], acc[2][1], acc[3][1]);
        }
        if (selB) {
            *reinterpret_cast<float4*>(dstB + 32 * nb) = make_float4(acc[0][2], acc[1][2], acc[2][2], acc[3][2]);
            *reinterpret_cast<float4*>(dstB + 32 * nb + 4) = make_float4(acc[0][3], acc[1][3], acc[2][3], acc[3][3]);
        }
    }
    __syncwarp();   // the block is overwritten by the next call
}

// Rank-64 four-core shape: the stage K-1 product of one group is 8 x 64 by 64 x 256 and there are few groups (tens of
// thousands), so the whole CTA works on one pair of groups at a time: the four warps each compute two of the eight
// column blocks of the stacked 16-row tensor-core product into one shared C buffer (16 KB per CTA instead of per
// warp), then two warps per group produce its rows.  Four times the parallelism per pair of the warp-per-pair form.
template <int PM, int RB>
__device__ __forceinline__ void tt_sweep_pair_cta(const WsView& w, const TableDesc& td, uint32_t g0, uint32_t g1, float* Cs2,
                                                  int lane, int wid)
{
    constexpr int MROWS = 8, COLS = PM / MROWS * RB;
    static_assert(COLS == 256, "four warps x 64 columns");
    __shared__ uint32_t m_val[2], m_im[2], m_u0[2], m_u1[2];
    __shared__ const float* m_src[2];
    const int K = w.K, km = K - 2;
    const int ra = td.r[km];
    const uint32_t nK = (uint32_t)td.n[K - 1];
    uint32_t staged = 0xffffffffu;   // slice whose blocks the warps hold in shared memory (the same for all four warps)
    for (uint32_t base = g0; base < g1; base += 2) {
        const int cnt = (int)min(2u, g1 - base);
        if (threadIdx.x < 2) {
            const int q = threadIdx.x;
            if (q < cnt) {
                const uint32_t pos = base + q;
                const uint32_t gq = (w.ablation & 1) ? pos : w.tnode[K - 1][pos];
                const uint32_t v = w.val[K - 1][gq];
                m_val[q] = v;
                m_im[q] = v % (uint32_t)td.n[km];
                m_src[q] = tt_left_operand(w, td, K - 1, gq);
                m_u0[q] = w.cstart[K - 1][gq];
                m_u1[q] = w.cstart[K - 1][gq + 1];
            } else {
                m_val[q] = 0; m_im[q] = 0xffffffffu; m_src[q] = nullptr; m_u0[q] = 0; m_u1[q] = 0;
            }
        }
        __syncthreads();
        const float* B0 = td.core[km] + (size_t)m_im[0] * td.slice_floats[km];
        float* stg = Cs2 + 2 * PM * RB + (size_t)wid * (64 * 68);   // this warp's staged 64 x 64 block of the slice
        // neighbouring pairs of the digit-major order share the slice: its 64 KB are fetched again only when it changes
        if (cnt == 2 && m_im[1] == m_im[0]) {
            tt_pair_mid_staged<COLS>(B0, ra, m_src[0], m_src[1], true, true, Cs2, stg, lane, wid, staged != m_im[0]);
            staged = m_im[0];
        } else {
            tt_pair_mid_staged<COLS>(B0, ra, m_src[0], m_src[1], true, false, Cs2, stg, lane, wid, staged != m_im[0]);
            staged = m_im[0];
            if (cnt == 2) {
                tt_pair_mid_staged<COLS>(td.core[km] + (size_t)m_im[1] * td.slice_floats[km], ra, m_src[0], m_src[1], false, true, Cs2,
                                         stg, lane, wid, true);
                staged = m_im[1];
            }
        }
        __syncthreads();
        {
            const int q = wid >> 1;   // warps 0,1: first group; warps 2,3: second group
            if (q < cnt) tt_warp_rows<PM, RB, 2>(Cs2 + (size_t)q * (PM * RB), w, td, m_u0[q], m_u1[q], m_val[q] * nK, lane, wid & 1, 2);
        }
        __syncthreads();
    }
}

// generic fallback: the whole CTA works on one group at a time (any shape)
__device__ __forceinline__ void tt_sweep_generic(const WsView& w, const TableDesc& td, uint32_t g0, uint32_t g1, float* Pl, float* Cs)
{
    const int K = w.K, kl = K - 1, km = K - 2;
    const int Pm = td.P[K - 1], rb = td.r[K - 1], dK = td.d[kl], D = w.D;
    const uint32_t nK = (uint32_t)td.n[kl];
    for (uint32_t jpos = g0; jpos < g1; ++jpos) {
        const uint32_t g = (K >= 3 && !(w.ablation & 1)) ? w.tnode[K - 1][jpos] : jpos;
        const uint32_t val = w.val[K - 1][g];
        if (K >= 3) {
            const int M = td.P[km], ra = td.r[km], cols = td.d[km] * rb;
            const float* src = tt_left_operand(w, td, K - 1, g);
            for (int i = threadIdx.x; i < M * ra; i += blockDim.x) Pl[i] = src[i];
            __syncthreads();
            const uint32_t im = val % (uint32_t)td.n[km];
            tt_mid_product(Pl, td.core[km] + (size_t)im * td.slice_floats[km], Cs, M, ra, cols);
        } else {
            const float* src = td.core[0] + (size_t)val * td.slice_floats[0];
            for (int i = threadIdx.x; i < Pm * rb; i += blockDim.x) Cs[i] = src[i];
        }
        __syncthreads();
        const uint32_t u0 = w.cstart[K - 1][g], u1 = w.cstart[K - 1][g + 1];
        const int items = (int)(u1 - u0) * D;
        for (int it = threadIdx.x; it < items; it += blockDim.x) {
            const int rr = it / D, e = it - rr * D;
            const int p = e / dK, j = e - p * dK;
            const uint32_t u = u0 + rr;
            const uint32_t iK = w.val[K][u] % nK;
            const float* Dsl = td.core[kl] + (size_t)iK * td.slice_floats[kl];
            const float* c = Cs + p * rb;
            float acc = 0.f;
            for (int b = 0; b < rb; ++b) acc = fmaf(c[b], __ldg(Dsl + b * dK + j), acc);
            w.E[(size_t)u * D + e] = acc;
        }
        __syncthreads();
    }
}

// fused levels K-1 and K: C stays on chip, rows go to w.E.  One CTA (4 warps) per work unit (table, q);
// one instantiation per shape variant V so that each gets its own register budget.  blockIdx.y walks the
// tables of variant V (w.vlist), blockIdx.x the table's equal-cost slices.
template <int V>
__global__ void __launch_bounds__(128, (V >= 0 && V != 3 && V != 4) ? 6 : 1) k_sweep_fwd(WsView w, int pl_floats, int c_floats, int vbase)
{
    tt_pdl_enter();
    extern __shared__ __align__(16) float sm[];
    __shared__ uint32_t next;
    const int t = w.vlist[vbase + blockIdx.y];
    const uint2 rng = w.unit_rng[t * w.units_per_table + blockIdx.x];
    const uint32_t g0 = rng.x, g1 = rng.y;
    const TableDesc& td = w.tdesc[t];
    if (V < 0) {
        tt_sweep_generic(w, td, g0, g1, sm, sm + pl_floats);
        return;
    }
    if (threadIdx.x == 0) next = g0;
    __syncthreads();
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    if (V == 0) tt_sweep_quad<16, 32, 4, 4, 0>(w, td, g1, sm + (size_t)wid * (4 * 16 * 36), &next, lane);
    if (V == 1) tt_sweep_quad<16, 16, 4, 4, 0>(w, td, g1, sm + (size_t)wid * (4 * 16 * 20), &next, lane);
    if (V == 3) tt_sweep_quad<32, 32, 4, 4, 0>(w, td, g1, sm + (size_t)wid * (4 * 32 * 36), &next, lane);
    if (V == 4) tt_sweep_pair_cta<32, 64>(w, td, g0, g1, sm, lane, wid);
    float* As = sm + (size_t)wid * (pl_floats + c_floats);
    float* Cs = As + pl_floats;
    if (V == 2) tt_sweep_quad<16, 8, 4, 4, 0>(w, td, g1, sm + (size_t)wid * (4 * 16 * 12), &next, lane);
    if (V == 5) tt_sweep_quad<8, 32, 2, 4, 0>(w, td, g1, sm + (size_t)wid * (8 * 8 * 36), &next, lane);
    if (V == 6) tt_sweep_quad<8, 16, 2, 4, 0>(w, td, g1, sm + (size_t)wid * (8 * 8 * 20), &next, lane);
    if (V == 7) tt_sweep_quad<8, 8, 2, 4, 0>(w, td, g1, sm + (size_t)wid * (8 * 8 * 12), &next, lane);
    if (V == 8) tt_sweep_quad<4, 32, 2, 4, 0>(w, td, g1, sm + (size_t)wid * (8 * 4 * 36), &next, lane);
    if (V == 9) tt_sweep_quad<4, 16, 2, 4, 0>(w, td, g1, sm + (size_t)wid * (8 * 4 * 20), &next, lane);
    if (V == 10) tt_sweep_fast<4, 8, 2, 2, 1, false>(w, td, g1, As, Cs, &next, lane);
}

// dynamic shared memory of k_sweep_fwd<V> / k_sweep_bwd<V>: four C tiles per warp for the tensor-core variants
static size_t tt_sweep_smem(int V, int max_pl, int max_c)
{
    if (V == 0) return (size_t)4 * 4 * 16 * 36 * sizeof(float);   // C rows padded by four floats (conflict-free fragment loads)
    if (V == 1) return (size_t)4 * 4 * 16 * 20 * sizeof(float);
    if (V == 3) return (size_t)4 * 4 * 32 * 36 * sizeof(float);
    if (V == 5) return (size_t)4 * 8 * 8 * 36 * sizeof(float);    // eight C tiles of 8 rows per warp
    if (V == 6) return (size_t)4 * 8 * 8 * 20 * sizeof(float);
    if (V == 2) return (size_t)4 * 4 * 16 * 12 * sizeof(float);
    if (V == 7) return (size_t)4 * 8 * 8 * 12 * sizeof(float);
    if (V == 8) return (size_t)4 * 8 * 4 * 36 * sizeof(float);
    if (V == 9) return (size_t)4 * 8 * 4 * 20 * sizeof(float);
    if (V == 4) return (size_t)(2 * 32 * 64 + 4 * 64 * 68) * sizeof(float);   // one pair of C tiles per CTA + a staged slice block per warp
    return (size_t)4 * (max_pl + max_c) * sizeof(float);
}

template <int V>
static cudaError_t launch_sweep_fwd(tt_emb* h, int max_pl, int max_c, cudaStream_t s)
{
    const int n = h->vcount[V + 1];
    if (n == 0) return cudaSuccess;
    const size_t smem = tt_sweep_smem(V, max_pl, max_c);
    cudaError_t e = cudaFuncSetAttribute(k_sweep_fwd<V>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    if ((e = tt_stage_begin(h, 9 + V + 1, s)) != cudaSuccess) return e;
    if ((e = tt_launch_pdl(k_sweep_fwd<V>, dim3(h->units_per_table, n), dim3(128), smem, s, h->v, max_pl, max_c, h->vbase[V + 1])) != cudaSuccess) return e;
    tt_note_launch();
    if ((e = tt_stage_end(h, 9 + V + 1, s)) != cudaSuccess) return e;
    return cudaGetLastError();
}

cudaError_t tt_launch_contraction(tt_emb* h, cudaStream_t s)
{
    WsView& w = h->v;
    int max_pl = 4, max_c = 4;
    for (int t = 0; t < h->T; ++t) {
        const TableDesc& td = h->tab[t];
        for (int k = 1; k < h->K; ++k) {
            int f = (td.P[k] * td.r[k] + 3) / 4 * 4;
            if (k <= h->K - 2 && f > max_pl) max_pl = f;
            if (k == h->K - 1 && f > max_c) max_c = f;
        }
    }
    for (int k = 2; k <= h->K - 2; ++k) {
        int grid = h->sm_count * 16;
        cudaError_t e0 = tt_launch_pdl(k_mid_level, dim3(grid), dim3(128), (size_t)max_pl * sizeof(float), s, w, k);
        if (e0 != cudaSuccess) return e0;
        tt_note_launch();
    }
    cudaError_t e;
    // tables of different shape variants are independent: their kernels run side by side on forked streams
    int nvar = 0;
    for (int vi = 0; vi <= TT_NUM_VARIANTS; ++vi) nvar += h->vcount[vi] > 0 ? 1 : 0;
    const bool fork = nvar > 1 && !h->serial;
    if (fork && (e = tt_fork(h, s, 4)) != cudaSuccess) return e;
    int slot = 0;
    auto next_stream = [&](int vi) { return (fork && h->vcount[vi] > 0) ? h->side[(slot++) & 3] : s; };
    if ((e = launch_sweep_fwd<-1>(h, max_pl, max_c, next_stream(0))) != cudaSuccess) return e;
    if ((e = launch_sweep_fwd<0>(h, max_pl, max_c, next_stream(1))) != cudaSuccess) return e;
    if ((e = launch_sweep_fwd<1>(h, max_pl, max_c, next_stream(2))) != cudaSuccess) return e;
    if ((e = launch_sweep_fwd<2>(h, max_pl, max_c, next_stream(3))) != cudaSuccess) return e;
    if ((e = launch_sweep_fwd<3>(h, max_pl, max_c, next_stream(4))) != cudaSuccess) return e;
    if ((e = launch_sweep_fwd<4>(h, max_pl, max_c, next_stream(5))) != cudaSuccess) return e;
    if ((e = launch_sweep_fwd<5>(h, max_pl, max_c, next_stream(6))) != cudaSuccess) return e;
    if ((e = launch_sweep_fwd<6>(h, max_pl, max_c, next_stream(7))) != cudaSuccess) return e;
    if ((e = launch_sweep_fwd<7>(h, max_pl, max_c, next_stream(8))) != cudaSuccess) return e;
    if ((e = launch_sweep_fwd<8>(h, max_pl, max_c, next_stream(9))) != cudaSuccess) return e;
    if ((e = launch_sweep_fwd<9>(h, max_pl, max_c, next_stream(10))) != cudaSuccess) return e;
    if ((e = launch_sweep_fwd<10>(h, max_pl, max_c, next_stream(11))) != cudaSuccess) return e;
    if (fork && (e = tt_join(h, s, 4)) != cudaSuccess) return e;
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------- pooling

// One warp per bag.  A row of D floats is read as D/4 float4 chunks by a sub-warp of LPR lanes
// (LPR = power of two >= min(32, D/4)); 32/LPR rows are fetched per load instruction, up to NF such
// instructions are issued back to back before any result is consumed (the kernel is bound by memory
// latency, so bytes in flight per warp are what counts), the rank look-ups of the next 32 lookups are
// started before the current ones are gathered, and the sub-warps' partial sums are combined with
// __shfl_xor at the end.
__device__ __forceinline__ uint32_t tt_lookup_slot(const WsView& w, const TableDesc& td, int64_t l, uint32_t capK)
{
    const int64_t g = tt_index<true>(w, l);    // streamed once: evict-first, keeps L2 for rows and rank words
    uint32_t slot = 0xffffffffu;
    if (w.ablation & 4) return (g >= 0 && g < td.N && l < (int64_t)capK) ? (uint32_t)l : slot;   // no de-duplication: lookup l is row slot l
    if (g >= 0 && g < td.N) {
        const uint2 e = __ldg(&w.bm[td.word_base + ((uint32_t)g >> 5)]);
        if (e.x >> (g & 31) & 1u) {
            slot = e.y + __popc(e.x & ((1u << (g & 31)) - 1u));
            if (slot >= capK) slot = 0xffffffffu;
        }
    }
    return slot;
}

// Pooling partition: the lookups are cut into C = W * chunks equal shares of whole bags (k_pool_bounds), and the
// warps take the shares in order from a counter.  All resident warps therefore work inside one moving window of
// about W shares at a time - a few tables - so the rows that several bags share are still in L2 when the next
// bag asks for them; one contiguous share per warp would spread the warps over all tables at once.  Equal lookups are
// not equal time (a share of popular rows is served by L2, one of unpopular rows by HBM): with a fixed assignment the
// first warp finished at 84 % of the kernel, the median one at 90 %.  Eight shares per warp: more of them cost more
// in pipeline fill and drain per share than they give in balance (4 / 8 / 16 / 32: 2.62 / 2.39 / 2.50 / 2.76 ms).
#define TT_POOL_MAX_CHUNKS 8
__host__ __device__ __forceinline__ int64_t tt_pool_chunks(int64_t L, int64_t W)
{
    int64_t c = L / (W * 512);                          // at least 512 lookups per share
    c = c < 1 ? 1 : (c > TT_POOL_MAX_CHUNKS ? TT_POOL_MAX_CHUNKS : c);
    while (W * c > TT_POOL_MAX_SHARES && c > 1) --c;
    return c;
}

// first bag of every share: share ci starts at the first bag whose offset is >= L ci / C (the same search for both
// neighbours of a boundary, whatever the offsets hold).  One thread per boundary: the bisections (21 dependent loads for
// two million bags) run side by side here instead of at the start of every share in the pooling warps.
__global__ void __launch_bounds__(256) k_pool_bounds(WsView w, int64_t C)
{
    tt_pdl_enter();
    const int64_t nb = (int64_t)w.T * w.B;
    for (int64_t ci = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; ci <= C; ci += (int64_t)gridDim.x * blockDim.x) {
        const int64_t target = (w.L * ci) / C;
        int64_t lo = 0, hi = nb;
        while (lo < hi) {
            const int64_t mid = (lo + hi) >> 1;
            if (__ldg(w.offsets + mid) < target) lo = mid + 1; else hi = mid;
        }
        w.pool_bounds[ci] = ci == 0 ? 0 : (ci == C ? nb : lo);
    }
}

static cudaError_t launch_pool_bounds(tt_emb* h, int64_t W, cudaStream_t s)
{
    const int64_t C = W * tt_pool_chunks(h->v.L, W);
    const int64_t want = (C + 1 + 255) / 256;
    const int grid = (int)(want < (int64_t)h->sm_count * 8 ? want : (int64_t)h->sm_count * 8);
    cudaError_t e = tt_launch_pdl(k_pool_bounds, dim3(grid), dim3(256), 0, s, h->v, C);
    if (e == cudaSuccess) tt_note_launch();
    return e;
}

template <int LPR, int CPL, bool WT>  // lanes per row, float4 chunks per lane, weighted / mean pooling
__global__ void __launch_bounds__(256, (CPL == 1 ? 6 : (CPL == 2 ? 2 : 1))) k_pool_vec(WsView w, float* __restrict__ out)
{
    tt_pdl_enter();
    const int lane = threadIdx.x & 31;
    const int sub = lane / LPR, lr = lane % LPR;
    constexpr int RPI = 32 / LPR;                       // rows per load instruction
    constexpr int NIT = 32 / RPI;                       // load instructions per 32 lookups
    constexpr int NF = NIT < 4 ? NIT : 4;               // load instructions in flight
    const int D4 = w.D >> 2;
    const float4* __restrict__ E4 = reinterpret_cast<const float4*>(w.E);
    const uint32_t capK = w.cap[w.K];
    // Skew-aware split: the grid is exactly resident (persistent warps); a share holds the bags whose first
    // lookup falls into it (offsets is the cost prefix sum).
    const int64_t W = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const int64_t C = W * tt_pool_chunks(w.L, W);
    auto clampL = [&](int64_t x) { return x < 0 ? (int64_t)0 : (x > w.L ? w.L : x); };
    for (;;) {
    // shares are handed out in order through a counter: a warp whose shares hold popular (L2-resident) rows takes more of them
    int64_t ci = 0;
    if (lane == 0) ci = (int64_t)atomicAdd(&w.counters[CTR_POOL_NEXT], 1u);
    ci = __shfl_sync(0xffffffffu, ci, 0);
    if (ci >= C) break;
    const int64_t b0 = __ldg(w.pool_bounds + ci), b1 = __ldg(w.pool_bounds + ci + 1);
    if (b0 >= b1) continue;
    // every bag is summed over its own (offsets[bag], offsets[bag + 1]) pair, clamped to [0, L]; an inverted pair (malformed
    // offsets) is an empty bag.  o_next: start of the next bag = this bag's end as stored, before the inversion fix
    int64_t o_lo = clampL(__ldg(w.offsets + b0)), o_next = clampL(__ldg(w.offsets + b0 + 1));
    int64_t o_hi = o_next < o_lo ? o_lo : o_next;
    int t = (int)(b0 / w.B);
    uint32_t slot_next;
    float wt_next = 1.f;
    auto fetch = [&](int64_t base, int64_t lim, int tt) {   // rank look-up (and weight) of lookup base + lane
        slot_next = (base + lane < lim) ? tt_lookup_slot(w, w.tdesc[tt], base + lane, capK) : 0xffffffffu;
        if (WT) wt_next = (w.psw && base + lane < lim) ? __ldg(w.psw + base + lane) : 1.f;
    };
    fetch(o_lo, o_hi, t);
    for (int64_t bag = b0; bag < b1; ++bag) {
        const int64_t b = bag - (int64_t)t * w.B;
        // next bag (for the prefetch of its first 32 rank look-ups)
        const bool has_next = bag + 1 < b1;
        const int64_t n_lo = o_next;
        const int64_t n_next = has_next ? clampL(__ldg(w.offsets + bag + 2)) : o_next;
        const int64_t n_hi = n_next < n_lo ? n_lo : n_next;
        const int tn = (has_next && b + 1 == w.B) ? t + 1 : t;
        float4 acc[CPL];
#pragma unroll
        for (int c = 0; c < CPL; ++c) acc[c] = make_float4(0.f, 0.f, 0.f, 0.f);
        if (o_lo >= o_hi && has_next) fetch(n_lo, n_hi, tn);
        for (int64_t l0 = o_lo; l0 < o_hi; l0 += 32) {
            const uint32_t slot = slot_next;
            const float wt = wt_next;
            if (w.upairs && l0 + lane < o_hi) __stcs(&w.upairs[l0 + lane], make_uint2(slot, (uint32_t)b));  // kept for the backward sort
            if (l0 + 32 < o_hi) fetch(l0 + 32, o_hi, t);
            else if (has_next) fetch(n_lo, n_hi, tn);
            const int n = (int)min((int64_t)32, o_hi - l0);
            float4 part[CPL];   // two-level sum: per-batch partial, added to the bag's sum once per batch
#pragma unroll
            for (int c = 0; c < CPL; ++c) part[c] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
            for (int j0 = 0; j0 < NIT; j0 += NF) {
                if (j0 * RPI >= n) break;
                float4 v[NF][CPL];
#pragma unroll
                for (int jj = 0; jj < NF; ++jj) {
                    const int j = (j0 + jj) * RPI + sub;
                    const uint32_t sl = __shfl_sync(0xffffffffu, slot, j & 31);
                    const bool ok = j < n && sl != 0xffffffffu;
                    const float4* row = E4 + (size_t)(ok ? sl : 0u) * D4;
#pragma unroll
                    for (int c = 0; c < CPL; ++c) {
                        const int ch = lr + c * LPR;
                        v[jj][c] = (ok && ch < D4) ? __ldg(row + ch) : make_float4(0.f, 0.f, 0.f, 0.f);
                    }
                }
#pragma unroll
                for (int jj = 0; jj < NF; ++jj) {
                    const float wj = WT ? __shfl_sync(0xffffffffu, wt, ((j0 + jj) * RPI + sub) & 31) : 1.f;
#pragma unroll
                    for (int c = 0; c < CPL; ++c) {
                        if (WT) {
                            part[c].x = fmaf(wj, v[jj][c].x, part[c].x); part[c].y = fmaf(wj, v[jj][c].y, part[c].y);
                            part[c].z = fmaf(wj, v[jj][c].z, part[c].z); part[c].w = fmaf(wj, v[jj][c].w, part[c].w);
                        } else {
                            part[c].x += v[jj][c].x; part[c].y += v[jj][c].y; part[c].z += v[jj][c].z; part[c].w += v[jj][c].w;
                        }
                    }
                }
            }
#pragma unroll
            for (int c = 0; c < CPL; ++c) { acc[c].x += part[c].x; acc[c].y += part[c].y; acc[c].z += part[c].z; acc[c].w += part[c].w; }
        }
#pragma unroll
        for (int o = LPR; o < 32; o <<= 1) {
#pragma unroll
            for (int c = 0; c < CPL; ++c) {
                acc[c].x += __shfl_xor_sync(0xffffffffu, acc[c].x, o);
                acc[c].y += __shfl_xor_sync(0xffffffffu, acc[c].y, o);
                acc[c].z += __shfl_xor_sync(0xffffffffu, acc[c].z, o);
                acc[c].w += __shfl_xor_sync(0xffffffffu, acc[c].w, o);
            }
        }
        if (sub == 0) {
            float4* o4 = reinterpret_cast<float4*>(out + (size_t)b * w.T * w.D + (size_t)t * w.D);
            const float inv = (WT && w.pool_mean && o_hi > o_lo) ? 1.f / (float)(o_hi - o_lo) : 1.f;
#pragma unroll
            for (int c = 0; c < CPL; ++c) {
                const int ch = lr + c * LPR;
                if (WT) { acc[c].x *= inv; acc[c].y *= inv; acc[c].z *= inv; acc[c].w *= inv; }
                if (ch < D4) __stcs(o4 + ch, acc[c]);
            }
        }
        o_lo = n_lo;
        o_hi = n_hi;
        o_next = n_next;
        t = tn;
    }
    }
}

// Rows of up to 256 bytes (D <= 64): the gather is bound by bytes in flight, and registers cap what LDG can keep in
// flight.  Here every warp owns an 8 KB shared-memory buffer and fills it with cp.async (16 bytes per lane, two
// rows per instruction, no staging registers): the 32 rows of a batch are all in flight at once.  Same bag
// partition (equal shares of the lookups per warp), same prefetch of the next batch's rank look-ups.
#define POOL_WARPS 7   // 4 CTAs x 7 warps x 8 KB = 224 KB of the SM's shared memory
template <int R4, bool WT>   // R4: float4 pieces per staged row, 16 (D <= 64) or 8 (D <= 32)
__global__ void __launch_bounds__(32 * POOL_WARPS, 4) k_pool_async(WsView w, float* __restrict__ out)
{
    tt_pdl_enter();
    static_assert(R4 == 16 || R4 == 8, "two or four rows per cp.async instruction");
    constexpr int RPI = 32 / R4;
    constexpr int PGRP = 4;              // load instructions per group: a window is cut short and tested for validity per group
                                         // (half of all windows end a bag and are short; groups of two measured slower)
    extern __shared__ __align__(16) float4 pool_buf[];   // [POOL_WARPS][32 rows][R4 float4]
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const int sub = lane / R4, lr = lane % R4;
    float4* buf = pool_buf + (size_t)wid * 32 * R4;
    const int D4 = w.D >> 2;
    const bool lane_on = lr < D4;
    const float4* __restrict__ E4 = reinterpret_cast<const float4*>(w.E);
    const uint32_t capK = w.cap[w.K];
    const int64_t W = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const int64_t C = W * tt_pool_chunks(w.L, W);
    // lookup positions and bag indices fit in 32 bits (L and T * B are below 2^31, checked when the handle is made)
    typedef int32_t pos_t;
    auto clampL = [&](int64_t x) { return x < 0 ? (pos_t)0 : (x > w.L ? (pos_t)w.L : (pos_t)x); };
    for (;;) {
    // shares are handed out in order through a counter: a warp whose shares hold popular (L2-resident) rows takes more of them
    int64_t ci = 0;
    if (lane == 0) ci = (int64_t)atomicAdd(&w.counters[CTR_POOL_NEXT], 1u);
    ci = __shfl_sync(0xffffffffu, ci, 0);
    if (ci >= C) break;
    const pos_t b0 = (pos_t)__ldg(w.pool_bounds + ci), b1 = (pos_t)__ldg(w.pool_bounds + ci + 1);
    if (b0 >= b1) continue;
    // every bag is summed over its own (offsets[bag], offsets[bag + 1]) pair, clamped to [0, L]; an inverted pair (malformed
    // offsets) is an empty bag.  o_next: start of the next bag = this bag's end as stored, before the inversion fix
    pos_t o_lo = clampL(__ldg(w.offsets + b0)), o_next = clampL(__ldg(w.offsets + b0 + 1));
    pos_t o_hi = o_next < o_lo ? o_lo : o_next;
    int t = (int)(b0 / w.B);
    uint32_t slot_next;
    float wt_next = 1.f;
    auto fetch = [&](pos_t base, pos_t lim, int tt) {   // rank look-up (and weight) of lookup base + lane
        slot_next = (base + lane < lim) ? tt_lookup_slot(w, w.tdesc[tt], base + lane, capK) : 0xffffffffu;
        if (WT) wt_next = (w.psw && base + lane < lim) ? __ldg(w.psw + base + lane) : 1.f;
    };
    fetch(o_lo, o_hi, t);
    for (pos_t bag = b0; bag < b1; ++bag) {
        const pos_t b = bag - (pos_t)t * w.B;
        const bool has_next = bag + 1 < b1;
        const pos_t n_lo = o_next;
        const pos_t n_next = has_next ? clampL(__ldg(w.offsets + bag + 2)) : o_next;
        const pos_t n_hi = n_next < n_lo ? n_lo : n_next;
        const int tn = (has_next && b + 1 == w.B) ? t + 1 : t;
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        if (o_lo >= o_hi && has_next) fetch(n_lo, n_hi, tn);
        for (pos_t l0 = o_lo; l0 < o_hi; l0 += 32) {
            const uint32_t slot = slot_next;
            const float wt = wt_next;
            if (w.upairs && l0 + lane < o_hi) __stcs(&w.upairs[l0 + lane], make_uint2(slot, (uint32_t)b));
            const int n = (int)min((pos_t)32, o_hi - l0);
            const unsigned valid = __ballot_sync(0xffffffffu, lane < n && slot != 0xffffffffu);
            // two-level sum: the batch's rows go into a partial that is added to the bag's sum once per batch, so the
            // rounding error of a bag with thousands of lookups grows with the number of batches, not of rows
            float4 part = make_float4(0.f, 0.f, 0.f, 0.f);
            // all rows of the batch in flight
            // (groups of four instructions; a short window -- half of all windows end a bag -- leaves early)
            // a group whose rows are all valid (the usual case) needs no per-row test
            const bool plain = valid == (n == 32 ? 0xffffffffu : (1u << n) - 1u) && D4 == R4;
#pragma unroll
            for (int jq = 0; jq < 32 / RPI; jq += PGRP) {
                if (RPI * jq >= n) break;
                if (plain && RPI * (jq + PGRP) <= n) {
#pragma unroll
                    for (int jj = jq; jj < jq + PGRP; ++jj) {
                        const int j = RPI * jj + sub;
                        const uint32_t sl = __shfl_sync(0xffffffffu, slot, j);
                        tt_cp_async16(buf + j * R4 + lr, E4 + (size_t)sl * R4 + lr);
                    }
                } else {
#pragma unroll
                    for (int jj = jq; jj < jq + PGRP; ++jj) {
                        const int j = RPI * jj + sub;
                        const uint32_t sl = __shfl_sync(0xffffffffu, slot, j);
                        if (((valid >> j) & 1u) && lane_on) tt_cp_async16(buf + j * R4 + lr, E4 + (size_t)sl * D4 + lr);
                    }
                }
            }
            asm volatile("cp.async.commit_group;" ::: "memory");
            // the rank look-ups of the next batch (or of the next bag) overlap the gather
            if (l0 + 32 < o_hi) fetch(l0 + 32, o_hi, t);
            else if (has_next) fetch(n_lo, n_hi, tn);
            asm volatile("cp.async.wait_group 0;" ::: "memory");
            __syncwarp();
#pragma unroll
            for (int jq = 0; jq < 32 / RPI; jq += PGRP) {
                if (RPI * jq >= n) break;
                if (!WT && plain && RPI * (jq + PGRP) <= n) {
#pragma unroll
                    for (int jj = jq; jj < jq + PGRP; ++jj) {
                        const float4 v = buf[(RPI * jj + sub) * R4 + lr];
                        tt_add4(part, v);
                    }
                } else {
#pragma unroll
                    for (int jj = jq; jj < jq + PGRP; ++jj) {
                        const int j = RPI * jj + sub;
                        const float wj = WT ? __shfl_sync(0xffffffffu, wt, j) : 1.f;
                        if (((valid >> j) & 1u) && lane_on) {
                            const float4 v = buf[j * R4 + lr];
                            if (WT) { part.x = fmaf(wj, v.x, part.x); part.y = fmaf(wj, v.y, part.y); part.z = fmaf(wj, v.z, part.z); part.w = fmaf(wj, v.w, part.w); }
                            else tt_add4(part, v);
                        }
                    }
                }
            }
            acc.x += part.x; acc.y += part.y; acc.z += part.z; acc.w += part.w;
            __syncwarp();
        }
#pragma unroll
        for (int o = R4; o < 32; o <<= 1) {
            acc.x += __shfl_xor_sync(0xffffffffu, acc.x, o); acc.y += __shfl_xor_sync(0xffffffffu, acc.y, o);
            acc.z += __shfl_xor_sync(0xffffffffu, acc.z, o); acc.w += __shfl_xor_sync(0xffffffffu, acc.w, o);
        }
        if (WT && w.pool_mean && o_hi > o_lo) {
            const float inv = 1.f / (float)(o_hi - o_lo);
            acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
        }
        if (sub == 0 && lane_on) __stcs(reinterpret_cast<float4*>(out + (size_t)b * w.T * w.D + (size_t)t * w.D) + lr, acc);
        o_lo = n_lo;
        o_hi = n_hi;
        o_next = n_next;
        t = tn;
    }
    }
}

// The same gather for batches with few lookups per bag (on average below TT_POOL_STREAM_BELOW, or ..._WIDE for rows
// of more than 128 bytes): a window is 32 consecutive lookups of the warp's share, whatever bags they belong to.  One
// bag per window, as in k_pool_async, costs the latency of a window per bag: 2 million bags took 0.82 ms there whether
// they held 2 or 16 lookups each, and 7.9 million one-lookup bags 3.0 ms.  Here a window of one-lookup bags goes
// straight from the staged rows to out (those 7.9 million bags: 0.40 ms, 5 TB/s of rows read and written); a full
// window with one boundary is summed into two partial sums in one unrolled pass; a window with several bags in it is
// summed by the whole warp at once, each sub-warp taking consecutive rows and the pieces of a bag that crosses
// sub-warps being joined afterwards (from two boundaries on for rows of up to 128 bytes, from five on for wider rows,
// where a sub-warp has sixteen rows to walk); a window with empty bags, weights or mean pooling is summed bag by bag.
// 2 million bags of 128-byte rows, stream against one bag per window: 2 / 4 / 8 lookups each 0.20 / 0.28 / 0.51 ms
// against 0.82; 1 to 15 lookups 0.54 against 0.83, 1 to 31 0.83 against 0.91, 1 to 63 1.22 against 1.27, 1 to 100 1.69
// against 1.72, 1 to 200 3.09 against 3.00 ms.  256-byte rows: 2 / 4 / 8 lookups 0.29 / 0.44 / 0.74 ms against 0.88-0.92;
// 1 to 15 lookups 0.78 against 0.95; 1 to 31 1.11-1.19 against 1.10; on the benchmark configuration (1 to 100 lookups)
// 2.34-2.36 against 2.39 ms.  Hence the thresholds (the benchmark configuration stays with the per-bag kernel).  A
// window ends early only at the end of the share or of a table (the rank look-up of a window uses one table).  With
// malformed offsets (status bit set by the offsets check earlier in the stream) every bag is summed over its own
// clamped (offsets[bag], offsets[bag + 1]) pair as the header promises, and windows stop at the end of their bag.
#define TT_POOL_STREAM_BELOW 33        // rows of up to 128 bytes
#define TT_POOL_STREAM_BELOW_WIDE 12   // rows of up to 256 bytes
template <int R4, bool WT>   // R4: float4 pieces per staged row, 16 (D <= 64) or 8 (D <= 32)
__global__ void __launch_bounds__(32 * POOL_WARPS, 4) k_pool_stream(WsView w, float* __restrict__ out)
{
    tt_pdl_enter();
    static_assert(R4 == 16 || R4 == 8, "two or four rows per cp.async instruction");
    constexpr int RPI = 32 / R4;
    constexpr int PGRP = 4;              // load instructions per group: a window is cut short and tested for validity per group
    extern __shared__ __align__(16) float4 pool_buf[];   // [POOL_WARPS][32 rows][R4 float4]
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const int sub = lane / R4, lr = lane % R4;
    float4* buf = pool_buf + (size_t)wid * 32 * R4;
    const int D4 = w.D >> 2;
    const bool lane_on = lr < D4;
    const float4* __restrict__ E4 = reinterpret_cast<const float4*>(w.E);
    const uint32_t capK = w.cap[w.K];
    const int64_t W = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const int64_t C = W * tt_pool_chunks(w.L, W);
    const bool stream_ok = !(*w.status & TT_EMB_STATUS_OFFSETS);
    // lookup positions and bag indices fit in 32 bits (L and T * B are below 2^31, checked when the handle is made)
    typedef int32_t pos_t;
    auto clampL = [&](int64_t x) { return x < 0 ? (pos_t)0 : (x > w.L ? (pos_t)w.L : (pos_t)x); };
    for (;;) {
    int64_t ci = 0;     // shares are handed out in order through a counter (see k_pool_async)
    if (lane == 0) ci = (int64_t)atomicAdd(&w.counters[CTR_POOL_NEXT], 1u);
    ci = __shfl_sync(0xffffffffu, ci, 0);
    if (ci >= C) break;
    const pos_t b0 = (pos_t)__ldg(w.pool_bounds + ci), b1 = (pos_t)__ldg(w.pool_bounds + ci + 1);
    if (b0 >= b1) continue;
    // the ends of the share's bags, 32 at a time and one vector ahead: lane i holds the clamped offsets[ebase + 1 + i]
    // (ends_nx: the 32 bags after those), so that no bag waits for a load of its own end
    auto load_ends = [&](pos_t base) { const pos_t i = base + lane; return i < b1 ? clampL(__ldg(w.offsets + i + 1)) : (pos_t)0x7fffffff; };   // past the share: never inside a window
    pos_t ebase = b0;
    pos_t ends_reg = load_ends(b0), ends_nx = load_ends(b0 + 32);
    auto end_of = [&](pos_t bg) {     // bg >= ebase, and below ebase + 64 (a step moves on by at most 32 bags)
        while (bg - ebase >= 32) {
            ends_reg = ends_nx;
            ebase += 32;
            ends_nx = load_ends(ebase + 32);
        }
        return __shfl_sync(0xffffffffu, ends_reg, (int)(bg - ebase));
    };
    // the bag being summed: its table, its (clamped) range, the end of the bag as stored
    pos_t bag = b0;
    int t = (int)(b0 / w.B);
    pos_t o_lo = clampL(__ldg(w.offsets + b0)), o_next = end_of(b0);
    pos_t o_hi = o_next < o_lo ? o_lo : o_next;
    const pos_t share_end = stream_ok ? clampL(__ldg(w.offsets + b1)) : 0;
    pos_t t_end = stream_ok ? (pos_t)__ldg(w.tl_start + t + 1) : 0;
    pos_t pos = o_lo;                                 // next lookup of the stream
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    // rank look-up (and weight) of lookup base + lane, for the window that starts at `base`
    uint32_t slot_next = 0xffffffffu;
    float wt_next = 1.f;
    pos_t pre_pos = -1;
    int pre_t = -1;
    auto fetch = [&](pos_t base, pos_t lim, int tt) {
        slot_next = (base + lane < lim) ? tt_lookup_slot(w, w.tdesc[tt], base + lane, capK) : 0xffffffffu;
        if (WT) wt_next = (w.psw && base + lane < lim) ? __ldg(w.psw + base + lane) : 1.f;
        pre_pos = base;
        pre_t = tt;
    };
    // bag `nb_`, which starts at lookup `lo_`, becomes the one being summed (nb_ > bag, at most 32 bags on)
    auto seek_bag = [&](pos_t nb_, pos_t lo_) {
        acc = make_float4(0.f, 0.f, 0.f, 0.f);
        bag = nb_;
        if (bag < b1) {
            if (bag >= (pos_t)(t + 1) * w.B) {
                ++t;
                if (stream_ok) t_end = (pos_t)__ldg(w.tl_start + t + 1);
            }
            o_lo = lo_;
            o_next = end_of(bag);
            o_hi = o_next < o_lo ? o_lo : o_next;
        }
    };
    auto advance_bag = [&]() { seek_bag(bag + 1, o_next); };
    // the bag is complete: combine the sub-warps, write its row of out, move on to the next bag
    auto close_bag = [&]() {
#pragma unroll
        for (int o = R4; o < 32; o <<= 1) {
            acc.x += __shfl_xor_sync(0xffffffffu, acc.x, o); acc.y += __shfl_xor_sync(0xffffffffu, acc.y, o);
            acc.z += __shfl_xor_sync(0xffffffffu, acc.z, o); acc.w += __shfl_xor_sync(0xffffffffu, acc.w, o);
        }
        if (WT && w.pool_mean && o_hi > o_lo) {
            const float inv = 1.f / (float)(o_hi - o_lo);
            acc.x *= inv; acc.y *= inv; acc.z *= inv; acc.w *= inv;
        }
        const pos_t b = bag - (pos_t)t * w.B;
        if (sub == 0 && lane_on) __stcs(reinterpret_cast<float4*>(out + (size_t)b * w.T * w.D + (size_t)t * w.D) + lr, acc);
        advance_bag();
    };
    while (bag < b1) {
        if (pos >= o_hi) {              // the bag has no (more) lookups
            close_bag();
            pos = o_lo;
            continue;
        }
        const pos_t lim = stream_ok ? (share_end < t_end ? share_end : t_end) : o_hi;   // > pos: the bag ends no later
        const int n = (int)min((pos_t)32, lim - pos);
        if (pre_pos != pos || pre_t != t) fetch(pos, lim, t);
        const uint32_t slot = slot_next;
        const float wt = wt_next;
        const unsigned valid = __ballot_sync(0xffffffffu, lane < n && slot != 0xffffffffu);
        // all rows of the window in flight (groups of four instructions; a short window leaves early);
        // a group whose rows are all valid (the usual case) needs no per-row test
        const bool plain = valid == (n == 32 ? 0xffffffffu : (1u << n) - 1u) && D4 == R4;
#pragma unroll
        for (int jq = 0; jq < 32 / RPI; jq += PGRP) {
            if (RPI * jq >= n) break;
            if (plain && RPI * (jq + PGRP) <= n) {
#pragma unroll
                for (int jj = jq; jj < jq + PGRP; ++jj) {
                    const int j = RPI * jj + sub;
                    const uint32_t sl = __shfl_sync(0xffffffffu, slot, j);
                    tt_cp_async16(buf + j * R4 + lr, E4 + (size_t)sl * R4 + lr);
                }
            } else {
#pragma unroll
                for (int jj = jq; jj < jq + PGRP; ++jj) {
                    const int j = RPI * jj + sub;
                    const uint32_t sl = __shfl_sync(0xffffffffu, slot, j);
                    if (((valid >> j) & 1u) && lane_on) tt_cp_async16(buf + j * R4 + lr, E4 + (size_t)sl * D4 + lr);
                }
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
        // the rank look-ups of the next window overlap the gather (the next window of the stream; in the per-bag mode
        // only while the bag goes on)
        {
            const pos_t np = pos + n;
            if (stream_ok) {
                if (np < lim) fetch(np, lim, t);
                else if (np < share_end) {               // the table ends here: the next window belongs to the next one
                    const pos_t te = (pos_t)__ldg(w.tl_start + t + 2);
                    fetch(np, share_end < te ? share_end : te, t + 1);
                }
            } else if (np < o_hi) fetch(np, o_hi, t);
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncwarp();
        // Windows with bag boundaries in them are summed by the whole warp at once.  Lane i looks at bag + i, which ends at
        // e_mine; a bag starts at row e - pos of the window for every end e inside it.
        if (!WT && stream_ok && o_hi < pos + n) {
            const pos_t wend = pos + n;
            const int ei = (int)(bag - ebase) + lane;
            const pos_t e0 = __shfl_sync(0xffffffffu, ends_reg, ei & 31), e1 = __shfl_sync(0xffffffffu, ends_nx, ei & 31);
            const pos_t e_mine = ei < 32 ? e0 : e1;
            // one-lookup bags only (lane i: bag + i ends at pos + i + 1): every staged row is a row of out
            if (o_lo == pos && __all_sync(0xffffffffu, lane >= n || e_mine == pos + lane + 1)) {
                const pos_t bf = bag - (pos_t)t * w.B;       // the window lies in table t: bf + n <= B
                if (w.upairs && lane < n) __stcs(&w.upairs[pos + lane], make_uint2(slot, (uint32_t)(bf + lane)));
                float4* o4 = reinterpret_cast<float4*>(out + (size_t)bf * w.T * w.D + (size_t)t * w.D) + lr;
                const size_t ostride = (size_t)w.T * D4;
#pragma unroll
                for (int jj = 0; jj < 32 / RPI; ++jj) {
                    const int j = RPI * jj + sub;
                    if (j < n && lane_on)
                        __stcs(o4 + (size_t)j * ostride, ((valid >> j) & 1u) ? buf[j * R4 + lr] : make_float4(0.f, 0.f, 0.f, 0.f));
                }
                __syncwarp();
                pos += n;
                seek_bag(bag + n, pos);
                continue;
            }
            // no empty bag among those that start inside the window (an empty bag needs a row of zeros: left to the
            // bag-by-bag loop below)
            const pos_t e_prev = __shfl_up_sync(0xffffffffu, e_mine, 1);
            const int inside = __popc(__ballot_sync(0xffffffffu, e_mine > pos && e_mine < wend));   // bag ends inside the window
            if (inside == 1 && plain && n == 32) {
                // one boundary, at row c: the rows before it complete the open bag, the others start the next one
                const int c = (int)(o_hi - pos);
                if (w.upairs) __stcs(&w.upairs[pos + lane], make_uint2(slot, (uint32_t)(bag - (pos_t)t * w.B) + (lane >= c ? 1u : 0u)));
                float4 pa = make_float4(0.f, 0.f, 0.f, 0.f), pb = pa;
#pragma unroll
                for (int jj = 0; jj < 32 / RPI; ++jj) {
                    const int j = RPI * jj + sub;
                    const float4 v = buf[j * R4 + lr];
                    if (j < c) tt_add4(pa, v); else tt_add4(pb, v);
                }
                acc.x += pa.x; acc.y += pa.y; acc.z += pa.z; acc.w += pa.w;
                close_bag();
                acc = pb;
                __syncwarp();
                pos = wend;
                continue;
            }
            const bool many = inside >= (R4 == 16 ? 5 : 2);   // fewer: cheaper bag by bag
            if (many && !__any_sync(0xffffffffu, lane >= 1 && e_prev < wend && e_mine == e_prev)) {
                // starts: bit j = row j is the first of its bag; closes: bit j = row j is the last of its bag
                const unsigned starts = __reduce_or_sync(0xffffffffu, (e_mine > pos && e_mine < wend) ? 1u << (int)(e_mine - pos) : 0u)
                                      | (o_lo == pos ? 1u : 0u);
                const bool last_closed = __any_sync(0xffffffffu, e_mine == wend);
                const unsigned closes = (starts >> 1) | (last_closed ? 1u << (n - 1) : 0u);
                const pos_t bt = bag - (pos_t)t * w.B;       // bag of row j: bt + bags started in rows 1..j
                auto row_of = [&](int j) {
                    const pos_t b = bt + __popc(starts & ((2u << j) - 2u));
                    return reinterpret_cast<float4*>(out + (size_t)b * w.T * w.D + (size_t)t * w.D) + lr;
                };
                if (w.upairs && lane < n)
                    __stcs(&w.upairs[pos + lane], make_uint2(slot, (uint32_t)(bt + __popc(starts & ((2u << lane) - 2u)))));
                // the open bag's sum so far, the same in every sub-warp
                float4 carry = acc;
#pragma unroll
                for (int o = R4; o < 32; o <<= 1) {
                    carry.x += __shfl_xor_sync(0xffffffffu, carry.x, o); carry.y += __shfl_xor_sync(0xffffffffu, carry.y, o);
                    carry.z += __shfl_xor_sync(0xffffffffu, carry.z, o); carry.w += __shfl_xor_sync(0xffffffffu, carry.w, o);
                }
                // sub-warp s sums the R4 consecutive rows from s * R4 on, in step with the others: a bag that lies inside
                // them is written at its last row; the piece of a bag that came in from before (head) is kept, the piece
                // of a bag that goes on after them is what `run` holds at the end
                float4 run = make_float4(0.f, 0.f, 0.f, 0.f), head = run;
                bool head_open = !((starts >> (sub * R4)) & 1u), head_closed = false;
                // (not unrolled: the kernel's warps are spread over its four summing paths, and with this loop unrolled
                // they waited for instructions: 2.39 -> 1.90 ms on the 240-table workload, ncu `no_instruction` stalls)
                // (the row of out of the bag being summed moves on by one bag per segment end; masks shifted to the sub-warp)
                {
                    const int j0 = sub * R4, ns = min(R4, n - j0);
                    unsigned vs = valid >> j0, cs = closes >> j0;
                    float4* orow = row_of(j0);
                    const size_t ostride = (size_t)w.T * D4;
                    const float4* src = buf + j0 * R4 + lr;
#pragma unroll 1
                    for (int jj = 0; jj < ns; ++jj, vs >>= 1, cs >>= 1, src += R4) {
                        if (vs & 1u) {
                            const float4 v = *src;
                            tt_add4(run, v);
                        }
                        if (cs & 1u) {
                            if (head_open) { head = run; head_closed = true; head_open = false; }
                            else if (lane_on) __stcs(orow, run);
                            run = make_float4(0.f, 0.f, 0.f, 0.f);
                            orow += ostride;
                        }
                    }
                }
                // the pieces across the sub-warps, in order: a head closes the bag carried so far; rows that all belong to
                // the carried bag add to it; otherwise the carried bag ended with the sub-warp before (nothing carried)
                const unsigned hc = __ballot_sync(0xffffffffu, head_closed), ho = __ballot_sync(0xffffffffu, head_open);
#pragma unroll
                for (int s2 = 0; s2 < RPI; ++s2) {
                    if (((hc >> (s2 * R4)) & 1u) && sub == s2 && lane_on) {
                        float4 sum = carry;
                        tt_add4(sum, head);
                        __stcs(row_of(s2 * R4), sum);
                    }
                    float4 tail;
                    tail.x = __shfl_sync(0xffffffffu, run.x, s2 * R4 + lr); tail.y = __shfl_sync(0xffffffffu, run.y, s2 * R4 + lr);
                    tail.z = __shfl_sync(0xffffffffu, run.z, s2 * R4 + lr); tail.w = __shfl_sync(0xffffffffu, run.w, s2 * R4 + lr);
                    if ((ho >> (s2 * R4)) & 1u) tt_add4(carry, tail);
                    else carry = tail;
                }
                __syncwarp();
                const pos_t bl = bag + __popc(starts & 0xfffffffeu);     // the bag of the window's last row
                pos = wend;
                if (last_closed) seek_bag(bl + 1, pos);
                else {
                    if (bl > bag) {
                        const pos_t lo_ = end_of(bl - 1);
                        seek_bag(bl, lo_);
                    }
                    acc = sub == 0 ? carry : make_float4(0.f, 0.f, 0.f, 0.f);
                }
                continue;
            }
        }
        // the window's rows, bag by bag.  Two-level sum: the rows of a (piece of a) bag go into a partial that is added to
        // the bag's sum once, so the rounding error of a bag with thousands of lookups grows with the number of windows
        int r = 0;
        while (r < n) {
            if (pos + r >= o_hi) {       // a bag ends inside the window (and empty bags after it)
                close_bag();
                if (bag >= b1) break;    // cannot happen with checked offsets; never spin on it
                continue;
            }
            const pos_t room = o_hi - (pos + r);
            const int seg = room < (pos_t)(n - r) ? (int)room : n - r;
            if (w.upairs && lane >= r && lane < r + seg)    // kept for the backward sort
                __stcs(&w.upairs[pos + lane], make_uint2(slot, (uint32_t)(bag - (pos_t)t * w.B)));
            if (!WT && seg == 1 && pos + r == o_lo && o_hi - o_lo == 1) {
                // a bag of one lookup: its row of out is the staged row (or zeros for an id outside the table); the
                // sub-warp that staged it writes it, nothing to combine
                if (sub == (r & (RPI - 1)) && lane_on) {
                    const float4 v = ((valid >> r) & 1u) ? buf[r * R4 + lr] : make_float4(0.f, 0.f, 0.f, 0.f);
                    __stcs(reinterpret_cast<float4*>(out + (size_t)(bag - (pos_t)t * w.B) * w.T * w.D + (size_t)t * w.D) + lr, v);
                }
                advance_bag();
                r += 1;
                if (bag >= b1) break;
                continue;
            }
            float4 part = make_float4(0.f, 0.f, 0.f, 0.f);
            if (!WT && plain && seg == 32) {
#pragma unroll
                for (int jj = 0; jj < 32 / RPI; ++jj) {
                    const float4 v = buf[(RPI * jj + sub) * R4 + lr];
                    tt_add4(part, v);
                }
            } else {
                for (int jj = r / RPI; RPI * jj < r + seg; ++jj) {
                    const int j = RPI * jj + sub;
                    const float wj = WT ? __shfl_sync(0xffffffffu, wt, j) : 1.f;
                    if (j >= r && j < r + seg && ((valid >> j) & 1u) && lane_on) {
                        const float4 v = buf[j * R4 + lr];
                        if (WT) { part.x = fmaf(wj, v.x, part.x); part.y = fmaf(wj, v.y, part.y); part.z = fmaf(wj, v.z, part.z); part.w = fmaf(wj, v.w, part.w); }
                        else tt_add4(part, v);
                    }
                }
            }
            acc.x += part.x; acc.y += part.y; acc.z += part.z; acc.w += part.w;
            r += seg;
        }
        __syncwarp();
        pos += n;
    }
    }
}


template <int R4, bool WT>
static cudaError_t launch_pool_async(tt_emb* h, float* out, cudaStream_t s)
{
    const size_t smem = (size_t)POOL_WARPS * 32 * R4 * sizeof(float4);
    cudaError_t e = cudaFuncSetAttribute(k_pool_async<R4, WT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    int per_sm = 0;
    if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_pool_async<R4, WT>, 32 * POOL_WARPS, smem)) != cudaSuccess) return e;
    if (per_sm < 1) per_sm = 1;
    const int64_t nb = (int64_t)h->v.T * h->v.B;
    int64_t grid = (int64_t)per_sm * h->sm_count;
    const int64_t need = (nb + POOL_WARPS - 1) / POOL_WARPS;
    if (grid > need) grid = need;
    if (grid < 1) grid = 1;
    if ((e = launch_pool_bounds(h, grid * POOL_WARPS, s)) != cudaSuccess) return e;
    if (h->v.L < (int64_t)(R4 == 16 ? TT_POOL_STREAM_BELOW_WIDE : TT_POOL_STREAM_BELOW) * nb) {   // few lookups per bag: windows across bags
        if ((e = cudaFuncSetAttribute(k_pool_stream<R4, WT>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)) != cudaSuccess) return e;
        if ((e = tt_launch_pdl(k_pool_stream<R4, WT>, dim3((int)grid), dim3(32 * POOL_WARPS), smem, s, h->v, out)) != cudaSuccess) return e;
        tt_note_launch();
        return cudaGetLastError();
    }
    if ((e = tt_launch_pdl(k_pool_async<R4, WT>, dim3((int)grid), dim3(32 * POOL_WARPS), smem, s, h->v, out)) != cudaSuccess) return e;
    tt_note_launch();
    return cudaGetLastError();
}

template <int LPR, int CPL, bool WT>
static cudaError_t launch_pool_vec(tt_emb* h, float* out, cudaStream_t s)
{
    int per_sm = 0;
    cudaError_t e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, k_pool_vec<LPR, CPL, WT>, 256, 0);
    if (e != cudaSuccess) return e;
    if (per_sm < 1) per_sm = 1;
    const int64_t nb = (int64_t)h->v.T * h->v.B;
    int64_t grid = (int64_t)per_sm * h->sm_count;
    const int64_t need = (nb + 7) / 8;
    if (grid > need) grid = need;
    if (grid < 1) grid = 1;
    if ((e = launch_pool_bounds(h, grid * 8, s)) != cudaSuccess) return e;
    if ((e = tt_launch_pdl(k_pool_vec<LPR, CPL, WT>, dim3((int)grid), dim3(256), 0, s, h->v, out)) != cudaSuccess) return e;
    tt_note_launch();
    return cudaGetLastError();
}

// any D (scalar path): lane handles elements lane, lane + 32, ... (NC of them per pass over the bag); 32 / NC rows in flight
template <int NC>
__global__ void __launch_bounds__(256) k_pool_scalar(WsView w, float* __restrict__ out)
{
    tt_pdl_enter();
    constexpr int RF = 32 / NC;     // rows in flight
    const int lane = threadIdx.x & 31;
    const int D = w.D;
    const int64_t nb = (int64_t)w.T * w.B;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const uint32_t capK = w.cap[w.K];
    for (int64_t bag = (((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5); bag < nb; bag += nwarps) {
        const int t = (int)(bag / w.B);
        const int64_t b = bag - (int64_t)t * w.B;
        const TableDesc& td = w.tdesc[t];
        int64_t lo = w.offsets[bag], hi = w.offsets[bag + 1];
        lo = lo < 0 ? 0 : (lo > w.L ? w.L : lo);
        hi = hi < lo ? lo : (hi > w.L ? w.L : hi);
        float* o = out + (size_t)b * w.T * D + (size_t)t * D;
        for (int e0 = 0; e0 < D; e0 += 32 * NC) {
            float acc[NC];
#pragma unroll
            for (int c = 0; c < NC; ++c) acc[c] = 0.f;
            // 32 lookups at a time: every lane looks one slot up (the two dependent loads of a lookup run 32 wide instead of
            // one after the other), then the rows are added in lookup order, RF row loads in flight
            for (int64_t l0 = lo; l0 < hi; l0 += 32) {
                const int n = (int)min((int64_t)32, hi - l0);
                const uint32_t slot = lane < n ? tt_lookup_slot(w, td, l0 + lane, capK) : 0xffffffffu;
                const float a = (w.psw && lane < n) ? __ldg(w.psw + l0 + lane) : 1.f;
                if (w.upairs && e0 == 0 && lane < n) w.upairs[l0 + lane] = make_uint2(slot, (uint32_t)b);
                for (int j0 = 0; j0 < n; j0 += RF) {
                    float v[RF][NC], aj[RF];
#pragma unroll
                    for (int jj = 0; jj < RF; ++jj) {
                        const uint32_t sj = __shfl_sync(0xffffffffu, slot, (j0 + jj) & 31);
                        aj[jj] = __shfl_sync(0xffffffffu, a, (j0 + jj) & 31);
                        const bool ok = j0 + jj < n && sj != 0xffffffffu;
                        const float* row = w.E + (size_t)(ok ? sj : 0u) * D;
#pragma unroll
                        for (int c = 0; c < NC; ++c) {
                            const int idx = e0 + lane + c * 32;
                            v[jj][c] = (ok && idx < D) ? __ldg(row + idx) : 0.f;
                        }
                    }
#pragma unroll
                    for (int jj = 0; jj < RF; ++jj)
#pragma unroll
                        for (int c = 0; c < NC; ++c) acc[c] = fmaf(aj[jj], v[jj][c], acc[c]);
                }
            }
            const float inv = (w.pool_mean && hi > lo) ? 1.f / (float)(hi - lo) : 1.f;
#pragma unroll
            for (int c = 0; c < NC; ++c) {
                const int idx = e0 + lane + c * 32;
                if (idx < D) o[idx] = acc[c] * inv;
            }
        }
    }
}

template <bool WT>
static cudaError_t launch_pool_sized(tt_emb* h, int D4, float* out, cudaStream_t s)
{
    if (D4 > 8 && D4 <= 16) return launch_pool_async<16, WT>(h, out, s);
    if (D4 > 4 && D4 <= 8) return launch_pool_async<8, WT>(h, out, s);
    if (D4 <= 4) return launch_pool_vec<4, 1, WT>(h, out, s);
    if (D4 <= 8) return launch_pool_vec<8, 1, WT>(h, out, s);
    if (D4 <= 16) return launch_pool_vec<16, 1, WT>(h, out, s);
    if (D4 <= 32) return launch_pool_vec<32, 1, WT>(h, out, s);
    if (D4 <= 64) return launch_pool_vec<32, 2, WT>(h, out, s);
    if (D4 <= 128) return launch_pool_vec<32, 4, WT>(h, out, s);
    return launch_pool_vec<32, 8, WT>(h, out, s);
}

cudaError_t tt_launch_pooling(tt_emb* h, float* out, cudaStream_t s)
{
    WsView& w = h->v;
    const int64_t nb = (int64_t)w.T * w.B;
    const int64_t want = (nb + 7) / 8;  // 8 warps per CTA, one warp per bag
    int grid = (int)want;
    if (grid < 1) grid = 1;
    const int D = w.D;
    const bool vec_ok = (D % 4 == 0) && ((reinterpret_cast<uintptr_t>(out) & 15) == 0);
    if (!vec_ok) {
        int pgrid = (int)(want < (int64_t)h->sm_count * 8 ? want : (int64_t)h->sm_count * 8);
        const dim3 pg(pgrid < 1 ? 1 : pgrid);
        cudaError_t e0 = D <= 32 ? tt_launch_pdl(k_pool_scalar<1>, pg, dim3(256), 0, s, w, out)
                       : D <= 64 ? tt_launch_pdl(k_pool_scalar<2>, pg, dim3(256), 0, s, w, out)
                       : D <= 128 ? tt_launch_pdl(k_pool_scalar<4>, pg, dim3(256), 0, s, w, out)
                                  : tt_launch_pdl(k_pool_scalar<8>, pg, dim3(256), 0, s, w, out);
        if (e0 != cudaSuccess) return e0;
        tt_note_launch();
        return cudaGetLastError();
    }
    const int D4 = D / 4;
    (void)grid;
    return (w.psw || w.pool_mean) ? launch_pool_sized<true>(h, D4, out, s) : launch_pool_sized<false>(h, D4, out, s);
}
