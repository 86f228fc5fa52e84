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

// ---------------------------------------------------------------------------------------------- schedule

struct CostScan {
    WsView w;
    int shift;
    __device__ uint32_t size() const { return w.counters[CTR_LEVEL0 + w.K - 1]; }
    __device__ uint32_t value(uint32_t g) const
    {
        const int K = w.K;
        const int t = tt_find_table(w.tb[K - 1], w.T, g);
        const TableDesc& td = w.tdesc[t];
        const uint32_t nchild = w.cstart[K - 1][g + 1] - w.cstart[K - 1][g];
        // c_k = P_{k-1} r_{k-1} d_k r_k
        uint64_t c_last = (uint64_t)td.P[K - 1] * td.r[K - 1] * td.d[K - 1];
        uint64_t c_mid = K >= 3 ? (uint64_t)td.P[K - 2] * td.r[K - 2] * td.d[K - 2] * td.r[K - 1] : 0;
        uint64_t c = ((c_mid + (uint64_t)nchild * c_last) >> shift) + 1;
        return (uint32_t)c;
    }
    __device__ void emit(uint32_t g, uint32_t excl, uint32_t) const { w.cost[g] = excl; }
    __device__ void total(uint32_t tot) const
    {
        w.cost[size()] = tot;
        w.counters[CTR_COST_TOTAL] = tot;
    }
};

cudaError_t tt_launch_schedule(tt_emb* h, cudaStream_t s)
{
    // cost unit: 2^shift FMAs, chosen at create time so that the worst-case total fits 32 bits
    CostScan cs{h->v, h->cost_shift};
    return tt_scan(cs, h->v.cap[h->v.K - 1], h->v.scan_tmp, s);
}

// group range [g0, g1) of work unit `unit` (global id) -- equal-cost slice of its table
__device__ __forceinline__ void tt_unit_range(const WsView& w, int unit, int& t_out, uint32_t& g0, uint32_t& g1)
{
    int t = 0;
    for (int i = 0; i < w.T; ++i)
        if (w.tdesc[i].unit_base <= unit) t = i;
    const TableDesc& td = w.tdesc[t];
    const int q = unit - td.unit_base, Q = td.units;
    const int lvl = w.K - 1;
    const uint32_t a = w.tb[lvl][t], b = w.tb[lvl][t + 1];
    const uint64_t ca = w.cost[a], cb = w.cost[b];
    const uint64_t lo_c = ca + (cb - ca) * (uint64_t)q / Q, hi_c = ca + (cb - ca) * (uint64_t)(q + 1) / Q;
    // first group whose exclusive cost >= target
    auto lower = [&](uint64_t target) {
        uint32_t lo = a, hi = b;
        while (lo < hi) {
            uint32_t mid = lo + ((hi - lo) >> 1);
            if ((uint64_t)w.cost[mid] < target) lo = mid + 1; else hi = mid;
        }
        return lo;
    };
    g0 = q == 0 ? a : lower(lo_c);
    g1 = q == Q - 1 ? b : lower(hi_c);
    t_out = t;
}

// ---------------------------------------------------------------------------------------------- products

// out[m*cols + c] = sum_a Pl[m*ra + a] * Bsl[a*cols + c]   (Pl in shared memory, Bsl in global, out anywhere)
__device__ __forceinline__ void tt_mid_product(const float* __restrict__ Pl, const float* __restrict__ Bsl, float* out,
                                               int M, int ra, int cols)
{
    for (int c = threadIdx.x; c < cols; c += blockDim.x) {
        for (int m0 = 0; m0 < M; m0 += 8) {
            float acc[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[i] = 0.f;
            const int mm = min(8, M - m0);
            for (int a = 0; a < ra; ++a) {
                const float b = __ldg(Bsl + (size_t)a * cols + c);
#pragma unroll
                for (int i = 0; i < 8; ++i)
                    if (i < mm) acc[i] = fmaf(Pl[(m0 + i) * ra + a], b, acc[i]);
            }
#pragma unroll
            for (int i = 0; i < 8; ++i)
                if (i < mm) out[(size_t)(m0 + i) * cols + c] = acc[i];
        }
    }
}

// left operand of level k (0-based core index kc = k-1 >= 1) for node v: P_{k-1} of its parent
__device__ __forceinline__ const float* tt_left_operand(const WsView& w, const TableDesc& td, int k, uint32_t v)
{
    // k = level of the node being produced (2..K-1)
    if (k == 2) {
        const uint32_t i1 = w.val[2][v] / (uint32_t)td.n[1];
        return td.core[0] + (size_t)i1 * td.slice_floats[0];
    }
    return w.pbuf[k - 1] + (size_t)w.parent[k][v] * w.stride[k - 1];
}

// P_k for every level-k node, 2 <= k <= K-2 (only K = 4 has such a level); one CTA per node, grid-stride
__global__ void __launch_bounds__(128) k_mid_level(WsView w, int k)
{
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

// fused levels K-1 and K: C in shared memory, rows to w.E
__global__ void __launch_bounds__(128) k_sweep_fwd(WsView w, int pl_floats)
{
    extern __shared__ float sm[];
    float* Pl = sm;
    float* Cs = sm + pl_floats;
    int t;
    uint32_t g0, g1;
    tt_unit_range(w, blockIdx.x, t, g0, g1);
    const TableDesc& td = w.tdesc[t];
    const int K = w.K, kl = K - 1, km = K - 2;
    const int Pm = td.P[K - 1], rb = td.r[K - 1], dK = td.d[kl], D = w.D;
    const uint32_t nK = (uint32_t)td.n[kl];
    for (uint32_t g = g0; g < g1; ++g) {
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

cudaError_t tt_launch_contraction(tt_emb* h, cudaStream_t s)
{
    WsView& w = h->v;
    int max_pl = 1, max_c = 1;
    for (int t = 0; t < h->T; ++t) {
        const TableDesc& td = h->tab[t];
        for (int k = 1; k < h->K; ++k) {
            int f = td.P[k] * td.r[k];
            if (k <= h->K - 2 && f > max_pl) max_pl = f;
            if (k == h->K - 1 && f > max_c) max_c = f;
        }
    }
    for (int k = 2; k <= h->K - 2; ++k) {
        int grid = h->sm_count * 16;
        k_mid_level<<<grid, 128, (size_t)max_pl * sizeof(float), s>>>(w, k);
    }
    const size_t smem = (size_t)(max_pl + max_c) * sizeof(float);
    k_sweep_fwd<<<h->units_total, 128, smem, s>>>(w, max_pl);
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------- pooling

// One warp per bag.  A row of D floats is read as D/4 float4 chunks by a sub-warp of LPR lanes
// (LPR = power of two >= min(32, D/4)); 32/LPR rows are in flight per load instruction, and the
// sub-warps' partial sums are combined with __shfl_xor at the end.
template <int LPR, int CPL>  // lanes per row, float4 chunks per lane
__global__ void __launch_bounds__(256) k_pool_vec(WsView w, float* __restrict__ out)
{
    const int lane = threadIdx.x & 31;
    const int sub = lane / LPR, lr = lane % LPR;
    constexpr int RPI = 32 / LPR;  // rows per iteration
    const int D4 = w.D >> 2;
    const int64_t nb = (int64_t)w.T * w.B;
    const int64_t nwarps = ((int64_t)gridDim.x * blockDim.x) >> 5;
    const float4* __restrict__ E4 = reinterpret_cast<const float4*>(w.E);
    const uint32_t capK = w.cap[w.K];
    bool bad = false;
    for (int64_t bag = (((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5); bag < nb; bag += nwarps) {
        const int t = (int)(bag / w.B);
        const int64_t b = bag - (int64_t)t * w.B;
        const TableDesc& td = w.tdesc[t];
        int64_t lo = w.offsets[bag], hi = w.offsets[bag + 1];
        lo = lo < 0 ? 0 : (lo > w.L ? w.L : lo);
        hi = hi < lo ? lo : (hi > w.L ? w.L : hi);
        float4 acc[CPL];
#pragma unroll
        for (int c = 0; c < CPL; ++c) acc[c] = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int64_t l0 = lo; l0 < hi; l0 += 32) {
            uint32_t slot = 0xffffffffu;
            if (l0 + lane < hi) {
                const int64_t g = __ldg(w.indices + l0 + lane);
                if (g >= 0 && g < td.N) {
                    const uint2 e = __ldg(&w.bm[td.word_base + ((uint32_t)g >> 5)]);
                    if (e.x >> (g & 31) & 1u) {
                        slot = e.y + __popc(e.x & ((1u << (g & 31)) - 1u));
                        if (slot >= capK) slot = 0xffffffffu;
                    }
                }
                if (w.upairs) w.upairs[l0 + lane] = make_uint2(slot, (uint32_t)b);  // kept for the backward sort
            }
            const int n = (int)min((int64_t)32, hi - l0);
#pragma unroll 4
            for (int j = 0; j < n; j += RPI) {
                const uint32_t sl = __shfl_sync(0xffffffffu, slot, (j + sub) & 31);
                if (j + sub < n && sl != 0xffffffffu) {
                    const float4* row = E4 + (size_t)sl * D4;
#pragma unroll
                    for (int c = 0; c < CPL; ++c) {
                        const int ch = lr + c * LPR;
                        if (ch < D4) {
                            const float4 v = __ldg(row + ch);
                            acc[c].x += v.x; acc[c].y += v.y; acc[c].z += v.z; acc[c].w += v.w;
                        }
                    }
                }
            }
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
#pragma unroll
            for (int c = 0; c < CPL; ++c) {
                const int ch = lr + c * LPR;
                if (ch < D4) o4[ch] = acc[c];
            }
        }
    }
    (void)bad;
}

// any D (scalar path): lane handles elements lane, lane+32, ...
__global__ void __launch_bounds__(256) k_pool_scalar(WsView w, float* __restrict__ out)
{
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
        if (w.upairs)
            for (int64_t l = lo + lane; l < hi; l += 32) {
                const int64_t g = __ldg(w.indices + l);
                uint32_t slot = 0xffffffffu;
                if (g >= 0 && g < td.N) {
                    const uint2 e = __ldg(&w.bm[td.word_base + ((uint32_t)g >> 5)]);
                    if (e.x >> (g & 31) & 1u) slot = e.y + __popc(e.x & ((1u << (g & 31)) - 1u));
                    if (slot >= capK) slot = 0xffffffffu;
                }
                w.upairs[l] = make_uint2(slot, (uint32_t)b);
            }
        for (int e0 = 0; e0 < D; e0 += 32 * 8) {
            float acc[8];
#pragma unroll
            for (int c = 0; c < 8; ++c) acc[c] = 0.f;
            for (int64_t l = lo; l < hi; ++l) {
                const int64_t g = __ldg(w.indices + l);
                if (g < 0 || g >= td.N) continue;
                const uint2 e = __ldg(&w.bm[td.word_base + ((uint32_t)g >> 5)]);
                if (!(e.x >> (g & 31) & 1u)) continue;
                const uint32_t slot = e.y + __popc(e.x & ((1u << (g & 31)) - 1u));
                if (slot >= capK) continue;
                const float* row = w.E + (size_t)slot * D;
#pragma unroll
                for (int c = 0; c < 8; ++c) {
                    const int idx = e0 + lane + c * 32;
                    if (idx < D) acc[c] += __ldg(row + idx);
                }
            }
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const int idx = e0 + lane + c * 32;
                if (idx < D) o[idx] = acc[c];
            }
        }
    }
}

cudaError_t tt_launch_pooling(tt_emb* h, float* out, cudaStream_t s)
{
    WsView& w = h->v;
    const int64_t nb = (int64_t)w.T * w.B;
    int64_t want = (nb + 7) / 8;  // 8 warps per CTA
    int grid = (int)(want < (int64_t)h->sm_count * 8 ? want : (int64_t)h->sm_count * 8);
    if (grid < 1) grid = 1;
    const int D = w.D;
    const bool vec_ok = (D % 4 == 0) && ((reinterpret_cast<uintptr_t>(out) & 15) == 0);
    if (!vec_ok) {
        k_pool_scalar<<<grid, 256, 0, s>>>(w, out);
        return cudaGetLastError();
    }
    const int D4 = D / 4;
    if (D4 <= 4) k_pool_vec<4, 1><<<grid, 256, 0, s>>>(w, out);
    else if (D4 <= 8) k_pool_vec<8, 1><<<grid, 256, 0, s>>>(w, out);
    else if (D4 <= 16) k_pool_vec<16, 1><<<grid, 256, 0, s>>>(w, out);
    else if (D4 <= 32) k_pool_vec<32, 1><<<grid, 256, 0, s>>>(w, out);
    else if (D4 <= 64) k_pool_vec<32, 2><<<grid, 256, 0, s>>>(w, out);
    else if (D4 <= 128) k_pool_vec<32, 4><<<grid, 256, 0, s>>>(w, out);
    else k_pool_vec<32, 8><<<grid, 256, 0, s>>>(w, out);
    return cudaGetLastError();
}
