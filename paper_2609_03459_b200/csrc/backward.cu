// Backward path (paper Sec. 3.2 backward, Eq. 2) and SGD.
//
//   1. sort:  the forward left one (slot, bag) pair per lookup; a counting sort by slot (counts -> exclusive
//             scan -> scatter) groups the lookups of every distinct row.  Hot rows would serialise global
//             atomics, so each CTA first aggregates the duplicates of its tile in shared memory (owner tags) and
//             issues one global atomic per aggregated row per tile.
//   2. dE:    segmented sum of grad_out rows over the sorted pairs.  Fixed-size chunks of sorted positions per
//             warp (skew-proof); segments that cross chunk borders leave partial sums which a second kernel
//             adds in position order.
//   3. last level: per group, C is rebuilt in shared memory; every row contributes C^T.dE to the slice of
//             the last core it selects and dE.D^T to the group's dC (summed over the rows sharing C before
//             going up, Eq. 2; the sum is the k-loop of the tensor-core product, so dC is written once).
//             The last core's slices are accumulated with vector reductions into TT_STRIPES L2-resident
//             partial copies, which are then added in a fixed order (shared-memory fp32 atomics measured
//             at 2.6 per clock per SM on this part, too slow for a CTA-private copy).
//   4. middle cores: dP_{k-1} of a parent = sum over its (contiguous) children; the gradient of slice i_k
//             = sum over the level-k nodes with that digit, enumerated by a second, digit-major bitmap sort.
//             Each output has exactly one owner, which sums in sorted order: no atomics.
#include "common.cuh"
#include "scan.cuh"
#include "mma.cuh"
#include "quad_mid.cuh"

#define HT_SIZE 4096
#define HT_TILE 2048
#define HT_EMPTY 0xffffffffu
#define RB 8  // rows per batch in the last-level kernel

// ---------------------------------------------------------------------------------------------- small utilities

__global__ void k_zero_u32_dev(uint32_t* p, const uint32_t* count, uint32_t extra)
{
    tt_pdl_enter();
    const uint32_t n = *count + extra;
    for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x) p[i] = 0u;
}

// zero the gradient that is not fully written by an owner kernel: core 0 (only the slices of present
// first digits are written later)
__global__ void k_zero_grads(WsView w)
{
    tt_pdl_enter();
    const int t = blockIdx.y;
    const TableDesc& td = w.tdesc[t];
    const int K = w.K;
    float* g0 = td.grad[0];
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < td.core_floats[0]; i += (int64_t)gridDim.x * blockDim.x) g0[i] = 0.f;
    (void)K;
}

// ---------------------------------------------------------------------------------------------- 1. sort by slot

// MODE 0: cnt[slot] += occurrences.  MODE 1: pairs[seg_start[slot] + claimed position] = (slot, bag).
//
// Aggregation of a tile's duplicates without a probing hash table (two shared-memory atomics per pair made the
// shared-memory atomic unit the limit of both passes): every pair stores a tag (low key bits, its number in the tile)
// into bucket h(key) with a plain store; after a barrier the bucket holds the tag of one of its writers.  That pair
// owns the bucket.  A pair with the owner's key is a duplicate: it counts itself in extra[h] (the only shared-memory
// atomic left, and only duplicates issue it) and the owner makes one global atomic for all of them.  A pair with another
// key lost the bucket and goes to the global counter by itself.  h takes the key bits above bit 19 as they are, so that
// bucket and the 20 low bits together identify the key and a 32-bit tag is enough.
#define TT_SORT0_TILES 24
#define HT_LOW_BITS 20
#define HT_ID_BITS 11
template <int MODE>
__global__ void __launch_bounds__(256) k_sort_pass(WsView w)
{
    tt_pdl_enter();
    static_assert(HT_TILE == (1 << HT_ID_BITS) && HT_SIZE == (1 << (32 - HT_LOW_BITS)) && HT_LOW_BITS + HT_ID_BITS <= 32, "tag layout");
    const uint2* __restrict__ upairs = w.upairs;
    const uint32_t capK = w.cap[w.K];
    __shared__ uint32_t tag[HT_SIZE];
    __shared__ uint32_t extra[HT_SIZE];   // duplicates of the owner's key; MODE 1: then the claimed base position
    const int64_t L = w.L;
    const int64_t ntiles = (L + HT_TILE - 1) / HT_TILE;
    const bool weighted = MODE == 1 && w.wsorted && (w.psw || w.pool_mean);
    for (int i = threadIdx.x; i < HT_SIZE; i += blockDim.x) extra[i] = 0u;
    // the first barrier of the tile loop orders this before the first atomic on extra
    auto emit = [&](uint32_t pos, const uint2& pr, int64_t l) {
        w.pairs[pos] = pr;
        if (weighted) {   // weighted / mean pooling: the pair's factor travels with it
            float a = w.psw ? __ldg(w.psw + l) : 1.f;
            if (w.pool_mean) {
                const int64_t gb = (int64_t)tt_find_table(w.tb[w.K], w.T, pr.x) * w.B + pr.y;
                const int64_t len = __ldg(w.offsets + gb + 1) - __ldg(w.offsets + gb);
                a /= (float)(len > 0 ? len : 1);
            }
            w.wsorted[pos] = a;
        }
    };
    enum { ROLE_NONE = 0, ROLE_OWNER = 1, ROLE_DUP = 2 };
    for (int64_t tile = blockIdx.x; tile < ntiles; tile += gridDim.x) {
        uint2 pr[HT_TILE / 256];
        uint32_t st[HT_TILE / 256];   // bucket (12 bits) | rank among the duplicates (12 bits) << 12 | role << 24
#pragma unroll
        for (int j = 0; j < HT_TILE / 256; ++j) {
            const int64_t l = tile * HT_TILE + j * 256 + threadIdx.x;
            pr[j] = l < L ? __ldcs(upairs + l) : make_uint2(HT_EMPTY, 0u);
            if (pr[j].x >= capK || (int64_t)pr[j].y >= w.B) pr[j].x = HT_EMPTY;  // invalid lookup (or malformed offsets)
        }
#pragma unroll
        for (int j = 0; j < HT_TILE / 256; ++j) {
            if (pr[j].x == HT_EMPTY) continue;
            const uint32_t low = pr[j].x & ((1u << HT_LOW_BITS) - 1u);
            const uint32_t h = ((pr[j].x >> HT_LOW_BITS) ^ ((low * 2654435761u) >> HT_LOW_BITS)) & (HT_SIZE - 1);
            st[j] = h;
            tag[h] = (low << HT_ID_BITS) | (uint32_t)(j * 256 + threadIdx.x);
        }
        __syncthreads();
#pragma unroll
        for (int j = 0; j < HT_TILE / 256; ++j) {
            if (pr[j].x == HT_EMPTY) continue;
            const uint32_t low = pr[j].x & ((1u << HT_LOW_BITS) - 1u);
            const uint32_t h = st[j];
            const uint32_t tg = tag[h];
            if ((tg >> HT_ID_BITS) == low) {
                if ((tg & (HT_TILE - 1)) == (uint32_t)(j * 256 + threadIdx.x)) st[j] = h | (ROLE_OWNER << 24);
                else if (MODE == 0) { atomicAdd(&extra[h], 1u); st[j] = h | (ROLE_DUP << 24); }
                else st[j] = h | ((atomicAdd(&extra[h], 1u) + 1u) << 12) | (ROLE_DUP << 24);
            } else {   // another key holds the bucket
                if (MODE == 0) atomicAdd(&w.cnt[pr[j].x], 1u);
                else emit(atomicAdd(&w.cnt[pr[j].x], 1u), pr[j], tile * HT_TILE + j * 256 + threadIdx.x);
            }
        }
        __syncthreads();
        // one global atomic per owner.  MODE 1 claims a run of positions directly on the scanned count array:
        // cnt[slot] starts as the segment start and ends as the segment end (= next segment's start)
#pragma unroll
        for (int j = 0; j < HT_TILE / 256; ++j) {
            if (pr[j].x == HT_EMPTY || (st[j] >> 24) != ROLE_OWNER) continue;
            const uint32_t h = st[j] & (HT_SIZE - 1);
            const uint32_t n = 1u + extra[h];
            if (MODE == 0) {
                atomicAdd(&w.cnt[pr[j].x], n);
                extra[h] = 0u;
            } else {
                const uint32_t base = atomicAdd(&w.cnt[pr[j].x], n);
                extra[h] = base;
                emit(base, pr[j], tile * HT_TILE + j * 256 + threadIdx.x);
            }
        }
        if (MODE == 1) {
            __syncthreads();
#pragma unroll
            for (int j = 0; j < HT_TILE / 256; ++j) {
                if (pr[j].x == HT_EMPTY || (st[j] >> 24) != ROLE_DUP) continue;
                emit(extra[st[j] & (HT_SIZE - 1)] + ((st[j] >> 12) & 0xfffu), pr[j], tile * HT_TILE + j * 256 + threadIdx.x);
            }
            __syncthreads();
#pragma unroll
            for (int j = 0; j < HT_TILE / 256; ++j)
                if (pr[j].x != HT_EMPTY && (st[j] >> 24) == ROLE_OWNER) extra[st[j] & (HT_SIZE - 1)] = 0u;
        }
    }
}

struct CntScan {
    WsView w;
    __device__ uint32_t size() const { return w.counters[CTR_LEVEL0 + w.K]; }
    __device__ int locate(uint32_t) const { return 0; }
    __device__ uint32_t value(uint32_t i, int) const { return w.cnt[i]; }
    __device__ void emit(uint32_t i, uint32_t excl, uint32_t, int) const { w.cnt[i] = excl; }
    __device__ void total(uint32_t tot) const { w.cnt[size()] = tot; }
};

cudaError_t tt_launch_bwd_sort(tt_emb* h, cudaStream_t s)
{
    WsView& w = h->v;
    const int zgrid = h->sm_count * 8;
    cudaError_t e;
    if ((e = tt_launch_pdl(k_zero_u32_dev, dim3(zgrid), dim3(256), 0, s, w.cnt, (const uint32_t*)(w.counters + CTR_LEVEL0 + w.K), 1u)) != cudaSuccess) return e;
    tt_note_launch();
    const int64_t ntiles = (w.L + HT_TILE - 1) / HT_TILE;
    int per_sm0 = 0, per_sm1 = 0;   // persistent grids sized to what is actually resident (no partial second wave)
    if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm0, k_sort_pass<0>, 256, 0)) != cudaSuccess) return e;
    if ((e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm1, k_sort_pass<1>, 256, 0)) != cudaSuccess) return e;
    auto grid_of = [&](int per_sm) {
        int64_t g = (int64_t)(per_sm < 1 ? 1 : per_sm) * h->sm_count;
        if (g > ntiles) g = ntiles;
        return (int)(g < 1 ? 1 : g);
    };
    // the counting pass as a grid of more CTAs than fit at once, TT_SORT0_TILES tiles each: the block scheduler then
    // balances the tiles' very different costs (a tile of popular rows aggregates to a few claims, one of unpopular rows
    // makes two thousand; as a resident grid the first CTA was done at 58 % of the kernel).  4 / 8 / 16 / 24 / 32 / 48
    // tiles per CTA: 2.92 / 2.68 / 2.57 / 2.52 / 2.54 / 2.68 ms for the sort, 2.62 ms with the resident grid
    int g0 = grid_of(per_sm0);
    {
        const int64_t many = (ntiles + TT_SORT0_TILES - 1) / TT_SORT0_TILES;
        if (many > g0) g0 = (int)many;
    }
    if ((e = tt_launch_pdl(k_sort_pass<0>, dim3(g0), dim3(256), 0, s, w)) != cudaSuccess) return e;
    tt_note_launch();
    CntScan cs{w};
    if ((e = tt_scan(cs, w.cap[w.K], w.scan_tmp, s)) != cudaSuccess) return e;
    if ((e = tt_launch_pdl(k_sort_pass<1>, dim3(grid_of(per_sm1)), dim3(256), 0, s, w)) != cudaSuccess) return e;
    tt_note_launch();
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------- 2. dE

// lane l of the warp owns float4 chunks l, l+32, ... of a row (VEC) or floats l, l+32, ... (!VEC)
template <bool VEC, int CPL>
struct RowAcc {
    float v[VEC ? 4 * CPL : CPL];
    __device__ void clear()
    {
#pragma unroll
        for (int i = 0; i < (VEC ? 4 * CPL : CPL); ++i) v[i] = 0.f;
    }
    // v += a * row (a = 1 gives exactly v + row)
    __device__ void add_row(const float* __restrict__ row, int D, int lane, float a = 1.f)
    {
        if (VEC) {
            const float4* r4 = reinterpret_cast<const float4*>(row);
#pragma unroll
            for (int c = 0; c < CPL; ++c) {
                const int ch = lane + c * 32;
                if (ch * 4 < D) {
                    const float4 x = __ldg(r4 + ch);
                    v[4 * c] = fmaf(a, x.x, v[4 * c]); v[4 * c + 1] = fmaf(a, x.y, v[4 * c + 1]);
                    v[4 * c + 2] = fmaf(a, x.z, v[4 * c + 2]); v[4 * c + 3] = fmaf(a, x.w, v[4 * c + 3]);
                }
            }
        } else {
#pragma unroll
            for (int c = 0; c < CPL; ++c) {
                const int i = lane + c * 32;
                if (i < D) v[c] = fmaf(a, __ldg(row + i), v[c]);
            }
        }
    }
    __device__ void store(float* __restrict__ row, int D, int lane) const
    {
        if (VEC) {
            float4* r4 = reinterpret_cast<float4*>(row);
#pragma unroll
            for (int c = 0; c < CPL; ++c) {
                const int ch = lane + c * 32;
                if (ch * 4 < D) r4[ch] = make_float4(v[4 * c], v[4 * c + 1], v[4 * c + 2], v[4 * c + 3]);
            }
        } else {
#pragma unroll
            for (int c = 0; c < CPL; ++c) {
                const int i = lane + c * 32;
                if (i < D) row[i] = v[c];
            }
        }
    }
};

template <bool VEC, int CPL>
__global__ void __launch_bounds__(256) k_dE(WsView w, const float* __restrict__ grad_out)
{
    tt_pdl_enter();
    const int lane = threadIdx.x & 31;
    const int64_t chunk = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint32_t U = w.counters[CTR_LEVEL0 + w.K];
    const uint32_t Ltot = w.cnt[U];
    const int64_t a64 = chunk * TT_DE_CHUNK;
    if (a64 >= Ltot) return;
    const uint32_t a = (uint32_t)a64;
    const uint32_t b = min(a + (uint32_t)TT_DE_CHUNK, Ltot);
    const int D = w.D;
    const size_t gstride = (size_t)w.T * D;
    const uint32_t prev = a > 0 ? w.pairs[a - 1].x : HT_EMPTY;
    const uint32_t next = b < Ltot ? w.pairs[b].x : HT_EMPTY;
    RowAcc<VEC, CPL> acc;
    acc.clear();
    uint32_t cur = w.pairs[a].x;
    int tcur = tt_find_table(w.tb[w.K], w.T, cur);
    bool seg_first = true;
    float* carry = w.carry + (size_t)chunk * 2 * D;
    for (uint32_t p0 = a; p0 < b; p0 += 32) {
        const uint2 mine = (p0 + lane < b) ? __ldg(&w.pairs[p0 + lane]) : make_uint2(HT_EMPTY, 0u);
        const bool weighted = w.wsorted && (w.psw || w.pool_mean);
        const float wmine = (weighted && p0 + lane < b) ? __ldg(&w.wsorted[p0 + lane]) : 1.f;
        const int n = (int)min(32u, b - p0);
        // four rows of grad_out in flight at a time (their addresses need the table of each pair's slot; positions are
        // sorted, so the table changes rarely), then the rows are folded in position order
        const int tmine = lane < n ? tt_find_table_from(w.tb[w.K], w.T, mine.x, tcur) : tcur;
        for (int j0 = 0; j0 < n; j0 += 4) {
            RowAcc<VEC, CPL> rowv[4];
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) {
                const int j = min(j0 + jj, n - 1);
                const uint32_t bag = __shfl_sync(0xffffffffu, mine.y, j);
                const int tj = __shfl_sync(0xffffffffu, tmine, j);
                rowv[jj].clear();
                if (j0 + jj < n) rowv[jj].add_row(grad_out + (size_t)bag * gstride + (size_t)tj * D, D, lane, 1.f);
            }
#pragma unroll
            for (int jj = 0; jj < 4; ++jj) {
                const int j = j0 + jj;
                if (j >= n) break;
                const uint32_t sl = __shfl_sync(0xffffffffu, mine.x, j);
                const float wj = __shfl_sync(0xffffffffu, wmine, j);
                if (sl != cur) {
                    const bool open_start = seg_first && prev == cur;
                    if (open_start) acc.store(carry, D, lane);  // head: started in an earlier chunk, ends here
                    else acc.store(w.E + (size_t)cur * D, D, lane);
                    acc.clear();
                    cur = sl;
                    seg_first = false;
                }
#pragma unroll
                for (int i = 0; i < (VEC ? 4 * CPL : CPL); ++i) acc.v[i] = fmaf(wj, rowv[jj].v[i], acc.v[i]);
            }
        }
        tcur = __shfl_sync(0xffffffffu, tmine, n - 1);
    }
    const bool open_start = seg_first && prev == cur;
    const bool open_end = next == cur;
    if (open_end) acc.store(carry + D, D, lane);        // tail: continues in the next chunk
    else if (open_start) acc.store(carry, D, lane);     // head
    else acc.store(w.E + (size_t)cur * D, D, lane);
}

// the chunk in which a border-crossing segment starts adds up the pieces in position order
template <bool VEC, int CPL>
__global__ void __launch_bounds__(256) k_dE_fix(WsView w)
{
    tt_pdl_enter();
    const int lane = threadIdx.x & 31;
    const int64_t chunk = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint32_t U = w.counters[CTR_LEVEL0 + w.K];
    const uint32_t Ltot = w.cnt[U];
    const int64_t a64 = chunk * TT_DE_CHUNK;
    if (a64 >= Ltot) return;
    const uint32_t a = (uint32_t)a64;
    const uint32_t b = min(a + (uint32_t)TT_DE_CHUNK, Ltot);
    if (b >= Ltot) return;
    const uint32_t first = w.pairs[a].x, last = w.pairs[b - 1].x;
    const uint32_t prev = a > 0 ? w.pairs[a - 1].x : HT_EMPTY;
    const uint32_t next = w.pairs[b].x;
    if (next != last) return;                         // nothing continues past this chunk
    if (first == last && prev == first) return;       // the segment started earlier: not the owner
    const int D = w.D;
    RowAcc<VEC, CPL> acc;
    acc.clear();
    acc.add_row(w.carry + ((size_t)chunk * 2 + 1) * D, D, lane);
    const int64_t nchunks = ((int64_t)Ltot + TT_DE_CHUNK - 1) / TT_DE_CHUNK;
    // A popular row spans thousands of chunks.  Look at 32 following chunks at once: every lane classifies one
    // ("whole chunk is this row and it goes on" = a tail piece to add; otherwise its head piece ends the row),
    // a ballot finds where the row ends, and the pieces are added in position order.
    for (int64_t c0 = chunk + 1; c0 < nchunks; c0 += 32) {
        const int64_t c2 = c0 + lane;
        bool through = false;
        if (c2 < nchunks) {
            const uint32_t a2 = (uint32_t)(c2 * TT_DE_CHUNK);
            const uint32_t b2 = min(a2 + (uint32_t)TT_DE_CHUNK, Ltot);
            const uint32_t last2 = w.pairs[b2 - 1].x;
            const uint32_t next2 = b2 < Ltot ? w.pairs[b2].x : HT_EMPTY;
            through = last2 == last && next2 == last;
        }
        const unsigned stops = __ballot_sync(0xffffffffu, !through);   // chunks beyond the end count as stops
        const int nthrough = stops ? __ffs(stops) - 1 : 32;
#pragma unroll 8
        for (int i = 0; i < nthrough; ++i) acc.add_row(w.carry + ((size_t)(c0 + i) * 2 + 1) * D, D, lane);
        if (nthrough < 32) {
            if (c0 + nthrough < nchunks) acc.add_row(w.carry + (size_t)(c0 + nthrough) * 2 * D, D, lane);
            break;
        }
    }
    acc.store(w.E + (size_t)last * D, D, lane);
}

// Fast variant for D/4 <= 32 float4 chunks per row: LPR lanes cover a row, 32/LPR rows per load instruction,
// NF load instructions issued back to back, then the rows are folded in position order.  Each sub-warp keeps
// its own partial sum; the sub-warps are combined only when a segment ends.  Segment starts inside a batch of
// 32 positions are found once with a ballot, so a window without a start costs 4 adds per load and nothing else.
template <int LPR, bool WT>
__global__ void __launch_bounds__(256, 5) k_dE_fast(WsView w, const float* __restrict__ grad_out)
{
    tt_pdl_enter();
    constexpr int RPI = 32 / LPR, NF = 4;
    const int lane = threadIdx.x & 31, sub = lane / LPR, lr = lane % LPR;
    const int64_t chunk = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint32_t U = w.counters[CTR_LEVEL0 + w.K];
    const uint32_t Ltot = w.cnt[U];
    const int64_t a64 = chunk * TT_DE_CHUNK;
    if (a64 >= Ltot) return;
    const uint32_t a = (uint32_t)a64;
    const uint32_t b = min(a + (uint32_t)TT_DE_CHUNK, Ltot);
    const int D = w.D, D4 = D >> 2;
    const bool lane_on = lr < D4;
    const uint32_t prev = a > 0 ? w.pairs[a - 1].x : HT_EMPTY;
    const uint32_t next = b < Ltot ? w.pairs[b].x : HT_EMPTY;
    const float4* __restrict__ G4 = reinterpret_cast<const float4*>(grad_out);
    float4* __restrict__ E4 = reinterpret_cast<float4*>(w.E);
    float4* carry4 = reinterpret_cast<float4*>(w.carry + (size_t)chunk * 2 * D);
    float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
    uint32_t cur = w.pairs[a].x;
    bool seg_first = true;
    // close the running segment: combine the sub-warps, store (sub-warp 0 writes), clear
    auto close_segment = [&]() {
        float4* dst = (seg_first && prev == cur) ? carry4 : E4 + (size_t)cur * D4;   // head piece or whole segment
#pragma unroll
        for (int o = LPR; o < 32; o <<= 1) {
            acc.x += __shfl_xor_sync(0xffffffffu, acc.x, o); acc.y += __shfl_xor_sync(0xffffffffu, acc.y, o);
            acc.z += __shfl_xor_sync(0xffffffffu, acc.z, o); acc.w += __shfl_xor_sync(0xffffffffu, acc.w, o);
        }
        if (sub == 0 && lane_on) dst[lr] = acc;
        acc = make_float4(0.f, 0.f, 0.f, 0.f);
        seg_first = false;
    };
    uint32_t last_slot = cur;  // slot of the position before the current batch
    for (uint32_t p0 = a; p0 < b; p0 += 32) {
        const uint2 mine = (p0 + lane < b) ? __ldcs(&w.pairs[p0 + lane]) : make_uint2(HT_EMPTY, 0u);
        const float wmine = (WT && p0 + lane < b) ? __ldcs(&w.wsorted[p0 + lane]) : 1.f;   // factor of this lane's pair
        const int n = (int)min(32u, b - p0);
        // row index of this lane's pair inside grad_out viewed as [B*T][D]
        const uint32_t grow = lane < n ? mine.y * (uint32_t)w.T + (uint32_t)tt_find_table(w.tb[w.K], w.T, mine.x) : 0u;
        uint32_t before = __shfl_up_sync(0xffffffffu, mine.x, 1);
        if (lane == 0) before = last_slot;
        const unsigned starts = __ballot_sync(0xffffffffu, lane < n && mine.x != before);  // bit j: position j opens a segment
        last_slot = __shfl_sync(0xffffffffu, mine.x, n - 1);
        for (int j0 = 0; j0 < n; j0 += NF * RPI) {
            float4 v[NF];
#pragma unroll
            for (int jj = 0; jj < NF; ++jj) {
                const int j = j0 + jj * RPI + sub;
                const uint32_t gr = __shfl_sync(0xffffffffu, grow, j & 31);
                v[jj] = (j < n && lane_on) ? __ldg(G4 + (size_t)gr * D4 + lr) : make_float4(0.f, 0.f, 0.f, 0.f);
                if (WT) {
                    const float wj = __shfl_sync(0xffffffffu, wmine, j & 31);
                    v[jj].x *= wj; v[jj].y *= wj; v[jj].z *= wj; v[jj].w *= wj;
                }
            }
#pragma unroll
            for (int jj = 0; jj < NF; ++jj) {
                const int j = j0 + jj * RPI;
                if (((starts >> j) & ((1u << RPI) - 1u)) == 0u) {
                    acc.x += v[jj].x; acc.y += v[jj].y; acc.z += v[jj].z; acc.w += v[jj].w;
                } else {
#pragma unroll
                    for (int h = 0; h < RPI; ++h) {
                        if ((starts >> (j + h)) & 1u) {
                            close_segment();
                            cur = __shfl_sync(0xffffffffu, mine.x, (j + h) & 31);
                        }
                        if (sub == h) { acc.x += v[jj].x; acc.y += v[jj].y; acc.z += v[jj].z; acc.w += v[jj].w; }
                    }
                }
            }
        }
    }
    // last segment of the chunk
    {
        const bool open_start = seg_first && prev == cur;
        float4* dst = next == cur ? carry4 + D4 : (open_start ? carry4 : E4 + (size_t)cur * D4);  // tail / head / whole
#pragma unroll
        for (int o = LPR; o < 32; o <<= 1) {
            acc.x += __shfl_xor_sync(0xffffffffu, acc.x, o); acc.y += __shfl_xor_sync(0xffffffffu, acc.y, o);
            acc.z += __shfl_xor_sync(0xffffffffu, acc.z, o); acc.w += __shfl_xor_sync(0xffffffffu, acc.w, o);
        }
        if (sub == 0 && lane_on) dst[lr] = acc;
    }
}

// D = 64 (256-byte rows): the 32 grad_out rows of a batch of sorted positions are fetched into an 8 KB per-warp
// buffer with cp.async (all in flight at once, no staging registers), then every lane walks the batch in position
// order owning two of the 64 columns: one shared-memory load and two adds per row, a coalesced 256-byte store when a
// segment ends, and no shuffles to combine partial sums.  About half the instructions per lookup of k_dE_fast, which
// was bound by instruction issue.  Chunks, carries and the fix-up pass are those of k_dE / k_dE_fast.
#define DE_WARPS 7   // 4 CTAs x 7 warps x 8 KB of staging per SM
template <int DD, bool WT>   // DD = D: 64 (two columns per lane), 32 (one) or 16 (one, lanes 0..15)
__global__ void __launch_bounds__(32 * DE_WARPS, 4) k_dE_stage(WsView w, const float* __restrict__ grad_out)
{
    tt_pdl_enter();
    static_assert(DD == 64 || DD == 32 || DD == 16, "a lane owns DD / 32 columns (one column on the first DD lanes below 32)");
    constexpr int R4 = DD / 4;          // float4 pieces per row
    constexpr int RPI = 32 / R4;        // rows per cp.async instruction
    constexpr int VPL = DD >= 32 ? DD / 32 : 1;   // columns per lane
    extern __shared__ __align__(16) float4 de_buf[];   // [DE_WARPS][32 rows][R4 float4]
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, sub = lane / R4, lr = lane % R4;
    float4* buf = de_buf + (size_t)wid * 32 * R4;
    const float* bufv = reinterpret_cast<const float*>(buf);
    const int64_t chunk = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const uint32_t U = w.counters[CTR_LEVEL0 + w.K];
    const uint32_t Ltot = w.cnt[U];
    const int64_t a64 = chunk * TT_DE_CHUNK;
    if (a64 >= Ltot) return;
    const uint32_t a = (uint32_t)a64;
    const uint32_t b = min(a + (uint32_t)TT_DE_CHUNK, Ltot);
    const uint32_t prev = a > 0 ? w.pairs[a - 1].x : HT_EMPTY;
    const uint32_t next = b < Ltot ? w.pairs[b].x : HT_EMPTY;
    const float4* __restrict__ G4 = reinterpret_cast<const float4*>(grad_out);
    float* carry = w.carry + (size_t)chunk * 2 * DD;
    const uint32_t* __restrict__ tbK = w.tb[w.K];
    float acc[VPL], part[VPL];
#pragma unroll
    for (int x = 0; x < VPL; ++x) { acc[x] = 0.f; part[x] = 0.f; }
    uint32_t cur = w.pairs[a].x;
    bool seg_first = true;
    uint32_t last_slot = cur;
    // slot range of the table the chunk is in: positions are sorted, so a batch rarely leaves it
    int tcur = tt_find_table(tbK, w.T, cur);
    uint32_t t_lo = tbK[tcur], t_hi = tbK[tcur + 1];
    // two-level sum: rows are added into a per-batch partial (at most 32 terms) which is added to the segment's sum at
    // the end of the batch, so the rounding error of a long segment grows with sqrt(length / 32), not sqrt(length)
    auto store_row = [&](float* dst, bool with_part) {
        if (VPL == 2) reinterpret_cast<float2*>(dst)[lane] = make_float2(acc[0] + (with_part ? part[0] : 0.f), acc[VPL - 1] + (with_part ? part[VPL - 1] : 0.f));
        else if (lane < DD) dst[lane] = acc[0] + (with_part ? part[0] : 0.f);
    };
    auto close_segment = [&]() {
        store_row((seg_first && prev == cur) ? carry : w.E + (size_t)cur * DD, true);   // head piece or whole segment
#pragma unroll
        for (int x = 0; x < VPL; ++x) { acc[x] = 0.f; part[x] = 0.f; }
        seg_first = false;
    };
    uint2 mine = (a + lane < b) ? __ldcs(&w.pairs[a + lane]) : make_uint2(HT_EMPTY, 0u);
    float wmine = (WT && a + lane < b) ? __ldcs(&w.wsorted[a + lane]) : 1.f;
    for (uint32_t p0 = a; p0 < b; p0 += 32) {
        const int n = (int)min(32u, b - p0);
        int tl = tcur;
        if (!__all_sync(0xffffffffu, lane >= n || (mine.x >= t_lo && mine.x < t_hi))) {
            tl = lane < n ? tt_find_table(tbK, w.T, mine.x) : tcur;
            tcur = __shfl_sync(0xffffffffu, tl, n - 1);
            t_lo = tbK[tcur];
            t_hi = tbK[tcur + 1];
        }
        const uint32_t grow = mine.y * (uint32_t)w.T + (uint32_t)tl;   // row of grad_out viewed as [B*T][DD]
        uint32_t before = __shfl_up_sync(0xffffffffu, mine.x, 1);
        if (lane == 0) before = last_slot;
        const unsigned starts = __ballot_sync(0xffffffffu, lane < n && mine.x != before);   // bit j: position j opens a segment
        last_slot = __shfl_sync(0xffffffffu, mine.x, n - 1);
        if (n == 32) {   // all windows of a chunk but its last: no per-row test
#pragma unroll
            for (int jj = 0; jj < 32 / RPI; ++jj) {
                const int j = RPI * jj + sub;
                const uint32_t gr = __shfl_sync(0xffffffffu, grow, j);
                tt_cp_async16(buf + j * R4 + lr, G4 + (size_t)gr * R4 + lr);
            }
        } else {
#pragma unroll
            for (int jj = 0; jj < 32 / RPI; ++jj) {
                const int j = RPI * jj + sub;
                const uint32_t gr = __shfl_sync(0xffffffffu, grow, j);
                if (j < n) tt_cp_async16(buf + j * R4 + lr, G4 + (size_t)gr * R4 + lr);
            }
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
        // the pairs of the next batch arrive while the rows are in flight
        const uint2 cur_pairs = mine;
        const float cur_w = wmine;
        if (p0 + 32 < b) {
            mine = (p0 + 32 + lane < b) ? __ldcs(&w.pairs[p0 + 32 + lane]) : make_uint2(HT_EMPTY, 0u);
            if (WT) wmine = (p0 + 32 + lane < b) ? __ldcs(&w.wsorted[p0 + 32 + lane]) : 1.f;
        }
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncwarp();
        auto add_row = [&](int j) {
            float x[VPL];
            if (VPL == 2) {
                const float2 v = reinterpret_cast<const float2*>(bufv)[j * 32 + lane];
                x[0] = v.x; x[VPL - 1] = v.y;
            } else x[0] = bufv[j * DD + (lane & (DD - 1))];
            if (WT) {
                const float wj = __shfl_sync(0xffffffffu, cur_w, j);
#pragma unroll
                for (int c = 0; c < VPL; ++c) x[c] *= wj;
            }
#pragma unroll
            for (int c = 0; c < VPL; ++c) part[c] += x[c];
        };
        // eight rows at a time; a run of eight without a segment start (popular rows: most lookups sit in segments far
        // longer than a batch) is added without looking at the start bits
        for (int j0 = 0; j0 < n; j0 += 8) {
            if (j0 + 8 <= n && ((starts >> j0) & 0xffu) == 0u) {
#pragma unroll
                for (int jj = 0; jj < 8; ++jj) add_row(j0 + jj);
            } else if (j0 + 8 <= n && ((starts >> j0) & 0xffu) == 0xffu) {
                // eight starts in a row (rows looked up once: most distinct rows): the first closes the running segment,
                // the next seven rows are whole segments of one row each and are copied out, the eighth opens a new one
                close_segment();
#pragma unroll
                for (int jj = 0; jj < 7; ++jj) {
                    const uint32_t sj = __shfl_sync(0xffffffffu, cur_pairs.x, j0 + jj);
                    add_row(j0 + jj);
                    float* dst = w.E + (size_t)sj * DD;
                    if (VPL == 2) reinterpret_cast<float2*>(dst)[lane] = make_float2(part[0], part[VPL - 1]);
                    else if (lane < DD) dst[lane] = part[0];
#pragma unroll
                    for (int c = 0; c < VPL; ++c) part[c] = 0.f;
                }
                cur = __shfl_sync(0xffffffffu, cur_pairs.x, j0 + 7);
                add_row(j0 + 7);
            } else {
                const int j1 = min(j0 + 8, n);
                for (int j = j0; j < j1; ++j) {
                    if ((starts >> j) & 1u) {
                        close_segment();
                        cur = __shfl_sync(0xffffffffu, cur_pairs.x, j);
                    }
                    add_row(j);
                }
            }
        }
#pragma unroll
        for (int c = 0; c < VPL; ++c) { acc[c] += part[c]; part[c] = 0.f; }
        __syncwarp();
    }
    {   // last segment of the chunk: tail / head / whole
        const bool open_start = seg_first && prev == cur;
        store_row(next == cur ? carry + DD : (open_start ? carry : w.E + (size_t)cur * DD), false);
    }
}

template <bool VEC, int CPL>
static cudaError_t launch_dE_t(tt_emb* h, const float* grad_out, cudaStream_t s)
{
    const int64_t chunks = (h->v.L + TT_DE_CHUNK - 1) / TT_DE_CHUNK;
    const int grid = (int)((chunks + 7) / 8);
    if (grid > 0) {
        const int D4 = h->D / 4;
        const bool wt = h->v.wsorted && (h->v.psw || h->v.pool_mean);
        if (VEC && (h->D == 64 || h->D == 32 || h->D == 16)) {
            const size_t smem = (size_t)DE_WARPS * 32 * (h->D / 4) * sizeof(float4);
            auto kern = h->D == 64 ? (wt ? k_dE_stage<64, true> : k_dE_stage<64, false>)
                      : h->D == 32 ? (wt ? k_dE_stage<32, true> : k_dE_stage<32, false>) : (wt ? k_dE_stage<16, true> : k_dE_stage<16, false>);
            cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
            if (e != cudaSuccess) return e;
            const int sgrid = (int)((chunks + DE_WARPS - 1) / DE_WARPS);
            if ((e = tt_launch_pdl(kern, dim3(sgrid), dim3(32 * DE_WARPS), smem, s, h->v, grad_out)) != cudaSuccess) return e;
            tt_note_launch();
        } else
        if (VEC && D4 <= 8) { if (wt) k_dE_fast<8, true><<<grid, 256, 0, s>>>(h->v, grad_out); else k_dE_fast<8, false><<<grid, 256, 0, s>>>(h->v, grad_out); tt_note_launch(); }
        else if (VEC && D4 <= 16) { if (wt) k_dE_fast<16, true><<<grid, 256, 0, s>>>(h->v, grad_out); else k_dE_fast<16, false><<<grid, 256, 0, s>>>(h->v, grad_out); tt_note_launch(); }
        else if (VEC && D4 <= 32) { if (wt) k_dE_fast<32, true><<<grid, 256, 0, s>>>(h->v, grad_out); else k_dE_fast<32, false><<<grid, 256, 0, s>>>(h->v, grad_out); tt_note_launch(); }
        else { k_dE<VEC, CPL><<<grid, 256, 0, s>>>(h->v, grad_out); tt_note_launch(); }
        cudaError_t ef = tt_launch_pdl(k_dE_fix<VEC, CPL>, dim3(grid), dim3(256), 0, s, h->v);
        if (ef != cudaSuccess) return ef;
        tt_note_launch();
    }
    return cudaGetLastError();
}

cudaError_t tt_launch_bwd_dE(tt_emb* h, const float* grad_out, cudaStream_t s)
{
    const int D = h->D;
    const bool vec = (D % 4 == 0) && ((reinterpret_cast<uintptr_t>(grad_out) & 15) == 0);
    if (vec) {
        if (D <= 128) return launch_dE_t<true, 1>(h, grad_out, s);
        if (D <= 256) return launch_dE_t<true, 2>(h, grad_out, s);
        if (D <= 512) return launch_dE_t<true, 4>(h, grad_out, s);
        return launch_dE_t<true, 8>(h, grad_out, s);
    }
    if (D <= 128) return launch_dE_t<false, 4>(h, grad_out, s);
    if (D <= 256) return launch_dE_t<false, 8>(h, grad_out, s);
    if (D <= 512) return launch_dE_t<false, 16>(h, grad_out, s);
    return launch_dE_t<false, 32>(h, grad_out, s);
}

// ---------------------------------------------------------------------------------------------- 3. last level

// generic fallback (any shape): the whole CTA works on one group at a time
__device__ __forceinline__ void tt_sweep_bwd_generic(const WsView& w, const TableDesc& td, uint32_t g0, uint32_t g1,
                                                     float* gk, float* Pl, float* Cs, float* dCs, float* dEs)
{
    const int K = w.K, kl = K - 1, km = K - 2;
    const int Pm = td.P[K - 1], rb = td.r[K - 1], dK = td.d[kl], D = w.D;
    const int sliceK = td.slice_floats[kl];
    const uint32_t nK = (uint32_t)td.n[kl];
    for (int i = threadIdx.x; i < Pm * rb; i += blockDim.x) dCs[i] = 0.f;
    __syncthreads();
    for (uint32_t jpos = g0; jpos < g1; ++jpos) {
        const uint32_t g = K >= 3 ? w.tnode[K - 1][jpos] : jpos;
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
        for (uint32_t ub = u0; ub < u1; ub += RB) {
            const int nr = (int)min((uint32_t)RB, u1 - ub);
            for (int i = threadIdx.x; i < nr * D; i += blockDim.x) dEs[i] = w.E[(size_t)ub * D + i];
            __syncthreads();
            // dG_K[i_K][b][j] += sum_p C[p][b] * dE[p][j]     ("dD = C^T . dE")
            for (int it = threadIdx.x; it < nr * sliceK; it += blockDim.x) {
                const int rr = it / sliceK, e = it - rr * sliceK;
                const int bb = e / dK, j = e - bb * dK;
                const float* de = dEs + rr * D + j;
                float acc = 0.f;
                for (int p = 0; p < Pm; ++p) acc = fmaf(Cs[p * rb + bb], de[p * dK], acc);
                const uint32_t iK = w.val[K][ub + rr] % nK;
                atomicAdd(gk + (size_t)iK * sliceK + e, acc);
            }
            // dC[p][b] += sum_j dE[p][j] * D[b][j]             ("dC = dE . D^T", summed over the group: Eq. 2)
            for (int it = threadIdx.x; it < Pm * rb; it += blockDim.x) {
                const int p = it / rb, bb = it - p * rb;
                float acc = 0.f;
                for (int rr = 0; rr < nr; ++rr) {
                    const uint32_t iK = w.val[K][ub + rr] % nK;
                    const float* Dsl = td.core[kl] + (size_t)iK * sliceK + bb * dK;
                    const float* de = dEs + rr * D + p * dK;
                    for (int j = 0; j < dK; ++j) acc = fmaf(de[j], __ldg(Dsl + j), acc);
                }
                dCs[it] += acc;
            }
            __syncthreads();
        }
        // hand dC to the level above (K = 2: it is the gradient of the first core's slice itself)
        float* dst = K >= 3 ? w.dP[K - 1] + (size_t)g * w.stride[K - 1] : td.grad[0] + (size_t)val * td.slice_floats[0];
        for (int i = threadIdx.x; i < Pm * rb; i += blockDim.x) { dst[i] = dCs[i]; dCs[i] = 0.f; }
        __syncthreads();
    }
}

// ---- register-tiled backward of the last two levels (same shape variants as the forward sweep) ----------------
//
// One warp per group.  C is rebuilt in shared memory, then two passes over the group's rows:
//   pass A  dC[p][b] += sum_j dE_u[p][j] * D_u[b][j]: a lane owns TP rows p for all b (TP*RB accumulators) and
//           one of 32*TP/PM concurrent rows; D streams as float4 (16 FMAs per load at TP = 4).  The row-slots
//           are then combined by a reduce-scatter of warp shuffles and each lane writes its share of dC (Eq. 2:
//           the sum over the rows sharing C is formed before anything moves up a level).
//   pass B  dG_K[i_K][b][j] += sum_p C[p][b] * dE_u[p][j]: a lane owns RB*TP/PM values of b for all p
//           (PM*RB*TP/PM registers of C) and streams the float4 rows of dE (8*TP FMAs per load at PM = 16).
//           The lane's 4*RB*TP/PM results are contiguous in the slice and go out as vector reductions.

__device__ __forceinline__ void tt_red_v4(float* p, float x, float y, float z, float wv)
{
    asm volatile("red.global.add.v4.f32 [%0], {%1, %2, %3, %4};" ::"l"(p), "f"(x), "f"(y), "f"(z), "f"(wv) : "memory");
}

// RBP > 0: C is stored as [P][RBP + 8] (rows of r_{K-1} = RBP values, stride RBP + 8 floats), the layout whose transposed
// fragment loads in the tensor-core dG pass are free of bank conflicts; RBP = 0: plain [M][cols].
template <int M, int CPL, int RBP = 0>
__device__ __forceinline__ void tt_warp_mid_b(const float* As, const float* __restrict__ Bsl, float* Cs, int ra, int cols, int lane)
{
    const int c4n = cols >> 2;
    const int LA = (c4n / CPL) < 32 ? (c4n / CPL) : 32;
    const int NS = 32 / LA;
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
            for (int m = 0; m < M; ++m) {
                const int col = 4 * (ll + i * LA);
                float* dst = RBP > 0 ? Cs + (m * (cols / (RBP > 0 ? RBP : 1)) + col / (RBP > 0 ? RBP : 1)) * (RBP + 8) + col % (RBP > 0 ? RBP : 1)
                                     : Cs + m * cols + col;
                *reinterpret_cast<float4*>(dst) = make_float4(acc[i][m][0], acc[i][m][1], acc[i][m][2], acc[i][m][3]);
            }
    }
}

template <int PM, int RB_, int TP>
__device__ __forceinline__ void tt_warp_rows_dC(const WsView& w, const TableDesc& td, uint32_t u0, uint32_t u1, uint32_t row_base,
                                                float* dPdst, int lane)
{
    constexpr int LR = PM / TP, RW = 32 / LR, NV = TP * RB_;
    const int q = lane % LR, slot = lane / LR;
    const int K = w.K;
    const float* __restrict__ GK = td.core[K - 1];
    const uint32_t* __restrict__ rows = w.val[K];
    const float4* __restrict__ E4 = reinterpret_cast<const float4*>(w.E);
    float dc[NV];
#pragma unroll
    for (int i = 0; i < NV; ++i) dc[i] = 0.f;
    for (uint32_t ub = u0; ub < u1; ub += RW) {
        const uint32_t u = ub + slot;
        const bool act = u < u1;
        const uint32_t iK = act ? rows[u] - row_base : 0u;
        const float4* __restrict__ D4 = reinterpret_cast<const float4*>(GK + (size_t)iK * (RB_ * 4));
        float4 e[TP];
#pragma unroll
        for (int i = 0; i < TP; ++i) e[i] = act ? __ldg(E4 + (size_t)u * PM + TP * q + i) : make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int b = 0; b < RB_; ++b) {
            const float4 d = __ldg(D4 + b);
#pragma unroll
            for (int i = 0; i < TP; ++i) {
                float a = dc[i * RB_ + b];
                a = fmaf(e[i].x, d.x, a); a = fmaf(e[i].y, d.y, a); a = fmaf(e[i].z, d.z, a); a = fmaf(e[i].w, d.w, a);
                dc[i * RB_ + b] = a;
            }
        }
    }
    // reduce-scatter over the RW row-slots: after the step with lane bit o, a lane keeps the half selected by that bit
    int base = 0;
    int n = NV;
#pragma unroll
    for (int o = 16; o >= LR; o >>= 1) {
        n >>= 1;
        const bool hi = (lane & o) != 0;
#pragma unroll
        for (int i = 0; i < NV / 2; ++i) {
            if (i < n) {
                const float send = hi ? dc[i] : dc[i + n];
                const float recv = __shfl_xor_sync(0xffffffffu, send, o);
                dc[i] = (hi ? dc[i + n] : dc[i]) + recv;
            }
        }
        base += hi ? n : 0;
    }
    // the lane now holds dc[0..n) = dC values [base, base+n) of its TP rows (value v <-> row v / RB_, column v % RB_)
    constexpr int NF = NV / RW;
    float* dst = dPdst + (TP * q + base / RB_) * RB_ + base % RB_;
    if constexpr (NF >= 4) {
#pragma unroll
        for (int i = 0; i < NF / 4; ++i)
            *reinterpret_cast<float4*>(dst + 4 * i) = make_float4(dc[4 * i], dc[4 * i + 1], dc[4 * i + 2], dc[4 * i + 3]);
    } else {
#pragma unroll
        for (int i = 0; i < NF; ++i) dst[i] = dc[i];
    }
}

template <int PM, int RB_, int TP>
__device__ __forceinline__ void tt_warp_rows_dG(const float* Cs, const WsView& w, uint32_t u0, uint32_t u1, uint32_t row_base,
                                                float* gk, int lane)
{
    constexpr int LR = PM / TP, RW = 32 / LR, BQ = RB_ / LR;
    const int q = lane % LR, slot = lane / LR;
    const uint32_t* __restrict__ rows = w.val[w.K];
    const float4* __restrict__ E4 = reinterpret_cast<const float4*>(w.E);
    float c2[PM][BQ];
#pragma unroll
    for (int p = 0; p < PM; ++p)
#pragma unroll
        for (int bi = 0; bi < BQ; ++bi) c2[p][bi] = Cs[p * RB_ + BQ * q + bi];
    for (uint32_t ub = u0; ub < u1; ub += RW) {
        const uint32_t u = ub + slot;
        const bool act = u < u1;
        const uint32_t ur = act ? u : u0;
        float4 acc[BQ];
#pragma unroll
        for (int bi = 0; bi < BQ; ++bi) acc[bi] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int p = 0; p < PM; ++p) {
            const float4 e = __ldg(E4 + (size_t)ur * PM + p);
#pragma unroll
            for (int bi = 0; bi < BQ; ++bi) {
                acc[bi].x = fmaf(c2[p][bi], e.x, acc[bi].x);
                acc[bi].y = fmaf(c2[p][bi], e.y, acc[bi].y);
                acc[bi].z = fmaf(c2[p][bi], e.z, acc[bi].z);
                acc[bi].w = fmaf(c2[p][bi], e.w, acc[bi].w);
            }
        }
        if (act) {
            const uint32_t iK = rows[u] - row_base;
            float* dst = gk + (size_t)iK * (RB_ * 4) + (BQ * q) * 4;
#pragma unroll
            for (int bi = 0; bi < BQ; ++bi) tt_red_v4(dst + 4 * bi, acc[bi].x, acc[bi].y, acc[bi].z, acc[bi].w);
        }
    }
}

// ---- tensor-core (3xTF32, m16n8k8) forms of the two row passes, d_K = 4 ---------------------------------------
//
// pass A  dC[p][b] = sum over the group's rows u and j of dE_u[p][j] * D_u[b][j]:  M = 16 rows p, N = 8 values of b,
//         K = 8 = two rows x 4 columns j.  The sum over the rows that share C (Eq. 2) is the accumulation over
//         k-steps, so dC ends up complete in the accumulator fragments (PM*RB/32 registers) and is written once:
//         no cross-lane reduction at all.
// pass B  dG_K[i_K(u)][b][j] += sum_p C[p][b] * dE_u[p][j]:  M = 16 values of b, K = 8 rows p, N = 8 = two rows x 4
//         columns j; C^T fragments are fixed per group.  Results leave as 8-byte vector reductions.
__device__ __forceinline__ void tt_red_v2(float* p, float x, float y)
{
    asm volatile("red.global.add.v2.f32 [%0], {%1, %2};" ::"l"(p), "f"(x), "f"(y) : "memory");
}

template <int PM, int RB_>
__device__ __forceinline__ void tt_warp_rows_dC_mma(const WsView& w, const TableDesc& td, uint32_t u0, uint32_t u1, uint32_t row_base,
                                                    float* dPdst, int lane)
{
    static_assert(PM == 4 || PM == 8 || PM % 16 == 0, "4 or 8 rows of dC fill the first rows of one row tile, else whole tiles");
    constexpr bool HALF = PM < 16;   // rows PM..15 of the tile stay zero and are not stored
    constexpr int MT = HALF ? 1 : PM / 16, NT = RB_ / 8;
    const int g = lane >> 2, t = lane & 3;
    const bool rowok = !HALF || g < PM;
    const int K = w.K;
    const float* __restrict__ GK = td.core[K - 1];
    const uint32_t* __restrict__ rows = w.val[K];
    // acc: tensor-core accumulators, folded into tot (rounded fp32 adds) every sixteen row pairs: the tensor core adds
    // with truncation, so a long chain (a group can have hundreds of rows) would drift by chain length * 2^-24
    float acc[MT][NT][4], tot[MT][NT][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int x = 0; x < 4; ++x) { acc[mt][nt][x] = 0.f; tot[mt][nt][x] = 0.f; }
    for (uint32_t ub0 = u0; ub0 < u1; ub0 += 32) {
    const uint32_t ub1 = min(ub0 + 32u, u1);
#pragma unroll 2
    for (uint32_t ub = ub0; ub < ub1; ub += 2) {
        const bool two = ub + 1 < u1;
        const uint32_t ua = ub, uc = two ? ub + 1 : ub;
        const float* __restrict__ Ea = w.E + (size_t)ua * (PM * 4) + t;
        const float* __restrict__ Ec = w.E + (size_t)uc * (PM * 4) + t;
        const float* __restrict__ Da = GK + (size_t)(rows[ua] - row_base) * (RB_ * 4) + t;
        const float* __restrict__ Dc = GK + (size_t)(rows[uc] - row_base) * (RB_ * 4) + t;
        Tf32Pair a[MT][4];
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
            a[mt][0] = tt_split_tf32(rowok ? __ldg(Ea + (16 * mt + g) * 4) : 0.f);
            a[mt][1] = tt_split_tf32(HALF ? 0.f : __ldg(Ea + (16 * mt + g + 8) * 4));
            a[mt][2] = tt_split_tf32(two && rowok ? __ldg(Ec + (16 * mt + g) * 4) : 0.f);
            a[mt][3] = tt_split_tf32(two && !HALF ? __ldg(Ec + (16 * mt + g + 8) * 4) : 0.f);
        }
        float bv[NT][2];
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            bv[nt][0] = __ldg(Da + (8 * nt + g) * 4);
            bv[nt][1] = __ldg(Dc + (8 * nt + g) * 4);
        }
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            Tf32Pair b[2];
            b[0] = tt_split_tf32(bv[nt][0]);
            b[1] = tt_split_tf32(bv[nt][1]);
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) tt_mma_3xtf32(acc[mt][nt], a[mt], b);
        }
    }
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt)
#pragma unroll
            for (int x = 0; x < 4; ++x) { tot[mt][nt][x] += acc[mt][nt][x]; acc[mt][nt][x] = 0.f; }
    }
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            if (rowok) *reinterpret_cast<float2*>(dPdst + (16 * mt + g) * RB_ + 8 * nt + 2 * t) = make_float2(tot[mt][nt][0], tot[mt][nt][1]);
            if (!HALF) *reinterpret_cast<float2*>(dPdst + (16 * mt + g + 8) * RB_ + 8 * nt + 2 * t) = make_float2(tot[mt][nt][2], tot[mt][nt][3]);
        }
}

template <int PM, int RB_>
__device__ __forceinline__ void tt_warp_rows_dG_mma(const float* Cs, const WsView& w, uint32_t u0, uint32_t u1, uint32_t row_base,
                                                    float* gk, int lane)
{
    constexpr bool KHALF = PM == 4;   // p = 4..7 of the one k step do not exist: zero operands
    constexpr bool BHALF = RB_ == 8;  // b = 8..15 of the one row tile do not exist: zero operands, not reduced
    constexpr int MT = BHALF ? 1 : RB_ / 16, KT = KHALF ? 1 : PM / 8;
    const int g = lane >> 2, t = lane & 3;
    const uint32_t* __restrict__ rows = w.val[w.K];
    Tf32Pair a[MT][KT][4];   // A[m = b][k = p] = C[p][b]
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int kt = 0; kt < KT; ++kt) {
            a[mt][kt][0] = tt_split_tf32(Cs[(8 * kt + t) * (RB_ + 8) + 16 * mt + g]);
            a[mt][kt][1] = tt_split_tf32(BHALF ? 0.f : Cs[(8 * kt + t) * (RB_ + 8) + 16 * mt + g + 8]);
            a[mt][kt][2] = tt_split_tf32(KHALF ? 0.f : Cs[(8 * kt + t + 4) * (RB_ + 8) + 16 * mt + g]);
            a[mt][kt][3] = tt_split_tf32(KHALF || BHALF ? 0.f : Cs[(8 * kt + t + 4) * (RB_ + 8) + 16 * mt + g + 8]);
        }
    const int rb_ = g >> 2, jb = g & 3;       // B fragment: row rb_ of the pair, column jb of dE
    const int rc = t >> 1, jc = 2 * (t & 1);  // C fragment: row rc of the pair, columns jc, jc+1
#pragma unroll 2
    for (uint32_t ub = u0; ub < u1; ub += 2) {
        const uint32_t ul = min(ub + (uint32_t)rb_, u1 - 1);
        const bool valid = ub + (uint32_t)rb_ < u1;
        const float* __restrict__ El = w.E + (size_t)ul * (PM * 4) + jb;
        float acc[MT][4];
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) { acc[mt][0] = 0.f; acc[mt][1] = 0.f; acc[mt][2] = 0.f; acc[mt][3] = 0.f; }
        float bv[KT][2];
#pragma unroll
        for (int kt = 0; kt < KT; ++kt) {
            bv[kt][0] = valid ? __ldg(El + (8 * kt + t) * 4) : 0.f;
            bv[kt][1] = valid && !KHALF ? __ldg(El + (8 * kt + t + 4) * 4) : 0.f;
        }
#pragma unroll
        for (int kt = 0; kt < KT; ++kt) {
            Tf32Pair b[2];
            b[0] = tt_split_tf32(bv[kt][0]);
            b[1] = tt_split_tf32(bv[kt][1]);
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) tt_mma_3xtf32(acc[mt], a[mt][kt], b);
        }
        const uint32_t us = ub + (uint32_t)rc;
        if (us < u1) {
            float* dst = gk + (size_t)(rows[us] - row_base) * (RB_ * 4) + jc;
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
                tt_red_v2(dst + (16 * mt + g) * 4, acc[mt][0], acc[mt][1]);
                if (!BHALF) tt_red_v2(dst + (16 * mt + g + 8) * 4, acc[mt][2], acc[mt][3]);
            }
        }
    }
}

// Both row passes in one loop over the group's row pairs: the row ids and the dE rows come from memory once (the
// second fragment layout of dE is served by L1), dC accumulates across the loop, dG_K tiles leave per pair.
template <int PM, int RB_, int CS = RB_ + 8>   // CS: row stride of C in shared memory
__device__ __forceinline__ void tt_warp_rows_bwd_mma(const float* Cs, const WsView& w, const TableDesc& td, uint32_t u0, uint32_t u1,
                                                     uint32_t row_base, float* dPdst, float* gk, int lane)
{
    static_assert(PM == 4 || PM == 8 || PM % 16 == 0, "4 or 8 rows of dC fill the first rows of one row tile, else whole tiles");
    constexpr bool HALF = PM < 16;                // rows PM..15 of the dC tile stay zero and are not stored
    constexpr bool KHALF = PM == 4;               // p = 4..7 of the one dG k step do not exist: zero operands
    constexpr int MT = HALF ? 1 : PM / 16, NT = RB_ / 8;     // dC tiles: rows p, columns b
    constexpr bool BHALF = RB_ == 8;              // b = 8..15 of the one dG row tile do not exist: zero operands, not reduced
    constexpr int MT2 = BHALF ? 1 : RB_ / 16, KT2 = KHALF ? 1 : PM / 8;   // dG tiles: rows b, k = p
    const int g = lane >> 2, t = lane & 3;
    const bool rowok = !HALF || g < PM;
    const int K = w.K;
    const float* __restrict__ GK = td.core[K - 1];
    const uint32_t* __restrict__ rows = w.val[K];
    Tf32Pair ct[MT2][KT2][4];   // A[m = b][k = p] = C[p][b]
#pragma unroll
    for (int mt = 0; mt < MT2; ++mt)
#pragma unroll
        for (int kt = 0; kt < KT2; ++kt) {
            ct[mt][kt][0] = tt_split_tf32(Cs[(8 * kt + t) * CS + 16 * mt + g]);
            ct[mt][kt][1] = tt_split_tf32(BHALF ? 0.f : Cs[(8 * kt + t) * CS + 16 * mt + g + 8]);
            ct[mt][kt][2] = tt_split_tf32(KHALF ? 0.f : Cs[(8 * kt + t + 4) * CS + 16 * mt + g]);
            ct[mt][kt][3] = tt_split_tf32(KHALF || BHALF ? 0.f : Cs[(8 * kt + t + 4) * CS + 16 * mt + g + 8]);
        }
    // C of 8 or 4 rows would fill half or a quarter of the row tiles of dC: there the product runs transposed,
    // dC^T[b][p] += sum_{(row, j)} D_row[b][j] * dE_row[p][j], M = b, N = 8 columns p (PM = 4: four of them zero), K = 8 =
    // two rows x 4 columns j: RB_/16 tiles per pair instead of RB_/8
    constexpr bool TR = HALF && RB_ >= 16;
    constexpr int MTT = RB_ / 16;
    constexpr int DM = TR ? MTT : MT, DN = TR ? 1 : NT;
    float dc[DM][DN][4], dct[DM][DN][4];   // tensor-core accumulators and their rounded running sums (see tt_warp_rows_dC_mma)
#pragma unroll
    for (int mt = 0; mt < DM; ++mt)
#pragma unroll
        for (int nt = 0; nt < DN; ++nt)
#pragma unroll
            for (int x = 0; x < 4; ++x) { dc[mt][nt][x] = 0.f; dct[mt][nt][x] = 0.f; }
    const int rb_ = g >> 2, jb = g & 3;       // dG B fragment: row rb_ of the pair, column jb of dE
    const int rc = t >> 1, jc = 2 * (t & 1);  // dG C fragment: row rc of the pair, columns jc, jc+1
    for (uint32_t ub0 = u0; ub0 < u1; ub0 += 32) {
    const uint32_t ub1 = min(ub0 + 32u, u1);
    for (uint32_t ub = ub0; ub < ub1; ub += 2) {
        const bool two = ub + 1 < u1;
        const uint32_t ua = ub, uc = two ? ub + 1 : ub;
        const uint32_t iKa = rows[ua] - row_base, iKc = rows[uc] - row_base;
        const float* __restrict__ Ea = w.E + (size_t)ua * (PM * 4);
        const float* __restrict__ Ec = w.E + (size_t)uc * (PM * 4);
        // ---- loads: dE as A fragments (dC), slices as B fragments (dC), dE as B fragments (dG)
        float av[MT][4], bv[NT][2], ev[KT2][2];
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
            // (transposed: av[0][0], av[0][2] are the B fragment dE_a[p = g][j = t], dE_c[g][t])
            av[mt][0] = rowok ? __ldg(Ea + (16 * mt + g) * 4 + t) : 0.f;
            av[mt][1] = HALF ? 0.f : __ldg(Ea + (16 * mt + g + 8) * 4 + t);
            av[mt][2] = two && rowok ? __ldg(Ec + (16 * mt + g) * 4 + t) : 0.f;
            av[mt][3] = two && !HALF ? __ldg(Ec + (16 * mt + g + 8) * 4 + t) : 0.f;
        }
        const float* __restrict__ Da = GK + (size_t)iKa * (RB_ * 4) + t;
        const float* __restrict__ Dc = GK + (size_t)iKc * (RB_ * 4) + t;
#pragma unroll
        for (int nt = 0; nt < NT; ++nt) {
            // (transposed: bv[2 mt][.], bv[2 mt + 1][.] are the A fragment rows b = 16 mt + g and + 8 of D_a, D_c)
            bv[nt][0] = __ldg(Da + (8 * nt + g) * 4);
            bv[nt][1] = two || !TR ? __ldg(Dc + (8 * nt + g) * 4) : 0.f;
        }
        const bool valid = rb_ == 0 || two;
        const float* __restrict__ El = (rb_ == 0 ? Ea : Ec) + jb;
#pragma unroll
        for (int kt = 0; kt < KT2; ++kt) {
            ev[kt][0] = valid ? __ldg(El + (8 * kt + t) * 4) : 0.f;
            ev[kt][1] = valid && !KHALF ? __ldg(El + (8 * kt + t + 4) * 4) : 0.f;
        }
        // ---- dC += dE . D^T
        if constexpr (TR) {
            Tf32Pair b[2];
            b[0] = tt_split_tf32(av[0][0]);
            b[1] = tt_split_tf32(av[0][2]);
#pragma unroll
            for (int mt = 0; mt < MTT; ++mt) {
                Tf32Pair a[4];
                a[0] = tt_split_tf32(bv[2 * mt][0]);
                a[1] = tt_split_tf32(bv[2 * mt + 1][0]);
                a[2] = tt_split_tf32(bv[2 * mt][1]);
                a[3] = tt_split_tf32(bv[2 * mt + 1][1]);
                tt_mma_3xtf32(dc[mt][0], a, b);
            }
        } else {
            Tf32Pair a[MT][4];
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                for (int x = 0; x < 4; ++x) a[mt][x] = tt_split_tf32(av[mt][x]);
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                Tf32Pair b[2];
                b[0] = tt_split_tf32(bv[nt][0]);
                b[1] = tt_split_tf32(bv[nt][1]);
#pragma unroll
                for (int mt = 0; mt < MT; ++mt) tt_mma_3xtf32(dc[mt][nt], a[mt], b);
            }
        }
        // ---- dG_K[i_K] += C^T . dE
        {
            float acc[MT2][4];
#pragma unroll
            for (int mt = 0; mt < MT2; ++mt) { acc[mt][0] = 0.f; acc[mt][1] = 0.f; acc[mt][2] = 0.f; acc[mt][3] = 0.f; }
#pragma unroll
            for (int kt = 0; kt < KT2; ++kt) {
                Tf32Pair b[2];
                b[0] = tt_split_tf32(ev[kt][0]);
                b[1] = tt_split_tf32(ev[kt][1]);
#pragma unroll
                for (int mt = 0; mt < MT2; ++mt) tt_mma_3xtf32(acc[mt], ct[mt][kt], b);
            }
            if (rc == 0 || two) {
                float* dst = gk + (size_t)(rc == 0 ? iKa : iKc) * (RB_ * 4) + jc;
#pragma unroll
                for (int mt = 0; mt < MT2; ++mt) {
                    tt_red_v2(dst + (16 * mt + g) * 4, acc[mt][0], acc[mt][1]);
                    if (!BHALF) tt_red_v2(dst + (16 * mt + g + 8) * 4, acc[mt][2], acc[mt][3]);
                }
            }
        }
    }
#pragma unroll
    for (int mt = 0; mt < DM; ++mt)
#pragma unroll
        for (int nt = 0; nt < DN; ++nt)
#pragma unroll
            for (int x = 0; x < 4; ++x) { dct[mt][nt][x] += dc[mt][nt][x]; dc[mt][nt][x] = 0.f; }
    }
    if constexpr (TR) {
        // the lane holds dC[p = 2t][b], dC[2t + 1][b] for b = 16 mt + g and b + 8
        if (2 * t < PM) {
#pragma unroll
            for (int mt = 0; mt < MTT; ++mt) {
                dPdst[(2 * t) * RB_ + 16 * mt + g] = dct[mt][0][0];
                dPdst[(2 * t + 1) * RB_ + 16 * mt + g] = dct[mt][0][1];
                dPdst[(2 * t) * RB_ + 16 * mt + g + 8] = dct[mt][0][2];
                dPdst[(2 * t + 1) * RB_ + 16 * mt + g + 8] = dct[mt][0][3];
            }
        }
    } else {
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int nt = 0; nt < NT; ++nt) {
                if (rowok) *reinterpret_cast<float2*>(dPdst + (16 * mt + g) * RB_ + 8 * nt + 2 * t) = make_float2(dct[mt][nt][0], dct[mt][nt][1]);
                if (!HALF) *reinterpret_cast<float2*>(dPdst + (16 * mt + g + 8) * RB_ + 8 * nt + 2 * t) = make_float2(dct[mt][nt][2], dct[mt][nt][3]);
            }
    }
}

template <int PM, int RB_, int TP, int M, int CPL, bool MMA>
__device__ __forceinline__ void tt_sweep_bwd_fast(const WsView& w, const TableDesc& td, uint32_t g1, float* gk,
                                                  float* As, float* Cs, uint32_t* next, int lane)
{
    const int K = w.K, km = K - 2;
    const int ra = td.r[km], cols = td.d[km] * RB_;
    const uint32_t nK = (uint32_t)td.n[K - 1];
    for (;;) {   // groups are handed out through a shared counter: their row counts differ widely
        uint32_t j = 0;
        if (lane == 0) j = atomicAdd(next, 1u);
        j = __shfl_sync(0xffffffffu, j, 0);
        if (j >= g1) break;
        const uint32_t g = w.tnode[K - 1][j];   // units are cut from the digit-major order (see forward.cu)
        const uint32_t val = w.val[K - 1][g];
        const float* src = tt_left_operand(w, td, K - 1, g);
        for (int i = lane; i < M * ra; i += 32) {
            const int m = i / ra, a = i - m * ra;
            As[a * M + m] = __ldg(src + i);
        }
        __syncwarp();
        const uint32_t im = val % (uint32_t)td.n[km];
        tt_warp_mid_b<M, CPL, (MMA ? RB_ : 0)>(As, td.core[km] + (size_t)im * td.slice_floats[km], Cs, ra, cols, lane);
        __syncwarp();
        const uint32_t u0 = w.cstart[K - 1][g], u1 = w.cstart[K - 1][g + 1];
        if constexpr (MMA) {
            // small C (rank 16): one fused loop over the row pairs is faster; larger C: two passes keep the register
            // footprint low enough for twice the resident warps (measured on the 60-table configuration)
            if constexpr (PM * RB_ <= 256) {
                tt_warp_rows_bwd_mma<PM, RB_>(Cs, w, td, u0, u1, val * nK, w.dP[K - 1] + (size_t)g * w.stride[K - 1], gk, lane);
            } else {
                tt_warp_rows_dC_mma<PM, RB_>(w, td, u0, u1, val * nK, w.dP[K - 1] + (size_t)g * w.stride[K - 1], lane);
                tt_warp_rows_dG_mma<PM, RB_>(Cs, w, u0, u1, val * nK, gk, lane);
            }
        } else {
            tt_warp_rows_dC<PM, RB_, TP>(w, td, u0, u1, val * nK, w.dP[K - 1] + (size_t)g * w.stride[K - 1], lane);
            tt_warp_rows_dG<PM, RB_, TP>(Cs, w, u0, u1, val * nK, gk, lane);
        }
        __syncwarp();
    }
}

// The fused-loop shapes with the intermediate products of NG = 16 / MROWS neighbouring groups formed together on the
// tensor cores, as in the forward sweep (quad_mid.cuh): one group at a time, every group read its whole slice of core
// K-1 (16 KB at rank 32) for a product of MROWS rows, which made the L1/L2 path the limit where groups hold few rows.
template <int PM, int RB_, int MROWS, int KTMAX>
__device__ __forceinline__ void tt_sweep_bwd_quad(const WsView& w, const TableDesc& td, uint32_t g1, float* gk, float* Cs4,
                                                  uint32_t* next, int lane)
{
    constexpr int COLS = PM / MROWS * RB_;   // d_{K-1} * r_{K-1}
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
        uint32_t gq = 0, valq = 0, imq = 0, u0q = 0, u1q = 0;
        const float* srcq = nullptr;
        if (lane < cnt) {
            gq = w.tnode[K - 1][base + lane];   // position in the digit-major order -> group
            valq = w.val[K - 1][gq];
            imq = valq % (uint32_t)td.n[km];
            srcq = tt_left_operand(w, td, K - 1, gq);
            u0q = w.cstart[K - 1][gq];
            u1q = w.cstart[K - 1][gq + 1];
        }
        tt_quad_mid<COLS, MROWS, KTMAX, RB_>(td.core[km], td.slice_floats[km], ra, cnt, imq, srcq, Cs4, lane);
        __syncwarp();
        for (int q = 0; q < cnt; ++q) {
            const uint32_t g = __shfl_sync(0xffffffffu, gq, q), val = __shfl_sync(0xffffffffu, valq, q);
            const uint32_t u0 = __shfl_sync(0xffffffffu, u0q, q), u1 = __shfl_sync(0xffffffffu, u1q, q);
            tt_warp_rows_bwd_mma<PM, RB_, RB_ + 4>(Cs4 + (size_t)q * (PM * (RB_ + 4)), w, td, u0, u1, val * nK,
                                                   w.dP[K - 1] + (size_t)g * w.stride[K - 1], gk, lane);
        }
        __syncwarp();
    }
}

// One CTA (4 warps) per work unit (table, q); last-core gradients go to one of TT_STRIPES L2-resident partial
// copies with vector reductions, added up in fixed stripe order by k_reduce_gpart.
template <int V>
__global__ void __launch_bounds__(128, (V == 5 || V == 6 || V == 8 || V == 9 || V == 1) ? 6 : 0) k_sweep_bwd(WsView w, int pl_floats, int c_floats, int vbase)
{
    tt_pdl_enter();
    extern __shared__ __align__(16) float sm[];
    const int t = w.vlist[vbase + blockIdx.y], q = blockIdx.x;
    const uint2 rng = w.unit_rng[t * w.units_per_table + q];
    const uint32_t g0 = rng.x, g1 = rng.y;
    const TableDesc& td = w.tdesc[t];
    const int stripe = (blockIdx.x + blockIdx.y) % TT_STRIPES;
    float* gk = w.gpart + (size_t)stripe * w.gpart_stride + td.gpart_off;
    if (V < 0) {
        float* Pl = sm;
        float* Cs = Pl + pl_floats;
        float* dCs = Cs + c_floats;
        float* dEs = dCs + c_floats;
        tt_sweep_bwd_generic(w, td, g0, g1, gk, Pl, Cs, dCs, dEs);
        return;
    }
    __shared__ uint32_t next;
    if (threadIdx.x == 0) next = g0;
    __syncthreads();
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    float* As = sm + (size_t)wid * (pl_floats + c_floats);
    float* Cs = As + pl_floats;
    if (V == 0) tt_sweep_bwd_fast<16, 32, 4, 4, 1, true>(w, td, g1, gk, As, Cs, &next, lane);
    if (V == 1) tt_sweep_bwd_quad<16, 16, 4, 4>(w, td, g1, gk, sm + (size_t)wid * (4 * 16 * 20), &next, lane);
    if (V == 2) tt_sweep_bwd_fast<16, 8, 4, 4, 1, true>(w, td, g1, gk, As, Cs, &next, lane);
    if (V == 3) tt_sweep_bwd_fast<32, 32, 4, 4, 2, true>(w, td, g1, gk, As, Cs, &next, lane);
    if (V == 4) tt_sweep_bwd_fast<32, 64, 2, 8, 2, false>(w, td, g1, gk, As, Cs, &next, lane);
    if (V == 5) tt_sweep_bwd_quad<8, 32, 2, 4>(w, td, g1, gk, sm + (size_t)wid * (8 * 8 * 36), &next, lane);
    if (V == 6) tt_sweep_bwd_quad<8, 16, 2, 4>(w, td, g1, gk, sm + (size_t)wid * (8 * 8 * 20), &next, lane);
    if (V == 7) tt_sweep_bwd_fast<8, 8, 2, 2, 1, false>(w, td, g1, gk, As, Cs, &next, lane);   // 8 x 8: the FP32 pipe wins (0.39 against 0.41 ms)
    if (V == 8) tt_sweep_bwd_quad<4, 32, 2, 4>(w, td, g1, gk, sm + (size_t)wid * (8 * 4 * 36), &next, lane);
    if (V == 9) tt_sweep_bwd_quad<4, 16, 2, 4>(w, td, g1, gk, sm + (size_t)wid * (8 * 4 * 20), &next, lane);
    if (V == 10) tt_sweep_bwd_fast<4, 8, 2, 2, 1, false>(w, td, g1, gk, As, Cs, &next, lane);
}

// fixed-order sum of the partial copies of the last core's gradient
__global__ void __launch_bounds__(256) k_reduce_gpart(WsView w)
{
    tt_pdl_enter();
    const int t = blockIdx.y;
    const TableDesc& td = w.tdesc[t];
    const int kl = w.K - 1;
    const int64_t n = td.core_floats[kl];
    const float* src = w.gpart + td.gpart_off;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x) {
        float s = 0.f;
#pragma unroll
        for (int q = 0; q < TT_STRIPES; ++q) s += src[(size_t)q * w.gpart_stride + i];
        td.grad[kl][i] = s;
        if (w.fused_lr != 0.f) td.core[kl][i] = td.core[kl][i] - w.fused_lr * s;   // nothing reads the last core after the sweeps
    }
}

template <int V>
static cudaError_t launch_sweep_bwd(tt_emb* h, int max_pl, int max_c, cudaStream_t s)
{
    const int n = h->vcount[V + 1];
    if (n == 0) return cudaSuccess;
    // tensor-core variants keep C with padded rows (stride r_{K-1} + 8 floats)
    if (V == 0) max_c = 16 * (32 + 8);
    if (V == 1) max_c = 16 * (16 + 8);
    if (V == 2) max_c = 16 * (8 + 8);
    if (V == 3) max_c = 32 * (32 + 8);
    if (V == 5) max_c = 8 * (32 + 8);
    if (V == 6) max_c = 8 * (16 + 8);
    if (V == 8) max_c = 4 * (32 + 8);
    if (V == 9) max_c = 4 * (16 + 8);
    size_t smem = V < 0 ? (size_t)(max_pl + 2 * max_c + RB * h->D) * sizeof(float)
                        : (size_t)4 * (max_pl + max_c) * sizeof(float);
    if (V == 5) smem = (size_t)4 * 8 * 8 * 36 * sizeof(float);    // eight C tiles per warp, rows padded by four floats
    if (V == 6) smem = (size_t)4 * 8 * 8 * 20 * sizeof(float);
    if (V == 8) smem = (size_t)4 * 8 * 4 * 36 * sizeof(float);
    if (V == 9) smem = (size_t)4 * 8 * 4 * 20 * sizeof(float);
    if (V == 1) smem = (size_t)4 * 4 * 16 * 20 * sizeof(float);   // four C tiles per warp
    cudaError_t e = cudaFuncSetAttribute(k_sweep_bwd<V>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    if ((e = tt_stage_begin(h, 9 + TT_NUM_VARIANTS + 1 + V + 1, s)) != cudaSuccess) return e;
    if ((e = tt_launch_pdl(k_sweep_bwd<V>, dim3(h->units_per_table, n), dim3(128), smem, s, h->v, max_pl, max_c, h->vbase[V + 1])) != cudaSuccess) return e;
    tt_note_launch();
    if ((e = tt_stage_end(h, 9 + TT_NUM_VARIANTS + 1 + V + 1, s)) != cudaSuccess) return e;
    return cudaGetLastError();
}

cudaError_t tt_launch_bwd_contraction(tt_emb* h, cudaStream_t s)
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
    cudaError_t e;
    if ((e = cudaMemsetAsync(w.gpart, 0, (size_t)TT_STRIPES * w.gpart_stride * sizeof(float), s)) != cudaSuccess) return e;
    k_zero_grads<<<dim3(64, h->T), 256, 0, s>>>(w);
    tt_note_launch();
    // P_k of the levels below K-1 are still in pbuf from the forward (K = 4 only)
    // tables of different shape variants are independent: their kernels run side by side on forked streams
    int nvar = 0;
    for (int vi = 0; vi <= TT_NUM_VARIANTS; ++vi) nvar += h->vcount[vi] > 0 ? 1 : 0;
    const bool fork = nvar > 1 && !h->serial;
    if (fork && (e = tt_fork(h, s, 4)) != cudaSuccess) return e;
    int slot = 0;
    auto next_stream = [&](int vi) { return (fork && h->vcount[vi] > 0) ? h->side[(slot++) & 3] : s; };
    if ((e = launch_sweep_bwd<-1>(h, max_pl, max_c, next_stream(0))) != cudaSuccess) return e;
    if ((e = launch_sweep_bwd<0>(h, max_pl, max_c, next_stream(1))) != cudaSuccess) return e;
    if ((e = launch_sweep_bwd<1>(h, max_pl, max_c, next_stream(2))) != cudaSuccess) return e;
    if ((e = launch_sweep_bwd<2>(h, max_pl, max_c, next_stream(3))) != cudaSuccess) return e;
    if ((e = launch_sweep_bwd<3>(h, max_pl, max_c, next_stream(4))) != cudaSuccess) return e;
    if ((e = launch_sweep_bwd<4>(h, max_pl, max_c, next_stream(5))) != cudaSuccess) return e;
    if ((e = launch_sweep_bwd<5>(h, max_pl, max_c, next_stream(6))) != cudaSuccess) return e;
    if ((e = launch_sweep_bwd<6>(h, max_pl, max_c, next_stream(7))) != cudaSuccess) return e;
    if ((e = launch_sweep_bwd<7>(h, max_pl, max_c, next_stream(8))) != cudaSuccess) return e;
    if ((e = launch_sweep_bwd<8>(h, max_pl, max_c, next_stream(9))) != cudaSuccess) return e;
    if ((e = launch_sweep_bwd<9>(h, max_pl, max_c, next_stream(10))) != cudaSuccess) return e;
    if ((e = launch_sweep_bwd<10>(h, max_pl, max_c, next_stream(11))) != cudaSuccess) return e;
    if (fork && (e = tt_join(h, s, 4)) != cudaSuccess) return e;
    if ((e = tt_launch_pdl(k_reduce_gpart, dim3(32, h->T), dim3(256), 0, s, w)) != cudaSuccess) return e;
    tt_note_launch();
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------- 4. middle cores

__device__ __forceinline__ uint32_t tt_tkey(const TableDesc& td, int k, uint32_t val)
{
    // digit-major key of a level-k node: i_k * (number of possible parents) + parent prefix value
    const uint32_t nk = (uint32_t)td.n[k - 1];
    return (val % nk) * td.prefix_space[k - 1] + val / nk;
}

__global__ void k_tmark(WsView w, int k)
{
    tt_pdl_enter();
    const uint32_t count = w.counters[CTR_LEVEL0 + k];
    for (uint32_t v = blockIdx.x * blockDim.x + threadIdx.x; v < count; v += gridDim.x * blockDim.x) {
        const int t = tt_find_table(w.tb[k], w.T, v);
        const TableDesc& td = w.tdesc[t];
        const uint32_t key = tt_tkey(td, k, w.val[k][v]);
        atomicOr(&w.tbm[k][td.tword_base[k] + (key >> 5)].x, 1u << (key & 31));
    }
}

struct TPopScan {
    WsView w;
    int k;
    __device__ uint32_t size() const { return w.ttotal_words[k]; }
    __device__ int locate(uint32_t) const { return 0; }
    __device__ uint32_t value(uint32_t i, int) const { return __popc(w.tbm[k][i].x); }
    __device__ void emit(uint32_t i, uint32_t excl, uint32_t, int) const { w.tbm[k][i].y = excl; }
    __device__ void total(uint32_t) const {}
};

__device__ __forceinline__ uint32_t tt_trank(const WsView& w, const TableDesc& td, int k, uint32_t key)
{
    const uint2 e = w.tbm[k][td.tword_base[k] + (key >> 5)];
    return e.y + __popc(e.x & ((1u << (key & 31)) - 1u));
}

__global__ void k_tfill(WsView w, int k)
{
    tt_pdl_enter();
    const uint32_t count = w.counters[CTR_LEVEL0 + k];
    for (uint32_t v = blockIdx.x * blockDim.x + threadIdx.x; v < count; v += gridDim.x * blockDim.x) {
        const int t = tt_find_table(w.tb[k], w.T, v);
        const TableDesc& td = w.tdesc[t];
        w.tnode[k][tt_trank(w, td, k, tt_tkey(td, k, w.val[k][v]))] = v;
    }
}

// dP_{k-1}[parent] (or the first core's gradient slice when k = 2) = sum over children v of
//   out[m][a] = sum_{j,b} dP_k[v][(m*d_k + j)*r_k + b] * G_k[i_k(v)][a][j][b]
// one CTA per parent, children in sorted order; the slice is staged in shared memory (padded rows)
__global__ void __launch_bounds__(256) k_mid_down(WsView w, int k)
{
    tt_pdl_enter();
    extern __shared__ float sm[];
    const uint32_t count = w.counters[CTR_LEVEL0 + k - 1];
    for (uint32_t pn = blockIdx.x; pn < count; pn += gridDim.x) {
        const int t = tt_find_table(w.tb[k - 1], w.T, pn);
        const TableDesc& td = w.tdesc[t];
        if (td.midfast[k] >= 0) continue;  // handled by k_mid_mma + k_mid_sum
        const int kc = k - 1;
        const int M = td.P[kc], ra = td.r[kc], cols = td.d[kc] * td.r[kc + 1];
        const int ld = cols + 1;
        float* Bs = sm;                  // ra * ld
        float* dPs = sm + ra * ld;       // M * cols
        const int nout = M * ra;
        // each thread owns outputs o = tid, tid + 256, ... (at most 16 per thread: M*ra <= 4096)
        float acc[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) acc[i] = 0.f;
        const uint32_t c0 = w.cstart[k - 1][pn], c1 = w.cstart[k - 1][pn + 1];
        for (uint32_t v = c0; v < c1; ++v) {
            const uint32_t ik = w.val[k][v] % (uint32_t)td.n[kc];
            const float* Bsl = td.core[kc] + (size_t)ik * td.slice_floats[kc];
            for (int i = threadIdx.x; i < ra * cols; i += blockDim.x) Bs[(i / cols) * ld + (i % cols)] = __ldg(Bsl + i);
            const float* dp = w.dP[k] + (size_t)v * w.stride[k];
            for (int i = threadIdx.x; i < M * cols; i += blockDim.x) dPs[i] = dp[i];
            __syncthreads();
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const int o = threadIdx.x + i * 256;
                if (o < nout) {
                    const int m = o / ra, a = o - m * ra;
                    const float* x = dPs + m * cols;
                    const float* y = Bs + a * ld;
                    float s = 0.f;
                    for (int c = 0; c < cols; ++c) s = fmaf(x[c], y[c], s);
                    acc[i] += s;
                }
            }
            __syncthreads();
        }
        float* dst;
        if (k == 2) dst = td.grad[0] + (size_t)w.val[1][pn] * td.slice_floats[0];
        else dst = w.dP[k - 1] + (size_t)pn * w.stride[k - 1];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const int o = threadIdx.x + i * 256;
            if (o < nout) dst[o] = acc[i];
        }
    }
}

// gradient of slice i_k of core k (1-based, 2 <= k <= K-1) of table t:
//   dG_k[i_k][a][c] = sum over level-k nodes v with digit i_k of sum_m P_{k-1}[parent(v)][m][a] * dP_k[v][m*cols + c]
// one CTA per (table, slice); nodes come from the digit-major list, i.e. in ascending parent order
__global__ void __launch_bounds__(256) k_mid_slice(WsView w, int k)
{
    tt_pdl_enter();
    extern __shared__ float sm[];
    const int t = blockIdx.y;
    const TableDesc& td = w.tdesc[t];
    const int kc = k - 1;
    if ((int)blockIdx.x >= td.n[kc] || td.midfast[k] >= 0) return;
    const uint32_t ik = blockIdx.x;
    const int M = td.P[kc], ra = td.r[kc], cols = td.d[kc] * td.r[kc + 1];
    const int nout = ra * cols;
    float* Pls = sm;             // M * ra
    float* dPs = sm + M * ra;    // M * cols
    const uint32_t space = td.prefix_space[k - 1];
    const uint32_t j0 = tt_trank(w, td, k, ik * space), j1 = tt_trank(w, td, k, (ik + 1) * space);
    float* dst = td.grad[kc] + (size_t)ik * td.slice_floats[kc];
    for (int o0 = 0; o0 < nout; o0 += 256 * 16) {
        float acc[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) acc[i] = 0.f;
        for (uint32_t jn = j0; jn < j1; ++jn) {
            const uint32_t v = w.tnode[k][jn];
            const float* pl = tt_left_operand(w, td, k, v);
            for (int i = threadIdx.x; i < M * ra; i += blockDim.x) Pls[i] = pl[i];
            const float* dp = w.dP[k] + (size_t)v * w.stride[k];
            for (int i = threadIdx.x; i < M * cols; i += blockDim.x) dPs[i] = dp[i];
            __syncthreads();
#pragma unroll
            for (int i = 0; i < 16; ++i) {
                const int o = o0 + threadIdx.x + i * 256;
                if (o < nout) {
                    const int a = o / cols, c = o - a * cols;
                    float s = 0.f;
                    for (int m = 0; m < M; ++m) s = fmaf(Pls[m * ra + a], dPs[m * cols + c], s);
                    acc[i] += s;
                }
            }
            __syncthreads();
        }
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const int o = o0 + threadIdx.x + i * 256;
            if (o < nout) dst[o] = acc[i];
        }
    }
}

// ---- tensor-core middle-core backward (P_{k-1} = 4 or 2 rows, r_{k-1} in {16,32}, d_k * r_k in {32,64,128}) ----
//
// One CTA of 4 warps per (table, slice i_k).  The nodes with digit i_k arrive in ascending parent order from the
// digit-major list, 16 or 32 stacked rows (node, m) per pass: NQ = 4..16 nodes, staged with cp.async into padded
// shared-memory tiles (two stages, two barriers per pass), and both products run as 3xTF32 m16n8k8 tiles (mma.cuh):
//   dG_k[a][c] += sum_{node, m} P_{k-1}[node][m][a] * dP_k[node][m][c]   M = a, N = c, K = 8 stacked rows (node, m);
//                 a warp owns COLS/4 columns c of the slice, accumulators stay in registers over the whole list
//   Y[node][m][a] = sum_c dP_k[node][m][c] * G_k[a][c]                   M = 16 stacked rows, N = 8 values of a,
//                 K = c; the slice sits unsplit in shared memory (its 64 registers of split fragments per thread
//                 held the kernel at three CTAs per SM; at ~95 registers five are resident);
//                 warp -> (n-tile of a, tile of sixteen stacked rows)
// k_mid_sum then adds the Y rows of each parent's (contiguous) children.
// Row strides RA + 8 and COLS + 8 floats make every fragment load from shared memory conflict-free or 2-way.
// The tensor core adds into its fp32 accumulator with truncation, so an accumulation chain of N products drifts by
// up to N * 2^-24 of the sum; the dG accumulators are therefore folded into running sums (a rounded fp32
// add into the CTA's own gradient slice, which stays in L2) every eighth pass, which keeps every chain at 48 or 96
// products whatever the length of the node list.
template <int M, int RA, int COLS, int NQF = 1>
constexpr size_t tt_mid_smem_bytes()
{
    constexpr int NQ = NQF * 512 / (RA * M);
    return sizeof(float) * (size_t)(2 * NQ * M * (RA + 8) + 2 * NQ * M * (COLS + 8) + RA * (COLS + 4));
}

template <int M, int RA, int COLS, int NQF = 1>   // M = P_{k-1}: 4 or 2 rows per node; NQF: 2 = twice the nodes per pass
__global__ void __launch_bounds__(128, 5) k_mid_mma(WsView w, int k, int variant, int lbase)
{
    tt_pdl_enter();
    static_assert((M == 4 || M == 2) && (RA == 8 || RA % 16 == 0) && (COLS % 32 == 0 || COLS == 16), "rows per node; r_{k-1}; columns per warp");
    static_assert(NQF == 1 || NQF == 2, "one or two Y row tiles per warp");
    constexpr int NQ = NQF * 512 / (RA * M), AP = RA + 8, CP = COLS + 8;   // NQ * M = 16, 32 or 64 stacked rows per pass (x NQF)
    constexpr bool AHALF = RA == 8;          // dG: a = 8..15 of the one m-tile do not exist: zero operands, not stored
    constexpr int MT = AHALF ? 1 : RA / 16;  // dG: m-tiles over a
    constexpr int CW = COLS >= 32 ? COLS / 4 : 8;   // dG: columns per warp (16 columns: warps 0 and 1 only)
    constexpr int NTW = CW / 8;              // dG: n-tiles per warp
    constexpr int NTY = RA / 8;              // Y: n-tiles over a (4 or 2); NQ * M / 16 row tiles; NTY * NQ * M / 16 = 4 NQF tasks, NQF per warp
    constexpr int KTY = COLS / 8;            // Y: k steps over c
    extern __shared__ __align__(16) float mid_sm[];   // [2][NQ M AP] P rows, [2][NQ M CP] dP rows, [RA][COLS + 4] slice (tt_mid_smem_bytes)
    float* const sA = mid_sm;
    float* const sD = sA + 2 * NQ * M * AP;
    const int t_ = w.vlist[lbase + blockIdx.y];   // the tables of this variant, largest first: their long node lists start early
    const TableDesc& td = w.tdesc[t_];
    const int kc = k - 1;
    if (td.midfast[k] != variant || (int)blockIdx.x >= td.n[kc]) return;
    const uint32_t ik = blockIdx.x;
    const int tid = threadIdx.x, lane = tid & 31, wid = tid >> 5, g = lane >> 2, t = lane & 3;
    const float* __restrict__ Bsl = td.core[kc] + (size_t)ik * td.slice_floats[kc];
    // Y: this warp's n-tile of a and its four nodes
    const int ynt = wid % NTY, yrt0 = wid / NTY;   // task wid + 4 yi: the same n-tile, row tile yrt0 + yi * 4 / NTY
    // the slice G_k[i_k] for the Y product: unsplit in shared memory (row pitch COLS + 4: the fragment loads of a warp hit
    // 32 different banks), split at every use: registers for a fifth CTA per SM count for more than the 2 x 3 integer
    // operations per fragment
    constexpr int BP = COLS + 4;
    float* const sB = sD + 2 * NQ * M * CP;
    for (int i = tid; i < RA * (COLS / 4); i += 128) {
        const int a_ = i / (COLS / 4), c4 = i - a_ * (COLS / 4);
        tt_cp_async16(&sB[a_ * BP + 4 * c4], reinterpret_cast<const float4*>(Bsl + (size_t)a_ * COLS) + c4);
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
    // (asynchronous, so that the look-ups below do not queue behind it; it is the oldest copy group, so the wait for the
    // first pass's rows covers it, and the barrier after that wait orders it before its first use)
    const float* const sBw = sB + (8 * ynt + g) * BP + t;
    float acc[MT][NTW][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int nt = 0; nt < NTW; ++nt) { acc[mt][nt][0] = 0.f; acc[mt][nt][1] = 0.f; acc[mt][nt][2] = 0.f; acc[mt][nt][3] = 0.f; }
    // fold: this CTA is the only writer of its slice of the gradient, so the running sums live there (L2) instead of
    // in a second register set; each thread adds its accumulators to the elements it owns
    float* const gdst = td.grad[kc] + (size_t)ik * td.slice_floats[kc];
    bool first_fold = true;
    // last: the sums are final; the fused update of this CTA's slice goes with them (its fragments were read at the start,
    // and no other CTA or later kernel of the backward reads this slice)
    float* const cdst = td.core[kc] + (size_t)ik * td.slice_floats[kc];
    auto fold = [&](bool last) {
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
            // all loads of a row tile first, then the sums and stores: one round trip per tile instead of one per
            // column block (the compiler cannot move a load above a store it cannot tell apart)
            float2 v0[NTW], v1[NTW], u0[NTW], u1[NTW];
            const bool upd = last && w.fused_lr != 0.f;
#pragma unroll
            for (int nt = 0; nt < NTW; ++nt) {
                const int c = wid * CW + 8 * nt + 2 * t;
                v0[nt] = make_float2(0.f, 0.f); v1[nt] = v0[nt]; u0[nt] = v0[nt]; u1[nt] = v0[nt];
                if (c >= COLS) continue;     // this warp owns no columns of the slice gradient
                const size_t o0 = (size_t)(16 * mt + g) * COLS + c, o1 = (size_t)(16 * mt + g + 8) * COLS + c;
                if (!first_fold) {
                    v0[nt] = *reinterpret_cast<const float2*>(gdst + o0);
                    if (!AHALF) v1[nt] = *reinterpret_cast<const float2*>(gdst + o1);
                }
                if (upd) {   // the slice as it was read at the start (nobody else writes it): from its shared-memory copy
                    u0[nt] = *reinterpret_cast<const float2*>(sB + (16 * mt + g) * BP + c);
                    if (!AHALF) u1[nt] = *reinterpret_cast<const float2*>(sB + (16 * mt + g + 8) * BP + c);
                }
            }
#pragma unroll
            for (int nt = 0; nt < NTW; ++nt) {
                const int c = wid * CW + 8 * nt + 2 * t;
                if (c >= COLS) continue;
                const size_t o0 = (size_t)(16 * mt + g) * COLS + c, o1 = (size_t)(16 * mt + g + 8) * COLS + c;
                v0[nt].x += acc[mt][nt][0]; v0[nt].y += acc[mt][nt][1]; v1[nt].x += acc[mt][nt][2]; v1[nt].y += acc[mt][nt][3];
                *reinterpret_cast<float2*>(gdst + o0) = v0[nt];
                if (!AHALF) *reinterpret_cast<float2*>(gdst + o1) = v1[nt];
                if (upd) {
                    u0[nt].x = u0[nt].x - w.fused_lr * v0[nt].x; u0[nt].y = u0[nt].y - w.fused_lr * v0[nt].y;
                    *reinterpret_cast<float2*>(cdst + o0) = u0[nt];
                    if (!AHALF) {
                        u1[nt].x = u1[nt].x - w.fused_lr * v1[nt].x; u1[nt].y = u1[nt].y - w.fused_lr * v1[nt].y;
                        *reinterpret_cast<float2*>(cdst + o1) = u1[nt];
                    }
                }
                acc[mt][nt][0] = 0.f; acc[mt][nt][1] = 0.f; acc[mt][nt][2] = 0.f; acc[mt][nt][3] = 0.f;
            }
        }
        first_fold = false;
    };
    const uint32_t space = td.prefix_space[k - 1];
    const uint32_t j0 = tt_trank(w, td, k, ik * space), j1 = tt_trank(w, td, k, (ik + 1) * space);
    const int strideY = w.stride[k - 1];
    const uint32_t passes = (j1 - j0 + NQ - 1) / NQ;
    // The node ids of a pass and the addresses of the nodes' left operands are looked up two passes ahead by NQ threads
    // (digit-major list -> node -> prefix value or parent -> operand: a chain of dependent loads) and handed to the
    // CTA through a ring in shared memory, so that staging a pass starts with its cp.async instructions.
    __shared__ uint32_t s_node[3][NQ];
    __shared__ const float* s_left[3][NQ];
    uint32_t pre_node = 0xffffffffu;
    const float* pre_left = nullptr;
    auto lookup_ids = [&](uint32_t r) {          // into registers (threads 0..NQ-1)
        pre_node = 0xffffffffu;
        pre_left = nullptr;
        if (tid < NQ && j0 + r * NQ + tid < j1) {
            pre_node = w.tnode[k][j0 + r * NQ + tid];
            pre_left = tt_left_operand(w, td, k, pre_node);
        }
    };
    auto publish_ids = [&](uint32_t r) {         // registers -> ring slot of pass r
        if (tid < NQ) { s_node[r % 3u][tid] = pre_node; s_left[r % 3u][tid] = pre_left; }
    };
    // stage the NQ nodes of pass r (missing nodes of the last pass are zero-filled)
    auto issue = [&](uint32_t r) {
        const int st = (int)(r & 1u);
        const uint32_t* ids = s_node[r % 3u];
        const float* const* lefts = s_left[r % 3u];
        for (int i = tid; i < NQ * M * (COLS / 4); i += 128) {   // dP_k rows: M * COLS / 4 float4 per node
            const int q = i / (M * (COLS / 4)), rem = i - q * (M * (COLS / 4)), m = rem / (COLS / 4), c4 = rem - m * (COLS / 4);
            float4* dst = reinterpret_cast<float4*>(&sD[st * NQ * M * CP + (q * M + m) * CP + 4 * c4]);
            const uint32_t v = ids[q];
            if (v != 0xffffffffu) tt_cp_async16(dst, reinterpret_cast<const float4*>(w.dP[k] + (size_t)v * w.stride[k] + m * COLS) + c4);
            else *dst = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        for (int i = tid; i < NQ * M * (RA / 4); i += 128) {     // P_{k-1} of the parent: M * RA / 4 float4 per node
            const int q = i / (M * (RA / 4)), rem = i - q * (M * (RA / 4)), m = rem / (RA / 4), a4 = rem - m * (RA / 4);
            float4* dst = reinterpret_cast<float4*>(&sA[st * NQ * M * AP + (q * M + m) * AP + 4 * a4]);
            if (ids[q] != 0xffffffffu) tt_cp_async16(dst, reinterpret_cast<const float4*>(lefts[q] + m * RA) + a4);
            else *dst = make_float4(0.f, 0.f, 0.f, 0.f);
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };
    // passes 0 and 1 are looked up side by side (threads 0..NQ-1 and NQ..2NQ-1): one chain of round trips, not two
    if (tid < 2 * NQ) {
        const uint32_t r = (uint32_t)tid / NQ, q = (uint32_t)tid % NQ;
        uint32_t nd = 0xffffffffu;
        const float* lf = nullptr;
        if (j0 + r * NQ + q < j1) {
            nd = w.tnode[k][j0 + r * NQ + q];
            lf = tt_left_operand(w, td, k, nd);
        }
        s_node[r][q] = nd;
        s_left[r][q] = lf;
    }
    __syncthreads();
    if (passes > 0) issue(0);
    for (uint32_t r = 0; r < passes; ++r) {
        lookup_ids(r + 2);          // in flight while this pass is staged and computed; published at the end of the iteration
        if (r + 1 < passes) {
            issue(r + 1);
            asm volatile("cp.async.wait_group 1;" ::: "memory");
        } else {
            asm volatile("cp.async.wait_group 0;" ::: "memory");
        }
        __syncthreads();
        const float* A_ = sA + (r & 1u) * (NQ * M * AP);
        const float* D_ = sD + (r & 1u) * (NQ * M * CP);
        // ---- dG: eight stacked rows (node, m) give k = 8
#pragma unroll
        for (int p = 0; p < NQ * M / 8; ++p) {
            const float* Aa = A_ + (8 * p + t) * AP;       // stacked row 8p + t:     node (8p + t) / M, row (8p + t) % M
            const float* Ab = A_ + (8 * p + t + 4) * AP;   // stacked row 8p + t + 4
            if (wid * CW >= COLS) break;     // this warp owns no columns of the slice gradient
            const float* Da = D_ + (8 * p + t) * CP + wid * CW + g;
            const float* Db = D_ + (8 * p + t + 4) * CP + wid * CW + g;
            Tf32Pair a[MT][4];
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
                a[mt][0] = tt_split_tf32(Aa[16 * mt + g]);
                a[mt][1] = tt_split_tf32(AHALF ? 0.f : Aa[16 * mt + g + 8]);
                a[mt][2] = tt_split_tf32(Ab[16 * mt + g]);
                a[mt][3] = tt_split_tf32(AHALF ? 0.f : Ab[16 * mt + g + 8]);
            }
#pragma unroll
            for (int nt = 0; nt < NTW; ++nt) {
                Tf32Pair b[2];
                b[0] = tt_split_tf32(Da[8 * nt]);
                b[1] = tt_split_tf32(Db[8 * nt]);
#pragma unroll
                for (int mt = 0; mt < MT; ++mt) tt_mma_3xtf32(acc[mt][nt], a[mt], b);
            }
        }
        // ---- Y of this warp's sixteen stacked rows (NQF times) and eight values of a
#pragma unroll
        for (int yi = 0; yi < NQF; ++yi) {
            const int yrt = yrt0 + yi * (4 / NTY);
            float y[4] = {0.f, 0.f, 0.f, 0.f};
            const float* Ra = D_ + (16 * yrt + g) * CP;       // row g of the tile: stacked row 16 yrt + g
            const float* Rb = D_ + (16 * yrt + g + 8) * CP;   // row g + 8
#pragma unroll
            for (int kt = 0; kt < KTY; ++kt) {
                Tf32Pair a[4];
                a[0] = tt_split_tf32(Ra[8 * kt + t]);
                a[1] = tt_split_tf32(Rb[8 * kt + t]);
                a[2] = tt_split_tf32(Ra[8 * kt + t + 4]);
                a[3] = tt_split_tf32(Rb[8 * kt + t + 4]);
                Tf32Pair by[2];
                by[0] = tt_split_tf32(sBw[8 * kt]);
                by[1] = tt_split_tf32(sBw[8 * kt + 4]);
                tt_mma_3xtf32(y, a, by);
            }
            const uint32_t ja = j0 + r * NQ + (16 * yrt + g) / M, jb2 = j0 + r * NQ + (16 * yrt + g + 8) / M;
            const int ma = (16 * yrt + g) % M;   // the same row of P for g and g + 8 (M divides 8)
            if (ja < j1) {
                const uint32_t v = s_node[r % 3u][(16 * yrt + g) / M];
                *reinterpret_cast<float2*>(&w.Y[k][(size_t)v * strideY + ma * RA + 8 * ynt + 2 * t]) = make_float2(y[0], y[1]);
            }
            if (jb2 < j1) {
                const uint32_t v = s_node[r % 3u][(16 * yrt + g + 8) / M];
                *reinterpret_cast<float2*>(&w.Y[k][(size_t)v * strideY + ma * RA + 8 * ynt + 2 * t]) = make_float2(y[2], y[3]);
            }
        }
        if ((r & (8u / NQF - 1u)) == 8u / NQF - 1u) fold(false);   // rounded running sums every eighth pass (fourth with twice the nodes)
        publish_ids(r + 2);   // its ring slot held pass r - 1
        __syncthreads();   // everyone is done with this stage before pass r + 2 overwrites it
    }
    if (passes == 0) {   // no pass has waited for the slice copy
        asm volatile("cp.async.wait_group 0;" ::: "memory");
        __syncthreads();
    }
    fold(true);   // also writes the zeros of a slice without nodes
}

// dP_{k-1}[parent] (k = 2: the first core's gradient slice) = sum of the Y rows of the parent's children,
// which are contiguous in sorted order; one warp per parent
__global__ void __launch_bounds__(256) k_mid_sum(WsView w, int k)
{
    tt_pdl_enter();
    const int lane = threadIdx.x & 31;
    const uint32_t count = w.counters[CTR_LEVEL0 + k - 1];
    const uint32_t nwarps = (gridDim.x * blockDim.x) >> 5;
    const int strideY = w.stride[k - 1];
    for (uint32_t pn = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; pn < count; pn += nwarps) {
        const int t = tt_find_table(w.tb[k - 1], w.T, pn);
        const TableDesc& td = w.tdesc[t];
        if (td.midfast[k] < 0) continue;
        const int nout4 = td.P[k - 1] * td.r[k - 1] / 4;
        const uint32_t c0 = w.cstart[k - 1][pn], c1 = w.cstart[k - 1][pn + 1];
        float* dst = k == 2 ? td.grad[0] + (size_t)w.val[1][pn] * td.slice_floats[0] : w.dP[k - 1] + (size_t)pn * w.stride[k - 1];
        for (int f = lane; f < nout4; f += 32) {
            float4 s = make_float4(0.f, 0.f, 0.f, 0.f);
            for (uint32_t v = c0; v < c1; ++v) {
                const float4 x = __ldg(reinterpret_cast<const float4*>(w.Y[k] + (size_t)v * strideY) + f);
                s.x += x.x; s.y += x.y; s.z += x.z; s.w += x.w;
            }
            reinterpret_cast<float4*>(dst)[f] = s;
            if (k == 2 && w.fused_lr != 0.f) {   // first core: the slices of present first digits are final here
                float4* c4 = reinterpret_cast<float4*>(td.core[0] + (size_t)w.val[1][pn] * td.slice_floats[0]) + f;
                float4 u = *c4;
                u.x = u.x - w.fused_lr * s.x; u.y = u.y - w.fused_lr * s.y; u.z = u.z - w.fused_lr * s.z; u.w = u.w - w.fused_lr * s.w;
                *c4 = u;
            }
        }
    }
}

// Digit-major ("transposed") list of the level-k nodes: a second presence-bitmap sort, keyed by
// (i_k, parent prefix) instead of (parent prefix, i_k); tnode[k][rank] = node.
cudaError_t tt_launch_tlist(tt_emb* h, int k, cudaStream_t s)
{
    WsView& w = h->v;
    cudaError_t e;
    if ((e = cudaMemsetAsync(w.tbm[k], 0, (size_t)w.ttotal_words[k] * sizeof(uint2), s)) != cudaSuccess) return e;
    const int g = h->sm_count * 8;
    if ((e = tt_launch_pdl(k_tmark, dim3(g), dim3(256), 0, s, w, k)) != cudaSuccess) return e;
    tt_note_launch();
    TPopScan tp{w, k};
    if ((e = tt_scan(tp, w.ttotal_words[k], w.scan_tmp, s)) != cudaSuccess) return e;
    if ((e = tt_launch_pdl(k_tfill, dim3(g), dim3(256), 0, s, w, k)) != cudaSuccess) return e;
    tt_note_launch();
    return cudaGetLastError();
}

template <int M, int RA, int COLS>
static cudaError_t tt_launch_mid(dim3 grid, cudaStream_t st, const WsView& w, int k, int variant, int lbase)
{
    constexpr size_t smem = tt_mid_smem_bytes<M, RA, COLS>();
    cudaError_t e = cudaFuncSetAttribute(k_mid_mma<M, RA, COLS>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    return tt_launch_pdl(k_mid_mma<M, RA, COLS>, grid, dim3(128), smem, st, w, k, variant, lbase);
}

cudaError_t tt_launch_bwd_middle(tt_emb* h, cudaStream_t s)
{
    WsView& w = h->v;
    cudaError_t e;
    for (int k = h->K - 1; k >= 2; --k) {
        int max_n = 1, max_down = 1, max_slice = 1;
        bool any_generic = false, any_fast[11] = {false, false, false, false, false, false, false, false, false, false, false};
        for (int t = 0; t < h->T; ++t) {
            const TableDesc& td = h->tab[t];
            const int kc = k - 1;
            const int M = td.P[kc], ra = td.r[kc], cols = td.d[kc] * td.r[kc + 1];
            if (td.n[kc] > max_n) max_n = td.n[kc];
            if (ra * (cols + 1) + M * cols > max_down) max_down = ra * (cols + 1) + M * cols;
            if (M * ra + M * cols > max_slice) max_slice = M * ra + M * cols;
            if (td.midfast[k] < 0) any_generic = true; else any_fast[td.midfast[k]] = true;
        }
        // level K-1's digit-major list already exists: the forward built it to order its sweep
        if (k != h->K - 1 && (e = tt_launch_tlist(h, k, s)) != cudaSuccess) return e;
        const dim3 sg(max_n, h->T);
        // the shape variants are independent (different tables): run them side by side so that the tail of one
        // (a few long node lists) overlaps the others
        int nfast = 0;
        for (int v = 0; v < 11; ++v) nfast += any_fast[v] ? 1 : 0;
        const bool fork = nfast > 1 && !h->serial;
        if (fork && (e = tt_fork(h, s, 4)) != cudaSuccess) return e;
        int slot = 0;
        auto st = [&]() { return fork ? h->side[(slot++) & 3] : s; };
        // grid of variant v: its own tables only, slices up to the largest n_k among them
        auto mgrid = [&](int v) { return dim3(h->mmaxn[k][v + 1], h->mcount[k][v + 1]); };
        auto mlist = [&](int v) { return (2 + k) * h->T + h->mbase[k][v + 1]; };
        if (any_fast[0]) { if ((e = tt_launch_mid<4, 32, 128>(mgrid(0), st(), w, k, 0, mlist(0))) != cudaSuccess) return e; tt_note_launch(); }
        if (any_fast[1]) { if ((e = tt_launch_mid<4, 16, 128>(mgrid(1), st(), w, k, 1, mlist(1))) != cudaSuccess) return e; tt_note_launch(); }
        if (any_fast[2]) { if ((e = tt_launch_mid<4, 32, 64>(mgrid(2), st(), w, k, 2, mlist(2))) != cudaSuccess) return e; tt_note_launch(); }
        if (any_fast[3]) { if ((e = tt_launch_mid<4, 16, 64>(mgrid(3), st(), w, k, 3, mlist(3))) != cudaSuccess) return e; tt_note_launch(); }
        if (any_fast[4]) { if ((e = tt_launch_mid<2, 32, 128>(mgrid(4), st(), w, k, 4, mlist(4))) != cudaSuccess) return e; tt_note_launch(); }
        if (any_fast[5]) { if ((e = tt_launch_mid<2, 16, 64>(mgrid(5), st(), w, k, 5, mlist(5))) != cudaSuccess) return e; tt_note_launch(); }
        if (any_fast[6]) { if ((e = tt_launch_mid<2, 32, 64>(mgrid(6), st(), w, k, 6, mlist(6))) != cudaSuccess) return e; tt_note_launch(); }
        if (any_fast[7]) { if ((e = tt_launch_mid<2, 16, 32>(mgrid(7), st(), w, k, 7, mlist(7))) != cudaSuccess) return e; tt_note_launch(); }
        if (any_fast[8]) { if ((e = tt_launch_mid<4, 8, 32>(mgrid(8), st(), w, k, 8, mlist(8))) != cudaSuccess) return e; tt_note_launch(); }
        if (any_fast[9]) { if ((e = tt_launch_mid<2, 8, 32>(mgrid(9), st(), w, k, 9, mlist(9))) != cudaSuccess) return e; tt_note_launch(); }
        if (any_fast[10]) { if ((e = tt_launch_mid<2, 8, 16>(mgrid(10), st(), w, k, 10, mlist(10))) != cudaSuccess) return e; tt_note_launch(); }
        if (fork && (e = tt_join(h, s, 4)) != cudaSuccess) return e;
        if (nfast > 0) {
            if ((e = tt_launch_pdl(k_mid_sum, dim3(h->sm_count * 8), dim3(256), 0, s, w, k)) != cudaSuccess) return e;
            tt_note_launch();
        }
        if (any_generic) {
            if ((e = cudaFuncSetAttribute(k_mid_slice, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(max_slice * sizeof(float)))) != cudaSuccess) return e;
            k_mid_slice<<<sg, 256, (size_t)max_slice * sizeof(float), s>>>(w, k);
            tt_note_launch();
            if ((e = cudaFuncSetAttribute(k_mid_down, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)(max_down * sizeof(float)))) != cudaSuccess) return e;
            k_mid_down<<<h->sm_count * 8, 256, (size_t)max_down * sizeof(float), s>>>(w, k);
            tt_note_launch();
        }
    }
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------- SGD

__global__ void __launch_bounds__(256) k_sgd(WsView w, float lr, int only_unfused)
{
    tt_pdl_enter();
    const int t = blockIdx.y / w.K, k = blockIdx.y % w.K;
    const TableDesc& td = w.tdesc[t];
    if (only_unfused && ((td.sgd_mask >> k) & 1)) return;   // updated by the kernel that finalised its gradient
    float* __restrict__ G = td.core[k];
    const float* __restrict__ dG = td.grad[k];
    const int64_t n = td.core_floats[k];
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i < n; i += (int64_t)gridDim.x * blockDim.x)
        G[i] = G[i] - lr * dG[i];
}

cudaError_t tt_launch_sgd(tt_emb* h, float lr, bool only_unfused, cudaStream_t s)
{
    k_sgd<<<dim3(64, h->T * h->K), 256, 0, s>>>(h->v, lr, only_unfused ? 1 : 0);
    tt_note_launch();
    return cudaGetLastError();
}
