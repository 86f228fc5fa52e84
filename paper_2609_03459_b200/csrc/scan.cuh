// Device-wide exclusive scan of uint32 values produced by a functor, as two kernels: tile sums, where the CTA that
// reports last (a ticket counter; nobody waits) also scans the tile sums, then per-tile scan + apply.
//
// Functor F:
//   __device__ uint32_t size() const;                       number of elements (may read device memory)
//   __device__ int locate(uint32_t i0) const;               once per tile, for its first element: a hint handed to value / emit
//                                                           (e.g. the table the tile starts in, so that elements need no search)
//   __device__ uint32_t value(uint32_t i, int hint) const;  input i
//   __device__ uint32_t weight(uint32_t v) const;           optional: the amount that input v adds to the scan (default: v
//                                                           itself); emit is handed v, so that a functor whose input is a
//                                                           word of flags does not have to load it a second time
//   __device__ void emit(uint32_t i, uint32_t excl, uint32_t v, int hint) const;   called once per element in the apply pass
//   __device__ void total(uint32_t tot) const;              called by one thread with the grand total
//   __device__ uint32_t tile_of(uint32_t cta) const;        optional: the tile that CTA `cta` of the apply pass takes
//                                                           (0xffffffff: none), for an order other than ascending,
//                                                           e.g. the tiles with the most output first
//   WsView w;                                               w.counters[CTR_SCAN_TICKET] is the ticket (zero between scans)
// ITEMS = elements per thread (tile = TT_SCAN_THREADS * ITEMS): the default for long inputs, fewer for short ones whose
// tiles should still spread over the SMs.
#pragma once
#include "common.cuh"

template <class F>
__device__ __forceinline__ auto tt_scan_amount(const F& f, uint32_t v, int) -> decltype(f.weight(v)) { return f.weight(v); }
template <class F>
__device__ __forceinline__ uint32_t tt_scan_amount(const F&, uint32_t v, long) { return v; }
template <class F>
__device__ __forceinline__ auto tt_scan_tile(const F& f, uint32_t cta, int) -> decltype(f.tile_of(cta)) { return f.tile_of(cta); }
template <class F>
__device__ __forceinline__ uint32_t tt_scan_tile(const F&, uint32_t cta, long) { return cta; }

__device__ __forceinline__ uint32_t tt_block_excl_scan(uint32_t x, uint32_t* sm /* [34] */, uint32_t& block_total)
{
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5, nw = blockDim.x >> 5;
    uint32_t incl = x;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        uint32_t y = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += y;
    }
    if (lane == 31) sm[wid] = incl;
    __syncthreads();
    if (wid == 0) {
        uint32_t wv = lane < nw ? sm[lane] : 0u, wi = wv;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            uint32_t y = __shfl_up_sync(0xffffffffu, wi, o);
            if (lane >= o) wi += y;
        }
        sm[lane] = wi - wv;
        if (lane == 31) sm[33] = wi;
    }
    __syncthreads();
    uint32_t res = sm[wid] + incl - x;
    block_total = sm[33];
    __syncthreads();
    return res;
}

// exclusive scan of the tile sums in place (one CTA), grand total to the functor
template <class F>
__device__ __forceinline__ void tt_scan_spine_cta(const F& f, uint32_t* tile_sums, uint32_t ntiles, uint32_t* sm)
{
    uint32_t carry = 0;
    for (uint32_t b0 = 0; b0 < ntiles; b0 += blockDim.x) {
        const uint32_t i = b0 + threadIdx.x;
        const uint32_t x = i < ntiles ? __ldcg(tile_sums + i) : 0u;   // written by other CTAs: read past L1
        uint32_t tot;
        const uint32_t ex = tt_block_excl_scan(x, sm, tot);
        if (i < ntiles) tile_sums[i] = carry + ex;
        carry += tot;
    }
    if (threadIdx.x == 0) f.total(carry);
}

template <class F, int ITEMS>
__global__ void __launch_bounds__(TT_SCAN_THREADS) tt_scan_reduce(F f, uint32_t* tile_sums)
{
    tt_pdl_enter();
    constexpr int TILE = TT_SCAN_THREADS * ITEMS;
    __shared__ uint32_t sm[34];
    __shared__ uint32_t ticket;
    const uint32_t n = f.size();
    const uint32_t ntiles = (uint32_t)(((uint64_t)n + TILE - 1) / TILE);
    if (ntiles == 0) {   // nothing to scan: the first CTA still reports the total
        if (blockIdx.x == 0 && threadIdx.x == 0) f.total(0u);
        return;
    }
    if (blockIdx.x >= ntiles) return;
    const uint64_t base = (uint64_t)blockIdx.x * TILE;
    uint32_t s = 0;
    const int hint = f.locate((uint32_t)base);
    // a sum has no order: neighbouring threads take neighbouring elements (coalesced)
#pragma unroll 4
    for (int j = 0; j < ITEMS; ++j) {
        const uint64_t i = base + (uint64_t)j * TT_SCAN_THREADS + threadIdx.x;
        if (i < n) s += tt_scan_amount(f, f.value((uint32_t)i, hint), 0);
    }
    uint32_t tot;
    tt_block_excl_scan(s, sm, tot);
    if (threadIdx.x == 0) {
        tile_sums[blockIdx.x] = tot;
        __threadfence();                                   // the sum is visible before the ticket is
        ticket = atomicAdd(f.w.counters + CTR_SCAN_TICKET, 1u);
    }
    __syncthreads();
    if (ticket != ntiles - 1) return;
    // every tile has reported: this CTA scans the sums and leaves the ticket at zero for the next scan
    __threadfence();
    tt_scan_spine_cta(f, tile_sums, ntiles, sm);
    if (threadIdx.x == 0) f.w.counters[CTR_SCAN_TICKET] = 0u;
}

// Elements are read and emitted striped (thread t takes elements t, t + 256, ...: coalesced for the functor's loads and
// stores), scanned blocked (thread t owns elements ITEMS t .. ITEMS t + ITEMS - 1); the two orders meet in shared memory, padded by
// one word per 32 so that both access patterns are free of bank conflicts.
__device__ __forceinline__ int tt_scan_pad(int i) { return i + (i >> 5); }

template <class F, int ITEMS>
__global__ void __launch_bounds__(TT_SCAN_THREADS, 4) tt_scan_apply(F f, const uint32_t* __restrict__ tile_sums)
{
    tt_pdl_enter();
    constexpr int TILE = TT_SCAN_THREADS * ITEMS;
    __shared__ uint32_t sm[34];
    __shared__ uint32_t sv[TILE + TILE / 32];
    const uint32_t n = f.size();
    const uint32_t tile = tt_scan_tile(f, blockIdx.x, 0);
    if (tile == 0xffffffffu) return;
    const uint64_t base = (uint64_t)tile * TILE;
    if (base >= n) return;
    uint32_t v[ITEMS];
    const int hint = f.locate((uint32_t)base);
#pragma unroll
    for (int j = 0; j < ITEMS; ++j) {
        const uint64_t i = base + (uint64_t)j * TT_SCAN_THREADS + threadIdx.x;
        v[j] = i < n ? f.value((uint32_t)i, hint) : 0u;
        sv[tt_scan_pad(j * TT_SCAN_THREADS + threadIdx.x)] = i < n ? tt_scan_amount(f, v[j], 0) : 0u;
    }
    __syncthreads();
    uint32_t s = 0;
    uint32_t mine[ITEMS];
#pragma unroll
    for (int j = 0; j < ITEMS; ++j) {
        mine[j] = sv[tt_scan_pad(threadIdx.x * ITEMS + j)];
        s += mine[j];
    }
    uint32_t tot;
    uint32_t ex = tile_sums[tile] + tt_block_excl_scan(s, sm, tot);
#pragma unroll
    for (int j = 0; j < ITEMS; ++j) {
        sv[tt_scan_pad(threadIdx.x * ITEMS + j)] = ex;   // exclusive prefix of element ITEMS t + j
        ex += mine[j];
    }
    __syncthreads();
#pragma unroll
    for (int j = 0; j < ITEMS; ++j) {
        const uint64_t i = base + (uint64_t)j * TT_SCAN_THREADS + threadIdx.x;
        if (i < n) f.emit((uint32_t)i, sv[tt_scan_pad(j * TT_SCAN_THREADS + threadIdx.x)], v[j], hint);
    }
}

// capacity = host-known upper bound of f.size(); tmp must hold ceil(capacity / tile) + 1 words; apply_ctas: size of the
// apply grid for a functor with tile_of (default: one CTA per tile)
template <class F, int ITEMS = TT_SCAN_ITEMS>
static inline cudaError_t tt_scan(const F& f, uint64_t capacity, uint32_t* tmp, cudaStream_t s, unsigned apply_ctas = 0)
{
    constexpr int TILE = TT_SCAN_THREADS * ITEMS;
    unsigned tiles = (unsigned)((capacity + TILE - 1) / TILE);
    if (tiles == 0) tiles = 1;
    cudaError_t e = tt_launch_pdl(tt_scan_reduce<F, ITEMS>, dim3(tiles), dim3(TT_SCAN_THREADS), 0, s, f, tmp);
    if (e != cudaSuccess) return e;
    tt_note_launch();
    if ((e = tt_launch_pdl(tt_scan_apply<F, ITEMS>, dim3(apply_ctas ? apply_ctas : tiles), dim3(TT_SCAN_THREADS), 0, s, f, (const uint32_t*)tmp)) != cudaSuccess) return e;
    tt_note_launch();
    return cudaGetLastError();
}
