// Prefix grouping (paper Sec. 3.3: sort, unique, mixed-radix conversion, run-length encoding), integer only.
//
// B200 design: the sort + unique of a table's row ids is a distribution (counting) sort over the row-id
// domain with one presence bit per row.  The bitmaps of all tables (N_t / 8 bytes each) stay resident in
// the 126 MB L2, so marking costs one L2 access per lookup, and an exclusive scan of the word popcounts
// yields (a) the ascending list of distinct rows, (b) a rank structure {bits, base} that maps any row id
// to its slot with one 8-byte load, so no per-lookup inverse map is ever written.  The prefix levels are
// built the same way: the marking pass also sets one bit per length-k prefix (k < K) in a small bitmap over
// the prefix space, and a scan of its word popcounts yields the ascending distinct prefixes; the first child of
// a prefix is a rank look-up in the next level's bitmap, so the run-length encoding of the sorted rows is never
// walked.  A prefix is present when the scanned bitmap of the level below counts at least one node in its range of
// children (two rank look-ups per possible prefix, k_prefix_bits), so the cost of a prefix level is proportional
// to the size of its prefix space, not to the lookups or the rows.  No kernel waits on another CTA.
#include "common.cuh"
#include "scan.cuh"

// ---------------------------------------------------------------------------------------------- prologue

__global__ void k_check_offsets(WsView w)
{
    tt_pdl_enter();
    const int64_t nb = (int64_t)w.T * w.B;
    const int64_t stride = (int64_t)gridDim.x * blockDim.x;
    bool bad = false;
    for (int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; i <= nb; i += stride) {
        const int64_t o = w.offsets[i];
        if (o < 0 || o > w.L) bad = true;
        if (i == 0 && o != 0) bad = true;
        if (i == nb && o != w.L) bad = true;
        if (i < nb && w.offsets[i + 1] < o) bad = true;
        if (i % w.B == 0 || i == nb) {
            int64_t c = o < 0 ? 0 : (o > w.L ? w.L : o);
            w.tl_start[i == nb ? w.T : i / w.B] = c;
        }
    }
    if (bad) atomicOr(w.status, TT_EMB_STATUS_OFFSETS);
}

// ---------------------------------------------------------------------------------------------- mark

__global__ void __launch_bounds__(256) k_mark(WsView w)
{
    tt_pdl_enter();
    const int64_t L = w.L;
    const int64_t step = (int64_t)gridDim.x * blockDim.x * 4;
    int t = 0;
    bool bad = false;
    // the table of the last lookup, kept in registers: lookup range, row count, first presence word
    int64_t l_lo = 0, l_hi = 0, tN = 0;
    uint32_t twb = 0;
    for (int64_t base = (int64_t)blockIdx.x * blockDim.x * 4 + threadIdx.x; base < L; base += step) {
        int64_t g[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int64_t l = base + (int64_t)j * blockDim.x;
            g[j] = l < L ? tt_index(w, l) : -1;
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int64_t l = base + (int64_t)j * blockDim.x;
            if (l >= L) continue;
            if (!(l_lo <= l && l < l_hi)) {
                t = tt_find_table64(w.tl_start, w.T, l);
                l_lo = w.tl_start[t];
                l_hi = w.tl_start[t + 1];
                tN = w.tdesc[t].N;
                twb = w.tdesc[t].word_base;
            }
            if (g[j] < 0 || g[j] >= tN) { bad = true; continue; }
            const uint32_t row = (uint32_t)g[j];
            unsigned* word = &w.bm[twb + (row >> 5)].x;
            const unsigned m = 1u << (row & 31);
            if (!(__ldca(word) & m)) atomicOr(word, m);   // L1 may hold a stale word: at worst a redundant atomic
        }
    }
    if (bad) atomicOr(w.status, TT_EMB_STATUS_INDEX);
}

// val[excl ..] = v0 + (positions of the set bits of `bits`), clipped at `cap`.  Called by all lanes that emit a word
// (also with bits == 0).  A lane writes the first bits of its own word; a word with more is handed to the whole warp,
// one lane per bit: a densely set word then is one coalesced store instead of 32 stores that each touch another
// sector (a tile of the popular first rows of a table took 80 us against 20 us for a sparse one).
#define EMIT_OWN 8
__device__ __forceinline__ void tt_emit_set_bits(uint32_t* __restrict__ val, uint32_t cap, unsigned bits, uint32_t excl, uint32_t v0)
{
    const unsigned act = __activemask();
    const int lane = threadIdx.x & 31;
    const bool dense = __popc(bits) > EMIT_OWN;
    if (!dense) {
        uint32_t slot = excl;
#pragma unroll
        for (int it = 0; it < EMIT_OWN; ++it)
            if (bits) {
                const int b = __ffs(bits) - 1;
                bits &= bits - 1;
                if (slot < cap) val[slot] = v0 + b;
                ++slot;
            }
    }
    unsigned todo = __ballot_sync(act, dense);
    while (todo) {
        const int src = __ffs(todo) - 1;
        todo &= todo - 1;
        const unsigned wb = __shfl_sync(act, bits, src);
        const uint32_t we = __shfl_sync(act, excl, src);
        const uint32_t wv = __shfl_sync(act, v0, src);
        if ((wb >> lane) & 1u) {
            const uint32_t sl = we + __popc(wb & ((1u << lane) - 1u));
            if (sl < cap) val[sl] = wv + lane;
        }
    }
}

// ---------------------------------------------------------------------------------------------- level K: rows

struct PopScan {
    WsView w;
    __device__ uint32_t size() const { return w.total_words; }
    // every table starts on a scan-tile boundary: the table of a tile's first word is the table of all its words
    __device__ int locate(uint32_t i0) const
    {
        int lo = 0, hi = w.T;
        while (hi - lo > 1) {
            int mid = (lo + hi) >> 1;
            if (w.tdesc[mid].word_base <= i0) lo = mid; else hi = mid;
        }
        return lo;
    }
    __device__ uint32_t value(uint32_t i, int) const { return w.bm[i].x; }
    __device__ uint32_t weight(uint32_t bits) const { return __popc(bits); }
    // The first TT_HEAD_TILES tiles of every table go first (CTAs 0 .. HEAD * T - 1, tile position major), the others
    // follow in ascending order.  With the identity rank-to-row mapping the popular rows are the first rows of a table:
    // those tiles are densely set and emit a hundred times the rows of a tile further down (70 us against 6), and in
    // ascending order the dense tiles of the last tables ran alone at the end of the kernel.
    __device__ uint32_t tile_of(uint32_t cta) const
    {
        const uint32_t head = (uint32_t)TT_HEAD_TILES * (uint32_t)w.T;
        if (cta < head) {
            const uint32_t p = cta / (uint32_t)w.T, t = cta % (uint32_t)w.T;
            const TableDesc& td = w.tdesc[t];
            return p < td.num_words / TT_SCAN_TILE ? td.word_base / TT_SCAN_TILE + p : 0xffffffffu;
        }
        const uint32_t m = cta - head;
        if (m >= w.rest_tiles) return 0xffffffffu;
        int lo = 0, hi = w.T;                    // the table whose remaining tiles hold number m
        while (hi - lo > 1) {
            const int mid = (lo + hi) >> 1;
            if (w.tdesc[mid].rest_base <= m) lo = mid; else hi = mid;
        }
        return w.tdesc[lo].word_base / TT_SCAN_TILE + TT_HEAD_TILES + (m - w.tdesc[lo].rest_base);
    }
    __device__ void emit(uint32_t i, uint32_t excl, uint32_t bits, int t) const
    {
        w.bm[i].y = excl;
        const int K = w.K;
        const uint32_t wb = w.tdesc[t].word_base;
        if (i == wb) w.tb[K][t] = excl < w.cap[K] ? excl : w.cap[K];
        const uint32_t row0 = (i - wb) << 5;
        tt_emit_set_bits(w.val[K], w.cap[K], bits, excl, row0);
    }
    __device__ void total(uint32_t tot) const
    {
        const int K = w.K;
        if (tot > w.cap[K]) { atomicOr(w.status, TT_EMB_STATUS_OVERFLOW); tot = w.cap[K]; }
        w.counters[CTR_LEVEL0 + K] = tot;
        w.tb[K][w.T] = tot;
    }
};

// ---------------------------------------------------------------------------------------------- prefix levels

// number of level-c nodes before the first one whose value is >= pos (c = K: rows; c < K: length-c prefixes)
__device__ __forceinline__ uint32_t tt_rank_at(const WsView& w, const TableDesc& td, int c, uint32_t pos)
{
    const uint2 e = c == w.K ? w.bm[td.word_base + (pos >> 5)] : w.bml[c][td.lword_base[c] + (pos >> 5)];
    const uint32_t r = e.y + __popc(e.x & ((1u << (pos & 31)) - 1u));
    const uint32_t lim = w.counters[CTR_LEVEL0 + c];
    return r < lim ? r : lim;
}

// number of level-c nodes of all tables before position x of table td (x inside the table's space), from the scanned bitmap
__device__ __forceinline__ uint32_t tt_rank_excl(const WsView& w, const TableDesc& td, int c, uint32_t x)
{
    const uint2 e = c == w.K ? w.bm[td.word_base + (x >> 5)] : w.bml[c][td.lword_base[c] + (x >> 5)];
    return e.y + __popc(e.x & ((1u << (x & 31)) - 1u));
}
// ... up to and including position x
__device__ __forceinline__ uint32_t tt_rank_incl(const WsView& w, const TableDesc& td, int c, uint32_t x)
{
    const uint2 e = c == w.K ? w.bm[td.word_base + (x >> 5)] : w.bml[c][td.lword_base[c] + (x >> 5)];
    return e.y + __popc(e.x & (0xffffffffu >> (31 - (x & 31))));
}

// Presence bitmap of level k < K (one bit per possible length-k prefix of every table) from the scanned bitmap of level
// k + 1: prefix p is present when some node of level k + 1 lies in [p n_{k+1}, (p + 1) n_{k+1}).  One warp per word, one
// lane per prefix (the two rank look-ups of a prefix are dependent loads: 32 of them one after the other per thread
// took 25 us even for the few words of level 1); the words are written whole (no memset, no atomics).
__global__ void __launch_bounds__(256) k_prefix_bits(WsView w, int k)
{
    tt_pdl_enter();
    const int c = k + 1;
    const int lane = threadIdx.x & 31;
    const uint32_t nwords = w.total_words_l[k];
    const uint32_t nwarps = (gridDim.x * blockDim.x) >> 5;
    for (uint32_t i = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; i < nwords; i += nwarps) {
        int lo_t = 0, hi_t = w.T;
        while (hi_t - lo_t > 1) {
            const int mid = (lo_t + hi_t) >> 1;
            if (w.tdesc[mid].lword_base[k] <= i) lo_t = mid; else hi_t = mid;
        }
        const TableDesc& td = w.tdesc[lo_t];
        const uint32_t p = ((i - td.lword_base[k]) << 5) + lane;
        const uint32_t radix = (uint32_t)td.n[k];                       // radix of digit k + 1
        const uint32_t space_c = c == w.K ? (uint32_t)td.N : td.prefix_space[c];
        const uint64_t lo = (uint64_t)p * radix;
        bool present = false;
        if (p < td.prefix_space[k] && lo < space_c) {                    // rows past N do not exist
            uint64_t hi = lo + radix;
            if (hi > space_c) hi = space_c;
            present = tt_rank_incl(w, td, c, (uint32_t)hi - 1u) != tt_rank_excl(w, td, c, (uint32_t)lo);
        }
        const unsigned bits = __ballot_sync(0xffffffffu, present);
        if (lane == 0) w.bml[k][i] = make_uint2(bits, 0u);
    }
}

// Level k < K from its own presence bitmap: the ascending distinct prefixes of every table.  Runs after the scan of
// level k + 1 and k_prefix_bits, which sets this level's bits.
struct LevelScan {
    WsView w;
    int k;
    __device__ uint32_t size() const { return w.total_words_l[k]; }
    __device__ int locate(uint32_t i0) const
    {
        int lo = 0, hi = w.T;
        while (hi - lo > 1) {
            int mid = (lo + hi) >> 1;
            if (w.tdesc[mid].lword_base[k] <= i0) lo = mid; else hi = mid;
        }
        return lo;
    }
    __device__ uint32_t value(uint32_t i, int) const { return w.bml[k][i].x; }
    __device__ uint32_t weight(uint32_t bits) const { return __popc(bits); }
    __device__ void emit(uint32_t i, uint32_t excl, uint32_t bits, int t) const
    {
        w.bml[k][i].y = excl;
        const TableDesc& td = w.tdesc[t];
        const uint32_t wb = td.lword_base[k];
        if (i == wb) w.tb[k][t] = excl < w.cap[k] ? excl : w.cap[k];
        const uint32_t p0 = (i - wb) << 5;
        tt_emit_set_bits(w.val[k], w.cap[k], bits, excl, p0);
    }
    __device__ void total(uint32_t tot) const
    {
        if (tot > w.cap[k]) { atomicOr(w.status, TT_EMB_STATUS_OVERFLOW); tot = w.cap[k]; }
        w.counters[CTR_LEVEL0 + k] = tot;
        w.tb[k][w.T] = tot;
    }
};

// Links of every level-k node, one thread each (the rank look-ups are random 8-byte loads: kept out of the scan, where
// one thread would walk them one after the other): first child at the level below (k + 1; with the "no prefix reuse"
// study switch the groups of level K-1 are the rows themselves, so level K-2 points at rows), and, for the levels
// whose left operand is looked up through it (3..K-1), the parent at level k-1.
__global__ void __launch_bounds__(256) k_links(WsView w, int k)
{
    tt_pdl_enter();
    const int K = w.K;
    const uint32_t count = w.counters[CTR_LEVEL0 + k];
    const bool rows = (w.ablation & 1) && k == K - 1;          // level k holds one node per row, not per prefix
    const int c = ((w.ablation & 1) && k + 1 == K - 1) ? K : k + 1;
    const uint32_t first = blockIdx.x * blockDim.x + threadIdx.x;
    if (first == 0 && !rows) w.cstart[k][count] = w.counters[CTR_LEVEL0 + c];
    for (uint32_t v = first; v < count; v += gridDim.x * blockDim.x) {
        const int t = tt_find_table(w.tb[k], w.T, v);
        const TableDesc& td = w.tdesc[t];
        if (!rows) {
            const uint32_t mult = c == k + 1 ? (uint32_t)td.n[k] : td.suffix[k];   // value of the first possible child
            w.cstart[k][v] = tt_rank_at(w, td, c, w.val[k][v] * mult);
        }
        if (w.parent[k]) {
            const uint32_t up = rows ? w.val[K][v] / td.suffix[k - 1] : w.val[k][v] / (uint32_t)td.n[k - 1];
            w.parent[k][v] = tt_rank_at(w, td, k - 1, up);
        }
    }
}

// Study switch "no prefix reuse": every distinct row is a group of its own at level K-1
__global__ void __launch_bounds__(256) k_unique_groups(WsView w)
{
    tt_pdl_enter();
    const int K = w.K, k = K - 1;
    const uint32_t count = w.counters[CTR_LEVEL0 + K] < w.cap[k] ? w.counters[CTR_LEVEL0 + K] : w.cap[k];
    const uint32_t first = blockIdx.x * blockDim.x + threadIdx.x;
    if (first == 0) {
        w.counters[CTR_LEVEL0 + k] = count;
        w.cstart[k][count] = count;
    }
    if (first <= (uint32_t)w.T) w.tb[k][first] = w.tb[K][first] < count ? w.tb[K][first] : count;
    for (uint32_t v = first; v < count; v += gridDim.x * blockDim.x) {
        const int t = tt_find_table(w.tb[K], w.T, v);
        w.val[k][v] = w.val[K][v] / (uint32_t)w.tdesc[t].n[K - 1];
        w.cstart[k][v] = v;
    }
}

// Study switch "no de-duplication" (the first arm of the paper's reuse ablation): lookup l is row slot l and a group of
// its own at every prefix level, so nothing is shared: every lookup rebuilds its whole chain of products.
// Lookups with a row id outside the table keep the row 0 (the pooling pass skips them by their id).
__global__ void __launch_bounds__(256) k_nodedup_levels(WsView w)
{
    tt_pdl_enter();
    const int K = w.K;
    const int64_t L = w.L < (int64_t)w.cap[K] ? w.L : (int64_t)w.cap[K];
    const int64_t first = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (first == 0) {
        if (w.L > (int64_t)w.cap[K]) atomicOr(w.status, TT_EMB_STATUS_OVERFLOW);
        for (int k = 1; k <= K; ++k) {
            w.counters[CTR_LEVEL0 + k] = (uint32_t)L;
            if (k < K) w.cstart[k][L] = (uint32_t)L;
        }
    }
    if (first <= w.T)
        for (int k = 1; k <= K; ++k) {
            const int64_t v = w.tl_start[first];
            w.tb[k][first] = (uint32_t)(v < L ? v : L);
        }
    int t = 0;
    for (int64_t l = first; l < L; l += (int64_t)gridDim.x * blockDim.x) {
        if (!(w.tl_start[t] <= l && l < w.tl_start[t + 1])) t = tt_find_table64(w.tl_start, w.T, l);
        const TableDesc& td = w.tdesc[t];
        const int64_t g = tt_index(w, l);
        if (g < 0 || g >= td.N) atomicOr(w.status, TT_EMB_STATUS_INDEX);
        uint32_t v = (g >= 0 && g < td.N) ? (uint32_t)g : 0u;
        for (int k = K; k >= 1; --k) {
            w.val[k][l] = v;
            if (k < K) w.cstart[k][l] = (uint32_t)l;
            if (w.parent[k]) w.parent[k][l] = (uint32_t)l;
            v /= (uint32_t)td.n[k - 1];
        }
    }
}

cudaError_t tt_launch_grouping(tt_emb* h, cudaStream_t s)
{
    WsView& w = h->v;
    cudaError_t e;
    // status word + counters are adjacent; bitmap follows its own region
    if ((e = cudaMemsetAsync(w.status, 0, (16 + 64) * sizeof(uint32_t), s)) != cudaSuccess) return e;
    const int64_t nb = (int64_t)w.T * w.B + 1;
    int g0 = (int)((nb + 255) / 256);
    if (g0 > h->sm_count * 8) g0 = h->sm_count * 8;
    if (w.ablation & 4) {
        if ((e = tt_launch_pdl(k_check_offsets, dim3(g0), dim3(256), 0, s, w)) != cudaSuccess) return e;
        tt_note_launch();
        if ((e = tt_launch_pdl(k_nodedup_levels, dim3(h->sm_count * 8), dim3(256), 0, s, w)) != cudaSuccess) return e;
        tt_note_launch();
        return cudaGetLastError();
    }
    if ((e = cudaMemsetAsync(w.bm, 0, (size_t)w.total_words * sizeof(uint2), s)) != cudaSuccess) return e;
    if ((e = tt_launch_pdl(k_check_offsets, dim3(g0), dim3(256), 0, s, w)) != cudaSuccess) return e;
    tt_note_launch();
    if (w.L > 0) {
        int64_t want = (w.L + 1023) / 1024;
        int g1 = (int)(want < (int64_t)h->sm_count * 8 ? want : (int64_t)h->sm_count * 8);
        if ((e = tt_launch_pdl(k_mark, dim3(g1), dim3(256), 0, s, w)) != cudaSuccess) return e;
        tt_note_launch();
    }
    PopScan ps{w};
    if ((e = tt_scan(ps, w.total_words, w.scan_tmp, s, (unsigned)(TT_HEAD_TILES * w.T) + w.rest_tiles)) != cudaSuccess) return e;
    for (int k = w.K - 1; k >= 1; --k) {
        {
            const uint32_t want = (w.total_words_l[k] + 7u) / 8u;   // a warp per word
            const uint32_t g = want < (uint32_t)h->sm_count * 8u ? (want ? want : 1u) : (uint32_t)h->sm_count * 8u;
            if ((e = tt_launch_pdl(k_prefix_bits, dim3(g), dim3(256), 0, s, w, k)) != cudaSuccess) return e;
            tt_note_launch();
        }
        LevelScan ls{w, k};
        if ((e = tt_scan<LevelScan, TT_LSCAN_ITEMS>(ls, w.total_words_l[k], w.scan_tmp, s)) != cudaSuccess) return e;
        if ((w.ablation & 1) && k == w.K - 1) {   // the scan still sets the bits of level K-2; its nodes are replaced
            if ((e = tt_launch_pdl(k_unique_groups, dim3(h->sm_count * 8), dim3(256), 0, s, w)) != cudaSuccess) return e;
            tt_note_launch();
        }
    }
    for (int k = w.K - 1; k >= 1; --k) {   // after all the scans: a node's links look into the levels on both sides
        if ((e = tt_launch_pdl(k_links, dim3(h->sm_count * 8), dim3(256), 0, s, w, k)) != cudaSuccess) return e;
        tt_note_launch();
    }
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------- export (inspection)

// first leaf (level-K node) under node v of level k
__device__ __forceinline__ uint32_t tt_first_leaf(const WsView& w, int k, uint32_t v)
{
    for (int j = k; j < w.K; ++j) v = w.cstart[j][v];
    return v;
}

__global__ void k_export_mult(WsView w, int table)
{
    // lookups per distinct row of one table -> cursor[] (scratch), via the rank structure
    const TableDesc& td = w.tdesc[table];
    const int64_t lo = w.tl_start[table], hi = w.tl_start[table + 1];
    for (int64_t l = lo + (int64_t)blockIdx.x * blockDim.x + threadIdx.x; l < hi; l += (int64_t)gridDim.x * blockDim.x) {
        const int64_t g = tt_index(w, l);
        if (g < 0 || g >= td.N) continue;
        const uint2 e = w.bm[td.word_base + ((uint32_t)g >> 5)];
        const uint32_t slot = e.y + __popc(e.x & ((1u << (g & 31)) - 1u));
        if (slot < w.cap[w.K]) atomicAdd(&w.cursor[slot], 1u);
    }
}

__global__ void k_export_level(WsView w, int table, int k, int64_t* vals, int32_t* rc, int32_t* lc, int have_mult)
{
    const uint32_t v0 = w.tb[k][table], v1 = w.tb[k][table + 1];
    for (uint32_t v = v0 + blockIdx.x * blockDim.x + threadIdx.x; v < v1; v += gridDim.x * blockDim.x) {
        if (vals) vals[v - v0] = (int64_t)w.val[k][v];
        const uint32_t l0 = tt_first_leaf(w, k, v);
        const uint32_t l1 = (v + 1 < w.counters[CTR_LEVEL0 + k]) ? tt_first_leaf(w, k, v + 1) : w.counters[CTR_LEVEL0 + w.K];
        if (rc) rc[v - v0] = (int32_t)(l1 - l0);
        if (lc && have_mult) {
            uint32_t s = 0;
            for (uint32_t u = l0; u < l1; ++u) s += w.cursor[u];
            lc[v - v0] = (int32_t)s;
        }
    }
}

cudaError_t tt_launch_export_level(tt_emb* h, int table, int level, int64_t* vals, int32_t* rc, int32_t* lc, cudaStream_t s)
{
    WsView& w = h->v;
    if (lc) {
        cudaError_t e = cudaMemsetAsync(w.cursor, 0, (size_t)w.cap[w.K] * sizeof(uint32_t), s);
        if (e != cudaSuccess) return e;
        k_export_mult<<<h->sm_count * 4, 256, 0, s>>>(w, table);
        tt_note_launch();
    }
    k_export_level<<<h->sm_count * 4, 256, 0, s>>>(w, table, level, vals, rc, lc, lc ? 1 : 0);
    tt_note_launch();
    return cudaGetLastError();
}

__global__ void k_export_inverse(WsView w, int table, int32_t* inv)
{
    const TableDesc& td = w.tdesc[table];
    const int64_t lo = w.tl_start[table], hi = w.tl_start[table + 1];
    const uint32_t base = w.tb[w.K][table];
    for (int64_t l = lo + (int64_t)blockIdx.x * blockDim.x + threadIdx.x; l < hi; l += (int64_t)gridDim.x * blockDim.x) {
        const int64_t g = tt_index(w, l);
        int32_t r = -1;
        if (g >= 0 && g < td.N) {
            const uint2 e = w.bm[td.word_base + ((uint32_t)g >> 5)];
            r = (w.ablation & 4) ? (int32_t)(l - lo) : (int32_t)(e.y + __popc(e.x & ((1u << (g & 31)) - 1u)) - base);
        }
        inv[l - lo] = r;
    }
}

cudaError_t tt_launch_export_inverse(tt_emb* h, int table, int32_t* inv, cudaStream_t s)
{
    k_export_inverse<<<h->sm_count * 4, 256, 0, s>>>(h->v, table, inv);
    tt_note_launch();
    return cudaGetLastError();
}

// ---------------------------------------------------------------------------------------------- core layout conversion

__global__ void k_pack(const float* __restrict__ src, float* __restrict__ dst, int rp, int n, int d, int rn, int to_canonical)
{
    // canonical [n][rp][d][rn]  <->  index order [rp][n][d][rn]
    const int64_t total = (int64_t)rp * n * d * rn;
    const int inner = d * rn;
    for (int64_t c = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; c < total; c += (int64_t)gridDim.x * blockDim.x) {
        const int x = (int)(c % inner);
        const int64_t q = c / inner;
        const int a = (int)(q % rp);
        const int i = (int)(q / rp);
        const int64_t o = ((int64_t)a * n + i) * inner + x;
        if (to_canonical) dst[c] = src[o]; else dst[o] = src[c];
    }
}

cudaError_t tt_launch_pack(const TableDesc& td, int core, const float* src, float* dst, bool to_canonical, cudaStream_t s)
{
    const int64_t total = td.core_floats[core];
    int grid = (int)((total + 255) / 256);
    if (grid > 4096) grid = 4096;
    if (grid < 1) grid = 1;
    k_pack<<<grid, 256, 0, s>>>(src, dst, td.r[core], td.n[core], td.d[core], td.r[core + 1], to_canonical ? 1 : 0);
    tt_note_launch();
    return cudaGetLastError();
}
