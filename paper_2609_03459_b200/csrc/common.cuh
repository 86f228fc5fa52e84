// Internal declarations shared by the translation units of libtt_emb.so (sm_100a only).
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>
#include <stddef.h>

#include "tt_emb.h"

#define TT_MAXK 4
#define TT_SCAN_THREADS 256
#define TT_SCAN_ITEMS 16
#define TT_SCAN_TILE (TT_SCAN_THREADS * TT_SCAN_ITEMS)  // elements per scan tile
#define TT_POOL_MAX_SHARES 262144                       // shares of the lookups that the pooling warps take in order
#define TT_HEAD_TILES 4                                 // leading scan tiles of a table that are emitted first (see PopScan)
#define TT_LSCAN_ITEMS 2                                // the short scans of the prefix-level bitmaps
#define TT_LSCAN_TILE (TT_SCAN_THREADS * TT_LSCAN_ITEMS)
#define TT_DE_CHUNK 1024                                  // sorted lookups per warp in the dE segment reduction
#define TT_NUM_STAGES 33                                // 0..8 pipeline stages, 9..20 forward sweep variants -1..10, 21..32 backward sweep variants
#define TT_STRIPES 8                                     // L2-resident partial copies of the last core's gradient
#define TT_NUM_MIDFAST 11                                // tensor-core instances of the middle-core backward (backward.cu)
#define TT_NUM_VARIANTS 11                               // register-tiled shape variants (forward.cu)

// Per-table descriptor, resident in the workspace.  k below is 0-based (core k+1 of the paper).
struct TableDesc {
    int64_t N;
    int32_t n[TT_MAXK];
    int32_t d[TT_MAXK];
    int32_t r[TT_MAXK + 1];
    int32_t P[TT_MAXK + 1];             // P[0] = 1, P[k] = d_1 * .. * d_k
    int32_t slice_floats[TT_MAXK];      // r[k] * d[k] * r[k+1]
    int64_t core_floats[TT_MAXK];       // n[k] * slice_floats[k]
    float* core[TT_MAXK];
    float* grad[TT_MAXK];
    uint32_t word_base;                 // first 32-row word of this table in the presence bitmap
    uint32_t num_words;
    uint32_t rest_base;                 // scan tiles of the tables before this one, their first TT_HEAD_TILES each left out
    uint32_t lword_base[TT_MAXK];       // the same for the presence bitmaps of the length-k prefixes, k = 1..K-1
    uint32_t suffix[TT_MAXK];           // n_{k+1} * .. * n_K: row id / suffix[k] = length-k prefix value, k = 1..K-1
    uint32_t tword_base[TT_MAXK];       // same for the digit-major ("transposed") node bitmaps, levels 2..K-1
    uint32_t tnum_words[TT_MAXK];
    uint32_t prefix_space[TT_MAXK + 1]; // n_1 * .. * n_k (number of possible length-k prefixes), k = 1..K-1
    int64_t gpart_off;                  // float offset of this table's last core inside one stripe
    int32_t units;                      // work units (CTAs) this table is cut into
    int32_t unit_base;                  // first global unit id
    int32_t sgd_mask;                   // bit k: the fused backward + SGD call updates core k inside the kernel that finalises its gradient
    int32_t fast;                       // register-tiled kernel variant for this table's shapes, -1 = generic path
    int32_t midfast[TT_MAXK];           // same for the middle-core backward of level k (index k), -1 = generic
};

// Device-side view of the workspace handed to kernels by value.
struct WsView {
    int32_t T, K, D;
    int32_t ablation;                   // study switches: bit 0 no prefix reuse, bit 1 static (equal-count) schedule,
                                        // bit 2 no de-duplication (every lookup is its own row and its own group; implies bit 0)
    float fused_lr;                     // != 0: the kernels that finalise a gradient also apply G -= fused_lr * dG (cores in sgd_mask)
    int32_t stride[TT_MAXK + 1];        // floats per node of the level-k partial-product buffers (max over tables)
    int64_t B, L;                       // current batch / lookups
    int64_t capU;                       // capacity in distinct rows
    uint32_t cap[TT_MAXK + 1];          // node capacity per level 1..K
    uint32_t total_words;
    uint32_t ttotal_words[TT_MAXK];
    int32_t* status;
    uint32_t* counters;                 // [k] = number of level-k nodes (k = 1..K); [8+k] transposed counts
    TableDesc* tdesc;
    int32_t* vlist;                     // [0,T): table ids grouped by kernel variant (generic first); [T,2T): all tables;
                                        // largest tables first inside each list
    int64_t* tl_start;                  // [T+1] first lookup of each table
    uint2* bm;                          // {32 presence bits, number of set bits before this word (global)}
    uint2* bml[TT_MAXK];                // the same for the length-k prefixes, k = 1..K-1 (one bit per possible prefix)
    uint32_t total_words_l[TT_MAXK];
    uint32_t rest_tiles;                // scan tiles of the row bitmap beyond the first TT_HEAD_TILES of every table
    uint32_t* scan_tmp;
    uint32_t* val[TT_MAXK + 1];         // level k: prefix value within the table (k = K: row id)
    uint32_t* cstart[TT_MAXK + 1];      // level k < K: first child (level k+1 node); [count] = sentinel
    uint32_t* parent[TT_MAXK + 1];      // levels 3..K-1: parent node at level k-1 (null elsewhere: nothing reads it)
    uint32_t* tb[TT_MAXK + 1];          // [T+1] node range of each table at level k
    uint32_t* cost;                     // [cap_{K-1}+1] exclusive scan of per-group cost (+ total)
    int64_t* pool_bounds;               // [shares + 1] first bag of every share of the pooling pass (k_pool_bounds)
    uint2* unit_rng;                    // [T * units per table] group range of every work unit (k_unit_ranges)
    int32_t units_per_table;
    float* pbuf[TT_MAXK + 1];           // partial products P_k of level-k nodes, 2 <= k <= K-2
    float* E;                           // [capU][D] rows (forward) / dE (backward)
    // backward
    uint32_t* cnt;                      // [capU+1] lookups per distinct row -> exclusive scan
    uint32_t* cursor;                   // [capU]
    uint2* pairs;                       // [L] (slot, bag) sorted by slot
    uint2* upairs;                      // [L] (slot, bag) in lookup order, written by the pooling kernel (null: forward only)
    float* dP[TT_MAXK + 1];             // dP_k per level-k node, 2 <= k <= K-1
    float* Y[TT_MAXK + 1];              // per level-k node: its contribution to dP_{k-1} of its parent
    float* carry;                       // [chunks][2][D]
    float* gpart;                       // [TT_STRIPES][gpart_stride] partial copies of all tables' last-core gradients
    int64_t gpart_stride;               // floats per stripe
    uint2* tbm[TT_MAXK + 1];            // digit-major node bitmaps, levels 2..K-1
    uint32_t* tnode[TT_MAXK + 1];       // nodes of level k ordered by (table, i_k, parent prefix)
    const int64_t* indices;
    const int64_t* offsets;
    // pooling beyond the plain sum (tt_emb_set_pooling)
    const float* psw;                   // per-lookup weights [L] or null
    float* wsorted;                     // [L] factor of every sorted pair (weight, or 1 / bag length), backward only
    int32_t pool_mean;                  // 1: mean pooling
    int32_t idx32;                      // 1: `indices` points at int32 row ids (tt_emb_forward_i32)
};

// row id of lookup l (int64 or int32 storage); STREAM: read-once hint
template <bool STREAM = false>
__device__ __forceinline__ int64_t tt_index(const WsView& w, int64_t l)
{
    if (w.idx32) {
        const int32_t* p = reinterpret_cast<const int32_t*>(w.indices) + l;
        return (int64_t)(STREAM ? __ldcs(p) : __ldg(p));
    }
    return STREAM ? __ldcs(w.indices + l) : __ldg(w.indices + l);
}

enum { CTR_LEVEL0 = 0 /* +k */, CTR_TLEVEL0 = 8 /* +k */, CTR_COST_TOTAL = 16, CTR_SCAN_TICKET = 32 /* tiles of the running scan that have reported */,
       CTR_POOL_NEXT = 34 /* next share of the lookups to be pooled (shares are handed out in order) */ };

struct tt_emb {
    int T, K, D;
    int64_t max_batch, max_lookups, capU;
    int enable_backward;
    int enable_weighted;
    int ablation;
    int sm_count;
    int units_total;
    int units_per_table;
    int vcount[TT_NUM_VARIANTS + 1];   // tables per variant, index 0 = generic (-1)
    int vbase[TT_NUM_VARIANTS + 1];    // first entry of each variant in vlist
    // middle-core kernels of level k: tables grouped by their variant (index 0 = generic), largest first, in
    // vlist[(2 + k) * T ..); first entry, count and largest n_k of each group
    int mbase[TT_MAXK + 1][TT_NUM_MIDFAST + 1], mcount[TT_MAXK + 1][TT_NUM_MIDFAST + 1], mmaxn[TT_MAXK + 1][TT_NUM_MIDFAST + 1];
    int32_t* vlist_host;
    size_t off_vlist;
    int cost_shift;       // cost unit of the schedule = 2^cost_shift FMAs
    TableDesc* tab;       // host copy [T]
    size_t ws_bytes;
    size_t off_status, off_counters, off_tdesc, off_tlstart, off_bm, off_scan, off_cost, off_E;
    size_t off_bml[TT_MAXK];
    size_t off_val[TT_MAXK + 1], off_cstart[TT_MAXK + 1], off_parent[TT_MAXK + 1], off_tb[TT_MAXK + 1];
    size_t off_pbuf[TT_MAXK + 1], off_dP[TT_MAXK + 1], off_tbm[TT_MAXK + 1], off_tnode[TT_MAXK + 1];
    size_t off_Y[TT_MAXK + 1];
    size_t off_cnt, off_cursor, off_pairs, off_carry, off_gpart, off_wsorted, off_unit_rng, off_pool_bounds;
    // guard bytes after every workspace region (tt_emb_check_guards): [guard_off[i], guard_off[i] + guard_len[i])
    int num_regions;
    size_t guard_off[96], guard_len[96];
    const char* region_name[96];
    size_t off_guard_list;      // device copy of the (offset, length) pairs + the check's result word
    void* ws_base;
    size_t scan_tmp_elems;
    int64_t gpart_floats;
    WsView v;             // filled at bind
    bool bound, have_forward;
    bool timing;
    bool serial;          // timing mode 2: shape-variant kernels run one after the other (per-kernel durations)
    cudaEvent_t ev[TT_NUM_STAGES][2];
    bool ev_valid[TT_NUM_STAGES];
    bool ev_created;
    // side streams for kernels of different shape variants that may overlap (created on first use)
    cudaStream_t side[4];
    cudaEvent_t side_ev[5];
    bool side_created;
};

// every kernel launch of the library is noted here (api.cu); read with tt_emb_launch_count
void tt_note_launch(int n = 1);
// remember a failing CUDA call for tt_emb_last_cuda_error (api.cu)
void tt_set_last_cuda_error(cudaError_t e);
// compute capability 10.x device current? (api.cu)
int tt_device_ok(int* sm_count);

// fork/join helpers (api.cu): side streams wait for everything enqueued on `s` so far / `s` waits for the side streams
cudaError_t tt_fork(tt_emb* h, cudaStream_t s, int n);
cudaError_t tt_join(tt_emb* h, cudaStream_t s, int n);

// stage timing (api.cu): no-ops unless timing is enabled
cudaError_t tt_stage_begin(tt_emb* h, int stage, cudaStream_t s);
cudaError_t tt_stage_end(tt_emb* h, int stage, cudaStream_t s);

// ---- launchers implemented in the .cu files (all enqueue on `s`, return cudaGetLastError()) ----
cudaError_t tt_launch_grouping(tt_emb* h, cudaStream_t s);
cudaError_t tt_launch_schedule(tt_emb* h, cudaStream_t s);
cudaError_t tt_launch_tlist(tt_emb* h, int k, cudaStream_t s);   // digit-major list of the level-k nodes
cudaError_t tt_launch_contraction(tt_emb* h, cudaStream_t s);
cudaError_t tt_launch_pooling(tt_emb* h, float* out, cudaStream_t s);
cudaError_t tt_launch_bwd_sort(tt_emb* h, cudaStream_t s);
cudaError_t tt_launch_bwd_dE(tt_emb* h, const float* grad_out, cudaStream_t s);
cudaError_t tt_launch_bwd_contraction(tt_emb* h, cudaStream_t s);
cudaError_t tt_launch_bwd_middle(tt_emb* h, cudaStream_t s);
cudaError_t tt_launch_sgd(tt_emb* h, float lr, bool only_unfused, cudaStream_t s);
cudaError_t tt_launch_export_level(tt_emb* h, int table, int level, int64_t* vals, int32_t* rc, int32_t* lc, cudaStream_t s);
cudaError_t tt_launch_export_inverse(tt_emb* h, int table, int32_t* inv, cudaStream_t s);
cudaError_t tt_launch_pack(const TableDesc& td, int core, const float* src, float* dst, bool to_canonical, cudaStream_t s);

// ---- programmatic dependent launch: the kernels of the forward chain are launched with the attribute below and
// begin with tt_pdl_enter().  A kernel's CTAs may then become resident while its predecessor in the stream is still
// running and wait (griddepcontrol.wait) until that grid has completed and its writes are visible, so the launch
// latency of a chain of short kernels overlaps the previous kernel instead of following it.  Without the attribute
// (or after a non-kernel operation in the stream) the wait returns at once.
__device__ __forceinline__ void tt_pdl_enter()
{
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

template <class... KArgs, class... Args>
static inline cudaError_t tt_launch_pdl(void (*kern)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t s, Args&&... args)
{
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, static_cast<KArgs>(args)...);
}

// a += v as two packed fp32 additions (add.rn.f32x2 of sm_100: two IEEE additions per instruction and lane, the same
// results as four scalar additions; the row sums of the gathers are bound by issue slots)
__device__ __forceinline__ void tt_add4(float4& a, const float4& v)
{
    const float2 lo = __fadd2_rn(make_float2(a.x, a.y), make_float2(v.x, v.y));
    const float2 hi = __fadd2_rn(make_float2(a.z, a.w), make_float2(v.z, v.w));
    a = make_float4(lo.x, lo.y, hi.x, hi.y);
}

// ---- small device helpers ----
__device__ __forceinline__ int tt_find_table(const uint32_t* __restrict__ tb, int T, uint32_t v)
{
    // largest t with tb[t] <= v  (tb non-decreasing, tb[0] = 0)
    int lo = 0, hi = T;
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if (tb[mid] <= v) lo = mid; else hi = mid;
    }
    return lo;
}

// the same, starting from a table known not to lie after v's (elements of a tile are ascending: the table of the
// tile's first element); usually no step at all
__device__ __forceinline__ int tt_find_table_from(const uint32_t* __restrict__ tb, int T, uint32_t v, int t)
{
    while (t + 1 < T && tb[t + 1] <= v) ++t;
    return t;
}

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

// 16-byte asynchronous copy global -> shared, past L1
__device__ __forceinline__ void tt_cp_async16(void* smem_dst, const void* gsrc)
{
    const unsigned d = (unsigned)__cvta_generic_to_shared(smem_dst);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(d), "l"(gsrc) : "memory");
}

// left operand of level k (2..K-1) for node v: P_{k-1} of its parent (k = 2: the slice of the first core)
__device__ __forceinline__ const float* tt_left_operand(const WsView& w, const TableDesc& td, int k, uint32_t v)
{
    if (k == 2) {
        const uint32_t i1 = w.val[2][v] / (uint32_t)td.n[1];
        return td.core[0] + (size_t)i1 * td.slice_floats[0];
    }
    return w.pbuf[k - 1] + (size_t)w.parent[k][v] * w.stride[k - 1];
}

// group range [g0, g1) of work unit q of table t: an equal-cost slice of the table's level-(K-1) groups in sweep order
// (called by one thread per unit, once per forward: k_unit_ranges)
__device__ __forceinline__ void tt_unit_range(const WsView& w, int t, int q, uint32_t& g0, uint32_t& g1)
{
    const TableDesc& td = w.tdesc[t];
    const int lvl = w.K - 1;
    const uint32_t a = w.tb[lvl][t], b = w.tb[lvl][t + 1];
    // the host sizes the grid for the largest possible number of groups; with fewer groups in this batch the table is
    // cut into fewer units (at least 16 groups each) and the surplus CTAs leave at once
    int Q = td.units;
    {
        const int by_groups = (int)((b - a) >> 4);
        if (Q > by_groups) Q = by_groups < 1 ? 1 : by_groups;
    }
    if (q >= Q) { g0 = a; g1 = a; return; }
    const uint64_t ca = w.cost[a], cb = w.cost[b];
    if (w.ablation & 2) {   // study switch: static schedule, equal group counts
        g0 = a + (uint32_t)((uint64_t)(b - a) * (uint64_t)q / Q);
        g1 = a + (uint32_t)((uint64_t)(b - a) * (uint64_t)(q + 1) / Q);
        return;
    }
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
}

__device__ __forceinline__ int tt_find_table64(const int64_t* __restrict__ tb, int T, int64_t v)
{
    int lo = 0, hi = T;
    while (hi - lo > 1) {
        int mid = (lo + hi) >> 1;
        if (tb[mid] <= v) lo = mid; else hi = mid;
    }
    return lo;
}
