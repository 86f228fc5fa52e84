/*
 * tt_emb.h -- C ABI of the B200 (sm_100a) Tensor-Train embedding-bag library.
 *
 * What the library computes (paper sections in brackets):
 *   * an embedding table of N rows x D columns is stored as K TT-cores G_k[a][i][j][b],
 *     a < r_{k-1}, i < n_k, j < d_k, b < r_k, r_0 = r_K = 1, prod n_k >= N, prod d_k = D   [Sec. 2.1]
 *   * a row id g is split mixed-radix into digits (i_1..i_K), i_1 most significant          [Eq. 1]
 *   * the row is the chain of slice products G_1[i_1] . G_2[i_2] ... G_K[i_K], flattened
 *     row-major over (j_1..j_K)                                   [Sec. 3.2, "C = A.B, E = C.D"]
 *   * rows are sum-pooled per bag (duplicates counted, empty bag = zeros)    [Sec. 3.2, "V"]
 *   * looked-up rows are de-duplicated and grouped by shared digit prefixes so that every
 *     distinct prefix product is formed once                                         [Sec. 3.3]
 *   * backward: dE per distinct row, dD = C^T.dE, dC = dE.D^T summed over the rows that share C
 *     before going up a level, then dA, dB                                   [Sec. 3.2, Eq. 2]
 *
 * General rules
 *   * Every function returns 0 (TT_EMB_OK) or a negative tt_emb_error code.  Nothing throws,
 *     aborts or traps.  There is no CPU fallback: without a CUDA device of compute capability
 *     10.x the compute entry points return TT_EMB_ERR_ARCH.
 *   * "device" pointers are CUDA device memory of the current device, "host" pointers ordinary
 *     host memory.  The library allocates no device memory: the caller provides one workspace.
 *   * `stream` is a cudaStream_t passed as void* (NULL = legacy default stream).  All device work
 *     is enqueued on it; no entry point synchronises the host unless its comment says so.
 *   * Data-dependent problems (row id out of range, malformed offsets, more distinct rows than
 *     max_unique_rows) are detected on the device; the offending lookups contribute nothing and a
 *     bit is set in the device status word, read back with tt_emb_status().
 *   * Core layout on the device ("slice-major"): core k of a table is float[n_k][r_{k-1}][d_k][r_k],
 *     i.e. the slice of one digit value is one contiguous block.  tt_emb_pack_core /
 *     tt_emb_unpack_core convert from / to the index order [r_{k-1}][n_k][d_k][r_k].
 *     Gradients use the same slice-major layout.
 *   * Limits: 2 <= K <= 4; N_t < 2^31; num_lookups < 2^31; batch * num_tables < 2^31;
 *     D <= 1024; every r_k <= 128; prod_{m<k} d_m * r_k <= 4096 floats per partial product.
 */
#ifndef TT_EMB_H
#define TT_EMB_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct tt_emb* tt_emb_t; /* opaque host-side handle */
typedef void* tt_emb_stream_t;   /* cudaStream_t */

enum tt_emb_error {
    TT_EMB_OK = 0,
    TT_EMB_ERR_ARG = -1,       /* null pointer, bad shape, limit exceeded */
    TT_EMB_ERR_WORKSPACE = -2, /* workspace missing, misaligned or too small */
    TT_EMB_ERR_ARCH = -3,      /* no CUDA device of compute capability 10.x */
    TT_EMB_ERR_STATE = -4,     /* call order: not bound, backward before forward, ... */
    TT_EMB_ERR_CUDA = -5       /* a CUDA runtime call failed (see tt_emb_last_cuda_error) */
};

/* bits of the device status word (tt_emb_status) */
enum tt_emb_status_bits {
    TT_EMB_STATUS_INDEX = 1,    /* some row id was < 0 or >= N_t; it contributed nothing */
    TT_EMB_STATUS_OFFSETS = 2,  /* offsets not non-decreasing / not starting at 0 / not ending at L */
    TT_EMB_STATUS_OVERFLOW = 4  /* more distinct rows than max_unique_rows; surplus rows dropped */
};

typedef struct {
    int32_t num_tables;         /* T >= 1 */
    int32_t num_cores;          /* K, 2..4, same for every table */
    const int64_t* num_rows;    /* host [T]        N_t */
    const int32_t* row_factors; /* host [T*K]      n_{t,k}, product >= N_t */
    const int32_t* dim_factors; /* host [T*K]      d_{t,k}, product = D, the same D for every table */
    const int32_t* ranks;       /* host [T*(K+1)]  r_{t,0} = 1 .. r_{t,K} = 1 */
    int64_t max_batch;          /* upper bound on `batch` (bags per table) */
    int64_t max_lookups;        /* upper bound on `num_lookups` (all tables together) */
    int64_t max_unique_rows;    /* upper bound on distinct (table,row) pairs per call; 0 = min(max_lookups, sum N_t) */
    int32_t enable_backward;    /* 0: forward only (smaller workspace); 1: tt_emb_backward may be called */
    int32_t ablation;           /* 0 = the full method.  Study switches (forward only; tt_emb_create rejects them together
                                   with enable_backward): bit 0 = no prefix reuse, every distinct row forms its own group
                                   and rebuilds its prefix product ("unique only", cf. the paper's reuse ablation);
                                   bit 1 = static schedule, every table cut into units of equal group COUNT instead of
                                   equal cost (cf. the paper's scheduling ablation); bit 2 = no de-duplication, every
                                   lookup is a row and a group of its own ("no dedup", the first arm of the reuse
                                   ablation; sizes the row buffer for max_lookups rows; implies bit 0) */
    int32_t enable_weighted;    /* 1: tt_emb_set_pooling may select mean pooling or per-lookup weights (with the
                                   backward enabled the workspace grows by 4 bytes per lookup) */
} tt_emb_config_t;

/* Host only.  Copies everything it needs out of *cfg.  [data model: Sec. 2.1] */
int tt_emb_create(const tt_emb_config_t* cfg, tt_emb_t* out_handle);
int tt_emb_destroy(tt_emb_t h);

/* Bytes of device workspace tt_emb_bind needs (256-byte aligned base). */
int tt_emb_workspace_bytes(tt_emb_t h, size_t* bytes);
/* Number of floats of core `core` (0-based) of table `table`: n*r_prev*d*r_next. */
int tt_emb_core_floats(tt_emb_t h, int32_t table, int32_t core, int64_t* count);
/* Embedding dimension D. */
int tt_emb_dim(tt_emb_t h, int32_t* D);

/*
 * Attach the cores and the workspace.  core_ptrs: HOST array of T*K DEVICE pointers
 * (table-major: table 0 core 0..K-1, table 1 ...), each slice-major fp32, 16-byte aligned.
 * The caller owns cores and workspace and keeps them alive while the handle is used.
 * Enqueues a small upload on `stream`; the host array may be freed on return.
 */
int tt_emb_bind(tt_emb_t h, float* const* core_ptrs, void* workspace, size_t workspace_bytes,
                tt_emb_stream_t stream);

/*
 * Forward: out[b, t*D + j] = sum over lookups l of bag (t,b) of row_t(indices[l])[j].
 *   [Eq. 1 digits; Sec. 3.3 grouping; Sec. 3.2 stages 1-3]
 * indices  device int64[num_lookups], table-major: all bags of table 0, then table 1, ...
 * offsets  device int64[T*batch + 1], CSR over (table, bag): bag (t,b) owns
 *          indices[offsets[t*batch+b] .. offsets[t*batch+b+1]); offsets[0] = 0, last = num_lookups
 * out      device fp32[batch][T*D], row-major, fully overwritten (also when a status bit reports malformed
 *          offsets: every bag is then summed over its offsets clamped to [0, num_lookups], an inverted pair
 *          counting as an empty bag)
 * The forward keeps what the backward needs (one (row slot, bag) pair per lookup) in the workspace: `indices` may be
 * freed or overwritten once the forward has completed.  `offsets` must stay valid and unchanged until the backward
 * has completed if mean pooling is selected (the bag lengths are re-read); the inspection calls
 * tt_emb_export_level (with lookup_counts) and tt_emb_export_inverse re-read both arrays.  Asynchronous.
 */
int tt_emb_forward(tt_emb_t h, const int64_t* indices, const int64_t* offsets, int64_t batch,
                   int64_t num_lookups, float* out, tt_emb_stream_t stream);

/*
 * The same forward with 32-bit row ids (every N_t is below 2^31 anyway): half the bytes to bring to the device and to
 * read in the grouping and pooling passes.  indices: device int32[num_lookups]; everything else as tt_emb_forward.
 * The paper's interface has 64-bit ids only; this entry point is an addition for callers that hold 32-bit ids.
 */
int tt_emb_forward_i32(tt_emb_t h, const int32_t* indices, const int64_t* offsets, int64_t batch,
                       int64_t num_lookups, float* out, tt_emb_stream_t stream);

/*
 * Pooling mode of the forward / backward calls that follow (default: TT_EMB_POOL_SUM without weights, the paper's
 * pooling [Sec. 3.2]).  The two other forms are extensions that follow the usual embedding-bag operator; the paper
 * has no counterpart.
 *   TT_EMB_POOL_MEAN    out = bag's sum / number of lookups of the bag (an empty bag gives zeros)
 *   per_sample_weights  device fp32[num_lookups] (or NULL): lookup l contributes weights[l] * row; sum mode only.
 *                       Must stay valid and unchanged until the backward of the forward that used it has completed.
 * The backward differentiates the mode its forward used.  Needs cfg.enable_weighted (TT_EMB_ERR_STATE otherwise,
 * unless mode is SUM and the pointer NULL); weights together with MEAN is TT_EMB_ERR_ARG.  Host only.
 */
enum tt_emb_pooling { TT_EMB_POOL_SUM = 0, TT_EMB_POOL_MEAN = 1 };
int tt_emb_set_pooling(tt_emb_t h, int32_t mode, const float* per_sample_weights);

/*
 * Backward of the most recent forward on this handle, for loss = sum(grad_out * out).
 *   [Sec. 3.2 backward; Eq. 2: dC of rows sharing a prefix are summed before going up]
 * grad_out   device fp32[batch][T*D]
 * core_grads HOST array of T*K DEVICE pointers, each shaped like the matching core (slice-major);
 *            fully OVERWRITTEN (untouched slices become zero), not accumulated.
 * Lookups are sorted by row and reduced by segments (dE); first- and middle-core slices each have a single
 * owner that sums its sorted contributions; last-core slices are accumulated with vector reductions into a
 * few L2-resident partial copies that are then added in a fixed order.  Needs enable_backward = 1.
 * Asynchronous.
 */
int tt_emb_backward(tt_emb_t h, const float* grad_out, float* const* core_grads, tt_emb_stream_t stream);

/*
 * Forward for callers that cannot allocate device memory (no counterpart in the paper; added for embedding in
 * hosts with a fixed memory pool, plug-ins that only receive raw pointers, and allocation-frozen regions).
 * Same result as tt_emb_bind(core_ptrs, <workspace>) followed by tt_emb_forward(...), but the workspace is a
 * fixed 32 MiB array inside the library (tt_emb_static_workspace_limit()); nothing is allocated.
 *   - returns TT_EMB_ERR_WORKSPACE, launching nothing, if tt_emb_workspace_bytes(h) exceeds that limit;
 *   - the first call on a device looks up the array's address, and the first forward of a handle creates the
 *     handle's side streams and events and sets kernel attributes (host-side objects, no device memory): make those
 *     first calls outside any stream capture;
 *   - all calls on a device share the array (it keeps the previous call's contents; what must start at zero is
 *     cleared by the call); calls whose GPU work overlaps (other streams, other handles) race: serialise them;
 *   - afterwards the handle is bound to the array; a call on a handle that already is, with the same core
 *     pointers, enqueues nothing but the forward itself.
 * TT_EMB_ERR_ARCH without a compute-capability-10 device; TT_EMB_ERR_ARG if the current device's index is 64 or more.
 * core_ptrs as in tt_emb_bind; the remaining arguments as in tt_emb_forward.  Asynchronous.
 */
int tt_emb_forward_static(tt_emb_t h, float* const* core_ptrs, const int64_t* indices, const int64_t* offsets,
                          int64_t batch, int64_t num_lookups, float* out, tt_emb_stream_t stream);
size_t tt_emb_static_workspace_limit(void);

/* Plain SGD on every bound core: G <- G - lr * dG, elementwise fp32.  Asynchronous. */
int tt_emb_sgd_step(tt_emb_t h, float* const* core_grads, float lr, tt_emb_stream_t stream);

/*
 * tt_emb_backward followed by tt_emb_sgd_step(lr) as one call, with the update fused into the backward
 *   [Sec. 3.2 backward; the paper mentions a fused update and leaves it switched off]:
 * every core's gradient has a kernel that writes its final value (the fixed-order sum of the last core's partial
 * copies, the owner CTA of a middle-core slice, the sum over the children of a first digit); with lr != 0 that
 * kernel also applies G <- G - lr * dG to the elements it has just finished, so the gradient is not read again.
 * Cores whose gradient is finalised by a kernel that other blocks still read the core in (generic shape path,
 * K = 2 first core) are updated by the plain kernel at the end of the call.  core_grads is still fully written
 * (gradients at the pre-update cores), the result equals the two separate calls up to the rounding of identical
 * expressions.  Arguments and errors as tt_emb_backward; lr = 0 is tt_emb_backward.  Asynchronous.
 */
int tt_emb_backward_sgd(tt_emb_t h, const float* grad_out, float* const* core_grads, float lr, tt_emb_stream_t stream);

/*
 * Copy the device status word (OR of tt_emb_status_bits since the last forward began) to *status_host.
 * SYNCHRONISES `stream`.
 */
int tt_emb_status(tt_emb_t h, int32_t* status_host, tt_emb_stream_t stream);

/* ---- inspection of the grouping of the most recent forward (tests, diagnostics).  All SYNCHRONISE. ---- */

/*
 * counts_host: host int64[T*K]; entry t*K + (k-1) = number of distinct length-k digit prefixes of
 * table t among its lookups (k = K: distinct rows).  [Sec. 3.3]
 */
int tt_emb_grouping_counts(tt_emb_t h, int64_t* counts_host, tt_emb_stream_t stream);
/*
 * Prefix level k (1..K) of one table, ascending by prefix value, into DEVICE buffers with room for
 * the count reported by tt_emb_grouping_counts:
 *   vals           int64  prefix value floor(row / prod_{j>k} n_j)   (k = K: the row id)
 *   row_counts     int32  distinct rows under the prefix
 *   lookup_counts  int32  lookups under the prefix (with multiplicity)
 * Any of the three may be NULL.
 */
int tt_emb_export_level(tt_emb_t h, int32_t table, int32_t level, int64_t* vals, int32_t* row_counts,
                        int32_t* lookup_counts, tt_emb_stream_t stream);
/*
 * inv: DEVICE int32[lookups of this table]; inv[l] = position of lookup l's row among the table's
 * ascending distinct rows (-1 for an out-of-range row id).
 */
int tt_emb_export_inverse(tt_emb_t h, int32_t table, int32_t* inv, tt_emb_stream_t stream);

/* Register-tiled kernel variant that serves the last two levels of `table` (-1: the generic any-shape path). */
int tt_emb_table_variant(tt_emb_t h, int32_t table, int32_t* sweep_variant);

/*
 * Debug aid, a stand-in for a memory checker: tt_emb_bind writes guard bytes behind every region of the workspace
 * (status, bitmap, level arrays, row buffer, ...); this call reports in *first_bad the index of the first region whose
 * guard bytes no longer hold the pattern, i.e. that some kernel wrote past (-1: all intact), and
 * tt_emb_region_name(h, index) names it.  The paper has no counterpart.  SYNCHRONISES.
 */
int tt_emb_check_guards(tt_emb_t h, int32_t* first_bad, tt_emb_stream_t stream);
const char* tt_emb_region_name(tt_emb_t h, int32_t index);

/* Layout conversion, device to device.  rndr = [r_{k-1}][n_k][d_k][r_k], canonical = slice-major. */
int tt_emb_pack_core(tt_emb_t h, int32_t table, int32_t core, const float* rndr, float* canonical,
                     tt_emb_stream_t stream);
int tt_emb_unpack_core(tt_emb_t h, int32_t table, int32_t core, const float* canonical, float* rndr,
                       tt_emb_stream_t stream);

/* ---- measurement helpers (used by the benchmark to obtain roofline denominators) ---- */

/*
 * Device events: time of stage `stage` of the most recent call, in milliseconds, measured with CUDA
 * events recorded on the call's stream when timing is enabled.  SYNCHRONISES on the stage's end event.
 * Stages: 0 grouping, 1 schedule, 2 contraction, 3 pooling, 4 backward sort, 5 backward dE,
 * 6 backward contraction, 7 backward middle cores + reductions, 8 sgd; 9..20 the forward sweep kernel of shape
 * variant -1 (generic), 0..10; 21..32 the backward sweep kernel of the same variants (TT_EMB_ERR_STATE for a
 * variant no table uses).
 * on = 0: no events; 1: events, normal execution; 2: events, and kernels of different shape variants, which
 * normally run side by side on forked streams, run one after the other, so that a per-kernel duration is that
 * kernel's alone (the step is slower in this mode; it is for per-kernel figures, not for throughput).
 */
int tt_emb_enable_timing(tt_emb_t h, int32_t on);
int tt_emb_stage_ms(tt_emb_t h, int32_t stage, float* ms);

/* Independent-FMA-chain micro-benchmark: FP32 lane-instructions per second of the current device. SYNCHRONISES. */
int tt_emb_probe_fp32(double* slots_per_second, tt_emb_stream_t stream);
/*
 * Independent-chain micro-benchmark of the tensor path the contraction kernels use: warp-level
 * mma.sync.m16n8k8 TF32 instructions (1024 multiply-adds each) per second of the current device.  A product of the
 * path (Sec. 3.2: C = A.B, E = C.D) costs three of them per 1024 multiply-adds (3xTF32).  SYNCHRONISES.
 */
int tt_emb_probe_mma(double* mma_per_second, tt_emb_stream_t stream);
/*
 * The same question for the fifth-generation tensor cores: D[128 x n_cols] = A[128 x 32] . B[32 x n_cols] as
 * tcgen05.mma kind::tf32 instructions (M 128, N n_cols, k 8; operands in shared memory, accumulator in tensor
 * memory).  One product is checked against a plain FP32 loop on operands that are exact in TF32 (*max_abs_err, 0
 * when the instruction does what this file says), then one CTA per SM issues a long run of them
 * (*mma_per_second: M128.N.k8 instructions per second of the device = 128 * n_cols * 8 multiply-adds each).
 * n_cols must be 32 or 128 (TT_EMB_ERR_ARG otherwise): the widths of the middle-core products (Sec. 3.2, dB) and of
 * the stacked intermediate product (C = A.B).  Allocates two floats of device memory for its result.  SYNCHRONISES.
 */
int tt_emb_probe_tcgen05(int32_t n_cols, double* mma_per_second, double* max_abs_err, tt_emb_stream_t stream);
/*
 * Random 256-byte-row gather bandwidth (bytes/s) from a caller-provided DEVICE buffer of `bytes`
 * bytes (<= L2 size measures L2, >> L2 measures HBM).  scratch_idx: DEVICE int32[num_rows_read].  SYNCHRONISES.
 */
int tt_emb_probe_gather(const void* buffer, size_t bytes, int32_t* scratch_idx, int64_t num_rows_read,
                        double* bytes_per_second, tt_emb_stream_t stream);

/* Kernels launched by this thread's library calls since the last reset (counted at the launch sites). */
int tt_emb_launch_count(int64_t* count, int32_t reset);

const char* tt_emb_strerror(int code);
/* cudaError_t of the last failing CUDA call made by this thread's most recent library call (0 = none). */
int tt_emb_last_cuda_error(void);

#ifdef __cplusplus
}
#endif
#endif /* TT_EMB_H */
