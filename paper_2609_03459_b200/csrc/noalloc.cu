// Forward pass for callers that cannot allocate device memory.
//
// Who needs this: code that runs where cudaMalloc is forbidden or harmful -- inside a latency-critical serving
// loop whose memory pool is fixed at start-up, in a plug-in that is handed raw pointers by a host application
// and must not grow the process's footprint, or between the begin and end of a region in which the owner of the
// device has frozen allocation (allocating there can synchronise the whole device).  Such callers can pass their
// inputs, cores and the output buffer, but they have nowhere to get the library's workspace from.
//
// What it does: tt_emb_forward_static runs exactly the same kernels as tt_emb_bind + tt_emb_forward, with the
// workspace (scan partial sums, presence bitmap, prefix levels, row buffer, ...) placed in the fixed array below
// instead of caller memory.  It allocates nothing: no cudaMalloc/cudaFree, no allocating library routine.
//
// Limits and rules:
//   * the handle's workspace need (tt_emb_workspace_bytes) must not exceed TT_EMB_STATIC_WORKSPACE_BYTES (32 MiB);
//     larger configurations are rejected with TT_EMB_ERR_WORKSPACE before anything is launched;
//   * every GPU that loads the library holds those 32 MiB until the process exits;
//   * the first call on a device looks the array's device address up (once per device, with that device current),
//     and the first forward of a handle creates the handle's side streams and events and raises the shared-memory
//     limit of the kernels it uses (host-side driver objects and function attributes, no device memory); make those
//     first calls outside any stream capture;
//   * a call binds the handle to the array (a small upload of the table descriptors) unless the handle is already
//     bound to it with the same core pointers, in which case nothing but the forward itself is enqueued;
//   * all calls on a device share the one array and it keeps the previous call's contents; the forward clears
//     what must start at zero (status, counters, bitmap) itself.  Two calls whose GPU work overlaps -- different
//     streams, or different handles -- race on the array: serialise them;
//   * threads: the per-device address is published once with an atomic store, so concurrent first calls are safe;
//     the handle itself, as everywhere in this library, belongs to one thread at a time.
#include <atomic>

#include "common.cuh"

#define TT_EMB_STATIC_WORKSPACE_BYTES (32u << 20)
#define TT_MAX_DEVICES 64

// The scratch itself.  In host code this name is only a stand-in for the symbol, not a device address: it must go
// through cudaGetSymbolAddress before a kernel can be given it.
static __device__ __align__(256) unsigned char g_static_workspace[TT_EMB_STATIC_WORKSPACE_BYTES];

static std::atomic<void*> g_static_ptr[TT_MAX_DEVICES];  // device address of the array, per device (null = not looked up yet)

extern "C" int tt_emb_forward_static(tt_emb_t h, float* const* core_ptrs, const int64_t* indices, const int64_t* offsets,
                                     int64_t batch, int64_t num_lookups, float* out, tt_emb_stream_t stream)
{
    if (!h || !core_ptrs) return TT_EMB_ERR_ARG;
    size_t need = 0;
    int rc = tt_emb_workspace_bytes(h, &need);
    if (rc != TT_EMB_OK) return rc;
    if (need > (size_t)TT_EMB_STATIC_WORKSPACE_BYTES) return TT_EMB_ERR_WORKSPACE;  // configuration too large for the fixed array
    if (!tt_device_ok(nullptr)) return TT_EMB_ERR_ARCH;   // the array exists only in the sm_100a image
    int dev = -1;
    cudaError_t ce = cudaGetDevice(&dev);
    if (ce != cudaSuccess) { tt_set_last_cuda_error(ce); cudaGetLastError(); return TT_EMB_ERR_CUDA; }
    if (dev < 0 || dev >= TT_MAX_DEVICES) return TT_EMB_ERR_ARG;   // more devices than the per-device address table holds
    void* ws = g_static_ptr[dev].load(std::memory_order_acquire);
    if (!ws) {
        ce = cudaGetSymbolAddress(&ws, g_static_workspace);
        if (ce != cudaSuccess || !ws) { tt_set_last_cuda_error(ce); cudaGetLastError(); return TT_EMB_ERR_CUDA; }
        g_static_ptr[dev].store(ws, std::memory_order_release);
    }
    bool same = h->bound && h->ws_base == ws;
    for (int t = 0; same && t < h->T; ++t)
        for (int k = 0; k < h->K; ++k)
            if (h->tab[t].core[k] != core_ptrs[t * h->K + k]) { same = false; break; }
    if (!same) {
        rc = tt_emb_bind(h, core_ptrs, ws, (size_t)TT_EMB_STATIC_WORKSPACE_BYTES, stream);
        if (rc != TT_EMB_OK) return rc;
    }
    return tt_emb_forward(h, indices, offsets, batch, num_lookups, out, stream);
}

extern "C" size_t tt_emb_static_workspace_limit(void) { return (size_t)TT_EMB_STATIC_WORKSPACE_BYTES; }
