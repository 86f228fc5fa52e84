"""ctypes binding of libtt_emb.so: argument marshalling only, every step of the path runs in the CUDA library.

Two layers:
  * the raw C functions, under their C names (tt_emb_create, tt_emb_forward, ...), taking integers that are
    device or host addresses;
  * TTEmbeddingBag, a small convenience object that owns torch tensors for the cores / workspace / outputs
    and passes their data_ptr() and the current torch stream down.  torch is used for device memory and
    streams only.

There is no CPU fallback: if the shared library cannot be loaded, importing this module raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import List, Optional, Sequence

import numpy as np

from . import build as _build

_HERE = os.path.dirname(os.path.abspath(__file__))

STAGES = ["grouping", "schedule", "contraction", "pooling", "bwd_sort", "bwd_dE", "bwd_contraction",
          "bwd_middle", "sgd"] + [f"k_sweep_fwd<{v}>" for v in range(-1, 11)] + [f"k_sweep_bwd<{v}>" for v in range(-1, 11)]

TT_EMB_OK = 0
TT_EMB_ERR_ARG, TT_EMB_ERR_WORKSPACE, TT_EMB_ERR_ARCH, TT_EMB_ERR_STATE, TT_EMB_ERR_CUDA = -1, -2, -3, -4, -5
STATUS_INDEX, STATUS_OFFSETS, STATUS_OVERFLOW = 1, 2, 4


class tt_emb_config_t(ctypes.Structure):
    _fields_ = [
        ("num_tables", ctypes.c_int32),
        ("num_cores", ctypes.c_int32),
        ("num_rows", ctypes.c_void_p),
        ("row_factors", ctypes.c_void_p),
        ("dim_factors", ctypes.c_void_p),
        ("ranks", ctypes.c_void_p),
        ("max_batch", ctypes.c_int64),
        ("max_lookups", ctypes.c_int64),
        ("max_unique_rows", ctypes.c_int64),
        ("enable_backward", ctypes.c_int32),
        ("ablation", ctypes.c_int32),
        ("enable_weighted", ctypes.c_int32),
    ]


def _load() -> ctypes.CDLL:
    so = _build.SO
    if not os.path.exists(so):
        raise ImportError(f"{so} is missing: run `python -m paper_2609_03459_b200.build` (needs nvcc); "
                          "this package has no CPU fallback")
    return ctypes.CDLL(so)


lib = _load()

_vp, _i32, _i64, _f32 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_float
_SIGS = {
    "tt_emb_create": (ctypes.c_int, [ctypes.POINTER(tt_emb_config_t), ctypes.POINTER(_vp)]),
    "tt_emb_destroy": (ctypes.c_int, [_vp]),
    "tt_emb_workspace_bytes": (ctypes.c_int, [_vp, ctypes.POINTER(ctypes.c_size_t)]),
    "tt_emb_core_floats": (ctypes.c_int, [_vp, _i32, _i32, ctypes.POINTER(_i64)]),
    "tt_emb_dim": (ctypes.c_int, [_vp, ctypes.POINTER(_i32)]),
    "tt_emb_bind": (ctypes.c_int, [_vp, _vp, _vp, ctypes.c_size_t, _vp]),
    "tt_emb_forward": (ctypes.c_int, [_vp, _vp, _vp, _i64, _i64, _vp, _vp]),
    "tt_emb_forward_i32": (ctypes.c_int, [_vp, _vp, _vp, _i64, _i64, _vp, _vp]),
    "tt_emb_forward_static": (ctypes.c_int, [_vp, _vp, _vp, _vp, _i64, _i64, _vp, _vp]),
    "tt_emb_static_workspace_limit": (ctypes.c_size_t, []),
    "tt_emb_backward": (ctypes.c_int, [_vp, _vp, _vp, _vp]),
    "tt_emb_sgd_step": (ctypes.c_int, [_vp, _vp, _f32, _vp]),
    "tt_emb_backward_sgd": (ctypes.c_int, [_vp, _vp, _vp, _f32, _vp]),
    "tt_emb_status": (ctypes.c_int, [_vp, ctypes.POINTER(_i32), _vp]),
    "tt_emb_grouping_counts": (ctypes.c_int, [_vp, _vp, _vp]),
    "tt_emb_export_level": (ctypes.c_int, [_vp, _i32, _i32, _vp, _vp, _vp, _vp]),
    "tt_emb_export_inverse": (ctypes.c_int, [_vp, _i32, _vp, _vp]),
    "tt_emb_pack_core": (ctypes.c_int, [_vp, _i32, _i32, _vp, _vp, _vp]),
    "tt_emb_unpack_core": (ctypes.c_int, [_vp, _i32, _i32, _vp, _vp, _vp]),
    "tt_emb_set_pooling": (ctypes.c_int, [_vp, _i32, _vp]),
    "tt_emb_enable_timing": (ctypes.c_int, [_vp, _i32]),
    "tt_emb_stage_ms": (ctypes.c_int, [_vp, _i32, ctypes.POINTER(_f32)]),
    "tt_emb_probe_fp32": (ctypes.c_int, [ctypes.POINTER(ctypes.c_double), _vp]),
    "tt_emb_probe_mma": (ctypes.c_int, [ctypes.POINTER(ctypes.c_double), _vp]),
    "tt_emb_probe_tcgen05": (ctypes.c_int, [ctypes.c_int32, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double), _vp]),
    "tt_emb_probe_gather": (ctypes.c_int, [_vp, ctypes.c_size_t, _vp, _i64, ctypes.POINTER(ctypes.c_double), _vp]),
    "tt_emb_launch_count": (ctypes.c_int, [ctypes.POINTER(_i64), _i32]),
    "tt_emb_table_variant": (ctypes.c_int, [_vp, _i32, ctypes.POINTER(_i32)]),
    "tt_emb_check_guards": (ctypes.c_int, [_vp, ctypes.POINTER(_i32), _vp]),
    "tt_emb_region_name": (ctypes.c_char_p, [_vp, _i32]),
    "tt_emb_strerror": (ctypes.c_char_p, [ctypes.c_int]),
    "tt_emb_last_cuda_error": (ctypes.c_int, []),
}
for _name, (_res, _args) in _SIGS.items():
    _fn = getattr(lib, _name)
    _fn.restype = _res
    _fn.argtypes = _args
    globals()[_name] = _fn

EXPORTED_SYMBOLS = sorted(_SIGS)


class TTEmbError(RuntimeError):
    def __init__(self, code: int, where: str):
        msg = lib.tt_emb_strerror(code).decode()
        if code == TT_EMB_ERR_CUDA:
            msg += f" [cudaError {lib.tt_emb_last_cuda_error()}]"
        super().__init__(f"{where}: {msg} ({code})")
        self.code = code


def _check(code: int, where: str):
    if code != TT_EMB_OK:
        raise TTEmbError(code, where)


def make_config(num_rows: Sequence[int], row_factors: Sequence[Sequence[int]], dim_factors: Sequence[Sequence[int]],
                ranks: Sequence[Sequence[int]], max_batch: int, max_lookups: int, max_unique_rows: int = 0,
                enable_backward: bool = False, ablation: int = 0, enable_weighted: bool = False):
    """Returns (tt_emb_config_t, keepalive list of numpy arrays)."""
    T = len(num_rows)
    K = len(row_factors[0])
    nr = np.ascontiguousarray(np.asarray(num_rows, dtype=np.int64))
    rf = np.ascontiguousarray(np.asarray(row_factors, dtype=np.int32).reshape(T * K))
    df = np.ascontiguousarray(np.asarray(dim_factors, dtype=np.int32).reshape(T * K))
    rk = np.ascontiguousarray(np.asarray(ranks, dtype=np.int32).reshape(T * (K + 1)))
    cfg = tt_emb_config_t(T, K, nr.ctypes.data, rf.ctypes.data, df.ctypes.data, rk.ctypes.data,
                          int(max_batch), int(max_lookups), int(max_unique_rows), 1 if enable_backward else 0, int(ablation),
                          1 if enable_weighted else 0)
    return cfg, [nr, rf, df, rk]


def _stream_ptr(stream=None) -> int:
    import torch
    s = torch.cuda.current_stream() if stream is None else stream
    return int(s.cuda_stream)


class TTEmbeddingBag:
    """T TT-compressed tables behind one handle.  Cores are given in index order [r_{k-1}, n_k, d_k, r_k]
    (numpy or torch, fp32) and converted on the device to the library's slice-major layout."""

    def __init__(self, num_rows, row_factors, dim_factors, ranks, max_batch, max_lookups, *,
                 max_unique_rows: int = 0, enable_backward: bool = False, ablation: int = 0,
                 enable_weighted: bool = False, device="cuda:0"):
        import torch
        self.torch = torch
        self.device = torch.device(device)
        self.T, self.K = len(num_rows), len(row_factors[0])
        self.shapes = [[(ranks[t][k], row_factors[t][k], dim_factors[t][k], ranks[t][k + 1]) for k in range(self.K)]
                       for t in range(self.T)]
        self.enable_backward = enable_backward
        cfg, keep = make_config(num_rows, row_factors, dim_factors, ranks, max_batch, max_lookups,
                                max_unique_rows, enable_backward, ablation, enable_weighted)
        h = ctypes.c_void_p()
        _check(lib.tt_emb_create(ctypes.byref(cfg), ctypes.byref(h)), "tt_emb_create")
        self.h = h
        d = ctypes.c_int32()
        _check(lib.tt_emb_dim(self.h, ctypes.byref(d)), "tt_emb_dim")
        self.D = int(d.value)
        nbytes = ctypes.c_size_t()
        _check(lib.tt_emb_workspace_bytes(self.h, ctypes.byref(nbytes)), "tt_emb_workspace_bytes")
        self.workspace_bytes = int(nbytes.value)
        self.workspace = None
        self.cores: List[List] = []
        self.grads: Optional[List[List]] = None

    def __del__(self):
        h = getattr(self, "h", None)
        if h and lib is not None:   # at interpreter shutdown the module globals may already be gone
            lib.tt_emb_destroy(h)
            self.h = None

    # ---- set-up
    def set_cores(self, cores):
        """cores[t][k]: fp32 array of shape (r_{k-1}, n_k, d_k, r_k).  Packs to slice-major and binds.
        All cores live in one flat device buffer (self.flat_cores), all gradients in another
        (self.flat_grads), so a multi-GPU job can all-reduce the gradients with a single collective."""
        torch = self.torch
        with torch.cuda.device(self.device):
            s = _stream_ptr()
            sizes = [int(np.prod(self.shapes[t][k])) for t in range(self.T) for k in range(self.K)]
            offs, tot = [], 0
            for n in sizes:
                offs.append(tot)
                tot += (n + 3) // 4 * 4  # keep every core 16-byte aligned
            self.flat_cores = torch.empty(max(tot, 4), dtype=torch.float32, device=self.device)
            self.cores = []
            i = 0
            for t in range(self.T):
                row = []
                for k in range(self.K):
                    src = cores[t][k]
                    if not torch.is_tensor(src):
                        src = torch.from_numpy(np.ascontiguousarray(src, dtype=np.float32))
                    src = src.to(self.device, dtype=torch.float32).contiguous()
                    assert tuple(src.shape) == tuple(self.shapes[t][k]), (t, k, src.shape, self.shapes[t][k])
                    dst = self.flat_cores[offs[i]:offs[i] + sizes[i]]
                    _check(lib.tt_emb_pack_core(self.h, t, k, src.data_ptr(), dst.data_ptr(), s), "tt_emb_pack_core")
                    row.append(dst)
                    i += 1
                self.cores.append(row)
            torch.cuda.current_stream().synchronize()
            if self.workspace is None:
                self.workspace = torch.empty(self.workspace_bytes + 256, dtype=torch.uint8, device=self.device)
            base = (self.workspace.data_ptr() + 255) // 256 * 256
            ptrs = (ctypes.c_void_p * (self.T * self.K))(*[c.data_ptr() for row in self.cores for c in row])
            _check(lib.tt_emb_bind(self.h, ptrs, base, self.workspace_bytes, s), "tt_emb_bind")
            if self.enable_backward:
                self.flat_grads = torch.zeros_like(self.flat_cores)
                self.grads, i = [], 0
                for t in range(self.T):
                    row = []
                    for k in range(self.K):
                        row.append(self.flat_grads[offs[i]:offs[i] + sizes[i]])
                        i += 1
                    self.grads.append(row)

    def get_cores(self):
        """Cores back in index order [r_{k-1}, n_k, d_k, r_k] as numpy fp32."""
        return self._unpack(self.cores)

    def get_grads(self):
        return self._unpack(self.grads)

    def _unpack(self, tensors):
        torch = self.torch
        out = []
        with torch.cuda.device(self.device):
            s = _stream_ptr()
            for t in range(self.T):
                row = []
                for k in range(self.K):
                    dst = torch.empty(self.shapes[t][k], dtype=torch.float32, device=self.device)
                    _check(lib.tt_emb_unpack_core(self.h, t, k, tensors[t][k].data_ptr(), dst.data_ptr(), s),
                           "tt_emb_unpack_core")
                    row.append(dst)
                torch.cuda.current_stream().synchronize()
                out.append([x.cpu().numpy() for x in row])
        return out

    # ---- hot path
    def forward(self, indices, offsets, batch: int, out=None):
        """indices int64[L] (or int32[L]) / offsets int64[T*batch+1] device tensors -> out fp32 [batch, T*D] (device)."""
        torch = self.torch
        assert indices.dtype in (torch.int64, torch.int32) and offsets.dtype == torch.int64
        assert indices.is_cuda and offsets.is_cuda
        if out is None:
            out = torch.empty((batch, self.T * self.D), dtype=torch.float32, device=self.device)
        self._keep = (indices, offsets)
        fn = lib.tt_emb_forward if indices.dtype == torch.int64 else lib.tt_emb_forward_i32   # 32-bit row ids
        _check(fn(self.h, indices.data_ptr(), offsets.data_ptr(), int(batch), int(indices.numel()),
                  out.data_ptr(), _stream_ptr()), "tt_emb_forward")
        return out

    def capture_forward(self, indices, offsets, batch: int, out):
        """CUDA graph of one forward on fixed buffers (same batch and number of lookups at every replay; the CONTENTS
        of `indices` / `offsets` may change between replays: grouping, schedule and all counts are computed on the
        device).  For launch-latency-bound small batches: replaying the graph saves the per-kernel launch cost of
        the ~25 small kernels of a forward.  Returns a torch.cuda.CUDAGraph; call .replay()."""
        torch = self.torch
        self.forward(indices, offsets, batch, out=out)      # first call outside the capture: creates streams, sets attributes
        torch.cuda.synchronize()
        g = torch.cuda.CUDAGraph()
        with torch.cuda.graph(g):
            self.forward(indices, offsets, batch, out=out)
        return g

    def set_pooling(self, mode: str = "sum", per_sample_weights=None):
        """Pooling of the following forward/backward calls: "sum" (default), "mean", or "sum" with per-lookup
        weights (fp32 device tensor [L]).  Needs enable_weighted=True unless plain sum is selected."""
        torch = self.torch
        if per_sample_weights is not None:
            assert per_sample_weights.dtype == torch.float32 and per_sample_weights.is_cuda and per_sample_weights.is_contiguous()
        self._keep_w = per_sample_weights
        _check(lib.tt_emb_set_pooling(self.h, {"sum": 0, "mean": 1}[mode],
                                      None if per_sample_weights is None else per_sample_weights.data_ptr()),
               "tt_emb_set_pooling")

    def forward_static(self, indices, offsets, batch: int, out=None):
        """Forward through the library's built-in 32 MiB workspace: for callers that must not allocate device
        memory.  Only for configurations whose workspace fits (TTEmbError with ERR_WORKSPACE otherwise).  Calls
        must not overlap on the GPU; the handle stays bound to the built-in workspace afterwards."""
        torch = self.torch
        assert indices.dtype == torch.int64 and offsets.dtype == torch.int64 and indices.is_cuda and offsets.is_cuda
        if out is None:
            out = torch.empty((batch, self.T * self.D), dtype=torch.float32, device=self.device)
        self._keep = (indices, offsets)
        ptrs = (ctypes.c_void_p * (self.T * self.K))(*[c.data_ptr() for row in self.cores for c in row])
        _check(lib.tt_emb_forward_static(self.h, ptrs, indices.data_ptr(), offsets.data_ptr(), int(batch),
                                         int(indices.numel()), out.data_ptr(), _stream_ptr()), "tt_emb_forward_static")
        return out

    def backward(self, grad_out):
        torch = self.torch
        assert grad_out.dtype == torch.float32 and grad_out.is_cuda and grad_out.is_contiguous()
        ptrs = (ctypes.c_void_p * (self.T * self.K))(*[g.data_ptr() for row in self.grads for g in row])
        _check(lib.tt_emb_backward(self.h, grad_out.data_ptr(), ptrs, _stream_ptr()), "tt_emb_backward")
        return self.grads

    def backward_sgd(self, grad_out, lr: float):
        """Backward and SGD update in one call, the update fused into the kernels that finalise each gradient."""
        torch = self.torch
        assert grad_out.dtype == torch.float32 and grad_out.is_cuda and grad_out.is_contiguous()
        ptrs = (ctypes.c_void_p * (self.T * self.K))(*[g.data_ptr() for row in self.grads for g in row])
        _check(lib.tt_emb_backward_sgd(self.h, grad_out.data_ptr(), ptrs, float(lr), _stream_ptr()), "tt_emb_backward_sgd")
        return self.grads

    def sgd_step(self, lr: float):
        ptrs = (ctypes.c_void_p * (self.T * self.K))(*[g.data_ptr() for row in self.grads for g in row])
        _check(lib.tt_emb_sgd_step(self.h, ptrs, float(lr), _stream_ptr()), "tt_emb_sgd_step")

    def forward_host(self, indices_pinned, offsets_pinned, batch: int, out_pinned=None):
        """End-to-end call with HOST buffers: copies inputs to the device, runs forward, copies `out` back."""
        torch = self.torch
        idx = indices_pinned.to(self.device, non_blocking=True)
        off = offsets_pinned.to(self.device, non_blocking=True)
        out = self.forward(idx, off, batch)
        if out_pinned is None:
            return out.cpu()
        out_pinned.copy_(out, non_blocking=True)
        torch.cuda.current_stream().synchronize()
        return out_pinned

    # ---- inspection
    def status(self) -> int:
        st = ctypes.c_int32()
        _check(lib.tt_emb_status(self.h, ctypes.byref(st), _stream_ptr()), "tt_emb_status")
        return int(st.value)

    def grouping_counts(self) -> np.ndarray:
        c = np.zeros(self.T * self.K, dtype=np.int64)
        _check(lib.tt_emb_grouping_counts(self.h, c.ctypes.data, _stream_ptr()), "tt_emb_grouping_counts")
        return c.reshape(self.T, self.K)

    def export_level(self, table: int, level: int, count: int, with_lookup_counts: bool = True):
        torch = self.torch
        vals = torch.empty(count, dtype=torch.int64, device=self.device)
        rc = torch.empty(count, dtype=torch.int32, device=self.device)
        lc = torch.empty(count, dtype=torch.int32, device=self.device) if with_lookup_counts else None
        _check(lib.tt_emb_export_level(self.h, table, level, vals.data_ptr(), rc.data_ptr(),
                                       lc.data_ptr() if lc is not None else None, _stream_ptr()), "tt_emb_export_level")
        return vals.cpu().numpy(), rc.cpu().numpy(), (lc.cpu().numpy() if lc is not None else None)

    def export_inverse(self, table: int, num_lookups: int) -> np.ndarray:
        torch = self.torch
        inv = torch.empty(max(num_lookups, 1), dtype=torch.int32, device=self.device)
        _check(lib.tt_emb_export_inverse(self.h, table, inv.data_ptr(), _stream_ptr()), "tt_emb_export_inverse")
        return inv.cpu().numpy()[:num_lookups]

    def table_variant(self, table: int) -> int:
        """Register-tiled sweep kernel variant of a table (-1: generic path)."""
        v = ctypes.c_int32()
        _check(lib.tt_emb_table_variant(self.h, table, ctypes.byref(v)), "tt_emb_table_variant")
        return int(v.value)

    def check_guards(self):
        """None if the guard bytes behind every workspace region are intact, else the name of the first damaged region."""
        bad = ctypes.c_int32()
        _check(lib.tt_emb_check_guards(self.h, ctypes.byref(bad), _stream_ptr()), "tt_emb_check_guards")
        return None if bad.value < 0 else lib.tt_emb_region_name(self.h, bad.value).decode()

    def enable_timing(self, on=True):
        """False/0: off; True/1: stage events; 2: stage events with the shape-variant kernels serialised."""
        _check(lib.tt_emb_enable_timing(self.h, int(on)), "tt_emb_enable_timing")

    def stage_ms(self) -> dict:
        res = {}
        for i, name in enumerate(STAGES):
            ms = ctypes.c_float()
            if lib.tt_emb_stage_ms(self.h, i, ctypes.byref(ms)) == TT_EMB_OK:
                res[name] = float(ms.value)
        return res


def from_workload(wl, *, enable_backward: bool = False, max_unique_rows: int = 0, ablation: int = 0,
                  enable_weighted: bool = False, device="cuda:0") -> TTEmbeddingBag:
    """Build a TTEmbeddingBag for a workloads.Workload-like object (tables with N, n, d, r; B; L; cores)."""
    emb = TTEmbeddingBag([s.N for s in wl.tables], [s.n for s in wl.tables], [s.d for s in wl.tables],
                         [s.r for s in wl.tables], wl.B, max(wl.L, 1), max_unique_rows=max_unique_rows,
                         enable_backward=enable_backward, ablation=ablation, enable_weighted=enable_weighted, device=device)
    emb.set_cores(wl.cores)
    return emb


def launch_count(reset: bool = False) -> int:
    v = ctypes.c_int64()
    _check(lib.tt_emb_launch_count(ctypes.byref(v), 1 if reset else 0), "tt_emb_launch_count")
    return int(v.value)


def probe_fp32() -> float:
    v = ctypes.c_double()
    _check(lib.tt_emb_probe_fp32(ctypes.byref(v), _stream_ptr()), "tt_emb_probe_fp32")
    return float(v.value)


def probe_mma() -> float:
    v = ctypes.c_double()
    _check(lib.tt_emb_probe_mma(ctypes.byref(v), _stream_ptr()), "tt_emb_probe_mma")
    return float(v.value)


def probe_tcgen05(n_cols: int):
    """(M128.N.k8 tcgen05 TF32 instructions per second, max |error| of the checked product)."""
    rate, err = ctypes.c_double(), ctypes.c_double()
    _check(lib.tt_emb_probe_tcgen05(int(n_cols), ctypes.byref(rate), ctypes.byref(err), _stream_ptr()), "tt_emb_probe_tcgen05")
    return float(rate.value), float(err.value)


def probe_gather(nbytes: int, rows_read: int = 1 << 22, device="cuda:0") -> float:
    import torch
    buf = torch.zeros(nbytes // 4, dtype=torch.float32, device=device)
    idx = torch.empty(rows_read, dtype=torch.int32, device=device)
    v = ctypes.c_double()
    _check(lib.tt_emb_probe_gather(buf.data_ptr(), nbytes, idx.data_ptr(), rows_read, ctypes.byref(v), _stream_ptr()),
           "tt_emb_probe_gather")
    return float(v.value)
