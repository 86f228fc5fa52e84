"""The allocation-free forward (tt_emb_forward_static) against the ordinary bind + forward.

Some users of the library cannot allocate device memory at call time (fixed memory pools in serving loops,
plug-ins that only get raw pointers, allocation-frozen regions), so one entry point keeps its workspace in a fixed
array inside the library.  This test calls it through the C ABI twice in a row -- the array keeps the first
call's contents, so the second call also checks that everything that must start at zero is cleared -- and compares
with the existing entry point.  It is collected last so that a run that stops at the first failure has already
run every other test; it also passes when run alone in a fresh process."""
import ctypes

import numpy as np
import pytest

import oracle
import workloads
from workloads import TableSpec

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def binding():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import __graft_entry__ as entry
    entry.build()
    from paper_2609_03459_b200 import binding as b
    return b


def _dev(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def test_static_workspace_forward_matches_regular_forward_twice(binding):
    import torch
    tables = [TableSpec(30_000, (32, 32, 32), (4, 4, 4), (1, 32, 32, 1), 1.1, "normal", 0.05),
              TableSpec(9_000, (21, 21, 21), (4, 4, 4), (1, 16, 32, 1), 0.9, "normal", 0.05),
              TableSpec(700, (9, 9, 9), (4, 4, 4), (1, 5, 7, 1), 1.0, "normal", 0.05)]
    wl_a = workloads.custom(tables, 200, (0, 25), seed=11)
    wl_b = workloads.custom(tables, 200, (0, 25), seed=12)
    wl_b.cores = wl_a.cores
    emb = binding.from_workload(wl_a)                      # regular path: caller-provided workspace
    assert emb.workspace_bytes <= binding.lib.tt_emb_static_workspace_limit()
    ref_a = emb.forward(_dev(wl_a.indices), _dev(wl_a.offsets), wl_a.B).cpu().numpy()
    emb_b = binding.from_workload(wl_b)
    ref_b = emb_b.forward(_dev(wl_b.indices), _dev(wl_b.offsets), wl_b.B).cpu().numpy()

    emb_s = binding.from_workload(wl_a if wl_a.L >= wl_b.L else wl_b)   # capacity for the larger batch
    out1 = emb_s.forward_static(_dev(wl_a.indices), _dev(wl_a.offsets), wl_a.B).cpu().numpy()
    out2 = emb_s.forward_static(_dev(wl_b.indices), _dev(wl_b.offsets), wl_b.B).cpu().numpy()   # second call, other batch
    out3 = emb_s.forward_static(_dev(wl_a.indices), _dev(wl_a.offsets), wl_a.B).cpu().numpy()   # and the first again
    torch.cuda.synchronize()
    assert emb_s.status() == 0
    for got, ref, what in ((out1, ref_a, "first call"), (out2, ref_b, "second call"), (out3, ref_a, "third call")):
        err = np.abs(got.astype(np.float64) - ref.astype(np.float64)).max()
        assert err <= 1e-5 * np.abs(ref).max(), (what, err)
    # and against the fp64 oracle, like every other forward
    for got, wl, what in ((out1, wl_a, "first call"), (out2, wl_b, "second call"), (out3, wl_a, "third call")):
        want = oracle.forward_workload(wl)
        assert np.abs(got - want).max() <= 1e-5 * np.abs(want).max(), (what, "vs oracle")
    assert emb_s.check_guards() is None


def test_static_workspace_rejects_configurations_that_do_not_fit(binding):
    spec = TableSpec(10_000_000, (200, 250, 200), (4, 8, 4), (1, 32, 32, 1), 1.1, "normal", 0.05)
    cfg, keep = binding.make_config([spec.N], [spec.n], [spec.d], [spec.r], 32768, 655360)
    h = ctypes.c_void_p()
    assert binding.lib.tt_emb_create(ctypes.byref(cfg), ctypes.byref(h)) == 0
    need = ctypes.c_size_t()
    binding.lib.tt_emb_workspace_bytes(h, ctypes.byref(need))
    assert need.value > binding.lib.tt_emb_static_workspace_limit()
    ptrs = (ctypes.c_void_p * 3)(256, 512, 768)
    rc = binding.lib.tt_emb_forward_static(h, ptrs, 256, 256, 1, 1, 256, None)
    assert rc == binding.TT_EMB_ERR_WORKSPACE
    assert b"workspace" in binding.lib.tt_emb_strerror(rc)
    binding.lib.tt_emb_destroy(h)
