"""Parity at the benchmark's full sizes, in the launch configuration bench.py times: EVERY element of `out`,
of every core gradient and of every core after the SGD step is compared with the fp64 oracle.

  * configs 1, 2, 4 (single table): the plain per-lookup oracle redoes the whole batch (seconds), and the
    memoised oracle must agree with it on the same full inputs;
  * configs 3 and 5 (60 tables, 99 million lookups; identity and scattered rank -> row mapping): the memoised
    oracle (every distinct row built once, grad_out summed per distinct row in fp64; pinned against the plain
    oracle by the CPU tests, among them a 1/64 sub-sample of this very batch);
  * grouping: distinct-row / prefix counts of every table against numpy sets, sampled tables in full.
Tolerance: max|err| <= 1e-5 * max|ref| per compared tensor (per table block of `out`, per core gradient, per core)."""
import numpy as np
import pytest

import oracle
import workloads

pytestmark = pytest.mark.gpu
TOL = 1e-5


@pytest.fixture(scope="module")
def binding():
    import torch
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    import __graft_entry__ as entry
    entry.build()
    from paper_2609_03459_b200 import binding as b
    return b


def dev(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def close(got, ref, what):
    ref = np.asarray(ref, np.float64); got = np.asarray(got, np.float64)
    scale = np.abs(ref).max()
    err = np.abs(got - ref).max()
    assert err <= TOL * max(scale, 1e-300), f"{what}: max|err| {err:.3e} vs 1e-5 * {scale:.3e}"
    return err / max(scale, 1e-300)


def check_counts(emb, wl, full_tables=()):
    counts = emb.grouping_counts()
    for t, s in enumerate(wl.tables):
        idx, _ = wl.table_slice(t)
        uniq = np.unique(idx)
        assert counts[t, s.K - 1] == uniq.shape[0]
        suffix = 1
        for k in range(s.K - 1, 0, -1):
            suffix *= s.n[k]
            assert counts[t, k - 1] == np.unique(uniq // suffix).shape[0]
    for t in full_tables:
        s = wl.tables[t]
        idx, _ = wl.table_slice(t)
        g = oracle.grouping(s.n, idx)
        vals, rc, _ = emb.export_level(t, s.K, int(counts[t, s.K - 1]), with_lookup_counts=False)
        np.testing.assert_array_equal(vals, g["uniq"])
        for k in range(1, s.K):
            vals, rc, _ = emb.export_level(t, k, int(counts[t, k - 1]), with_lookup_counts=False)
            np.testing.assert_array_equal(vals, g["levels"][k - 1]["vals"])
            np.testing.assert_array_equal(rc, g["levels"][k - 1]["row_counts"])
        np.testing.assert_array_equal(emb.export_inverse(t, idx.shape[0]), g["inv"])


def check_out_all(wl, out, ref, what):
    """Every pooled output, table block by table block (the scale of a block is its own largest reference value)."""
    worst = 0.0
    D = wl.D
    for t in range(wl.T):
        worst = max(worst, close(out[:, t * D:(t + 1) * D], ref[:, t * D:(t + 1) * D], f"{what} out, table {t}"))
    return worst


def check_training_all(wl, emb, ref_grads, what):
    """Every gradient entry and every core entry after the update, tensor by tensor."""
    grads = emb.get_grads()
    cores = emb.get_cores()
    worst = 0.0
    for t in range(wl.T):
        want = oracle.sgd(wl.cores[t], ref_grads[t], wl.lr)
        for k in range(wl.tables[t].K):
            worst = max(worst, close(grads[t][k], ref_grads[t][k], f"{what} grad[{t}][{k}]"))
            close(cores[t][k], want[k], f"{what} core[{t}][{k}] after SGD")
    # slices of padding digits (never looked up) must have exactly zero gradient and unchanged cores
    for t in range(wl.T):
        s = wl.tables[t]
        rest = int(np.prod(s.n[1:]))
        last_i1 = (s.N - 1) // rest
        if last_i1 + 1 < s.n[0]:
            assert np.count_nonzero(grads[t][0][:, last_i1 + 1:]) == 0
            np.testing.assert_array_equal(cores[t][0][:, last_i1 + 1:], wl.cores[t][0][:, last_i1 + 1:])
    return worst


def test_config1_full(binding):
    wl = workloads.make(1)
    emb = binding.from_workload(wl)
    out = emb.forward(dev(wl.indices), dev(wl.offsets), wl.B).cpu().numpy()
    assert emb.status() == 0
    close(out, oracle.forward_workload(wl), "cfg1 out (all bags)")
    check_counts(emb, wl, full_tables=(0,))


@pytest.mark.parametrize("cfg", [2, 4])
@pytest.mark.parametrize("mapping", ["identity", "scattered"])
def test_single_table_configs_full(binding, cfg, mapping):
    wl = workloads.make(cfg, mapping=mapping)
    emb = binding.from_workload(wl)
    out = emb.forward(dev(wl.indices), dev(wl.offsets), wl.B).cpu().numpy()
    assert emb.status() == 0
    ref = oracle.forward_workload(wl)                    # the plain per-lookup oracle over the whole batch
    close(out, ref, f"cfg{cfg} {mapping} out (all bags)")
    memo = oracle.forward_workload(wl, memo=True)        # the two oracles agree on the full inputs as well
    np.testing.assert_allclose(memo, ref, rtol=1e-11, atol=1e-13 * np.abs(ref).max())
    check_counts(emb, wl, full_tables=(0,))


class _Full:
    """The 60-table training workload of one mapping with its oracle results (memoised oracle, fp64)."""
    def __init__(self, mapping):
        self.wl = workloads.make(5, mapping=mapping)
        self.ref_out = oracle.forward_workload(self.wl, memo=True)
        self.ref_grads = oracle.backward_workload(self.wl, memo=True)


@pytest.fixture(scope="module", params=["identity", "scattered"])
def full(request):
    f = _Full(request.param)
    yield f
    del f


def test_config3_forward_every_output(binding, full):
    wl = full.wl
    emb = binding.from_workload(wl)                       # forward-only handle: the launch configuration of config 3
    out = emb.forward(dev(wl.indices), dev(wl.offsets), wl.B).cpu().numpy()
    assert emb.status() == 0
    check_out_all(wl, out, full.ref_out, f"cfg3 {wl.mapping}")
    check_counts(emb, wl, full_tables=(0, 17))
    del emb


def test_config5_training_step_every_gradient_and_core(binding, full):
    wl = full.wl
    emb = binding.from_workload(wl, enable_backward=True)
    out = emb.forward(dev(wl.indices), dev(wl.offsets), wl.B)
    emb.backward_sgd(dev(wl.grad_out), wl.lr)     # the call the benchmark's training step makes
    assert emb.status() == 0
    check_out_all(wl, out.cpu().numpy(), full.ref_out, f"cfg5 {wl.mapping}")
    del out
    check_training_all(wl, emb, full.ref_grads, f"cfg5 {wl.mapping}")
    del emb


def test_config5_separate_backward_and_update_every_gradient_and_core(binding, full):
    # the three calls of the multi-GPU step (backward, [all-reduce], sgd_step) instead of the fused one
    wl = full.wl
    if wl.mapping != "identity":
        pytest.skip("one mapping is enough for the unfused call sequence")
    emb = binding.from_workload(wl, enable_backward=True)
    emb.forward(dev(wl.indices), dev(wl.offsets), wl.B)
    emb.backward(dev(wl.grad_out))
    emb.sgd_step(wl.lr)
    assert emb.status() == 0
    check_training_all(wl, emb, full.ref_grads, "cfg5 unfused")
    del emb


def test_many_tables_training_step_every_output_gradient_and_core(binding):
    # the many-tables bench workload at full size (240 tables, D = 32, ranks 32, every table with its own bag lengths:
    # the short-bag pooling kernel, the transposed row products and the stacked backward products), in the launch
    # configuration bench.py times, against the memoised oracle
    wl = workloads.many_tables_point(32768)
    ref_out = oracle.forward_workload(wl, memo=True)
    ref_grads = oracle.backward_workload(wl, memo=True)
    emb = binding.from_workload(wl, enable_backward=True, max_unique_rows=wl.L // 2)
    out = emb.forward(dev(wl.indices), dev(wl.offsets), wl.B)
    emb.backward_sgd(dev(wl.grad_out), wl.lr)
    assert emb.status() == 0
    check_out_all(wl, out.cpu().numpy(), ref_out, "many-tables")
    del out
    check_training_all(wl, emb, ref_grads, "many-tables")
    del emb
