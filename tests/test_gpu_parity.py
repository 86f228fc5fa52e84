"""Parity of the CUDA path (through the C ABI) against the fp64 CPU oracle, on the same seeded inputs.

Bar: integers (distinct rows, prefix groups, counts, inverse map) bit-exact after canonical ordering;
fp32 tensors within max|err| <= 1e-5 * max|ref|, per output tensor."""
import numpy as np
import pytest

import oracle
import workloads
from workloads import TableSpec

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


def assert_close(got, ref, what):
    ref = np.asarray(ref, dtype=np.float64)
    got = np.asarray(got, dtype=np.float64)
    assert got.shape == ref.shape, (what, got.shape, ref.shape)
    scale = np.abs(ref).max() if ref.size else 0.0
    err = np.abs(got - ref).max() if ref.size else 0.0
    if scale == 0.0:
        assert err == 0.0, f"{what}: reference is all zero but max|got| = {err}"
    else:
        assert err <= TOL * scale, f"{what}: max|err| = {err:.3e} > 1e-5 * {scale:.3e}"


def run_forward(binding, wl, **kw):
    emb = binding.from_workload(wl, **kw)
    out = emb.forward(dev(wl.indices), dev(wl.offsets), wl.B)
    return emb, out.cpu().numpy()


def check_grouping(emb, wl):
    counts = emb.grouping_counts()
    for t, s in enumerate(wl.tables):
        idx, _ = wl.table_slice(t)
        g = oracle.grouping(s.n, idx)
        K = s.K
        assert counts[t, K - 1] == g["uniq"].shape[0], (t, counts[t], g["uniq"].shape)
        vals, rc, lc = emb.export_level(t, K, int(counts[t, K - 1]), with_lookup_counts=emb.enable_backward)
        np.testing.assert_array_equal(vals, g["uniq"])
        np.testing.assert_array_equal(rc, np.ones_like(rc))
        if lc is not None:
            np.testing.assert_array_equal(lc, g["mult"])
        for k in range(1, K):
            lev = g["levels"][k - 1]
            assert counts[t, k - 1] == lev["vals"].shape[0]
            vals, rc, lc = emb.export_level(t, k, int(counts[t, k - 1]), with_lookup_counts=emb.enable_backward)
            np.testing.assert_array_equal(vals, lev["vals"])
            np.testing.assert_array_equal(rc, lev["row_counts"])
            if lc is not None:
                np.testing.assert_array_equal(lc, lev["lookup_counts"])
        inv = emb.export_inverse(t, idx.shape[0])
        np.testing.assert_array_equal(inv, g["inv"])


# ------------------------------------------------------------------------------------------ tiny forms of the five configs

@pytest.mark.parametrize("cfg", [1, 2, 3, 4, 5])
@pytest.mark.parametrize("mapping", ["identity", "scattered"])
def test_tiny_configs_forward_and_grouping(binding, cfg, mapping):
    wl = workloads.make(cfg, tiny=True, mapping=mapping)
    emb, out = run_forward(binding, wl, enable_backward=True)
    assert emb.status() == 0
    assert_close(out, oracle.forward_workload(wl), f"cfg{cfg}-tiny out")
    check_grouping(emb, wl)


@pytest.mark.parametrize("cfg", [1, 2, 3, 4, 5])
def test_tiny_configs_backward_and_sgd(binding, cfg):
    wl = workloads.make(cfg, tiny=True)
    rng = np.random.default_rng(cfg)
    go = wl.grad_out if wl.grad_out is not None else rng.standard_normal((wl.B, wl.T * wl.D)).astype(np.float32)
    emb, out = run_forward(binding, wl, enable_backward=True)
    emb.backward(dev(go))
    grads = emb.get_grads()
    ref = oracle.backward_workload(wl, grad_out=go)
    for t in range(wl.T):
        for k in range(wl.tables[t].K):
            assert_close(grads[t][k], ref[t][k], f"cfg{cfg}-tiny dG[{t}][{k}]")
    emb.sgd_step(0.01)
    cores = emb.get_cores()
    for t in range(wl.T):
        want = oracle.sgd(wl.cores[t], ref[t], 0.01)
        for k in range(wl.tables[t].K):
            assert_close(cores[t][k], want[k], f"cfg{cfg}-tiny core[{t}][{k}] after SGD")
    assert emb.status() == 0


@pytest.mark.parametrize("cfg", [1, 2, 3, 4, 5])
def test_tiny_configs_fused_backward_sgd(binding, cfg):
    # backward and update in one call: gradients at the pre-update cores, cores after the step
    wl = workloads.make(cfg, tiny=True)
    rng = np.random.default_rng(cfg)
    go = wl.grad_out if wl.grad_out is not None else rng.standard_normal((wl.B, wl.T * wl.D)).astype(np.float32)
    emb, out = run_forward(binding, wl, enable_backward=True)
    emb.backward_sgd(dev(go), 0.01)
    grads = emb.get_grads()
    cores = emb.get_cores()
    ref = oracle.backward_workload(wl, grad_out=go)
    for t in range(wl.T):
        want = oracle.sgd(wl.cores[t], ref[t], 0.01)
        for k in range(wl.tables[t].K):
            assert_close(grads[t][k], ref[t][k], f"cfg{cfg}-tiny fused dG[{t}][{k}]")
            assert_close(cores[t][k], want[k], f"cfg{cfg}-tiny core[{t}][{k}] after the fused step")
    assert emb.status() == 0
    # the handle is back to the plain backward afterwards: cores stay as they are
    out2 = emb.forward(dev(wl.indices), dev(wl.offsets), wl.B)
    emb.backward(dev(go))
    after = emb.get_cores()
    for t in range(wl.T):
        for k in range(wl.tables[t].K):
            assert np.array_equal(after[t][k], cores[t][k]), "a plain backward after a fused one must not touch the cores"


# ------------------------------------------------------------------------------------------ medium cases: several tiles, ragged tails

MEDIUM = [
    # name, tables, B, pooling
    ("k3-mixed", [TableSpec(200_003, (59, 59, 59), (4, 4, 4), (1, 16, 32, 1), 1.05, "normal", 0.05),
                  TableSpec(1_500, (12, 12, 12), (4, 4, 4), (1, 32, 16, 1), 0.9, "normal", 0.05),
                  TableSpec(150_000, (54, 54, 54), (4, 4, 4), (1, 7, 5, 1), 1.2, "normal", 0.05)], 300, (0, 40)),
    # every register-tiled shape variant: (r1, r2) in {16,32}^2 and rank 8 with d = 4x4x4, the d = 4x8x4 rank-32
    # shape, and the 4-core rank-64 shape
    ("tiled-r16-r32", [TableSpec(30_000, (32, 32, 32), (4, 4, 4), (1, 32, 32, 1), 1.1, "normal", 0.05),
                       TableSpec(20_000, (28, 28, 28), (4, 4, 4), (1, 16, 16, 1), 0.9, "normal", 0.05),
                       TableSpec(25_000, (30, 30, 30), (4, 4, 4), (1, 16, 32, 1), 1.0, "normal", 0.05),
                       TableSpec(12_000, (23, 23, 23), (4, 4, 4), (1, 32, 16, 1), 1.2, "normal", 0.05),
                       TableSpec(8_000, (20, 20, 20), (4, 4, 4), (1, 8, 8, 1), 1.05, "uniform", 0.1),
                       # first ranks that are not multiples of 8: the stacked tensor-core product pads its k range
                       TableSpec(9_000, (21, 21, 21), (4, 4, 4), (1, 12, 32, 1), 1.0, "normal", 0.05),
                       TableSpec(7_000, (19, 20, 19), (4, 4, 4), (1, 21, 16, 1), 1.1, "normal", 0.05)], 150, (0, 30)),
    # long accumulation chains: groups with hundreds of rows (dC summed over a whole group) and middle-core slices
    # with hundreds of nodes; nearly uniform lookups so that most rows are present.  The tensor core adds into its
    # accumulator with truncation, which drifts by chain length * 2^-24 unless the chains are kept short.
    ("long-chains", [TableSpec(72_000, (6, 40, 300), (4, 4, 4), (1, 32, 32, 1), 0.2, "normal", 0.05),
                     TableSpec(64_000, (200, 8, 40), (4, 4, 4), (1, 16, 32, 1), 0.2, "normal", 0.05),
                     TableSpec(60_000, (5, 40, 300), (4, 4, 4), (1, 16, 16, 1), 0.2, "normal", 0.05)], 96, (500, 900)),
    ("tiled-d484", [TableSpec(10_000, (20, 25, 20), (4, 8, 4), (1, 32, 32, 1), 1.1, "normal", 0.05)], 100, 20),
    ("tiled-k4-r64", [TableSpec(20_736, (12, 12, 12, 12), (2, 4, 4, 4), (1, 64, 64, 64, 1), 1.2, "normal", 0.02)], 120, 8),
    ("k2", [TableSpec(9_999, (100, 100), (8, 8), (1, 12, 1), 1.0, "uniform", 0.1)], 257, (1, 9)),
    ("k4", [TableSpec(40_000, (15, 14, 14, 14), (2, 4, 4, 4), (1, 6, 9, 5, 1), 1.1, "normal", 0.05)], 200, 8),
    ("odd-D", [TableSpec(30_000, (32, 32, 32), (3, 3, 5), (1, 4, 6, 1), 1.0, "normal", 0.1)], 123, (0, 12)),
    ("wide-D", [TableSpec(5_000, (18, 18, 18), (8, 8, 8), (1, 4, 4, 1), 1.0, "normal", 0.1)], 64, (1, 6)),
]


@pytest.mark.parametrize("case", MEDIUM, ids=[c[0] for c in MEDIUM])
def test_medium_forward_backward(binding, case):
    name, tables, B, pooling = case
    wl = workloads.custom(tables, B, pooling, seed=77, with_grad=True, name=name)
    emb, out = run_forward(binding, wl, enable_backward=True)
    assert emb.status() == 0
    assert_close(out, oracle.forward_workload(wl), f"{name} out")
    check_grouping(emb, wl)
    emb.backward(dev(wl.grad_out))
    grads = emb.get_grads()
    ref = oracle.backward_workload(wl)
    for t in range(wl.T):
        for k in range(wl.tables[t].K):
            assert_close(grads[t][k], ref[t][k], f"{name} dG[{t}][{k}]")


# Few lookups per bag: the pooling gather takes windows of 32 lookups across bags there.  One lookup in every bag
# (rows go straight to out), empty bags in between, two to four bags per window, bags longer than a window among short
# ones; batch sizes that put table boundaries and share boundaries inside windows.
SHORT_BAG_TABLES = {
    64: [TableSpec(30_000, (32, 32, 32), (4, 4, 4), (1, 16, 16, 1), 1.1, "normal", 0.05),
         TableSpec(900, (10, 10, 10), (4, 4, 4), (1, 8, 8, 1), 0.8, "normal", 0.05),
         TableSpec(20_000, (28, 28, 28), (4, 4, 4), (1, 16, 32, 1), 1.0, "normal", 0.05)],
    32: [TableSpec(30_000, (32, 32, 32), (2, 4, 4), (1, 16, 16, 1), 1.1, "normal", 0.05),
         TableSpec(700, (9, 9, 9), (2, 4, 4), (1, 8, 8, 1), 0.8, "normal", 0.05),
         TableSpec(20_000, (28, 28, 28), (2, 4, 4), (1, 8, 16, 1), 1.0, "normal", 0.05)],
    20: [TableSpec(9_000, (21, 21, 21), (2, 2, 5), (1, 4, 6, 1), 1.0, "normal", 0.1),
         TableSpec(500, (8, 8, 8), (2, 2, 5), (1, 4, 4, 1), 1.0, "normal", 0.1)],
}


@pytest.mark.parametrize("pooling", [1, (0, 1), (0, 2), (1, 4), (0, 7), (1, 13), (0, 27)], ids=str)
@pytest.mark.parametrize("D", [64, 32, 20])
@pytest.mark.parametrize("B", [33, 1000])
def test_short_bags(binding, D, B, pooling):
    wl = workloads.custom(SHORT_BAG_TABLES[D], B, pooling, seed=123, with_grad=True, name=f"short-D{D}")
    emb, out = run_forward(binding, wl, enable_backward=True)
    assert emb.status() == 0
    assert_close(out, oracle.forward_workload(wl), f"short bags D{D} B{B} {pooling} out")
    emb.backward(dev(wl.grad_out))
    grads = emb.get_grads()
    ref = oracle.backward_workload(wl)
    for t in range(wl.T):
        for k in range(wl.tables[t].K):
            assert_close(grads[t][k], ref[t][k], f"short bags D{D} B{B} {pooling} dG[{t}][{k}]")
    assert emb.check_guards() is None


@pytest.mark.parametrize("mode", ["weighted", "mean"])
@pytest.mark.parametrize("pooling", [1, (0, 3), (1, 13)], ids=str)
def test_short_bags_weighted_and_mean(binding, pooling, mode):
    wl = workloads.custom(SHORT_BAG_TABLES[64], 500, pooling, seed=124, with_grad=True, name="short-wt")
    wts = np.random.default_rng(18).normal(size=wl.L).astype(np.float32) if mode == "weighted" else None
    omode = "mean" if mode == "mean" else "sum"
    emb = binding.from_workload(wl, enable_backward=True, enable_weighted=True)
    emb.set_pooling(omode, None if wts is None else dev(wts))
    out = emb.forward(dev(wl.indices), dev(wl.offsets), wl.B).cpu().numpy()
    assert emb.status() == 0
    assert_close(out, oracle.forward_workload(wl, weights=wts, mode=omode), f"short bags {pooling} {mode} out")
    emb.backward(dev(wl.grad_out))
    grads = emb.get_grads()
    ref = oracle.backward_workload(wl, weights=wts, mode=omode)
    for t in range(wl.T):
        for k in range(wl.tables[t].K):
            assert_close(grads[t][k], ref[t][k], f"short bags {pooling} {mode} dG[{t}][{k}]")


@pytest.mark.parametrize("B", [1, 2, 97])
@pytest.mark.parametrize("D", [64, 32])
def test_short_bags_with_whole_tables_empty(binding, D, B):
    # tables without a single lookup between, before and after tables with short bags; one-bag batches
    tabs = SHORT_BAG_TABLES[D]
    tables = [tabs[0], tabs[1], tabs[2], tabs[0], tabs[1]]
    for pooling in ([0, (0, 3), 0, (1, 5), 0], [(1, 2), 0, 0, 1, (0, 40)], [1, 1, 0, 1, 1]):
        wl = workloads.custom(tables, B, pooling, seed=131, with_grad=True, name="short-empty-tables")
        emb, out = run_forward(binding, wl, enable_backward=True)
        assert emb.status() == 0
        assert_close(out, oracle.forward_workload(wl), f"empty tables D{D} B{B} {pooling} out")
        emb.backward(dev(wl.grad_out))
        grads = emb.get_grads()
        ref = oracle.backward_workload(wl)
        for t in range(wl.T):
            for k in range(wl.tables[t].K):
                assert_close(grads[t][k], ref[t][k], f"empty tables D{D} B{B} {pooling} dG[{t}][{k}]")


def test_many_tables_point_reduced(binding):
    # the many-tables bench workload (D = 32, ranks 32, every table with its own bag-length law) at a size the oracle
    # finishes in seconds: both pooling kernels' territory in one batch, fused update
    wl = workloads.many_tables_point(700, num_tables=16, with_grad=True)
    emb, out = run_forward(binding, wl, enable_backward=True)
    assert emb.status() == 0
    assert_close(out, oracle.forward_workload(wl, memo=True), "many-tables out")
    emb.backward_sgd(dev(wl.grad_out), 0.01)
    grads = emb.get_grads()
    cores = emb.get_cores()
    ref = oracle.backward_workload(wl, memo=True)
    for t in range(wl.T):
        want = oracle.sgd(wl.cores[t], ref[t], 0.01)
        for k in range(3):
            assert_close(grads[t][k], ref[t][k], f"many-tables dG[{t}][{k}]")
            assert_close(cores[t][k], want[k], f"many-tables core[{t}][{k}]")
    assert emb.check_guards() is None


def test_short_bags_with_rows_outside_the_table(binding):
    # ids outside the table among one- and two-lookup bags: flagged, and they add nothing to their bag
    wl = workloads.custom(SHORT_BAG_TABLES[32], 777, (0, 3), seed=125, name="short-oor")
    idx = wl.indices.copy()
    rng = np.random.default_rng(5)
    bad = rng.choice(wl.L, size=wl.L // 7, replace=False)
    t_of = np.searchsorted(wl.offsets[:: wl.B][1:], bad, side="right")
    idx[bad] = np.array([wl.tables[t].N for t in t_of]) + rng.integers(0, 5, size=bad.size)
    wl_bad = workloads.Workload(wl.name, wl.tables, wl.B, idx, wl.offsets, wl.cores, wl.grad_out)
    emb, out = run_forward(binding, wl_bad)
    assert emb.status() & binding.STATUS_INDEX
    assert_close(out, oracle.forward_workload(wl_bad), "short bags with bad ids out")   # the oracle skips them as well


@pytest.mark.parametrize("D,rank", [(16, 8), (16, 16), (16, 32), (32, 8), (32, 16), (32, 32), (64, 8), (64, 16), (64, 32)])
def test_sweep_point_shapes(binding, D, rank):
    # the shapes of the dimension / rank sweep (dim factors 2x2x4, 2x4x4, 4x4x4) at a batch the oracle finishes fast
    wl = workloads.sweep_point(D, rank, 96, num_tables=3, with_grad=True)
    emb, out = run_forward(binding, wl, enable_backward=True)
    assert emb.status() == 0
    assert_close(out, oracle.forward_workload(wl), f"sweep D{D} r{rank} out")
    check_grouping(emb, wl)
    emb.backward(dev(wl.grad_out))
    grads = emb.get_grads()
    ref = oracle.backward_workload(wl)
    for t in range(wl.T):
        for k in range(3):
            assert_close(grads[t][k], ref[t][k], f"sweep D{D} r{rank} dG[{t}][{k}]")
    assert emb.check_guards() is None      # no kernel of these shape variants wrote past its workspace region


@pytest.mark.parametrize("D,rank", [(16, 16), (16, 32), (32, 8), (32, 32), (64, 8)])
def test_sweep_point_shapes_many_groups(binding, D, rank):
    # the same shape classes with thousands of prefix groups per table (several work units per table, long node lists
    # for the middle cores, rows of 64 / 128 / 256 bytes through the staged pooling and dE kernels), fused update
    wl = workloads.sweep_point(D, rank, 2048, num_tables=2, with_grad=True)
    emb, out = run_forward(binding, wl, enable_backward=True)
    assert emb.status() == 0
    assert_close(out, oracle.forward_workload(wl), f"sweep-large D{D} r{rank} out")
    emb.backward_sgd(dev(wl.grad_out), 0.01)
    grads = emb.get_grads()
    cores = emb.get_cores()
    ref = oracle.backward_workload(wl)
    for t in range(wl.T):
        want = oracle.sgd(wl.cores[t], ref[t], 0.01)
        for k in range(3):
            assert_close(grads[t][k], ref[t][k], f"sweep-large D{D} r{rank} dG[{t}][{k}]")
            assert_close(cores[t][k], want[k], f"sweep-large D{D} r{rank} core[{t}][{k}]")


POOLING_CASES = [MEDIUM[0], MEDIUM[1], MEDIUM[3], MEDIUM[5], MEDIUM[7], MEDIUM[8]]   # D = 64 (cp.async pooling), D = 128, K = 2, odd D, wide D


@pytest.mark.parametrize("mode", ["weighted", "mean"])
@pytest.mark.parametrize("case", POOLING_CASES, ids=[c[0] for c in POOLING_CASES])
def test_weighted_and_mean_pooling(binding, case, mode):
    # per-lookup weights and mean pooling (extensions beyond the plain sum), forward and backward
    name, tables, B, pooling = case
    wl = workloads.custom(tables, B, pooling, seed=91, with_grad=True, name=name)
    wts = np.random.default_rng(17).normal(size=wl.L).astype(np.float32) if mode == "weighted" else None
    omode = "mean" if mode == "mean" else "sum"
    emb = binding.from_workload(wl, enable_backward=True, enable_weighted=True)
    emb.set_pooling(omode, None if wts is None else dev(wts))
    out = emb.forward(dev(wl.indices), dev(wl.offsets), wl.B).cpu().numpy()
    assert emb.status() == 0
    assert_close(out, oracle.forward_workload(wl, weights=wts, mode=omode), f"{name} {mode} out")
    emb.backward(dev(wl.grad_out))
    grads = emb.get_grads()
    ref = oracle.backward_workload(wl, weights=wts, mode=omode)
    for t in range(wl.T):
        for k in range(wl.tables[t].K):
            assert_close(grads[t][k], ref[t][k], f"{name} {mode} dG[{t}][{k}]")
    # back to the plain sum on the same handle
    emb.set_pooling("sum")
    out = emb.forward(dev(wl.indices), dev(wl.offsets), wl.B).cpu().numpy()
    assert_close(out, oracle.forward_workload(wl), f"{name} sum after {mode}")


def test_pooling_modes_need_the_config_flag(binding):
    name, tables, B, pooling = MEDIUM[0]
    wl = workloads.custom(tables, B, pooling, seed=5)
    emb = binding.from_workload(wl)
    emb.set_pooling("sum")                       # the default is always allowed
    with pytest.raises(binding.TTEmbError):
        emb.set_pooling("mean")
    emb2 = binding.from_workload(wl, enable_weighted=True)
    with pytest.raises(binding.TTEmbError):     # weights go with the sum mode only
        import ctypes
        from paper_2609_03459_b200.binding import lib, _check
        _check(lib.tt_emb_set_pooling(emb2.h, 1, dev(np.ones(4, np.float32)).data_ptr()), "tt_emb_set_pooling")


def test_long_accumulation_chains_of_one_sign(binding):
    # all cores and all output gradients positive: every partial sum grows monotonically, the worst case for an
    # accumulator that truncates (the tensor core's): groups with hundreds of rows, middle-core slices with hundreds of
    # nodes.  Chains that are not folded into rounded sums miss the tolerance here.
    name, tables, B, pooling = [c for c in MEDIUM if c[0] == "long-chains"][0]
    wl = workloads.custom(tables, B, pooling, seed=78, with_grad=True, name=name)
    wl.cores = [[np.abs(c) for c in tc] for tc in wl.cores]
    wl.grad_out = np.abs(wl.grad_out)
    emb, out = run_forward(binding, wl, enable_backward=True)
    assert_close(out, oracle.forward_workload(wl), "one-sign out")
    emb.backward(dev(wl.grad_out))
    grads = emb.get_grads()
    ref = oracle.backward_workload(wl)
    for t in range(wl.T):
        for k in range(3):
            assert_close(grads[t][k], ref[t][k], f"one-sign dG[{t}][{k}]")


def test_int32_row_ids_give_the_same_result(binding):
    # the 32-bit index entry point: same grouping, same output bit for bit, same gradients; bad ids still flagged
    import torch
    name, tables, B, pooling = MEDIUM[0]
    wl = workloads.custom(tables, B, pooling, seed=41, with_grad=True, name=name)
    emb = binding.from_workload(wl, enable_backward=True)
    out64 = emb.forward(dev(wl.indices), dev(wl.offsets), wl.B).cpu().numpy()
    idx32 = dev(wl.indices.astype(np.int32))
    out32 = emb.forward(idx32, dev(wl.offsets), wl.B).cpu().numpy()
    np.testing.assert_array_equal(out32, out64)
    check_grouping(emb, wl)
    emb.backward(dev(wl.grad_out))
    grads = emb.get_grads()
    ref = oracle.backward_workload(wl)
    for t in range(wl.T):
        for k in range(wl.tables[t].K):
            assert_close(grads[t][k], ref[t][k], f"int32 ids dG[{t}][{k}]")
    bad = wl.indices.astype(np.int32).copy()
    bad[3] = -5
    emb.forward(dev(bad), dev(wl.offsets), wl.B)
    assert emb.status() & binding.STATUS_INDEX


def test_forward_replayed_from_a_cuda_graph(binding):
    # the forward is capturable (no host synchronisation, fork/join of the side streams inside the capture); a replay
    # on new contents of the same buffers gives the new result
    import torch
    name, tables, B, pooling = MEDIUM[1]
    wl = workloads.custom(tables, B, 7, seed=31, name=name)
    wl2 = workloads.custom(tables, B, 7, seed=32, name=name)      # same shapes and lookup count, other rows
    assert wl.L == wl2.L
    wl2.cores = wl.cores
    emb = binding.from_workload(wl)
    d_idx, d_off = dev(wl.indices), dev(wl.offsets)
    out = torch.empty((wl.B, wl.T * wl.D), dtype=torch.float32, device="cuda")
    g = emb.capture_forward(d_idx, d_off, wl.B, out)
    g.replay()
    torch.cuda.synchronize()
    assert_close(out.cpu().numpy(), oracle.forward_workload(wl), "graph replay 1")
    d_idx.copy_(dev(wl2.indices))
    d_off.copy_(dev(wl2.offsets))
    g.replay()
    torch.cuda.synchronize()
    assert emb.status() == 0
    assert_close(out.cpu().numpy(), oracle.forward_workload(wl2), "graph replay 2")


def test_forward_only_handle_and_repeat_calls(binding):
    # a forward-only handle (no backward workspace) gives the same output, and calling twice is idempotent
    name, tables, B, pooling = MEDIUM[0]
    wl = workloads.custom(tables, B, pooling, seed=5)
    emb, out1 = run_forward(binding, wl, enable_backward=False)
    out2 = emb.forward(dev(wl.indices), dev(wl.offsets), wl.B).cpu().numpy()
    np.testing.assert_array_equal(out1, out2)
    assert_close(out1, oracle.forward_workload(wl), "forward-only out")
    # a different batch through the same handle (smaller batch, fewer lookups)
    wl2 = workloads.custom(tables, B // 2, pooling, seed=6)
    emb.forward(dev(wl.indices), dev(wl.offsets), wl.B)
    out3 = emb.forward(dev(wl2.indices), dev(wl2.offsets), wl2.B).cpu().numpy()
    wl2.cores = wl.cores
    assert_close(out3, oracle.forward_workload(wl2), "second batch out")


@pytest.mark.parametrize("case", ["tiled-r16-r32", "tiled-k4-r64", "k2", "k4"])
@pytest.mark.parametrize("flags", [1, 2, 3, 4, 6])
def test_ablation_switches_keep_the_result(binding, flags, case):
    # the study switches (no prefix reuse / static schedule / no de-duplication) change cost, never values;
    # with two, three and four cores (the prefix levels above a level of per-row groups link to rows, not to prefixes)
    name, tables, B, pooling = next(c for c in MEDIUM if c[0] == case)
    wl = workloads.custom(tables, B, pooling, seed=21)
    emb = binding.from_workload(wl, ablation=flags)
    out = emb.forward(dev(wl.indices), dev(wl.offsets), wl.B).cpu().numpy()
    assert emb.status() == 0
    assert_close(out, oracle.forward_workload(wl), f"ablation {flags} out")
    counts = emb.grouping_counts()
    if flags & 1:   # every distinct row is its own group
        assert np.array_equal(counts[:, -2], counts[:, -1])
    if flags == 1:  # ... and the prefix levels above it are the ordinary ones, counting rows under each prefix
        for t, s in enumerate(wl.tables):
            g = oracle.grouping(s.n, wl.table_slice(t)[0])
            for k in range(1, s.K - 1):
                lev = g["levels"][k - 1]
                assert counts[t, k - 1] == lev["vals"].shape[0]
                vals, rc, _ = emb.export_level(t, k, int(counts[t, k - 1]), with_lookup_counts=False)
                np.testing.assert_array_equal(vals, lev["vals"])
                np.testing.assert_array_equal(rc, lev["row_counts"])
    if flags & 4:   # every lookup is a row, a group and a first-level node of its own
        per_table = wl.offsets[np.arange(1, wl.T + 1) * wl.B] - wl.offsets[np.arange(wl.T) * wl.B]
        for k in range(counts.shape[1]):
            assert np.array_equal(counts[:, k], per_table)
    with pytest.raises(binding.TTEmbError):
        binding.from_workload(wl, ablation=flags, enable_backward=True)


# ------------------------------------------------------------------------------------------ degenerate inputs

def test_hot_row_and_long_segments(binding):
    # one row takes ~70 % of 60k lookups: exercises chunk-crossing segments of the dE reduction,
    # the hash-aggregated sort and a bag with thousands of lookups
    spec = TableSpec(50_000, (37, 37, 37), (4, 4, 4), (1, 8, 16, 1), 1.0, "normal", 0.1)
    wl = workloads.custom([spec], 40, (500, 2500), seed=3, with_grad=True)
    rng = np.random.default_rng(0)
    hot = rng.random(wl.L) < 0.7
    wl.indices[hot] = 31_337
    wl.indices[rng.random(wl.L) < 0.1] = 31_338
    emb, out = run_forward(binding, wl, enable_backward=True)
    assert_close(out, oracle.forward_workload(wl), "hot out")
    check_grouping(emb, wl)
    emb.backward(dev(wl.grad_out))
    grads = emb.get_grads()
    ref = oracle.backward_workload(wl)
    for k in range(3):
        assert_close(grads[0][k], ref[0][k], f"hot dG[{k}]")


def test_all_bags_empty(binding):
    spec = TableSpec(1000, (10, 10, 10), (4, 4, 4), (1, 4, 4, 1), 1.0, "normal", 0.1)
    wl = workloads.custom([spec, spec], 9, 0, seed=1, with_grad=True)
    assert wl.L == 0
    import torch
    emb = binding.from_workload(wl, enable_backward=True)
    idx = torch.zeros(1, dtype=torch.int64, device="cuda")[:0]
    out = emb.forward(idx, dev(wl.offsets), wl.B).cpu().numpy()
    assert emb.status() == 0
    assert np.count_nonzero(out) == 0
    emb.backward(dev(wl.grad_out))
    for row in emb.get_grads():
        for g in row:
            assert np.count_nonzero(g) == 0


def test_out_of_range_indices_are_flagged_and_ignored(binding):
    spec = TableSpec(997, (10, 10, 10), (4, 4, 4), (1, 4, 4, 1), 1.0, "normal", 0.1)
    wl = workloads.custom([spec], 20, (1, 6), seed=2, with_grad=True)
    bad = wl.indices.copy()
    bad[3] = 997       # first padding row: not a valid row id
    bad[10] = -5
    bad[11] = 1 << 40
    wl_bad = workloads.Workload(wl.name, wl.tables, wl.B, bad, wl.offsets, wl.cores, wl.grad_out)
    emb, out = run_forward(binding, wl_bad, enable_backward=True)
    assert emb.status() & binding.STATUS_INDEX
    assert_close(out, oracle.forward_workload(wl_bad), "oob out")   # the oracle skips them as well
    emb.backward(dev(wl.grad_out))
    ref = oracle.backward_workload(wl_bad)
    grads = emb.get_grads()
    for k in range(3):
        assert_close(grads[0][k], ref[0][k], f"oob dG[{k}]")


@pytest.mark.parametrize("d", [(4, 4, 4), (4, 8, 4), (2, 4, 4), (3, 3, 5)])
def test_bad_offsets_are_flagged_and_out_is_still_fully_written(binding, d):
    # malformed offsets set the status bit; `out` is still defined everywhere: every bag is the sum over its own
    # (offsets[b], offsets[b+1]) range, an inverted pair being an empty bag -- which is what the oracle's loop does too
    spec = TableSpec(997, (10, 10, 10), d, (1, 4, 4, 1), 1.0, "normal", 0.1)
    wl = workloads.custom([spec], 700, 3, seed=2)
    off = wl.offsets.copy()
    for b in (5, 77, 300, 301, 650):
        off[b], off[b + 1] = off[b + 1], off[b] - 1
    emb = binding.from_workload(wl)
    out = torch_full((wl.B, wl.D), float("nan"))
    emb.forward(dev(wl.indices), dev(off), wl.B, out=out)
    assert emb.status() & binding.STATUS_OFFSETS
    s = wl.tables[0]
    ref = oracle.forward(s.n, s.d, s.r, s.N, wl.cores[0], wl.indices, off)
    assert_close(out.cpu().numpy(), ref, "out with malformed offsets")


def torch_full(shape, value):
    import torch
    return torch.full(shape, value, dtype=torch.float32, device="cuda")


@pytest.mark.parametrize("cfg", [1, 2, 3, 4, 5])
def test_no_kernel_writes_past_its_workspace_region(binding, cfg):
    # guard bytes behind every workspace region (the stand-in for a memory checker) after a whole step
    wl = workloads.make(cfg, tiny=True)
    emb = binding.from_workload(wl, enable_backward=True, enable_weighted=True)
    emb.forward(dev(wl.indices), dev(wl.offsets), wl.B)
    go = wl.grad_out if wl.grad_out is not None else np.ones((wl.B, wl.T * wl.D), np.float32)
    emb.backward_sgd(dev(go), 0.01)
    assert emb.status() == 0
    assert emb.check_guards() is None


def test_guard_check_medium_shapes_and_detection(binding):
    for name, tables, B, pooling in MEDIUM:
        wl = workloads.custom(tables, B, pooling, seed=5, with_grad=True)
        emb = binding.from_workload(wl, enable_backward=True)
        emb.forward(dev(wl.indices), dev(wl.offsets), wl.B)
        emb.backward(dev(wl.grad_out))
        emb.sgd_step(0.01)
        assert emb.check_guards() is None, name
    # the check does see damage: the last byte of the workspace is a guard byte of the last region
    base_off = (-emb.workspace.data_ptr()) % 256
    emb.workspace[base_off + emb.workspace_bytes - 1] = 0
    assert emb.check_guards() == "guard_list"


@pytest.mark.parametrize("spec", [
    TableSpec(5000, (18, 18, 18), (4, 4, 4), (1, 4, 4, 1), 0.5, "normal", 0.1),
    TableSpec(30_000, (14, 13, 13, 13), (2, 4, 4, 4), (1, 6, 9, 5, 1), 0.5, "normal", 0.1),
    TableSpec(9_999, (100, 100), (8, 8), (1, 12, 1), 0.5, "uniform", 0.1),
], ids=["k3", "k4", "k2"])
@pytest.mark.parametrize("pooling,B", [(20, 50), ((0, 3), 600)], ids=["long-bags", "short-bags"])
def test_unique_row_capacity_overflow_is_flagged(binding, spec, pooling, B):
    # more distinct rows than the handle was sized for: flagged, and every kernel of the forward and of the backward
    # still stays inside its workspace region (the rows past the capacity are dropped, prefix levels are clipped to them);
    # with long bags (one bag per pooling window) and with short ones (windows across bags)
    wl = workloads.custom([spec, spec], B, pooling, seed=4, with_grad=True)
    emb = binding.from_workload(wl, max_unique_rows=100, enable_backward=True)
    out = emb.forward(dev(wl.indices), dev(wl.offsets), wl.B)
    assert emb.status() & binding.STATUS_OVERFLOW
    assert np.isfinite(out.cpu().numpy()).all()
    emb.backward(dev(wl.grad_out))
    assert emb.check_guards() is None
    # the same handle is fine again with a batch that fits
    small = workloads.custom([spec, spec], 4, 5, seed=5)
    small.cores = wl.cores
    out2 = emb.forward(dev(small.indices), dev(small.offsets), small.B).cpu().numpy()
    assert emb.status() == 0
    assert_close(out2, oracle.forward_workload(small), "after overflow")


def test_pack_unpack_round_trip(binding):
    wl = workloads.make(4, tiny=True)
    emb = binding.from_workload(wl)
    back = emb.get_cores()
    for k in range(4):
        np.testing.assert_array_equal(back[0][k], wl.cores[0][k])


def test_invariants_index_order_and_bag_additivity(binding):
    # results do not depend on the order of indices inside a bag; a bag holding two bags' lookups is their sum
    spec = TableSpec(20_000, (28, 28, 28), (4, 4, 4), (1, 8, 8, 1), 1.1, "normal", 0.1)
    wl = workloads.custom([spec], 64, 16, seed=9)
    emb, out = run_forward(binding, wl)
    rng = np.random.default_rng(1)
    perm = wl.indices.reshape(64, 16).copy()
    for b in range(64):
        rng.shuffle(perm[b])
    out_p = emb.forward(dev(perm.reshape(-1)), dev(wl.offsets), 64).cpu().numpy()
    assert np.abs(out_p - out).max() <= 2e-6 * np.abs(out).max()
    merged_off = wl.offsets[::2].copy()
    out_m = emb.forward(dev(wl.indices), dev(merged_off), 32).cpu().numpy()
    assert np.abs(out_m - (out[0::2] + out[1::2])).max() <= 2e-6 * np.abs(out).max()


def test_forward_and_grouping_are_bit_reproducible(binding):
    # two runs of the same training step on fresh handles: `out` and the grouping are identical bit for bit (nothing in
    # the forward depends on timing).  The gradients agree to rounding only: the backward sort claims positions with
    # atomics and the last core's slices are accumulated with vector reductions, so their summation order varies.
    name, tables, B, pooling = MEDIUM[1]
    wl = workloads.custom(tables, B, pooling, seed=33, with_grad=True)
    runs = []
    for _ in range(2):
        emb = binding.from_workload(wl, enable_backward=True)
        out = emb.forward(dev(wl.indices), dev(wl.offsets), wl.B).cpu().numpy()
        counts = emb.grouping_counts()
        levels = [emb.export_level(t, k, int(counts[t, k - 1])) for t in range(wl.T) for k in range(1, wl.tables[t].K + 1)]
        inv = [emb.export_inverse(t, wl.table_slice(t)[0].shape[0]) for t in range(wl.T)]
        emb.backward(dev(wl.grad_out))
        runs.append((out, counts, levels, inv, emb.get_grads()))
    a, b = runs
    assert np.array_equal(a[0], b[0])
    assert np.array_equal(a[1], b[1])
    for la, lb in zip(a[2], b[2]):
        for x, y in zip(la, lb):
            assert np.array_equal(x, y)
    for x, y in zip(a[3], b[3]):
        assert np.array_equal(x, y)
    for t in range(wl.T):
        for k in range(wl.tables[t].K):
            scale = max(np.abs(a[4][t][k]).max(), 1e-30)
            assert np.abs(a[4][t][k] - b[4][t][k]).max() <= 2e-6 * scale


@pytest.mark.parametrize("n_cols", [32, 128])
def test_tcgen05_probe_product_is_exact(binding, n_cols):
    # the measurement helper's tile product D[128 x N] = A[128 x 32] . B[32 x N] on the fifth-generation tensor cores
    # against a plain FP32 loop over the same operands (multiples of 1/4: exact in TF32, sums exact in fp32)
    rate, err = binding.probe_tcgen05(n_cols)
    assert err == 0.0
    assert rate > 1e9    # M128.N.k8 instructions per second of the whole device
