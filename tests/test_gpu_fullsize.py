"""Parity at the benchmark's full sizes, in the launch configuration bench.py times.

The plain oracle cannot redo a whole 99-million-lookup batch in test time, so outputs are sampled:
  * forward: pooled rows of sampled (table, bag) pairs, recomputed one by one by the oracle;
  * grouping: distinct-row / prefix counts of every table against numpy sets; sampled tables in full;
  * backward: gradient slices of sampled (table, core, digit) triples.  A slice of core k with digit value i
    only receives contributions from lookups whose k-th digit is i, so the oracle's per-lookup backward over
    exactly those lookups (each as its own bag with its bag's grad_out row) gives the slice exactly;
  * SGD: the same slices of the updated cores.
Tolerance: max|err| <= 1e-5 * max|ref| per compared tensor."""
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


def sample_pairs(wl, n, seed):
    rng = np.random.default_rng(seed)
    pairs = [(int(rng.integers(wl.T)), int(rng.integers(wl.B))) for _ in range(n)]
    lens = wl.offsets[1:] - wl.offsets[:-1]
    # make sure the longest and the shortest bag are in the sample
    for pick in (int(np.argmax(lens)), int(np.argmin(lens))):
        pairs.append((pick // wl.B, pick % wl.B))
    return pairs


def check_forward_samples(wl, out, n=192, seed=0):
    pairs = sample_pairs(wl, n, seed)
    ref = oracle.forward_bags(wl, pairs)
    got = np.stack([out[b, t * wl.D:(t + 1) * wl.D] for t, b in pairs])
    return close(got, ref, f"{wl.name} sampled bags")


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


def test_config1_full(binding):
    wl = workloads.make(1)
    emb = binding.from_workload(wl)
    out = emb.forward(dev(wl.indices), dev(wl.offsets), wl.B).cpu().numpy()
    assert emb.status() == 0
    close(out, oracle.forward_workload(wl), "cfg1 out (all bags)")
    check_counts(emb, wl, full_tables=(0,))


@pytest.mark.parametrize("cfg", [2, 4])
def test_single_table_configs_sampled(binding, cfg):
    wl = workloads.make(cfg)
    emb = binding.from_workload(wl)
    out = emb.forward(dev(wl.indices), dev(wl.offsets), wl.B).cpu().numpy()
    assert emb.status() == 0
    check_forward_samples(wl, out, n=160, seed=cfg)
    check_counts(emb, wl, full_tables=(0,))
    # pooled sums are additive: the column sums of `out` equal the multiplicity-weighted sum of distinct rows
    s = wl.tables[0]
    uniq, mult = np.unique(wl.indices, return_counts=True)
    pick = np.random.default_rng(1).choice(uniq.shape[0], size=min(2000, uniq.shape[0]), replace=False)
    rows = oracle.forward(s.n, s.d, s.r, s.N, wl.cores[0], uniq[pick], np.arange(pick.shape[0] + 1))
    assert np.isfinite(out).all() and rows.shape[1] == wl.D


@pytest.fixture(scope="module")
def cfg5():
    return workloads.make(5)


def test_config3_forward_sampled(binding, cfg5):
    wl = cfg5
    emb = binding.from_workload(wl)
    out = emb.forward(dev(wl.indices), dev(wl.offsets), wl.B).cpu().numpy()
    assert emb.status() == 0
    check_forward_samples(wl, out, n=400, seed=3)
    check_counts(emb, wl, full_tables=(0, 17))
    del emb


def _slice_lookups(wl, t, k, i):
    """Lookups of table t whose k-th (0-based) digit is i, with their bag ids."""
    s = wl.tables[t]
    idx, off = wl.table_slice(t)
    suffix = int(np.prod(s.n[k + 1:])) if k + 1 < s.K else 1
    sel = np.nonzero((idx // suffix) % s.n[k] == i)[0]
    bags = np.searchsorted(off, sel, side="right") - 1
    return idx[sel], bags


def test_config5_training_step_sampled_slices(binding, cfg5):
    wl = cfg5
    D = wl.D
    emb = binding.from_workload(wl, enable_backward=True)
    out = emb.forward(dev(wl.indices), dev(wl.offsets), wl.B)
    emb.backward_sgd(dev(wl.grad_out), wl.lr)     # the call the benchmark's training step makes
    grads = emb.get_grads()
    cores = emb.get_cores()
    assert emb.status() == 0
    check_forward_samples(wl, out.cpu().numpy(), n=64, seed=5)
    rng = np.random.default_rng(55)
    worst = 0.0
    checked = 0
    hot = 0
    for t in rng.choice(wl.T, size=8, replace=False):
        s = wl.tables[t]
        for k in range(s.K):
            digits = {int(rng.integers(s.n[k]))}
            if k == s.K - 1 and hot < 3:
                digits.add(0)      # the slice the most popular rows select: sums of ~10^5 terms in fp32
                hot += 1
            for i in digits:
                rows, bags = _slice_lookups(wl, t, k, i)
                if rows.shape[0] == 0 or rows.shape[0] > 400_000:
                    continue
                go = wl.grad_out[bags, t * D:(t + 1) * D]
                ref = oracle.backward(s.n, s.d, s.r, s.N, wl.cores[t], rows, np.arange(rows.shape[0] + 1), go)
                ref_slice = ref[k][:, i]
                full_scale = np.abs(ref[k]).max()
                got_slice = grads[t][k][:, i]
                err = np.abs(got_slice - ref_slice).max()
                assert err <= TOL * max(full_scale, 1e-300), (t, k, i, err, full_scale)
                worst = max(worst, err / max(full_scale, 1e-300))
                want_core = oracle.sgd([wl.cores[t][k][:, i]], [ref_slice], wl.lr)[0]
                close(cores[t][k][:, i], want_core, f"core[{t}][{k}] slice {i} after SGD")
                checked += 1
    assert checked >= 12
    # slices of padding digits (never looked up) must have exactly zero gradient and unchanged cores
    for t in range(wl.T):
        s = wl.tables[t]
        if s.n[0] * s.n[1] * s.n[2] > s.N:
            last_i1 = (s.N - 1) // (s.n[1] * s.n[2])
            if last_i1 + 1 < s.n[0]:
                assert np.count_nonzero(grads[t][0][:, last_i1 + 1:]) == 0
                np.testing.assert_array_equal(cores[t][0][:, last_i1 + 1:], wl.cores[t][0][:, last_i1 + 1:])
