"""Pins for the fp64 CPU oracle: every check here compares the oracle with something that is NOT the
oracle's own contraction code -- the paper's definitions written another way, closed forms, exact
finite differences, library routines (torch.einsum / embedding_bag), or brute force on tiny inputs."""
import itertools

import numpy as np
import pytest
import torch

import oracle
import workloads
from workloads import TableSpec

SHAPES = [
    # (n, d, r)
    ((3, 4), (2, 3), (1, 3, 1)),
    ((3, 2, 4), (2, 3, 2), (1, 3, 5, 1)),
    ((5, 6, 4), (4, 4, 4), (1, 8, 8, 1)),
    ((2, 3, 2, 3), (2, 2, 3, 2), (1, 2, 3, 2, 1)),
    ((3, 3, 3), (1, 5, 2), (1, 1, 4, 1)),
]


def rand_cores(rng, n, d, r, scale=1.0):
    return [rng.normal(0, scale, size=(r[k], n[k], d[k], r[k + 1])) for k in range(len(n))]


# ------------------------------------------------------------------ A. digit decomposition (Eq. 1)

def test_digits_decimal_case_fixes_msb_first():
    # with radices 100,100,100 the digits are the decimal pairs of the number, most significant first
    assert oracle.digits(123456, (100, 100, 100)) == (12, 34, 56)
    assert oracle.digits(7, (100, 100, 100)) == (0, 0, 7)
    assert oracle.digits(999999, (100, 100, 100)) == (99, 99, 99)


@pytest.mark.parametrize("n", [(3, 4), (2, 3, 5), (4, 1, 3), (2, 3, 2, 3), (7, 5, 3)])
def test_digits_exhaustive_matches_lexicographic_enumeration(n):
    # enumerating digit tuples in lexicographic order (first digit slowest) visits g = 0,1,2,..
    for g, tup in enumerate(itertools.product(*[range(x) for x in n])):
        assert oracle.digits(g, n) == tup


def test_digits_round_trip_large(rng):
    n = (200, 250, 200)
    for g in rng.integers(0, 10_000_000, size=200):
        dg = oracle.digits(int(g), n)
        assert all(0 <= dg[k] < n[k] for k in range(3))
        assert dg[0] * 250 * 200 + dg[1] * 200 + dg[2] == g


# ------------------------------------------------------------------ B. row reconstruction vs the definition

@pytest.mark.parametrize("n,d,r", SHAPES)
def test_row_matches_dense_definition(rng, n, d, r):
    cores = rand_cores(rng, n, d, r)
    W = oracle.dense(n, d, r, cores)
    for g in range(int(np.prod(n))):
        np.testing.assert_allclose(oracle.row(n, d, r, cores, g), W[g], rtol=1e-12, atol=1e-13)


@pytest.mark.parametrize("n,d,r", SHAPES)
def test_dense_matches_einsum(rng, n, d, r):
    # library routine: chain the cores with einsum into the full tensor, then reorder to [rows, cols]
    cores = rand_cores(rng, n, d, r)
    K = len(n)
    full = torch.from_numpy(cores[0])[0]  # [n1, d1, r1]
    for k in range(1, K):
        full = torch.einsum("...a,anjb->...njb", full, torch.from_numpy(cores[k]))
    full = full[..., 0]  # [n1,d1,n2,d2,...]
    perm = [2 * k for k in range(K)] + [2 * k + 1 for k in range(K)]
    Wt = full.permute(*perm).reshape(int(np.prod(n)), int(np.prod(d))).numpy()
    np.testing.assert_allclose(oracle.dense(n, d, r, cores), Wt, rtol=1e-12, atol=1e-13)


# ------------------------------------------------------------------ C. closed forms

def test_rank_one_is_product_of_entries(rng):
    n, d, r = (3, 4, 2), (2, 3, 2), (1, 1, 1, 1)
    cores = rand_cores(rng, n, d, r)
    for g in (0, 5, 17, 23):
        i = oracle.digits(g, n)
        E = oracle.row(n, d, r, cores, g)
        for j, (j1, j2, j3) in enumerate(itertools.product(range(2), range(3), range(2))):
            want = cores[0][0, i[0], j1, 0] * cores[1][0, i[1], j2, 0] * cores[2][0, i[2], j3, 0]
            assert abs(E[j] - want) < 1e-14


def test_all_ones_cores_give_product_of_inner_ranks():
    n, d, r = (3, 2, 4), (2, 2, 3), (1, 5, 7, 1)
    cores = [np.ones((r[k], n[k], d[k], r[k + 1])) for k in range(3)]
    E = oracle.row(n, d, r, cores, 11)
    assert np.all(E == 35.0)


def test_sum_separable_table_rank_two(rng):
    # W[i, j] = f1(i1,j1) + f2(i2,j2) + f3(i3,j3) has an exact TT of rank 2:
    # G1 = [f1 1], G2 = [[1 0],[f2 1]], G3 = [1; f3]
    n, d = (3, 4, 2), (2, 3, 2)
    f = [rng.normal(size=(n[k], d[k])) for k in range(3)]
    G1 = np.zeros((1, n[0], d[0], 2)); G1[0, :, :, 0] = f[0]; G1[0, :, :, 1] = 1
    G2 = np.zeros((2, n[1], d[1], 2)); G2[0, :, :, 0] = 1; G2[1, :, :, 0] = f[1]; G2[1, :, :, 1] = 1
    G3 = np.zeros((2, n[2], d[2], 1)); G3[0, :, :, 0] = 1; G3[1, :, :, 0] = f[2]
    # check the construction on paper: [f1 1] [[1 0],[f2 1]] = [f1+f2, 1]; times [1; f3] = f1+f2+f3
    for g in range(24):
        i = oracle.digits(g, n)
        E = oracle.row(n, d, (1, 2, 2, 1), [G1, G2, G3], g)
        for j, (j1, j2, j3) in enumerate(itertools.product(range(2), range(3), range(2))):
            assert abs(E[j] - (f[0][i[0], j1] + f[1][i[1], j2] + f[2][i[2], j3])) < 1e-13


def test_scaling_one_core_scales_output(rng):
    n, d, r = SHAPES[1]
    cores = rand_cores(rng, n, d, r)
    idx = np.array([1, 5, 5, 20, 3]); off = np.array([0, 2, 5])
    base = oracle.forward(n, d, r, 24, cores, idx, off)
    cores2 = [c.copy() for c in cores]; cores2[1] *= -2.5
    np.testing.assert_allclose(oracle.forward(n, d, r, 24, cores2, idx, off), -2.5 * base, rtol=1e-13)


# ------------------------------------------------------------------ D. pooling

def test_pooling_is_sum_of_rows_with_duplicates_and_empty_bags(rng):
    n, d, r = SHAPES[2]
    N = int(np.prod(n)) - 3
    cores = rand_cores(rng, n, d, r, 0.3)
    W = oracle.dense(n, d, r, cores)
    lens = np.array([3, 0, 1, 7, 0, 2])
    off = np.concatenate([[0], np.cumsum(lens)])
    idx = rng.integers(0, N, size=off[-1]); idx[4] = idx[5] = idx[6]  # duplicates inside bag 3
    out = oracle.forward(n, d, r, N, cores, idx, off)
    for b in range(len(lens)):
        want = W[idx[off[b]:off[b + 1]]].sum(axis=0) if lens[b] else np.zeros(W.shape[1])
        np.testing.assert_allclose(out[b], want, rtol=1e-12, atol=1e-13)
    # library routine on the brute-force table
    eb = torch.nn.functional.embedding_bag(torch.from_numpy(idx), torch.from_numpy(W),
                                           torch.from_numpy(off[:-1]), mode="sum").numpy()
    np.testing.assert_allclose(out, eb, rtol=1e-12, atol=1e-13)


def test_pooling_order_invariance_and_additivity(rng):
    n, d, r = SHAPES[1]
    cores = rand_cores(rng, n, d, r)
    idx = rng.integers(0, 24, size=12); off = np.array([0, 5, 12])
    out = oracle.forward(n, d, r, 24, cores, idx, off)
    idx2 = idx.copy(); idx2[:5] = idx[:5][::-1]; idx2[5:] = np.roll(idx[5:], 3)
    np.testing.assert_allclose(oracle.forward(n, d, r, 24, cores, idx2, off), out, rtol=1e-12, atol=1e-14)
    # one bag holding both bags' lookups = sum of the two bags
    both = oracle.forward(n, d, r, 24, cores, idx, np.array([0, 12]))
    np.testing.assert_allclose(both[0], out[0] + out[1], rtol=1e-12, atol=1e-14)
    # out-of-range indices contribute nothing
    idx3 = np.concatenate([idx, [-1, 24, 10**9]]); off3 = np.array([0, 5, 15])
    np.testing.assert_allclose(oracle.forward(n, d, r, 24, cores, idx3, off3), out, rtol=1e-12, atol=1e-14)


# ------------------------------------------------------------------ E. backward

def _loss(n, d, r, N, cores, idx, off, go):
    return float((oracle.forward(n, d, r, N, cores, idx, off) * go).sum())


@pytest.mark.parametrize("n,d,r", SHAPES[:4])
def test_backward_exact_finite_difference(rng, n, d, r):
    # the loss sum(grad_out * out) is linear in each single core entry, so a difference quotient
    # is exact for any step size
    N = int(np.prod(n))
    cores = rand_cores(rng, n, d, r, 0.5)
    lens = rng.integers(0, 5, size=6); off = np.concatenate([[0], np.cumsum(lens)])
    idx = rng.integers(0, N, size=off[-1])
    go = rng.normal(size=(6, int(np.prod(d))))
    grads = oracle.backward(n, d, r, N, cores, idx, off, go)
    base = _loss(n, d, r, N, cores, idx, off, go)
    for k in range(len(n)):
        flat = cores[k].reshape(-1)
        for e in rng.choice(flat.size, size=min(flat.size, 25), replace=False):
            for step in (1e-3, 1.0, 37.0):
                c2 = [c.copy() for c in cores]
                c2[k].reshape(-1)[e] += step
                fd = (_loss(n, d, r, N, c2, idx, off, go) - base) / step
                assert abs(fd - grads[k].reshape(-1)[e]) < 1e-9 * max(1.0, abs(fd)), (k, e, step)


@pytest.mark.parametrize("n,d,r", SHAPES[:4])
def test_backward_matches_dense_route(rng, n, d, r):
    # dW = scatter-add of grad_out over the looked-up rows; dL/dG_k[entry] = <dW, dW/dG_k[entry]> and,
    # W being linear in core k, dW/dG_k[entry] is the dense table built with core k replaced by a one-hot
    N = int(np.prod(n))
    cores = rand_cores(rng, n, d, r, 0.5)
    lens = rng.integers(1, 4, size=5); off = np.concatenate([[0], np.cumsum(lens)])
    idx = rng.integers(0, N, size=off[-1])
    go = rng.normal(size=(5, int(np.prod(d))))
    grads = oracle.backward(n, d, r, N, cores, idx, off, go)
    dW = np.zeros((N, int(np.prod(d))))
    for b in range(5):
        for l in range(off[b], off[b + 1]):
            dW[idx[l]] += go[b]
    for k in range(len(n)):
        for e in rng.choice(cores[k].size, size=min(cores[k].size, 12), replace=False):
            c2 = [c.copy() for c in cores]
            c2[k] = np.zeros_like(cores[k]); c2[k].reshape(-1)[e] = 1.0
            want = float((oracle.dense(n, d, r, c2) * dW).sum())
            assert abs(want - grads[k].reshape(-1)[e]) < 1e-10 * max(1.0, abs(want))


def test_backward_matches_torch_autograd(rng):
    n, d, r = (4, 3, 5), (4, 4, 4), (1, 6, 3, 1)
    N = 57
    cores = rand_cores(rng, n, d, r, 0.4)
    lens = rng.integers(0, 6, size=9); off = np.concatenate([[0], np.cumsum(lens)])
    idx = rng.integers(0, N, size=off[-1])
    go = rng.normal(size=(9, 64))
    grads = oracle.backward(n, d, r, N, cores, idx, off, go)
    tc = [torch.from_numpy(c).clone().requires_grad_(True) for c in cores]
    i1, i2, i3 = idx // 15, (idx // 5) % 3, idx % 5
    A = tc[0][0][i1]                      # [L, d1, r1]
    Bm = tc[1][:, i2].permute(1, 0, 2, 3)  # [L, r1, d2, r2]
    Dm = tc[2][:, i3, :, 0].permute(1, 0, 2)  # [L, r2, d3]
    C = torch.einsum("lpa,lajb->lpjb", A, Bm)
    E = torch.einsum("lpjb,lbk->lpjk", C, Dm).reshape(len(idx), 64)
    bag = np.repeat(np.arange(9), lens)
    loss = (E * torch.from_numpy(go)[bag]).sum()
    loss.backward()
    for k in range(3):
        np.testing.assert_allclose(grads[k], tc[k].grad.numpy(), rtol=1e-11, atol=1e-12)


@pytest.mark.parametrize("mode,weighted", [("sum", True), ("mean", False)])
def test_weighted_and_mean_pooling_match_library_embedding_bag(rng, mode, weighted):
    # extensions beyond the paper's plain sum: forward against torch's embedding_bag on the brute-force table,
    # backward against autograd through that same library call (gradient w.r.t. the dense table, contracted with
    # the other cores by the brute-force definition of d table / d core entry)
    n, d, r = (3, 4, 3), (2, 3, 2), (1, 3, 2, 1)
    N = 33
    cores = rand_cores(rng, n, d, r, 0.5)
    W = oracle.dense(n, d, r, cores)
    lens = np.array([4, 0, 1, 6, 2]); off = np.concatenate([[0], np.cumsum(lens)])
    idx = rng.integers(0, N, size=off[-1]); idx[5] = idx[6]
    wts = rng.normal(size=off[-1]) if weighted else None
    go = rng.normal(size=(len(lens), 12))
    out = oracle.forward(n, d, r, N, cores, idx, off, wts, mode)
    Wt = torch.from_numpy(W).clone().requires_grad_(True)
    eb = torch.nn.functional.embedding_bag(torch.from_numpy(idx), Wt, torch.from_numpy(off[:-1]), mode=mode,
                                           per_sample_weights=None if wts is None else torch.from_numpy(wts))
    np.testing.assert_allclose(out, eb.detach().numpy(), rtol=1e-12, atol=1e-13)
    (eb * torch.from_numpy(go)).sum().backward()
    dW = Wt.grad.numpy()
    grads = oracle.backward(n, d, r, N, cores, idx, off, go, wts, mode)
    pick = np.random.default_rng(5)
    for k in range(3):
        for e in pick.choice(cores[k].size, size=12, replace=False):
            c2 = [c.copy() for c in cores]
            c2[k] = np.zeros_like(cores[k]); c2[k].reshape(-1)[e] = 1.0
            want = float((oracle.dense(n, d, r, c2) * dW).sum())   # the table is linear in each core
            assert abs(want - grads[k].reshape(-1)[e]) < 1e-10 * max(1.0, abs(want))
    # special cases that reduce to the plain sum: unit weights; mean over bags of one lookup
    ones = oracle.forward(n, d, r, N, cores, idx, off, np.ones(off[-1]), "sum")
    np.testing.assert_allclose(ones, oracle.forward(n, d, r, N, cores, idx, off), rtol=0, atol=0)
    off1 = np.arange(off[-1] + 1)
    np.testing.assert_allclose(oracle.forward(n, d, r, N, cores, idx, off1, None, "mean"),
                               oracle.forward(n, d, r, N, cores, idx, off1), rtol=0, atol=0)


def test_backward_prefix_regrouping_identity_eq2(rng):
    # Eq. 2: for lookups that share the first two digits, (sum_n dC_n).B^T equals sum_n (dC_n.B^T):
    # the gradient of one bag holding all rows of a prefix group equals the sum over single-row bags
    n, d, r = (3, 3, 4), (2, 2, 2), (1, 3, 2, 1)
    cores = rand_cores(rng, n, d, r)
    rows = np.array([4 * 5 + j for j in range(4)])  # prefix (1, 2), all four last digits
    go = rng.normal(size=(1, 8))
    together = oracle.backward(n, d, r, 36, cores, rows, np.array([0, 4]), go)
    apart = [oracle.backward(n, d, r, 36, cores, rows[j:j + 1], np.array([0, 1]), go) for j in range(4)]
    for k in range(3):
        np.testing.assert_allclose(together[k], sum(a[k] for a in apart), rtol=1e-12, atol=1e-14)
    # and only the touched slices are non-zero
    assert np.count_nonzero(together[0][:, [0, 2]]) == 0 and np.count_nonzero(together[1][:, [0, 1]]) == 0


# ------------------------------------------------------------------ F. SGD

def test_sgd_closed_form(rng):
    c = [rng.normal(size=(2, 3, 2, 2))]; g = [rng.normal(size=(2, 3, 2, 2))]; g[0][:, 1] = 0.0
    new = oracle.sgd(c, g, 0.01)[0]
    np.testing.assert_array_equal(new, c[0] - 0.01 * g[0])
    np.testing.assert_array_equal(new[:, 1], c[0][:, 1])  # untouched slice is bit-identical


# ------------------------------------------------------------------ G. grouping (integers)

def test_grouping_matches_python_sets(rng):
    n = (4, 3, 5)
    idx = rng.integers(0, 57, size=200)
    g = oracle.grouping(n, idx)
    uniq = sorted(set(int(x) for x in idx))
    assert g["uniq"].tolist() == uniq
    assert all(g["uniq"][g["inv"][l]] == idx[l] for l in range(200))
    assert g["mult"].sum() == 200
    for u, row in enumerate(uniq):
        assert tuple(g["digits"][u]) == oracle.digits(row, n)
        assert g["mult"][u] == int((idx == row).sum())
    for k, s in ((1, 15), (2, 5)):
        lev = g["levels"][k - 1]
        rows_by, looks_by = {}, {}
        for row in uniq:
            rows_by[row // s] = rows_by.get(row // s, 0) + 1
        for x in idx:
            looks_by[int(x) // s] = looks_by.get(int(x) // s, 0) + 1
        assert lev["vals"].tolist() == sorted(rows_by)
        assert lev["row_counts"].tolist() == [rows_by[v] for v in sorted(rows_by)]
        assert lev["lookup_counts"].tolist() == [looks_by[v] for v in sorted(rows_by)]


def test_grouping_empty():
    g = oracle.grouping((2, 2, 2), np.zeros(0, np.int64))
    assert g["uniq"].size == 0 and all(lv["vals"].size == 0 for lv in g["levels"])


# ------------------------------------------------------------------ workloads + multi-table wrapper

@pytest.mark.parametrize("cfg", [1, 2, 3, 4, 5])
def test_tiny_configs_forward_matches_dense(cfg):
    wl = workloads.make(cfg, tiny=True)
    out = oracle.forward_workload(wl)
    D = wl.D
    for t, s in enumerate(wl.tables):
        W = oracle.dense(s.n, s.d, s.r, wl.cores[t])
        idx, off = wl.table_slice(t)
        for b in range(wl.B):
            want = W[idx[off[b]:off[b + 1]]].sum(axis=0)
            np.testing.assert_allclose(out[b, t * D:(t + 1) * D], want, rtol=1e-11, atol=1e-13)
    assert wl.offsets[0] == 0 and wl.offsets[-1] == wl.L and np.all(np.diff(wl.offsets) >= 0)
    for t, s in enumerate(wl.tables):
        idx, _ = wl.table_slice(t)
        assert idx.min() >= 0 and idx.max() < s.N and int(np.prod(s.n)) >= s.N


def test_forward_bags_sampling_agrees_with_full():
    wl = workloads.make(3, tiny=True)
    full = oracle.forward_workload(wl)
    pairs = [(0, 3), (2, 7), (3, 15)]
    got = oracle.forward_bags(wl, pairs)
    for i, (t, b) in enumerate(pairs):
        np.testing.assert_array_equal(got[i], full[b, t * wl.D:(t + 1) * wl.D])


def test_per_table_bag_lengths_and_the_many_tables_point():
    # a list gives every table its own bag-length law; the many-tables point (the paper's operating shape, Sec. 4.1:
    # D = 32, ranks 32, three cores) draws one per table and records it
    spec = workloads.TableSpec(500, (8, 8, 8), (2, 4, 4), (1, 4, 4, 1), 1.0, "normal", 0.1)
    wl = workloads.custom([spec, spec, spec], 50, [1, (0, 3), (5, 9)], seed=3)
    lens = np.diff(wl.offsets).reshape(3, 50)
    assert (lens[0] == 1).all() and lens[1].min() >= 0 and lens[1].max() <= 3 and lens[2].min() >= 5 and lens[2].max() <= 9
    assert wl.L == int(lens.sum()) and wl.indices.min() >= 0 and wl.indices.max() < 500
    mt = workloads.many_tables_point(16, num_tables=6, with_grad=True)
    assert mt.T == 6 and mt.D == 32 and all(s.r == (1, 32, 32, 1) and s.d == (2, 4, 4) for s in mt.tables)
    lens = np.diff(mt.offsets).reshape(6, 16)
    for t, cap in enumerate(mt.meta["max_bag"]):
        assert 1 <= cap <= 64 and lens[t].min() >= 1 and lens[t].max() <= cap
    again = workloads.many_tables_point(16, num_tables=6, with_grad=True)
    assert np.array_equal(mt.indices, again.indices) and np.array_equal(mt.grad_out, again.grad_out)
