"""Pins for the memoised oracle (oracle/tt_oracle_memo.c): the same plain definition as tt_oracle.c with every
distinct row built once.  The two files share no code, so agreement to fp64 rounding pins both; on top of that
the memoised one is held against things that are neither: the brute-force dense table with the library's
embedding_bag (forward) and autograd through it (backward), and an exact finite difference."""
import numpy as np
import pytest
import torch

import oracle
import workloads
from workloads import TableSpec

SHAPES = [
    ((3, 4), (2, 3), (1, 3, 1)),
    ((3, 2, 4), (2, 3, 2), (1, 3, 5, 1)),
    ((5, 6, 4), (4, 4, 4), (1, 8, 8, 1)),
    ((2, 3, 2, 3), (2, 2, 3, 2), (1, 2, 3, 2, 1)),
    ((3, 3, 3), (1, 5, 2), (1, 1, 4, 1)),
]


def rand_cores(rng, n, d, r):
    return [rng.normal(0, 1.0, size=(r[k], n[k], d[k], r[k + 1])) for k in range(len(n))]


def ragged_batch(rng, N, B, max_len, bad=0):
    lens = rng.integers(0, max_len + 1, size=B)
    off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int64)
    idx = rng.integers(0, N, size=int(off[-1])).astype(np.int64)
    if idx.size:
        idx[rng.integers(0, idx.size, size=idx.size // 3)] = idx[0]        # a popular row
        for j in range(min(bad, idx.size)):
            idx[(7 * j + 3) % idx.size] = N + j if j % 2 else -1 - j        # ids outside [0, N) contribute nothing
    return idx, off


@pytest.mark.parametrize("n,d,r", SHAPES)
@pytest.mark.parametrize("mode,weighted", [("sum", False), ("sum", True), ("mean", False)])
def test_memo_equals_plain_oracle(rng, n, d, r, mode, weighted):
    N = int(np.prod(n)) - 1
    cores = rand_cores(rng, n, d, r)
    idx, off = ragged_batch(rng, N, 23, 9, bad=3)
    w = rng.normal(size=idx.shape[0]) if weighted else None
    go = rng.normal(size=(23, int(np.prod(d))))
    np.testing.assert_allclose(oracle.forward(n, d, r, N, cores, idx, off, w, mode, memo=True),
                               oracle.forward(n, d, r, N, cores, idx, off, w, mode), rtol=1e-12, atol=1e-12)
    gm = oracle.backward(n, d, r, N, cores, idx, off, go, w, mode, memo=True)
    gp = oracle.backward(n, d, r, N, cores, idx, off, go, w, mode)
    for a, b in zip(gm, gp):
        np.testing.assert_allclose(a, b, rtol=1e-11, atol=1e-11)


@pytest.mark.parametrize("n,d,r", SHAPES[:4])
def test_memo_forward_and_backward_match_library_embedding_bag_on_the_dense_table(rng, n, d, r):
    # forward: embedding_bag(sum) on the brute-force table; backward: autograd through an einsum chain of the cores
    N = int(np.prod(n))
    cores = rand_cores(rng, n, d, r)
    idx, off = ragged_batch(rng, N, 11, 6)
    W = torch.from_numpy(oracle.dense(n, d, r, cores))
    ref = torch.nn.functional.embedding_bag(torch.from_numpy(idx), W, torch.from_numpy(off[:-1]), mode="sum")
    got = oracle.forward(n, d, r, N, cores, idx, off, memo=True)
    np.testing.assert_allclose(got, ref.numpy(), rtol=1e-11, atol=1e-11)
    K = len(n)
    tc = [torch.from_numpy(c).clone().requires_grad_(True) for c in cores]
    full = tc[0][0]
    for k in range(1, K):
        full = torch.einsum("...a,anjb->...njb", full, tc[k])
    full = full[..., 0]
    perm = [2 * k for k in range(K)] + [2 * k + 1 for k in range(K)]
    Wt = full.permute(*perm).reshape(N, int(np.prod(d)))
    go = rng.normal(size=(11, int(np.prod(d))))
    out = torch.nn.functional.embedding_bag(torch.from_numpy(idx), Wt, torch.from_numpy(off[:-1]), mode="sum")
    (out * torch.from_numpy(go)).sum().backward()
    gm = oracle.backward(n, d, r, N, cores, idx, off, go, memo=True)
    for a, b in zip(gm, tc):
        np.testing.assert_allclose(a, b.grad.numpy(), rtol=1e-10, atol=1e-11)


def test_memo_backward_exact_finite_difference(rng):
    # the loss sum(grad_out * out) is linear in every single core entry: a finite difference of any step is exact
    n, d, r = (3, 2, 4), (2, 3, 2), (1, 3, 5, 1)
    N = int(np.prod(n))
    cores = rand_cores(rng, n, d, r)
    idx, off = ragged_batch(rng, N, 9, 5)
    go = rng.normal(size=(9, int(np.prod(d))))
    g = oracle.backward(n, d, r, N, cores, idx, off, go, memo=True)
    base = float((oracle.forward(n, d, r, N, cores, idx, off, memo=True) * go).sum())
    for k in range(3):
        for _ in range(12):
            pos = tuple(int(rng.integers(s)) for s in cores[k].shape)
            for step in (1e-3, 1.0, 37.0):
                c2 = [c.copy() for c in cores]
                c2[k][pos] += step
                fd = (float((oracle.forward(n, d, r, N, c2, idx, off, memo=True) * go).sum()) - base) / step
                assert abs(fd - g[k][pos]) <= 1e-9 * max(1.0, abs(g[k][pos]))


@pytest.mark.parametrize("cfg", [1, 2, 3, 4, 5])
def test_memo_equals_plain_on_tiny_configs(cfg):
    wl = workloads.make(cfg, tiny=True)
    np.testing.assert_allclose(oracle.forward_workload(wl, memo=True), oracle.forward_workload(wl), rtol=1e-12, atol=1e-13)
    if cfg == 5:
        for tm, tp in zip(oracle.backward_workload(wl, memo=True), oracle.backward_workload(wl)):
            for a, b in zip(tm, tp):
                np.testing.assert_allclose(a, b, rtol=1e-11, atol=1e-12)


def test_memo_equals_plain_on_a_reduced_multi_table_training_batch():
    # the 60-table recipe with 6 tables and 192 bags: real table sizes (up to 10^7 rows), real skew, ~10^4 lookups
    wl = workloads.make(5, num_tables=6, batch=192)
    np.testing.assert_allclose(oracle.forward_workload(wl, memo=True), oracle.forward_workload(wl), rtol=1e-12, atol=1e-13)
    for tm, tp in zip(oracle.backward_workload(wl, memo=True), oracle.backward_workload(wl)):
        for a, b in zip(tm, tp):
            np.testing.assert_allclose(a, b, rtol=1e-10, atol=1e-12)


def test_memo_four_core_medium_case():
    spec = TableSpec(4096, (8, 8, 8, 8), (2, 4, 4, 4), (1, 6, 7, 5, 1), 1.2, "normal", 0.3)
    wl = workloads.custom([spec], 64, (0, 12), seed=77, with_grad=True)
    np.testing.assert_allclose(oracle.forward_workload(wl, memo=True), oracle.forward_workload(wl), rtol=1e-12, atol=1e-13)
    for a, b in zip(oracle.backward_workload(wl, memo=True)[0], oracle.backward_workload(wl)[0]):
        np.testing.assert_allclose(a, b, rtol=1e-11, atol=1e-12)


def _every_kth_bag(wl, stride):
    """The workload restricted to bags 0, stride, 2*stride, ... of every table (same tables and cores)."""
    bags = np.arange(0, wl.B, stride)
    idx_parts, lens = [], []
    for t in range(wl.T):
        idx, off = wl.table_slice(t)
        lens.append((off[1:] - off[:-1])[bags])
        idx_parts.extend(idx[off[b]:off[b + 1]] for b in bags)
    offsets = np.concatenate([[0], np.cumsum(np.concatenate(lens))]).astype(np.int64)
    return workloads.Workload(name=wl.name + f"-every{stride}", tables=wl.tables, B=len(bags),
                              indices=np.concatenate(idx_parts).astype(np.int64), offsets=offsets, cores=wl.cores,
                              grad_out=wl.grad_out[bags], lr=wl.lr, mapping=wl.mapping)


def test_memo_equals_plain_on_every_64th_bag_of_the_full_training_configuration():
    # the 60-table, 99-million-lookup batch the GPU tests compare in full with the memoised oracle: on every 64th bag
    # of every table (1.5 million lookups) the plain per-lookup oracle is affordable, and the two must agree
    sub = _every_kth_bag(workloads.make(5), 64)
    assert sub.T == 60 and sub.B == 512 and sub.L > 1_000_000
    ref = oracle.forward_workload(sub)
    np.testing.assert_allclose(oracle.forward_workload(sub, memo=True), ref, rtol=1e-11, atol=1e-13 * np.abs(ref).max())
    for tm, tp in zip(oracle.backward_workload(sub, memo=True), oracle.backward_workload(sub)):
        for a, b in zip(tm, tp):
            np.testing.assert_allclose(a, b, rtol=1e-9, atol=1e-12 * max(np.abs(b).max(), 1e-300))
