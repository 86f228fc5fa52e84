"""Seeded random shapes against the oracle: core counts, row / dim factors, ranks, batch sizes and pooling laws that no
hand-picked case covers (ranks that are not multiples of 8, first dim factor 1, 2 or 4, last dim factor 4 or not, tables
of different shape variants behind one handle, empty bags, hot rows).  Forward and backward, the tolerance of the path."""
import numpy as np
import pytest

import oracle
import workloads
from workloads import TableSpec

pytestmark = pytest.mark.gpu
TOL = 1e-5


@pytest.fixture(scope="module")
def binding():
    from paper_2609_03459_b200 import binding as b
    return b


def dev(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def close(got, ref, what):
    ref = np.asarray(ref, dtype=np.float64)
    got = np.asarray(got, dtype=np.float64)
    assert got.shape == ref.shape, (what, got.shape, ref.shape)
    scale = np.abs(ref).max() if ref.size else 0.0
    err = np.abs(got - ref).max() if ref.size else 0.0
    if scale == 0.0:
        assert err == 0.0, f"{what}: reference is all zero but max|got| = {err}"
    else:
        assert err <= TOL * scale, f"{what}: max|err| = {err:.3e} > 1e-5 * {scale:.3e}"


def random_case(seed):
    rng = np.random.default_rng(1000 + seed)
    K = int(rng.choice([2, 3, 3, 3, 4]))
    # all tables of a handle share K and D: draw the dim factors once, ranks and row factors per table
    if rng.random() < 0.6:
        d = tuple(int(x) for x in rng.choice([[4, 4, 4], [2, 4, 4], [2, 2, 4], [4, 8, 4]])) if K == 3 else \
            ((8, 8) if K == 2 else (2, 4, 4, 4))
    else:
        d = tuple(int(rng.integers(1, 6)) for _ in range(K))
    T = int(rng.integers(1, 4))
    tables = []
    for _ in range(T):
        n = tuple(int(rng.integers(3, 40)) for _ in range(K))
        N = int(np.prod(n)) - int(rng.integers(0, max(1, n[-1] - 1)))
        if rng.random() < 0.6:
            ranks = [int(rng.choice([8, 16, 32])) for _ in range(K - 1)]
        else:
            ranks = [int(rng.integers(1, 40)) for _ in range(K - 1)]
        r = (1,) + tuple(ranks) + (1,)
        tables.append(TableSpec(N, n, d, r, float(rng.uniform(0.3, 1.3)), "normal", 0.1))
    B = int(rng.integers(1, 200))
    pooling = (0, int(rng.integers(1, 60))) if rng.random() < 0.7 else int(rng.integers(1, 30))
    return tables, B, pooling


@pytest.mark.parametrize("seed", range(24))
def test_random_shape_forward_backward(binding, seed):
    tables, B, pooling = random_case(seed)
    wl = workloads.custom(tables, B, pooling, seed=500 + seed, with_grad=True, name=f"random-{seed}")
    if wl.L and seed % 3 == 0:      # a hot row: a fifth of the lookups of table 0 hit one row
        idx, _ = wl.table_slice(0)
        lo = int(wl.offsets[0])
        hot = np.random.default_rng(seed).random(idx.shape[0]) < 0.2
        wl.indices[lo:lo + idx.shape[0]][hot] = tables[0].N // 2
    emb = binding.from_workload(wl, enable_backward=True)
    out = emb.forward(dev(wl.indices), dev(wl.offsets), wl.B).cpu().numpy()
    assert emb.status() == 0
    close(out, oracle.forward_workload(wl), f"random {seed} out")
    emb.backward(dev(wl.grad_out))
    grads = emb.get_grads()
    ref = oracle.backward_workload(wl)
    for t in range(wl.T):
        for k in range(wl.tables[t].K):
            close(grads[t][k], ref[t][k], f"random {seed} dG[{t}][{k}] (d={tables[t].d}, r={tables[t].r}, n={tables[t].n})")


@pytest.mark.parametrize("seed", range(24, 40))
def test_random_shape_weighted_mean_int32(binding, seed):
    # the same draw of shapes under the other pooling laws, ids handed over as int32 on the even seeds
    tables, B, pooling = random_case(seed)
    wl = workloads.custom(tables, B, pooling, seed=500 + seed, with_grad=True, name=f"random-{seed}")
    weighted = seed % 4 < 2
    wts = np.random.default_rng(seed).normal(size=wl.L).astype(np.float32) if weighted else None
    mode = "sum" if weighted else "mean"
    emb = binding.from_workload(wl, enable_backward=True, enable_weighted=True)
    emb.set_pooling(mode, None if wts is None else dev(wts))
    ids = wl.indices.astype(np.int32) if seed % 2 == 0 else wl.indices
    out = emb.forward(dev(ids), dev(wl.offsets), wl.B).cpu().numpy()
    assert emb.status() == 0
    close(out, oracle.forward_workload(wl, weights=wts, mode=mode), f"random {seed} {mode} out")
    emb.backward(dev(wl.grad_out))
    grads = emb.get_grads()
    ref = oracle.backward_workload(wl, weights=wts, mode=mode)
    for t in range(wl.T):
        for k in range(wl.tables[t].K):
            close(grads[t][k], ref[t][k], f"random {seed} {mode} dG[{t}][{k}] (d={tables[t].d}, r={tables[t].r}, n={tables[t].n})")


@pytest.mark.parametrize("seed", range(40, 64))
def test_random_shape_fused_backward_sgd(binding, seed):
    # every shape class finalises its gradients in another kernel: the fused update must reach each core exactly once
    tables, B, pooling = random_case(seed)
    wl = workloads.custom(tables, B, pooling, seed=500 + seed, with_grad=True, name=f"random-{seed}")
    lr = 0.05
    emb = binding.from_workload(wl, enable_backward=True)
    emb.forward(dev(wl.indices), dev(wl.offsets), wl.B)
    emb.backward_sgd(dev(wl.grad_out), lr)
    assert emb.status() == 0
    grads = emb.get_grads()
    cores = emb.get_cores()
    ref = oracle.backward_workload(wl)
    for t in range(wl.T):
        want = oracle.sgd(wl.cores[t], ref[t], lr)
        for k in range(wl.tables[t].K):
            what = f"(d={tables[t].d}, r={tables[t].r}, n={tables[t].n})"
            close(grads[t][k], ref[t][k], f"random {seed} fused dG[{t}][{k}] {what}")
            # the update itself is exact in the gradient: compare the applied step with lr * gradient
            step = (np.asarray(wl.cores[t][k], np.float64) - np.asarray(cores[t][k], np.float64))
            want_step = lr * np.asarray(ref[t][k], np.float64)
            slack = TOL * np.abs(want_step).max() + 2.0 ** -23 * np.abs(np.asarray(wl.cores[t][k])).max()   # + the rounding of the fp32 core
            assert np.abs(step - want_step).max() <= slack, f"random {seed} fused step[{t}][{k}] {what}"
            close(cores[t][k], want[k], f"random {seed} core[{t}][{k}] after the fused step {what}")
