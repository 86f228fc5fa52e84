"""Stored expected values: a hand-worked example, and a frozen snapshot written by the oracle itself."""
import os

import numpy as np

import oracle
import workloads

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _read(name):
    d = {}
    for line in open(os.path.join(GOLD, name)):
        if line.startswith("#") or not line.strip():
            continue
        k, *v = line.split()
        d[k] = np.array([float(x) for x in v])
    return d


def test_hand_worked_example():
    g = _read("hand_worked_k2.txt")
    n, d, r = (2, 2), (1, 2), (1, 2, 1)
    G1 = np.array([[1., 2.], [3., 4.]]).reshape(1, 2, 1, 2)
    G2 = np.zeros((2, 2, 2, 1))
    G2[0, 0, :, 0] = [1, 0]; G2[1, 0, :, 0] = [0, 1]; G2[0, 1, :, 0] = [2, 1]; G2[1, 1, :, 0] = [1, 3]
    rows = np.concatenate([oracle.row(n, d, r, [G1, G2], i) for i in range(4)])
    np.testing.assert_array_equal(rows, g["rows"])
    idx = np.array([0, 3, 3, 1, 2]); off = np.array([0, 3, 5, 5])
    np.testing.assert_array_equal(oracle.forward(n, d, r, 4, [G1, G2], idx, off).reshape(-1), g["out"])
    go = np.array([[1., 0.], [0., 1.], [5., 5.]])
    dG1, dG2 = oracle.backward(n, d, r, 4, [G1, G2], idx, off, go)
    np.testing.assert_array_equal(dG1.reshape(-1), g["dG1"])
    np.testing.assert_array_equal(dG2[0].reshape(-1), g["dG2_a0"])
    np.testing.assert_array_equal(dG2[1].reshape(-1), g["dG2_a1"])


def test_frozen_snapshot_of_tiny_configs():
    g = _read("oracle_cfg_tiny.txt")
    for cfg in (1, 2, 3, 4, 5):
        wl = workloads.make(cfg, tiny=True)
        out = oracle.forward_workload(wl)
        vals = np.array([out.sum(), (out ** 2).sum(), *out[0, :4]])
        np.testing.assert_allclose(vals, g[f"cfg{cfg}"], rtol=1e-12, atol=1e-14)
        if wl.grad_out is not None:   # per table: the sum of all its core-gradient entries (plain and memoised oracle)
            for memo in (False, True):
                sums = [sum(float(c.sum()) for c in tg) for tg in oracle.backward_workload(wl, memo=memo)]
                np.testing.assert_allclose(sums, g[f"cfg{cfg}_grad_sums"], rtol=1e-10, atol=1e-13)
