"""Pins of the oracle's steps beyond the worker-side pass: the uniform-ratio policy (Section 3.1), the
receiver's estimator update and the model step (Algorithm 1, server lines).  Each is checked against
something other than itself: the hand-computed example, brute force, numpy float32 arithmetic, the
sender/receiver identity of EF21, a closed form."""
import os

import numpy as np
import pytest

from oracle import kimad_oracle as ko

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "three_layer_example.txt")


def _golden_uniform():
    layers, grid, cases = [], None, []
    for line in open(GOLDEN):
        t = line.split()
        if not t or t[0].startswith("#"):
            continue
        if t[0] == "layer":
            layers.append(np.float32([float(x) for x in t[2:]]))
        elif t[0] == "grid":
            grid = [float(x) for x in t[1:]]
        elif t[0] == "uniform":
            f = [s.split() for s in line[len("uniform"):].split(":")]
            cases.append((int(f[0][0]), int(f[1][0]), [int(x) for x in f[2]], float(f[3][0]), int(f[4][0])))
    return layers, grid, cases


def test_uniform_policy_hand_example():
    layers, grid, cases = _golden_uniform()
    assert len(cases) == 6
    sizes = [x.size for x in layers]
    d = np.concatenate(layers)[None]
    for c, j, k, err, status in cases:
        res = ko.step(sizes, 1, grid, 1000, 0, d, np.zeros_like(d), [float(c)], 1.0, policy=1)
        assert res.status[0] == status
        assert list(res.j[0]) == [j] * 3 and list(res.k[0]) == k
        assert float(res.total_err[0]) == err
        if status != ko.STATUS_INFEASIBLE:
            assert int(res.used_bytes[0]) <= c


@pytest.mark.parametrize("seed", range(5))
def test_uniform_policy_brute_force(seed):
    rng = np.random.default_rng(seed)
    L, K = int(rng.integers(1, 9)), int(rng.integers(1, 7))
    sizes = rng.integers(1, 400, L)
    grid = np.sort(rng.uniform(0.01, 1.0, K))
    grid[-1] = 1.0 if seed % 2 else grid[-1]
    kt = ko.k_table(sizes, grid)
    for vd, bpe in ((0, 8), (1, 6)):
        totals = [int(kt[:, j].sum()) * bpe for j in range(K)]
        for c in sorted({0, 1, *totals, *[t - 1 for t in totals], *[t + 1 for t in totals], 10 ** 9}):
            fits = [j for j in range(K) if totals[j] <= c]
            status, j = ko.uniform(kt, vd, c)
            if not fits:
                assert (status, j) == (ko.STATUS_INFEASIBLE, 0)
            else:
                assert j == max(fits)
                assert status == (ko.STATUS_PLATEAU if j == K - 1 else ko.STATUS_OK)


def test_layer_adaptive_search_never_worse_than_uniform():
    """Section 4.3: at the same budget the layer-adaptive choice has at most the uniform choice's error,
    whenever the uniform assignment also fits the discretised budget (the ceil of the cells can exclude it)."""
    rng = np.random.default_rng(7)
    sizes = [300, 50, 1200, 7, 640]
    grid = [0.05, 0.1, 0.2, 0.4, 0.8]
    D = 1000
    kt = ko.k_table(sizes, grid)
    checked = 0
    for trial in range(20):
        d = (rng.standard_normal(sum(sizes)) * np.repeat(rng.uniform(0.01, 10, len(sizes)), sizes)).astype(np.float32)[None]
        c = float(rng.integers(200, 16000))
        uni = ko.step(sizes, 1, grid, D, 0, d, np.zeros_like(d), [c], 1.0, policy=1)
        dp = ko.step(sizes, 1, grid, D, 0, d, np.zeros_like(d), [c], 1.0, policy=0)
        if uni.status[0] != ko.STATUS_OK:
            continue
        status, units = ko.units(kt, 0, int(c), D)
        if sum(int(units[l, uni.j[0, l]]) for l in range(len(sizes))) > D:
            continue
        assert float(dp.total_err[0]) <= float(uni.total_err[0])
        checked += 1
    assert checked >= 5


@pytest.mark.parametrize("value_dtype", [0, 1])
def test_receiver_copy_tracks_the_senders_estimator(value_dtype):
    """EF21 keeps u^_m identical on both ends: adding every message to the receiver's copy reproduces the
    sender's state bit for bit, over several rounds."""
    rng = np.random.default_rng(3 + value_dtype)
    sizes = [257, 4, 1000, 33]
    grid = [0.02, 0.1, 0.5, 1.0]
    N = sum(sizes)
    W = 2
    state = np.zeros((W, N), np.float32)
    copy = np.zeros((W, N), np.float32)
    for rnd in range(4):
        grads = rng.standard_normal((W, N)).astype(np.float32)
        res = ko.step(sizes, W, grid, 1000, value_dtype, grads, state, [3000.0 + 900 * rnd, 700.0], 1.0)
        for w in range(W):
            copy[w] = ko.apply_packed(sizes, res.idx[w], res.val[w], res.offs[w], value_dtype, copy[w])
        state = res.state
        assert np.array_equal(copy.view(np.uint32), state.view(np.uint32))


def test_apply_packed_matches_numpy_scatter_add():
    sizes = [5, 3]
    idx = np.uint32([1, 4, 0, 2])      # layer 0: entries 1, 4; layer 1: entries 0, 2
    val = np.float32([0.5, -2.0, 3.25, 1e-3])
    offs = np.uint64([0, 2, 4])
    est = np.float32([1, 1, 1, 1, 1, 10, 10, 10])
    want = est.copy()
    np.add.at(want, [1, 4, 5 + 0, 5 + 2], val)
    assert np.array_equal(ko.apply_packed(sizes, idx, val, offs, 0, est), want)
    with pytest.raises(Exception):
        ko.apply_packed(sizes, np.uint32([5, 0, 0, 0]), val, offs, 0, est)  # index outside its layer


def test_aggregate_matches_float32_recomputation_and_closed_form():
    rng = np.random.default_rng(11)
    W, N = 5, 1003
    est = rng.standard_normal((W, N)).astype(np.float32)
    x = rng.standard_normal(N).astype(np.float32)
    w = rng.uniform(0.1, 1.0, W).astype(np.float32)
    gamma = np.float32(0.37)
    acc = np.zeros(N, np.float32)
    for m in range(W):
        acc = acc + w[m] * est[m]          # float32 product, then float32 sum
    want = x - gamma * acc
    got = ko.aggregate(x, est, w, float(gamma))
    assert got.dtype == np.float32 and np.array_equal(got, want)
    # equal estimators, weights 1/2 + 1/2, gamma a power of two: exact
    e = rng.integers(-1000, 1000, N).astype(np.float32)
    got = ko.aggregate(np.ones(N, np.float32), np.stack([e, e]), [0.5, 0.5], 0.25)
    assert np.array_equal(got, 1.0 - 0.25 * e)
    # hand example: the c = 96, D = 12 allocation keeps A[5:], all of B, C[:3]
    est1 = np.float32([0, 0, 0, 0, 0, 6, 7, 8, 9, 10, -8, 0.5, 8, -0.5, 3, -3, 3, 0, 0, 0])
    got = ko.aggregate(np.zeros(20, np.float32), est1[None], [1.0], 0.5)
    assert np.array_equal(got, -0.5 * est1)
    layers, grid, _ = _golden_uniform()
    d = np.concatenate(layers)[None]
    res = ko.step([x.size for x in layers], 1, grid, 12, 0, d, np.zeros_like(d), [96.0], 1.0)
    recv = ko.apply_packed([x.size for x in layers], res.idx[0], res.val[0], res.offs[0], 0, np.zeros(20, np.float32))
    assert np.array_equal(recv, est1)


def test_error_axis_dp_hand_example():
    layers, grid, _ = _golden_uniform()
    cases = []
    for line in open(GOLDEN):
        if line.startswith("erroraxis"):
            f = [s.split() for s in line[len("erroraxis"):].split(":")]
            cases.append((int(f[0][0]), int(f[0][1]), [int(x) for x in f[1]], int(f[2][0]), int(f[3][0])))
    assert len(cases) == 4
    sizes = [x.size for x in layers]
    kt = ko.k_table(sizes, grid)
    d = np.concatenate(layers)[None]
    for c, D, k, cell, status in cases:
        res = ko.step(sizes, 1, grid, D, 0, d, np.zeros_like(d), [float(c)], 1.0, policy=2)
        assert res.status[0] == status and list(res.k[0]) == k
        st, j, got_cell = ko.dp_error_axis(res.err[0], kt, D, 0, c)
        assert st == status and (status != ko.STATUS_OK or got_cell == cell)


@pytest.mark.parametrize("seed", range(4))
def test_error_axis_dp_brute_force(seed):
    """Every assignment enumerated: the DP returns the lowest discretised error level that fits the budget and,
    at that level, the fewest kept entries."""
    import itertools
    rng = np.random.default_rng(100 + seed)
    for trial in range(40):
        L, K = int(rng.integers(1, 6)), int(rng.integers(1, 5))
        D = int(rng.integers(max(L, 2), 40))
        sizes = rng.integers(1, 60, L)
        grid = np.sort(rng.uniform(0.05, 1, K))
        kt = ko.k_table(sizes, grid)
        err = np.sort(rng.uniform(0, 10, (L, K)).astype(np.float32), axis=1)[:, ::-1].copy()
        vd = trial % 2
        bpe = 6 if vd else 8
        c = int(rng.integers(0, int(kt[:, -1].sum()) * bpe + 20))
        st, j, cell = ko.dp_error_axis(err, kt, D, vd, c)
        emax = 0.0
        for l in range(L):
            emax = emax + float(err[l, 0])
        cells = [[int(np.floor(float(err[l, q]) * float(D) / emax)) if emax > 0 else 0 for q in range(K)] for l in range(L)]
        if c >= int(kt[:, -1].sum()) * bpe:
            assert st == ko.STATUS_PLATEAU and all(j == K - 1)
            continue
        best = None
        for a in itertools.product(range(K), repeat=L):
            e = sum(cells[l][a[l]] for l in range(L))
            b = sum(int(kt[l, a[l]]) for l in range(L)) * bpe
            assert e <= D  # rounding down keeps every assignment on the axis
            if b <= c and (best is None or (e, b) < best):
                best = (e, b)
        if best is None:
            assert st == ko.STATUS_INFEASIBLE and all(j == 0)
        else:
            assert st == ko.STATUS_OK and cell == best[0]
            assert sum(int(kt[l, j[l]]) for l in range(L)) * bpe == best[1]
            assert sum(cells[l][j[l]] for l in range(L)) == best[0]
