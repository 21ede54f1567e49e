"""Pins of the oracle's Kimad ratio sized to the budget (Section 3.1; O9b) and of the sizes with a dense
fallback (O13), against something other than themselves: the hand-computed lines of the golden example, exact
rational arithmetic over every breakpoint of the ratio, closed forms, exhaustive enumeration."""
import itertools
import os
from fractions import Fraction

import numpy as np
import pytest

from oracle import kimad_oracle as ko

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "three_layer_example.txt")


def _golden(tag):
    layers, grid, cases = [], None, []
    for line in open(GOLDEN):
        t = line.split()
        if not t or t[0].startswith("#"):
            continue
        if t[0] == "layer":
            layers.append(np.float32([float(x) for x in t[2:]]))
        elif t[0] == "grid":
            grid = [float(x) for x in t[1:]]
        elif t[0] == tag:
            cases.append([[float(x) for x in s.split()] for s in line[len(tag):].split(":")])
    return layers, grid, cases


# ----------------------------------------------------------------------------- O9b
def test_fitted_ratio_hand_example():
    layers, _, cases = _golden("fitted")
    assert len(cases) == 6
    sizes = [x.size for x in layers]
    d = np.concatenate(layers)[None]
    for (c,), k, (err,), (used,), (status,) in cases:
        r = ko.step(sizes, 1, [1.0], 1000, 0, d, np.zeros_like(d), [c], 1.0, policy=3)
        assert r.k[0].tolist() == [int(x) for x in k], c
        assert float(r.total_err[0]) == err
        assert int(r.used_bytes[0]) == int(used) and int(r.status[0]) == int(status)
        assert int(r.budget_bytes[0]) == int(c)


def _fit_by_breakpoints(sizes, entries):
    """The definition with exact rationals: walk the breakpoints m / n_l of r -> sum_l max(1, floor(r n_l)) in
    ascending order; the answer is the k-vector just before the first breakpoint whose sum exceeds `entries`."""
    k_at = lambda r: [min(n, max(1, (r.numerator * n) // r.denominator)) for n in sizes]
    points = sorted({Fraction(m, n) for n in sizes for m in range(1, n + 1)})
    best = k_at(Fraction(0))
    if sum(best) > entries:
        return None
    for r in points:
        k = k_at(r)
        if sum(k) > entries:
            break
        best = k
    return best


@pytest.mark.parametrize("seed", range(8))
def test_fitted_ratio_against_exact_rationals(seed):
    rng = np.random.default_rng(seed)
    sizes = [int(x) for x in rng.integers(1, 60, int(rng.integers(1, 6)))]
    N = sum(sizes)
    for entries in range(0, N + 3):
        status, q, k = ko.fit_ratio(sizes, entries)
        want = _fit_by_breakpoints(sizes, entries)
        if want is None:
            assert status == ko.STATUS_INFEASIBLE and k.tolist() == [1] * len(sizes) and q == 0
            continue
        assert k.tolist() == want, (sizes, entries)
        assert status == (ko.STATUS_PLATEAU if entries >= N else ko.STATUS_OK)
        assert sum(want) <= entries
        # k really is floor(q n / 2^32) for the returned q, and q + 1 would not fit (or q is the top)
        assert k.tolist() == [min(n, max(1, (q * n) >> 32)) for n in sizes]
        if status == ko.STATUS_OK:
            assert sum(min(n, max(1, ((q + 1) * n) >> 32)) for n in sizes) > entries


def test_fitted_ratio_one_layer_is_whole_model_topk():
    """With one layer spanning the model the fitted ratio keeps exactly K = floor(c / 8) entries (Section 4.3:
    TopK with the whole model information), for every K between 1 and N."""
    for N in (1, 7, 1000, 50257 * 768, 2 ** 32 - 1):
        for entries in {1, 2, 3, N // 3, N - 1, N, N + 5} - {0}:
            status, q, k = ko.fit_ratio([N], entries)
            assert int(k[0]) == min(N, entries)
    rng = np.random.default_rng(4)
    d = (rng.standard_normal((1, 5000)) * np.exp(rng.uniform(-3, 3, (1, 5000)))).astype(np.float32)
    r = ko.step([5000], 1, [1.0], 1000, 0, d, np.zeros_like(d), [8.0 * 321 + 5], 1.0, policy=3)
    assert int(r.k[0, 0]) == 321
    want = np.sort(np.argsort(-np.abs(d[0]), kind="stable")[:321])
    assert np.array_equal(r.idx[0, :321], want.astype(np.uint32))


def test_fitted_ratio_uses_the_budget_better_than_the_grid():
    """The grid variant (policy 1) may leave a large part of c unused; the fitted ratio leaves less than one entry
    per layer (the next breakpoint adds at most one entry to each layer)."""
    sizes = [40000, 300, 7000, 12, 90000]
    L, N = len(sizes), sum(sizes)
    grid = [10 ** (-3 + 3 * j / 15) for j in range(16)]
    kt = ko.k_table(sizes, grid)
    for frac in (0.003, 0.02, 0.11, 0.37, 0.8):
        c = int(frac * 8 * N)
        st_g, j = ko.uniform(kt, 0, c)
        st_f, q, k = ko.fit_ratio(sizes, c // 8)
        used_f = 8 * int(k.sum())
        assert used_f <= c and c - used_f < 8 * (L + 1)
        if st_g == ko.STATUS_OK:
            assert 8 * int(kt[:, j].sum()) <= used_f + 8 * L  # ceil on the grid against floor here: L entries at most


# ----------------------------------------------------------------------------- O13
def test_dense_fallback_hand_example():
    layers, grid, cases = _golden("dense")
    assert len(cases) == 4
    sizes = [x.size for x in layers]
    d = np.concatenate(layers)[None]
    for (c, D), k, dense, (err,), (used,), (status,) in cases:
        r = ko.step(sizes, 1, grid, int(D), 0, d, np.zeros_like(d), [c], 1.0, cost_model=1)
        assert r.k[0].tolist() == [int(x) for x in k], (c, D)
        assert r.dense[0].tolist() == [int(x) for x in dense]
        assert float(r.total_err[0]) == err and int(r.used_bytes[0]) == int(used) and int(r.status[0]) == int(status)
        # a dense layer is sent whole, in index order, and the estimator then equals the gradient there
        off = 0
        for l, n in enumerate(sizes):
            if r.dense[0, l]:
                o = int(r.offs[0, l])
                assert r.idx[0, o:o + n].tolist() == list(range(n))
                assert np.array_equal(r.val[0, o:o + n], d[0, off:off + n])
                assert np.array_equal(r.state[0, off:off + n], d[0, off:off + n])
            off += n


@pytest.mark.parametrize("vd,vb", [(0, 4), (1, 2)])
def test_candidate_sizes_closed_form(vd, vb):
    for n in (1, 2, 3, 10, 1001):
        for k in range(1, n + 1):
            assert ko.candidate(n, k, vd, 0) == (k * (4 + vb), k, 0)
            b, ke, dn = ko.candidate(n, k, vd, 1)
            if k * (4 + vb) >= vb * n:      # f32: k >= n/2; bf16: k >= n/3
                assert (b, ke, dn) == (vb * n, n, 1)
            else:
                assert (b, ke, dn) == (k * (4 + vb), k, 0)
            assert b == min(k * (4 + vb), vb * n)


@pytest.mark.parametrize("seed", range(6))
def test_dense_fallback_exhaustive(seed):
    """All K^L assignments with the cost model's sizes and errors, summed left to right in binary32: the step's
    decision is the first assignment (candidates ascending, cells ascending) that attains the minimum."""
    rng = np.random.default_rng(100 + seed)
    L, K, D = int(rng.integers(2, 5)), int(rng.integers(2, 5)), int(rng.integers(8, 40))
    sizes = [int(x) for x in rng.integers(3, 50, L)]
    grid = np.sort(rng.uniform(0.05, 1.0, K))
    vd = seed % 2
    vb = 4 if vd == 0 else 2
    d = (rng.standard_normal((1, sum(sizes))) * np.repeat(np.exp(rng.uniform(-2, 2, L)), sizes)).astype(np.float32)
    kt = ko.k_table(sizes, grid)
    for frac in (0.2, 0.45, 0.7):
        c = int(frac * vb * sum(sizes)) + 1
        r = ko.step(sizes, 1, grid, D, vd, d, np.zeros_like(d), [float(c)], 1.0, cost_model=1)
        byt = np.array([[ko.candidate(sizes[l], int(kt[l, j]), vd, 1)[0] for j in range(K)] for l in range(L)], np.uint64)
        dns = np.array([[ko.candidate(sizes[l], int(kt[l, j]), vd, 1)[2] for j in range(K)] for l in range(L)])
        err = np.where(dns == 1, np.float32(0), r.err[0]).astype(np.float32)
        if c >= int(byt[:, -1].sum()):
            assert r.status[0] == ko.STATUS_PLATEAU
            continue
        cells = (byt * np.uint64(D) + np.uint64(c - 1)) // np.uint64(c)
        best = None
        for js in itertools.product(range(K), repeat=L):
            cc = sum(int(cells[l, j]) for l, j in enumerate(js))
            if cc > D or any(int(cells[l, j]) > D for l, j in enumerate(js)):
                continue
            tot = np.float32(0)
            for l, j in enumerate(js):
                tot = np.float32(tot + err[l, j])
            if best is None or tot < best[0]:
                best = (tot, js)
        if best is None:
            assert r.status[0] == ko.STATUS_INFEASIBLE
            continue
        assert r.status[0] == ko.STATUS_OK
        assert r.total_err[0].view(np.uint32) == best[0].view(np.uint32)   # the optimum's value, bit for bit
        assert int(r.used_bytes[0]) == sum(int(byt[l, j]) for l, j in enumerate(r.j[0])) <= c
        for l in range(L):
            assert int(r.k[0, l]) == (sizes[l] if r.dense[0, l] else int(kt[l, r.j[0, l]]))


def test_cost_model_and_policy_combinations_are_validated():
    d = np.zeros((1, 20), np.float32)
    with pytest.raises(RuntimeError):
        ko.step([20], 1, [0.5, 1.0], 10, 0, d, d, [50.0], 1.0, policy=3)          # the fitted ratio takes one candidate
    with pytest.raises(RuntimeError):
        ko.step([20], 1, [1.0], 10, 0, d, d, [50.0], 1.0, policy=3, cost_model=1)
    with pytest.raises(RuntimeError):
        ko.step([20], 1, [0.5, 1.0], 10, 0, d, d, [50.0], 1.0, policy=2, cost_model=1)
