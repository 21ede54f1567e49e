"""Pins for the CPU oracle: each oracle routine is checked against something other than itself --
a library routine, a closed form, brute force, or the hand-computed example under tests/golden/."""
import itertools
import math
import os
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import kimad_oracle as ko

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "three_layer_example.txt")


# ----------------------------------------------------------------------------- brute-force helpers
def keys_of(d):
    return np.ascontiguousarray(d, np.float32).view(np.uint32) & np.uint32(0x7FFFFFFF)


def bf_order(d):
    """Indices by (|x| descending, index ascending) via Python's sort on tuples."""
    k = keys_of(d)
    return [i for _, i in sorted((-int(k[i]), i) for i in range(len(k)))]


def bf_err(d, k):
    """Exact (rational) sum of squares of the n-k smallest-magnitude entries."""
    order = bf_order(d)
    return sum((Fraction(float(d[i])) ** 2 for i in order[k:]), Fraction(0))


def bf_dp(err, units, D):
    """Exhaustive search over all K^L assignments; objective summed left to right in float32."""
    L, K = err.shape
    best, best_assign, n_best = None, None, 0
    for assign in itertools.product(range(K), repeat=L):
        cells = sum(int(units[l, j]) for l, j in enumerate(assign))
        if cells > D:
            continue
        tot = np.float32(0.0)
        for l, j in enumerate(assign):
            tot = np.float32(tot + err[l, j])
        if best is None or tot < best:
            best, best_assign, n_best = tot, assign, 1
        elif tot == best:
            n_best += 1
    return best, best_assign, n_best


# ----------------------------------------------------------------------------- O1 / O8 / bf16
def test_diff_matches_numpy_float32():
    rng = np.random.default_rng(1)
    a = (rng.standard_normal(10007) * 10.0 ** rng.uniform(-6, 3, 10007)).astype(np.float32)
    b = (rng.standard_normal(10007) * 10.0 ** rng.uniform(-6, 3, 10007)).astype(np.float32)
    d = ko.diff(a, b)
    assert d.dtype == np.float32
    assert np.array_equal(d.view(np.uint32), (a - b).view(np.uint32))
    # sign matters: grad - g, not g - grad
    assert ko.diff(np.float32([3.0]), np.float32([1.0]))[0] == 2.0


def test_bf16_rounding_matches_torch():
    rng = np.random.default_rng(2)
    x = (rng.standard_normal(4000) * 10.0 ** rng.uniform(-8, 8, 4000)).astype(np.float32)
    # exact halfway cases, both parities, and values that carry into the exponent
    special = np.array([0x3F808000, 0x3F818000, 0x3F80FFFF, 0x3FFFFFFF, 0x3F807FFF, 0x3F808001, 0x00000001,
                        0x80008000, 0x7F7F0000, 0x00800000], dtype=np.uint32).view(np.float32)
    x = np.concatenate([x, special, np.float32([0.0, -0.0, 1.0, -1.0])])
    mine = ko.bf16_rne(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(mine, ref)


def test_state_update_matches_numpy():
    rng = np.random.default_rng(3)
    g = rng.standard_normal(500).astype(np.float32)
    idx = np.sort(rng.choice(500, 60, replace=False)).astype(np.uint32)
    val = rng.standard_normal(60).astype(np.float32)
    out = ko.state_update(g, idx, val, 0)
    ref = g.copy()
    ref[idx] = ref[idx] + val
    assert np.array_equal(out.view(np.uint32), ref.view(np.uint32))
    # bf16 mode adds the value that was sent, i.e. the bf16 number widened back to float32
    vb = ko.bf16_rne(val)
    out = ko.state_update(g, idx, vb, 1)
    widened = (vb.astype(np.uint32) << 16).view(np.float32)
    ref = g.copy()
    ref[idx] = ref[idx] + widened
    assert np.array_equal(out.view(np.uint32), ref.view(np.uint32))


# ----------------------------------------------------------------------------- O3
def test_k_table_hand_values():
    kt = ko.k_table([10, 4, 6, 1, 64, 1000], [0.25, 0.5, 1.0])
    assert kt.tolist() == [[3, 5, 10], [1, 2, 4], [2, 3, 6], [1, 1, 1], [16, 32, 64], [250, 500, 1000]]
    kt = ko.k_table([64, 100352, 3], [0.001, 0.01, 0.02])
    # ceil(0.064)=1, ceil(0.64)=1, ceil(1.28)=2 ; 100352*0.001 = 100.352 -> 101 ; tiny layer never below 1
    assert kt.tolist() == [[1, 1, 2], [101, 1004, 2008], [1, 1, 1]]


def test_k_table_exact_ceiling():
    rng = np.random.default_rng(4)
    sizes = rng.integers(1, 5_000_000, 40)
    grid = sorted(set(rng.uniform(1e-4, 1.0, 12).tolist())) + [1.0]
    kt = ko.k_table(sizes, grid)
    for l, n in enumerate(sizes):
        for j, r in enumerate(grid):
            prod = float(r) * float(n)  # the binary64 product, as specified
            want = min(int(n), max(1, math.ceil(Fraction(prod))))
            assert int(kt[l, j]) == want
    assert np.all(np.diff(kt.astype(np.int64), axis=1) >= 0)
    assert np.all(kt[:, -1] == sizes)


def test_k_table_rejects_bad_grid():
    for bad in ([0.5, 0.2], [0.0, 0.5], [0.5, 1.5], [0.3, 0.3]):
        with pytest.raises(RuntimeError):
            ko.k_table([10], bad)


# ----------------------------------------------------------------------------- O2 / O4 / O7
def test_curve_closed_form_ramp():
    n = 1000
    for sign in (1.0, -1.0):
        d = (sign * np.arange(1, n + 1)).astype(np.float32)
        ks = np.array([1, 10, 250, 999, 1000], np.uint64)
        c = ko.layer_curve(d, ks)
        for j, k in enumerate(ks):
            m = n - int(k)
            assert c.err[j] == np.float32(m * (m + 1) * (2 * m + 1) // 6)
            assert c.tau[j] == keys_of(np.float32([n - int(k) + 1]))[0]
            assert c.keep_eq[j] == 1 and c.n_gt[j] == k - 1 and c.n_eq[j] == 1
        idx, val = ko.select_pack(d, 10)
        assert idx.tolist() == list(range(n - 10, n))
        assert np.array_equal(val, d[n - 10:])


def test_curve_shuffled_ramp_is_permutation_invariant():
    rng = np.random.default_rng(5)
    n = 777
    perm = rng.permutation(n)
    d = (perm + 1).astype(np.float32) * np.where(rng.uniform(size=n) < 0.5, -1, 1).astype(np.float32)
    ks = np.array([5, 77, 400, 777], np.uint64)
    c = ko.layer_curve(d, ks)
    for j, k in enumerate(ks):
        m = n - int(k)
        assert c.err[j] == np.float32(m * (m + 1) * (2 * m + 1) // 6)
    idx, _ = ko.select_pack(d, 77)
    assert sorted(idx.tolist()) == idx.tolist()
    assert set(idx.tolist()) == set(np.nonzero(perm + 1 > n - 77)[0].tolist())


@pytest.mark.parametrize("seed", range(6))
def test_curve_and_select_vs_bruteforce_with_ties(seed):
    rng = np.random.default_rng(100 + seed)
    n = int(rng.integers(1, 300))
    # few distinct magnitudes, both signs, exact zeros of both signs: plenty of ties
    pool = np.concatenate([rng.standard_normal(6).astype(np.float32), np.float32([0.0, -0.0, 1e-40, -1e-40])])
    d = rng.choice(pool, n).astype(np.float32)
    d *= np.where(rng.uniform(size=n) < 0.5, -1, 1).astype(np.float32)
    ks = np.unique(np.clip(rng.integers(1, n + 1, 8), 1, n)).astype(np.uint64)
    c = ko.layer_curve(d, ks)
    order = bf_order(d)
    key = keys_of(d)
    for j, k in enumerate(ks):
        k = int(k)
        exact = bf_err(d, k)
        assert c.err[j] == np.float32(float(exact)) or abs(float(c.err[j]) - float(exact)) <= 1e-6 * float(exact)
        t = int(key[order[k - 1]])
        assert int(c.tau[j]) == t
        assert int(c.n_gt[j]) == int(np.sum(key > t))
        assert int(c.n_eq[j]) == int(np.sum(key == t))
        assert int(c.keep_eq[j]) == k - int(np.sum(key > t))
        idx, val = ko.select_pack(d, k)
        assert idx.tolist() == sorted(order[:k])
        assert np.array_equal(val.view(np.uint32), d[idx].view(np.uint32))


def test_curve_matches_fsum_and_lexsort_on_random_data():
    rng = np.random.default_rng(7)
    n = 20000
    d = (rng.standard_t(3, n) * 1e-3).astype(np.float32)
    ks = ko.k_table([n], [0.001, 0.01, 0.1, 0.5, 1.0])[0]
    c = ko.layer_curve(d, ks)
    key = keys_of(d)
    order = np.lexsort((np.arange(n), -key.astype(np.int64)))  # library sort, same total order
    sq = d.astype(np.float64) ** 2
    for j, k in enumerate(ks):
        k = int(k)
        ref = math.fsum(sq[order[k:]].tolist())
        assert abs(float(c.err[j]) - ref) <= 2e-7 * ref + 1e-45
        idx, val = ko.select_pack(d, k)
        assert np.array_equal(idx, np.sort(order[:k]).astype(np.uint32))
    assert c.err[-1] == 0.0 and not np.signbit(c.err[-1])


def test_topk_set_matches_torch_topk_when_tie_free():
    rng = np.random.default_rng(8)
    n = 5000
    mag = rng.permutation(n).astype(np.float32) + 1.0  # distinct magnitudes
    d = mag * np.where(rng.uniform(size=n) < 0.5, -1, 1).astype(np.float32)
    for k in (1, 17, 500, n):
        idx, val = ko.select_pack(d, k)
        ref = torch.topk(torch.from_numpy(d).abs(), k).indices.numpy()
        assert set(idx.tolist()) == set(ref.tolist())
        assert np.array_equal(val, d[idx])


def test_curve_invariants_contractive_bound():
    rng = np.random.default_rng(9)
    n = 4096
    d = (rng.standard_normal(n) * 0.01).astype(np.float32)
    ks = np.arange(1, n + 1, 37, dtype=np.uint64)
    ks[-1] = n
    c = ko.layer_curve(d, ks)
    tot = float(np.sum(d.astype(np.float64) ** 2))
    assert np.all(np.diff(c.err) <= 0)  # non-increasing in k
    assert c.err[-1] == 0.0
    # TopK is contractive with alpha = k/n (the class C(alpha) used by the 3PC lemma)
    for j, k in enumerate(ks):
        assert float(c.err[j]) <= (1.0 - float(k) / n) * tot * (1 + 1e-6)
    # pushing k to 1 approaches the full squared norm minus the largest entry
    c1 = ko.layer_curve(d, np.array([1], np.uint64))
    assert abs(float(c1.err[0]) - (tot - float(np.max(np.abs(d))) ** 2)) <= 1e-6 * tot


def test_select_pack_bf16_values():
    rng = np.random.default_rng(10)
    d = rng.standard_normal(300).astype(np.float32)
    idx0, val0 = ko.select_pack(d, 40, 0)
    idx1, val1 = ko.select_pack(d, 40, 1)
    assert np.array_equal(idx0, idx1)  # selection is on the float32 magnitude in both modes
    ref = torch.from_numpy(val0).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(val1, ref)


# ----------------------------------------------------------------------------- O5
def test_budget_and_units_hand_values():
    assert ko.budget_bytes(125e6, 0.05) == 6_250_000
    assert ko.budget_bytes(40708.0, 1.0) == 40708
    assert ko.budget_bytes(10.9, 1.0) == 10
    assert ko.budget_bytes(0.0, 1.0) == 0
    kt = np.array([[3, 5, 10], [1, 2, 4], [2, 3, 6]], np.uint64)
    st, u = ko.units(kt, 0, 96, 1000)
    assert st == 0 and u.tolist() == [[250, 417, 834], [84, 167, 334], [167, 250, 500]]
    st, u = ko.units(kt, 0, 96, 12)
    assert st == 0 and u.tolist() == kt.tolist()
    st, u = ko.units(kt, 1, 96, 12)  # 6 bytes per entry in bf16 mode: ceil(6k*12/96) = ceil(0.75k)
    assert st == 0 and u.tolist() == [[3, 4, 8], [1, 2, 3], [2, 3, 5]]
    assert ko.units(kt, 0, 160, 1000)[0] == ko.STATUS_PLATEAU
    assert ko.units(kt, 0, 159, 1000)[0] == 0
    assert ko.units(kt, 1, 120, 1000)[0] == ko.STATUS_PLATEAU
    assert ko.units(kt, 0, 0, 1000)[0] == ko.STATUS_INFEASIBLE


# ----------------------------------------------------------------------------- O6
@pytest.mark.parametrize("seed", range(12))
def test_dp_equals_exhaustive_enumeration(seed):
    rng = np.random.default_rng(200 + seed)
    L = int(rng.integers(1, 7))
    K = int(rng.integers(1, 5))
    D = int(rng.integers(4, 40))
    units = np.sort(rng.integers(1, max(2, D // 2), (L, K)), axis=1).astype(np.uint64)
    err = -np.sort(-rng.uniform(0, 10, (L, K)), axis=1)
    err = err.astype(np.float32)
    st, j, val, cell = ko.dp(err, units, D)
    best, assign, n_best = bf_dp(err, units, D)
    if best is None:
        assert st == ko.STATUS_INFEASIBLE and j.tolist() == [0] * L
        return
    assert st == 0
    assert np.float32(val) == best  # bit for bit: float32 addition is monotone
    mine = np.float32(0)
    for l in range(L):
        mine = np.float32(mine + err[l, j[l]])
    assert mine == best
    assert sum(int(units[l, j[l]]) for l in range(L)) == cell <= D
    if n_best == 1:
        assert tuple(int(x) for x in j) == assign


def test_dp_reduces_to_01_knapsack():
    # K = 2 where candidate 0 ("skip the item") costs no cell is the textbook 0/1 knapsack:
    # minimising the left-over error is maximising the value packed.
    rng = np.random.default_rng(11)
    n_items, cap = 9, 25
    w = rng.integers(1, 12, n_items)
    v = rng.integers(1, 50, n_items).astype(np.float64)
    # textbook table
    tab = np.zeros(cap + 1)
    for i in range(n_items):
        for b in range(cap, w[i] - 1, -1):
            tab[b] = max(tab[b], tab[b - w[i]] + v[i])
    best_value = tab[cap]
    # as a Kimad+ instance: skipping item i leaves error v_i, taking it leaves 0 and costs w_i cells
    err = np.stack([v, np.zeros(n_items)], axis=1).astype(np.float32)
    units = np.stack([np.zeros(n_items), w], axis=1).astype(np.uint64)
    st, j, val, cell = ko.dp(err, units, cap)
    assert st == 0
    assert float(val) == float(v.sum() - best_value)
    assert int(np.sum(w[j == 1])) == cell <= cap


def test_dp_special_cases():
    rng = np.random.default_rng(12)
    L, K = 5, 4
    err = (-np.sort(-rng.uniform(1, 9, (L, K)), axis=1)).astype(np.float32)
    err[:, -1] = 0
    units = np.sort(rng.integers(1, 30, (L, K)), axis=1).astype(np.uint64)
    # budget large enough for every layer's largest candidate -> all-max, zero error
    st, j, val, _ = ko.dp(err, units, int(units[:, -1].sum()))
    assert st == 0 and j.tolist() == [K - 1] * L and val == 0.0
    # one candidate per layer -> forced
    st, j, val, cell = ko.dp(err[:, :1], units[:, :1], int(units[:, 0].sum()))
    assert st == 0 and j.tolist() == [0] * L and cell == int(units[:, 0].sum())
    # one cell short of the cheapest assignment -> infeasible, all-min returned
    st, j, _, _ = ko.dp(err, units, int(units[:, 0].sum()) - 1)
    assert st == ko.STATUS_INFEASIBLE and j.tolist() == [0] * L
    # candidates above D are unusable even if their error is lowest
    u2 = units.copy()
    u2[:, -1] = 10_000
    st, j, _, _ = ko.dp(err, u2, 200)
    assert st == 0 and np.all(j < K - 1)


def test_dp_tie_breaks():
    # two candidates with identical cost and error: the first (lower j) keeps the cell (strict '<')
    err = np.float32([[1.0, 1.0, 0.5]])
    units = np.uint64([[2, 2, 9]])
    st, j, val, cell = ko.dp(err, units, 5)
    assert (st, j.tolist(), float(val), cell) == (0, [0], 1.0, 2)
    # equal final values at several cells: the lowest cell wins
    err = np.float32([[3.0, 3.0]])
    units = np.uint64([[4, 2]])
    st, j, val, cell = ko.dp(err, units, 6)
    assert (j.tolist(), cell) == ([1], 2)


# ----------------------------------------------------------------------------- golden example
def _read_golden():
    layers, ktab, curves, kept, cases, grid = {}, {}, {}, [], [], None
    for line in open(GOLDEN):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        t = line.split()
        if t[0] == "layer":
            layers[t[1]] = np.float32([float(x) for x in t[2:]])
        elif t[0] == "grid":
            grid = [float(x) for x in t[1:]]
        elif t[0] == "ktable":
            ktab[t[1]] = [int(x) for x in t[2:]]
        elif t[0] == "curve":
            curves[t[1]] = [float(x) for x in t[2:]]
        elif t[0] == "kept":
            kept.append((t[1], int(t[2]), [int(x) for x in t[4:]]))
        elif t[0] == "case":
            f = [s.split() for s in line[4:].split(":")]
            cases.append((int(f[0][0]), int(f[0][1]), [int(x) for x in f[1]], float(f[2][0]), int(f[3][0]),
                          int(f[4][0])))
    return layers, grid, ktab, curves, kept, cases


def test_golden_three_layer_example():
    layers, grid, ktab, curves, kept, cases = _read_golden()
    names = ["A", "B", "C"]
    sizes = [layers[n].size for n in names]
    kt = ko.k_table(sizes, grid)
    assert kt.tolist() == [ktab[n] for n in names]
    for i, n in enumerate(names):
        c = ko.layer_curve(layers[n], kt[i])
        assert c.err.tolist() == curves[n]
    for n, k, want in kept:
        idx, val = ko.select_pack(layers[n], k)
        assert idx.tolist() == want
        assert np.array_equal(val.view(np.uint32), layers[n][want].view(np.uint32))
    flat = np.concatenate([layers[n] for n in names])[None, :]
    state = np.zeros_like(flat)
    for c, D, want_k, want_err, want_cells, want_status in cases:
        r = ko.step(sizes, 1, grid, D, 0, flat, state, [float(c)], 1.0)
        assert r.k[0].tolist() == want_k, (c, D)
        assert float(r.total_err[0]) == want_err
        assert int(r.status[0]) == want_status
        assert int(r.budget_bytes[0]) == c
        assert int(r.used_bytes[0]) == 8 * sum(want_k)
        if want_status == 0:
            st, u = ko.units(kt, 0, c, D)
            assert sum(int(u[l, r.j[0, l]]) for l in range(3)) == want_cells
            assert int(r.used_bytes[0]) <= c  # Eq. 3


# ----------------------------------------------------------------------------- whole step
@pytest.mark.parametrize("value_dtype", [0, 1])
def test_step_identities(value_dtype):
    rng = np.random.default_rng(13)
    sizes = [1000, 7, 333, 64, 2048, 1]
    W, N = 3, sum(sizes)
    grid = [0.01, 0.05, 0.1, 0.5, 1.0]
    grads = (rng.standard_t(3, (W, N)) * 0.01).astype(np.float32)
    state = (rng.standard_normal((W, N)) * 0.003).astype(np.float32)
    bpe = 8 if value_dtype == 0 else 6
    bw = np.array([0.03, 0.2, 0.6]) * N * bpe
    r = ko.step(sizes, W, grid, 1000, value_dtype, grads, state, bw, 1.0)
    kt = ko.k_table(sizes, grid)
    offs = np.concatenate([[0], np.cumsum(sizes)])
    for w in range(W):
        assert int(r.status[w]) == 0
        assert int(r.used_bytes[w]) <= int(r.budget_bytes[w]) == math.floor(bw[w])
        assert int(r.used_bytes[w]) == bpe * int(r.k[w].sum()) == bpe * int(r.n_selected[w])
        assert r.offs[w].tolist() == np.concatenate([[0], np.cumsum(r.k[w])]).tolist()
        tot = np.float32(0)
        for l in range(len(sizes)):
            assert int(r.k[w, l]) == int(kt[l, r.j[w, l]])
            tot = np.float32(tot + r.err[w, l, r.j[w, l]])
            lo, hi = offs[l], offs[l + 1]
            d = (grads[w, lo:hi] - state[w, lo:hi]).astype(np.float32)
            a, b = int(r.offs[w, l]), int(r.offs[w, l + 1])
            idx, val = r.idx[w, a:b], r.val[w, a:b]
            assert np.all(np.diff(idx.astype(np.int64)) > 0)
            sent = val if value_dtype == 0 else (val.astype(np.uint32) << 16).view(np.float32)
            if value_dtype == 0:
                assert np.array_equal(sent.view(np.uint32), d[idx].view(np.uint32))
            # EF21: g_new - g is C(d) on the kept entries and untouched elsewhere
            g_old, g_new = state[w, lo:hi], r.state[w, lo:hi]
            ref = g_old.copy()
            ref[idx] = ref[idx] + sent
            assert np.array_equal(ref.view(np.uint32), g_new.view(np.uint32))
            # ||d - C(d)||^2 = err_l(k_l)  (f32 values only: bf16 adds a quantisation residual)
            if value_dtype == 0:
                resid = d.astype(np.float64).copy()
                resid[idx] = 0.0
                want = math.fsum((resid ** 2).tolist())
                got = float(r.err[w, l, r.j[w, l]])
                assert abs(got - want) <= 2e-7 * want + 1e-45
            # no dropped entry is larger in magnitude than a kept one
            key = keys_of(d)
            mask = np.zeros(hi - lo, bool)
            mask[idx] = True
            if mask.any() and (~mask).any():
                assert key[mask].min() >= key[~mask].max()
        assert tot == r.total_err[w]


def test_step_dp_beats_uniform_ratio():
    # Kimad+ never does worse than one ratio for all layers whenever that uniform choice fits the budget cells
    rng = np.random.default_rng(14)
    sizes = [4000, 500, 12000, 64, 900]
    grid = [0.01, 0.02, 0.05, 0.1, 0.2, 0.5, 1.0]
    N = sum(sizes)
    grads = np.concatenate([(rng.standard_normal(n) * s).astype(np.float32)
                            for n, s in zip(sizes, [1e-3, 1.0, 1e-2, 5.0, 0.1])])[None, :]
    kt = ko.k_table(sizes, grid)
    for frac in (0.03, 0.12, 0.4):
        c = int(frac * N * 8)
        r = ko.step(sizes, 1, grid, 1000, 0, grads, np.zeros_like(grads), [float(c)], 1.0)
        st, u = ko.units(kt, 0, c, 1000)
        for j in range(len(grid)):
            if int(u[:, j].sum()) <= 1000:
                uni = np.float32(0)
                for l in range(len(sizes)):
                    uni = np.float32(uni + r.err[0, l, j])
                assert r.total_err[0] <= uni


def test_step_inject_err_drives_dp():
    rng = np.random.default_rng(15)
    sizes = [100, 200, 50]
    grid = [0.1, 0.5, 1.0]
    grads = rng.standard_normal((1, 350)).astype(np.float32)
    inj = np.float32([[[5, 4, 0], [100, 1, 0], [5, 4, 0]]])
    kt = ko.k_table(sizes, grid)
    c = int(8 * (10 + 100 + 5) + 8)
    r = ko.step(sizes, 1, grid, 1000, 0, grads, np.zeros_like(grads), [float(c)], 1.0, inject_err=inj)
    assert r.k[0].tolist() == [10, 100, 5]
    assert float(r.total_err[0]) == 11.0
