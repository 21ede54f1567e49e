"""GPU parity of Kimad's ratio sized to the budget (Section 3.1; whole-model TopK of Section 4.3 as its one-layer
case) and of the sizes with a dense fallback, against the oracle (O9b, O13) on the same seeded inputs."""
import numpy as np
import pytest
import torch

from oracle import kimad_oracle as ko
from paper_2312_08053_b200 import binding as kb
from paper_2312_08053_b200 import workloads
from tests._harness import Runner, u32

pytestmark = pytest.mark.gpu

GOLD = torch.tensor([list(range(1, 11)) + [-8, .5, 8, -.5] + [3, -3, 3, 0, -0., 1]], dtype=torch.float32)


def test_fitted_ratio_hand_example_on_gpu():
    budgets = [24.0, 40.0, 96.0, 152.0, 17.0, 160.0]
    r = Runner([10, 4, 6], len(budgets), [1.0], 1000, 0, policy=3)
    d = GOLD.repeat(len(budgets), 1).cuda()
    res = r.compare_step(d, torch.zeros_like(d), budgets, 1.0, check_inject=False)
    assert res["forced"].k.tolist() == [[1, 1, 1], [3, 1, 1], [6, 2, 4], [9, 3, 5], [1, 1, 1], [10, 4, 6]]
    assert res["forced"].status.tolist() == [0, 0, 0, 0, ko.STATUS_INFEASIBLE, ko.STATUS_PLATEAU]
    assert r.out.stats_host()["total_err"].tolist() == [368.5, 223.5, 30.5, 1.25, 368.5, 0.0]


@pytest.mark.parametrize("cfg,divisor", [(2, 8), (4, 64), (5, 512)])
def test_fitted_ratio_matches_oracle(cfg, divisor):
    wl = workloads.workload(cfg, divisor)
    r = Runner(wl.layer_sizes, wl.n_workers, [1.0], wl.D, wl.value_dtype, policy=3)
    bw = workloads.bandwidth_trace(wl, 60)
    state = torch.zeros((wl.n_workers, wl.N), dtype=torch.float32, device="cuda")
    bpe = 8 if wl.value_dtype == 0 else 6
    for s, b in enumerate((0, 17, 33, 59)):
        grads = workloads.gradients(wl, s, device="cuda")
        res = r.compare_step(grads, state, bw[b], wl.t_target, check_inject=False)
        st = r.out.stats_host()
        ok = res["forced"].status == 0
        # the budget is used up to less than one entry per layer
        assert np.all(st["used_bytes"][ok] <= st["budget_bytes"][ok])
        assert np.all(st["budget_bytes"][ok] - st["used_bytes"][ok] < bpe * (wl.L + 1))


def test_whole_model_topk_keeps_floor_c_over_8_entries():
    """One layer spanning the model + the fitted ratio = TopK with the whole model information at K = floor(c / 8)."""
    wl = workloads.workload(2, 16)
    N = wl.N
    r = Runner([N], 1, [1.0], 1000, 0, policy=3)
    grads = workloads.gradients(wl, 0, device="cuda")[:1].contiguous()
    state = torch.zeros_like(grads)
    for K in (1, 777, N // 5):
        res = r.compare_step(grads, state.clone(), [8.0 * K + 3], 1.0, check_inject=False)
        assert int(res["forced"].k[0, 0]) == K
        kept = u32(r.out.idx)[0, :K]
        top = np.argsort(-np.abs(grads.cpu().numpy()[0]), kind="stable")[:K]
        assert np.array_equal(np.sort(top), kept)


def test_layer_adaptive_beats_the_fitted_ratio_at_equal_budget():
    """Section 4.3: Kimad+ reaches a lower compression error than Kimad at the same size.  On layers whose scales
    spread over three orders of magnitude the knapsack's total error is far below the one ratio's, at every budget
    of the trace (both within the same byte budget)."""
    wl = workloads.workload(4, 64)
    plus = Runner(wl.layer_sizes, wl.n_workers, wl.ratio_grid, wl.D, 0)
    kimad = Runner(wl.layer_sizes, wl.n_workers, [1.0], wl.D, 0, policy=3)
    bw = workloads.bandwidth_trace(wl, 60)
    grads = workloads.gradients(wl, 0, device="cuda")
    for b in (0, int(np.argmax(bw[:, 0]))):  # the floor of the trace and a burst
        s1, s2 = torch.zeros_like(grads), torch.zeros_like(grads)
        plus.gpu_step(grads, s1, bw[b], wl.t_target)
        kimad.gpu_step(grads, s2, bw[b], wl.t_target)
        a, c = plus.out.stats_host(), kimad.out.stats_host()
        assert np.all(a["status"] == 0) and np.all(c["status"] == 0)
        assert np.all(a["used_bytes"] <= a["budget_bytes"]) and np.all(c["used_bytes"] <= c["budget_bytes"])
        assert np.all(a["total_err"] < c["total_err"])


# ----------------------------------------------------------------------------- dense fallback
def test_dense_fallback_hand_example_on_gpu():
    cases = [(96.0, 12), (79.0, 1000), (60.0, 12), (48.0, 12)]
    want_k = [[10, 4, 6], [10, 4, 2], [3, 1, 6], [3, 1, 2]]
    want_dense = [[1, 1, 1], [1, 1, 0], [0, 0, 1], [0, 0, 0]]
    for (c, D), k, dn in zip(cases, want_k, want_dense):
        r = Runner([10, 4, 6], 1, [0.25, 0.5, 1.0], D, 0, cost_model=1)
        d = GOLD.cuda()
        res = r.compare_step(d, torch.zeros_like(d), [c], 1.0)
        assert res["forced"].k.tolist() == [k] and u32(r.out.dense).tolist() == [dn]


@pytest.mark.parametrize("policy", [0, 1])
@pytest.mark.parametrize("cfg,divisor", [(2, 8), (5, 512)])
def test_dense_fallback_matches_oracle(cfg, divisor, policy):
    wl = workloads.workload(cfg, divisor)
    r = Runner(wl.layer_sizes, wl.n_workers, wl.ratio_grid, wl.D, wl.value_dtype, policy=policy, cost_model=1)
    state = torch.zeros((wl.n_workers, wl.N), dtype=torch.float32, device="cuda")
    any_dense = False
    for s, frac in enumerate((0.05, 0.3, 0.6, 0.9)):  # of the dense size: the larger ones make layers reach it
        grads = workloads.gradients(wl, s, device="cuda")
        bw = frac * 4.0 * wl.N / wl.t_target * np.linspace(0.8, 1.2, wl.n_workers)
        res = r.compare_step(grads, state, bw, wl.t_target, check_inject=(policy == 0))
        any_dense |= bool(res["forced"].dense.any())
    assert any_dense


def test_receiver_reads_dense_layers_like_any_other():
    wl = workloads.workload(3, 32)
    W, N = wl.n_workers, wl.N
    r = Runner(wl.layer_sizes, W, wl.ratio_grid, wl.D, 0, cost_model=1)
    state = torch.zeros((W, N), dtype=torch.float32, device="cuda")
    copy = torch.zeros((W, N), dtype=torch.float32, device="cuda")
    for s in range(2):
        grads = workloads.gradients(wl, s, device="cuda")
        r.gpu_step(grads, state, np.full(W, 0.5 * 4 * N / wl.t_target), wl.t_target)
        assert u32(r.out.dense).any()
        kb.kimad_apply_packed(r.ctx, r.out, copy)
        torch.cuda.synchronize()
        assert torch.equal(copy.view(torch.int32), state.view(torch.int32))


def test_create_validates_policy_and_cost_model():
    for kw in (dict(ratio_grid=[0.5, 1.0], policy=3), dict(ratio_grid=[0.5], policy=3),
               dict(ratio_grid=[1.0], policy=3, cost_model=1), dict(ratio_grid=[0.5, 1.0], policy=2, cost_model=1),
               dict(ratio_grid=[0.5, 1.0], cost_model=2)):
        with pytest.raises(kb.KimadError):
            kb.kimad_create([100, 20], 1, **kw)


@pytest.mark.parametrize("seed", [21, 22])
def test_randomized_policies_and_cost_models(seed):
    """Random layer lists, grids, worker counts, strides, value types and budgets under every policy (layer-adaptive,
    grid ratio, error axis, fitted ratio) and both cost models where they apply; two steps each, everything compared
    with the oracle."""
    for it in range(16):
        rng = np.random.default_rng(seed * 1000 + it)
        policy = int(rng.integers(0, 4))
        cost_model = int(rng.integers(0, 2)) if policy < 2 else 0
        L = int(rng.integers(1, 7))
        sizes = [int(v) for v in np.exp(rng.uniform(np.log(1), np.log(200000), L)).astype(int) + 1]
        if policy == 3:
            grid = [1.0]
        else:
            grid = np.unique(np.round(np.sort(rng.uniform(0.0005, 1.0, int(rng.integers(1, 12)))), 6))
            if rng.random() < 0.5:
                grid[-1] = 1.0
        W, vd = int(rng.integers(1, 4)), int(rng.integers(0, 2))
        D = max(int(rng.choice([L, 50, 1000])), L)
        N = sum(sizes)
        stride = N + int(rng.integers(0, 9))
        r = Runner(sizes, W, list(grid), D, vd, stride=stride, policy=policy, cost_model=cost_model)
        x = (rng.standard_normal((W, stride)) * np.exp(rng.uniform(-4, 4, (W, stride)))).astype(np.float32)
        if it % 5 == 4:
            x = np.round(x * 2) / 2  # heavy ties, many zeros
        grads = torch.from_numpy(x).cuda()
        state = torch.from_numpy((rng.standard_normal((W, stride)) * 0.1).astype(np.float32)).cuda()
        for rep in range(2):
            frac = float(np.exp(rng.uniform(np.log(0.002), np.log(1.5))))
            bw = [frac * (8 if vd == 0 else 6) * N * float(rng.uniform(0.5, 1.5)) for _ in range(W)]
            r.compare_step(grads, state, bw, 1.0, check_inject=bool(rng.integers(0, 2)))
