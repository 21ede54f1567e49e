"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle on the same seeded inputs."""
import numpy as np
import pytest
import torch

from oracle import kimad_oracle as ko
from paper_2312_08053_b200 import binding as kb
from paper_2312_08053_b200 import workloads
from tests._harness import Runner, u32

pytestmark = pytest.mark.gpu


def _run_workload(cfg, divisor, steps, grid=None, D=None, curve_mode=0, schedule=0):
    wl = workloads.workload(cfg, divisor)
    grid = grid or wl.ratio_grid
    r = Runner(wl.layer_sizes, wl.n_workers, grid, D or wl.D, wl.value_dtype, curve_mode=curve_mode, schedule=schedule)
    bw = workloads.bandwidth_trace(wl, max(steps, 60))
    pick = np.linspace(0, len(bw) - 1, steps).astype(int)  # spread over the trace: low and high budgets
    state = torch.zeros((wl.n_workers, wl.N), dtype=torch.float32, device="cuda")
    mismatched = 0
    for s in range(steps):
        grads = workloads.gradients(wl, s, device="cuda")
        res = r.compare_step(grads, state, bw[pick[s]], wl.t_target)
        mismatched += not res["same_k"]
    # the free-running state after `steps` steps was compared bit for bit at every step
    assert mismatched == 0, f"{mismatched} steps chose another k than the oracle on its own curve"
    n_reg = sum(1 for n in wl.layer_sizes if n > 4096) * wl.n_workers * steps * 2  # each step runs twice (inject check)
    handed = kb.kimad_debug_exact_path_layers(r.ctx)
    if curve_mode == 1:
        assert handed == n_reg
    else:  # the sampled bands must carry (nearly) all layers by themselves
        why = kb.kimad_debug_exact_path_layers(r.ctx, detail=True)
        # with 50 candidates the fine bins are shared by 50 bands and more error bounds come out too loose
        limit = n_reg // 50 if len(grid) <= 16 else n_reg // 4
        assert handed <= max(1, limit), f"{why} of {n_reg} layers fell back to the exact radix path"
    return handed, n_reg


def test_cfg1_mlp_full_size():
    _run_workload(1, 1, 3)


def test_cfg2_resnet18_shape_scaled():
    _run_workload(2, 8, 4)


def test_cfg3_resnet50_shape_scaled():
    _run_workload(3, 16, 3)


def test_cfg4_gpt2_shape_scaled():
    _run_workload(4, 64, 3)


def test_cfg5_llama_shape_scaled_bf16():
    _run_workload(5, 512, 4)


@pytest.mark.parametrize("cfg,divisor,curve_mode", [(2, 8, 0), (3, 16, 0), (4, 64, 0), (5, 512, 0), (3, 32, 1)])
def test_two_worker_groups(cfg, divisor, curve_mode):
    """The schedule large steps use (two groups of workers on two streams, each with work lists of its own),
    forced on the scaled workloads: every result as with one group."""
    _run_workload(cfg, divisor, 3, curve_mode=curve_mode, schedule=1)


def test_paper_grid_50_candidates():
    _run_workload(2, 32, 2, grid=workloads.paper_grid_50())


@pytest.mark.parametrize("cfg,divisor", [(2, 8), (4, 64), (5, 512)])
def test_exact_radix_everywhere(cfg, divisor):
    """curve_mode 1: every layer above the tiny size goes through the three-digit radix select."""
    _run_workload(cfg, divisor, 2, curve_mode=1)


def test_paper_grid_50_exact_radix():
    _run_workload(2, 32, 2, grid=workloads.paper_grid_50(), curve_mode=1)


def test_worked_example_on_gpu():
    a = np.arange(1, 11, dtype=np.float32)
    b = np.float32([-8, 0.5, 8, -0.5])
    c = np.float32([3, -3, 3, 0, -0.0, 1])
    flat = torch.from_numpy(np.concatenate([a, b, c])[None, :]).cuda()
    for budget, D, want in [(96, 12, [5, 4, 3]), (96, 1000, [5, 2, 3]), (100, 1000, [5, 4, 3]), (95, 12, [5, 2, 2]),
                            (200, 1000, [10, 4, 6]), (47, 1000, [3, 1, 2])]:
        r = Runner([10, 4, 6], 1, [0.25, 0.5, 1.0], D=D)
        state = torch.zeros_like(flat)
        res = r.compare_step(flat, state, [float(budget)], 1.0)
        assert u32(r.out.k)[0].tolist() == want
        assert res["same_k"]


def _adversarial_layers(rng):
    n = 70001
    layers = []
    layers.append(np.full(n, 0.5, np.float32) * np.where(rng.uniform(size=n) < 0.5, -1, 1))      # all equal magnitude
    layers.append(np.zeros(4097, np.float32))                                                      # all zero
    z = np.zeros(33000, np.float32); z[::2] = -0.0                                                 # +0 / -0 mix
    layers.append(z)
    one = np.zeros(40000, np.float32); one[31999] = -3.0                                           # a single nonzero
    layers.append(one)
    layers.append(np.float32([7.0]))                                                               # n = 1
    den = (rng.integers(1, 2 ** 22, 50000).astype(np.uint32)).view(np.float32)                     # denormals
    layers.append(den * np.where(rng.uniform(size=50000) < 0.5, -1, 1).astype(np.float32))
    dup = rng.choice(np.float32([1.0, 1.0000001, 0.9999999, 2.0, 1e-3]), 100003).astype(np.float32)  # few distinct values
    layers.append(dup)
    emb = np.zeros(64 * 3000, np.float32)                                                          # row-sparse "embedding"
    rows = rng.choice(3000, 90, replace=False)
    for r in rows:
        emb[r * 64:(r + 1) * 64] = rng.standard_normal(64).astype(np.float32) * 1e-2
    layers.append(emb)
    layers.append((rng.standard_normal(13) * 1e15).astype(np.float32))                             # huge, squares still finite
    layers.append((rng.standard_normal(65537) * 1e-30).astype(np.float32))                         # tiny normals
    return [np.ascontiguousarray(x, np.float32) for x in layers]


@pytest.mark.parametrize("curve_mode", [0, 1])
@pytest.mark.parametrize("value_dtype", [0, 1])
def test_adversarial_inputs(value_dtype, curve_mode):
    rng = np.random.default_rng(77)
    layers = _adversarial_layers(rng)
    sizes = [x.size for x in layers]
    N = sum(sizes)
    grid = [0.001, 0.01, 0.1, 0.5, 0.9, 1.0]
    r = Runner(sizes, 2, grid, value_dtype=value_dtype, curve_mode=curve_mode)
    flat = np.concatenate(layers)
    grads = torch.from_numpy(np.stack([flat, flat[::-1].copy()])).cuda()   # worker 1: same values, other layout
    bpe = 8 if value_dtype == 0 else 6
    state = torch.zeros_like(grads)
    for frac in (0.02, 0.3, 0.95):
        # several layers here have exactly linear error curves, so many assignments tie up to the last
        # rounding of the curve: the decision is compared on the SAME curve (inside compare_step) only
        r.compare_step(grads, state, [frac * N * bpe, 0.5 * frac * N * bpe], 1.0)


def test_unaligned_stride_and_offsets_take_scalar_path():
    rng = np.random.default_rng(5)
    sizes = [10, 1000, 50257, 3, 40001, 7]            # layer starts not 16-byte aligned
    N = sum(sizes)
    stride = N + 3                                     # worker rows not 16-byte aligned either
    grid = [0.01, 0.1, 0.5, 1.0]
    r = Runner(sizes, 3, grid, stride=stride)
    grads = torch.from_numpy((rng.standard_t(3, (3, stride)) * 1e-2).astype(np.float32)).cuda()
    state = torch.from_numpy((rng.standard_normal((3, stride)) * 1e-3).astype(np.float32)).cuda()
    pad_before = state[:, N:].clone()
    res = r.compare_step(grads, state, [0.05 * N * 8, 0.2 * N * 8, 0.6 * N * 8], 1.0)
    assert res["same_k"]
    assert torch.equal(state[:, N:], pad_before)       # padding between workers untouched


def test_statuses_plateau_infeasible_capacity_nonfinite():
    rng = np.random.default_rng(6)
    sizes = [5000, 300, 70000]
    N = sum(sizes)
    grid = [0.01, 0.1, 1.0]
    grads = torch.from_numpy(rng.standard_normal((2, N)).astype(np.float32)).cuda()
    # plateau on worker 0, infeasible on worker 1
    r = Runner(sizes, 2, grid)
    state = torch.zeros_like(grads)
    res = r.compare_step(grads, state, [8.0 * N, 100.0], 1.0)
    st = r.out.stats_host()
    assert st["status"].tolist() == [kb.KIMAD_STATUS_PLATEAU, kb.KIMAD_STATUS_INFEASIBLE]
    assert res["status"] == kb.KIMAD_STATUS_PLATEAU
    assert u32(r.out.k)[0].tolist() == sizes and st["total_err"][0] == 0.0
    assert torch.equal(state[0], grads[0] - torch.zeros_like(grads[0]))  # everything sent: g + (grad - g), g = 0
    # capacity: worker 0 wants more entries than the packed buffers hold -> error status, state untouched
    r = Runner(sizes, 2, grid, cap=1000)
    state = torch.zeros_like(grads)
    status, k = r.gpu_step(grads, state, [8.0 * N, 8.0 * 900], 1.0)
    st = r.out.stats_host()
    assert status == kb.KIMAD_ERR_CAPACITY
    assert st["status"][0] == kb.KIMAD_ERR_CAPACITY and st["status"][1] == 0
    assert int(st["n_selected"][0]) == 0 and not state[0].any()
    assert int(st["n_selected"][1]) <= 900 and state[1].any()
    # non-finite input with check_finite
    r = Runner(sizes, 2, grid, check_finite=1)
    bad = grads.clone()
    bad[1, 5100] = float("inf")
    state = torch.zeros_like(grads)
    status, k = r.gpu_step(bad, state, [8.0 * 800, 8.0 * 800], 1.0)
    st = r.out.stats_host()
    assert status == kb.KIMAD_ERR_NONFINITE
    assert st["status"].tolist() == [0, kb.KIMAD_ERR_NONFINITE]
    assert not state[1].any() and state[0].any()
    # the flag does not stick: the next clean step succeeds
    status, k = r.gpu_step(grads, state, [8.0 * 800, 8.0 * 800], 1.0)
    assert status == 0


def test_given_j_skips_the_dp():
    rng = np.random.default_rng(8)
    sizes = [3000, 50, 20000]
    grid = [0.01, 0.05, 0.25, 1.0]
    r = Runner(sizes, 1, grid)
    grads = torch.from_numpy(rng.standard_normal((1, sum(sizes))).astype(np.float32)).cuda()
    state = torch.zeros_like(grads)
    j = torch.tensor([[2, 0, 3]], dtype=torch.int32, device="cuda")
    kb.kimad_debug_step_with_j(r.ctx, grads, state, [1.0], 1.0, r.out, j)
    status, k = kb.kimad_get_k(r.ctx)
    assert k[0].tolist() == [750, 1, 20000]
    d = grads.cpu().numpy()[0]
    offs = np.concatenate([[0], np.cumsum(sizes)])
    pos = 0
    for l, kk in enumerate(k[0]):
        idx, val = ko.select_pack(d[offs[l]:offs[l + 1]], int(kk))
        assert np.array_equal(u32(r.out.idx)[0, pos:pos + kk], idx)
        assert np.array_equal(r.out.val.cpu().numpy()[0, pos:pos + kk], val)
        pos += int(kk)


def test_run_to_run_determinism_of_decisions():
    wl = workloads.workload(3, 32)
    bw = workloads.bandwidth_trace(wl, 10)[7]
    grads = workloads.gradients(wl, 0, device="cuda")
    outs = []
    for _ in range(3):
        r = Runner(wl.layer_sizes, wl.n_workers, wl.ratio_grid)
        state = torch.zeros_like(grads)
        r.gpu_step(grads, state, bw, wl.t_target)
        outs.append((u32(r.out.k).copy(), u32(r.out.idx).copy(), u32(state).copy()))
    for o in outs[1:]:
        assert all(np.array_equal(a, b) for a, b in zip(outs[0], o))


@pytest.mark.parametrize("cfg,divisor,schedule", [(1, 1, 0), (2, 16, 1)])
def test_step_is_capturable_in_a_cuda_graph(cfg, divisor, schedule):
    """All work of a step, the forked streams included (the tiny layers' side stream; with schedule 1 the two worker
    groups' sweep and short-kernel streams), is ordered through the caller's stream: the step can be captured once
    and replayed on new gradients (the budgets are baked into the captured launches)."""
    wl = workloads.workload(cfg, divisor)
    W, N = wl.n_workers, wl.N
    bw = workloads.bandwidth_trace(wl)[0]
    ctx = kb.new_context(wl.layer_sizes, W, wl.ratio_grid, D=wl.D, value_dtype=wl.value_dtype)
    kb.kimad_debug_set_schedule(ctx, schedule)
    out = kb.Packed(ctx)
    grads = workloads.gradients(wl, 0, device="cuda")
    state = torch.zeros((W, N), device="cuda")
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        kb.kimad_step(ctx, grads, state, bw, wl.t_target, out, s)  # warm-up outside the capture
    s.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph, stream=s):
        kb.kimad_step(ctx, grads, state, bw, wl.t_target, out, torch.cuda.current_stream())
    state.zero_()
    ref_state = np.zeros((W, N), np.float32)
    for step in range(3):
        fresh = workloads.gradients(wl, 10 + step, device="cuda")
        grads.copy_(fresh)
        graph.replay()
        torch.cuda.synchronize()
        ref = ko.step(wl.layer_sizes, W, wl.ratio_grid, wl.D, wl.value_dtype, fresh.cpu().numpy(), ref_state, bw,
                      wl.t_target)
        ref_state = ref.state
        assert np.array_equal(u32(out.k), ref.k)
        assert np.array_equal(u32(state), ref_state.view(np.uint32))


@pytest.mark.parametrize("K,D", [(127, 1000), (1, 1000), (16, 8191), (7, 5)])
def test_interface_limits(K, D):
    """The largest ratio grid (127), a single ratio, the largest number of budget cells (8191) and the smallest one
    the layer list allows (D = L)."""
    rng = np.random.default_rng(K + D)
    sizes = [70000, 33, 5000, 4097, 1]
    grid = np.linspace(1.0 / K, 1.0, K) if K > 1 else [0.25]
    r = Runner(sizes, 2, grid, D, 0)
    N = sum(sizes)
    grads = torch.from_numpy((rng.standard_normal((2, N)) * np.repeat([1.0, 30.0, 0.01, 3.0, 1.0], sizes)).astype(np.float32)).cuda()
    state = torch.zeros_like(grads)
    for budget in ([0.05 * 8 * N, 0.6 * 8 * N], [0.3 * 8 * N, 8.0 * N]):
        res = r.compare_step(grads, state, budget, 1.0)
        assert res["same_k"]


def test_many_workers_with_different_budgets():
    """40 workers on one GPU (the DP runs in several launches of workers), every worker with its own budget."""
    sizes = [30000, 128, 9000, 10]
    grid = [0.01, 0.02, 0.05, 0.1, 0.2, 0.5, 1.0]
    W, N = 40, sum(sizes)
    r = Runner(sizes, W, grid, 1000, 1)
    gen = torch.Generator(device="cuda").manual_seed(40)
    grads = torch.randn((W, N), device="cuda", generator=gen) * 0.01
    state = torch.zeros_like(grads)
    bw = np.linspace(0.0, 1.1, W) * 6 * N  # from nothing (infeasible) to more than everything (plateau)
    res = r.compare_step(grads, state, bw, 1.0)
    st = res["forced"].status
    assert st[0] == ko.STATUS_INFEASIBLE and st[-1] == ko.STATUS_PLATEAU and np.count_nonzero(st == 0) > 30


def test_huge_dynamic_range_in_a_tiny_layer():
    """Magnitudes spread over 26 orders: the curve's partial sums must not lose their small terms (an exclusive scan
    taken as inclusive minus own would cancel them)."""
    rng = np.random.default_rng(1095)
    sizes = [48, 3000, 70000]
    grid = [0.02, 0.1, 0.3, 0.6, 0.9, 1.0]
    N = sum(sizes)
    x = (rng.standard_normal((3, N)) * np.exp(rng.uniform(-30, 30, (3, N)))).astype(np.float32)
    r = Runner(sizes, 3, grid, 1000, 0)
    grads = torch.from_numpy(x).cuda()
    state = torch.from_numpy((rng.standard_normal((3, N)) * 0.1).astype(np.float32)).cuda()
    r.compare_step(grads, state, [0.1 * 8 * N, 0.5 * 8 * N, 2.0 * 8 * N], 1.0)


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_randomized_configurations(seed):
    """Random layer lists, grids, worker counts, strides, value types, cell counts and value patterns (ties, denormals,
    mostly zeros, huge dynamic range, all-equal magnitudes), two steps each, all compared with the oracle."""
    for it in range(25):
        rng = np.random.default_rng(seed * 1000 + it)
        L = int(rng.integers(1, 7))
        sizes = [int(v) for v in np.exp(rng.uniform(np.log(1), np.log(400000), L)).astype(int) + 1]
        grid = np.unique(np.round(np.sort(rng.uniform(0.0005, 1.0, int(rng.integers(1, 20)))), 6))
        if rng.random() < 0.5:
            grid[-1] = 1.0
        W, vd = int(rng.integers(1, 4)), int(rng.integers(0, 2))
        D = max(int(rng.choice([L, 50, 1000, 4000])), L)
        N = sum(sizes)
        stride = N + int(rng.integers(0, 9))
        r = Runner(sizes, W, list(grid), D, vd, stride=stride)
        kind = int(rng.integers(0, 6))
        x = rng.standard_normal((W, stride)).astype(np.float32)
        if kind == 1:
            x = np.round(x * 4) / 4
        elif kind == 2:
            x *= np.float32(1e-40)
        elif kind == 3:
            x[rng.random(x.shape) < 0.9] = 0
        elif kind == 4:
            x = (x * np.exp(rng.uniform(-30, 30, x.shape))).astype(np.float32)
        elif kind == 5:
            x = np.sign(x) * np.float32(0.5)
        grads = torch.from_numpy(x).cuda()
        state = torch.from_numpy((rng.standard_normal((W, stride)) * (0.0 if kind in (2, 5) else 0.1)).astype(np.float32)).cuda()
        for rep in range(2):
            frac = float(np.exp(rng.uniform(np.log(0.002), np.log(1.5))))
            bw = [frac * (8 if vd == 0 else 6) * N * float(rng.uniform(0.5, 1.5)) for _ in range(W)]
            r.compare_step(grads, state, bw, 1.0, check_inject=bool(rng.integers(0, 2)))


@pytest.mark.parametrize("seed", [3, 4])
def test_concentrated_magnitudes_second_select_round(seed):
    """Layers whose |d| sits within a third of an octave: the bin that holds a threshold is wide (many keys) and
    full, so the select stage overflows its per-chunk lists, narrows the interval with the coarse histogram and
    counts a second time.  Duplicates of the k-th value are planted in different chunks, so that kept ties span
    chunks and any double count of an entry shifts the packed positions."""
    rng = np.random.default_rng(seed)
    sizes = [20000, 300007, 1000003, 32768, 150001, 2000000]
    grid = [0.01, 0.1, 0.3, 0.5, 0.8, 1.0]
    N = sum(sizes)
    parts = []
    for n in sizes:
        a = np.float32(10.0 ** rng.uniform(-3, 0))
        v = (a * rng.uniform(1.0, 1.3, n)).astype(np.float32)
        for ratio in grid[:-1]:  # plant ties at every candidate's threshold value
            kth = np.partition(v, n - int(np.ceil(ratio * n)))[n - int(np.ceil(ratio * n))]
            v[rng.choice(n, 12, replace=False)] = kth
        parts.append(v * np.where(rng.random(n) < 0.5, -1, 1).astype(np.float32))
    x = np.concatenate(parts)[None, :]
    r = Runner(sizes, 1, grid)
    grads = torch.from_numpy(x).cuda()
    state = torch.zeros_like(grads)
    for frac in (0.05, 0.25, 0.45, 0.7):
        r.compare_step(grads, state.clone(), [frac * 8 * N], 1.0)


def test_traced_step_equals_a_plain_step():
    """The launch trace only adds events: results equal the oracle's, and the timeline names both groups' sweeps."""
    rng = np.random.default_rng(3)
    sizes = [90000, 700, 40000, 5000]
    W, N = 4, sum(sizes)
    r = Runner(sizes, W, [0.01, 0.1, 0.5, 1.0], 1000, 0, schedule=1)
    grads = torch.from_numpy(rng.standard_normal((W, N)).astype(np.float32)).cuda()
    state = torch.zeros_like(grads)
    r.compare_step(grads, state, [0.2 * 8 * N] * W, 1.0)
    ref_state = state.clone()
    state.zero_()
    text = kb.kimad_debug_trace_step(r.ctx, grads, state, [0.2 * 8 * N] * W, 1.0, r.out)
    assert torch.equal(state, ref_state)
    lines = [ln.split() for ln in text.strip().splitlines()]
    sweeps = [ln for ln in lines if ln[0].startswith("k_pass_a")]
    assert len(sweeps) == 2 and sweeps[0][2] != sweeps[1][2]  # one sweep per group, on different streams
    assert all(float(ln[3]) <= float(ln[5]) for ln in lines)
