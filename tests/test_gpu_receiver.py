"""GPU parity of the rows beyond the worker-side pass: the uniform-ratio policy (Section 3.1), the receiver's
estimator update and the model step (Algorithm 1, server lines), and the closed bidirectional EF21 loop."""
import numpy as np
import pytest
import torch

from oracle import kimad_oracle as ko
from paper_2312_08053_b200 import binding as kb
from paper_2312_08053_b200 import workloads
from tests._harness import Runner, u32

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("cfg,divisor", [(2, 8), (5, 512)])
def test_uniform_ratio_policy_matches_oracle(cfg, divisor):
    wl = workloads.workload(cfg, divisor)
    r = Runner(wl.layer_sizes, wl.n_workers, wl.ratio_grid, wl.D, wl.value_dtype, policy=1)
    bw = workloads.bandwidth_trace(wl, 60)
    state = torch.zeros((wl.n_workers, wl.N), dtype=torch.float32, device="cuda")
    seen = set()
    for s, b in enumerate((0, 17, 33, 59)):
        grads = workloads.gradients(wl, s, device="cuda")
        res = r.compare_step(grads, state, bw[b], wl.t_target, check_inject=False)
        j = res["forced"].j
        assert np.all(j == j[:, :1]), "one candidate index for all layers of a worker"
        seen.update(int(x) for x in j[:, 0])
    assert len(seen) > 1  # the budgets of the trace select different ratios


def test_uniform_ratio_statuses():
    sizes, grid = [10, 4, 6], [0.25, 0.5, 1.0]
    r = Runner(sizes, 3, grid, 1000, 0, policy=1)
    d = torch.tensor([list(range(1, 11)) + [-8, .5, 8, -.5] + [3, -3, 3, 0, -0., 1]] * 3, dtype=torch.float32, device="cuda")
    state = torch.zeros_like(d)
    res = r.compare_step(d, state, [47.0, 80.0, 160.0], 1.0, check_inject=False)
    assert list(res["forced"].status) == [ko.STATUS_INFEASIBLE, ko.STATUS_OK, ko.STATUS_PLATEAU]
    assert res["forced"].k.tolist() == [[3, 1, 2], [5, 2, 3], [10, 4, 6]]


def test_whole_model_topk_is_a_single_layer_context():
    """Section 4.3's whole-model baseline: one layer spanning the model, uniform policy; indices are global."""
    wl = workloads.workload(2, 16)
    N = wl.N
    r = Runner([N], 1, wl.ratio_grid, 1000, 0, policy=1)
    grads = workloads.gradients(wl, 0, device="cuda")[:1].contiguous()
    state = torch.zeros_like(grads)
    res = r.compare_step(grads, state, [0.3 * 8 * N], 1.0, check_inject=False)
    k = int(res["forced"].k[0, 0])
    assert 0 < k < N
    kept = u32(r.out.idx)[0, :k]
    top = np.argsort(-np.abs(grads.cpu().numpy()[0]), kind="stable")[:k]
    assert np.array_equal(np.sort(top), kept)


@pytest.mark.parametrize("value_dtype", [0, 1])
def test_receiver_copy_equals_sender_state(value_dtype):
    wl = workloads.workload(3, 32)
    W, N = wl.n_workers, wl.N
    stride = N + 12
    r = Runner(wl.layer_sizes, W, wl.ratio_grid, wl.D, value_dtype, stride=stride)
    bw = workloads.bandwidth_trace(wl, 60)
    state = torch.zeros((W, stride), dtype=torch.float32, device="cuda")
    copy = torch.zeros((W, stride), dtype=torch.float32, device="cuda")
    copy_ref = np.zeros((W, N), np.float32)
    for s, b in enumerate((3, 30, 55)):
        grads = workloads.gradients(wl, s, device="cuda", stride=stride)
        r.gpu_step(grads, state, bw[b], wl.t_target)
        kb.kimad_apply_packed(r.ctx, r.out, copy)
        torch.cuda.synchronize()
        assert torch.equal(copy.view(torch.int32)[:, :N], state.view(torch.int32)[:, :N])
        assert not copy[:, N:].any()
        # and against the oracle's receiver, fed the same message
        offs = r.out.offs.cpu().numpy().astype(np.uint64)
        idx, val = u32(r.out.idx), r.out.val.view(torch.int16 if value_dtype else torch.int32).cpu().numpy()
        for w in range(W):
            n = int(offs[w, -1])
            v = val[w, :n].view(np.uint16 if value_dtype else np.float32)
            copy_ref[w] = ko.apply_packed(wl.layer_sizes, idx[w, :n], v, offs[w], value_dtype, copy_ref[w])
        assert np.array_equal(copy.cpu().numpy()[:, :N].view(np.uint32), copy_ref.view(np.uint32))


def test_apply_skips_a_failed_worker_and_bad_indices():
    sizes, grid = [64, 5000], [0.1, 1.0]
    r = Runner(sizes, 2, grid, 1000, 0, check_finite=1)
    g = torch.randn((2, sum(sizes)), device="cuda")
    g[1, 7] = float("inf")
    state = torch.zeros_like(g)
    status, _ = r.gpu_step(g, state, [4000.0, 4000.0], 1.0)
    assert status == kb.KIMAD_ERR_NONFINITE
    copy = torch.zeros_like(g)
    kb.kimad_apply_packed(r.ctx, r.out, copy)
    torch.cuda.synchronize()
    assert torch.equal(copy[0], state[0]) and copy[0].any()
    assert not copy[1].any()
    # an index beyond its layer is skipped, the rest of the message is applied
    r.out.idx[0, 0] = 64
    copy2 = torch.zeros_like(g)
    kb.kimad_apply_packed(r.ctx, r.out, copy2)
    torch.cuda.synchronize()
    diff = (copy2[0] != copy[0]).nonzero().flatten().tolist()
    assert len(diff) == 1 and diff[0] < 64


@pytest.mark.parametrize("W,n,stride", [(1, 1, 1), (3, 4099, 4099), (4, 1 << 20, (1 << 20) + 8), (64, 2500, 2504),
                                        (2, 1000003, 1000003)])
def test_aggregate_matches_oracle_bit_for_bit(W, n, stride):
    g = torch.Generator(device="cuda").manual_seed(n + W)
    est = torch.randn((W, stride), device="cuda", generator=g)
    x = torch.randn(n, device="cuda", generator=g)
    w = np.random.default_rng(W).uniform(0.05, 1.0, W).astype(np.float32)
    want = ko.aggregate(x.cpu().numpy(), est.cpu().numpy()[:, :n], w, 0.013)
    kb.kimad_aggregate(x, est, w, 0.013)
    torch.cuda.synchronize()
    assert np.array_equal(x.cpu().numpy().view(np.uint32), want.view(np.uint32))


def test_aggregate_rejects_bad_arguments():
    x = torch.zeros(8, device="cuda")
    est = torch.zeros((65, 8), device="cuda")
    with pytest.raises(kb.KimadError):
        kb.kimad_aggregate(x, est, np.ones(65, np.float32), 0.1)


def test_bidirectional_ef21_loop_on_a_quadratic_matches_oracle_and_converges():
    """Algorithm 1 end to end on f_m(x) = 1/2 sum_i a_i (x_i - b_{m,i})^2: server compresses x - x^, workers
    compress grad f_m(x^) - u^_m, the server aggregates.  The GPU loop and the oracle loop stay bit-identical,
    and the loss falls."""
    sizes, grid = [6000, 300, 9000, 50], [0.05, 0.1, 0.2, 0.4, 0.8, 1.0]
    N, M, gamma, rounds = sum(sizes), 3, 0.2, 12
    rng = np.random.default_rng(5)
    a = rng.uniform(0.5, 2.0, N).astype(np.float32)
    b = rng.standard_normal((M, N)).astype(np.float32)
    wts = np.full(M, 1.0 / M, np.float32)
    up_bw, down_bw = [0.15 * 8 * N, 0.3 * 8 * N, 0.6 * 8 * N], [0.25 * 8 * N]

    def loss(x):
        return float(sum(0.5 * np.sum(a.astype(np.float64) * (x.astype(np.float64) - b[m]) ** 2) for m in range(M)) / M)

    # oracle loop
    x, xh, uh = np.zeros(N, np.float32), np.zeros((1, N), np.float32), np.zeros((M, N), np.float32)
    x[:] = 3.0
    losses = [loss(x)]
    xs_ref = []
    for k in range(rounds):
        xh = ko.step(sizes, 1, grid, 1000, 0, x[None], xh, down_bw, 1.0).state        # x^ += C(x - x^)
        u = a[None, :] * (xh - b)                                                      # float32
        uh = ko.step(sizes, M, grid, 1000, 0, u, uh, up_bw, 1.0).state                # u^_m += C_m(u_m - u^_m)
        x = ko.aggregate(x, uh, wts, gamma)
        xs_ref.append(x.copy())
        losses.append(loss(x))
    l_star = loss(b.mean(0).astype(np.float32))  # the minimiser is the mean of the b_m
    assert all(y < x_ for x_, y in zip(losses, losses[1:]))
    assert losses[-1] - l_star < 0.05 * (losses[0] - l_star)

    # GPU loop: server context (1 sender) and worker context (M senders); receivers apply the messages
    srv = Runner(sizes, 1, grid, 1000, 0)
    wrk = Runner(sizes, M, grid, 1000, 0)
    a_d, b_d = torch.from_numpy(a).cuda(), torch.from_numpy(b).cuda()
    x_d = torch.full((N,), 3.0, device="cuda")
    xh_srv, xh_wrk = torch.zeros((1, N), device="cuda"), torch.zeros((1, N), device="cuda")
    uh_wrk, uh_srv = torch.zeros((M, N), device="cuda"), torch.zeros((M, N), device="cuda")
    for k in range(rounds):
        kb.kimad_step(srv.ctx, x_d[None], xh_srv, down_bw, 1.0, srv.out)   # server: compress x - x^, update its x^
        kb.kimad_apply_packed(srv.ctx, srv.out, xh_wrk)                    # workers: the same update from the message
        u_d = a_d[None, :] * (xh_wrk - b_d)
        kb.kimad_step(wrk.ctx, u_d, uh_wrk, up_bw, 1.0, wrk.out)           # workers: compress u - u^, update u^
        kb.kimad_apply_packed(wrk.ctx, wrk.out, uh_srv)                    # server: its copies of u^_m
        kb.kimad_aggregate(x_d, uh_srv, wts, gamma)
        torch.cuda.synchronize()
        assert torch.equal(xh_srv, xh_wrk) and torch.equal(uh_srv, uh_wrk)
        assert np.array_equal(x_d.cpu().numpy().view(np.uint32), xs_ref[k].view(np.uint32)), f"round {k}"


def test_block_granularity_is_a_finer_layer_list():
    """Blocks instead of whole tensors as the unit of allocation: same pass, finer segment list.  At a budget
    where the cells' rounding-up costs little, the finer allocation reaches a lower error."""
    wl = workloads.workload(2, 8)
    blocks = workloads.block_layers(wl.layer_sizes, 16384)
    assert sum(blocks) == wl.N and len(blocks) > len(wl.layer_sizes) and max(blocks) == 16384
    fine = Runner(blocks, 1, wl.ratio_grid, 1000, 0)
    coarse = Runner(wl.layer_sizes, 1, wl.ratio_grid, 1000, 0)
    grads = workloads.gradients(wl, 0, device="cuda")[:1].contiguous()
    budget = [0.2 * 8 * wl.N]
    res_f = fine.compare_step(grads, torch.zeros_like(grads), budget, 1.0)
    res_c = coarse.compare_step(grads, torch.zeros_like(grads), budget, 1.0)
    assert res_f["same_k"] and res_c["same_k"]
    assert float(res_f["ref"].total_err[0]) < float(res_c["ref"].total_err[0])


@pytest.mark.parametrize("cfg,divisor", [(2, 8), (3, 16)])
def test_error_axis_dp_matches_oracle(cfg, divisor):
    """Algorithm 3 with the error as the knapsack axis (policy 2): decisions bit-identical to the oracle's, on its
    own curves and on injected ones."""
    wl = workloads.workload(cfg, divisor)
    r = Runner(wl.layer_sizes, wl.n_workers, wl.ratio_grid, wl.D, wl.value_dtype, policy=2)
    bw = workloads.bandwidth_trace(wl, 60)
    state = torch.zeros((wl.n_workers, wl.N), dtype=torch.float32, device="cuda")
    ks = set()
    for s, b in enumerate((5, 25, 50)):
        grads = workloads.gradients(wl, s, device="cuda")
        res = r.compare_step(grads, state, bw[b], wl.t_target)
        assert np.all(res["forced"].used_bytes <= res["forced"].budget_bytes)
        ks.add(tuple(res["forced"].k[0]))
    assert len(ks) > 1


def test_error_axis_dp_worked_example_and_statuses():
    sizes, grid = [10, 4, 6], [0.25, 0.5, 1.0]
    r = Runner(sizes, 4, grid, 12, 0, policy=2)
    d = torch.tensor([list(range(1, 11)) + [-8, .5, 8, -.5] + [3, -3, 3, 0, -0., 1]] * 4, dtype=torch.float32, device="cuda")
    res = r.compare_step(d, torch.zeros_like(d), [96.0, 112.0, 47.0, 160.0], 1.0)
    assert res["forced"].k.tolist() == [[5, 2, 2], [10, 2, 2], [3, 1, 2], [10, 4, 6]]
    assert list(res["forced"].status) == [0, 0, ko.STATUS_INFEASIBLE, ko.STATUS_PLATEAU]


def test_overlapped_host_driver_gives_the_serial_results_and_feeds_the_monitor():
    """The double-buffered driver (next step copied in and compressed while this step's message is copied out)
    against the plain one-after-the-other driver: same messages, same estimator; the message copies' sizes and
    durations reach the bandwidth monitor."""
    from paper_2312_08053_b200 import pipeline

    wl = workloads.workload(2, 8)
    W, N = wl.n_workers, wl.N
    bw = workloads.bandwidth_trace(wl, 12)
    host = [workloads.gradients(wl, s).pin_memory() for s in range(3)]
    results = {}
    for mode in ("serial", "overlapped"):
        ctx = kb.new_context(wl.layer_sizes, W, wl.ratio_grid, D=wl.D, max_packed_elems=N)
        mon = kb.kimad_monitor_create(window=4, alpha=1.0)
        drv = pipeline.HostDriver(ctx, wl, N, monitor=mon)
        state = torch.zeros((W, N), dtype=torch.float32, device="cuda")
        moved = drv.run(mode, host, state, bw, 7)
        torch.cuda.synchronize()
        last = 6 % 2 if mode == "overlapped" else 0
        st = drv.h_stats[last].numpy().view(kb.STATS_DTYPE).reshape(-1).copy()
        n = int(st["n_selected"][0])
        results[mode] = (moved, state.cpu().numpy().copy(), st, drv.h_idx[last][0, :n].numpy().copy(),
                         drv.h_val[last][0, :n].numpy().copy())
        assert kb.kimad_monitor_estimate(mon) > 0.0  # bytes per second of the message copies
    a, b = results["serial"], results["overlapped"]
    assert a[0] == b[0] and a[0] > 0
    assert np.array_equal(a[1].view(np.uint32), b[1].view(np.uint32))
    assert a[2].tobytes() == b[2].tobytes()
    assert np.array_equal(a[3], b[3]) and np.array_equal(a[4].view(np.uint32), b[4].view(np.uint32))
