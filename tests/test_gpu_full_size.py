"""Parity at the benchmark's full sizes, in the launch configuration bench.py times.

Every element: workload 4 (all layers of all workers) and one whole worker of workload 5 go through the oracle's
complete pass and everything is compared.  The quicker sampled variant below stays as well: (1) for a sample of
layers (always including the largest one) the oracle computes curve, threshold, packed entries and state one
layer at a time and every value is compared; (2) the DP is re-run by the oracle on the GPU's complete curve; (3)
properties that hold at any size are checked on ALL layers: counts, offsets, ascending indices, values
equal to d at the indices, no dropped entry larger than a kept one, untouched entries of the state."""
import numpy as np
import pytest
import torch

from oracle import kimad_oracle as ko
from paper_2312_08053_b200 import binding as kb
from paper_2312_08053_b200 import workloads

pytestmark = pytest.mark.gpu


def _full_size_step(cfg, step_of_trace, sample_layers, workers_checked):
    wl = workloads.workload(cfg)
    W, N, L, K = wl.n_workers, wl.N, wl.L, len(wl.ratio_grid)
    bw_all = workloads.bandwidth_trace(wl)
    bw = bw_all[step_of_trace]
    bpe = 8 if wl.value_dtype == 0 else 6
    cap = int(min(N, np.max(bw) * wl.t_target / bpe + L + 1))
    ctx = kb.new_context(wl.layer_sizes, W, wl.ratio_grid, D=wl.D, value_dtype=wl.value_dtype, max_packed_elems=cap)
    out = kb.Packed(ctx)
    state = torch.zeros((W, N), dtype=torch.float32, device="cuda")
    # one earlier step so that the EF state is not all zero
    g0 = workloads.gradients(wl, 0, device="cuda")
    kb.kimad_step(ctx, g0, state, bw_all[0], wl.t_target, out)
    del g0
    grads = workloads.gradients(wl, 1, device="cuda")
    state_before = state.clone()
    kb.kimad_step(ctx, grads, state, bw, wl.t_target, out)
    status, k_gpu = kb.kimad_get_k(ctx)
    assert status >= 0
    err_g, tau_g, keq_g, shift_g = kb.kimad_debug_get_curve(ctx)
    tau_s, keq_s = kb.kimad_debug_get_selection(ctx)
    st = out.stats_host()
    j_gpu = out.j.cpu().numpy().view(np.uint32)
    offs = out.offs.cpu().numpy().astype(np.int64)
    kt = ko.k_table(wl.layer_sizes, wl.ratio_grid)
    loff = np.concatenate([[0], np.cumsum(wl.layer_sizes)]).astype(np.int64)

    # (2) the DP on the GPU's own curve, and the bookkeeping
    for w in range(W):
        c = ko.budget_bytes(float(bw[w]), wl.t_target)
        s_units, units = ko.units(kt, wl.value_dtype, c, wl.D)
        assert s_units == 0
        s_dp, j_ref, val, cell = ko.dp(err_g[w], units, wl.D)
        assert s_dp == int(st["status"][w]) == 0
        assert np.array_equal(j_ref, j_gpu[w])
        k_ref = kt[np.arange(L), j_ref]
        assert np.array_equal(k_ref.astype(np.uint32), k_gpu[w])
        assert np.array_equal(offs[w], np.concatenate([[0], np.cumsum(k_ref)]).astype(np.int64))
        assert int(st["used_bytes"][w]) == bpe * int(k_ref.sum()) <= c == int(st["budget_bytes"][w])
        tot = np.float32(0)
        for l in range(L):
            tot = np.float32(tot + err_g[w, l, j_ref[l]])
        assert tot == st["total_err"][w]

    # (1) + (3) per layer, on the host copy of one worker at a time
    for w in workers_checked:
        d = (grads[w] - state_before[w]).cpu().numpy()
        g_old = state_before[w].cpu().numpy()
        g_new = state[w].cpu().numpy()
        n_sel = int(offs[w, L])
        idx_all = out.idx[w, :n_sel].cpu().numpy().view(np.uint32)
        val_all = out.val[w, :n_sel].view(torch.int16 if wl.value_dtype else torch.int32).cpu().numpy()
        for l in range(L):
            lo, hi = int(loff[l]), int(loff[l + 1])
            a, b = int(offs[w, l]), int(offs[w, l + 1])
            k = b - a
            idx = idx_all[a:b].astype(np.int64)
            dl = d[lo:hi]
            assert k == int(k_gpu[w, l]) and np.all(np.diff(idx) > 0) and (k == 0 or idx[-1] < hi - lo)
            sent32 = dl[idx]
            if wl.value_dtype == 0:
                assert np.array_equal(val_all[a:b], sent32.view(np.int32))
                sent = sent32
            else:
                ref16 = torch.from_numpy(sent32).to(torch.bfloat16)
                assert np.array_equal(val_all[a:b], ref16.view(torch.int16).numpy())
                sent = ref16.to(torch.float32).numpy()
            expect = g_old[lo:hi].copy()
            expect[idx] = expect[idx] + sent
            assert np.array_equal(expect.view(np.uint32), g_new[lo:hi].view(np.uint32))
            key = dl.view(np.uint32) & np.uint32(0x7FFFFFFF)
            if 0 < k < hi - lo:
                mask = np.zeros(hi - lo, bool)
                mask[idx] = True
                kmin = key[mask].min()
                assert kmin >= key[~mask].max()
                assert kmin == tau_s[w, l]
                eq = np.nonzero(key == kmin)[0]
                kept_eq = eq[mask[eq]]
                assert len(kept_eq) == keq_s[w, l] and np.array_equal(kept_eq, eq[:len(kept_eq)])  # lowest indices first
            if l in sample_layers:  # everything the oracle can say about this layer
                cv = ko.layer_curve(dl, kt[l])
                tol = 1e-5 * np.abs(cv.err.astype(np.float64))
                assert np.all((err_g[w, l] == cv.err) | (np.abs(err_g[w, l].astype(np.float64) - cv.err) <= tol)), (l, err_g[w, l], cv.err)
                ex = (shift_g[w, l] == 0) & (kt[l] < hi - lo)
                assert np.array_equal(tau_g[w, l][ex], cv.tau[ex]) and np.array_equal(keq_g[w, l][ex], cv.keep_eq[ex])
                if 0 < k:
                    oi, ov = ko.select_pack(dl, k, wl.value_dtype)
                    assert np.array_equal(oi.astype(np.int64), idx)
                    assert np.array_equal(ov.view(np.int16 if wl.value_dtype else np.int32), val_all[a:b])
        del d, g_old, g_new
    return kb.kimad_debug_exact_path_layers(ctx, detail=True)


def _every_element(cfg, step_of_trace, workers, zero_rows=0.0):
    """One full-size step in the benchmark's launch configuration, EVERY element of the listed workers compared
    with the oracle's whole pass (curves of all layers and candidates to the curve tolerance; decisions, packed
    indices and values, offsets, statistics and the EF21 state bit for bit)."""
    wl = workloads.workload(cfg)
    W, N, L = wl.n_workers, wl.N, wl.L
    bw_all = workloads.bandwidth_trace(wl)
    bw = bw_all[step_of_trace]
    bpe = 8 if wl.value_dtype == 0 else 6
    cap = int(min(N, np.max(bw_all) * wl.t_target / bpe + L + 1))  # as bench.py sizes the packed buffers
    ctx = kb.new_context(wl.layer_sizes, W, wl.ratio_grid, D=wl.D, value_dtype=wl.value_dtype, max_packed_elems=cap)
    out = kb.Packed(ctx)
    state = torch.zeros((W, N), dtype=torch.float32, device="cuda")
    g0 = workloads.gradients(wl, 0, device="cuda", zero_rows=zero_rows)
    kb.kimad_step(ctx, g0, state, bw_all[0], wl.t_target, out)  # an earlier step: the EF state is not all zero
    del g0
    grads = workloads.gradients(wl, 1, device="cuda", zero_rows=zero_rows)
    state_before = state.clone()
    kb.kimad_step(ctx, grads, state, bw, wl.t_target, out)
    status, k_gpu = kb.kimad_get_k(ctx)
    assert status == 0
    err_g, tau_g, keq_g, shift_g = kb.kimad_debug_get_curve(ctx)
    tau_s, keq_s = kb.kimad_debug_get_selection(ctx)
    st = out.stats_host()
    j_gpu = out.j.cpu().numpy().view(np.uint32)
    offs_g = out.offs.cpu().numpy().astype(np.uint64)
    sizes = np.array(wl.layer_sizes, np.uint32)
    kt = ko.k_table(wl.layer_sizes, wl.ratio_grid)
    for w in workers:
        g_host = grads[w:w + 1].cpu().numpy()
        s_host = state_before[w:w + 1].cpu().numpy()
        ref = ko.step(wl.layer_sizes, 1, wl.ratio_grid, wl.D, wl.value_dtype, g_host, s_host, [bw[w]], wl.t_target,
                      cap=cap)
        # (b) the curve of every layer and candidate
        tol = 1e-5 * np.abs(ref.err[0].astype(np.float64))
        bad = (err_g[w] != ref.err[0]) & ~(np.abs(err_g[w].astype(np.float64) - ref.err[0].astype(np.float64)) <= tol)
        assert not bad.any(), np.argwhere(bad)[:5]
        full = kt == sizes[:, None].astype(np.uint64)
        ex = (shift_g[w] == 0) & ~full
        assert np.array_equal(tau_g[w][ex], ref.tau[0][ex]) and np.array_equal(keq_g[w][ex], ref.keep_eq[0][ex])
        lazy = (shift_g[w] != 0) & ~full
        assert np.all((ref.tau[0][lazy] >= tau_g[w][lazy]) &
                      (ref.tau[0][lazy] - tau_g[w][lazy] < (1 << shift_g[w][lazy].astype(np.uint64))))
        # (c) decisions: the oracle's own curve must lead to the same k here; if the two curves (equal within the
        # tolerance) ever led to different decisions, the oracle's DP is run on the GPU's curve instead
        if not np.array_equal(ref.k[0], k_gpu[w]):
            ref = ko.step(wl.layer_sizes, 1, wl.ratio_grid, wl.D, wl.value_dtype, g_host, s_host, [bw[w]],
                          wl.t_target, cap=cap, inject_err=err_g[w:w + 1])
        assert np.array_equal(ref.j[0], j_gpu[w]) and np.array_equal(ref.k[0], k_gpu[w])
        assert np.array_equal(ref.offs[0], offs_g[w])
        assert int(st["status"][w]) == int(ref.status[0]) and int(st["used_bytes"][w]) == int(ref.used_bytes[0])
        assert int(st["n_selected"][w]) == int(ref.n_selected[0]) and int(st["budget_bytes"][w]) == int(ref.budget_bytes[0])
        # (d) exact thresholds of the chosen candidates
        jj = ref.j[0].astype(np.int64)
        part = (ref.k[0] > 0) & (ref.k[0] < sizes)
        assert np.array_equal(tau_s[w][part], ref.tau[0][np.arange(L), jj][part])
        assert np.array_equal(keq_s[w][part], ref.keep_eq[0][np.arange(L), jj][part])
        # (e) + (f) every packed entry and every element of the state
        n = int(ref.offs[0, L])
        assert np.array_equal(out.idx[w, :n].cpu().numpy().view(np.uint32), ref.idx[0, :n])
        val_g = out.val[w, :n].view(torch.int16 if wl.value_dtype else torch.int32).cpu().numpy()
        assert np.array_equal(val_g, ref.val[0, :n].view(np.int16 if wl.value_dtype else np.int32))
        assert np.array_equal(state[w].cpu().numpy().view(np.uint32), ref.state[0].view(np.uint32))
        del g_host, s_host, ref


def test_gpt2_small_shape_full_size_every_element():
    # all 148 layers of all 4 workers (4 x 124.4 M elements), a low-budget step of the trace
    _every_element(4, step_of_trace=7, workers=[0, 1, 2, 3])


def test_gpt2_small_shape_full_size_every_element_burst():
    # a burst of the trace (25 Gbit/s: about 16 % of the entries kept), one worker
    bw = workloads.bandwidth_trace(workloads.workload(4))
    _every_element(4, step_of_trace=int(np.argmax(bw[:, 0])), workers=[2])


def test_llama_1b_shape_full_size_sparse_embedding_rows():
    # 90 % of the token embedding's gradient rows exactly zero (drawn per worker and step): the 65.5 M-element layer
    # is swept without its zeros, its loose candidates are refined; a high-budget step, so that candidates whose
    # threshold lies among the zeros are in play; every element of one worker
    bw = workloads.bandwidth_trace(workloads.workload(5))
    _every_element(5, step_of_trace=int(np.argmax(bw[:, 0])), workers=[0], zero_rows=0.9)


def test_gpt2_small_shape_full_size_sparse_embedding_rows():
    _every_element(4, step_of_trace=7, workers=[1, 3], zero_rows=0.6)


def test_llama_1b_shape_full_size_every_element_of_one_worker():
    # all 201 layers of one worker (1.1 G elements, bf16 values)
    _every_element(5, step_of_trace=30, workers=[1])


@pytest.mark.parametrize("block,D", [(65536, 4096), (16384, 8191)])
def test_gpt2_small_shape_full_size_in_blocks(block, D):
    """Block granularity (the paper's Section 5: from layers to blocks) on a full-size workload: the GPT-2-small
    shaped gradient of one worker (124.4 M elements) cut into blocks of 64 K and of 16 K elements (1995 and 7686
    segments; every segment takes at least one budget cell, so D >= segments), every element compared."""
    from tests._harness import Runner

    wl = workloads.workload(4)
    blocks = workloads.block_layers(wl.layer_sizes, block)
    assert sum(blocks) == wl.N and max(blocks) == block and len(blocks) <= D
    r = Runner(blocks, 1, wl.ratio_grid, D, 0)
    grads = workloads.gradients(wl, 3, device="cuda", workers=[1])
    state = (workloads.gradients(wl, 2, device="cuda", workers=[1]) * 0.5).contiguous()  # a non-trivial estimator
    bw = workloads.bandwidth_trace(wl)
    res = r.compare_step(grads, state, [float(bw[int(np.argmax(bw[:, 0])), 0]) * 0.3], wl.t_target, check_inject=False)
    assert res["status"] == 0
    k = res["forced"].k[0]
    assert len(set(k.tolist())) > 3  # the blocks of one tensor do not all get the same k


def test_gpt2_small_shape_full_size():
    # 4 workers x 124.4 M elements; layers: the 38.6 M embedding, position table, one of each block tensor, last norm
    why = _full_size_step(4, step_of_trace=7, sample_layers={0, 1, 2, 4, 6, 10, 12, 147}, workers_checked=[0, 3])
    assert why[0] <= 8, why


def test_llama_1b_shape_full_size_bf16():
    # 2 workers x 1.1 G elements, bf16 values; layers: 65.5 M embedding, q/k proj, one FFN matrix, a norm, lm_head slot
    why = _full_size_step(5, step_of_trace=30, sample_layers={0, 2, 3, 7, 10}, workers_checked=[1])
    assert why[0] <= 60, why


@pytest.mark.parametrize("n", [(1 << 28) + 3, (1 << 31) + 5, (1 << 32) - 1])
def test_one_very_large_layer(n):
    """A single layer far larger than any in the workloads (8193 chunks and more, a ragged last one; the larger
    sizes cross 2^31 layer-local indices and reach the largest layer the interface takes): the curve of every candidate against a full sort done by torch on the
    device, and the selection properties on all entries.  The state starts at zero so that d = grad."""
    grid = [0.0001, 0.003, 0.05, 0.4, 1.0]
    torch.cuda.empty_cache()  # blocks cached from earlier tests do not count as free
    free_bytes, _ = torch.cuda.mem_get_info()
    if free_bytes < 30 * n:  # inputs, scratch and the reference sort take about 26 bytes per element at the peak
        pytest.skip(f"needs {30 * n / 2**30:.0f} GiB of free device memory")
    ctx = kb.new_context([n], 1, grid, D=1000, value_dtype=0, max_packed_elems=n // 64)
    out = kb.Packed(ctx)
    gen = torch.Generator(device="cuda").manual_seed(28)
    grads = torch.randn((1, n), device="cuda", generator=gen)
    grads.mul_(torch.randn((1, n), device="cuda", generator=gen).abs_())  # heavier tails than a normal
    state = torch.zeros((1, n), device="cuda")
    d = grads[0]
    kb.kimad_step(ctx, grads, state, [0.02 * 8 * n], 1.0, out)
    status, k_gpu = kb.kimad_get_k(ctx)
    assert status == 0
    kt = ko.k_table([n], grid)[0]
    err_g, tau_g, keq_g, shift_g = kb.kimad_debug_get_curve(ctx)
    # curve: squares of the n - k smallest magnitudes, summed in float64.  torch sorts at most 2^31 - 1 elements,
    # so the magnitudes are sorted in three parts; the k-th largest of the union is found by bisection over the
    # 31-bit keys with searchsorted on the parts, and the dropped squares come from the parts' prefix sums.
    third = n // 3
    parts = []
    for a, b in ((0, third), (third, 2 * third), (2 * third, n)):
        srt, _ = torch.sort(d[a:b].abs())
        parts.append((srt.view(torch.int32), torch.cumsum(srt.double().square_(), 0)))
        del srt

    def count_below(key, right):  # entries with magnitude key < `key` (right=False) or <= `key` (right=True)
        probe = torch.tensor([key], dtype=torch.int32, device="cuda")
        return [int(torch.searchsorted(p[0], probe, right=right)) for p in parts]

    for j, k in enumerate(kt):
        drop = n - int(k)
        want = 0.0
        if drop:
            lo, hi = 0, 0x7F800000  # smallest key with at least `drop` entries <= key: the largest dropped magnitude
            while lo < hi:
                mid = (lo + hi) // 2
                if sum(count_below(mid, True)) >= drop:
                    hi = mid
                else:
                    lo = mid + 1
            below = count_below(lo, False)
            for p, c in zip(parts, below):
                want += float(p[1][c - 1]) if c else 0.0
            v = float(torch.tensor([lo], dtype=torch.int32).view(torch.float32))
            want += (drop - sum(below)) * v * v  # dropped entries equal to that magnitude
        assert abs(float(err_g[0, 0, j]) - want) <= 1e-5 * want, (j, err_g[0, 0, j], want)
    del parts
    j = int(out.j[0, 0])
    assert j == 1 and int(k_gpu[0, 0]) == int(kt[1])  # 0.3 % fits 2 % of the dense bytes, 5 % does not
    k = int(kt[j])
    idx = out.idx[0, :k].long() & 0xFFFFFFFF  # u32 indices stored in an int32 tensor
    val = out.val[0, :k]
    assert bool(torch.all(idx[1:] > idx[:-1])) and int(idx[-1]) < n
    assert torch.equal(val.view(torch.int32), d[idx].view(torch.int32))
    kept = torch.zeros(n, dtype=torch.bool, device="cuda")
    kept[idx] = True
    key = d.view(torch.int32) & 0x7FFFFFFF
    assert int(key[kept].min()) >= int(key[~kept].max())
    del key
    assert int(torch.count_nonzero(state[0])) == int(torch.count_nonzero(val))  # nothing but the kept entries changed
    assert torch.equal(state[0][idx].view(torch.int32), val.view(torch.int32))
    assert kb.kimad_debug_exact_path_layers(ctx) == 0
