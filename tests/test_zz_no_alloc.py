"""The allocation-free entry point (scratch inside the library's device image) against kimad_step.

Collected last on purpose: a run that stops at the first failure has then already run every other test.
Who needs it: callers that may not allocate device memory -- a gradient hook running beside busy streams
(cudaMalloc would synchronise the device), or a plug-in in a runtime that owns all device memory."""
import numpy as np
import pytest
import torch

from paper_2312_08053_b200 import binding as kb
from paper_2312_08053_b200 import workloads

pytestmark = pytest.mark.gpu


def _outputs(out, state, n_sel):
    return (out.k.cpu().numpy().copy(), out.j.cpu().numpy().copy(), out.offs.cpu().numpy().copy(),
            out.stats.cpu().numpy().copy(), out.idx.cpu().numpy()[:, :n_sel].copy(),
            out.val.view(torch.int32).cpu().numpy()[:, :n_sel].copy(), state.cpu().numpy().view(np.uint32).copy())


def test_builtin_scratch_matches_kimad_step_twice_in_a_row():
    wl = workloads.workload(1)  # 101,770 elements: well inside the built-in scratch
    bw = workloads.bandwidth_trace(wl, 1)[0]
    # reference: the ordinary entry point with a caller-owned workspace
    ref_ctx = kb.new_context(wl.layer_sizes, wl.n_workers, wl.ratio_grid, D=wl.D)
    assert kb.kimad_workspace_bytes(ref_ctx) <= kb.KIMAD_BUILTIN_SCRATCH_BYTES
    ref_out = kb.Packed(ref_ctx)
    ref_state = torch.zeros((wl.n_workers, wl.N), dtype=torch.float32, device="cuda")
    # under test: a context that never gets a workspace
    ctx = kb.kimad_create(wl.layer_sizes, wl.n_workers, wl.ratio_grid, D=wl.D)
    out = kb.Packed(ctx)
    state = torch.zeros_like(ref_state)
    for step in range(2):  # two calls in a row: the second one meets the first one's leftovers in the array
        grads = workloads.gradients(wl, step, device="cuda")
        kb.kimad_step(ref_ctx, grads, ref_state, bw, wl.t_target, ref_out)
        st_ref, _ = kb.kimad_get_k(ref_ctx)
        kb.kimad_step_builtin_scratch(ctx, grads, state, bw, wl.t_target, out)
        st_new, _ = kb.kimad_get_k(ctx)
        assert st_ref == st_new == 0
        n_sel = int(ref_out.stats_host()["n_selected"].max())
        assert n_sel > 0
        for a, b in zip(_outputs(ref_out, ref_state, n_sel), _outputs(out, state, n_sel)):
            assert np.array_equal(a, b)


def test_builtin_scratch_is_shared_by_contexts_of_different_shape():
    """Every context on a device uses the one built-in array.  A step of another context (other layer list, worker
    count, ratio grid; exact radix path everywhere, so that its histograms, lists and tables land on other offsets
    and get dirtied) runs between two calls of the first one: each call must bring in its own tables and clear what
    has to start at zero, whatever the previous call left."""
    wl = workloads.workload(1)
    bw = workloads.bandwidth_trace(wl, 1)[0]
    ref_ctx = kb.new_context(wl.layer_sizes, wl.n_workers, wl.ratio_grid, D=wl.D)
    ref_out = kb.Packed(ref_ctx)
    ref_state = torch.zeros((wl.n_workers, wl.N), dtype=torch.float32, device="cuda")
    ctx = kb.kimad_create(wl.layer_sizes, wl.n_workers, wl.ratio_grid, D=wl.D)
    out = kb.Packed(ctx)
    state = torch.zeros_like(ref_state)
    # the other context: 3 workers, 5 layers, 4 ratios, exact path for every layer above the tiny size
    o_sizes, o_grid, o_W = [9000, 17, 30011, 4097, 5], [0.003, 0.04, 0.3, 1.0], 3
    o_ref = kb.new_context(o_sizes, o_W, o_grid, D=200, curve_mode=1)
    o_ctx = kb.kimad_create(o_sizes, o_W, o_grid, D=200, curve_mode=1)
    assert kb.kimad_workspace_bytes(o_ctx) <= kb.KIMAD_BUILTIN_SCRATCH_BYTES
    o_out_ref, o_out = kb.Packed(o_ref), kb.Packed(o_ctx)
    gen = torch.Generator(device="cuda").manual_seed(5)
    o_N = sum(o_sizes)
    for step in range(3):
        grads = workloads.gradients(wl, step, device="cuda")
        kb.kimad_step(ref_ctx, grads, ref_state, bw, wl.t_target, ref_out)
        kb.kimad_step_builtin_scratch(ctx, grads, state, bw, wl.t_target, out)
        assert kb.kimad_get_k(ref_ctx)[0] == kb.kimad_get_k(ctx)[0] == 0
        n_sel = int(ref_out.stats_host()["n_selected"].max())
        for a, b in zip(_outputs(ref_out, ref_state, n_sel), _outputs(out, state, n_sel)):
            assert np.array_equal(a, b)
        # the other context's step on the same array
        o_grads = torch.randn((o_W, o_N), device="cuda", generator=gen) * 0.01
        s1, s2 = torch.zeros_like(o_grads), torch.zeros_like(o_grads)
        o_bw = [0.1 * 8 * o_N, 0.3 * 8 * o_N, 0.02 * 8 * o_N]
        kb.kimad_step(o_ref, o_grads, s1, o_bw, 1.0, o_out_ref)
        kb.kimad_step_builtin_scratch(o_ctx, o_grads, s2, o_bw, 1.0, o_out)
        assert kb.kimad_get_k(o_ref)[0] == kb.kimad_get_k(o_ctx)[0] == 0
        n_sel = int(o_out_ref.stats_host()["n_selected"].max())
        for a, b in zip(_outputs(o_out_ref, s1, n_sel), _outputs(o_out, s2, n_sel)):
            assert np.array_equal(a, b)


def test_builtin_scratch_refuses_bad_arguments_before_touching_the_array():
    import ctypes
    wl = workloads.workload(1)
    ctx = kb.kimad_create(wl.layer_sizes, wl.n_workers, wl.ratio_grid)
    out = kb.kimad_packed(1, 1, 1, 1, 1, 1)
    bw = (ctypes.c_double * 1)(1.0)
    L = kb.load()
    assert L.kimad_step_builtin_scratch(ctx.handle, None, 1, bw, 1.0, ctypes.byref(out), None) == kb.KIMAD_ERR_INVALID_ARG
    assert L.kimad_step_builtin_scratch(ctx.handle, 1, 1, bw, -1.0, ctypes.byref(out), None) == kb.KIMAD_ERR_INVALID_ARG
    assert L.kimad_step_builtin_scratch(None, 1, 1, bw, 1.0, ctypes.byref(out), None) == kb.KIMAD_ERR_INVALID_ARG


def test_builtin_scratch_rejects_large_problems():
    wl = workloads.workload(2)  # 4 workers x 11.7 M elements
    ctx = kb.kimad_create(wl.layer_sizes, wl.n_workers, wl.ratio_grid)
    assert kb.kimad_workspace_bytes(ctx) > kb.KIMAD_BUILTIN_SCRATCH_BYTES
    out = kb.kimad_packed(1, 1, 1, 1, 1, 1)
    import ctypes
    rc = kb.load().kimad_step_builtin_scratch(ctx.handle, 1, 1, (ctypes.c_double * 4)(1, 1, 1, 1), 1.0,
                                             ctypes.byref(out), None)
    assert rc == kb.KIMAD_ERR_TOO_LARGE
    assert "built-in" in kb.kimad_strerror(rc)
