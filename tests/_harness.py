"""Shared driver for the GPU parity tests: runs the CUDA library through its C ABI and the CPU oracle on
the same seeded inputs and compares stage by stage."""
from __future__ import annotations

import os

import numpy as np
import torch

from oracle import kimad_oracle as ko
from paper_2312_08053_b200 import binding as kb

ERR_RTOL = 1e-5  # acceptance bound on the error curve (relative, float32)


def u32(t):
    return t.cpu().numpy().view(np.uint32)


class Runner:
    def __init__(self, layer_sizes, W, grid, D=1000, value_dtype=0, stride=None, cap=None, check_finite=0,
                 curve_mode=0, policy=0, cost_model=0, schedule=0):
        self.ls, self.W, self.grid, self.D, self.vd = list(layer_sizes), W, list(grid), D, value_dtype
        self.policy, self.cost_model = policy, cost_model
        self.N = int(sum(self.ls))
        self.stride = stride or self.N
        self.cap = cap or self.N
        self.ctx = kb.new_context(self.ls, W, self.grid, D=D, value_dtype=value_dtype, worker_stride=self.stride,
                                  max_packed_elems=self.cap, check_finite=check_finite, curve_mode=curve_mode,
                                  policy=policy, cost_model=cost_model)
        kb.kimad_debug_set_schedule(self.ctx, schedule)  # 1: two groups of workers on two streams whenever W >= 2
        self.out = kb.Packed(self.ctx)
        self.kt = ko.k_table(self.ls, self.grid)

    def gpu_step(self, grads, state, bw, t):
        kb.kimad_step(self.ctx, grads, state, bw, t, self.out)
        status, k = kb.kimad_get_k(self.ctx)
        return status, k

    def compare_step(self, grads, state, bw, t, check_inject=True):
        """One teacher-forced step: GPU and oracle both start from (grads, state).  `state` (cuda tensor) is
        updated in place by the GPU.  Returns a dict of observations."""
        W, L, K = self.W, len(self.ls), len(self.grid)
        g_host = grads.cpu().numpy()
        s_host = state.cpu().numpy().copy()
        status, k_gpu = self.gpu_step(grads, state, bw, t)
        err_g, tau_g, keq_g, shift_g = kb.kimad_debug_get_curve(self.ctx)
        tau_s, keq_s = kb.kimad_debug_get_selection(self.ctx)
        # oracle on its own curves
        ref = ko.step(self.ls, W, self.grid, self.D, self.vd, g_host, s_host, bw, t, cap=self.cap,
                      policy=self.policy, cost_model=self.cost_model)
        # (b) curve: thresholds exact, error within tolerance
        # where all 31 bits were resolved the threshold must be the oracle's; elsewhere the oracle's
        # threshold must lie in the reported key interval
        exact = shift_g == 0
        if self.policy == 3:  # the one candidate of every (worker, layer) is the ratio fitted to the worker's budget
            full = (ref.k == np.array(self.ls, np.uint32)[None, :])[:, :, None]
        else:
            full = np.broadcast_to((self.kt == np.array(self.ls, np.uint64)[:, None])[None], exact.shape)  # k = n: no threshold
        chk = exact & ~full
        assert np.array_equal(tau_g[chk], ref.tau[chk]), "tau differs"
        assert np.array_equal(keq_g[chk], ref.keep_eq[chk]), "keep_eq differs"
        lazy = ~exact & ~full
        assert np.all(shift_g <= 15)
        assert np.all((ref.tau[lazy] >= tau_g[lazy]) & (ref.tau[lazy] - tau_g[lazy] < (1 << shift_g[lazy].astype(np.uint64))))
        self.n_exact, self.n_lazy = int(chk.sum()), int(lazy.sum())
        tol = ERR_RTOL * np.abs(ref.err.astype(np.float64))
        with np.errstate(invalid="ignore"):
            bad = (err_g != ref.err) & ~(np.abs(err_g.astype(np.float64) - ref.err.astype(np.float64)) <= tol)
        assert not bad.any(), f"err off at {np.argwhere(bad)[:5]}: {err_g[bad][:5]} vs {ref.err[bad][:5]}"
        # (c)-(f): oracle DP fed the GPU's curve must reproduce the GPU bit for bit
        forced = ko.step(self.ls, W, self.grid, self.D, self.vd, g_host, s_host, bw, t, cap=self.cap,
                         inject_err=err_g, policy=self.policy, cost_model=self.cost_model)
        st = self.out.stats_host()
        assert np.array_equal(st["status"], forced.status), (st["status"], forced.status)
        assert np.array_equal(u32(self.out.j), forced.j), "chosen candidates differ from oracle DP on the same curve"
        assert np.array_equal(k_gpu, forced.k)
        assert np.array_equal(u32(self.out.dense), forced.dense), "dense flags differ"
        # the exact threshold found for the chosen candidate of every layer
        jj = forced.j.astype(np.int64)
        t_ref = np.take_along_axis(ref.tau, jj[:, :, None], axis=2)[:, :, 0]
        q_ref = np.take_along_axis(ref.keep_eq, jj[:, :, None], axis=2)[:, :, 0]
        part = (forced.k > 0) & (forced.k < np.array(self.ls, np.uint32)[None, :]) & (forced.status[:, None] >= 0)
        assert np.array_equal(tau_s[part], t_ref[part]), "chosen thresholds differ"
        assert np.array_equal(keq_s[part], q_ref[part]), "kept ties differ"
        assert np.array_equal(self.out.offs.cpu().numpy().astype(np.uint64), forced.offs)
        assert np.array_equal(st["budget_bytes"], forced.budget_bytes)
        assert np.array_equal(st["used_bytes"], forced.used_bytes)
        assert np.array_equal(st["n_selected"], forced.n_selected)
        assert np.array_equal(st["total_err"].view(np.uint32), forced.total_err.view(np.uint32))
        idx_g = u32(self.out.idx)
        val_g = self.out.val.view(torch.int16 if self.vd else torch.int32).cpu().numpy()
        val_r = forced.val.view(np.int16 if self.vd else np.int32)
        for w in range(W):
            n = int(forced.offs[w, L])
            assert np.array_equal(idx_g[w, :n], forced.idx[w, :n]), f"packed indices differ (worker {w})"
            assert np.array_equal(val_g[w, :n], val_r[w, :n]), f"packed values differ (worker {w})"
        assert np.array_equal(u32(state), forced.state.view(np.uint32)), "EF21 state differs"
        same_k = np.array_equal(ref.k, forced.k)
        # DP fed the ORACLE's curve must give the oracle's decisions bit for bit
        if check_inject:
            scratch = torch.from_numpy(s_host).cuda()
            out2 = kb.Packed(self.ctx)
            kb.kimad_debug_step_with_err(self.ctx, grads, scratch, bw, t, out2, torch.from_numpy(ref.err).cuda())
            torch.cuda.synchronize()
            assert np.array_equal(u32(out2.j), ref.j), "DP on injected oracle curves differs"
            assert np.array_equal(u32(out2.k), ref.k)
            assert np.array_equal(u32(scratch), ref.state.view(np.uint32))
            assert np.array_equal(out2.stats_host()["total_err"].view(np.uint32), ref.total_err.view(np.uint32))
        # checked build of the library (KIMAD_CHECKED=1): no index test failed, no canary between workspace regions damaged
        checked, failed, damaged = kb.kimad_debug_check(self.ctx)
        assert checked == (os.environ.get("KIMAD_CHECKED") == "1")
        assert failed == 0 and damaged == 0, (hex(failed), damaged)
        return dict(status=status, same_k=same_k, ref=ref, forced=forced)
