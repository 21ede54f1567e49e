"""Host-side pieces around the pass (no GPU): the issue plan of the double-buffered driver and the bandwidth
monitor of the C ABI (Section 2.4: every device estimates its bandwidth from what it observed; Section 5: the
pass can be overlapped with communication)."""
import random

import numpy as np
import pytest

from paper_2312_08053_b200 import binding as kb
from paper_2312_08053_b200 import pipeline


# ----------------------------------------------------------------------------- plan
@pytest.mark.parametrize("n", [0, 1, 2, 3, 4, 9])
def test_plans_are_hazard_free(n):
    assert pipeline.check_plan(pipeline.plan(n, "serial"), 1, 1)
    assert pipeline.check_plan(pipeline.plan(n, "overlapped"), 2, 2)


def test_overlapped_plan_queues_the_next_pass_before_the_host_waits():
    ops = pipeline.plan(5, "overlapped")
    kinds = [(o.kind, o.step) for o in ops]
    for s in range(4):  # the pass of step s + 1 is enqueued before the host blocks on step s's statistics
        assert kinds.index(("step", s + 1)) < kinds.index(("host_wait_stats", s))
    # the message copy runs on a stream of its own, the input copy on another
    assert {o.stream for o in ops if o.kind == "d2h"} == {pipeline.S_OUT}
    assert {o.stream for o in ops if o.kind == "h2d"} == {pipeline.S_IN}


@pytest.mark.parametrize("drop", [("step", "h2d"), ("step", "d2h")])
def test_checker_catches_a_missing_wait(drop):
    """Removing either kind of event wait of the passes (input copied, output buffer uploaded) leaves a buffer
    hazard that the checker reports.  (The waits of the copies on earlier passes are implied by the host having
    waited for those passes' statistics; they stay in the plan so that it does not depend on that.)"""
    ops = pipeline.plan(6, "overlapped")
    hit = False
    for o in ops:
        if o.kind == drop[0]:
            before = len(o.waits)
            o.waits = [w for w in o.waits if w[0] != drop[1]]
            hit |= len(o.waits) != before
    assert hit
    with pytest.raises(AssertionError):
        pipeline.check_plan(ops, 2, 2)


def _linearize(ops, rng):
    """A random execution order the plan allows: stream order, event waits and host waits are respected, nothing
    else (ops of different streams run as late or as early as the rules permit)."""
    pos = {(o.kind, o.step): i for i, o in enumerate(ops)}
    n = len(ops)
    deps = [set() for _ in range(n)]
    last = {}
    barrier = None
    for i, o in enumerate(ops):
        if o.kind.startswith("host_wait"):
            barrier = pos[("stats" if o.kind == "host_wait_stats" else "d2h", o.step)]
            continue
        if o.stream in last:
            deps[i].add(last[o.stream])
        deps[i] |= {pos[w] for w in o.waits}
        if barrier is not None:
            deps[i].add(barrier)
        last[o.stream] = i
        if o.host_sync:
            barrier = i
    real = [i for i, o in enumerate(ops) if not o.kind.startswith("host_wait")]
    done, order = set(), []
    while len(order) < len(real):
        ready = [i for i in real if i not in done and deps[i] <= done]
        pick = rng.choice(ready)
        done.add(pick)
        order.append(pick)
    return order


def test_overlapped_execution_gives_the_serial_results():
    """A stand-in pass (a fixed integer function of input and state) run under random legal interleavings of the
    overlapped plan produces, step by step, what the serial plan produces."""
    n_steps, size = 7, 16
    rng_np = np.random.default_rng(1)
    host_in = [rng_np.integers(0, 1000, size) for _ in range(n_steps)]

    def execute(ops, order):
        dev_in = [np.zeros(size, np.int64) for _ in range(2)]
        dev_out = [np.zeros(size, np.int64) for _ in range(2)]
        stats = [0, 0]
        state = np.zeros(size, np.int64)
        result = {}
        for i in order:
            o = ops[i]
            if o.kind == "h2d":
                dev_in[o.in_buf][:] = host_in[o.step]
            elif o.kind == "step":
                dev_out[o.out_buf][:] = dev_in[o.in_buf] * 3 + state
                state += dev_in[o.in_buf] % 7
            elif o.kind == "stats":
                stats[o.out_buf] = int(dev_out[o.out_buf].sum())
            elif o.kind == "d2h":
                result[o.step] = (stats[o.out_buf], dev_out[o.out_buf].copy())
        return result

    serial = pipeline.plan(n_steps, "serial")
    want = execute(serial, [i for i in range(len(serial))])
    ops = pipeline.plan(n_steps, "overlapped")
    for seed in range(50):
        got = execute(ops, _linearize(ops, random.Random(seed)))
        assert got.keys() == want.keys()
        for s in want:
            assert got[s][0] == want[s][0] and np.array_equal(got[s][1], want[s][1]), (seed, s)


# ----------------------------------------------------------------------------- monitor
def test_monitor_constant_link_is_reported_exactly():
    m = kb.kimad_monitor_create(window=4, alpha=1.0)
    assert kb.kimad_monitor_estimate(m) == 0.0
    for _ in range(9):
        kb.kimad_monitor_observe(m, 1 << 20, 0.5)
        assert kb.kimad_monitor_estimate(m) == (1 << 20) / 0.5


def test_monitor_window_forgets_the_old_link_after_window_transfers():
    m = kb.kimad_monitor_create(window=3, alpha=1.0)
    for _ in range(5):
        kb.kimad_monitor_observe(m, 1000, 1.0)       # 1000 B/s
    kb.kimad_monitor_observe(m, 4000, 1.0)           # link got faster: 4000 B/s
    assert kb.kimad_monitor_estimate(m) == (1000 + 1000 + 4000) / 3.0
    kb.kimad_monitor_observe(m, 4000, 1.0)
    kb.kimad_monitor_observe(m, 4000, 1.0)
    assert kb.kimad_monitor_estimate(m) == 4000.0    # three transfers later nothing of the old link is left


def test_monitor_weighs_by_time_not_by_transfer():
    # 10 s at 100 B/s and 1 s at 1000 B/s: 2000 B in 11 s, not the mean of the two rates
    m = kb.kimad_monitor_create(window=8, alpha=1.0)
    kb.kimad_monitor_observe(m, 1000, 10.0)
    kb.kimad_monitor_observe(m, 1000, 1.0)
    assert kb.kimad_monitor_estimate(m) == pytest.approx(2000.0 / 11.0, rel=1e-15)


def test_monitor_smoothing_follows_the_geometric_closed_form():
    # window 1, alpha a: after a jump from r0 to r1 the estimate is r1 + (r0 - r1) (1 - a)^t after t transfers
    a, r0, r1 = 0.25, 800.0, 200.0
    m = kb.kimad_monitor_create(window=1, alpha=a)
    kb.kimad_monitor_observe(m, 800, 1.0)
    assert kb.kimad_monitor_estimate(m) == r0
    for t in range(1, 12):
        kb.kimad_monitor_observe(m, 200, 1.0)
        assert kb.kimad_monitor_estimate(m) == pytest.approx(r1 + (r0 - r1) * (1 - a) ** t, rel=1e-12)


def test_monitor_rejects_bad_arguments():
    import ctypes as C

    L = kb.load()
    h = C.c_void_p()
    assert L.kimad_monitor_create(C.byref(h), 0, 1.0) == kb.KIMAD_ERR_INVALID_ARG
    assert L.kimad_monitor_create(C.byref(h), 4, 0.0) == kb.KIMAD_ERR_INVALID_ARG
    assert L.kimad_monitor_create(C.byref(h), 4, 1.5) == kb.KIMAD_ERR_INVALID_ARG
    m = kb.kimad_monitor_create(window=2, alpha=1.0)
    for sec in (0.0, -1.0, float("nan"), float("inf")):
        assert L.kimad_monitor_observe(m.handle, 10, sec) == kb.KIMAD_ERR_INVALID_ARG
    assert kb.kimad_monitor_estimate(m) == 0.0  # nothing was recorded


def test_monitor_estimate_drives_the_budget_of_section_3_1():
    """The estimate is the B of Eq. 2: with a 50 ms one-way target the budget is floor(B * t) bytes."""
    m = kb.kimad_monitor_create(window=4, alpha=1.0)
    kb.kimad_monitor_observe(m, 6_250_000, 0.05)      # 1 Gbit/s
    ctx = kb.kimad_create([1000, 10], 1, [0.1, 1.0])
    st, c, _ = kb.kimad_plan_budget(ctx, kb.kimad_monitor_estimate(m), 0.05)
    assert c == 6_250_000
