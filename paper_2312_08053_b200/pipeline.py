"""Host side of a training loop around the compression pass: copy a step's gradients to the device, run
``kimad_step``, bring the packed message back (the "upload"), and feed the measured upload times to the
bandwidth monitor.  The paper notes that the Kimad+ pass "can be overlapped with communication" (Section 5);
``plan()`` lays the three activities of consecutive steps over three streams with two buffers each, and
``HostDriver`` issues that plan through torch streams and events.  No method arithmetic lives here: the pass
itself is ``kimad_step`` of the CUDA library.

The plan is plain data (a list of ``Op``), so that its ordering rules can be checked without a GPU: every
buffer hazard must be covered by stream order or by an event wait (``check_plan``).
"""
from __future__ import annotations

from dataclasses import dataclass, field

# streams
S_IN, S_COMPUTE, S_OUT = 0, 1, 2


@dataclass
class Op:
    kind: str            # "h2d" | "step" | "stats" | "d2h"
    step: int
    stream: int
    in_buf: int = -1     # device input buffer read or written
    out_buf: int = -1    # packed-output buffer read or written
    waits: list = field(default_factory=list)  # (kind, step) of ops on OTHER streams that must have finished
    host_sync: bool = False  # the host waits for this op before it issues what follows


def plan(n_steps: int, mode: str = "overlapped"):
    """Issue order of the host for ``n_steps`` steps.

    serial: copy in, step, copy the statistics out and wait for them, copy the message out, wait; one buffer.
    overlapped: two input buffers and two output buffers.  Step s + 1 is copied in and its pass enqueued BEFORE
    the host waits for step s's statistics (they size the message copy), so the device always has the next
    step's work queued while the host sizes and the copy engine uploads step s's message."""
    ops = []
    if mode == "serial":
        for s in range(n_steps):
            ops.append(Op("h2d", s, S_COMPUTE, in_buf=0))
            ops.append(Op("step", s, S_COMPUTE, in_buf=0, out_buf=0))
            ops.append(Op("stats", s, S_COMPUTE, out_buf=0, host_sync=True))
            ops.append(Op("d2h", s, S_COMPUTE, out_buf=0, host_sync=True))
        return ops
    if mode != "overlapped":
        raise ValueError(mode)

    def issue_in_and_step(s):
        b = s % 2
        w_in = [("step", s - 2)] if s >= 2 else []           # the pass that last read this input buffer
        ops.append(Op("h2d", s, S_IN, in_buf=b, waits=w_in))
        w_c = [("h2d", s)] + ([("d2h", s - 2)] if s >= 2 else [])  # input there; output buffer uploaded
        ops.append(Op("step", s, S_COMPUTE, in_buf=b, out_buf=b, waits=w_c))
        ops.append(Op("stats", s, S_COMPUTE, out_buf=b))      # small copy right behind the pass, same stream

    if n_steps > 0:
        issue_in_and_step(0)
    for s in range(n_steps):
        if s + 1 < n_steps:
            issue_in_and_step(s + 1)
        # the host needs step s's entry counts to size the upload
        ops.append(Op("host_wait_stats", s, S_COMPUTE, out_buf=s % 2, host_sync=True))
        ops.append(Op("d2h", s, S_OUT, out_buf=s % 2, waits=[("step", s)]))
    if n_steps > 0:
        ops.append(Op("host_wait_d2h", n_steps - 1, S_OUT, host_sync=True))
    return ops


def check_plan(ops, n_in_bufs=2, n_out_bufs=2):
    """Checks a plan without running it: every step has its four activities in order, and every pair of ops that
    touch the same buffer with at least one writer is ordered by stream order or by a chain of event waits.
    Raises AssertionError with the offending pair."""
    pos = {(o.kind, o.step): i for i, o in enumerate(ops)}
    # happens-before: earlier op on the same stream, or an explicit wait; closed transitively
    preds = [set() for _ in ops]
    last_on_stream = {}
    host_barrier = -1  # index of the last op the host waited for: everything issued later comes after it
    for i, o in enumerate(ops):
        if o.stream in last_on_stream:
            preds[i].add(last_on_stream[o.stream])
        for w in o.waits:
            assert w in pos and pos[w] < i, f"{o.kind}({o.step}) waits for {w}, which is not issued before it"
            preds[i].add(pos[w])
        if host_barrier >= 0:
            preds[i].add(host_barrier)
        if not o.kind.startswith("host_wait"):
            last_on_stream[o.stream] = i
        if o.host_sync:
            # waiting for an op means waiting for its stream up to that op
            host_barrier = i if not o.kind.startswith("host_wait") else (
                pos[("stats", o.step)] if o.kind == "host_wait_stats" else pos[("d2h", o.step)])
    before = [set() for _ in ops]
    for i in range(len(ops)):
        for p in preds[i]:
            before[i] |= before[p] | {p}
    writes = {"h2d": ("in",), "step": ("out",), "stats": (), "d2h": ()}
    reads = {"h2d": (), "step": ("in",), "stats": ("out",), "d2h": ("out",)}

    def touches(o):
        t = []
        for kind, acc in (("w", writes), ("r", reads)):
            for which in acc.get(o.kind, ()):
                buf = o.in_buf if which == "in" else o.out_buf
                t.append((which, buf, kind))
        return t

    real = [i for i, o in enumerate(ops) if not o.kind.startswith("host_wait")]
    for a in real:
        for b in real:
            if a >= b:
                continue
            for (wa, ba, ka) in touches(ops[a]):
                for (wb, bb, kb_) in touches(ops[b]):
                    if wa == wb and ba == bb and "w" in (ka, kb_):
                        assert a in before[b], (f"hazard on {wa} buffer {ba}: {ops[a].kind}({ops[a].step}) and "
                                                f"{ops[b].kind}({ops[b].step}) are not ordered")
    steps = sorted({o.step for o in ops})
    for s in steps:
        idx = [pos[(k, s)] for k in ("h2d", "step", "stats", "d2h")]
        assert idx == sorted(idx), f"step {s}: activities issued out of order"
        assert 0 <= ops[pos[("h2d", s)]].in_buf < n_in_bufs and 0 <= ops[pos[("step", s)]].out_buf < n_out_bufs
    return True


class HostDriver:
    """Runs a plan with torch streams: pinned host gradients in, packed messages out (pinned), statistics read on
    the host to size the message copy.  ``run`` returns the device-to-host bytes it moved; when ``monitor`` is
    given, every message copy's size and duration (CUDA events around it) are reported to it."""

    def __init__(self, ctx, wl, cap, device="cuda", monitor=None):
        import torch

        from . import binding as kb

        self.kb, self.torch, self.ctx, self.wl, self.cap, self.dev = kb, torch, ctx, wl, cap, device
        self.monitor = monitor
        W, N = wl.n_workers, wl.N
        self.bpe = 8 if wl.value_dtype == 0 else 6
        self.dev_in = [torch.empty((W, N), dtype=torch.float32, device=device) for _ in range(2)]
        self.out = [kb.Packed(ctx, device=device) for _ in range(2)]
        self.h_stats = [torch.empty_like(o.stats, device="cpu").pin_memory() for o in self.out]
        self.h_idx = [torch.empty((W, cap), dtype=torch.int32).pin_memory() for _ in range(2)]
        self.h_val = [torch.empty((W, cap), dtype=self.out[0].val.dtype).pin_memory() for _ in range(2)]
        self.streams = [torch.cuda.Stream(device=device) for _ in range(3)]

    def run(self, mode, host_grads, state, bw, n_steps, first_step=0):
        torch, kb = self.torch, self.kb
        ops = plan(n_steps, mode)
        done = {}    # (kind, step) -> event recorded behind the op
        moved = 0
        cur = torch.cuda.current_stream()
        for st in self.streams:
            st.wait_stream(cur)
        timing = []  # (bytes, start event, end event) of the message copies
        for o in ops:
            if o.kind.startswith("host_wait"):
                done[("stats" if o.kind == "host_wait_stats" else "d2h", o.step)].synchronize()
                continue
            stream = self.streams[o.stream]
            for w in o.waits:
                stream.wait_event(done[w])
            s = first_step + o.step
            with torch.cuda.stream(stream):
                if o.kind == "h2d":
                    self.dev_in[o.in_buf].copy_(host_grads[s % len(host_grads)], non_blocking=True)
                elif o.kind == "step":
                    kb.kimad_step(self.ctx, self.dev_in[o.in_buf], state, bw[s % len(bw)], self.wl.t_target,
                                  self.out[o.out_buf], stream)
                elif o.kind == "stats":
                    self.h_stats[o.out_buf].copy_(self.out[o.out_buf].stats, non_blocking=True)
                elif o.kind == "d2h":
                    stats = self.h_stats[o.out_buf].numpy().view(kb.STATS_DTYPE).reshape(-1)
                    n_bytes = self.h_stats[o.out_buf].numel()
                    e0 = torch.cuda.Event(enable_timing=self.monitor is not None)
                    e0.record(stream)
                    for w in range(self.wl.n_workers):
                        n = int(stats["n_selected"][w])
                        self.h_idx[o.out_buf][w, :n].copy_(self.out[o.out_buf].idx[w, :n], non_blocking=True)
                        self.h_val[o.out_buf][w, :n].copy_(self.out[o.out_buf].val[w, :n], non_blocking=True)
                        n_bytes += n * self.bpe
                    moved += n_bytes
                    if self.monitor is not None:
                        e1 = torch.cuda.Event(enable_timing=True)
                        e1.record(stream)
                        timing.append((n_bytes, e0, e1))
                ev = torch.cuda.Event()
                ev.record(stream)
                done[(o.kind, o.step)] = ev
            if o.host_sync:
                ev.synchronize()
        for st in self.streams:
            cur.wait_stream(st)
        if self.monitor is not None:
            torch.cuda.synchronize()
            for n_bytes, e0, e1 in timing:
                sec = e0.elapsed_time(e1) * 1e-3
                if sec > 0:
                    kb.kimad_monitor_observe(self.monitor, n_bytes, sec)
        return moved
