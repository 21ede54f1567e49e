"""Seeded synthetic workloads: layer lists, ratio grids, gradient and bandwidth generators.

This module only *produces inputs*.  It holds none of the compression method's
arithmetic and is the one module that both the CUDA path's callers (tests, bench,
smoke) and the CPU oracle's callers draw their inputs from.

The five workloads follow the benchmark configurations: tensor shapes of the named
architectures (no weights, no data), per-layer gradient scales log-uniform in
[1e-4, 1e-1], and gradient value distributions per configuration.  They stand in
for the paper's ResNet18/CIFAR10 gradients and bandwidth traces (Section 4.2),
which need a dataset and a training run.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np


# ----------------------------------------------------------------------------- layer lists
def _mlp_layers():
    return [784 * 128, 128, 128 * 10, 10]


def _resnet18_layers(num_classes=1000):
    out = [64 * 3 * 7 * 7, 64, 64]
    cin = 64
    for stage, w in enumerate([64, 128, 256, 512]):
        for b in range(2):
            out += [w * cin * 9, w, w, w * w * 9, w, w]
            if b == 0 and stage > 0:
                out += [w * cin, w, w]
            cin = w
    out += [512 * num_classes, num_classes]
    return out


def _resnet50_layers(num_classes=1000):
    out = [64 * 3 * 7 * 7, 64, 64]
    cin = 64
    for w, nb in zip([64, 128, 256, 512], [3, 4, 6, 3]):
        for b in range(nb):
            out += [w * cin, w, w, w * w * 9, w, w, 4 * w * w, 4 * w, 4 * w]
            if b == 0:
                out += [4 * w * cin, 4 * w, 4 * w]
            cin = 4 * w
    out += [2048 * num_classes, num_classes]
    return out


def _gpt2_small_layers(d=768, vocab=50257, n_ctx=1024, blocks=12):
    out = [vocab * d, n_ctx * d]
    for _ in range(blocks):
        out += [d, d, d * 3 * d, 3 * d, d * d, d, d, d, d * 4 * d, 4 * d, 4 * d * d, d]
    out += [d, d]
    return out


def _llama_1b_layers(d=2048, ffn=5632, vocab=32000, blocks=22, kv=256):
    out = [vocab * d]
    for _ in range(blocks):
        out += [d, d * d, kv * d, kv * d, d * d, d, ffn * d, ffn * d, ffn * d]
    out += [d, vocab * d]
    return out


GRID_7 = [0.01, 0.02, 0.05, 0.10, 0.20, 0.50, 1.00]


def block_layers(layer_sizes, block_elems: int):
    """Block granularity (the paper's Section 5 names it as the next step after per-layer compression): every
    tensor is cut into consecutive blocks of ``block_elems`` elements (the last one shorter) and each block is
    handed to the compression pass as a segment of its own.  Returns the list of segment sizes; the flat
    gradient vector is unchanged."""
    out = []
    for n in layer_sizes:
        n = int(n)
        out.extend([block_elems] * (n // block_elems))
        if n % block_elems:
            out.append(n % block_elems)
    return out


def _log_grid(lo_exp, n=16):
    g = [10.0 ** (lo_exp + (-lo_exp) * j / (n - 1)) for j in range(n)]
    g[-1] = 1.0
    return g


def paper_grid_50():
    """The ratio grid of Section 4.3: {0.01 + 0.02 k} within [0.01, 1] (50 values, largest 0.99)."""
    return [0.01 + 0.02 * k for k in range(50)]


@dataclass
class Workload:
    cfg: int                 # 1..5
    name: str
    layer_sizes: list
    n_workers: int
    ratio_grid: list
    value_dtype: int         # 0 = f32 packed values, 1 = bf16
    dist: str                # "normal" | "mix" | "student3"
    n_steps: int
    D: int = 1000
    t_target: float = 0.05
    divisor: int = 1
    scales: np.ndarray = field(default=None, repr=False)

    @property
    def N(self):
        return int(sum(self.layer_sizes))

    @property
    def L(self):
        return len(self.layer_sizes)


def workload(cfg: int, divisor: int = 1, n_workers: int | None = None) -> Workload:
    """Configuration ``cfg`` (1..5).  ``divisor`` > 1 shrinks every tensor (ceil(n / divisor),
    at least 1 element) for cases the CPU oracle must finish in seconds; the layer count,
    the size ratios between layers and the ragged, non-16-byte-aligned offsets remain."""
    table = {
        1: ("mlp-101k", _mlp_layers(), 1, GRID_7, 0, "normal", 1, 1.0),
        2: ("resnet18-shape", _resnet18_layers(), 4, GRID_7, 0, "mix", 100, 0.05),
        3: ("resnet50-shape", _resnet50_layers(), 8, _log_grid(-3.0), 0, "mix", 200, 0.05),
        4: ("gpt2-small-shape", _gpt2_small_layers(), 4, _log_grid(-3.0), 0, "student3", 100, 0.05),
        5: ("llama-1.1b-shape", _llama_1b_layers(), 2, _log_grid(-4.0), 1, "student3", 50, 1.0),
    }
    name, layers, W, grid, vd, dist, steps, t = table[cfg]
    if divisor > 1:
        layers = [max(1, -(-n // divisor)) for n in layers]
        name = f"{name}/div{divisor}"
    rng = np.random.default_rng(cfg - 1)
    scales = np.exp(rng.uniform(math.log(1e-4), math.log(1e-1), size=len(layers)))
    return Workload(cfg, name, list(layers), n_workers or W, list(grid), vd, dist, steps, 1000, t,
                    max(1, divisor), scales.astype(np.float64))


# ----------------------------------------------------------------------------- gradients
EMBED_COLS = {4: 768, 5: 2048}  # row length of layer 0 (the token embedding) of the two language-model shapes


def gradients(wl: Workload, step: int, device="cpu", workers=None, stride: int | None = None, zero_rows: float = 0.0):
    """float32 tensor [W][stride] of fresh gradients for ``step`` (seeded per (cfg, step, worker)).
    Padding beyond N (when stride > N) is zero.  ``zero_rows`` > 0 (workloads 4 and 5, undivided): that fraction of the
    rows of the token embedding's gradient, drawn per worker and step, is exactly zero -- the rows of the tokens
    a batch does not contain."""
    import torch

    W = wl.n_workers
    workers = list(range(W)) if workers is None else list(workers)
    N = wl.N
    stride = stride or N
    dev = torch.device(device)
    out = torch.zeros((len(workers), stride), dtype=torch.float32, device=dev)
    sizes = torch.tensor(wl.layer_sizes, dtype=torch.int64, device=dev)
    sc = torch.tensor(wl.scales, dtype=torch.float32, device=dev)
    scale_vec = torch.repeat_interleave(sc, sizes)
    for row, w in enumerate(workers):
        gen = torch.Generator(device=dev)
        gen.manual_seed(1_000_000 * wl.cfg + step * W + w)
        z = torch.randn(N, generator=gen, device=dev, dtype=torch.float32)
        if wl.dist == "normal":
            x = z
        elif wl.dist == "mix":
            pick = torch.rand(N, generator=gen, device=dev) < 0.05
            u = torch.rand(N, generator=gen, device=dev) - 0.5
            lap = -10.0 * torch.sign(u) * torch.log1p(-2.0 * u.abs()).clamp_(min=-80.0)
            x = torch.where(pick, lap, z)
            del pick, u, lap
        elif wl.dist == "student3":
            chi = torch.zeros(N, device=dev, dtype=torch.float32)
            for _ in range(3):
                q = torch.randn(N, generator=gen, device=dev, dtype=torch.float32)
                chi.addcmul_(q, q)
                del q
            x = z / torch.sqrt(chi / 3.0).clamp_(min=1e-12)
            del chi
        else:
            raise ValueError(wl.dist)
        out[row, :N] = x * scale_vec
        del x, z
        if zero_rows > 0.0:
            cols = EMBED_COLS[wl.cfg]
            emb = out[row, :wl.layer_sizes[0]].view(-1, cols)
            emb[torch.rand(emb.shape[0], generator=gen, device=dev) < zero_rows] = 0.0
    return out


# ----------------------------------------------------------------------------- bandwidth
def bandwidth_trace(wl: Workload, n_steps: int | None = None) -> np.ndarray:
    """float64 [steps][W] monitored bandwidth in bytes/s (the boundary input B_m^k); pair it with
    ``wl.t_target``.  Shapes: cfg 1 fixed budget (10 % of dense bytes); cfg 2 random 1-10 Gbit/s
    levels held 20 steps; cfg 3 the sinusoid eta*sin^2(theta*step)+delta of Section 4.2 scaled to
    0.5-5 Gbit/s; cfg 4 bursts of 25 Gbit/s over a 1 Gbit/s floor; cfg 5 a budget sweep over
    0.1 %-10 % of dense bytes."""
    steps = n_steps or wl.n_steps
    W = wl.n_workers
    rng = np.random.default_rng(100 + wl.cfg)
    gbit = 1e9 / 8.0 / wl.divisor  # shrunk tensors get a proportionally shrunk link
    dense = 4.0 * wl.N
    out = np.zeros((steps, W), dtype=np.float64)
    if wl.cfg == 1:
        out[:] = float((4 * wl.N) // 10)
    elif wl.cfg == 2:
        level = 1.0
        for s in range(steps):
            if s % 20 == 0:
                level = rng.uniform(1.0, 10.0)
            out[s] = np.clip(level * rng.uniform(0.9, 1.1, size=W), 1.0, 10.0) * gbit
    elif wl.cfg == 3:
        for s in range(steps):
            base = 4.5 * math.sin(math.pi / 200.0 * s) ** 2 + 0.5
            out[s] = base * rng.uniform(0.95, 1.05, size=W) * gbit
    elif wl.cfg == 4:
        left = 0
        for s in range(steps):
            if left == 0 and rng.uniform() < 0.1:
                left = int(rng.geometric(1.0 / 3.0))
            out[s] = (25.0 if left > 0 else 1.0) * gbit
            left = max(0, left - 1)
    elif wl.cfg == 5:
        for s in range(steps):
            frac = 10.0 ** (-3.0 + 2.0 * (s % 50) / 49.0)
            out[s] = frac * dense
    else:
        raise ValueError(wl.cfg)
    return out
