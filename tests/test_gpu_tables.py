"""GPU parity on inputs that stress the sweep's tables: a window of cells wider than the cell table (table entries
then stand for several cells), sparse gradients whose thresholds fall among exact zeros, and the byte codes the
sweep leaves for the counting sweep (layers with and without a histogram, both worker groups)."""
import numpy as np
import pytest
import torch

from paper_2312_08053_b200 import binding as kb
from tests._harness import Runner

pytestmark = pytest.mark.gpu


def _meta(r):
    n_reg = sum(1 for n in r.ls if n > 4096)
    return kb.kimad_debug_get_band_meta(r.ctx, n_reg)


@pytest.mark.parametrize("schedule", [0, 1])
def test_window_wider_than_the_cell_table(schedule):
    """Two populations 83 octaves apart, thresholds in both: the window between the lowest and the highest band
    has about 10,000 cells, more than the table's 4096 entries.  The sweep must run with its histograms (tables with
    several cells per entry) and everything must match the oracle bit for bit; layers whose error bound comes out
    too loose (the fine bins are shared by bands in both populations) may still be handed to the exact path afterwards."""
    rng = np.random.default_rng(7)
    sizes = [300000, 5000, 120000]
    grid = [0.01, 0.05, 0.2, 0.45, 0.7, 0.9, 1.0]  # 0.45 .. 0.9 fall into the small population
    W, N = 2, sum(sizes)
    x = rng.standard_normal((W, N)).astype(np.float32)
    small = rng.random((W, N)) < 0.6
    x[small] *= np.float32(1e-25)
    r = Runner(sizes, W, grid, 1000, 0, schedule=schedule)
    grads = torch.from_numpy(x).cuda()
    state = torch.zeros_like(grads)
    res = r.compare_step(grads, state, [0.05 * 8 * N, 0.3 * 8 * N], 1.0)
    assert res["same_k"]
    m = _meta(r)
    assert np.all(m[:, :, 2] == 0), "a layer was swept without its histogram"
    assert np.all(m[:, :, 1] <= 4096) and np.all(m[:, [0, 2], 1] > 1500)  # table entries in use: several cells per entry
    why = kb.kimad_debug_exact_path_layers(r.ctx, detail=True)
    assert why[1] == 0 and why[2] == 0 and why[3] == 0  # none forced, none without tables, no threshold outside its band
    # with the state of that step the kept entries difference to exactly zero: a third population at key 0 (the
    # window then starts at cell 0; layers whose widened bands no longer fit are handed to the exact path)
    res = r.compare_step(grads, state, [0.6 * 8 * N, 0.02 * 8 * N], 1.0)
    assert res["same_k"]


@pytest.mark.parametrize("value_dtype", [0, 1])
def test_sparse_gradients_thresholds_among_zeros(value_dtype):
    """90 % exact zeros (of both signs): candidates beyond the non-zero count have their threshold at key 0, where
    only the index order decides; the state of the step before makes some differences non-zero again."""
    rng = np.random.default_rng(21)
    sizes = [200000, 70000, 4097, 900]
    grid = [0.02, 0.08, 0.15, 0.5, 1.0]
    W, N = 2, sum(sizes)
    r = Runner(sizes, W, grid, 1000, value_dtype, schedule=1)
    state = torch.zeros((W, N), dtype=torch.float32, device="cuda")
    for step in range(3):
        x = rng.standard_normal((W, N)).astype(np.float32)
        x[rng.random((W, N)) < 0.9] = 0.0
        x[rng.random((W, N)) < 0.05] *= -0.0  # some negative zeros
        grads = torch.from_numpy(x).cuda()
        bpe = 8 if value_dtype == 0 else 6
        res = r.compare_step(grads, state, [0.3 * bpe * N, 0.12 * bpe * N], 1.0)
        assert res["same_k"]


def test_codes_of_layers_without_a_histogram():
    """curve_mode 1 sweeps every layer without a histogram (codes = upper bits of the key) and resolves through the
    exact path; mixed with tiny layers and a layer of one repeated magnitude, on two worker groups."""
    rng = np.random.default_rng(5)
    sizes = [150000, 12, 40000, 3000, 65536]
    grid = [0.001, 0.01, 0.1, 0.5, 1.0]
    W, N = 3, sum(sizes)
    x = rng.standard_normal((W, N)).astype(np.float32)
    x[:, -65536:] = np.sign(x[:, -65536:]) * np.float32(0.75)
    r = Runner(sizes, W, grid, 1000, 0, curve_mode=1, schedule=1)
    grads = torch.from_numpy(x).cuda()
    state = torch.from_numpy((rng.standard_normal((W, N)) * 0.01).astype(np.float32)).cuda()
    for budget in ([0.05 * 8 * N] * 3, [0.4 * 8 * N, 0.01 * 8 * N, 0.9 * 8 * N]):
        r.compare_step(grads, state, budget, 1.0)


def _row_sparse(rng, W, rows, cols, zero_frac, tail):
    """[W][rows * cols + tail]: a matrix whose untouched rows are exactly zero (an embedding gradient), then a dense tail."""
    x = rng.standard_normal((W, rows * cols + tail)).astype(np.float32)
    m = x[:, :rows * cols].reshape(W, rows, cols)
    m[rng.random((W, rows)) < zero_frac] = 0.0
    return x


@pytest.mark.parametrize("zero_frac,schedule", [(0.5, 0), (0.9, 1), (0.995, 1)])
def test_row_sparse_layer(zero_frac, schedule):
    """A 1.2 M-element layer with whole rows of exact zeros: candidates below the number of non-zeros have ordinary
    thresholds, the others have threshold 0 and keep zeros in index order.  Nothing of it may need the exact path:
    zeros are counted apart, loose candidates are refined from the code bytes."""
    rng = np.random.default_rng(int(zero_frac * 1000))
    rows, cols, tail = 600, 2048, 70000
    sizes = [rows * cols, tail]
    grid = [0.001, 0.004, 0.02, 0.05, 0.1, 0.2, 0.4, 0.6, 0.9, 1.0]
    W, N = 2, sum(sizes)
    r = Runner(sizes, W, grid, 1000, 0, schedule=schedule)
    state = torch.zeros((W, N), dtype=torch.float32, device="cuda")
    for step, frac in enumerate([0.02, 0.3, 0.7]):  # the last budget reaches candidates whose threshold is 0
        grads = torch.from_numpy(_row_sparse(rng, W, rows, cols, zero_frac, tail)).cuda()
        res = r.compare_step(grads, state, [frac * 8 * N, 0.5 * frac * 8 * N], 1.0)
        assert res["same_k"]
    why = kb.kimad_debug_exact_path_layers(r.ctx, detail=True)
    assert why[0] == 0, f"exact path taken: {why[:6]}"


def test_loose_candidates_are_refined():
    """Few, very wide bands (two populations 40 octaves apart under a coarse grid) leave bins whose error bound is too
    loose; those candidates are refined, and the refined curve, thresholds and selection equal the oracle's."""
    rng = np.random.default_rng(77)
    sizes = [900000, 50000]
    grid = [0.02, 0.3, 0.55, 0.8, 1.0]
    W, N = 2, sum(sizes)
    x = rng.standard_normal((W, N)).astype(np.float32)
    x[rng.random((W, N)) < 0.5] *= np.float32(1e-12)
    r = Runner(sizes, W, grid, 1000, 0, schedule=1)
    grads = torch.from_numpy(x).cuda()
    state = torch.zeros_like(grads)
    for budget in ([0.1 * 8 * N] * 2, [0.6 * 8 * N, 0.35 * 8 * N]):
        res = r.compare_step(grads, state, budget, 1.0)
        assert res["same_k"]
    why = kb.kimad_debug_exact_path_layers(r.ctx, detail=True)
    assert why[1] == 0 and why[2] == 0


@pytest.mark.parametrize("schedule", [0, 1])
def test_steps_issued_back_to_back(schedule):
    """Seven steps issued without a host synchronisation in between -- sparse, quantised and dense gradients in turn,
    so that the lists of the refinement and of the second select round fill and empty from step to step -- leave
    the same messages and states as the same steps run one by one, each of which is compared with the oracle."""
    rng = np.random.default_rng(11)
    cols, sizes = 1024, [400 * 1024, 3000, 150000, 768]
    grid = [0.001, 0.005, 0.02, 0.05, 0.1, 0.2, 0.4, 0.7, 1.0]
    W, N, S = 4, sum(sizes), 7
    grads = []
    for kind in [1, 0, 2, 1, 3, 0, 1]:
        x = rng.standard_normal((W, N)).astype(np.float32)
        if kind == 1:
            m = x[:, :sizes[0]].reshape(W, -1, cols)
            m[rng.random((W, m.shape[1])) < 0.9] = 0
        elif kind == 2:
            x = np.round(x * 3) / 3
        elif kind == 3:
            x[rng.random(x.shape) < 0.5] *= np.float32(1e-15)
        grads.append(torch.from_numpy(x).cuda())
    bws = [rng.uniform(0.005, 0.9, W) * 8 * N for _ in range(S)]
    one = Runner(sizes, W, grid, 1000, 0, schedule=schedule)
    state = torch.zeros((W, N), dtype=torch.float32, device="cuda")
    ref = []
    for s in range(S):
        one.compare_step(grads[s], state, bws[s], 1.0, check_inject=False)
        ref.append((one.out.idx.clone(), one.out.val.clone(), one.out.offs.clone(), state.clone()))
    run = Runner(sizes, W, grid, 1000, 0, schedule=schedule)
    state2 = torch.zeros((W, N), dtype=torch.float32, device="cuda")
    got = []
    for s in range(S):
        kb.kimad_step(run.ctx, grads[s], state2, bws[s], 1.0, run.out)
        got.append((run.out.idx.clone(), run.out.val.clone(), run.out.offs.clone(), state2.clone()))
    torch.cuda.synchronize()
    for s in range(S):
        offs = ref[s][2].cpu().numpy()
        assert torch.equal(ref[s][2], got[s][2]) and torch.equal(ref[s][3], got[s][3]), f"step {s}"
        for w in range(W):
            n = int(offs[w, len(sizes)])
            assert torch.equal(ref[s][0][w, :n], got[s][0][w, :n]) and torch.equal(ref[s][1][w, :n], got[s][1][w, :n]), f"step {s}"
