"""CPU-only checks of the C-ABI library: it loads without a GPU, exports every symbol the header
declares, and its host-side planner (candidate table, budget cells, argument validation) agrees with
the oracle.  No kernel is launched here."""
import ctypes
import os
import re

import numpy as np
import pytest

from oracle import kimad_oracle as ko
from paper_2312_08053_b200 import binding as kb
from paper_2312_08053_b200 import build as kbuild
from paper_2312_08053_b200 import workloads

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    kbuild.build()


def _declared_symbols():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        if fn.endswith(".h"):
            text = open(os.path.join(ROOT, "include", fn)).read()
            text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
            names |= set(re.findall(r"\b(kimad_[a-z0-9_]+)\s*\(", text))
    return names


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(kbuild.LIB_PATH)
    names = _declared_symbols()
    assert {"kimad_create", "kimad_step", "kimad_set_workspace", "kimad_get_k", "kimad_destroy"} <= names
    for n in sorted(names):
        assert hasattr(lib, n), n


def test_binding_names_match_header():
    for n in _declared_symbols():
        assert hasattr(kb, n), f"binding lacks {n}"


@pytest.mark.parametrize("cfg", [1, 2, 3, 4, 5])
def test_k_table_and_budget_cells_match_oracle(cfg):
    wl = workloads.workload(cfg)
    ctx = kb.kimad_create(wl.layer_sizes, wl.n_workers, wl.ratio_grid, D=wl.D, value_dtype=wl.value_dtype)
    kt = kb.kimad_get_k_table(ctx)
    assert np.array_equal(kt, ko.k_table(wl.layer_sizes, wl.ratio_grid))
    bw = workloads.bandwidth_trace(wl, 5)
    for b in list(bw[:, 0]) + [0.0, 1e18, 7.5]:
        st, c, cells = kb.kimad_plan_budget(ctx, float(b), wl.t_target)
        assert c == ko.budget_bytes(float(b), wl.t_target)
        ost, ocells = ko.units(kt, wl.value_dtype, c, wl.D)
        assert st == ost
        if st == 0:
            assert np.array_equal(cells, ocells)
    assert kb.kimad_workspace_bytes(ctx) > wl.N * wl.n_workers  # at least one code byte per element
    kb.kimad_destroy(ctx)


def test_create_rejects_bad_arguments():
    good = dict(layer_sizes=[10, 20], n_workers=1, ratio_grid=[0.1, 1.0])
    kb.kimad_destroy(kb.kimad_create(**good))
    bad = [dict(good, ratio_grid=[0.5, 0.1]), dict(good, ratio_grid=[0.0, 0.1]), dict(good, ratio_grid=[0.5, 1.5]),
           dict(good, layer_sizes=[0, 3]), dict(good, n_workers=0), dict(good, layer_sizes=[2 ** 32]),
           dict(good, D=1), dict(good, D=70000), dict(good, value_dtype=2), dict(good, worker_stride=5),
           dict(good, ratio_grid=list(np.linspace(0.001, 1, 200)))]
    for kw in bad:
        with pytest.raises(kb.KimadError) as e:
            kb.kimad_create(**kw)
        assert e.value.code == kb.KIMAD_ERR_INVALID_ARG


def test_step_without_workspace_is_refused():
    ctx = kb.kimad_create([8], 1, [1.0])
    out = kb.kimad_packed(1, 1, 1, 1, 1, 1)
    bw = (ctypes.c_double * 1)(1.0)
    rc = kb.load().kimad_step(ctx.handle, 1, 1, bw, 1.0, ctypes.byref(out), None)
    assert rc == kb.KIMAD_ERR_WORKSPACE
    assert "workspace" in kb.kimad_strerror(rc)
    assert kb.load().kimad_set_workspace(ctx.handle, None, 0) == kb.KIMAD_ERR_WORKSPACE


def test_schedule_modes_are_validated():
    ctx = kb.kimad_create([8, 9000], 3, [0.5, 1.0])
    for mode in (0, 1, 2):
        kb.kimad_debug_set_schedule(ctx, mode)
    for mode in (-1, 3):
        with pytest.raises(kb.KimadError) as e:
            kb.kimad_debug_set_schedule(ctx, mode)
        assert e.value.code == kb.KIMAD_ERR_INVALID_ARG
    kb.kimad_destroy(ctx)
