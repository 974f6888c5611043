"""CPU-only checks of the C-ABI library: it loads, exports what the header declares,
and its host-side logic (argument checks, workspace sizing, work split) is right.
No compute call is made here."""
import ctypes
import re
from pathlib import Path

import numpy as np
import pytest

from paper_2201_06227_b200 import binding as eg
from paper_2201_06227_b200 import workloads as wl

HEADER = Path(__file__).resolve().parent.parent / "include" / "egeria.h"


def declared_symbols():
    text = re.sub(r"/\*.*?\*/", "", HEADER.read_text(), flags=re.S)
    return sorted(set(re.findall(r"\b(egeria_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    L = eg.lib()
    names = declared_symbols()
    assert len(names) >= 12
    for name in names:
        assert hasattr(L, name), f"{name} is declared in egeria.h but not exported"
    assert sorted(eg.EXPORTS) == names


def test_header_is_plain_c(tmp_path):
    """The boundary is a C ABI: the header must compile as C99 on its own, and a C program that
    only uses the host-side calls must link against the library."""
    import shutil
    import subprocess
    if shutil.which("gcc") is None:
        pytest.skip("no gcc")
    src = tmp_path / "use_header.c"
    src.write_text(
        '#include "egeria.h"\n'
        '#include <stdio.h>\n'
        'int main(void) {\n'
        '    int64_t d[2] = {4096, 8192};\n'
        '    size_t n = egeria_workspace_bytes(2, d, 64, 10, EGERIA_FLAG_KEEP_GRAMS | EGERIA_FLAG_FRONTMOST);\n'
        '    printf("%zu %s\\n", n, egeria_status_string(EGERIA_ERR_TIMEOUT));\n'
        '    return n > 0 ? 0 : 1;\n'
        '}\n')
    exe = tmp_path / "use_header"
    lib_dir = Path(eg._LIB_PATH).parent
    subprocess.run(["gcc", "-std=c99", "-Wall", "-Werror", "-pedantic", "-I", str(HEADER.parent), str(src), "-o", str(exe),
                    "-L", str(lib_dir), "-legeria", f"-Wl,-rpath,{lib_dir}"], check=True)
    out = subprocess.run([str(exe)], check=True, capture_output=True, text=True).stdout.split(" ", 1)
    assert int(out[0]) == eg.egeria_workspace_bytes(2, [4096, 8192], 64, 10, eg.FLAG_KEEP_GRAMS | eg.FLAG_FRONTMOST)
    assert out[1].strip() == eg.status_string(eg.ERR_TIMEOUT)


def test_status_strings():
    for s in range(7):
        assert eg.status_string(s) not in ("", "unknown status")
    assert eg.status_string(99) == "unknown status"


def test_workspace_bytes_is_pure_and_monotone():
    d = [4096, 8192]
    base = eg.egeria_workspace_bytes(2, d, 64, 10)
    assert base > 0 and base % eg.WORKSPACE_ALIGN == 0
    assert eg.egeria_workspace_bytes(2, d, 64, 10) == base
    assert eg.egeria_workspace_bytes(2, d, 128, 10) > base
    assert eg.egeria_workspace_bytes(2, d, 256, 10) > eg.egeria_workspace_bytes(2, d, 128, 10)
    keep = eg.egeria_workspace_bytes(2, d, 64, 10, eg.FLAG_KEEP_GRAMS)
    assert keep >= base + 2 * 2 * 64 * 64 * 4
    stage = eg.egeria_workspace_bytes(2, d, 64, 10, eg.FLAG_HOST_STAGING)
    assert stage >= base + 2 * 64 * sum(d) * 2


@pytest.mark.parametrize("M,d,b,W", [(0, [8], 8, 5), (1, [0], 8, 5), (1, [8], 1, 5), (1, [8], 257, 5),
                                     (1, [8], 8, 0), (1, [8], 8, 100000), (1, [2 ** 31], 8, 5)])
def test_workspace_bytes_rejects_bad_arguments(M, d, b, W):
    assert eg.egeria_workspace_bytes(M, d, b, W) == 0


def _create(M, d, b_max, W, ws_ptr, ws_bytes, flags=0):
    h = ctypes.c_void_p()
    st = eg.lib().egeria_plasticity_create(ctypes.byref(h), M, eg._i64(d), b_max, W, None,
                                           ctypes.c_float(1e-3), ctypes.c_void_p(ws_ptr), ws_bytes, flags)
    return st, h


def test_create_error_paths_need_no_gpu():
    assert _create(0, [8], 8, 5, 0, 0)[0] == eg.ERR_INVALID_ARG
    assert _create(1, [8], 1, 5, 0, 0)[0] == eg.ERR_INVALID_ARG
    assert _create(1, [8], 300, 5, 0, 0)[0] == eg.ERR_UNSUPPORTED_SHAPE
    assert _create(1, [-4], 8, 5, 0, 0)[0] == eg.ERR_UNSUPPORTED_SHAPE
    assert _create(1, [8], 8, 5, 0, 0)[0] == eg.ERR_WORKSPACE             # NULL workspace
    assert _create(1, [8], 8, 5, 1024 + 8, 1 << 30)[0] == eg.ERR_WORKSPACE  # misaligned
    assert _create(1, [8], 8, 5, 4096, 16)[0] == eg.ERR_WORKSPACE          # too small
    L = eg.lib()
    assert L.egeria_plasticity_create(None, 1, eg._i64([8]), 8, 5, None, ctypes.c_float(0), None, 0, 0) \
        == eg.ERR_INVALID_ARG
    assert L.egeria_plasticity_destroy(None) == eg.ERR_INVALID_ARG
    assert L.egeria_device_status(None) == eg.ERR_INVALID_ARG
    assert L.egeria_plasticity_step(None, None, None, None, None) == eg.ERR_INVALID_ARG
    assert L.egeria_plasticity_window(None) == 0


def test_create_without_a_device_fails_loudly():
    """With a valid workspace pointer but no sm_100 device the call must fail, never fall back."""
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    n = eg.egeria_workspace_bytes(1, [64], 8, 5)
    st, h = _create(1, [64], 8, 5, 1 << 20, n)
    assert st in (eg.ERR_CUDA, eg.ERR_UNSUPPORTED_DEVICE)
    assert not h.value


# ----------------------------------------------------------------------------- the work split

def _check_plan(d, b, n_ctas):
    units = eg.egeria_debug_plan(d, b, n_ctas)
    M = len(d)
    sides = [2] if b <= 64 else [0, 1]
    nkb = [(x + 63) // 64 for x in d]
    # every (module, side) is covered exactly once, by contiguous ascending ranges
    for m in range(M):
        for s in sides:
            rows = units[(units[:, 0] == m) & (units[:, 1] == s)]
            assert len(rows) >= 1
            pos = 0
            for r in rows:
                assert r[2] == pos and r[3] >= 1
                pos += r[3]
            assert pos == nkb[m]
    assert len(units) == sum(len(units[(units[:, 0] == m)]) for m in range(M))
    # unit count bound used for workspace sizing
    assert len(units) <= len(sides) * M + 2 * n_ctas
    # balance among tensor-core-eligible work: per-CTA block counts differ by at most 1
    tc = units[np.isin(units[:, 0], [m for m in range(M) if d[m] % 8 == 0])]
    if len(tc):
        per = np.bincount(tc[:, 4], weights=tc[:, 3], minlength=n_ctas)
        busy = per[per > 0]
        assert busy.max() - busy.min() <= 1
        # small problems use fewer CTAs (at least 8 blocks each), never more than there are
        assert len(busy) == min(n_ctas, max(1, -(-int(per.sum()) // 8)))
    # CTAs are visited in order
    assert np.all(np.diff(tc[:, 4]) >= 0)
    return units


@pytest.mark.parametrize("name", wl.ORDER)
def test_plan_covers_named_workloads(name):
    w = wl.WORKLOADS[name]
    _check_plan(list(w.d), w.b, 148)


@pytest.mark.parametrize("d,b,n", [([8], 2, 148), ([64, 72, 4104], 17, 148), ([4096] * 5, 100, 7),
                                   ([1000, 24, 8], 256, 3), ([63, 65, 130], 129, 148), ([4096], 8, 1)])
def test_plan_odd_shapes(d, b, n):
    _check_plan(d, b, n)


@pytest.mark.parametrize("name", ["resnet50", "gpt2_medium", "resnet56"])
def test_weighted_plan_gives_shares_in_proportion(name):
    w = wl.WORKLOADS[name]
    d, n = list(w.d), 148
    rng = np.random.default_rng(7)
    weights = (1.0 + 0.08 * rng.standard_normal(n)).astype(np.float32)
    units = eg.egeria_debug_plan_weighted(d, w.b, n, weights)
    # still an exact cover, in order
    sides = [2] if w.b <= 64 else [0, 1]
    for m in range(len(d)):
        for s in sides:
            rows = units[(units[:, 0] == m) & (units[:, 1] == s)]
            pos = 0
            for r in rows:
                assert r[2] == pos and r[3] >= 1
                pos += r[3]
            assert pos == (d[m] + 63) // 64
    assert np.all(np.diff(units[:, 4]) >= 0)
    assert len(units) <= len(sides) * len(d) + 2 * n
    per = np.bincount(units[:, 4], weights=units[:, 3], minlength=n)
    want = per.sum() * weights.astype(np.float64) / weights.astype(np.float64).sum()
    assert np.max(np.abs(per - want)) <= 1.0 + 1e-6 * per.sum()
    # equal weights and no weights are the same split
    eq = eg.egeria_debug_plan_weighted(d, w.b, n, np.ones(n, dtype=np.float32))
    per_eq = np.bincount(eq[:, 4], weights=eq[:, 3], minlength=n)
    assert per_eq.max() - per_eq.min() <= 1
    assert np.array_equal(eg.egeria_debug_plan_weighted(d, w.b, n, None), eg.egeria_debug_plan(d, w.b, n))


def test_weighted_plan_ignores_bad_weights_and_small_problems():
    d, b, n = [802816, 401408], 64, 148
    base = eg.egeria_debug_plan(d, b, n)
    for bad in (np.zeros(n), np.full(n, np.nan), -np.ones(n), np.full(n, np.inf)):
        got = eg.egeria_debug_plan_weighted(d, b, n, bad.astype(np.float32))
        assert np.array_equal(got, base)
    # a problem that does not fill every CTA keeps the equal split
    small = eg.egeria_debug_plan([4096], 8, n)
    w = np.linspace(0.5, 1.5, n).astype(np.float32)
    assert np.array_equal(eg.egeria_debug_plan_weighted([4096], 8, n, w), small)


def test_plan_rejects_bad_arguments():
    out = np.zeros((4, 5), dtype=np.int32)
    n = ctypes.c_int()
    L = eg.lib()
    p = out.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))
    assert L.egeria_debug_plan(1, eg._i64([8]), 8, 0, p, 4, ctypes.byref(n)) == eg.ERR_INVALID_ARG
    assert L.egeria_debug_plan(1, eg._i64([8]), 400, 4, p, 4, ctypes.byref(n)) == eg.ERR_UNSUPPORTED_SHAPE
    assert L.egeria_debug_plan(1, eg._i64([8]), 8, 4, None, 4, ctypes.byref(n)) == eg.ERR_INVALID_ARG


def test_planned_help_goes_from_well_off_modules_to_needy_ones():
    """End-of-launch help (CtaHelp): CTAs whose module has more warps than rows to do lend some to
    the modules that have many rows per warp; balanced workloads plan none."""
    for name in ("bert_base", "gpt2_medium", "tiny"):
        w = wl.WORKLOADS[name]
        assert not (eg.egeria_debug_plan_help(list(w.d), w.b, 148)[:, 1] > 0).any(), name
    w = wl.WORKLOADS["resnet56"]
    d, n = list(w.d), 148
    units = eg.egeria_debug_plan(d, w.b, n)
    help_ = eg.egeria_debug_plan_help(d, w.b, n)
    blocks = np.zeros((n, len(d)))
    for m, _, _, nkb, c in units:
        blocks[c, m] += nkb
    have = (12.0 * blocks / blocks.sum(axis=1, keepdims=True)).sum(axis=0)      # warps credited to each module
    rows_per_warp = w.b / have
    donors = np.nonzero(help_[:, 1] > 0)[0]
    assert len(donors) > 20
    assert np.all(help_[donors, 1] <= 8) and np.all(help_[help_[:, 1] == 0, 0] == -1)
    avg = w.b * len(d) / have.sum()
    for c in donors:
        own = int(np.argmax(blocks[c]))
        assert rows_per_warp[own] < avg < rows_per_warp[help_[c, 0]]         # from the well-off to the needy
    got = np.bincount(help_[donors, 0], weights=help_[donors, 1], minlength=len(d))
    after = w.b / (have + got - np.bincount([int(np.argmax(blocks[c])) for c in donors],
                                            weights=help_[donors, 1], minlength=len(d)))
    assert after.max() < 0.6 * rows_per_warp.max()                             # the worst module is much better off
    assert after.max() / after.min() < 1.6


def test_first_tasks_of_the_finish_are_a_partition():
    """Who starts the end of a launch with which task (Plan::first_task): every task with a warp of
    its own is named exactly once, by a warp of a CTA that worked on the module (or lends it warps),
    the tasks are spread over the CTAs, the cursor's share is the rest, and the choice of protocol
    follows from it."""
    for name, only in (("tiny", -1), ("bert_base", -1), ("resnet50", -1), ("resnet56", -1), ("gpt2_medium", -1),
                       ("resnet50", 0), ("bert_base", 3), ("gpt2_medium", 0), ("resnet56", 26), ("resnet56", 0)):
        w = wl.WORKLOADS[name]
        d, n = list(w.d), 148
        first, tasks, validate = eg.egeria_debug_plan_tasks(d, w.b, n, only)
        help_ = eg.egeria_debug_plan_help(d, w.b, n) if only < 0 else np.full((n, 2), -1)
        worked = [set() for _ in range(n)]
        if only < 0:
            for m, _, _, _, c in eg.egeria_debug_plan(d, w.b, n):
                worked[c].add(int(m))
        else:                                        # the module alone over all CTAs
            for _, _, _, _, c in eg.egeria_debug_plan([d[only]], w.b, n):
                worked[c].add(only)
        seen = {}
        for c in range(n):
            for wp in range(12):
                ft = int(first[c, wp])
                if ft < 0:
                    continue
                m, t = ft >> 16, ft & 0xffff
                assert m in worked[c] or (help_[c, 1] > 0 and m == help_[c, 0]), (name, c, wp, m)
                assert (m, t) not in seen, (name, m, t)
                seen[(m, t)] = c
        active = [m for m in range(len(d)) if only < 0 or m == only]
        for m in range(len(d)):
            n_tasks, n_static = int(tasks[m, 0]), int(tasks[m, 1])
            mine = sorted(t for (mm, t) in seen if mm == m)
            if m not in active:
                assert mine == []
                continue
            assert mine == list(range(n_static)), (name, m)
            assert 0 < n_static <= n_tasks
            assert n_tasks % w.b == 0
            if n_tasks > w.b:                       # two levels: only a module alone, stacked modes
                assert len(active) == 1 and w.b <= 64
            ctas = {seen[(m, t)] for t in mine}
            assert len(ctas) >= min(n_static, len([c for c in range(n) if m in worked[c]])) * 0.9   # spread
        # partial rows announce themselves (no counters) at b <= 128 where every task has a warp of its
        # own and its partial rows fit one pass of the warp's 16 KB stage
        plan_units = eg.egeria_debug_plan(d, w.b, n) if only < 0 else eg.egeria_debug_plan([d[only]], w.b, n)
        pitch = 32 if w.b <= 32 else 64 if w.b <= 64 else 128 if w.b <= 128 else 256
        one_pass = True
        for m in active:
            mm = m if only < 0 else 0
            rows = sum(2 if side == 2 else 1 for (um, side, _, _, _) in plan_units if um == mm)
            if tasks[m, 0] > w.b:
                rows = min(rows, 2 * (16384 // (pitch * 4) // 2))
            one_pass = one_pass and rows * pitch * 4 <= 16384
        every_task_static = all(tasks[m, 0] == tasks[m, 1] for m in active)
        assert validate == (w.b <= 128 and one_pass and every_task_static), (name, only)
        assert validate == (name in ("tiny", "bert_base", "resnet50") or (name, only) == ("resnet56", 26)), (name, only)
        assert every_task_static == (name in ("tiny", "bert_base", "resnet50") or only >= 0), (name, only)


def test_two_level_tasks_only_for_a_module_alone_at_small_b():
    d = [64 * 148 * 40]
    for b, two in ((8, True), (32, True), (64, True), (128, False), (256, False)):
        first, tasks, validate = eg.egeria_debug_plan_tasks(d, b, 148)
        assert (tasks[0, 0] > b) == two, b
        if two:                                   # about 8 slots per chunk, and never more tasks than warps
            assert tasks[0, 0] == b * min(-(-148 // 8), (148 * 12) // b)
    first, tasks, validate = eg.egeria_debug_plan_tasks(d + d, 32, 148)   # two modules: one level
    assert tasks[0, 0] == 32 and tasks[1, 0] == 32
