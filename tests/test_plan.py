"""The sweep planner (host logic, no GPU): every element of every tensor is covered by exactly one work item,
whatever the shapes, ranks, storage types and alignment, for the single-seed and the multi-seed plan, with and
without the tcgen05 path.  Checked by brute-force counting on small random models and by interval arithmetic on
the full-size configurations."""
import ctypes

import numpy as np
import pytest

from paper_2601_12917_b200 import synth, zgr


class PlanItem(ctypes.Structure):
    _fields_ = [("path", ctypes.c_int32), ("kpad", ctypes.c_int32), ("tensor", ctypes.c_int32), ("ncols", ctypes.c_int32),
                ("row0_or_e0", ctypes.c_int64), ("nrows_or_count", ctypes.c_int64), ("col0", ctypes.c_int64)]


def plan(shapes, ranks, dtypes, bits=16, sm_count=148, tcgen05=1, multi=0, alpha=0.5, misalign=()):
    L = zgr.lib()
    L.zgr_debug_plan.restype = ctypes.c_int
    n = len(shapes)
    arr = (zgr.ZgrTensor * n)()
    for l, ((m, c), r, dt) in enumerate(zip(shapes, ranks, dtypes)):
        base = 0x100000 * (l + 1) + (2 if l in misalign and dt != zgr.F32 else (4 if l in misalign else 0))
        arr[l] = zgr.ZgrTensor(base, m, c, dt, r, 0x40000000 if r else None)     # addresses are never dereferenced
    cfg = zgr.ZgrConfig(alpha, 1e-3, zgr.SCALE_UNIT, bits)
    count = ctypes.c_int64()
    rc = L.zgr_debug_plan(arr, n, ctypes.byref(cfg), sm_count, tcgen05, multi, None, ctypes.c_int64(0), ctypes.byref(count))
    assert rc == zgr.OK
    items = (PlanItem * count.value)()
    rc = L.zgr_debug_plan(arr, n, ctypes.byref(cfg), sm_count, tcgen05, multi, items, ctypes.c_int64(count.value), ctypes.byref(count))
    assert rc == zgr.OK and count.value == len(items)
    return list(items)


def check_exact_cover(items, shapes):
    per_tensor = {}
    for it in items:
        per_tensor.setdefault(it.tensor, []).append(it)
    assert sorted(per_tensor) == list(range(len(shapes)))          # every tensor is served
    for l, (m, c) in enumerate(shapes):
        its = per_tensor[l]
        paths = {it.path for it in its}
        assert len(paths) == 1, f"tensor {l} is split over kernel families {paths}"
        if paths == {0}:                                           # flat chunks of elements
            iv = sorted((it.row0_or_e0, it.nrows_or_count) for it in its)
            pos = 0
            for e0, cnt in iv:
                assert e0 == pos and cnt > 0 and e0 % 8 == 0
                pos += cnt
            assert pos == m * c
        else:                                                      # strips of columns x ranges of rows
            strips = {}
            for it in its:
                strips.setdefault((it.col0, it.ncols), []).append((it.row0_or_e0, it.nrows_or_count))
            pos = 0
            for (c0, nc) in sorted(strips):
                assert c0 == pos and nc > 0
                pos += nc
                r = 0
                for r0, nr in sorted(strips[(c0, nc)]):
                    assert r0 == r and nr > 0
                    r += nr
                assert r == m
            assert pos == c


def brute_force_counts(items, shapes):
    counts = [np.zeros(m * c, dtype=np.int32) for m, c in shapes]
    for it in items:
        m, c = shapes[it.tensor]
        if it.path == 0:
            counts[it.tensor][it.row0_or_e0: it.row0_or_e0 + it.nrows_or_count] += 1
        else:
            view = counts[it.tensor].reshape(m, c)
            view[it.row0_or_e0: it.row0_or_e0 + it.nrows_or_count, it.col0: it.col0 + it.ncols] += 1
    return counts


@pytest.mark.parametrize("multi", [0, 1])
@pytest.mark.parametrize("tcgen05", [0, 1])
@pytest.mark.parametrize("trial", range(6))
def test_random_models_are_covered_exactly_once(trial, tcgen05, multi):
    rng = np.random.default_rng(100 + trial)
    n = int(rng.integers(3, 9))
    shapes, ranks, dtypes = [], [], []
    for _ in range(n):
        if rng.random() < 0.3:
            shapes.append((1, int(rng.integers(1, 5000)))); ranks.append(0)
        else:
            m = int(rng.integers(1, 700))
            c = int(rng.integers(1, 160)) * (8 if rng.random() < 0.7 else 1)
            shapes.append((m, c)); ranks.append(int(rng.choice([0, 1, 3, 4, 8, 12, 16, 20, 32, 40, 64])))
        dtypes.append(int(rng.choice([zgr.F32, zgr.F16, zgr.BF16])))
    misalign = {int(rng.integers(0, n))} if rng.random() < 0.5 else set()
    items = plan(shapes, ranks, dtypes, bits=int(rng.choice([16, 32])), sm_count=int(rng.choice([1, 4, 148])), tcgen05=tcgen05, multi=multi,
                 misalign=misalign)
    check_exact_cover(items, shapes)
    for cnt in brute_force_counts(items, shapes):
        assert cnt.min() == 1 and cnt.max() == 1
    if multi:
        assert all(it.path != 2 for it in items)                   # the legacy tensor-core kernel serves one seed per sweep only
    if not tcgen05:
        assert all(it.path != 4 for it in items)


@pytest.mark.parametrize("name", ["tiny", "roberta_large", "opt_1p3b", "llama_7b", "llama_13b"])
def test_full_size_configurations(name):
    wl = synth.workload(name)
    shapes = [(t.rows, t.cols) for t in wl.tensors]
    ranks = [t.rank for t in wl.tensors]
    dt = {"f32": zgr.F32, "f16": zgr.F16, "bf16": zgr.BF16}[wl.dtype]
    items = plan(shapes, ranks, [dt] * len(shapes))
    check_exact_cover(items, shapes)
    covered = sum(it.nrows_or_count if it.path == 0 else it.nrows_or_count * it.ncols for it in items)
    assert covered == wl.params
    expected_path = {"f32": 1, "f16": 4, "bf16": 4}[wl.dtype]
    assert {it.path for it in items if ranks[it.tensor] > 0} == {expected_path}
    assert {it.path for it in items if ranks[it.tensor] == 0} == {0}
    # enough items to balance 148 persistent CTAs: the tail of a fixed round-robin stays below 3 % (the tcgen05 kernel
    # assigns its items that way; the CUDA-core contraction kernel hands them out by a counter and needs less)
    guided = [it for it in items if it.path != 0]
    per_cta = np.zeros(148)
    for i, it in enumerate(guided):
        per_cta[i % 148] += it.nrows_or_count * it.ncols
    if name != "tiny":
        assert per_cta.max() / per_cta.mean() < 1.03


def test_alpha_one_plans_everything_as_isotropic_and_errors_are_reported():
    items = plan([(64, 256), (1, 100)], [8, 0], [zgr.BF16, zgr.BF16], alpha=1.0)
    assert {it.path for it in items} == {0}
    L = zgr.lib()
    cnt = ctypes.c_int64()
    cfg = zgr.ZgrConfig(0.5, 1e-3, zgr.SCALE_UNIT, 16)
    arr = (zgr.ZgrTensor * 1)(zgr.ZgrTensor(0x1000, 4, 4, zgr.F32, 0, None))
    assert L.zgr_debug_plan(arr, 1, ctypes.byref(cfg), 0, 1, 0, None, ctypes.c_int64(0), ctypes.byref(cnt)) == zgr.EINVAL   # sm_count
    assert L.zgr_debug_plan(arr, 1, ctypes.byref(cfg), 148, 1, 0, None, ctypes.c_int64(0), None) == zgr.EINVAL
    bad = (zgr.ZgrTensor * 1)(zgr.ZgrTensor(0x1000, 4, 4, 7, 0, None))
    assert L.zgr_debug_plan(bad, 1, ctypes.byref(cfg), 148, 1, 0, None, ctypes.c_int64(0), ctypes.byref(cnt)) == zgr.EINVAL
