"""Fixtures under tests/golden/: the hand-worked scalars of the smallest configuration, and the digests that
freeze the oracle's outputs (written by tests/golden/make_digests.py from the oracle alone)."""
import importlib.util
import math
import os

import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def _numbers():
    vals = {}
    for line in open(os.path.join(GOLDEN, "tiny_worked_numbers.txt")):
        line = line.split("#")[0].split()
        if len(line) == 2:
            vals[line[0]] = float(line[1])
    return vals


def test_worked_scalars_of_the_smallest_configuration():
    v = _numbers()
    g = oracle.projected_grad(v["loss_plus"], v["loss_minus"], v["eps"])
    assert g == pytest.approx(v["g"], rel=1e-12)
    assert v["lr"] * g == pytest.approx(v["lr_times_g"], rel=1e-12)
    assert abs(v["eps"] - v["lr"] * g) < 1e-15                      # vanishes up to the rounding of the decimal inputs
    # the fused restore + update coefficient: with -eps still applied it cancels, on the server side (nothing
    # applied) it is the bare step -lr g
    assert abs(oracle.update_coefficient(-v["eps"], v["loss_plus"], v["loss_minus"], v["eps"], v["lr"])) < 1e-15
    assert oracle.update_coefficient(0.0, v["loss_plus"], v["loss_minus"], v["eps"], v["lr"]) == pytest.approx(-v["lr_times_g"], rel=1e-12)
    d, K = int(v["d"]), int(v["K"])
    assert d == 4 * 256 * 256 + 4 * 256 and K == 4 * 4 * 256
    a, b = oracle.mix_scalars(0.5, d, K, oracle.SCALE_PAPER)
    assert a == pytest.approx(v["a_paper"], rel=1e-7) and b == pytest.approx(v["b_paper"], rel=1e-7)
    assert a == pytest.approx(math.sqrt(0.5 / d), rel=1e-14) and b == pytest.approx(math.sqrt(0.5 / K), rel=1e-14)
    a, b = oracle.mix_scalars(0.5, d, K, oracle.SCALE_UNIT)
    assert a == pytest.approx(v["a_unit"], rel=1e-7) and b == pytest.approx(v["b_unit"], rel=1e-7)


def test_oracle_outputs_match_the_stored_digests():
    spec = importlib.util.spec_from_file_location("make_digests", os.path.join(GOLDEN, "make_digests.py"))
    mod = importlib.util.module_from_spec(spec)
    spec.loader.exec_module(mod)
    stored = {}
    for line in open(os.path.join(GOLDEN, "oracle_digests.txt")):
        if line.startswith("#") or not line.strip():
            continue
        h, what = line.rstrip("\n").split("  ", 1)
        stored[what] = h
    now = dict(mod.digests())
    assert set(now) == set(stored)
    for what, h in now.items():
        assert stored[what] == h, f"oracle output changed: {what}"
