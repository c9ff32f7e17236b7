"""Pins of the oracle's adaptive mixing ratio (zgro_adapt_alpha): the rule is this build's candidate for the
adaptive choice announced in Sec. 1 -- balance the energies of the isotropic and the guided part of
Eq. (perturbation) -- so it is pinned by that balance itself, recomputed from the perturbation after the change,
and by a case worked by hand."""
import os

import numpy as np
import pytest

import oracle
from paper_2601_12917_b200 import synth

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def _numbers(name):
    vals = {}
    for line in open(os.path.join(GOLDEN, name)):
        line = line.split("#")[0].split()
        if len(line) == 2:
            vals[line[0]] = float(line[1])
    return vals


def test_hand_worked_two_tensor_case():
    v = _numbers("adapt_alpha_two_tensors.txt")
    d, K = int(v["d"]), int(v["K"])
    a0, b0 = oracle.mix_scalars(v["alpha_old"], d, K, oracle.SCALE_UNIT)
    stats = np.array([[v["iso_0"], v["guided_0"], 0.0], [v["iso_1"], v["guided_1"], 0.0]])
    assert oracle.adapt_alpha(stats, a0, b0, d, K, v["alpha_old"], 0.0, 1.0, 1.0) == pytest.approx(v["alpha_star"], rel=1e-14)
    assert oracle.adapt_alpha(stats, a0, b0, d, K, v["alpha_old"], 0.0, 1.0, 0.5) == pytest.approx(v["alpha_half_damped"], rel=1e-14)
    assert oracle.adapt_alpha(stats, a0, b0, d, K, v["alpha_old"], 0.05, 0.58, 1.0) == pytest.approx(v["alpha_clamped_at_0p58"], rel=1e-14)
    # the energies at alpha*: both equal the hand-worked 48
    a1, b1 = oracle.mix_scalars(v["alpha_star"], d, K, oracle.SCALE_UNIT)
    assert (a1 / a0) ** 2 * (v["iso_0"] + v["iso_1"]) == pytest.approx(v["balanced_energy"], rel=1e-13)
    assert (b1 / b0) ** 2 * (v["guided_0"] + v["guided_1"]) == pytest.approx(v["balanced_energy"], rel=1e-13)
    # the same in the paper's normalisation (a, b smaller by sqrt(d); the norms scale with them)
    a0p, b0p = oracle.mix_scalars(v["alpha_old"], d, K, oracle.SCALE_PAPER)
    assert oracle.adapt_alpha(stats / d, a0p, b0p, d, K, v["alpha_old"], 0.0, 1.0, 1.0) == pytest.approx(v["alpha_star"], rel=1e-13)


def _model(alpha, scale_mode, coeff_scale):
    """Two guided tensors and a vector; the second tensor's coefficients arrive compressed with a scale that
    is not that of a unit Gaussian, which is what moves the balance away from alpha = 1/2."""
    shapes, ranks = [(48, 64), (1, 40), (32, 96)], [4, 0, 8]
    tensors = []
    for l, ((m, n), r) in enumerate(zip(shapes, ranks)):
        U = synth.subspace(m, r, 40 + l) if r else None
        t = oracle.OracleTensor(theta=np.zeros(m * n, dtype=np.float32), rows=m, cols=n, dtype=oracle.F32, U=U)
        if l == 2:
            q, sc = synth.dtc_payload(r, n, seed=3)
            t.q, t.scale = q, (sc * coeff_scale).astype(np.float32)
        tensors.append(t)
    d = sum(m * n for m, n in shapes)
    K = sum(r * n for (m, n), r in zip(shapes, ranks))
    a, b = oracle.mix_scalars(alpha, d, K, scale_mode)
    return tensors, d, K, a, b


def _stats(tensors, a, b, seed=9):
    return np.array([oracle.stats_tensor(t, seed, l, 32, a, b) for l, t in enumerate(tensors)])


@pytest.mark.parametrize("scale_mode", [oracle.SCALE_PAPER, oracle.SCALE_UNIT])
@pytest.mark.parametrize("alpha0,coeff_scale", [(0.5, 1.0), (0.2, 3.0), (0.9, 0.25)])
def test_energies_are_balanced_after_the_change(alpha0, coeff_scale, scale_mode):
    tensors, d, K, a0, b0 = _model(alpha0, scale_mode, coeff_scale)
    st0 = _stats(tensors, a0, b0)
    alpha1 = oracle.adapt_alpha(st0, a0, b0, d, K, alpha0, 0.0, 1.0, 1.0)
    assert 0.0 < alpha1 < 1.0
    a1, b1 = oracle.mix_scalars(alpha1, d, K, scale_mode)
    st1 = _stats(tensors, a1, b1)                      # the perturbation itself, recomputed under the new ratio
    assert st1[:, 0].sum() == pytest.approx(st1[:, 1].sum(), rel=1e-12)
    # a fixed point: asking again changes nothing
    assert oracle.adapt_alpha(st1, a1, b1, d, K, alpha1, 0.0, 1.0, 1.0) == pytest.approx(alpha1, rel=1e-12)
    if coeff_scale > 1.0:
        assert alpha1 > 0.5        # a stronger guided part gets the smaller weight 1 - alpha
    if coeff_scale < 1.0:
        assert alpha1 < 0.5


def test_absent_parts_leave_alpha_alone():
    tensors, d, K, a0, b0 = _model(1.0, oracle.SCALE_UNIT, 1.0)          # alpha = 1: b = 0
    st = _stats(tensors, a0, b0)
    assert b0 == 0.0 and oracle.adapt_alpha(st, a0, b0, d, K, 1.0, 0.05, 0.95, 1.0) == 1.0
    tensors, d, K, a0, b0 = _model(0.0, oracle.SCALE_UNIT, 1.0)          # alpha = 0: a = 0
    st = _stats(tensors, a0, b0)
    assert a0 == 0.0 and oracle.adapt_alpha(st, a0, b0, d, K, 0.0, 0.05, 0.95, 1.0) == 0.0
    st = np.zeros((3, 3))
    assert oracle.adapt_alpha(st, 0.7, 0.7, 100, 0, 0.4, 0.05, 0.95, 1.0) == 0.4    # no guided coefficients at all
