"""Pins of the oracle's hybrid perturbation, Eq. (perturbation) (CPU only).

    z_h = sqrt(alpha/n) z + sqrt((1-alpha)/m) V z_g ,   V orthonormal,  z ~ N(0, I),  z_g ~ N(0, I)

Checked against what the equation and the mathematics fix, not against the oracle itself:
dense brute-force construction with an explicit V, the alpha = 1 and alpha = 0 special cases,
E|z_h|^2, the share of energy inside span(V), and the covariance (alpha/n) I + ((1-alpha)/m) V V^T.
"""
import math

import numpy as np
import pytest

import oracle
from paper_2601_12917_b200 import synth


def _tiny_model(shapes, ranks, seed=0):
    tensors = []
    for l, ((m, n), r) in enumerate(zip(shapes, ranks)):
        U = synth.subspace(m, r, seed * 100 + l) if r > 0 else None
        tensors.append(oracle.OracleTensor(theta=np.zeros(m * n), rows=m, cols=n, dtype=oracle.F64, U=U))
    return tensors


def _dense_V(tensors):
    """Explicit flat basis V = blockdiag_l(U_l kron I_cols) for row-major flattening: d x K."""
    d = sum(t.rows * t.cols for t in tensors)
    K = sum(t.rank * t.cols for t in tensors)
    V = np.zeros((d, K))
    ro = co = 0
    for t in tensors:
        if t.rank > 0:
            blk = np.kron(t.U.astype(np.float64), np.eye(t.cols))
            V[ro:ro + t.rows * t.cols, co:co + t.rank * t.cols] = blk
            co += t.rank * t.cols
        ro += t.rows * t.cols
    return V


@pytest.mark.parametrize("bits", [32, 16])
@pytest.mark.parametrize("scale_mode", [oracle.SCALE_PAPER, oracle.SCALE_UNIT])
def test_brute_force_dense_equation(bits, scale_mode):
    shapes, ranks = [(8, 8), (4, 12), (1, 9), (6, 5)], [2, 1, 0, 3]
    tensors = _tiny_model(shapes, ranks)
    V = _dense_V(tensors)
    d, K = V.shape
    np.testing.assert_allclose(V.T @ V, np.eye(K), atol=1e-6)       # V is orthonormal because each U_l is
    alpha, seed = 0.3, 42
    a, b = oracle.mix_scalars(alpha, d, K, scale_mode)
    s = math.sqrt(d) if scale_mode == oracle.SCALE_UNIT else 1.0
    assert a == pytest.approx(s * math.sqrt(alpha / d), rel=1e-15)
    assert b == pytest.approx(s * math.sqrt((1 - alpha) / K), rel=1e-15)
    # the two Gaussian vectors, taken from the generator streams (tag 0: z, tag 1: z_g)
    z_flat = np.concatenate([oracle.normals(seed, l, 0, bits, 0, t.rows * t.cols) for l, t in enumerate(tensors)])
    zg_flat = np.concatenate([oracle.normals(seed, l, 1, bits, 0, t.rank * t.cols) for l, t in enumerate(tensors) if t.rank > 0])
    zh = s * (math.sqrt(alpha / d) * z_flat + math.sqrt((1 - alpha) / K) * (V @ zg_flat))
    got = np.concatenate([oracle.z_tensor(t, seed, l, bits, a, b).ravel() for l, t in enumerate(tensors)])
    np.testing.assert_allclose(got, zh, rtol=0, atol=1e-13)
    # random access agrees with the full tensor
    for l, t in enumerate(tensors):
        idx = np.arange(t.rows * t.cols)[::3]
        np.testing.assert_array_equal(oracle.z_elements(t, seed, l, bits, a, b, idx), oracle.z_tensor(t, seed, l, bits, a, b).ravel()[idx])


def test_alpha_one_reduces_to_plain_zoo_perturbation():
    # Algorithm 1, non-guided round: z_h <- z.  With unit scaling alpha = 1 must give z itself.
    tensors = _tiny_model([(16, 8), (1, 7)], [4, 0])
    d = 16 * 8 + 7
    a, b = oracle.mix_scalars(1.0, d, 4 * 8, oracle.SCALE_UNIT)
    assert (a, b) == (1.0, 0.0)
    for l, t in enumerate(tensors):
        z = oracle.z_tensor(t, 5, l, 32, a, b).ravel()
        np.testing.assert_array_equal(z, oracle.normals(5, l, 0, 32, 0, t.rows * t.cols))
    a, b = oracle.mix_scalars(1.0, d, 4 * 8, oracle.SCALE_PAPER)
    assert a == pytest.approx(1 / math.sqrt(d)) and b == 0.0


def test_alpha_zero_lies_in_span_of_U():
    tensors = _tiny_model([(64, 24), (1, 10), (48, 16)], [4, 0, 8], seed=3)
    d = sum(t.rows * t.cols for t in tensors)
    K = sum(t.rank * t.cols for t in tensors)
    a, b = oracle.mix_scalars(0.0, d, K, oracle.SCALE_UNIT)
    assert a == 0.0
    for l, t in enumerate(tensors):
        Z = oracle.z_tensor(t, 11, l, 32, a, b)
        if t.rank == 0:
            assert np.all(Z == 0)          # 1-D tensors carry only the isotropic part
            continue
        U = t.U.astype(np.float64)
        resid = Z - U @ (U.T @ Z)
        assert np.abs(resid).max() <= 1e-6 * np.abs(Z).max()
        assert np.abs(Z).max() > 0.1


def test_no_guided_tensors_gives_b_zero():
    a, b = oracle.mix_scalars(0.5, 100, 0, oracle.SCALE_UNIT)
    assert b == 0.0 and a == pytest.approx(math.sqrt(0.5))


@pytest.mark.parametrize("scale_mode", [oracle.SCALE_PAPER, oracle.SCALE_UNIT])
def test_monte_carlo_energy_and_covariance(scale_mode):
    shapes, ranks = [(6, 4), (1, 5), (5, 3)], [2, 0, 1]
    tensors = _tiny_model(shapes, ranks, seed=9)
    V = _dense_V(tensors)
    d, K = V.shape
    alpha = 0.5
    a, b = oracle.mix_scalars(alpha, d, K, scale_mode)
    n_seeds = 6000
    Z = np.stack([np.concatenate([oracle.z_tensor(t, s, l, 32, a, b).ravel() for l, t in enumerate(tensors)]) for s in range(n_seeds)])
    unit = d if scale_mode == oracle.SCALE_UNIT else 1.0
    # E|z_h|^2 = alpha + (1 - alpha) = 1 (times d with unit scaling)
    e = (Z**2).sum(axis=1)
    assert abs(e.mean() / unit - 1.0) < 5 * e.std() / unit / math.sqrt(n_seeds)
    # energy inside span(V): (1 - alpha) + alpha K/d
    inside = ((Z @ V) ** 2).sum(axis=1).mean() / unit
    assert abs(inside - ((1 - alpha) + alpha * K / d)) < 0.03
    # covariance (alpha/n) I + ((1-alpha)/m) V V^T
    cov = (Z.T @ Z) / n_seeds / unit
    exp = (alpha / d) * np.eye(d) + ((1 - alpha) / K) * (V @ V.T)
    assert np.abs(cov - exp).max() < 6 * exp.max() / math.sqrt(n_seeds) * 2


def test_parts_add_up_and_stats():
    tensors = _tiny_model([(32, 16)], [4])
    t = tensors[0]
    a, b = 0.7, 1.9
    z, iso, gd = oracle.z_tensor(t, 1, 0, 32, a, b, parts=True)
    np.testing.assert_allclose(z, iso + gd, atol=1e-15)
    np.testing.assert_allclose(iso, a * oracle.normals(1, 0, 0, 32, 0, 32 * 16).reshape(32, 16), atol=1e-15)
    G = oracle.coeffs(1, 0, 32, 4, 16)
    np.testing.assert_allclose(gd, b * (t.U.astype(np.float64) @ G), atol=1e-14)
    st = oracle.stats_tensor(t, 1, 0, 32, a, b)
    np.testing.assert_allclose(st, [(iso**2).sum(), (gd**2).sum(), (z**2).sum()], rtol=1e-12)


# ------------------------------------------------------------------------------------- a proportion of the coefficients compressed
@pytest.mark.parametrize("qrows", [0, 1, 5, 8])
def test_mixed_coefficient_source(qrows):
    """Sec. 3.4, adaptive proportion: only part of the guided payload arrives compressed.  Here the first qrows
    rows of G_l are dequantised codes, x = lambda (x_q - delta), the other rows are drawn from the seed.  Checked
    against a dense construction from the two pure sources, and against them at the two ends."""
    rows, cols, r, seed, tid, bits = 24, 40, 8, 77, 3, 32
    U = synth.subspace(rows, r, 5)
    q_full, sc_full = synth.dtc_payload(r, cols, seed=4)
    ze_full = (np.arange(r) % 3 - 1).astype(np.float32)
    a, b = 0.6, 1.7
    t = oracle.OracleTensor(theta=np.zeros(rows * cols, dtype=np.float32), rows=rows, cols=cols, dtype=oracle.F32, U=U,
                            q=q_full[:qrows], scale=sc_full[:qrows], zero=ze_full[:qrows])
    z, iso, gd = oracle.z_tensor(t, seed, tid, bits, a, b, parts=True)
    G_seed = oracle.coeffs(seed, tid, bits, r, cols)
    G_code = oracle.dtc_dequantise(q_full, sc_full, ze_full)
    G = np.vstack([G_code[:qrows], G_seed[qrows:]])
    np.testing.assert_allclose(gd, b * (U.astype(np.float64) @ G), atol=1e-13)
    np.testing.assert_allclose(oracle.coeffs(seed, tid, bits, r, cols, q_full[:qrows], sc_full[:qrows], ze_full[:qrows]), G, atol=0)
    pure_seed = oracle.OracleTensor(theta=t.theta, rows=rows, cols=cols, dtype=oracle.F32, U=U)
    pure_code = oracle.OracleTensor(theta=t.theta, rows=rows, cols=cols, dtype=oracle.F32, U=U, q=q_full, scale=sc_full, zero=ze_full)
    if qrows == 0:
        np.testing.assert_array_equal(z, oracle.z_tensor(pure_seed, seed, tid, bits, a, b))
    if qrows == r:
        np.testing.assert_array_equal(z, oracle.z_tensor(pure_code, seed, tid, bits, a, b))
    # the random-access form and the norms see the same mixture
    idx = np.arange(0, rows * cols, 7)
    np.testing.assert_allclose(oracle.z_elements(t, seed, tid, bits, a, b, idx), z.ravel()[idx], atol=1e-14)
    st = oracle.stats_tensor(t, seed, tid, bits, a, b)
    np.testing.assert_allclose(st, [np.sum(iso**2), np.sum(gd**2), np.sum(z**2)], rtol=1e-13)
