"""Pins of the oracle's step: Eq. (ZOO), Eq. (grad), the update line of Algorithm 1, DTC (CPU only).

  * On a quadratic loss the central difference is exact, so (L+ - L-)/(2 eps) must equal the
    analytic directional derivative grad L . z for any eps; with a cubic term the gap is O(eps^2).
  * lr = 0 must give back theta (exactly up to double rounding with fp64 storage; within 2 ulp of
    the storage type otherwise, since three roundings cannot cancel bit for bit).
  * The update must move theta by -lr g z.
  * The worked numbers of the smallest configuration: (L+, L-) = (2.31, 2.29), eps = 1e-3,
    lr = 1e-4 give g = 10 and lr g = eps, so the fused restore+update coefficient vanishes.
  * DTC: x = lambda (x_q - delta), reconstruction error at most lambda/2.
"""
import math

import numpy as np
import pytest

import oracle
from paper_2601_12917_b200 import synth


def _model(dtype, shapes=((24, 16), (1, 12), (16, 24)), ranks=(4, 0, 2), seed=0):
    tensors = []
    for l, ((m, n), r) in enumerate(zip(shapes, ranks)):
        U = synth.subspace(m, r, seed + l) if r else None
        w = synth.weights_host(synth.TensorSpec(f"t{l}", m, n, r), seed + l).ravel()
        tensors.append(oracle.OracleTensor(theta=oracle.encode(w, dtype), rows=m, cols=n, dtype=dtype, U=U))
    return tensors


def _flat(tensors):
    return np.concatenate([oracle.decode(t.theta, t.dtype).ravel() for t in tensors])


def _flat_z(o, seed):
    return np.concatenate([oracle.z_tensor(t, seed, l, o.bits, o.a, o.b).ravel() for l, t in enumerate(o.tensors)])


@pytest.mark.parametrize("eps", [1e-1, 1e-3, 1e-5])
def test_two_point_estimate_is_exact_on_a_quadratic(eps):
    tensors = _model(oracle.F64)
    o = oracle.OracleZGR(tensors, alpha=0.5, eps=eps, scale_mode=oracle.SCALE_UNIT)
    theta0 = _flat(tensors)
    rng = np.random.default_rng(1)
    D = rng.uniform(0.5, 2.0, theta0.size)
    bvec = rng.standard_normal(theta0.size)
    loss = lambda th: 0.5 * np.sum(D * th * th) - np.sum(bvec * th)
    seed = 7
    z = _flat_z(o, seed)
    o.perturb(seed, +eps)
    lp = loss(_flat(tensors))
    np.testing.assert_allclose(_flat(tensors), theta0 + eps * z, atol=1e-15)
    o.perturb(seed, -2 * eps)
    lm = loss(_flat(tensors))
    np.testing.assert_allclose(_flat(tensors), theta0 - eps * z, atol=1e-15)
    g = oracle.projected_grad(lp, lm, eps)
    analytic = float(np.dot(D * theta0 - bvec, z))
    assert g == pytest.approx(analytic, rel=1e-7, abs=1e-7 / eps * 1e-3)
    # the update: theta <- theta0 - lr g z
    lr = 0.05
    c = o.restore_update(seed, lp, lm, lr)
    assert c == pytest.approx(eps - lr * g, rel=1e-12)
    np.testing.assert_allclose(_flat(tensors), theta0 - lr * g * z, atol=1e-13)
    assert o.active_seed is None and o.net == 0.0


def test_two_point_error_vanishes_quadratically_with_a_cubic_term():
    tensors0 = _model(oracle.F64)
    theta0 = _flat(tensors0)
    rng = np.random.default_rng(2)
    D = rng.uniform(0.5, 2.0, theta0.size)
    T = rng.standard_normal(theta0.size)
    loss = lambda th: 0.5 * np.sum(D * th * th) + np.sum(T * th**3)
    errs = []
    for eps in (1e-1, 1e-2):
        tensors = _model(oracle.F64)
        o = oracle.OracleZGR(tensors, alpha=0.5, eps=eps)
        z = _flat_z(o, 3)
        o.perturb(3, eps)
        lp = loss(_flat(tensors))
        o.perturb(3, -2 * eps)
        lm = loss(_flat(tensors))
        analytic = float(np.dot(D * theta0 + 3 * T * theta0**2, z))
        errs.append(abs(oracle.projected_grad(lp, lm, eps) - analytic))
        # the exact gap is eps^2 * sum T z^3
        assert errs[-1] == pytest.approx(abs(eps**2 * np.sum(T * z**3)), rel=1e-3)
    assert errs[1] == pytest.approx(errs[0] / 100, rel=1e-2)


def test_restore_is_exact_at_lr_zero_with_double_storage():
    tensors = _model(oracle.F64)
    theta0 = _flat(tensors)
    o = oracle.OracleZGR(tensors, alpha=0.5, eps=1e-3)
    o.perturb(5, 1e-3)
    assert np.abs(_flat(tensors) - theta0).max() > 1e-4
    o.perturb(5, -2e-3)
    c = o.restore_update(5, 2.0, 1.0, 0.0)
    assert c == pytest.approx(1e-3, rel=1e-12)
    assert np.abs(_flat(tensors) - theta0).max() <= 1e-15 * np.abs(theta0).max()


@pytest.mark.parametrize("dtype,mant", [(oracle.F32, 24), (oracle.F16, 11), (oracle.BF16, 8)])
def test_restore_at_lr_zero_within_two_ulp_in_real_storage(dtype, mant):
    tensors = _model(dtype)
    theta0 = _flat(tensors)
    o = oracle.OracleZGR(tensors, alpha=0.5, eps=1e-3)
    o.perturb(5, 1e-3)
    o.perturb(5, -2e-3)
    o.restore_update(5, 2.0, 1.0, 0.0)
    th = _flat(tensors)
    scale = np.maximum(np.abs(theta0), 1e-3 * 6)      # largest magnitude met on the way
    ulp = 2.0 ** (np.floor(np.log2(scale)) - (mant - 1))
    assert np.all(np.abs(th - theta0) <= 2 * ulp)
    assert np.mean(th == theta0) > 0.5


def test_worked_numbers_of_the_smallest_configuration():
    wl = synth.workload("tiny")
    lp, lm = wl.losses(0, 0)
    g = oracle.projected_grad(lp, lm, wl.eps)
    assert g == pytest.approx(10.0, rel=1e-12)
    assert wl.lr * g == pytest.approx(wl.eps, rel=1e-12)
    tensors = _model(oracle.F32)
    o = oracle.OracleZGR(tensors, alpha=wl.alpha, eps=wl.eps)
    o.perturb(0, wl.eps)
    o.perturb(0, -2 * wl.eps)
    before = _flat(tensors).copy()
    c = o.restore_update(0, lp, lm, wl.lr)
    assert abs(c) < 1e-15          # eps - lr g cancels: the third sweep leaves theta where it is
    np.testing.assert_array_equal(_flat(tensors), before)


def test_state_machine_rejects_mismatched_seeds():
    o = oracle.OracleZGR(_model(oracle.F32), alpha=0.5, eps=1e-3)
    with pytest.raises(RuntimeError):
        o.restore_update(1, 2.0, 1.0, 0.1)
    o.perturb(1, 1e-3)
    with pytest.raises(RuntimeError):
        o.perturb(2, 1e-3)
    with pytest.raises(RuntimeError):
        o.restore_update(2, 2.0, 1.0, 0.1)


@pytest.mark.parametrize("dtype", [oracle.F32, oracle.F16, oracle.BF16])
def test_sweep_elements_matches_full_sweep(dtype):
    tensors = _model(dtype)
    a, b, c = 0.7, 3.0, -2e-3
    for l, t in enumerate(tensors):
        idx = synth.sample_indices(t.rows * t.cols, 50, l)
        th_in = oracle.decode(t.theta, dtype).ravel()[idx]
        exp = oracle.sweep_elements(t, th_in, 9, l, 32, a, b, c, idx)
        oracle.sweep_tensor(t, 9, l, 32, a, b, c)
        np.testing.assert_array_equal(oracle.decode(t.theta, dtype).ravel()[idx], exp)


# ----------------------------------------------------------------------------------------- DTC
@pytest.mark.parametrize("symmetric", [True, False])
def test_dtc_roundtrip_error_bound(symmetric):
    rng = np.random.default_rng(8)
    G = rng.standard_normal((6, 500)) + (0.0 if symmetric else 0.7)
    q, sc, ze = oracle.dtc_quantise(G, bits=8, symmetric=symmetric)
    assert q.dtype == np.int8
    back = oracle.dtc_dequantise(q, sc, ze)
    # x = lambda (x_q - delta) by hand
    np.testing.assert_allclose(back, sc[:, None].astype(np.float64) * (q.astype(np.float64) - ze[:, None].astype(np.float64)), rtol=0, atol=0)
    assert np.all(np.abs(back - G) <= 0.5 * sc[:, None] * (1 + 1e-6))
    if symmetric:
        assert np.all(ze == 0)
        np.testing.assert_allclose(sc, np.abs(G).max(axis=1) / 127, rtol=1e-6)
        assert np.abs(q).max() == 127
    else:
        np.testing.assert_allclose(sc, (G.max(axis=1) - G.min(axis=1)) / 255, rtol=1e-6)
        assert q.min() == -128 and q.max() == 127


def test_dtc_coefficients_replace_seeded_ones():
    m, n, r = 32, 40, 4
    U = synth.subspace(m, r, 1)
    G = oracle.coeffs(3, 0, 32, r, n)
    q, sc, ze = oracle.dtc_quantise(G, 8, True)
    t_seed = oracle.OracleTensor(np.zeros(m * n), m, n, oracle.F64, U=U)
    t_dtc = oracle.OracleTensor(np.zeros(m * n), m, n, oracle.F64, U=U, q=q, scale=sc)
    a, b = 0.0, 1.0
    Zs = oracle.z_tensor(t_seed, 3, 0, 32, a, b)
    Zd = oracle.z_tensor(t_dtc, 3, 0, 32, a, b)
    np.testing.assert_allclose(Zd, U.astype(np.float64) @ oracle.dtc_dequantise(q, sc), atol=1e-14)
    # compressed coefficients perturb the guided part by at most the quantisation step
    bound = np.abs(U.astype(np.float64)) @ np.tile(0.5 * sc[:, None].astype(np.float64), (1, n))
    assert np.all(np.abs(Zd - Zs) <= bound * (1 + 1e-6))
    # zero-point form
    G2 = G + 0.3
    q2, sc2, ze2 = oracle.dtc_quantise(G2, 8, False)
    t2 = oracle.OracleTensor(np.zeros(m * n), m, n, oracle.F64, U=U, q=q2, scale=sc2, zero=ze2)
    np.testing.assert_allclose(oracle.z_tensor(t2, 3, 0, 32, a, b), U.astype(np.float64) @ oracle.dtc_dequantise(q2, sc2, ze2), atol=1e-14)


# ----------------------------------------------------------------------------- INT4 payload (Sec. 3.4)
def test_int4_quantiser_error_bound_and_code_range():
    rng = np.random.default_rng(5)
    G = rng.standard_normal((6, 101))
    q, sc, ze = oracle.dtc_quantise_int4(G)
    assert q.min() >= 0 and q.max() <= 15                       # x_quant in [0, 2^b - 1]
    for k in range(6):
        lam = float(sc[k])
        assert lam == pytest.approx((G[k].max() - G[k].min()) / 15.0, rel=1e-6)    # lambda = (max - min)/(2^b - 1)
    back = oracle.dtc_dequantise(q, sc, ze)
    assert np.all(np.abs(back - G) <= 0.5 * sc[:, None].astype(np.float64) * (1 + 1e-6) + 1e-12)   # |x - x'| <= lambda/2
    assert {0, 15} <= set(np.unique(q))                         # both ends of the range are used


def test_int4_packing_layout():
    codes = np.array([[1, 2, 3, 4, 5], [15, 0, 9, 8, 7]], dtype=np.int8)
    packed = oracle.dtc_pack4(codes)
    # column 2j in the low nibble, column 2j+1 in the high nibble; the odd tail is padded with 0
    assert packed.tolist() == [[0x21, 0x43, 0x05], [0x0F, 0x89, 0x07]]
    assert np.array_equal(oracle.dtc_unpack4(packed, 5), codes)
    rng = np.random.default_rng(6)
    c = rng.integers(0, 16, size=(7, 64)).astype(np.int8)
    assert np.array_equal(oracle.dtc_unpack4(oracle.dtc_pack4(c), 64), c)
