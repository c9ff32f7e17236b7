"""Pins of the oracle's multi-seed sweep  theta <- rnd(theta + sum_q c_q z(seed_q))  (CPU only).

Algorithm 1 sums the projected gradients of several seeds ("Recover gradient": sum_t g_t z_t) before the
update; the oracle applies that sum with one rounding.  What fixes it independently of itself:
  * with one term it is the single-seed sweep, bit for bit, in every storage type;
  * with double storage it equals the same terms applied one sweep at a time (linearity of the update);
  * brute force on a tiny tensor: Z, G and U G built as dense matrices from the raw normal stream;
  * the deferred schedule of a Q-query step (2Q+1 sweeps, restores fused with the next perturbation and
    one final multi-seed update) ends at the same weights as the 3Q-sweep schedule;
  * server-side aggregation: with no perturbation active, restore_update_multi is theta - lr sum_i g_i z_i.
"""
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


@pytest.mark.parametrize("dtype", [oracle.F32, oracle.F16, oracle.BF16, oracle.F64])
@pytest.mark.parametrize("bits", [32, 16])
def test_one_term_is_the_single_seed_sweep(dtype, bits):
    a_, b_ = _model(dtype), _model(dtype)
    oa = oracle.OracleZGR(a_, 0.5, 1e-3, bits=bits)
    ob = oracle.OracleZGR(b_, 0.5, 1e-3, bits=bits)
    oa.perturb(11, 1e-3)
    ob.sweep_multi([11], [1e-3])
    for ta, tb in zip(a_, b_):
        assert np.array_equal(ta.theta, tb.theta)
    assert ob.nets == {11: 1e-3}


def test_sum_of_terms_equals_the_terms_applied_one_by_one():
    seeds, coeffs = [3, 2**40 + 5, 17], [1e-3, -2.5e-3, 4e-4]
    a_, b_ = _model(oracle.F64), _model(oracle.F64)
    oa = oracle.OracleZGR(a_, 0.3, 1e-3, bits=16)
    ob = oracle.OracleZGR(b_, 0.3, 1e-3, bits=16)
    for l, t in enumerate(a_):
        for s, c in zip(seeds, coeffs):
            oracle.sweep_tensor(t, s, l, oa.bits, oa.a, oa.b, c)
    ob.sweep_multi(seeds, coeffs)
    np.testing.assert_allclose(_flat(b_), _flat(a_), rtol=0, atol=1e-17)
    assert _flat(b_).std() > 0


@pytest.mark.parametrize("bits", [32, 16])
def test_brute_force_dense_construction(bits):
    m, n, r = 8, 8, 2
    U = synth.subspace(m, r, 5)
    w = synth.weights_host(synth.TensorSpec("t", m, n, r), 5).ravel()
    t = oracle.OracleTensor(theta=oracle.encode(w, oracle.F64), rows=m, cols=n, dtype=oracle.F64, U=U)
    a, b = oracle.mix_scalars(0.4, m * n, r * n, oracle.SCALE_UNIT)
    seeds, coeffs = [21, 22, 23], [2e-3, -1e-3, 5e-4]
    expected = w.astype(np.float64).copy()
    for s, c in zip(seeds, coeffs):
        Z = oracle.normals(s, 0, 0, bits, 0, m * n).reshape(m, n)          # tag 0: isotropic part
        G = oracle.normals(s, 0, 1, bits, 0, r * n).reshape(r, n)          # tag 1: guided coefficients
        expected += c * (a * Z + b * (U.astype(np.float64) @ G)).ravel()   # Eq. (perturbation), per tensor
    oracle.sweep_multi_tensor(t, seeds, coeffs, 0, bits, a, b)
    np.testing.assert_allclose(oracle.decode(t.theta, t.dtype).ravel(), expected, rtol=0, atol=1e-16)


def test_deferred_schedule_matches_the_three_sweep_schedule():
    Q, eps, lr = 4, 1e-3, 1e-2
    seeds = [1000 + q for q in range(Q)]
    rng = np.random.default_rng(0)
    lp, lm = rng.uniform(1.5, 2.5, Q), rng.uniform(1.5, 2.5, Q)
    a_, b_ = _model(oracle.F64), _model(oracle.F64)
    oa = oracle.OracleZGR(a_, 0.5, eps, bits=16)
    ob = oracle.OracleZGR(b_, 0.5, eps, bits=16)
    for q in range(Q):                                           # 3Q sweeps
        oa.perturb(seeds[q], eps)
        oa.perturb(seeds[q], -2 * eps)
        oa.restore_update(seeds[q], lp[q], lm[q], lr / Q)
    sweeps = 0
    ob.sweep_multi([seeds[0]], [eps]); sweeps += 1               # 2Q + 1 sweeps
    ob.sweep_multi([seeds[0]], [-2 * eps]); sweeps += 1
    for q in range(1, Q):
        ob.sweep_multi([seeds[q - 1], seeds[q]], [eps, eps]); sweeps += 1    # restore q-1, perturb q
        assert seeds[q - 1] not in ob.nets
        ob.sweep_multi([seeds[q]], [-2 * eps]); sweeps += 1
    assert ob.nets == {seeds[-1]: pytest.approx(-eps)}
    ob.restore_update_multi(seeds, lp, lm, lr / Q); sweeps += 1
    assert sweeps == 2 * Q + 1 and ob.nets == {}
    np.testing.assert_allclose(_flat(b_), _flat(a_), rtol=0, atol=1e-15)


def test_server_side_aggregation_without_active_perturbation():
    eps, lr = 1e-3, 5e-3
    seeds = [7, 8, 9]
    lp, lm = [2.0, 1.7, 2.2], [1.9, 1.8, 2.0]
    ts = _model(oracle.F64)
    o = oracle.OracleZGR(ts, 0.5, eps, bits=32)
    theta0 = _flat(ts)
    zs = [np.concatenate([oracle.z_tensor(t, s, l, o.bits, o.a, o.b).ravel() for l, t in enumerate(ts)]) for s in seeds]
    coeffs = o.restore_update_multi(seeds, lp, lm, lr)
    g = [(p - m) / (2 * eps) for p, m in zip(lp, lm)]
    assert coeffs == pytest.approx([-lr * gi for gi in g])
    np.testing.assert_allclose(_flat(ts), theta0 - lr * sum(gi * zi for gi, zi in zip(g, zs)), rtol=0, atol=1e-13)


def test_sampled_elements_agree_with_the_whole_tensor():
    ts = _model(oracle.BF16, shapes=((40, 32),), ranks=(4,))
    t = ts[0]
    a, b = oracle.mix_scalars(0.5, 40 * 32, 4 * 32, oracle.SCALE_UNIT)
    idx = np.array([0, 5, 33, 700, 1279], dtype=np.int64)
    before = oracle.decode(t.theta, t.dtype).ravel()[idx]
    got = oracle.sweep_multi_elements(t, before, [4, 6], [1e-3, 2e-3], 0, 16, a, b, idx)
    oracle.sweep_multi_tensor(t, [4, 6], [1e-3, 2e-3], 0, 16, a, b)
    assert np.array_equal(got, oracle.decode(t.theta, t.dtype).ravel()[idx])
