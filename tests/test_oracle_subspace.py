"""Pins of the oracle's subspace construction (Algorithm 1, "Collect gradients to build basis V_r"; Sec. 3.2):
zgro_householder_qr against a hand-worked case, a library QR, and the properties that define the result."""
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def _numbers(name):
    vals = {}
    for line in open(os.path.join(GOLDEN, name)):
        line = line.split("#")[0].split()
        if len(line) == 2:
            vals[line[0]] = float(line[1])
    return vals


def test_hand_worked_three_by_two():
    v = _numbers("householder_3x2.txt")
    A = np.array([[v["a11"], v["a12"]], [v["a21"], v["a22"]], [v["a31"], v["a32"]]])
    Q, R = oracle.householder_qr(A, with_r=True)
    np.testing.assert_allclose(Q[:, 0], [v["q11"], v["q21"], v["q31"]], atol=1e-15)
    r22 = np.sqrt(v["r22_squared"])
    np.testing.assert_allclose(Q[:, 1] * r22, [v["q12_times_r22"], v["q22_times_r22"], v["q32_times_r22"]], atol=1e-14)
    np.testing.assert_allclose(R, [[v["r11"], v["r12"]], [0.0, r22]], atol=1e-14)


@pytest.mark.parametrize("rows,r", [(7, 1), (64, 4), (300, 16), (1000, 32), (513, 64), (64, 64)])
def test_against_library_qr_and_defining_properties(rows, r):
    rng = np.random.default_rng([rows, r])
    A = rng.standard_normal((rows, r)) * np.exp(rng.uniform(-3, 3, size=r))[None, :]     # columns of very different sizes
    Q, R = oracle.householder_qr(A, with_r=True)
    # defining properties: orthonormal columns, upper triangular R with positive diagonal, A = Q R
    np.testing.assert_allclose(Q.T @ Q, np.eye(r), atol=5e-14)
    assert np.all(np.diag(R) > 0) and np.all(np.tril(R, -1) == 0)
    np.testing.assert_allclose(Q @ R, A, atol=1e-12 * np.abs(A).max())
    # the library's factorisation, brought to the same sign convention
    q, rr = np.linalg.qr(A)
    sgn = np.sign(np.diag(rr))
    np.testing.assert_allclose(Q, q * sgn[None, :], atol=1e-11)
    # same span: the orthogonal projector of the normal equations
    P = A @ np.linalg.solve(A.T @ A, A.T)
    np.testing.assert_allclose(Q @ Q.T, P, atol=1e-8)


def test_leading_columns_do_not_depend_on_later_ones():
    # column k of Q spans, together with the earlier columns, the first k + 1 gradients: adding gradients leaves it alone
    rng = np.random.default_rng(5)
    A = rng.standard_normal((200, 12))
    Q12 = oracle.householder_qr(A)
    Q5 = oracle.householder_qr(A[:, :5].copy())
    np.testing.assert_allclose(Q12[:, :5], Q5, atol=1e-13)


def test_orthonormal_input_is_returned_unchanged_up_to_sign():
    rng = np.random.default_rng(6)
    q, rr = np.linalg.qr(rng.standard_normal((128, 8)))
    q = q * np.sign(np.diag(rr))[None, :]
    Q, R = oracle.householder_qr(q, with_r=True)
    np.testing.assert_allclose(R, np.eye(8), atol=1e-14)
    np.testing.assert_allclose(Q, q, atol=1e-14)


def test_zero_column_gives_no_nan():
    A = np.zeros((16, 3))
    A[:, 0] = 1.0
    A[:, 2] = np.arange(16)
    Q = oracle.householder_qr(A)
    assert np.all(np.isfinite(Q))
    np.testing.assert_allclose(Q[:, 0], np.full(16, 0.25), atol=1e-15)
