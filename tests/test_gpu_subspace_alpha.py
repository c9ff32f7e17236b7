"""Subspace construction on the device (zgr_build_subspace) and the adaptive mixing ratio (zgr_adapt_alpha)
against the oracle (needs a B200).

Algorithm 1, "Collect gradients to build basis V_r" (Sec. 3.2): the device builds the orthonormal basis of a stack
of gradient directions by Cholesky QR applied twice; the oracle does it by Householder QR in double.  Both keep
the diagonal of R positive, which makes the basis unique, so the two are compared column by column, through
their projectors, and by running a ZGR step on the device-built basis.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2601_12917_b200 import synth, zgr

from helpers import Pair, to_double

pytestmark = pytest.mark.gpu


def _directions(rows, r, seed, cond=1e3):
    """Gradient-like directions: correlated columns of very different sizes (condition number about `cond`)."""
    rng = np.random.default_rng([23, seed, rows, r])
    base = rng.standard_normal((rows, r))
    mix = np.eye(r) + 0.5 * rng.standard_normal((r, r)) / np.sqrt(r)
    scales = np.exp(np.linspace(0.0, np.log(cond), r))[rng.permutation(r)]
    return np.ascontiguousarray((base @ mix) * scales[None, :], dtype=np.float32)


@pytest.mark.parametrize("src", ["host", "device", "in_place"])
@pytest.mark.parametrize("rows,cols,r,dtype", [(300, 392, 16, "bf16"), (4096, 256, 32, "bf16"), (1000, 264, 64, "f16"), (200, 256, 8, "f32"),
                                               (64, 128, 64, "bf16"), (33000, 64, 24, "bf16")])
def test_device_built_basis_matches_householder(rows, cols, r, dtype, src):
    p = Pair([(rows, cols), (1, 24)], [r, 0], dtype, bits=16, seed=2)
    A = _directions(rows, r, seed=rows + r)
    if src == "host":
        p.lib.build_subspace(0, torch.from_numpy(A).pin_memory())
    elif src == "device":
        p.lib.build_subspace(0, torch.from_numpy(A).cuda())
    else:
        p.U[0].copy_(torch.from_numpy(A))
        p.lib.build_subspace(0, None)
    torch.cuda.synchronize()
    U = p.U[0].cpu().numpy().astype(np.float64)
    Q = oracle.householder_qr(A.astype(np.float64))
    orth = np.abs(U.T @ U - np.eye(r)).max()
    col = np.abs(U - Q).max()
    # the projector, compared through its action on random vectors (rows x rows is too large to form for the big case)
    rng = np.random.default_rng(1)
    X = rng.standard_normal((rows, 8))
    proj = np.abs(U @ (U.T @ X) - Q @ (Q.T @ X)).max() / np.abs(X).max()
    print(f"build_subspace {rows}x{r} [{src}]: |U^T U - I|_max = {orth:.2e}, |U - Q|_max = {col:.2e}, projector difference {proj:.2e}")
    assert orth <= 1e-6
    assert proj <= 1e-5
    assert col <= 1e-5
    # a ZGR step with the device-built basis, every call against the oracle (which reads the same U back)
    reports = p.step(seed=4, lp=2.2, lm=1.9, lr=1e-4)
    assert all(rep["moved"] > 0.3 for call in reports[:2] for rep in call)


def test_dependent_directions_are_refused_and_leave_the_basis_alone():
    p = Pair([(256, 128)], [16], "bf16", bits=16)
    before = p.U[0].clone()
    A = _directions(256, 16, seed=1)
    A[:, 7] = 2.0 * A[:, 3] - A[:, 5]                  # an exact linear combination of earlier columns
    with pytest.raises(zgr.ZgrError) as e:
        p.lib.build_subspace(0, torch.from_numpy(A).cuda())
    assert e.value.code == zgr.EINVAL
    torch.cuda.synchronize()
    assert torch.equal(before, p.U[0])
    p.step(seed=5, lp=2.0, lm=1.8, lr=1e-4)            # the context is still usable, on the old basis
    # more directions than rows, a tensor without subspace, an active perturbation
    q = Pair([(8, 64), (1, 16)], [4, 0], "f32")
    with pytest.raises(zgr.ZgrError) as e:
        q.lib.build_subspace(1, None)
    assert e.value.code == zgr.EINVAL
    q.lib.perturb(1, 1e-3)
    with pytest.raises(zgr.ZgrError) as e:
        q.lib.build_subspace(0, None)
    assert e.value.code == zgr.ESTATE
    q.lib.restore_update(1, 2.0, 2.0, 0.0)


# ------------------------------------------------------------------------------------- adaptive alpha
@pytest.mark.parametrize("scale_mode", [zgr.SCALE_UNIT, zgr.SCALE_PAPER])
def test_adaptive_alpha_balances_the_energies(scale_mode):
    shapes, ranks = [(96, 256), (1, 100), (300, 392), (64, 264)], [8, 0, 32, 4]
    p = Pair(shapes, ranks, "bf16", bits=16, alpha=0.3, scale_mode=scale_mode, seed=9)
    # compressed coefficients with a scale three times that of a unit Gaussian on one tensor: the balance moves
    q, sc = synth.dtc_payload(32, 392, seed=3)
    p.set_dtc(2, q, (3.0 * sc).astype(np.float32))
    seed = 21
    st0 = p.lib.get_stats(seed)
    exp0 = np.array([oracle.stats_tensor(p.oracle_tensor(l), seed, l, 16, p.a, p.b) for l in range(4)])
    np.testing.assert_allclose(st0, exp0, rtol=2e-5, atol=1e-12 * p.z_unit() ** 2)
    alpha_exp = oracle.adapt_alpha(exp0, p.a, p.b, p.d, p.K, 0.3, 0.05, 0.95, 1.0)
    alpha_got = p.lib.adapt_alpha(st0, 0.05, 0.95, 1.0)
    assert alpha_got == pytest.approx(alpha_exp, rel=1e-5) and alpha_got > 0.5
    a1, b1 = p.lib.scalars()
    a1_o, b1_o = oracle.mix_scalars(alpha_got, p.d, p.K, scale_mode)
    assert a1 == pytest.approx(a1_o, rel=1e-14) and b1 == pytest.approx(b1_o, rel=1e-14)
    # the norms under the new ratio: the two parts now carry the same energy, and asking again changes nothing
    st1 = p.lib.get_stats(seed)
    assert st1[:, 0].sum() == pytest.approx(st1[:, 1].sum(), rel=1e-4)
    assert p.lib.adapt_alpha(st1, 0.05, 0.95, 1.0) == pytest.approx(alpha_got, rel=1e-4)
    # damping and clamping
    p.lib.set_alpha(0.3)
    st0 = p.lib.get_stats(seed)
    assert p.lib.adapt_alpha(st0, 0.05, 0.95, 0.5) == pytest.approx(0.5 * 0.3 + 0.5 * alpha_exp, rel=1e-5)
    p.lib.set_alpha(0.3)
    assert p.lib.adapt_alpha(p.lib.get_stats(seed), 0.05, 0.4, 1.0) == pytest.approx(0.4, rel=1e-12)
    # a step under the adapted ratio still matches the oracle
    p.alpha = 0.4
    p.a, p.b = oracle.mix_scalars(0.4, p.d, p.K, scale_mode)
    p.step(seed=33, lp=2.1, lm=1.9, lr=1e-4)
    # argument checks
    L = zgr.lib()
    import ctypes
    out = ctypes.c_double()
    arr = (ctypes.c_double * (3 * 4))(*st0.ravel())
    assert L.zgr_adapt_alpha(p.lib._h, arr, 0.6, 0.4, 1.0, ctypes.byref(out)) == zgr.EINVAL
    assert L.zgr_adapt_alpha(p.lib._h, arr, 0.1, 0.9, 1.5, ctypes.byref(out)) == zgr.EINVAL
    assert L.zgr_adapt_alpha(p.lib._h, None, 0.1, 0.9, 1.0, ctypes.byref(out)) == zgr.EINVAL
    p.lib.perturb(1, 1e-3)
    assert L.zgr_adapt_alpha(p.lib._h, arr, 0.1, 0.9, 1.0, ctypes.byref(out)) == zgr.ESTATE
    p.lib.restore_update(1, 2.0, 2.0, 0.0)
