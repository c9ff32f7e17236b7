"""GPU tests of the remaining entry points of the C ABI: subspace updates (a guided round delivers
a new U), per-kernel timing, device status, and the choice between the tensor-core paths."""
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

import oracle
from paper_2601_12917_b200 import synth, zgr

from helpers import Pair, to_double

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.mark.parametrize("dtype,rank,src", [("bf16", 32, "host"), ("bf16", 16, "device"), ("f32", 8, "host"), ("f16", 64, "inplace")])
def test_update_subspace_is_followed_by_the_sweeps(dtype, rank, src):
    shapes, ranks = [(256, 384), (1, 40)], [rank, 0]
    p = Pair(shapes, ranks, dtype, seed=9)
    p.step(seed=1, lp=2.0, lm=1.9, lr=1e-4)                      # with the first subspace
    new_U = synth.subspace(256, rank, 4242)
    if src == "host":
        p.lib.update_subspace(0, torch.from_numpy(new_U).pin_memory())
    elif src == "device":
        p.lib.update_subspace(0, torch.from_numpy(new_U).cuda())
    else:
        p.U[0].copy_(torch.from_numpy(new_U))                     # caller rewrites its own buffer ...
        p.lib.update_subspace(0, None)                            # ... and tells the library
    torch.cuda.synchronize()
    np.testing.assert_array_equal(p.U[0].cpu().numpy(), new_U)   # the device buffer given at init now holds the new basis
    reports = p.step(seed=2, lp=1.7, lm=2.2, lr=1e-4)            # Pair.oracle_tensor reads U back from the device
    assert min(rep["moved"] for call in reports for rep in call) > 0.3
    # and the perturbation really lies in the new span when alpha = 0
    q = Pair(shapes, ranks, dtype, seed=9, alpha=0.0)
    q.lib.update_subspace(0, torch.from_numpy(new_U).cuda())
    Z = to_double(q.lib.debug_z(5, 0)).reshape(256, 384)
    U64 = new_U.astype(np.float64)
    assert np.abs(Z - U64 @ (U64.T @ Z)).max() <= 2e-4 * np.abs(Z).max()


def test_update_subspace_argument_and_state_errors():
    p = Pair([(64, 128), (1, 16)], [16, 0], "bf16")
    with pytest.raises(zgr.ZgrError) as e:
        p.lib.update_subspace(1, None)                            # tensor without a subspace
    assert e.value.code == zgr.EINVAL
    p.lib.perturb(3, 1e-3)
    with pytest.raises(zgr.ZgrError) as e:
        p.lib.update_subspace(0, None)                            # not between a perturb and its restore_update
    assert e.value.code == zgr.ESTATE
    p.lib.restore_update(3, 2.0, 2.0, 0.0)


def test_profile_reports_every_kernel_family_that_ran():
    p = Pair([(256, 256), (1, 64), (128, 264), (200, 100)], [32, 0, 8, 6], "bf16")
    p.lib.profile(True)
    p.lib.perturb(1, 1e-3)
    p.lib.restore_update(1, 2.0, 2.0, 0.0)
    entries = p.lib.profile_read()
    by_path = {k["path"]: k for k in entries}
    assert set(by_path) == {"umma", "iso", "fma", "generic"}
    assert by_path["umma"]["elements"] == 256 * 256 and by_path["iso"]["elements"] == 64
    assert by_path["fma"]["elements"] == 128 * 264 and by_path["generic"]["elements"] == 200 * 100
    for k in entries:
        assert k["launches"] == 2 and k["ms_total"] > 0
    assert p.lib.profile_read() == []                             # reading clears the record
    p.lib.profile(False)
    p.lib.perturb(2, 1e-3)
    p.lib.restore_update(2, 2.0, 2.0, 0.0)
    assert p.lib.profile_read() == []
    assert p.lib.device_status() == 0


def test_legacy_tensor_core_path_gives_the_same_results():
    """ZGR_TENSOR_PATH=legacy selects the mma.sync kernels for the same tensors; both paths must
    agree with the oracle, hence with each other up to the 1-ulp tolerance."""
    code = r'''
import sys
sys.path.insert(0, sys.argv[1]); sys.path.insert(0, sys.argv[1] + "/tests")
from helpers import Pair
p = Pair([(200, 520), (1, 64)], [32, 0], "bf16", seed=3, bits=16)
p.lib.profile(True)
p.step(seed=5, lp=2.2, lm=1.7, lr=1e-4)
print(sorted(k["path"] for k in p.lib.profile_read()))
'''
    env = dict(os.environ, ZGR_TENSOR_PATH="legacy")
    r = subprocess.run([sys.executable, "-c", code, ROOT], env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    assert "'mma'" in r.stdout and "umma" not in r.stdout


def test_set_alpha_between_steps():
    """zgr_set_alpha recomputes the mixing scalars of Eq. (perturbation); the following sweeps and norms use them."""
    p = Pair([(140, 520), (1, 64), (96, 256)], [32, 0, 8], "bf16", bits=16, seed=3, alpha=0.5)
    p.step(seed=1, lp=2.0, lm=1.9, lr=1e-4)
    for alpha in (0.2, 1.0, 0.0, 0.7):
        p.lib.set_alpha(alpha)
        p.alpha = alpha
        p.a, p.b = oracle.mix_scalars(alpha, p.d, p.K, p.scale_mode)
        a, b = p.lib.scalars()
        assert a == pytest.approx(p.a, rel=1e-14) and b == pytest.approx(p.b, rel=1e-14)
        p.step(seed=10 + int(alpha * 10), lp=2.2, lm=1.7, lr=1e-4)
        got = p.lib.get_stats(5)
        for l in range(3):
            exp = oracle.stats_tensor(p.oracle_tensor(l), 5, l, p.bits, p.a, p.b)
            np.testing.assert_allclose(got[l], exp, rtol=2e-5, atol=1e-12)
    with pytest.raises(zgr.ZgrError) as e:
        p.lib.set_alpha(1.5)
    assert e.value.code == zgr.EINVAL
    p.lib.perturb(3, 1e-3)
    with pytest.raises(zgr.ZgrError) as e:
        p.lib.set_alpha(0.5)
    assert e.value.code == zgr.ESTATE
    p.lib.restore_update(3, 2.0, 2.0, 0.0)
    # a context built without a guided part cannot grow one
    q = Pair([(64, 256)], [8], "f32", alpha=1.0)
    with pytest.raises(zgr.ZgrError) as e:
        q.lib.set_alpha(0.5)
    assert e.value.code == zgr.ESTATE
    q.lib.set_alpha(1.0)


def test_update_subspaces_in_one_call():
    """zgr_update_subspaces: all guided tensors at once (one fused rebuild of the operand copies), a subset
    (per-tensor rebuilds), device and host sources, then argument errors."""
    shapes, ranks = [(256, 384), (1, 40), (200, 512), (96, 256)], [32, 0, 16, 8]
    p = Pair(shapes, ranks, "bf16", seed=9, bits=16)
    p.step(seed=1, lp=2.0, lm=1.9, lr=1e-4)
    new = {l: synth.subspace(shapes[l][0], ranks[l], 500 + l) for l in (0, 2, 3)}
    launches0 = p.lib.launch_count()
    p.lib.update_subspaces([0, 2, 3], [torch.from_numpy(new[l]).pin_memory() for l in (0, 2, 3)])      # whole model, host
    assert p.lib.launch_count() - launches0 == 1                  # one fused launch for the two tensor-core tensors; rank 8 reads U directly
    torch.cuda.synchronize()
    for l in (0, 2, 3):
        np.testing.assert_array_equal(p.U[l].cpu().numpy(), new[l])
    reports = p.step(seed=2, lp=1.7, lm=2.2, lr=1e-4)
    assert min(rep["moved"] for call in reports for rep in call) > 0.3
    newer = synth.subspace(200, 16, 777)
    p.lib.update_subspaces([2], [torch.from_numpy(newer).cuda()])                                      # subset, device
    p.step(seed=3, lp=2.1, lm=2.0, lr=1e-4)
    p.U[0].copy_(torch.from_numpy(synth.subspace(256, 32, 778)))
    p.lib.update_subspaces([0, 2], [None, None])                                                       # rewritten in place
    p.step(seed=4, lp=2.1, lm=2.0, lr=1e-4)
    for bad in ([], [1], [0, 0], [9]):
        with pytest.raises((zgr.ZgrError, AssertionError)) as e:
            p.lib.update_subspaces(bad, [None] * len(bad))
        if isinstance(e.value, zgr.ZgrError):
            assert e.value.code == zgr.EINVAL
    p.lib.perturb(5, 1e-3)
    with pytest.raises(zgr.ZgrError) as e:
        p.lib.update_subspaces([0], [None])
    assert e.value.code == zgr.ESTATE
    p.lib.restore_update(5, 2.0, 2.0, 0.0)
