"""GPU parity of the multi-seed sweeps (zgr_sweep_multi, zgr_restore_update_multi) against the oracle.

One pass applies  sum_q c_q z(seed_q)  with a single rounding: the sum over seeds of Algorithm 1
("Recover gradient", "Update").  Every kernel family is exercised with two to eight terms, then the
deferred schedule of a Q-query step (2Q+1 sweeps), the server-side aggregation (nothing to restore),
compressed coefficients, the ledger of active seeds and the argument errors.
"""
import os
import subprocess
import sys

import numpy as np
import pytest
import torch

import oracle
from paper_2601_12917_b200 import zgr

from helpers import Pair

pytestmark = pytest.mark.gpu
ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

MODELS = {
    "iso+fma": ([(1, 777), (128, 256), (70, 520), (1, 8)], [0, 4, 8, 0]),
    "umma16": ([(150, 1032), (1, 100)], [16, 0]),
    "umma32": ([(200, 512), (64, 1024), (300, 392)], [32, 32, 32]),
    "umma64": ([(96, 776)], [64]),
    "generic": ([(45, 100), (33, 52)], [6, 20]),
}


@pytest.mark.parametrize("bits", [32, 16])
@pytest.mark.parametrize("dtype", ["f32", "f16", "bf16"])
@pytest.mark.parametrize("model", list(MODELS))
def test_multi_seed_sweep_per_call_parity(model, dtype, bits):
    shapes, ranks = MODELS[model]
    p = Pair(shapes, ranks, dtype, bits=bits, seed=13)
    seeds, coeffs = [5, 2**40 + 7, 6], [1e-3, -2e-3, 7e-4]
    reports = p.call_and_check_multi(seeds, coeffs, lambda: p.lib.sweep_multi(seeds, coeffs), "sweep_multi(3)")
    for rep in reports:
        assert rep["moved"] > 0.3, rep
        if dtype != "f32":
            assert rep["equal"] > 0.9, rep
    assert p.lib.active_seeds() == 3
    # undo two of them and check the ledger
    undo = [-c for c in coeffs[:2]]
    p.call_and_check_multi(seeds[:2], undo, lambda: p.lib.sweep_multi(seeds[:2], undo), "sweep_multi(2)")
    assert p.lib.active_seeds() == 1 and p.lib.state() == (True, seeds[1], 0.0)
    p.lib.restore_update(seeds[2], 2.0, 2.0, 0.0)
    assert p.lib.active_seeds() == 0


def test_eight_terms_in_one_pass():
    p = Pair([(140, 520), (1, 333), (64, 256)], [32, 0, 8], "bf16", bits=16, seed=2)
    seeds = [100 + i for i in range(8)]
    coeffs = [(-1) ** i * 1e-3 * (1 + 0.25 * i) for i in range(8)]
    reports = p.call_and_check_multi(seeds, coeffs, lambda: p.lib.sweep_multi(seeds, coeffs), "sweep_multi(8)")
    assert all(r["moved"] > 0.3 for r in reports)


@pytest.mark.parametrize("dtype,bits", [("bf16", 16), ("f32", 32)])
def test_deferred_schedule_of_a_four_query_step(dtype, bits):
    """2Q+1 sweeps: each restore is fused with the next query's perturbation, one final multi-seed update."""
    Q, lr = 4, 1e-4
    p = Pair([(200, 520), (1, 64), (96, 256)], [32, 0, 4], dtype, bits=bits, seed=4)
    eps = p.eps
    seeds = [1000 + q for q in range(Q)]
    rng = np.random.default_rng(3)
    lp, lm = rng.uniform(1.5, 2.5, Q).tolist(), rng.uniform(1.5, 2.5, Q).tolist()
    launches0 = p.lib.launch_count()
    p.call_and_check_multi([seeds[0]], [eps], lambda: p.lib.sweep_multi([seeds[0]], [eps]), "perturb q=0")
    launches_per_sweep = p.lib.launch_count() - launches0
    p.call_and_check_multi([seeds[0]], [-2 * eps], lambda: p.lib.sweep_multi([seeds[0]], [-2 * eps]), "perturb- q=0")
    for q in range(1, Q):
        pair = [seeds[q - 1], seeds[q]]
        p.call_and_check_multi(pair, [eps, eps], lambda: p.lib.sweep_multi(pair, [eps, eps]), f"restore {q-1} + perturb {q}")
        assert p.lib.active_seeds() == 1
        p.call_and_check_multi([seeds[q]], [-2 * eps], lambda: p.lib.sweep_multi([seeds[q]], [-2 * eps]), f"perturb- q={q}")
    coeffs = [-(lr / Q) * oracle.projected_grad(a, b, eps) for a, b in zip(lp, lm)]
    coeffs[-1] += eps                                           # the last query is still applied with -eps
    p.call_and_check_multi(seeds, coeffs, lambda: p.lib.restore_update_multi(seeds, lp, lm, lr / Q), "final update")
    assert p.lib.active_seeds() == 0
    assert p.lib.launch_count() - launches0 == (2 * Q + 1) * launches_per_sweep


def test_server_side_aggregation_and_single_seed_form():
    p = Pair([(130, 512), (1, 40)], [16, 0], "f16", bits=16, seed=9)
    eps, lr = p.eps, 2e-4
    seeds, lp, lm = [7, 8, 9], [2.0, 1.7, 2.2], [1.9, 1.8, 2.0]
    coeffs = [-lr * oracle.projected_grad(a, b, eps) for a, b in zip(lp, lm)]
    p.call_and_check_multi(seeds, coeffs, lambda: p.lib.restore_update_multi(seeds, lp, lm, lr), "aggregate 3 clients")
    assert p.lib.active_seeds() == 0
    # n = 1 is the plain restore_update
    p.lib.perturb(3, eps)
    c = -eps - lr * oracle.projected_grad(2.1, 2.0, eps)
    p.call_and_check_multi([3], [c], lambda: p.lib.restore_update_multi([3], [2.1], [2.0], lr), "restore_update_multi(1)")
    assert p.lib.active_seeds() == 0


@pytest.mark.parametrize("dtype,rank,cols", [("bf16", 32, 520), ("f32", 8, 264)])
def test_multi_seed_with_compressed_coefficients(dtype, rank, cols):
    """Compressed coefficients do not depend on the seed: the guided part is (sum_q c_q) b U G."""
    p = Pair([(96, cols)], [rank], dtype, bits=16 if dtype != "f32" else 32, seed=6)
    G = oracle.coeffs(1, 0, p.bits, rank, cols)
    q, sc, ze = oracle.dtc_quantise(G, 8, symmetric=True)
    p.set_dtc(0, q, sc)
    seeds, coeffs = [31, 32], [1e-3, 5e-4]
    reps = p.call_and_check_multi(seeds, coeffs, lambda: p.lib.sweep_multi(seeds, coeffs), "sweep_multi with DTC")
    assert reps[0]["moved"] > 0.3


def test_argument_and_state_errors():
    p = Pair([(32, 64), (1, 16)], [4, 0], "f32")
    before = [t.clone() for t in p.theta]
    L = zgr.lib()
    for seeds, coeffs in (([], []), (list(range(9)), [1e-3] * 9), ([1, 1], [1e-3, 1e-3]), ([1, 2], [1e-3, float("nan")])):
        with pytest.raises(zgr.ZgrError) as e:
            p.lib.sweep_multi(seeds, coeffs)
        assert e.value.code == zgr.EINVAL
    with pytest.raises(zgr.ZgrError) as e:
        p.lib.restore_update_multi([1, 2], [2.0, float("inf")], [1.0, 1.0], 0.1)
    assert e.value.code == zgr.EINVAL
    assert L.zgr_sweep_multi(None, 1, None, None, None) == zgr.EINVAL
    torch.cuda.synchronize()
    for t, b in zip(p.theta, before):
        assert torch.equal(t, b)
    p.lib.sweep_multi([1, 2], [1e-3, 1e-3])
    assert p.lib.active_seeds() == 2
    with pytest.raises(zgr.ZgrError) as e:
        p.lib.perturb(1, 1e-3)                       # zgr_perturb keeps its one-seed-at-a-time rule
    assert e.value.code == zgr.ESTATE
    with pytest.raises(zgr.ZgrError) as e:
        p.lib.set_coeffs_dtc(0, torch.zeros(4, 64, dtype=torch.int8, device="cuda"), torch.ones(4, device="cuda"))
    assert e.value.code == zgr.ESTATE
    p.lib.restore_update(1, 2.0, 2.0, 0.0)           # a single seed of several can be closed on its own
    p.lib.restore_update_multi([2], [2.0], [2.0], 0.0)
    assert p.lib.active_seeds() == 0


def test_multi_seed_sweeps_on_the_legacy_tensor_core_plan():
    """With ZGR_TENSOR_PATH=legacy the rank>8 tensors of a multi-seed sweep take the fallback kernel."""
    code = r'''
import sys
sys.path.insert(0, sys.argv[1]); sys.path.insert(0, sys.argv[1] + "/tests")
from helpers import Pair
p = Pair([(200, 520), (1, 64)], [32, 0], "bf16", seed=3, bits=16)
p.lib.profile(True)
p.call_and_check_multi([5, 6], [1e-3, -5e-4], lambda: p.lib.sweep_multi([5, 6], [1e-3, -5e-4]), "legacy multi")
print(sorted(k["path"] for k in p.lib.profile_read()))
'''
    env = dict(os.environ, ZGR_TENSOR_PATH="legacy")
    r = subprocess.run([sys.executable, "-c", code, ROOT], env=env, capture_output=True, text=True, timeout=600)
    assert r.returncode == 0, r.stderr[-2000:]
    assert "'generic'" in r.stdout and "umma" not in r.stdout and "'mma'" not in r.stdout
