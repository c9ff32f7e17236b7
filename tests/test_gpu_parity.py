"""GPU parity: the CUDA library, called through its C ABI, against the CPU oracle (needs a B200).

Element-by-element comparison on seeded inputs small enough for the oracle to replay in seconds
but spanning several tiles, strips and ragged tails of every kernel family; then the state
machine, the compressed-coefficient entry point and the norm bookkeeping.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2601_12917_b200 import synth, zgr

from helpers import Pair, check_sweep, to_double

pytestmark = pytest.mark.gpu


# ------------------------------------------------------------------------------------- generator
@pytest.mark.parametrize("seed,tensor,tag,first", [
    (0, 0, 0, 0), (1, 3, 1, 12345), (0xDEADBEEFCAFEF00D, 290, 1, 2**32 - 1000), (2**64 - 1, 7, 0, 2**40 + 5),
])
def test_generator_stream_is_bit_exact(seed, tensor, tag, first):
    p = Pair([(8, 8)], [0], "f32")
    n = 1 << 18
    got = p.lib.debug_philox(seed, tensor, tag, first, n).cpu().numpy().view(np.uint32)
    exp = oracle.blocks(seed, tensor, tag, first, n)
    np.testing.assert_array_equal(got, exp)


def test_generator_many_blocks():
    p = Pair([(8, 8)], [0], "f32")
    n = 1 << 24
    got = p.lib.debug_philox(42, 1, 0, 0, n).cpu().numpy().view(np.uint32)
    exp = oracle.blocks(42, 1, 0, 0, n)
    np.testing.assert_array_equal(got, exp)


# ------------------------------------------------------------------------------------- z itself
Z_CASES = [
    # (shape, rank, kernel family of 16-bit tensors, what it exercises)
    ((1, 1000), 0, "iso", "iso vector + ragged tail"),
    ((64, 256), 4, "fma", "fma R=4"),
    ((300, 520), 8, "fma", "fma R=8, three strips, last one ragged"),
    ((37, 264), 3, "fma", "fma rank 3 padded to 4"),
    ((50, 72), 5, "fma", "fma rank 5 padded to 8"),
    ((100, 1032), 16, "mma", "mma K=16, ragged strip and row tile"),
    ((130, 512), 32, "mma", "mma K=32"),
    ((96, 520), 64, "mma", "mma K=64"),
    ((48, 128), 12, "mma", "mma rank 12 padded to 16"),
    ((72, 64), 40, "mma", "mma rank 40 padded to 64"),
    ((45, 100), 6, "generic", "generic (columns not a multiple of 8), low rank"),
    ((45, 100), 20, "generic", "generic, high rank"),
]
# absolute tolerance on a unit-variance z: fp32 tensors use the accurate transform and an exact fp32
# contraction; 16-bit tensors use the hardware approximations and, above rank 8, split 16-bit operands on tensor cores
Z_TOL = {("f32", "iso"): 2e-6, ("f32", "fma"): 2e-6, ("f32", "mma"): 3e-6, ("f32", "generic"): 3e-6,
         ("bf16", "iso"): 1e-5, ("bf16", "fma"): 1e-5, ("bf16", "mma"): 4e-5, ("bf16", "generic"): 1e-5}
# ("mma" rows: zgr_debug_z runs the legacy mma.sync kernel for these tensors, whose operands are split into bf16
#  hi/lo (16 significant bits: 4.5e-6 rms, up to 4e-5 in the tail); the tcgen05 kernel that the sweeps use for them
#  splits into fp16 hi/lo and is compared with the oracle at 1.2e-5 in test_gpu_tcgen05_z.py)


@pytest.mark.parametrize("bits", [32, 16])
@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shape,rank,family,what", Z_CASES)
def test_perturbation_matches_oracle(shape, rank, family, what, dtype, bits):
    p = Pair([shape, (1, 40)], [rank, 0], dtype, bits=bits, seed=3)
    seed = 1234567
    tol = Z_TOL[(dtype, family)]
    for l in range(2):
        got = to_double(p.lib.debug_z(seed, l))
        exp = oracle.z_tensor(p.oracle_tensor(l), seed, l, bits, p.a, p.b).ravel()
        err = np.abs(got - exp).max()
        assert err <= tol, f"{what} [{dtype}]: max |z_gpu - z_oracle| = {err:.3e}"
        assert np.abs(exp).max() > 0.5


@pytest.mark.parametrize("scale_mode", [zgr.SCALE_PAPER, zgr.SCALE_UNIT])
@pytest.mark.parametrize("alpha", [0.0, 0.3, 1.0])
def test_perturbation_scalings_and_alpha_limits(scale_mode, alpha):
    shapes, ranks = [(64, 256), (1, 64), (64, 128)], [8, 0, 16]
    p = Pair(shapes, ranks, "bf16", alpha=alpha, scale_mode=scale_mode)
    a, b = p.lib.scalars()
    assert a == pytest.approx(p.a, rel=1e-14) and b == pytest.approx(p.b, rel=1e-14, abs=1e-300)
    for l in range(3):
        got = to_double(p.lib.debug_z(99, l))
        exp = oracle.z_tensor(p.oracle_tensor(l), 99, l, 32, p.a, p.b).ravel()
        unit = 1.0 if scale_mode == zgr.SCALE_UNIT else 1.0 / np.sqrt(p.d)
        assert np.abs(got - exp).max() <= 1e-4 * unit
        if alpha == 0.0 and ranks[l] == 0:
            assert np.all(got == 0)


# ------------------------------------------------------------------------------------- sweeps
SWEEP_MODELS = {
    "iso+fma": ([(1, 777), (128, 256), (70, 520), (1, 8)], [0, 4, 8, 0]),
    "mma16": ([(150, 1032), (1, 100)], [16, 0]),
    "mma32": ([(200, 512), (64, 1024)], [32, 32]),
    "mma64": ([(96, 776)], [64]),
    "generic": ([(45, 100), (33, 52)], [6, 20]),
}


@pytest.mark.parametrize("bits", [32, 16])
@pytest.mark.parametrize("dtype", ["f32", "f16", "bf16"])
@pytest.mark.parametrize("model", list(SWEEP_MODELS))
def test_step_per_call_parity(model, dtype, bits):
    shapes, ranks = SWEEP_MODELS[model]
    p = Pair(shapes, ranks, dtype, bits=bits, seed=11)
    reports = p.step(seed=5, lp=2.2, lm=1.7, lr=1e-4)
    for call in reports:
        for rep in call:
            assert rep["moved"] > 0.3, rep         # the sweep really changed the weights
            # (16-bit results: check_sweep holds the bit-identical fraction against what a z accurate to
            #  helpers.DELTA_Z_16BIT allows for this call's coefficient)
    assert p.lib.state()[0] is False


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_unaligned_weights_take_the_fallback_kernels(dtype):
    p = Pair([(40, 64), (1, 50), (24, 128)], [4, 0, 16], dtype, misalign=True)
    assert p.theta[0].data_ptr() % 16 != 0
    p.step(seed=8, lp=2.0, lm=1.9, lr=1e-4)


def test_tiny_configuration_full_cycle():
    wl = synth.workload("tiny")
    shapes = [(t.rows, t.cols) for t in wl.tensors]
    ranks = [t.rank for t in wl.tensors]
    for scale_mode in (zgr.SCALE_PAPER, zgr.SCALE_UNIT):
        p = Pair(shapes, ranks, "f32", alpha=wl.alpha, eps=wl.eps, scale_mode=scale_mode)
        theta0 = [to_double(t).copy() for t in p.theta]
        lp, lm = wl.losses(0, 0)
        p.step(seed=wl.seed(0, 0), lp=lp, lm=lm, lr=wl.lr)
        # (L+, L-) = (2.31, 2.29): g = 10, lr g = eps, so the fused third sweep adds (eps - lr g) z ~ 0:
        # theta ends at theta0 - eps z (rounded twice), not at theta0.
        for l, t in enumerate(p.theta):
            z = oracle.z_tensor(p.oracle_tensor(l), wl.seed(0, 0), l, 32, p.a, p.b).ravel()
            np.testing.assert_allclose(to_double(t), theta0[l] - wl.eps * z, atol=3e-8 + 1e-6 * p.theta_max)


def test_trajectory_parity_fp32_ten_steps():
    # both sides run 10 steps independently (no re-synchronisation between calls)
    shapes, ranks = [(96, 256), (1, 128), (64, 264)], [8, 0, 4]
    p = Pair(shapes, ranks, "f32", seed=21)
    ots = [p.oracle_tensor(l) for l in range(3)]
    o = oracle.OracleZGR(ots, alpha=p.alpha, eps=p.eps, scale_mode=p.scale_mode, bits=32)
    rng = np.random.default_rng(0)
    for step in range(10):
        lp, lm = rng.uniform(1.5, 2.5, 2)
        s = 1000 * step
        p.lib.perturb(s, p.eps); o.perturb(s, p.eps)
        p.lib.perturb(s, -2 * p.eps); o.perturb(s, -2 * p.eps)
        p.lib.restore_update(s, lp, lm, 1e-4); o.restore_update(s, lp, lm, 1e-4)
    torch.cuda.synchronize()
    theta_max = max(np.abs(oracle.decode(t.theta, t.dtype)).max() for t in ots)   # the updates have grown theta
    assert theta_max > p.theta_max
    for l, t in enumerate(ots):
        err = np.abs(to_double(p.theta[l]) - oracle.decode(t.theta, t.dtype)).max()
        assert err <= 1e-6 * theta_max


def test_results_do_not_depend_on_launch_history():
    shapes, ranks = [(200, 512), (1, 100)], [32, 0]
    a = Pair(shapes, ranks, "bf16", seed=2)
    b = Pair(shapes, ranks, "bf16", seed=2)
    a.lib.perturb(7, 1e-3)
    b.lib.perturb(3, 1e-3); b.lib.restore_update(3, 2.0, 2.0, 0.0)   # some other work first
    for l in range(2):
        b.theta[l].copy_(Pair(shapes, ranks, "bf16", seed=2).theta[l])
    b.lib.perturb(7, 1e-3)
    torch.cuda.synchronize()
    for l in range(2):
        assert torch.equal(a.theta[l], b.theta[l])


# ------------------------------------------------------------------------------------- DTC
@pytest.mark.parametrize("dtype,rank,cols", [("f32", 8, 264), ("bf16", 64, 520), ("bf16", 16, 512), ("f16", 20, 100)])
def test_compressed_coefficients(dtype, rank, cols):
    p = Pair([(80, cols), (1, 30)], [rank, 0], dtype, seed=4)
    q, sc = synth.dtc_payload(rank, cols, seed=1)
    p.set_dtc(0, q, sc)
    p.step(seed=77, lp=2.4, lm=1.6, lr=1e-4)
    # with zero points
    ze = (np.arange(rank) % 5 - 2).astype(np.float32)
    p.set_dtc(0, q, sc, ze)
    p.step(seed=78, lp=1.6, lm=2.4, lr=1e-4)
    # back to seed-drawn coefficients
    p.q[0] = p.scale[0] = p.zero[0] = None
    p.lib.clear_coeffs(0)
    p.step(seed=79, lp=2.0, lm=1.9, lr=1e-4)


@pytest.mark.parametrize("dtype,rank,cols", [("f32", 8, 264), ("bf16", 32, 520), ("bf16", 64, 384), ("f16", 16, 1032), ("f16", 20, 101)])
def test_int4_compressed_coefficients(dtype, rank, cols):
    """The paper's INT4 payload (Sec. 3.4): unsigned 4-bit codes, two to a byte, with per-row scale and zero point."""
    bits = 32 if dtype == "f32" else 16
    p = Pair([(80, cols), (1, 30)], [rank, 0], dtype, seed=4, bits=bits)
    G = oracle.coeffs(9, 0, bits, rank, cols)
    q, sc, ze = oracle.dtc_quantise_int4(G)
    p.set_dtc(0, q, sc, ze, bits=4)
    reports = p.step(seed=77, lp=2.4, lm=1.6, lr=1e-4)
    assert all(rep["moved"] > 0.3 for call in reports for rep in call)
    # the guided part really comes from the codes: z moves by at most the quantisation bound from the seed-drawn one
    if dtype == "f32":
        z4 = to_double(p.lib.debug_z(9, 0)).reshape(80, cols)
        p.q[0] = p.scale[0] = p.zero[0] = None
        p.lib.clear_coeffs(0)
        z_seed = to_double(p.lib.debug_z(9, 0)).reshape(80, cols)
        U = p.U[0].cpu().numpy().astype(np.float64)
        bound = p.b * (np.abs(U) @ np.tile(0.5 * sc[:, None].astype(np.float64), (1, cols)))
        assert np.all(np.abs(z4 - z_seed) <= bound * 1.001 + 1e-4) and np.abs(z4 - z_seed).max() > 0
    with pytest.raises(zgr.ZgrError) as e:
        p.lib.set_coeffs_dtc(0, torch.zeros(rank, cols, dtype=torch.int8, device="cuda"), torch.ones(rank, device="cuda"), None, 5)
    assert e.value.code == zgr.EINVAL


def test_dtc_path_agrees_with_quantised_seed_coefficients():
    # quantise the seed-drawn G with the oracle's quantiser (Sec. 3.4) and feed it back compressed:
    # z must move by at most the quantisation bound
    rank, cols, rows = 16, 512, 64
    p = Pair([(rows, cols)], [rank], "f32", alpha=0.0)
    seed = 31
    z_seed = to_double(p.lib.debug_z(seed, 0)).reshape(rows, cols)
    G = oracle.coeffs(seed, 0, 32, rank, cols)
    q, sc, _ = oracle.dtc_quantise(G, 8, True)
    p.set_dtc(0, q, sc)
    z_dtc = to_double(p.lib.debug_z(seed, 0)).reshape(rows, cols)
    U = p.U[0].cpu().numpy().astype(np.float64)
    bound = p.b * (np.abs(U) @ np.tile(0.5 * sc[:, None].astype(np.float64), (1, cols)))
    assert np.all(np.abs(z_dtc - z_seed) <= bound * 1.001 + 1e-4)
    assert np.abs(z_dtc - z_seed).max() > 0


# ------------------------------------------------------------------------------------- state machine / errors
def test_state_machine_and_argument_errors():
    p = Pair([(32, 64), (1, 16)], [4, 0], "f32")
    L = zgr.lib()
    before = [t.clone() for t in p.theta]
    with pytest.raises(zgr.ZgrError) as e:
        p.lib.restore_update(1, 2.0, 1.0, 0.1)
    assert e.value.code == zgr.ESTATE
    with pytest.raises(zgr.ZgrError) as e:
        p.lib.perturb(1, float("nan"))
    assert e.value.code == zgr.EINVAL
    torch.cuda.synchronize()
    for t, b in zip(p.theta, before):
        assert torch.equal(t, b)                      # failed calls leave theta untouched
    p.lib.perturb(1, 1e-3)
    assert p.lib.state() == (True, 1, 1e-3)
    with pytest.raises(zgr.ZgrError) as e:
        p.lib.perturb(2, 1e-3)
    assert e.value.code == zgr.ESTATE
    with pytest.raises(zgr.ZgrError) as e:
        p.lib.restore_update(2, 2.0, 1.0, 0.1)
    assert e.value.code == zgr.ESTATE
    with pytest.raises(zgr.ZgrError) as e:
        p.lib.restore_update(1, float("inf"), 1.0, 0.1)
    assert e.value.code == zgr.EINVAL
    with pytest.raises(zgr.ZgrError) as e:
        p.lib.set_coeffs_dtc(0, torch.zeros(4, 64, dtype=torch.int8, device="cuda"), torch.ones(4, device="cuda"))
    assert e.value.code == zgr.ESTATE                 # coefficients may not change mid-step
    p.lib.restore_update(1, 2.0, 2.0, 0.0)
    assert p.lib.state()[0] is False
    with pytest.raises(zgr.ZgrError) as e:
        p.lib.set_coeffs_dtc(1, torch.zeros(4, 16, dtype=torch.int8, device="cuda"), torch.ones(4, device="cuda"))
    assert e.value.code == zgr.EINVAL                 # tensor 1 has no subspace
    assert p.lib.launch_count() > 0
    assert L.zgr_perturb(None, 0, 1.0, None) == zgr.EINVAL


def test_init_rejects_bad_arguments():
    w = torch.zeros(8, 8, device="cuda")
    U = torch.zeros(8, 2, device="cuda")
    for kwargs in ({"alpha": 1.5}, {"eps": 0.0}, {"eps": float("nan")}, {"scale_mode": 7}, {"bits_per_normal": 24}):
        args = dict(alpha=0.5, eps=1e-3, scale_mode=zgr.SCALE_UNIT, bits_per_normal=32)
        args.update(kwargs)
        with pytest.raises(zgr.ZgrError) as e:
            zgr.Zgr([w], [U], **args)
        assert e.value.code == zgr.EINVAL
    with pytest.raises(zgr.ZgrError):
        zgr.Zgr([w], [torch.zeros(8, 65, device="cuda")], 0.5, 1e-3)      # rank above the maximum


def test_restore_is_within_two_ulp_at_lr_zero():
    for dtype in ("f32", "f16", "bf16"):
        p = Pair([(64, 256), (1, 99), (64, 512)], [8, 0, 32], dtype, seed=6)
        before = [to_double(t).copy() for t in p.theta]
        p.lib.perturb(3, p.eps); p.lib.perturb(3, -2 * p.eps); p.lib.restore_update(3, 2.0, 1.0, 0.0)
        torch.cuda.synchronize()
        from helpers import ulp
        for t, b in zip(p.theta, before):
            u = ulp(np.maximum(np.abs(b), 6e-3), dtype)
            assert np.all(np.abs(to_double(t) - b) <= 2 * u)


# ------------------------------------------------------------------------------------- norms
@pytest.mark.parametrize("bits", [32, 16])
def test_norm_bookkeeping(bits):
    # tensor-core tensors (ragged row blocks and strips included), CUDA-core, isotropic and fallback tensors
    shapes, ranks = [(64, 256), (1, 100), (40, 72), (48, 128), (300, 392), (130, 1032), (45, 100)], [8, 0, 3, 16, 32, 64, 20]
    p = Pair(shapes, ranks, "bf16", bits=bits, alpha=0.4)
    got = p.lib.get_stats(17)
    for l in range(len(shapes)):
        exp = oracle.stats_tensor(p.oracle_tensor(l), 17, l, bits, p.a, p.b)
        np.testing.assert_allclose(got[l], exp, rtol=2e-5, atol=1e-12)
    # the weights were not touched
    assert p.lib.state()[0] is False


@pytest.mark.parametrize("dtype,bits", [("bf16", 16), ("bf16", 32), ("f16", 16), ("f32", 32)])
def test_norm_bookkeeping_inside_the_sweep(dtype, bits):
    """zgr_config.stats: the first perturbation under a seed accumulates the three norms inside its sweep
    (every kernel family; ragged strips and row blocks), zgr_get_stats then only adds the partial sums up.
    The sweep itself must still match the oracle, the norms must match oracle.stats_tensor, repeated calls
    must give identical bits, and the pass of its own (bookkeeping off) must agree."""
    shapes, ranks = [(64, 256), (1, 100), (40, 72), (48, 128), (300, 392), (130, 1032), (45, 100), (1, 7)], [8, 0, 3, 16, 32, 64, 20, 0]
    p = Pair(shapes, ranks, dtype, bits=bits, alpha=0.4, stats=True, seed=13)
    seed, eps = 17, 1e-3
    launches = p.lib.launch_count()
    reports = p.call_and_check(seed, eps, lambda: p.lib.perturb(seed, eps), "perturb(+eps) with bookkeeping")
    assert all(rep["moved"] > 0.3 for rep in reports)
    swept = p.lib.launch_count() - launches
    got = p.lib.get_stats(seed)
    assert p.lib.launch_count() - launches == swept + 1          # one small finishing launch, no pass over the tensors
    for l in range(len(shapes)):
        exp = oracle.stats_tensor(p.oracle_tensor(l), seed, l, bits, p.a, p.b)
        np.testing.assert_allclose(got[l], exp, rtol=2e-5, atol=1e-12)
    assert np.array_equal(got, p.lib.get_stats(seed))             # fixed summation order
    # the rest of the step runs without bookkeeping (the seed is active) and still matches the oracle
    p.call_and_check(seed, -2 * eps, lambda: p.lib.perturb(seed, -2 * eps), "perturb(-2eps)")
    p.call_and_check(seed, eps, lambda: p.lib.restore_update(seed, 2.0, 2.0, 0.0), "restore")
    assert np.array_equal(got, p.lib.get_stats(seed))             # still held: nothing that the norms depend on has changed
    # another seed asked for: a pass of its own; and the same seed through that pass agrees with the sweep's figures
    other = p.lib.get_stats(seed + 1)
    exp = oracle.stats_tensor(p.oracle_tensor(4), seed + 1, 4, bits, p.a, p.b)
    np.testing.assert_allclose(other[4], exp, rtol=2e-5)
    p.lib.enable_stats(False)
    p.lib.set_alpha(0.4)                                          # same ratio, but the held norms are dropped
    by_pass = p.lib.get_stats(seed)
    np.testing.assert_allclose(by_pass, got, rtol=1e-5, atol=1e-12)
    assert np.array_equal(by_pass, p.lib.get_stats(seed))
    # a change of alpha drops the held norms
    p.lib.enable_stats(True)
    p.lib.perturb(seed + 2, eps); p.lib.restore_update(seed + 2, 2.0, 2.0, 0.0)
    p.lib.set_alpha(0.7)
    a2, b2 = oracle.mix_scalars(0.7, p.d, p.K, p.scale_mode)
    st = p.lib.get_stats(seed + 2)
    np.testing.assert_allclose(st[4], oracle.stats_tensor(p.oracle_tensor(4), seed + 2, 4, bits, a2, b2), rtol=2e-5)


@pytest.mark.parametrize("dtype,rows,cols,rank", [("f16", 16384, 2048, 16), ("bf16", 8192, 4096, 32), ("bf16", 6144, 1536, 64)])
def test_many_work_items_per_block(dtype, rows, cols, rank):
    """Tensors cut into ~1000 small work items, several per persistent block: the hand-over between items
    (coefficient strips rewritten while the pipeline still holds tiles of the previous item) is exercised
    hundreds of times per launch.  Every element is compared with the oracle."""
    p = Pair([(rows, cols)], [rank], dtype, bits=16, seed=21)
    reports = p.step(seed=12, lp=2.3, lm=1.8, lr=1e-4)
    for call in reports:
        assert call[0]["moved"] > 0.3 and call[0]["equal"] > 0.98, call
    seeds, coeffs = [31, 32], [1e-3, -7e-4]
    p.call_and_check_multi(seeds, coeffs, lambda: p.lib.sweep_multi(seeds, coeffs), "sweep_multi")
