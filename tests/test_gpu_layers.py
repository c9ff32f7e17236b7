"""Layer-wise perturbation with the compressed coefficients arriving from the host while earlier layers are swept
(zgr_perturb_layers; Sec. 3.3, the layer-wise sample -> transmit -> apply pipeline) and a proportion of the
coefficients compressed (zgr_set_coeffs_dtc_rows; Sec. 3.4, the adaptive proportion omega).  Needs a B200.

The oracle sweeps with the same mixed coefficient source; the device result must also be identical, bit for
bit, to copying every payload first and calling zgr_perturb."""
import numpy as np
import pytest
import torch

import oracle
from paper_2601_12917_b200 import synth, zgr

from helpers import Pair

pytestmark = pytest.mark.gpu

# three "layers": (matrix r=32, vector, matrix r=16) (matrix r=64, matrix r=8) (vector, matrix r=32)
SHAPES = [(300, 392), (1, 100), (150, 1032), (130, 520), (70, 264), (1, 64), (256, 512)]
RANKS = [32, 0, 16, 64, 8, 0, 32]
LAYER_END = [3, 5, 7]


def _payloads(ranks, shapes, omega, bits, seed):
    """Per guided tensor: (codes, scales, zeros or None, n_rows) for the first ceil(omega r) rows."""
    out = {}
    for l, ((m, n), r) in enumerate(zip(shapes, ranks)):
        if r == 0:
            continue
        n_rows = max(1, int(np.ceil(omega * r)))
        if bits == 8:
            q, sc = synth.dtc_payload(r, n, seed=seed + l)
            ze = None
        else:
            q, sc, ze = oracle.dtc_quantise_int4(oracle.coeffs(seed + l, l, 16, r, n))
        out[l] = (q, sc, ze, n_rows)
    return out


@pytest.mark.parametrize("dtype", ["bf16", "f16"])
@pytest.mark.parametrize("omega,bits", [(1.0, 8), (0.5, 8), (0.3, 4)])
def test_layerwise_delivery_matches_the_oracle_and_the_plain_sweep(omega, bits, dtype):
    pay = _payloads(RANKS, SHAPES, omega, bits, seed=40)
    pay2 = _payloads(RANKS, SHAPES, omega, bits, seed=90)       # what "arrives" in the pipelined call
    a = Pair(SHAPES, RANKS, dtype, bits=16, seed=7)
    b = Pair(SHAPES, RANKS, dtype, bits=16, seed=7)
    for p in (a, b):
        for l, (q, sc, ze, n_rows) in pay.items():             # register device buffers holding the first payload
            p.set_dtc(l, q, sc, ze, bits=bits, n_rows=None if n_rows == RANKS[l] else n_rows)
    # A: the pipelined call delivers the second payload layer by layer on a copy stream
    copy_stream = torch.cuda.Stream()
    deliveries = []
    for l, (q, sc, ze, n_rows) in pay2.items():
        hq = torch.from_numpy(np.ascontiguousarray(q[:n_rows]) if bits == 8 else oracle.dtc_pack4(q[:n_rows])).pin_memory()
        deliveries.append((l, hq, torch.from_numpy(np.ascontiguousarray(sc[:n_rows])).pin_memory(),
                           None if ze is None else torch.from_numpy(np.ascontiguousarray(ze[:n_rows])).pin_memory()))
    seed, eps = 11, 1e-3

    def pipelined():
        a.lib.perturb_layers(seed, eps, LAYER_END, deliveries, copy_stream=copy_stream)
        # the oracle sees the payload that arrived
        for l, (q, sc, ze, n_rows) in pay2.items():
            a.q[l] = torch.from_numpy(np.ascontiguousarray(q[:n_rows]))
            a.scale[l] = torch.from_numpy(np.ascontiguousarray(sc[:n_rows]))
            a.zero[l] = None if ze is None else torch.from_numpy(np.ascontiguousarray(ze[:n_rows]))

    # the oracle must start from theta before the call but use the delivered coefficients: take theta first
    ots_before = [a.oracle_tensor(l) for l in range(len(SHAPES))]
    pipelined()
    torch.cuda.synchronize()
    assert a.lib.device_status() == 0
    from helpers import check_sweep, to_double
    for l, t in enumerate(ots_before):
        before = oracle.decode(t.theta, t.dtype)
        t2 = a.oracle_tensor(l)                      # delivered coefficients ...
        t2.theta = t.theta                           # ... applied to the weights as they were
        oracle.sweep_tensor(t2, seed, l, 16, a.a, a.b, eps)
        exp = oracle.decode(t2.theta, t2.dtype)
        rep = check_sweep(to_double(a.theta[l]), exp, before, dtype, 1.0, f"perturb_layers tensor {l}", operand=eps * a.sigma_z(l), c_abs=eps)
        assert rep["moved"] > 0.3
    # B: copy everything first, then the plain call
    for l, (q, sc, ze, n_rows) in pay2.items():
        b.payload[l].copy_(deliveries[[d[0] for d in deliveries].index(l)][1])
        b.scale[l].copy_(torch.from_numpy(np.ascontiguousarray(sc[:n_rows])))
        if ze is not None:
            b.zero[l].copy_(torch.from_numpy(np.ascontiguousarray(ze[:n_rows])))
    b.lib.perturb(seed, eps)
    torch.cuda.synchronize()
    for l in range(len(SHAPES)):
        assert torch.equal(a.theta[l], b.theta[l]), f"tensor {l}"
    # the rest of the step on the delivered coefficients, then idle
    a.call_and_check(seed, -2 * eps, lambda: a.lib.perturb_layers(seed, -2 * eps, LAYER_END), "perturb_layers(-2eps)")
    a.call_and_check(seed, eps - 1e-4 * oracle.projected_grad(2.2, 1.9, eps), lambda: a.lib.restore_update(seed, 2.2, 1.9, 1e-4), "restore_update")
    assert a.lib.state()[0] is False


def test_layerwise_delivery_of_subspaces():
    """The subspaces themselves can travel the same way: a delivered U is copied into the tensor's subspace
    buffer and split for the tensor cores before its layer is swept."""
    a = Pair(SHAPES, RANKS, "bf16", bits=16, seed=3, stats=True)
    new_U = {l: torch.from_numpy(synth.subspace(SHAPES[l][0], RANKS[l], 900 + l)).pin_memory() for l in range(len(SHAPES)) if RANKS[l]}
    copy_stream = torch.cuda.Stream()
    deliveries = [(l, None, None, None, U) for l, U in new_U.items()]
    seed, eps = 21, 1e-3
    ots = [a.oracle_tensor(l) for l in range(len(SHAPES))]
    a.lib.perturb_layers(seed, eps, LAYER_END, deliveries, copy_stream=copy_stream)
    torch.cuda.synchronize()
    assert a.lib.device_status() == 0
    from helpers import check_sweep, to_double
    for l, t in enumerate(ots):
        assert RANKS[l] == 0 or torch.equal(a.U[l].cpu(), new_U[l])          # the subspace buffer holds what arrived
        before = oracle.decode(t.theta, t.dtype)
        t2 = a.oracle_tensor(l)
        t2.theta = t.theta
        oracle.sweep_tensor(t2, seed, l, 16, a.a, a.b, eps)
        rep = check_sweep(to_double(a.theta[l]), oracle.decode(t2.theta, t2.dtype), before, "bf16", 1.0, f"perturb_layers(U) tensor {l}",
                          operand=eps * a.sigma_z(l), c_abs=eps)
        assert rep["moved"] > 0.3
    # the norms kept by that layer-wise sweep are those of the delivered subspaces
    st = a.lib.get_stats(seed)
    for l in range(len(SHAPES)):
        np.testing.assert_allclose(st[l], oracle.stats_tensor(a.oracle_tensor(l), seed, l, 16, a.a, a.b), rtol=2e-5, atol=1e-12)
    a.call_and_check(seed, -2 * eps, lambda: a.lib.perturb(seed, -2 * eps), "perturb(-2eps)")
    a.call_and_check(seed, eps, lambda: a.lib.restore_update(seed, 2.0, 2.0, 0.0), "restore")
    with pytest.raises(zgr.ZgrError) as e:                      # a subspace for a vector
        a.lib.perturb_layers(5, eps, LAYER_END, [(1, None, None, None, new_U[0])], copy_stream=copy_stream)
    assert e.value.code == zgr.EINVAL
    with pytest.raises(zgr.ZgrError) as e:                      # a delivery that carries nothing
        a.lib.perturb_layers(5, eps, LAYER_END, [(0, None, None, None, None)], copy_stream=copy_stream)
    assert e.value.code == zgr.EINVAL


def test_layer_table_and_delivery_errors():
    p = Pair(SHAPES[:3], RANKS[:3], "bf16", bits=16)
    q, sc = synth.dtc_payload(32, 392, seed=1)
    p.set_dtc(0, q, sc)
    hq, hs = torch.from_numpy(q).pin_memory(), torch.from_numpy(sc).pin_memory()
    cs = torch.cuda.Stream()
    for bad in ([2, 2, 3], [3, 2], [1, 2], [1, 4]):
        with pytest.raises(zgr.ZgrError) as e:
            p.lib.perturb_layers(1, 1e-3, bad, copy_stream=cs)
        assert e.value.code == zgr.EINVAL
    with pytest.raises(zgr.ZgrError) as e:                      # tensor 2 has no compressed coefficients registered
        p.lib.perturb_layers(1, 1e-3, [1, 3], [(2, hq, hs, None)], copy_stream=cs)
    assert e.value.code == zgr.EINVAL
    with pytest.raises(zgr.ZgrError) as e:                      # the same tensor twice
        p.lib.perturb_layers(1, 1e-3, [1, 3], [(0, hq, hs, None), (0, hq, hs, None)], copy_stream=cs)
    assert e.value.code == zgr.EINVAL
    with pytest.raises(zgr.ZgrError) as e:
        p.lib.set_coeffs_dtc_rows(0, p.payload[0], p.scale[0], None, 8, 33)
    assert e.value.code == zgr.EINVAL
    p.lib.perturb_layers(1, 1e-3, [1, 3], [(0, hq, hs, None)], copy_stream=cs)
    with pytest.raises(zgr.ZgrError) as e:                      # no delivery while a perturbation is active
        p.lib.perturb_layers(1, -2e-3, [1, 3], [(0, hq, hs, None)], copy_stream=cs)
    assert e.value.code == zgr.ESTATE
    p.lib.perturb_layers(1, -2e-3, [1, 3], copy_stream=cs)
    p.lib.restore_update(1, 2.0, 2.0, 0.0)
    assert p.lib.state()[0] is False


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_layerwise_sweeps_of_low_rank_tensors_on_both_streams(dtype):
    """Every layer holds tensors of rank <= 8, so consecutive layers run the CUDA-core contraction kernel on the two
    alternating streams at the same time; that kernel hands its work items out through a counter per stream, which
    each launch must leave at zero for the next one.  Many layers of different sizes, layer-wise and whole-model
    sweeps in turn, every call against the oracle and against a context that only ever sweeps the whole model."""
    shapes, ranks, ends = [], [], []
    for L in range(9):
        shapes += [(96 + 40 * L, 264 + 256 * (L % 3)), (1, 72 + 8 * L), (64 + 8 * L, 520)]
        ranks += [8, 0, 4 if L % 2 else 6]
        ends.append(len(shapes))
    a = Pair(shapes, ranks, dtype, bits=16, seed=12)
    b = Pair(shapes, ranks, dtype, bits=16, seed=12)
    eps = 1e-3
    for step, seed in enumerate((5, 6, 7)):
        a.call_and_check(seed, eps, lambda: a.lib.perturb_layers(seed, eps, ends), f"perturb_layers(+eps) step {step}")
        b.lib.perturb(seed, eps)
        if step == 1:
            a.call_and_check(seed, -2 * eps, lambda: a.lib.perturb(seed, -2 * eps), f"perturb(-2eps) step {step}")
        else:
            a.call_and_check(seed, -2 * eps, lambda: a.lib.perturb_layers(seed, -2 * eps, ends), f"perturb_layers(-2eps) step {step}")
        b.lib.perturb(seed, -2 * eps)
        c = eps - 1e-4 * oracle.projected_grad(2.3, 1.8, eps)
        a.call_and_check(seed, c, lambda: a.lib.restore_update(seed, 2.3, 1.8, 1e-4), f"restore_update step {step}")
        b.lib.restore_update(seed, 2.3, 1.8, 1e-4)
        torch.cuda.synchronize()
        for l in range(len(shapes)):
            assert torch.equal(a.theta[l], b.theta[l]), f"step {step} tensor {l}"
    assert a.lib.device_status() == 0 and a.lib.state()[0] is False
