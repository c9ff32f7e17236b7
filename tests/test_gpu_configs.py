"""The five configurations at full size, in the launch configuration the benchmark times.

Configurations 2-5 are too large for the oracle to replay in full, so each call of one step
(perturb +eps, perturb -2 eps, restore_update) is checked on sampled elements that the oracle
computes one by one: a fixed set of tensors (first and last of every shape, the 1-D tensors of the
first layer, embedding and head) with 20,000 random elements each.  The values before the call are
read from the device, so every call is compared from the same starting point.  The smallest
configuration is replayed in full elsewhere (test_tiny_configuration_full_cycle).
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2601_12917_b200 import synth, zgr

from helpers import ORACLE_DTYPE, check_sweep

pytestmark = pytest.mark.gpu

SAMPLES_PER_TENSOR = 20000


def _pick_tensors(wl):
    """First and last tensor of every distinct (rows, cols, rank), at most 14 tensors."""
    first, last = {}, {}
    for l, t in enumerate(wl.tensors):
        key = (t.rows, t.cols, t.rank)
        first.setdefault(key, l)
        last[key] = l
    picked = sorted(set(first.values()) | set(last.values()))
    return picked[:14]


def _gather(t: torch.Tensor, idx: torch.Tensor) -> np.ndarray:
    return t.reshape(-1)[idx].to(torch.float64).cpu().numpy()


@pytest.mark.parametrize("name", ["roberta_large", "opt_1p3b", "llama_7b", "llama_13b"])
def test_full_size_configuration_sampled_parity(name):
    wl = synth.workload(name)
    free, _ = torch.cuda.mem_get_info()
    need = wl.params * synth.DTYPE_BYTES[wl.dtype] * 1.2 + 4e9
    if free < need:
        pytest.skip(f"needs {need / 1e9:.0f} GB of free device memory")
    dm = synth.materialise(wl, "cuda", seed=5)
    z = zgr.from_device_model(dm, bits_per_normal=16)
    a, b = z.scalars()
    a_o, b_o = oracle.mix_scalars(wl.alpha, wl.params, wl.coeffs, wl.scale_mode)
    assert a == pytest.approx(a_o, rel=1e-14) and b == pytest.approx(b_o, rel=1e-14)

    picked = _pick_tensors(wl)
    samples, otens = {}, {}
    for l in picked:
        spec = wl.tensors[l]
        idx = synth.sample_indices(spec.numel, SAMPLES_PER_TENSOR, seed=l)
        samples[l] = (idx, torch.from_numpy(idx).cuda())
        U = None if dm.U[l] is None else dm.U[l].cpu().numpy()
        q = None if dm.q[l] is None else dm.q[l].cpu().numpy()
        sc = None if dm.scale[l] is None else dm.scale[l].cpu().numpy()
        otens[l] = oracle.OracleTensor(theta=np.zeros(0, dtype=np.float32), rows=spec.rows, cols=spec.cols, dtype=ORACLE_DTYPE[wl.dtype], U=U, q=q, scale=sc)

    seed = wl.seed(0, 0)
    lp, lm = wl.losses(0, 0)
    lr = wl.lr / wl.queries
    g = oracle.projected_grad(lp, lm, wl.eps)
    calls = [("perturb(+eps)", wl.eps, lambda: z.perturb(seed, wl.eps)),
             ("perturb(-2eps)", -2 * wl.eps, lambda: z.perturb(seed, -2 * wl.eps)),
             ("restore_update", wl.eps - lr * g, lambda: z.restore_update(seed, lp, lm, lr))]
    for what, c, fn in calls:
        before = {l: _gather(dm.theta[l], samples[l][1]) for l in picked}
        fn()
        assert z.device_status() == 0
        after = {l: _gather(dm.theta[l], samples[l][1]) for l in picked}
        exps = {l: oracle.sweep_elements(otens[l], before[l], seed, l, 16, a_o, b_o, c, samples[l][0]) for l in picked}
        theta_max = max(max(np.abs(before[l]).max(), np.abs(exps[l]).max()) for l in picked)
        moved = []
        for l in picked:
            spec = wl.tensors[l]
            sigma = float(np.sqrt(a_o**2 + b_o**2 * spec.rank / spec.rows))
            rep = check_sweep(after[l], exps[l], before[l], wl.dtype, theta_max, f"{name} {what} tensor {l} ({spec.name})", operand=abs(c) * sigma)
            moved.append(rep["moved"])
            if wl.dtype != "f32":
                assert rep["equal"] > 0.9, (what, spec.name, rep)
        assert min(moved) > 0.3, (what, moved)       # no tensor was skipped by the sweep
    # one pass with two seeds (zgr_sweep_multi), sampled the same way
    seeds2, coeffs2 = [wl.seed(1, 0), wl.seed(1, 1)], [wl.eps, -0.5 * wl.eps]
    before = {l: _gather(dm.theta[l], samples[l][1]) for l in picked}
    z.sweep_multi(seeds2, coeffs2)
    assert z.device_status() == 0
    after = {l: _gather(dm.theta[l], samples[l][1]) for l in picked}
    exps = {l: oracle.sweep_multi_elements(otens[l], before[l], seeds2, coeffs2, l, 16, a_o, b_o, samples[l][0]) for l in picked}
    theta_max = max(max(np.abs(before[l]).max(), np.abs(exps[l]).max()) for l in picked)
    for l in picked:
        spec = wl.tensors[l]
        sigma = float(np.sqrt(a_o**2 + b_o**2 * spec.rank / spec.rows))
        rep = check_sweep(after[l], exps[l], before[l], wl.dtype, theta_max, f"{name} sweep_multi tensor {l} ({spec.name})",
                          operand=1.5 * wl.eps * sigma)
        assert rep["moved"] > 0.3, (spec.name, rep)
    assert z.active_seeds() == 2
    z.sweep_multi(seeds2, [-c for c in coeffs2])
    # nothing outside the model was touched and the state machine is idle again
    assert z.state()[0] is False
    z.close()


@pytest.mark.parametrize("dtype,rows,cols,rank", [
    ("bf16", 34000, 131072, 16),     # tcgen05 kernel, 4.46e9 elements: element indices beyond 2^32
    ("f32", 1100, 4194304, 8),       # CUDA-core kernel, 4.61e9 elements, very long rows
    ("bf16", 1, 4400000008, 0),      # isotropic kernel on one vector of 4.4e9 elements
])
def test_tensor_with_more_than_2_pow_32_elements(dtype, rows, cols, rank):
    """Largest sizes: linear element indices, generator block indices and byte offsets all pass 2^32.
    Sampled parity of one perturbation, with the samples concentrated at the far end of the tensor."""
    tdt = {"bf16": torch.bfloat16, "f32": torch.float32}[dtype]
    numel = rows * cols
    need = numel * (2 if dtype == "bf16" else 4) * 1.1 + 2e9
    free, _ = torch.cuda.mem_get_info()
    if free < need:
        pytest.skip(f"needs {need / 1e9:.0f} GB of free device memory")
    assert numel > 2**32
    g = torch.Generator(device="cuda").manual_seed(1)
    w = torch.empty((rows, cols) if rows > 1 else (cols,), dtype=tdt, device="cuda")
    chunk = 1 << 28
    flat = w.view(-1)
    for s in range(0, numel, chunk):                                  # N(0, 0.02^2) in slabs (bounded temporaries)
        n = min(chunk, numel - s)
        flat[s:s + n] = (0.02 * torch.randn(n, generator=g, device="cuda", dtype=torch.float32)).to(tdt)
    U = None
    if rank:
        qmat, _ = torch.linalg.qr(torch.randn(rows, rank, generator=g, device="cuda", dtype=torch.float64))
        U = qmat.to(torch.float32).contiguous()
    eps = 1e-3
    z = zgr.Zgr([w], [U], 0.5, eps, zgr.SCALE_UNIT, 16)
    a_o, b_o = oracle.mix_scalars(0.5, numel, rank * cols, oracle.SCALE_UNIT)
    rng = np.random.default_rng(0)
    idx = np.unique(np.concatenate([rng.integers(0, numel, 4000), rng.integers(2**32, numel, 12000),
                                    np.arange(numel - 2048, numel), np.arange(2**32 - 1024, 2**32 + 1024)])).astype(np.int64)
    didx = torch.from_numpy(idx).cuda()
    ot = oracle.OracleTensor(theta=np.zeros(0, dtype=np.float32), rows=rows, cols=cols, dtype=ORACLE_DTYPE[dtype],
                             U=None if U is None else U.cpu().numpy())
    before = _gather(w, didx)
    z.perturb(99, eps)
    assert z.device_status() == 0
    after = _gather(w, didx)
    exp = oracle.sweep_elements(ot, before, 99, 0, 16, a_o, b_o, eps, idx)
    sigma = float(np.sqrt(a_o**2 + b_o**2 * rank / rows))
    rep = check_sweep(after, exp, before, dtype, float(max(np.abs(before).max(), np.abs(exp).max())), f"{rows}x{cols} r={rank}",
                      operand=eps * sigma)
    assert rep["moved"] > 0.3, rep
    z.restore_update(99, 2.0, 2.0, 0.0)
    z.close()
