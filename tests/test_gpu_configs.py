"""The five configurations at full size, in the launch configuration the benchmark times.

Configurations 2-5 are too large for the oracle to replay in full, so each call of one step
(perturb +eps, perturb -2 eps, restore_update) is checked on a fixed set of tensors (first and last of
every shape, the 1-D tensors of the first layer, embedding and head): every element of those with at
most 2^24 elements on the RoBERTa- and OPT-shaped sets, and 75,000 random elements of each of the others
(a million of them on the embeddings of the two smaller sets), which the oracle computes one by one:
more than 10^6 samples per call on the LLaMA-shaped sets.  The values before the call are read from the
device, so every call is compared from the same starting point.  The smallest configuration is replayed
in full elsewhere (test_tiny_configuration_full_cycle).

test_trajectory_statistic runs the whole configuration (its 10 steps of Q queries) on both sides
independently and compares the end points of the sampled elements.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2601_12917_b200 import synth, zgr

from helpers import ORACLE_DTYPE, check_sweep

pytestmark = pytest.mark.gpu

SAMPLES_PER_TENSOR = 75000
WHOLE_TENSOR_LIMIT = 1 << 24      # configurations 2-3: tensors up to this size are compared in full
BIG_TENSOR_SAMPLES = 1000000      # ... and their larger tensors (the embeddings) on this many samples


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
    small_set = name in ("roberta_large", "opt_1p3b")
    for l in picked:
        spec = wl.tensors[l]
        if small_set:
            count = spec.numel if spec.numel <= WHOLE_TENSOR_LIMIT else BIG_TENSOR_SAMPLES
        else:
            count = SAMPLES_PER_TENSOR
        idx = synth.sample_indices(spec.numel, count, seed=l)
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
            rep = check_sweep(after[l], exps[l], before[l], wl.dtype, theta_max, f"{name} {what} tensor {l} ({spec.name})", operand=abs(c) * sigma,
                              c_abs=abs(c))
            moved.append(rep["moved"])
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
                          operand=1.5 * wl.eps * sigma, c_abs=1.5 * wl.eps)
        assert rep["moved"] > 0.3, (spec.name, rep)
    assert z.active_seeds() == 2
    z.sweep_multi(seeds2, [-c for c in coeffs2])
    # nothing outside the model was touched and the state machine is idle again
    assert z.state()[0] is False
    z.close()


@pytest.mark.parametrize("name", ["opt_1p3b", "llama_7b", "llama_13b"])
def test_trajectory_statistic(name):
    """The whole configuration on both sides independently: 10 steps x Q queries x (perturb +eps, perturb -2 eps,
    restore_update with lr/Q), no re-synchronisation in between, compared at the end on sampled elements of the
    picked tensors (Eq. (perturbation), Eq. (grad), Algorithm 1 "Update").  Per call the two sides agree to one
    ulp and differ in a fraction of a percent of the roundings; over 30-120 roundings an element can collect
    several such differences, so the statement is statistical: the histogram of the end-point differences in
    ulps, at least 1 - 1e-4 of the elements within 1 ulp and none beyond 3.  The ulp is taken as in the
    per-call check, at the largest magnitude that entered the element's arithmetic (the largest |theta| the
    element had along the oracle's trajectory -- a difference of one ulp picked up in a higher binade is two
    ulps once the weight has come back down -- and the largest |c| sigma_z); the strict figures (ulp of the
    oracle's end point alone) are printed beside it."""
    wl = synth.workload(name)
    free, _ = torch.cuda.mem_get_info()
    need = wl.params * synth.DTYPE_BYTES[wl.dtype] * 1.2 + 4e9
    if free < need:
        pytest.skip(f"needs {need / 1e9:.0f} GB of free device memory")
    dm = synth.materialise(wl, "cuda", seed=6)
    z = zgr.from_device_model(dm, bits_per_normal=16)
    a_o, b_o = oracle.mix_scalars(wl.alpha, wl.params, wl.coeffs, wl.scale_mode)
    picked = _pick_tensors(wl)
    per_tensor = 20000
    idx, didx, otens, theta_o, theta_0, theta_peak = {}, {}, {}, {}, {}, {}
    for l in picked:
        spec = wl.tensors[l]
        idx[l] = synth.sample_indices(spec.numel, per_tensor, seed=100 + l)
        didx[l] = torch.from_numpy(idx[l]).cuda()
        U = None if dm.U[l] is None else dm.U[l].cpu().numpy()
        q = None if dm.q[l] is None else dm.q[l].cpu().numpy()
        sc = None if dm.scale[l] is None else dm.scale[l].cpu().numpy()
        otens[l] = oracle.OracleTensor(theta=np.zeros(0, dtype=np.float32), rows=spec.rows, cols=spec.cols, dtype=ORACLE_DTYPE[wl.dtype], U=U, q=q, scale=sc)
        theta_0[l] = _gather(dm.theta[l], didx[l])
        theta_o[l] = theta_0[l].copy()
        theta_peak[l] = np.abs(theta_0[l])
    lr = wl.lr / wl.queries
    c_max = 0.0
    n_sweeps = 0
    for t in range(wl.steps):
        for qn in range(wl.queries):
            seed = wl.seed(t, qn)
            lp, lm = wl.losses(t, qn)
            z.perturb(seed, wl.eps)
            z.perturb(seed, -2.0 * wl.eps)
            z.restore_update(seed, lp, lm, lr)
            c3 = -(wl.eps + (-2.0 * wl.eps)) - lr * oracle.projected_grad(lp, lm, wl.eps)
            for c in (wl.eps, -2.0 * wl.eps, c3):
                for l in picked:
                    theta_o[l] = oracle.sweep_elements(otens[l], theta_o[l], seed, l, 16, a_o, b_o, c, idx[l])
                    theta_peak[l] = np.maximum(theta_peak[l], np.abs(theta_o[l]))
                c_max = max(c_max, abs(c))
                n_sweeps += 1
    assert z.device_status() == 0 and z.state()[0] is False
    assert n_sweeps == 3 * wl.queries * wl.steps
    from helpers import ulp
    hist = np.zeros(6, dtype=np.int64)
    hist_strict = np.zeros(6, dtype=np.int64)
    total, worst, worst_strict, moved = 0, 0.0, 0.0, 0
    for l in picked:
        spec = wl.tensors[l]
        got = _gather(dm.theta[l], didx[l])
        exp = theta_o[l]
        sigma = float(np.sqrt(a_o**2 + b_o**2 * spec.rank / spec.rows))
        u = ulp(np.maximum(theta_peak[l], c_max * sigma), wl.dtype)
        d = np.abs(got - exp) / u
        ds = np.abs(got - exp) / ulp(exp, wl.dtype)
        hist += np.bincount(np.minimum(np.ceil(d - 1e-9).astype(np.int64), 5), minlength=6)
        hist_strict += np.bincount(np.minimum(np.ceil(ds - 1e-9).astype(np.int64), 5), minlength=6)
        total += got.size
        worst, worst_strict = max(worst, float(d.max())), max(worst_strict, float(ds.max()))
        moved += int(np.sum(exp != theta_0[l]))
    print(f"trajectory {name}: {n_sweeps} sweeps, {total} sampled elements, {moved / total:.3f} moved; "
          f"ulp differences 0/1/2/3/4/5+ = {hist.tolist()} (worst {worst:.2f}); strict (ulp of the oracle's end point) = "
          f"{hist_strict.tolist()} (worst {worst_strict:.2f})")
    assert moved > 0.9 * total
    assert (hist[0] + hist[1]) >= (1.0 - 1e-4) * total, hist.tolist()
    assert worst <= 3.0, worst
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
