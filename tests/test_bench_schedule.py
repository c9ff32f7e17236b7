"""bench.py's two step schedules drive the same update (CPU only): run through an adapter that forwards the
library calls to the oracle in double storage, the 3Q-sweep step and the 2Q+1-sweep step must end at the same
weights, and the deferred one must issue exactly 2Q+1 passes and leave no seed active."""
import numpy as np

import bench
import oracle
from paper_2601_12917_b200 import synth


class _OracleBackedZgr:
    """The calls bench.run_step makes on a Zgr context, answered by the oracle."""

    def __init__(self, o):
        self.o, self.passes = o, 0

    def perturb(self, seed, scale):
        self.o.sweep_multi([seed], [scale]); self.passes += 1

    def restore_update(self, seed, lp, lm, lr):
        self.o.restore_update_multi([seed], [lp], [lm], lr); self.passes += 1

    def sweep_multi(self, seeds, coeffs):
        self.o.sweep_multi(seeds, coeffs); self.passes += 1

    def restore_update_multi(self, seeds, lps, lms, lr):
        self.o.restore_update_multi(seeds, lps, lms, lr); self.passes += 1


class _Workload:
    queries, eps, lr = 4, 1e-3, 1e-2

    def seed(self, t, q):
        return 1000 * t + q

    def losses(self, t, q):
        rng = np.random.default_rng(100 * t + q)
        return float(rng.uniform(1.5, 2.5)), float(rng.uniform(1.5, 2.5))


def _model():
    tensors = []
    for l, ((m, n), r) in enumerate(zip(((24, 16), (1, 12), (16, 24)), (4, 0, 2))):
        U = synth.subspace(m, r, l) if r else None
        w = synth.weights_host(synth.TensorSpec(f"t{l}", m, n, r), l).ravel()
        tensors.append(oracle.OracleTensor(theta=oracle.encode(w, oracle.F64), rows=m, cols=n, dtype=oracle.F64, U=U))
    return tensors


def test_sequential_and_deferred_schedules_agree():
    wl = _Workload()
    results, passes = [], []
    for schedule in ("sequential", "deferred"):
        tensors = _model()
        z = _OracleBackedZgr(oracle.OracleZGR(tensors, alpha=0.5, eps=wl.eps, bits=16))
        for t in range(2):
            bench.run_step(z, wl, t, schedule)
        assert z.o.nets == {}
        results.append(np.concatenate([oracle.decode(t_.theta, t_.dtype).ravel() for t_ in tensors]))
        passes.append(z.passes)
    assert passes == [2 * 3 * wl.queries, 2 * (2 * wl.queries + 1)]
    np.testing.assert_allclose(results[1], results[0], rtol=0, atol=1e-14)
    assert np.abs(results[0]).max() > 0


def test_layer_table_covers_every_tensor_once():
    """The layer table that bench.py hands to zgr_perturb_layers: strictly increasing, ends at the number of
    tensors, one layer for what precedes the blocks, one per Transformer block, one for what follows them."""
    expected_layers = {"roberta_large": 25, "opt_1p3b": 26, "llama_7b": 34, "llama_13b": 42}
    for name, n_layers in expected_layers.items():
        wl = synth.workload(name)
        ends = bench.layer_table(wl)
        assert len(ends) == n_layers and ends[-1] == len(wl.tensors)
        assert all(b > a for a, b in zip([0] + ends[:-1], ends))
        # a block's tensors share their name prefix, and no prefix is split over two layers
        start = 0
        seen = set()
        for end in ends:
            prefixes = {t.name.split(".")[0] for t in wl.tensors[start:end]}
            blocks = {p for p in prefixes if p.startswith("l") and p[1:].isdigit()}
            assert len(blocks) <= 1 and (not blocks or prefixes == blocks)
            assert not (prefixes & seen)
            seen |= prefixes
            start = end
