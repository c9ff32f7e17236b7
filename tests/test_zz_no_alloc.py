"""The allocation-free norms entry point (zgr_tensor_norms_noalloc) against the oracle and against zgr_get_stats.

Some users of the library cannot let it allocate device memory while they run -- an allocation
forces a device-wide synchronisation that stalls their other streams, or their framework has
already taken all free device memory for its own pool.  For them the library keeps the scratch of
this one entry point in a fixed array of its own image.  The test calls it through the C ABI twice in
a row (the array keeps the previous call's contents, so the second call must not be disturbed by
the first) and compares with the oracle's norms and with the allocating entry point, within the tolerance
of the other norm tests.

Collected last on purpose: a run that stops at the first failure has then already run everything else.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2601_12917_b200 import zgr

from helpers import Pair

pytestmark = pytest.mark.gpu


def test_noalloc_norms_match_get_stats_twice_in_a_row():
    shapes, ranks = [(1500, 200), (1, 300), (2100, 72)], [8, 0, 20]
    p = Pair(shapes, ranks, "bf16", alpha=0.4, bits=32)
    out = torch.full((3,), -1.0, dtype=torch.float64, device="cuda")
    for seed in (17, 18):                       # two calls in a row, different seeds
        ref = p.lib.get_stats(seed)             # the existing entry point (allocates on first use)
        for l in range(len(shapes)):
            p.lib.tensor_norms_noalloc(seed, l, out)
            torch.cuda.synchronize()
            got = out.cpu().numpy()
            np.testing.assert_allclose(got, ref[l], rtol=2e-5, atol=1e-12)
            # and against the oracle itself, so that a mistake shared by the two device routes cannot pass
            np.testing.assert_allclose(got, oracle.stats_tensor(p.oracle_tensor(l), seed, l, 32, p.a, p.b), rtol=2e-5, atol=1e-12)
            # fixed summation order: a repeat gives the same bits
            out2 = torch.empty_like(out)
            p.lib.tensor_norms_noalloc(seed, l, out2)
            torch.cuda.synchronize()
            assert torch.equal(out, out2)
    # a smaller tensor after a larger one: stale partial sums of the larger call must not leak in
    p.lib.tensor_norms_noalloc(18, 1, out)
    torch.cuda.synchronize()
    np.testing.assert_allclose(out.cpu().numpy(), p.lib.get_stats(18)[1], rtol=2e-5, atol=1e-12)


def test_noalloc_rejects_oversized_and_bad_arguments():
    # 8193 strips of 64 columns x 1 row tile: one tile more than the fixed scratch holds
    big = torch.zeros(1, 64 * zgr.NOALLOC_MAX_TILES + 8, dtype=torch.bfloat16, device="cuda")
    ok = torch.zeros(1, 64 * zgr.NOALLOC_MAX_TILES, dtype=torch.bfloat16, device="cuda")
    z = zgr.Zgr([big, ok], [None, None], 0.5, 1e-3)
    out = torch.zeros(3, dtype=torch.float64, device="cuda")
    with pytest.raises(zgr.ZgrError) as e:
        z.tensor_norms_noalloc(1, 0, out)
    assert e.value.code == zgr.ETOOBIG and "scratch" in str(e.value)
    z.tensor_norms_noalloc(1, 1, out)           # exactly at the limit is accepted
    torch.cuda.synchronize()
    assert out[0].item() == pytest.approx(0.5 * ok.numel(), rel=0.01)     # sum (a Z)^2 with a^2 = alpha
    L = zgr.lib()
    assert L.zgr_tensor_norms_noalloc(z._h, 1, 5, out.data_ptr(), None) == zgr.EINVAL
    assert L.zgr_tensor_norms_noalloc(z._h, 1, 0, None, None) == zgr.EINVAL
    assert L.zgr_tensor_norms_noalloc(None, 1, 0, out.data_ptr(), None) == zgr.EINVAL
