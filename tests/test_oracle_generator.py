"""Pins of the oracle's counter-based generator and Gaussian transform (CPU only).

The paper says only that client and edge server regenerate the same perturbation from a shared
seed (Algorithm 1, "Regenerate identical z_h via seed s"); the generator is Philox4x32-10 and is
pinned here against two independent library implementations of it, not against itself:
  * cuRAND's host generator (CURAND_RNG_PSEUDO_PHILOX4_32_10), whose default ordering emits block i
    as the output for counter (0, 0, i, 0) under key = seed;
  * Triton's ``tl.philox`` run through the Triton CPU interpreter, which takes all four counter
    words and the 64-bit seed.
The normal stream is pinned by exact uniforms, moments, a Kolmogorov-Smirnov test and its tail bound.
"""
import ctypes
import math
import os

import numpy as np
import pytest

import oracle


# ----------------------------------------------------------------------------------------- cuRAND
def _curand_blocks(seed: int, n_blocks: int) -> np.ndarray:
    path = None
    for cand in ("/usr/local/cuda/lib64/libcurand.so", "libcurand.so", "libcurand.so.10"):
        try:
            lib = ctypes.CDLL(cand)
            path = cand
            break
        except OSError:
            continue
    if path is None:
        pytest.skip("libcurand not found")
    gen = ctypes.c_void_p()
    if lib.curandCreateGeneratorHost(ctypes.byref(gen), 161) != 0:  # CURAND_RNG_PSEUDO_PHILOX4_32_10
        pytest.skip("cuRAND host generator unavailable")
    assert lib.curandSetPseudoRandomGeneratorSeed(gen, ctypes.c_ulonglong(seed)) == 0
    out = np.zeros(4 * n_blocks, dtype=np.uint32)
    assert lib.curandGenerate(gen, out.ctypes.data_as(ctypes.c_void_p), ctypes.c_size_t(out.size)) == 0
    lib.curandDestroyGenerator(gen)
    return out.reshape(n_blocks, 4)


@pytest.mark.parametrize("seed", [0, 1, 0xDEADBEEF, 0x0123456789ABCDEF, 2**64 - 1])
def test_philox_matches_curand_host(seed):
    n = 64
    ref = _curand_blocks(seed, n)
    # cuRAND block i <-> counter (0, 0, i, 0): in the oracle's layout that is block 0 of tensor i, tag 0.
    got = np.stack([oracle.blocks(seed, tensor=i, tag=0, first_block=0, n_blocks=1)[0] for i in range(n)])
    np.testing.assert_array_equal(got, ref)


# ----------------------------------------------------------------------------------------- Triton
def _triton_philox(seed, counters):
    os.environ["TRITON_INTERPRET"] = "1"
    try:
        import torch
        import triton
        import triton.language as tl
    except Exception as exc:  # pragma: no cover
        pytest.skip(f"triton interpreter unavailable: {exc}")

    @triton.jit
    def kern(out, ctr, seed, n, BLOCK: tl.constexpr):
        i = tl.arange(0, BLOCK)
        m = i < n
        c0 = tl.load(ctr + 4 * i + 0, mask=m, other=0)
        c1 = tl.load(ctr + 4 * i + 1, mask=m, other=0)
        c2 = tl.load(ctr + 4 * i + 2, mask=m, other=0)
        c3 = tl.load(ctr + 4 * i + 3, mask=m, other=0)
        a, b, c, d = tl.philox(seed, c0, c1, c2, c3)
        tl.store(out + 4 * i + 0, a, mask=m)
        tl.store(out + 4 * i + 1, b, mask=m)
        tl.store(out + 4 * i + 2, c, mask=m)
        tl.store(out + 4 * i + 3, d, mask=m)

    ctr = torch.from_numpy(np.asarray(counters, dtype=np.uint32).view(np.int32).copy())
    n = ctr.shape[0]
    out = torch.zeros((n, 4), dtype=torch.int32)
    # tl.philox takes the seed as a 64-bit integer; pass it as a signed value of the same bits
    s = seed if seed < 2**63 else seed - 2**64
    try:
        kern[(1,)](out, ctr, s, n, BLOCK=64)
    except Exception as exc:  # pragma: no cover
        pytest.skip(f"triton interpreter failed: {exc}")
    return out.numpy().view(np.uint32)


@pytest.mark.parametrize("seed", [0, 12345, 0xFEDCBA9876543210])
def test_philox_matches_triton_all_counter_words(seed):
    rng = np.random.default_rng(5)
    counters = rng.integers(0, 2**32, size=(48, 4), dtype=np.uint64).astype(np.uint32)
    counters[0] = 0
    counters[1] = 0xFFFFFFFF
    counters[2] = [0xFFFFFFFF, 0, 0, 0]      # low block word saturated
    counters[3] = [0, 1, 0, 0]               # block index 2^32
    ref = _triton_philox(seed, counters)
    key = [seed & 0xFFFFFFFF, seed >> 32]
    got = np.stack([oracle.philox4x32_10(c, key) for c in counters])
    np.testing.assert_array_equal(got, ref)
    # and through the stream layout (block lo, block hi, tensor, tag)
    for c in counters[:8]:
        j = int(c[0]) | (int(c[1]) << 32)
        blk = oracle.blocks(seed, tensor=int(c[2]), tag=int(c[3]), first_block=j, n_blocks=1)[0]
        np.testing.assert_array_equal(blk, oracle.philox4x32_10(c, key))


def test_stream_layout_and_block_carry():
    # consecutive blocks across the 2^32 boundary continue into the high counter word
    j0 = 2**32 - 2
    got = oracle.blocks(9, 3, 1, j0, 4)
    for i in range(4):
        j = j0 + i
        np.testing.assert_array_equal(got[i], oracle.philox4x32_10([j & 0xFFFFFFFF, j >> 32, 3, 1], [9, 0]))
    # distinct (block, tensor, tag, seed) give distinct blocks (the round function is a bijection
    # of the counter for a fixed key)
    seen = set()
    for seed in (0, 1):
        for tensor in range(4):
            for tag in range(2):
                for b in oracle.blocks(seed, tensor, tag, 0, 64):
                    seen.add(tuple(int(x) for x in b))
    assert len(seen) == 2 * 4 * 2 * 64


# ----------------------------------------------------------------------------------------- normals
def _expected_normals_from_block(x, bits):
    """Box-Muller of the block words, restated independently with Python's math module."""
    out = []
    if bits == 32:
        for p in range(2):
            u1 = (2 * (int(x[2 * p]) & 0x7FFFFF) + 1) / 2.0**24
            u2 = (2 * (int(x[2 * p + 1]) & 0x7FFFFF) + 1) / 2.0**24
            rho = math.sqrt(-2.0 * math.log(u1))
            out += [rho * math.cos(2 * math.pi * u2), rho * math.sin(2 * math.pi * u2)]
    else:
        for w in range(4):
            xw = int(x[w])
            k1 = (xw >> 7) & 0xFFFF                      # bits 7..22
            k2 = (xw >> 23) | ((xw & 0x7F) << 9)         # bits 23..31 (low) and 0..6 (high)
            u1 = (2 * k1 + 1) / 2.0**17
            u2 = (2 * k2 + 1) / 2.0**17
            rho = math.sqrt(-2.0 * math.log(u1))
            out += [rho * math.cos(2 * math.pi * u2), rho * math.sin(2 * math.pi * u2)]
    return np.array(out)


@pytest.mark.parametrize("bits", [32, 16])
def test_normals_index_to_block_mapping(bits):
    per = 4 if bits == 32 else 8
    seed, tensor, tag = 77, 5, 1
    e0 = 3 * per + 1  # start inside a block
    got = oracle.normals(seed, tensor, tag, bits, e0, 5 * per)
    for i, e in enumerate(range(e0, e0 + 5 * per)):
        blk = oracle.blocks(seed, tensor, tag, e // per, 1)[0]
        exp = _expected_normals_from_block(blk, bits)[e % per]
        assert abs(got[i] - exp) <= 1e-13


@pytest.mark.parametrize("bits", [32, 16])
def test_normals_moments_ks_and_tail(bits):
    from scipy import stats
    n = 1 << 22
    z = oracle.normals(2024, 0, 0, bits, 0, n)
    # 4-sigma bands of the sample moments of N(0,1): var(z)=1, var(z^2)=2, var(z^4)=96
    assert abs(z.mean()) < 4 / math.sqrt(n)
    assert abs((z**2).mean() - 1) < 4 * math.sqrt(2 / n)
    assert abs((z**4).mean() - 3) < 4 * math.sqrt(96 / n) + (0.02 if bits == 16 else 0.0)
    assert abs((z**3).mean()) < 4 * math.sqrt(15 / n)
    # tail bound from the smallest uniform: |z| <= sqrt(-2 ln 2^-(b+1))
    nb = 23 if bits == 32 else 16
    assert np.abs(z).max() <= math.sqrt(2 * (nb + 1) * math.log(2)) + 1e-12
    # KS against the normal CDF on a subsample
    ks = stats.kstest(z[: 1 << 18], "norm")
    assert ks.pvalue > 1e-3
    # the two outputs of a pair and neighbouring pairs are uncorrelated
    assert abs(np.mean(z[0::2] * z[1::2])) < 4 / math.sqrt(n / 2)
    assert abs(np.mean(z[1:-1:2] * z[2::2])) < 4 / math.sqrt(n / 2)


def test_streams_are_independent_across_tensor_tag_seed():
    n = 1 << 18
    base = oracle.normals(1, 0, 0, 32, 0, n)
    for other in (oracle.normals(2, 0, 0, 32, 0, n), oracle.normals(1, 1, 0, 32, 0, n), oracle.normals(1, 0, 1, 32, 0, n)):
        assert abs(np.mean(base * other)) < 5 / math.sqrt(n)
        assert not np.array_equal(base, other)
    # same arguments, same bits (determinism) and random access == bulk
    np.testing.assert_array_equal(base[1000:1010], oracle.normals(1, 0, 0, 32, 1000, 10))
