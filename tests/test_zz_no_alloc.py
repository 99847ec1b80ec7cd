"""The allocation-free ring product must give exactly what the allocating one gives.

Collected last on purpose (file name): if it fails, a run that stops at the first failure has
already been through every other test.  It also has to pass on its own in a fresh process, where
its first call is the one that resolves the scratch array's device address.
"""
import numpy as np
import pytest

from oracle import ckks
from tests.helpers import GpuSide, oracle_params

pytestmark = pytest.mark.gpu


def test_noalloc_product_equals_allocating_product_twice_in_a_row():
    par = oracle_params("n12")
    g = GpuSide(par, ckks.Plan(64, 1, 8, 8))
    try:
        bf = g.bf
        nb = par.r + 1
        N = par.N
        rng = np.random.default_rng(42)
        # two different batch sizes back to back: the second call finds the first call's leftovers in
        # the shared array, including in the region it has to clear for its padding polynomials
        for n_polys in (2 * nb + 3, nb + 1):
            moduli = [par.basis[t % nb] for t in range(n_polys)]
            a = np.stack([rng.integers(0, q, size=N, dtype=np.uint64) for q in moduli])
            b = np.stack([rng.integers(0, q, size=N, dtype=np.uint64) for q in moduli])
            da, db = g.to_dev(a), g.to_dev(b)
            ref = g.empty_u64(n_polys, N)
            out = g.empty_u64(n_polys, N)
            bf.bf_negacyclic_mul(g.ctx, da, db, ref, n_polys)
            bf.bf_negacyclic_mul_noalloc(g.ctx, da, db, out, n_polys)
            got, want = g.to_host_u64(out), g.to_host_u64(ref)
            assert np.array_equal(got, want)          # integer work: bit for bit
            assert np.array_equal(want, ckks.ring_mul(a, b, moduli, par))
        # beyond the fixed capacity: refused with its own error code, nothing enqueued
        too_many = bf.bf_noalloc_max_words() // N + nb
        big = g.empty_u64(too_many, N)
        with pytest.raises(bf.BifrostError) as ei:
            bf.bf_negacyclic_mul_noalloc(g.ctx, big, big, big, too_many)
        assert ei.value.code == bf.BF_ERR_TOO_LARGE
        # a count so large that rounding it up to whole groups of r + 1 would wrap 32 bits is refused the same way
        with pytest.raises(bf.BifrostError) as ei:
            bf.bf_negacyclic_mul_noalloc(g.ctx, big, big, big, 0xFFFFFFFF)
        assert ei.value.code == bf.BF_ERR_TOO_LARGE
    finally:
        g.close()


def test_noalloc_product_at_the_largest_ring_that_fits():
    # N = 2^15 with seven ciphertext primes: one group of r + 1 = 8 polynomials is 2^18 words, half of the fixed
    # array (two groups fill it exactly); the N = 2^16 chain (10 x 65536 words per group) can never fit
    par = oracle_params("n15")
    g = GpuSide(par, ckks.Plan(1024, 16, 16, 4))
    try:
        bf = g.bf
        nb, N = par.r + 1, par.N
        rng = np.random.default_rng(43)
        for n_polys in (nb, 2 * nb - 3):
            moduli = [par.basis[t % nb] for t in range(n_polys)]
            a = np.stack([rng.integers(0, q, size=N, dtype=np.uint64) for q in moduli])
            b = np.stack([rng.integers(0, q, size=N, dtype=np.uint64) for q in moduli])
            da, db = g.to_dev(a), g.to_dev(b)
            ref, out = g.empty_u64(n_polys, N), g.empty_u64(n_polys, N)
            bf.bf_negacyclic_mul(g.ctx, da, db, ref, n_polys)
            bf.bf_negacyclic_mul_noalloc(g.ctx, da, db, out, n_polys)
            assert np.array_equal(g.to_host_u64(out), g.to_host_u64(ref))
            assert np.array_equal(g.to_host_u64(out), ckks.ring_mul(a, b, moduli, par))
        with pytest.raises(bf.BifrostError) as ei:
            bf.bf_negacyclic_mul_noalloc(g.ctx, da, db, out, 2 * nb + 1)
        assert ei.value.code == bf.BF_ERR_TOO_LARGE
    finally:
        g.close()

    par16 = oracle_params("n16")
    g = GpuSide(par16, ckks.Plan(1024, 32, 8, 4))
    try:
        one = g.empty_u64(1, par16.N)
        with pytest.raises(g.bf.BifrostError) as ei:      # even one polynomial pads to a group of 10 x 2^16 words
            g.bf.bf_negacyclic_mul_noalloc(g.ctx, one, one, one, 1)
        assert ei.value.code == g.bf.BF_ERR_TOO_LARGE
    finally:
        g.close()
