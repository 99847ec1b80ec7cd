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
    finally:
        g.close()
