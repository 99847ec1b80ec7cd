"""Pins for the oracle's ring arithmetic: primes, NTT, negacyclic product, automorphism.

Every expected value here comes from Python big-integer arithmetic written out from the plain
definition, or from the golden prime table; none comes from the routine under test.
"""
import os
import random

import numpy as np
import pytest

from oracle import ckks

GOLD = os.path.join(os.path.dirname(__file__), "golden", "primes.txt")


def _fermat_probable_prime(n):
    return all(pow(a, n - 1, n) == 1 for a in (2, 3, 5, 7, 11))


def test_prime_chains_match_golden_table_and_rule():
    rows = [l.split() for l in open(GOLD) if l.strip() and not l.startswith("#")]
    table = {}
    for N, bits, p in rows:
        table.setdefault((int(N), int(bits)), []).append(int(p))
    for (N, bits), plist in table.items():
        assert ckks.find_primes(1 << bits, 2 * N, len(plist)) == plist
        # independent check of the rule with Python integers: each is 1 mod 2N, passes Fermat tests,
        # and no candidate between consecutive entries (or the bound) passes them
        prev = 1 << bits
        for p in plist:
            assert p % (2 * N) == 1 and p < prev and _fermat_probable_prime(p)
            c = ((prev - 2) // (2 * N)) * (2 * N) + 1
            while c > p:
                assert not _fermat_probable_prime(c), c
                c -= 2 * N
            prev = p


def test_is_prime_small_and_carmichael():
    L = ckks.lib()
    sieve = [n for n in range(2, 2000) if all(n % d for d in range(2, int(n ** 0.5) + 1))]
    assert [n for n in range(2000) if L.orc_is_prime(n)] == sieve
    for carmichael in (561, 1105, 1729, 2465, 6601, 825265, 321197185, 3825123056546413051):
        assert not L.orc_is_prime(carmichael)
    assert L.orc_is_prime((1 << 61) - 1)


@pytest.fixture(scope="module")
def small():
    N = 32
    primes, P = ckks.prime_chain(N, 2)
    return ckks.Params(N, primes, P, 2.0 ** 40)


def test_psi_is_primitive_2n_th_root(small):
    for q, psi in small.psi.items():
        assert pow(psi, small.N, q) == q - 1 and pow(psi, 2 * small.N, q) == 1


def test_ntt_equals_direct_evaluation_in_python_ints(small):
    rnd = random.Random(1)
    N = small.N
    for q in small.basis:
        a = [rnd.randrange(q) for _ in range(N)]
        psi = small.psi[q]
        expect = [sum(a[k] * pow(psi, (2 * i + 1) * k, q) for k in range(N)) % q for i in range(N)]
        got = ckks.ntt(np.array([a], dtype=np.uint64), [q], small)[0]
        assert [int(v) for v in got] == expect
        back = ckks.intt(got[None, :], [q], small)[0]
        assert [int(v) for v in back] == a


def test_ntt_direct_c_routine_agrees(small):
    # the O(N^2) C evaluation is itself only a pin; make sure it says the same as Python
    q = small.basis[1]
    a = np.arange(1, small.N + 1, dtype=np.uint64) * np.uint64(12345678901)
    a %= np.uint64(q)
    out = np.zeros_like(a)
    ckks.lib().orc_ntt_direct(ckks._p(a, ckks._u64p), ckks._p(out, ckks._u64p), small.N, q, small.psi[q])
    assert np.array_equal(out, ckks.ntt(a[None, :], [q], small)[0])


def test_ring_mul_equals_schoolbook_negacyclic(small):
    rnd = random.Random(2)
    N = small.N
    for q in small.basis:
        a = [rnd.randrange(q) for _ in range(N)]
        b = [rnd.randrange(q) for _ in range(N)]
        expect = [0] * N
        for i in range(N):
            for j in range(N):
                if i + j < N:
                    expect[i + j] = (expect[i + j] + a[i] * b[j]) % q
                else:
                    expect[i + j - N] = (expect[i + j - N] - a[i] * b[j]) % q
        got = ckks.ring_mul(np.array([a], dtype=np.uint64), np.array([b], dtype=np.uint64), [q], small)[0]
        assert [int(v) for v in got] == expect


def test_ntt_roundtrip_larger_ring():
    N = 1 << 12
    primes, P = ckks.prime_chain(N, 2)
    par = ckks.Params(N, primes, P, 2.0 ** 40)
    rng = np.random.default_rng(3)
    a = np.stack([rng.integers(0, q, size=N, dtype=np.uint64) for q in par.basis])
    f = ckks.ntt(a, par.basis, par)
    assert not np.array_equal(f, a)
    assert np.array_equal(ckks.intt(f, par.basis, par), a)
    # X * a(X): multiplying by the monomial X shifts coefficients and wraps with a minus sign
    x = np.zeros((len(par.basis), N), dtype=np.uint64)
    x[:, 1] = 1
    prod = ckks.ring_mul(a, x, par.basis, par)
    for i, q in enumerate(par.basis):
        expect = np.roll(a[i], 1)
        expect[0] = (np.uint64(q) - expect[0]) % np.uint64(q)
        assert np.array_equal(prod[i], expect)


def test_automorphism_definition_and_ntt_index_map(small):
    rnd = random.Random(4)
    N = small.N
    q = small.basis[0]
    psi = small.psi[q]
    a = [rnd.randrange(q) for _ in range(N)]
    for g in (5, 25, 3, 2 * N - 1):
        # definition: a(X^g) mod X^N + 1 with Python ints
        expect = [0] * N
        for i, v in enumerate(a):
            k = (i * g) % (2 * N)
            if k < N:
                expect[k] = (expect[k] + v) % q
            else:
                expect[k - N] = (expect[k - N] - v) % q
        got = ckks.automorphism(np.array(a, dtype=np.uint64), g, q)
        assert [int(v) for v in got] == expect
        # evaluation view: phi_g(a)(psi^e) = a(psi^(e*g)), so in natural order the NTT of phi_g(a)
        # is the NTT of a gathered at index ((2i+1)*g mod 2N - 1)/2
        fa = ckks.ntt(np.array([a], dtype=np.uint64), [q], small)[0]
        fg = ckks.ntt(got[None, :], [q], small)[0]
        idx = [(((2 * i + 1) * g) % (2 * N) - 1) // 2 for i in range(N)]
        assert np.array_equal(fg, fa[idx])
    assert small.psi[q] == psi
