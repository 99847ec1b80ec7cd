"""Pins for the oracle's canonical-embedding encoder and the host-stub decoder."""
import numpy as np
import pytest

from oracle import ckks


def slot_points(N):
    """zeta^(5^j) for j < N/2, in extended precision."""
    n = N // 2
    e = np.array([pow(5, j, 2 * N) for j in range(n)], dtype=np.int64)
    ang = np.pi * e.astype(np.longdouble) / np.longdouble(N)
    return np.cos(ang) + 1j * np.sin(ang), e


@pytest.mark.parametrize("N", [8, 16, 64])
def test_monomials_encode_to_unit_coefficients(N):
    # The slot vector of the polynomial X^k is (zeta_j^k)_j, so it must encode to scale * e_k.
    n = N // 2
    scale = 2.0 ** 40
    _, e = slot_points(N)
    for k in range(N):
        z = np.exp(1j * np.pi * ((e * k) % (2 * N)) / N)
        m = ckks.encode_coeffs(z, N, scale)
        expect = np.zeros(N, dtype=np.int64)
        expect[k] = 1 << 40
        assert np.array_equal(m, expect), k


@pytest.mark.parametrize("N", [16, 64])
def test_encode_matches_direct_formula(N):
    # u_k = (1/n) sum_j z_j zeta_j^(-k); m_k = round(scale Re u_k), m_{k+n} = round(scale Im u_k),
    # evaluated term by term in extended precision.
    n = N // 2
    rng = np.random.default_rng(N)
    scale = 2.0 ** 40
    z = rng.normal(size=n) + 1j * rng.normal(size=n)
    _, e = slot_points(N)
    expect = np.zeros(N, dtype=np.int64)
    for k in range(n):
        ang = -(np.pi * ((e * k) % (2 * N)).astype(np.longdouble)) / np.longdouble(N)
        w = np.cos(ang) + 1j * np.sin(ang)
        u = (z.astype(np.clongdouble) * w).sum() / n
        expect[k] = int(np.rint(u.real * scale))
        expect[k + n] = int(np.rint(u.imag * scale))
    got = ckks.encode_coeffs(z, N, scale)
    assert np.abs(got - expect).max() == 0


def test_constant_slots_encode_to_constant_polynomial():
    N = 256
    for c in (0.75, -3.0, 0.02):
        m = ckks.encode_coeffs(np.full(N // 2, c), N, 2.0 ** 40)
        assert m[0] == int(np.rint(c * 2.0 ** 40))
        assert not m[1:].any()


def test_rounding_is_ties_to_even():
    # constant c with scale*c = k + 0.5 exactly must round to the even neighbour
    N = 16
    scale = 2.0 ** 10
    for half, even in ((2.5, 2), (3.5, 4), (-2.5, -2), (-3.5, -4), (0.5, 0)):
        m = ckks.encode_coeffs(np.full(N // 2, half / scale), N, scale)
        assert m[0] == even and not m[1:].any()


def test_decode_inverts_encode():
    N = 1 << 10
    rng = np.random.default_rng(0)
    z = rng.normal(size=N // 2) + 1j * rng.normal(size=N // 2)
    m = ckks.encode_coeffs(z, N, 2.0 ** 40)
    assert np.abs(ckks.decode(m, N, 2.0 ** 40) - z).max() < 2.0 ** -28
    # decode from the definition z_j = m(zeta_j)/scale on a small ring
    N = 32
    z = rng.normal(size=N // 2)
    m = ckks.encode_coeffs(z, N, 2.0 ** 40)
    pts, _ = slot_points(N)
    direct = np.array([(m.astype(np.longdouble) * pt ** np.arange(N)).sum() for pt in pts]) / 2.0 ** 40
    assert np.abs(ckks.decode(m, N, 2.0 ** 40) - direct.astype(np.complex128)).max() < 1e-9


def test_real_batch_equals_single_and_has_conjugate_symmetry_free_form():
    N = 128
    rng = np.random.default_rng(5)
    z = rng.normal(size=(3, N // 2))
    batch = ckks.encode_real_batch(z, N, 2.0 ** 40)
    for i in range(3):
        assert np.array_equal(batch[i], ckks.encode_coeffs(z[i], N, 2.0 ** 40))


def test_automorphism_rotates_slots_left():
    N = 64
    n = N // 2
    rng = np.random.default_rng(6)
    z = rng.normal(size=n)
    q = ckks.find_primes(1 << 50, 2 * N, 1)[0]
    m = ckks.encode_coeffs(z, N, 2.0 ** 40)
    res = ckks.to_residues(m, [q])[0]
    for steps in (1, 2, 7, n - 1):
        g = ckks.galois_element(steps, N)
        rot = ckks.automorphism(res, g, q).astype(np.int64)
        rot = np.where(rot > q // 2, rot - q, rot)
        got = ckks.decode(rot, N, 2.0 ** 40)
        assert np.abs(got - np.roll(z, -steps)).max() < 1e-9      # out[s] = in[s + steps]


def test_overflow_is_reported():
    with pytest.raises(OverflowError):
        ckks.encode_coeffs(np.full(8, 1e10), 16, 2.0 ** 40)
