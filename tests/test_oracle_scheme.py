"""Pins for the oracle's scheme-level steps: key switch, ModDown, rescale, decrypt, packing, BSGS,
and the end-to-end encrypted matrix-vector product against an fp64 W.x."""
from functools import reduce

import numpy as np
import pytest

from oracle import ckks, slotsim
from oracle.ckks import Params, Plan
from paper_2606_17421_b200 import workloads as wl


def crt(residues, moduli):
    """Python-int CRT: the integer in [0, prod) with the given residues."""
    Q = reduce(lambda a, b: a * b, moduli)
    x = 0
    for r, q in zip(residues, moduli):
        Qi = Q // q
        x += int(r) * Qi * pow(Qi, -1, q)
    return x % Q, Q


def centred(x, Q):
    return x - Q if x > Q // 2 else x


@pytest.fixture(scope="module")
def ring64():
    N = 64
    primes, P = ckks.prime_chain(N, 2)
    par = Params(N, primes, P, 2.0 ** 40)
    s = ckks.keygen(par, 11)
    return par, s


def test_mod_down_of_exact_multiple_is_exact(ring64):
    par, _ = ring64
    rng = np.random.default_rng(0)
    v = ckks.sample_uniform(rng, par.primes, par.N)
    u = np.zeros((par.r + 1, par.N), dtype=np.uint64)
    for i, q in enumerate(par.primes):
        acc = np.zeros(par.N, dtype=np.uint64)
        ckks.mul_acc(acc, v[i], np.full(par.N, par.P % q, dtype=np.uint64), [q], par.N)
        u[i] = acc
    assert np.array_equal(ckks.mod_down(u, par), v)       # residue mod P is zero: P*v / P = v


def test_mod_down_is_rounded_division_by_P(ring64):
    par, _ = ring64
    rng = np.random.default_rng(1)
    u = ckks.sample_uniform(rng, par.basis, par.N)
    v = ckks.mod_down(u, par)
    Qp = reduce(lambda a, b: a * b, par.primes)
    for k in range(0, par.N, 7):
        x, QP = crt(u[:, k], par.basis)
        t = centred(x % par.P, par.P)
        expect = ((x - t) // par.P) % Qp                  # exact division, = round(x / P) mod Q
        assert (x - t) % par.P == 0
        assert abs(expect - round_div(x, par.P)) % Qp in (0,)
        got, _ = crt(v[:, k], par.primes)
        assert got == expect


def round_div(x, d):
    return (2 * x + d) // (2 * d)


def test_rescale_is_big_integer_round(ring64):
    par, _ = ring64
    rng = np.random.default_rng(2)
    ct = np.stack([ckks.sample_uniform(rng, par.primes, par.N) for _ in range(2)])
    out = ckks.rescale(par, ct)
    assert out.shape == (2, par.r - 1, par.N)
    qL = par.primes[-1]
    Qp = reduce(lambda a, b: a * b, par.primes[:-1])
    for comp in range(2):
        for k in range(0, par.N, 5):
            x, Q = crt(ct[comp, :, k], par.primes)
            xc = centred(x, Q)
            t = centred(xc % qL, qL)
            expect = ((xc - t) // qL) % Qp
            got, _ = crt(out[comp, :, k], par.primes[:-1])
            assert got == expect
            assert abs((xc - t) // qL - xc / qL) <= 0.5 + 1e-9


def test_decrypt_q0_only_equals_full_crt_decrypt(ring64):
    par, s = ring64
    rng = np.random.default_rng(3)
    m = rng.integers(-(1 << 45), 1 << 45, size=par.N)
    ct = ckks.encrypt(par, s, m, 7)
    got = ckks.decrypt(par, s, ct)
    # full decrypt with Python ints: c0 + c1*s in Z_Q[X]/(X^N+1), centred
    N = par.N
    c0 = [crt(ct[0, :, k], par.primes)[0] for k in range(N)]
    c1 = [crt(ct[1, :, k], par.primes)[0] for k in range(N)]
    Q = reduce(lambda a, b: a * b, par.primes)
    full = list(c0)
    for i in range(N):
        for j in range(N):
            if s[j] == 0:
                continue
            k = i + j
            term = c1[i] * int(s[j])
            if k < N:
                full[k] += term
            else:
                full[k - N] -= term
    full = np.array([centred(v % Q, Q) for v in full], dtype=np.int64)
    assert np.array_equal(got, full)
    noise = got - m
    assert np.abs(noise).max() <= 6 * 3.2 + 1            # fresh noise is the truncated Gaussian


def test_rotation_decrypts_to_left_rotation_with_bounded_noise(ring64):
    par, s = ring64
    N, n = par.N, par.n
    rng = np.random.default_rng(4)
    z = rng.normal(size=n)
    m = ckks.encode_coeffs(z, N, par.scale)
    ct = ckks.encrypt(par, s, m, 8)
    for steps in (1, 3, n - 1):
        g = ckks.galois_element(steps, N)
        key = ckks.galois_key(par, s, g, 9)
        rot = ckks.rotate_galois(par, ct, g, key)
        dec = ckks.decrypt(par, s, rot)
        assert np.abs(ckks.decode(dec, N, par.scale) - np.roll(z, -steps)).max() < 1e-8
        # coefficient-level: message moves by the automorphism; added noise stays under the loose
        # a-priori bound r*N*q_max*6sigma/P + N (in coefficient units), plus the fresh noise
        q0 = par.primes[0]
        moved = ckks.automorphism(ckks.to_residues(m, [q0])[0], g, q0).astype(np.int64)
        moved = np.where(moved > q0 // 2, moved - q0, moved)
        bound = par.r * N * max(par.primes) * 6 * 3.2 / par.P + N + 6 * 3.2 + 1
        assert np.abs(dec - moved).max() <= bound
    assert np.array_equal(ckks.rotate(par, ct, 0, {}), ct)


def test_rotation_composes(ring64):
    par, s = ring64
    rng = np.random.default_rng(5)
    z = rng.normal(size=par.n)
    ct = ckks.encrypt(par, s, ckks.encode_coeffs(z, par.N, par.scale), 10)
    keys = {ckks.galois_element(t, par.N): ckks.galois_key(par, s, ckks.galois_element(t, par.N), 12) for t in (2, 5)}
    a = ckks.rotate(par, ckks.rotate(par, ct, 2, keys), 5, keys)
    assert np.abs(ckks.decode(ckks.decrypt(par, s, a), par.N, par.scale) - np.roll(z, -7)).max() < 1e-8


# ------------------------------------------------------------------ packing / BSGS (slot level, no crypto)

PLANS = [(64, 1, 8, 8, 2048), (64, 4, 4, 4, 512), (1024, 16, 8, 8, 16384), (1024, 32, 8, 4, 32768), (8, 2, 2, 2, 32),
         # the plans the workloads ship with (ring sizes of their parameter sets)
         (1024, 16, 16, 4, 16384), (512, 32, 4, 4, 16384), (256, 64, 2, 2, 16384), (128, 128, 1, 1, 16384),
         (1024, 4, 16, 16, 4096)]


@pytest.mark.parametrize("D,tau,b,g,n", PLANS)
def test_slot_simulator_equals_matvec(D, tau, b, g, n):
    rng = np.random.default_rng(D + tau)
    for d_out, d_in in ((D, D), (D + 3, 2 * D - 5), (3 * D // 4, 3 * D)):
        W = rng.normal(size=(d_out, d_in))
        x = rng.normal(size=d_in)
        y = slotsim.linear_slots(W, x, Plan(D, tau, b, g), n)
        assert np.abs(y - W @ x).max() < 1e-10


def test_structured_matrices_localise_packing():
    plan, n, D = Plan(16, 4, 2, 2), 128, 16
    x = np.arange(1.0, D + 1)
    assert np.allclose(slotsim.linear_slots(np.eye(D), x, plan, n), x)
    shift = np.roll(np.eye(D), 3, axis=1)                     # y[i] = x[i+3]
    assert np.allclose(slotsim.linear_slots(shift, x, plan, n), np.roll(x, -3))
    for (row, col) in ((0, 0), (5, 11), (15, 2)):
        W = np.zeros((D, D))
        W[row, col] = 2.0
        y = slotsim.linear_slots(W, x, plan, n)
        expect = np.zeros(D)
        expect[row] = 2.0 * x[col]
        assert np.allclose(y, expect)
        # exactly one diagonal is non-zero, and only in the slots of (kappa=row, c=class of col)
        nz = [(j, k) for j in range(plan.g) for k in range(plan.b)
              if ckks.bsgs_plain_slots(W, plan, 0, 0, j, k, n).any()]
        assert len(nz) == 1


def test_worked_packing_example_n8():
    # n = 8, D = 4, tau = 2, M = 2: slots are (kappa, c) = (0,0),(0,1),(1,0),(1,1),...
    plan = Plan(4, 2, 2, 1)
    x = np.array([10.0, 11.0, 12.0, 13.0])
    assert list(ckks.pack_input(x, plan, 8)) == [10, 12, 11, 13, 12, 10, 13, 11]
    W = np.arange(16.0).reshape(4, 4)                            # W[i][j] = 4i + j
    d0 = ckks.diagonal_slots(W, plan, 0, 0, 0, 8)
    d1 = ckks.diagonal_slots(W, plan, 0, 0, 1, 8)
    assert list(d0) == [0, 2, 5, 7, 10, 8, 15, 13]               # W00 W02 W11 W13 W22 W20 W33 W31
    assert list(d1) == [1, 3, 6, 4, 11, 9, 12, 14]               # W01 W03 W12 W10 W23 W21 W30 W32


# ------------------------------------------------------------------ end to end

def run_linear(par, plan, W, x, seed, tol):
    s = ckks.keygen(par, seed)
    keys = ckks.make_rotation_keys(par, s, plan, seed)
    cts = ckks.encrypt_vector(par, plan, s, x, seed)
    out = ckks.linear(par, plan, cts, W, keys)
    d_out = W.shape[0]
    y = np.zeros(d_out)
    out_scale = par.scale * par.scale / par.primes[-1]
    for p, ct in out.items():
        low = ckks.rescale(par, ct)
        part = ckks.fold_output(ckks.decode(ckks.decrypt(par, s, low), par.N, out_scale), plan, p, d_out)
        y[p * plan.D:p * plan.D + len(part)] = part
    err = np.abs(y - W.astype(np.float64) @ x).max()
    assert err < tol, err
    return err


def test_end_to_end_small_ring_ragged_shape():
    N = 256
    primes, P = ckks.prime_chain(N, 2)
    par = Params(N, primes, P, 2.0 ** 40)
    plan = Plan(16, 4, 2, 2)
    W = wl.gen_weights(0, "t", 37, 41)
    x = wl.gen_activation(0, "t", 41)
    run_linear(par, plan, W, x, 1, 1e-6)


def test_end_to_end_tiny_config():
    w = wl.WORKLOADS["tiny"]
    ps = wl.PARAM_SETS[w.params]
    par = Params(ps["N"], ps["primes"], ps["special"], ps["scale"])
    plan = Plan(w.plan.D, w.plan.tau, w.plan.b, w.plan.g)
    W = wl.gen_weights(0, "tiny", 64, 64)
    x = wl.gen_activation(0, "tiny", 64)
    err = run_linear(par, plan, W, x, 0, 1e-2)
    assert err < 1e-6      # the stated tolerance is 1e-2; a scale-bookkeeping slip would sit near 1e-5


# ------------------------------------------------------------------ in-ciphertext fold of the tau partial sums

def test_fold_in_ciphertext_sums_each_group_of_tau_slots(ring64):
    # expected values come straight from the slot vector: slot kappa*tau of the folded ciphertext must
    # hold z[kappa*tau] + ... + z[kappa*tau + tau - 1]
    par, s = ring64
    plan = Plan(8, 4, 2, 1)                 # n = 32 slots = D * tau
    rng = np.random.default_rng(21)
    z = rng.normal(size=par.n)
    ct = ckks.encrypt(par, s, ckks.encode_coeffs(z, par.N, par.scale), 22)
    keys = {ckks.galois_element(t, par.N): ckks.galois_key(par, s, ckks.galois_element(t, par.N), 23)
            for t in ckks.fold_rotations(plan)}
    assert ckks.fold_rotations(plan) == [1, 2]
    folded = ckks.fold_in_ciphertext(par, plan, ct, keys)
    slots = ckks.decode(ckks.decrypt(par, s, folded), par.N, par.scale)
    expect = z.reshape(plan.D, plan.tau).sum(axis=1)
    assert np.abs(ckks.folded_output(slots, plan, 0, plan.D) - expect).max() < 1e-8
    # tau = 1: nothing to fold
    assert ckks.fold_rotations(Plan(32, 1, 2, 2)) == []
    assert np.array_equal(ckks.fold_in_ciphertext(par, Plan(32, 1, 2, 2), ct, {}), ct)


def test_linear_then_fold_in_ciphertext_gives_the_product():
    N = 256
    primes, P = ckks.prime_chain(N, 2)
    par = Params(N, primes, P, 2.0 ** 40)
    plan = Plan(16, 4, 2, 2)
    W = wl.gen_weights(3, "f", 37, 41)
    x = wl.gen_activation(3, "f", 41)
    s = ckks.keygen(par, 3)
    keys = ckks.make_rotation_keys(par, s, plan, 3, extra_steps=ckks.fold_rotations(plan))
    cts = ckks.encrypt_vector(par, plan, s, x, 3)
    out = ckks.linear(par, plan, cts, W, keys)
    y = np.zeros(37)
    out_scale = par.scale * par.scale / par.primes[-1]
    for p, ct in out.items():
        low = ckks.rescale(par, ckks.fold_in_ciphertext(par, plan, ct, keys))
        part = ckks.folded_output(ckks.decode(ckks.decrypt(par, s, low), par.N, out_scale), plan, p, 37)
        y[p * plan.D:p * plan.D + len(part)] = part
    assert np.abs(y - W.astype(np.float64) @ x).max() < 1e-6


# ------------------------------------------------------------------ key switch before the division by P

def negacyclic_int(a, b, N):
    """Schoolbook product of two integer polynomials modulo X^N + 1 (Python integers)."""
    out = [0] * N
    for i in range(N):
        if a[i] == 0:
            continue
        for j in range(N):
            if b[j] == 0:
                continue
            k = i + j
            if k < N:
                out[k] += a[i] * b[j]
            else:
                out[k - N] -= a[i] * b[j]
    return out


def test_key_switch_ext_is_P_times_the_rotated_product_plus_small_noise(ring64):
    # Over the full basis {q_i, P}: u0 + u1*s = P * (phi_g(c1) * phi_g(s) mod Q) + sum_j digit_j * e_j, with the
    # last term below r * N * q_max * 6 sigma.  Checked with Python integers through the CRT.
    par, s = ring64
    N = par.N
    rng = np.random.default_rng(31)
    c1 = ckks.sample_uniform(rng, par.primes, N)
    g = ckks.galois_element(3, N)
    key = ckks.galois_key(par, s, g, 32)
    u = ckks.key_switch_ext(par, c1, g, key)
    assert u.shape == (2, par.r + 1, N)
    Q = reduce(lambda a, b: a * b, par.primes)
    QP = Q * par.P
    u0 = [crt(u[0, :, k], par.basis)[0] for k in range(N)]
    u1 = [crt(u[1, :, k], par.basis)[0] for k in range(N)]
    lhs = [(a + b) % QP for a, b in zip(u0, negacyclic_int(u1, [int(v) for v in s], N))]
    # phi_g of c1 (as the integer in [0, Q)) and of s, by the definition i -> i*g mod 2N with X^N = -1
    def phi(poly):
        out = [0] * N
        for i, v in enumerate(poly):
            k = (i * g) % (2 * N)
            if k < N:
                out[k] = v
            else:
                out[k - N] = -v
        return out
    c1_int = [crt(c1[:, k], par.primes)[0] for k in range(N)]
    prod = [v % Q for v in negacyclic_int(phi(c1_int), phi([int(v) for v in s]), N)]
    bound = par.r * N * max(par.primes) * 6 * 3.2
    for k in range(N):
        diff = centred((lhs[k] - par.P * prod[k]) % QP, QP)
        assert abs(diff) <= bound


def test_rotate_galois_is_key_switch_ext_then_mod_down(ring64):
    par, s = ring64
    rng = np.random.default_rng(33)
    ct = np.stack([ckks.sample_uniform(rng, par.primes, par.N) for _ in range(2)])
    g = ckks.galois_element(5, par.N)
    key = ckks.galois_key(par, s, g, 34)
    u = ckks.key_switch_ext(par, ct[1], g, key)
    rot = ckks.rotate_galois(par, ct, g, key)
    for i, q in enumerate(par.primes):
        c0g = ckks.automorphism(ct[0, i], g, q)
        assert np.array_equal(rot[0, i], (c0g + ckks.mod_down(u[0], par)[i]) % np.uint64(q))
        assert np.array_equal(rot[1, i], ckks.mod_down(u[1], par)[i])


# ------------------------------------------------------------------ plan modes: complex packing, one division by P per output

COMPLEX_PLANS = [(64, 1, 8, 8, 2048), (64, 4, 4, 4, 512), (8, 2, 2, 2, 32), (1024, 16, 16, 4, 16384),
                 (1024, 32, 8, 4, 32768)]


@pytest.mark.parametrize("D,tau,b,g,n", COMPLEX_PLANS)
def test_slot_simulator_with_complex_packing_equals_matvec(D, tau, b, g, n):
    # two row blocks per output ciphertext (real and imaginary parts); shapes with an even and an odd number of
    # row blocks (the last ciphertext then carries one block only) and ragged edges
    rng = np.random.default_rng(D + tau + 1)
    plan = Plan(D, tau, b, g, pack="complex")
    for d_out, d_in in ((2 * D, D), (3 * D, D + 5), (D + 3, 2 * D - 5), (3 * D // 4, D)):
        W = rng.normal(size=(d_out, d_in))
        x = rng.normal(size=d_in)
        assert plan.n_out(d_out) == -(-d_out // (2 * D))
        y = slotsim.linear_slots(W, x, plan, n)
        assert np.abs(y - W @ x).max() < 1e-10


def test_complex_plaintext_is_the_two_real_ones_combined():
    # encode is linear up to rounding: the coefficients of (block 2p) + i (block 2p+1) differ from
    # enc(block 2p) + enc(i * block 2p+1) by at most one unit per coefficient (two roundings against one)
    N, n = 256, 128
    plan_r, plan_c = Plan(16, 4, 2, 2), Plan(16, 4, 2, 2, pack="complex")
    W = wl.gen_weights(5, "c", 40, 20)
    for (p, q, j, k) in ((0, 0, 0, 0), (0, 1, 1, 1), (1, 0, 1, 0)):
        zc = ckks.plain_slots(W, plan_c, p, q, j, k, n)
        za = ckks.plain_slots(W, plan_r, 2 * p, q, j, k, n)
        zb = ckks.plain_slots(W, plan_r, 2 * p + 1, q, j, k, n)
        assert np.array_equal(zc, za + 1j * zb)
        mc = ckks.encode_coeffs(zc, N, 2.0 ** 40)
        ma = ckks.encode_coeffs(za, N, 2.0 ** 40)
        mb = ckks.encode_coeffs(1j * zb, N, 2.0 ** 40)
        assert np.abs(mc - (ma + mb)).max() <= 1
        assert np.array_equal(ckks.encode_complex_batch(zc[None], N, 2.0 ** 40)[0], mc)
    # block 3 of a 40-row matrix with D = 16 does not exist: the imaginary part of ciphertext 1 is empty
    assert not ckks.plain_slots(W, plan_c, 1, 0, 0, 0, n).imag.any()


def run_linear_modes(par, plan, W, x, seed, tol):
    s = ckks.keygen(par, seed)
    keys = ckks.make_rotation_keys(par, s, plan, seed)
    cts = ckks.encrypt_vector(par, plan, s, x, seed)
    out = ckks.linear(par, plan, cts, W, keys)
    d_out = W.shape[0]
    assert sorted(out) == list(range(plan.n_out(d_out)))
    y = np.zeros(d_out)
    out_scale = par.scale * par.scale / par.primes[-1]
    for p, ct in out.items():
        low = ckks.rescale(par, ct)
        part = ckks.fold_output(ckks.decode(ckks.decrypt(par, s, low), par.N, out_scale), plan, p, d_out)
        y[p * plan.rows_per_ct:p * plan.rows_per_ct + len(part)] = part
    err = np.abs(y - W.astype(np.float64) @ x).max()
    assert err < tol, err
    return out, s, keys, cts


@pytest.mark.parametrize("pack,moddown", [("complex", "per_rotation"), ("real", "per_output"), ("complex", "per_output")])
def test_end_to_end_plan_modes_small_ring(pack, moddown):
    N = 256
    primes, P = ckks.prime_chain(N, 2)
    par = Params(N, primes, P, 2.0 ** 40)
    W = wl.gen_weights(0, "m", 37, 41)            # 3 row blocks of 16: with complex packing two ciphertexts
    x = wl.gen_activation(0, "m", 41)
    run_linear_modes(par, Plan(16, 4, 2, 2, pack=pack, moddown=moddown), W, x, 1, 1e-6)
    run_linear_modes(par, Plan(16, 1, 4, 4, pack=pack, moddown=moddown), W, x, 2, 1e-6)
    run_linear_modes(par, Plan(16, 8, 2, 1, pack=pack, moddown=moddown), W, x, 3, 1e-6)     # no giant step


def test_per_output_moddown_differs_from_per_rotation_only_by_rounding():
    # the two modes divide by P at different points, so residues differ, but only by the rounding of the g - 1
    # divisions: centred difference at most g - 1 units per coefficient (both are within 1/2 of the same real
    # quotient per rotation, summed), and the decrypted results agree to far below the tolerance
    N = 256
    primes, P = ckks.prime_chain(N, 2)
    par = Params(N, primes, P, 2.0 ** 40)
    W = wl.gen_weights(7, "pm", 30, 33)
    x = wl.gen_activation(7, "pm", 33)
    plan_a = Plan(16, 1, 4, 4)
    plan_b = Plan(16, 1, 4, 4, moddown="per_output")
    out_a, s, keys, cts = run_linear_modes(par, plan_a, W, x, 7, 1e-6)
    out_b = ckks.linear(par, plan_b, cts, W, keys)
    Q = reduce(lambda a, b: a * b, par.primes)
    differs = False
    for p in out_a:
        assert out_a[p].shape == out_b[p].shape
        differs = differs or not np.array_equal(out_a[p], out_b[p])
        for comp in range(2):
            for k in range(0, N, 3):
                a, _ = crt(out_a[p][comp, :, k], par.primes)
                b, _ = crt(out_b[p][comp, :, k], par.primes)
                assert abs(centred((a - b) % Q, Q)) <= plan_a.g - 1
    assert differs                                  # the mode is really read
    # with a single giant step there is nothing to merge: identical residues
    plan_c, plan_d = Plan(16, 4, 4, 1), Plan(16, 4, 4, 1, moddown="per_output")
    s2 = ckks.keygen(par, 8)
    keys2 = ckks.make_rotation_keys(par, s2, plan_c, 8)
    cts2 = ckks.encrypt_vector(par, plan_c, s2, x, 8)
    o_c, o_d = ckks.linear(par, plan_c, cts2, W, keys2), ckks.linear(par, plan_d, cts2, W, keys2)
    assert all(np.array_equal(o_c[p], o_d[p]) for p in o_c)


# ------------------------------------------------------------------ double hoisting

def test_extended_baby_rotation_divided_by_P_is_the_rotation(ring64):
    # (P*phi(c0) + u0, u1) differs from (u0, u1) by an exact multiple of P, so its division by P is
    # phi(c0) + ModDown(u0), ModDown(u1): exactly what the single-hoisted rotation produces
    par, s = ring64
    plan = Plan(8, 4, 4, 1)
    rng = np.random.default_rng(41)
    z = rng.normal(size=par.n)
    ct = ckks.encrypt(par, s, ckks.encode_coeffs(z, par.N, par.scale), 42)
    keys = ckks.make_rotation_keys(par, s, plan, 43)
    ext = ckks.baby_rotations_ext(par, plan, ct, keys)
    plain = ckks.baby_rotations(par, plan, ct, keys)
    for k in range(plan.b):
        assert ext[k].shape == (2, par.r + 1, par.N)
        got = np.stack([ckks.mod_down(ext[k][0], par), ckks.mod_down(ext[k][1], par)])
        assert np.array_equal(got, plain[k]), k
    assert not ext[0][:, par.r].any()                    # k = 0: P * ct has residue zero modulo P


@pytest.mark.parametrize("pack,moddown", [("real", "per_rotation"), ("complex", "per_output")])
def test_end_to_end_double_hoisting_small_ring(pack, moddown):
    N = 256
    primes, P = ckks.prime_chain(N, 2)
    par = Params(N, primes, P, 2.0 ** 40)
    W = wl.gen_weights(0, "dh", 37, 41)
    x = wl.gen_activation(0, "dh", 41)
    for plan_t in ((16, 4, 2, 2), (16, 1, 4, 4), (16, 8, 2, 1), (16, 1, 1, 16)):
        plan = Plan(*plan_t, pack=pack, moddown=moddown, hoist="double")
        out, s, keys, cts = run_linear_modes(par, plan, W, x, 1, 1e-6)
        single = ckks.linear(par, Plan(*plan_t, pack=pack, moddown=moddown), cts, W, keys)
        if plan.b > 1:            # the division by P moved: residues differ (the decrypted values do not, see above)
            assert any(not np.array_equal(out[p], single[p]) for p in out)
        else:                     # no baby rotation: only P * ct, whose division by P is exact
            assert all(np.array_equal(out[p], single[p]) for p in out)
    # the plaintexts carry the residue modulo P
    enc = ckks.encode_weights(par, Plan(16, 4, 2, 2, hoist="double"), W, blocks=[0])
    assert enc[(0, 0, 0, 0)].shape == (par.r + 1, N)
