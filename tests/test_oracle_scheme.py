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
