"""CPU oracle for the accelerator-side CKKS linear layer (ciphertext x encoded-plaintext weights).

TEST INFRASTRUCTURE ONLY.  Slow, plain and meant to be read next to the method: tests, the smoke
check and the benchmark's CPU-baseline leg are the only callers.  It shares no code with the CUDA
library and never imports it.

The paper (Sec. 4.2) delegates its CKKS arithmetic to a GPU library and states only what is
computed: a ciphertext--plaintext product with pre-encoded weight diagonals (Sec. 3.5 "Model
weights"), organised as baby-step/giant-step objects per projection (Sec. 4.2), over the ring
R_Q = Z_Q[X]/(X^N + 1) with N/2 slots, levels and rescaling (Sec. 2.1).  Everything finer is the
standard RNS-CKKS construction, fixed here step by step because the output residues depend on the
evaluation strategy (packing, BSGS split, key-switch variant, rounding points):

  canonical embedding   slot j <-> evaluation point zeta^(5^j), zeta = exp(i*pi/N)
  rotation by r         automorphism X -> X^(5^r mod 2N) followed by a key switch; rotates LEFT
  key switch            one special prime P, one ciphertext prime per digit; digits are the
                        residues of c1 mod q_j lifted to [0, q_j); decompose first, then apply the
                        automorphism; inner product with the key over the basis {q_0..q_L, P};
                        divide by P with a centred (round-to-nearest) lift, after every rotation
  packing               slot s = (rho*D + kappa)*tau + c; see `pack_input` and `diagonal_slots`
  BSGS                  diagonal i = j*b + k; Y_p = sum_j rot( sum_q sum_k Pt[p][q][j][k] * rot(ct_q, k*tau), j*b*tau )
  rescale               c'_i = (c_i - centred(c_L)) * q_L^{-1} mod q_i

Two variants change residues and are therefore modes of the plan, evaluated here step by step as well
(the paper leaves both open: Sec. 4.2 speaks of "key-switching primitives" and of weight diagonals kept
as BSGS objects, and Sec. 6.1 names the encoded-weight cache as the memory wall):
  pack = "complex"      two output row blocks share a plaintext: block 2P in the real parts of the slots,
                        block 2P+1 in the imaginary parts; the input ciphertexts stay real, so output
                        ciphertext P decrypts to (block 2P) + i (block 2P+1); half the diagonals
  moddown = "per_output"  the giant-step key switches of an output are summed in the extended basis
                        {q_0..q_L, P} and divided by P once per output ciphertext and component,
                        instead of once per rotation
  hoist = "double"      the baby-step rotations are not divided by P either: X[q][k] stays in the extended
                        basis as (P*phi_k(c0) + u0, u1), the plaintexts are reduced modulo P as well, the
                        products are summed over the extended basis, and each inner sum A[p][j] is divided
                        by P once (per output block and giant step instead of per input and baby step)

Array conventions (all numpy, C order):
  ciphertext  uint64 [2][r][N]   component, prime, coefficient; coefficient domain, residues in [0, q_i)
  plaintext   uint64 [r][N]      coefficient domain
  galois key  uint64 [r][2][r+1][N]   digit, component (0 = b, 1 = a), prime of the extended basis
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass, field

import numpy as np

from . import build as _build

_u64p = ctypes.POINTER(ctypes.c_uint64)
_i64p = ctypes.POINTER(ctypes.c_int64)
_f64p = ctypes.POINTER(ctypes.c_double)

_lib = None


def lib():
    """Load (building if needed) the C primitives."""
    global _lib
    if _lib is None:
        L = ctypes.CDLL(_build.build())
        L.orc_mulmod.restype = ctypes.c_uint64
        L.orc_mulmod.argtypes = [ctypes.c_uint64] * 3
        L.orc_powmod.restype = ctypes.c_uint64
        L.orc_powmod.argtypes = [ctypes.c_uint64] * 3
        L.orc_invmod.restype = ctypes.c_uint64
        L.orc_invmod.argtypes = [ctypes.c_uint64] * 2
        L.orc_is_prime.restype = ctypes.c_int
        L.orc_is_prime.argtypes = [ctypes.c_uint64]
        L.orc_find_primes.restype = ctypes.c_int
        L.orc_find_primes.argtypes = [ctypes.c_uint64, ctypes.c_uint64, ctypes.c_int, _u64p]
        L.orc_primitive_root_2n.restype = ctypes.c_uint64
        L.orc_primitive_root_2n.argtypes = [ctypes.c_uint64, ctypes.c_uint32]
        L.orc_ntt_batch.restype = None
        L.orc_ntt_batch.argtypes = [_u64p, ctypes.c_uint32, ctypes.c_uint32, _u64p, _u64p]
        L.orc_intt_batch.restype = None
        L.orc_intt_batch.argtypes = [_u64p, ctypes.c_uint32, ctypes.c_uint32, _u64p, _u64p]
        L.orc_ntt_direct.restype = None
        L.orc_ntt_direct.argtypes = [_u64p, _u64p, ctypes.c_uint32, ctypes.c_uint64, ctypes.c_uint64]
        L.orc_negacyclic_schoolbook.restype = None
        L.orc_negacyclic_schoolbook.argtypes = [_u64p, _u64p, _u64p, ctypes.c_uint32, ctypes.c_uint64]
        L.orc_mul_acc_batch.restype = None
        L.orc_mul_acc_batch.argtypes = [_u64p, _u64p, _u64p, ctypes.c_uint32, ctypes.c_uint32, _u64p]
        L.orc_automorphism.restype = None
        L.orc_automorphism.argtypes = [_u64p, _u64p, ctypes.c_uint32, ctypes.c_uint64, ctypes.c_uint64]
        L.orc_encode_slots.restype = ctypes.c_int
        L.orc_encode_slots.argtypes = [_f64p, _f64p, ctypes.c_uint32, ctypes.c_double, _i64p]
        L.orc_encode_real_batch.restype = ctypes.c_int
        L.orc_encode_real_batch.argtypes = [_f64p, ctypes.c_uint32, ctypes.c_uint32, ctypes.c_double, _i64p]
        L.orc_encode_complex_batch.restype = ctypes.c_int
        L.orc_encode_complex_batch.argtypes = [_f64p, _f64p, ctypes.c_uint32, ctypes.c_uint32, ctypes.c_double, _i64p]
        L.orc_num_threads.restype = ctypes.c_int
        _lib = L
    return _lib


def _p(a, t):
    return a.ctypes.data_as(t)


# --------------------------------------------------------------------------- parameters

def find_primes(below: int, two_n: int, count: int) -> list[int]:
    """The `count` largest primes < below that are 1 mod two_n, descending."""
    out = np.zeros(count, dtype=np.uint64)
    got = lib().orc_find_primes(below, two_n, count, _p(out, _u64p))
    assert got == count
    return [int(v) for v in out]


def prime_chain(N: int, n_small: int) -> tuple[list[int], int]:
    """The modulus chain the workloads prescribe: q0 = largest prime = 1 mod 2N below 2^50,
    then the n_small largest below 2^40; special prime = largest below 2^60."""
    q0 = find_primes(1 << 50, 2 * N, 1)
    qs = find_primes(1 << 40, 2 * N, n_small)
    P = find_primes(1 << 60, 2 * N, 1)[0]
    return q0 + qs, P


@dataclass
class Params:
    """Ring and modulus chain (Sec. 2.1; Sec. 4.2 lists the prototype's own choice)."""
    N: int
    primes: list[int]          # ciphertext primes q_0 .. q_L
    P: int                     # special prime for key switching
    scale: float               # Delta
    psi: dict = field(default_factory=dict)

    def __post_init__(self):
        for q in self.primes + [self.P]:
            assert lib().orc_is_prime(q) and q % (2 * self.N) == 1, q
            self.psi[q] = int(lib().orc_primitive_root_2n(q, self.N))
        assert len(set(self.primes + [self.P])) == len(self.primes) + 1

    @property
    def r(self) -> int:
        return len(self.primes)

    @property
    def n(self) -> int:
        return self.N // 2

    @property
    def basis(self) -> list[int]:
        return self.primes + [self.P]


@dataclass
class Plan:
    """Tiling of a projection: tile side D, replica split tau, M = D/tau diagonals per tile,
    baby steps b, giant steps g (b*g = M)."""
    D: int
    tau: int
    b: int
    g: int
    pack: str = "real"                 # "real" | "complex": see the module docstring
    moddown: str = "per_rotation"      # "per_rotation" | "per_output"
    hoist: str = "single"              # "single" | "double"

    @property
    def M(self) -> int:
        return self.D // self.tau

    @property
    def rows_per_ct(self) -> int:
        """Output rows one output ciphertext carries."""
        return self.D * (2 if self.pack == "complex" else 1)

    def n_out(self, d_out: int) -> int:
        """Number of output ciphertexts of a projection with d_out rows."""
        return -(-d_out // self.rows_per_ct)

    def check(self, n: int):
        assert self.D * self.tau <= n and n % (self.D * self.tau) == 0
        assert self.D % self.tau == 0 and self.b * self.g == self.M
        assert self.pack in ("real", "complex") and self.moddown in ("per_rotation", "per_output")
        assert self.hoist in ("single", "double")


def galois_element(steps: int, N: int) -> int:
    """5^steps mod 2N: the automorphism that rotates the slot vector left by `steps`."""
    return pow(5, steps % (N // 2), 2 * N)


# --------------------------------------------------------------------------- transforms

def ntt(polys: np.ndarray, moduli, params: Params) -> np.ndarray:
    """Forward negacyclic NTT of polys[..., N]; moduli gives one modulus per polynomial (flattened
    order).  Natural-order evaluations at psi^(2i+1)."""
    a = np.ascontiguousarray(polys, dtype=np.uint64).copy()
    flat = a.reshape(-1, params.N)
    q = np.array(list(moduli), dtype=np.uint64)
    assert q.shape[0] == flat.shape[0]
    psi = np.array([params.psi[int(v)] for v in q], dtype=np.uint64)
    lib().orc_ntt_batch(_p(flat, _u64p), flat.shape[0], params.N, _p(q, _u64p), _p(psi, _u64p))
    return a


def intt(polys: np.ndarray, moduli, params: Params) -> np.ndarray:
    a = np.ascontiguousarray(polys, dtype=np.uint64).copy()
    flat = a.reshape(-1, params.N)
    q = np.array(list(moduli), dtype=np.uint64)
    assert q.shape[0] == flat.shape[0]
    psi = np.array([params.psi[int(v)] for v in q], dtype=np.uint64)
    lib().orc_intt_batch(_p(flat, _u64p), flat.shape[0], params.N, _p(q, _u64p), _p(psi, _u64p))
    return a


def mul_acc(acc: np.ndarray, x: np.ndarray, y: np.ndarray, moduli, N: int) -> None:
    """acc += x * y pointwise, polynomial b modulo moduli[b] (in place on acc)."""
    assert acc.flags.c_contiguous and acc.dtype == np.uint64
    x = np.ascontiguousarray(x, dtype=np.uint64)
    y = np.ascontiguousarray(y, dtype=np.uint64)
    q = np.array(list(moduli), dtype=np.uint64)
    count = acc.size // N
    assert x.size == acc.size and y.size == acc.size and q.shape[0] == count
    lib().orc_mul_acc_batch(_p(acc, _u64p), _p(x, _u64p), _p(y, _u64p), count, N, _p(q, _u64p))


def ring_mul(a: np.ndarray, b: np.ndarray, moduli, params: Params) -> np.ndarray:
    """Product in Z_q[X]/(X^N+1) per polynomial: evaluate, multiply pointwise, interpolate."""
    fa, fb = ntt(a, moduli, params), ntt(b, moduli, params)
    acc = np.zeros_like(fa)
    mul_acc(acc, fa, fb, moduli, params.N)
    return intt(acc, moduli, params)


def automorphism(poly: np.ndarray, g: int, q: int) -> np.ndarray:
    """a(X) -> a(X^g) on one coefficient-domain polynomial modulo q."""
    a = np.ascontiguousarray(poly, dtype=np.uint64)
    out = np.empty_like(a)
    lib().orc_automorphism(_p(a, _u64p), _p(out, _u64p), a.shape[0], g, q)
    return out


# --------------------------------------------------------------------------- encode / decode

def encode_coeffs(z: np.ndarray, N: int, scale: float) -> np.ndarray:
    """Slot vector z (real or complex, length N/2) -> int64 coefficients round(scale * sigma^{-1}(z))."""
    z = np.asarray(z)
    zre = np.ascontiguousarray(z.real, dtype=np.float64)
    zim = np.ascontiguousarray(z.imag, dtype=np.float64) if np.iscomplexobj(z) else None
    m = np.zeros(N, dtype=np.int64)
    st = lib().orc_encode_slots(_p(zre, _f64p), _p(zim, _f64p) if zim is not None else None,
                                N, scale, _p(m, _i64p))
    if st != 0:
        raise OverflowError("encoded coefficient out of range")
    return m


def encode_real_batch(z: np.ndarray, N: int, scale: float) -> np.ndarray:
    """z[count][N/2] real -> int64 [count][N]."""
    z = np.ascontiguousarray(z, dtype=np.float64)
    m = np.zeros((z.shape[0], N), dtype=np.int64)
    st = lib().orc_encode_real_batch(_p(z, _f64p), z.shape[0], N, scale, _p(m, _i64p))
    if st != 0:
        raise OverflowError("encoded coefficient out of range")
    return m


def encode_complex_batch(z: np.ndarray, N: int, scale: float) -> np.ndarray:
    """z[count][N/2] complex -> int64 [count][N]."""
    z = np.asarray(z, dtype=np.complex128)
    zre = np.ascontiguousarray(z.real, dtype=np.float64)
    zim = np.ascontiguousarray(z.imag, dtype=np.float64)
    m = np.zeros((z.shape[0], N), dtype=np.int64)
    st = lib().orc_encode_complex_batch(_p(zre, _f64p), _p(zim, _f64p), z.shape[0], N, scale, _p(m, _i64p))
    if st != 0:
        raise OverflowError("encoded coefficient out of range")
    return m


def to_residues(m: np.ndarray, moduli) -> np.ndarray:
    """Signed integer coefficients m[..., N] -> residues [..., len(moduli), N] in [0, q)."""
    m = np.asarray(m, dtype=np.int64)
    out = np.empty(m.shape[:-1] + (len(moduli), m.shape[-1]), dtype=np.uint64)
    for i, q in enumerate(moduli):
        out[..., i, :] = np.mod(m, np.int64(q)).astype(np.uint64)   # numpy mod is non-negative for q > 0
    return out


def decode(coeffs: np.ndarray, N: int, scale: float) -> np.ndarray:
    """Centred integer coefficients -> complex slot vector z_j = (1/scale) * m(zeta^(5^j)).
    Host-stub arithmetic (not parity-relevant): z_t = sum_k (u_k zeta^k) omega^{tk}."""
    n = N // 2
    c = np.asarray(coeffs, dtype=np.float64)
    u = (c[:n] + 1j * c[n:]) * np.exp(1j * np.pi * np.arange(n) / N)
    v = np.fft.ifft(u) * n
    idx = np.array([(pow(5, j, 2 * N) - 1) // 4 for j in range(n)])
    return v[idx] / scale


# --------------------------------------------------------------------------- host stub: keys, encrypt, decrypt

def _rng(seed: int, *tag: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64([seed, *tag]))


def sample_ternary(rng, N: int) -> np.ndarray:
    return rng.integers(-1, 2, size=N, dtype=np.int64)


def sample_error(rng, N: int, sigma: float = 3.2) -> np.ndarray:
    """Rounded Gaussian, truncated at 6 sigma by resampling."""
    e = np.rint(rng.normal(0.0, sigma, size=N))
    bad = np.abs(e) > 6 * sigma
    while bad.any():
        e[bad] = np.rint(rng.normal(0.0, sigma, size=int(bad.sum())))
        bad = np.abs(e) > 6 * sigma
    return e.astype(np.int64)


def sample_uniform(rng, moduli, N: int) -> np.ndarray:
    return np.stack([rng.integers(0, q, size=N, dtype=np.uint64) for q in moduli])


def _add(a, b, q):
    return (a + b) % np.uint64(q)


def _sub(a, b, q):
    return (a + (np.uint64(q) - b)) % np.uint64(q)


def keygen(params: Params, seed: int) -> np.ndarray:
    """Secret key: uniform ternary coefficients."""
    return sample_ternary(_rng(seed, 1), params.N)


def galois_key(params: Params, s: np.ndarray, g: int, seed: int) -> np.ndarray:
    """Switching key from phi_g(s) to s.  For digit j:  a_j uniform over the extended basis,
    b_j = -a_j*s + e_j + [prime == q_j] * (P mod q_j) * phi_g(s).  Shape [r][2][r+1][N]."""
    N, r, basis = params.N, params.r, params.basis
    rng = _rng(seed, 2, g)
    s_res = to_residues(s, basis)                                   # [r+1][N]
    key = np.zeros((r, 2, r + 1, N), dtype=np.uint64)
    for j in range(r):
        a = sample_uniform(rng, basis, N)
        e = to_residues(sample_error(rng, N), basis)
        a_s = ring_mul(a, s_res, basis, params)
        for mi, m in enumerate(basis):
            b = _add(_sub(np.zeros(N, dtype=np.uint64), a_s[mi], m), e[mi], m)
            if mi == j:
                gs = automorphism(s_res[mi], g, m)
                acc = np.zeros(N, dtype=np.uint64)
                mul_acc(acc, gs, np.full(N, params.P % m, dtype=np.uint64), [m], N)
                b = _add(b, acc, m)
            key[j, 0, mi] = b
            key[j, 1, mi] = a[mi]
    return key


def encrypt(params: Params, s: np.ndarray, m: np.ndarray, seed: int, *tag: int) -> np.ndarray:
    """Symmetric encryption of integer coefficients m: c1 = a uniform, c0 = -a*s + e + m."""
    N, primes = params.N, params.primes
    rng = _rng(seed, 3, *tag)
    a = sample_uniform(rng, primes, N)
    e = to_residues(sample_error(rng, N), primes)
    mres = to_residues(m, primes)
    a_s = ring_mul(a, to_residues(s, primes), primes, params)
    ct = np.zeros((2, len(primes), N), dtype=np.uint64)
    for i, q in enumerate(primes):
        ct[0, i] = _add(_add(_sub(np.zeros(N, dtype=np.uint64), a_s[i], q), e[i], q), mres[i], q)
        ct[1, i] = a[i]
    return ct


def decrypt(params: Params, s: np.ndarray, ct: np.ndarray) -> np.ndarray:
    """c0 + c1*s modulo q_0 only, lifted to (-q_0/2, q_0/2]; valid while the message stays below
    q_0/2 in magnitude.  Returns int64 coefficients."""
    q0 = params.primes[0]
    c1s = ring_mul(ct[1, 0:1], to_residues(s, [q0]), [q0], params)[0]
    v = _add(ct[0, 0], c1s, q0).astype(np.int64)
    return np.where(v > (q0 - 1) // 2, v - q0, v)


# --------------------------------------------------------------------------- rotation (automorphism + key switch)

def mod_down(u: np.ndarray, params: Params) -> np.ndarray:
    """Divide by the special prime: u[r+1][N] over {q_0..q_L, P} -> v[r][N] with
    v_i = (u_i - t) * P^{-1} mod q_i, t = residue mod P lifted to the centred range."""
    N, P = params.N, params.P
    t = u[params.r]
    high = t > np.uint64((P - 1) // 2)
    v = np.zeros((params.r, N), dtype=np.uint64)
    for i, q in enumerate(params.primes):
        t_q = t % np.uint64(q)
        t_q = np.where(high, _sub(t_q, np.full(N, P % q, dtype=np.uint64), q), t_q)
        diff = _sub(u[i], t_q, q)
        p_inv = int(lib().orc_invmod(P % q, q))
        acc = np.zeros(N, dtype=np.uint64)
        mul_acc(acc, diff, np.full(N, p_inv, dtype=np.uint64), [q], N)
        v[i] = acc
    return v


def key_switch_ext(params: Params, c1: np.ndarray, g: int, key: np.ndarray, key_ntt=None) -> np.ndarray:
    """The key switch of phi_g(c1) from phi_g(s) to s, before the division by P:
    1. digit j = residues of c1 mod q_j as integers in [0, q_j), reduced into every modulus of the
       extended basis;  2. automorphism of each reduced digit;  3. (u0, u1) = sum_j digit_j *
       (key_j.b, key_j.a) in R_m for every m of the basis.  c1: [r][N]; returns u [2][r+1][N],
       coefficient domain, with u0 + u1*s = P * phi_g(c1) * phi_g(s) + small."""
    N, r, basis = params.N, params.r, params.basis
    assert c1.shape == (r, N)
    digits = np.zeros((r, r + 1, N), dtype=np.uint64)
    for j in range(r):
        for mi, m in enumerate(basis):
            digits[j, mi] = automorphism(c1[j] % np.uint64(m), g, m)
    moduli_d = basis * r
    dig_ntt = ntt(digits, moduli_d, params)
    if key_ntt is None:
        key_ntt = ntt(key, basis * (2 * r), params)
    u = np.zeros((2, r + 1, N), dtype=np.uint64)
    for comp in range(2):
        for j in range(r):
            mul_acc(u[comp], dig_ntt[j], key_ntt[j, comp], basis, N)
    return intt(u, basis * 2, params)


def rotate_galois(params: Params, ct: np.ndarray, g: int, key: np.ndarray, key_ntt=None) -> np.ndarray:
    """Apply X -> X^g to a full-level ciphertext and switch back to the secret key s.

    Steps 1-3: (u0, u1) = key_switch_ext(c1);  4. divide both by P (mod_down);
    5. result = (phi_g(c0) + v0, v1)."""
    N, r = params.N, params.r
    assert ct.shape == (2, r, N)
    u = key_switch_ext(params, ct[1], g, key, key_ntt)
    out = np.zeros_like(ct)
    v0, v1 = mod_down(u[0], params), mod_down(u[1], params)
    for i, q in enumerate(params.primes):
        out[0, i] = _add(automorphism(ct[0, i], g, q), v0[i], q)
        out[1, i] = v1[i]
    return out


def rotate(params: Params, ct: np.ndarray, steps: int, keys: dict) -> np.ndarray:
    """Left rotation of the slot vector by `steps` (identity when steps = 0 mod n)."""
    if steps % params.n == 0:
        return ct.copy()
    g = galois_element(steps, params.N)
    return rotate_galois(params, ct, g, keys[g])


def required_rotations(plan: Plan) -> list[int]:
    """Rotation amounts the BSGS evaluation needs: baby k*tau (k=1..b-1), giant j*b*tau (j=1..g-1)."""
    return [k * plan.tau for k in range(1, plan.b)] + [j * plan.b * plan.tau for j in range(1, plan.g)]


def fold_rotations(plan: Plan) -> list[int]:
    """Rotation amounts of the in-ciphertext fold of the tau partial sums: 1, 2, ..., tau/2."""
    return [1 << i for i in range(plan.tau.bit_length() - 1)]


def make_rotation_keys(params: Params, s: np.ndarray, plan: Plan, seed: int, extra_steps=()) -> dict:
    keys = {}
    for steps in list(required_rotations(plan)) + list(extra_steps):
        g = galois_element(steps, params.N)
        if g not in keys:
            keys[g] = galois_key(params, s, g, seed)
    return keys


# --------------------------------------------------------------------------- packing and the linear layer

def pack_input(x_chunk: np.ndarray, plan: Plan, n: int) -> np.ndarray:
    """Slot s = (rho*D + kappa)*tau + c holds x_chunk[(kappa + c*M) mod D]; x_chunk has D entries
    (zero-padded by the caller).  tau = 1 is the classical replicated layout x[s mod D]."""
    D, tau, M = plan.D, plan.tau, plan.M
    s = np.arange(n)
    c = s % tau
    kappa = (s // tau) % D
    return np.asarray(x_chunk, dtype=np.float64)[(kappa + c * M) % D]


def diagonal_slots(W: np.ndarray, plan: Plan, p: int, q: int, i: int, n: int) -> np.ndarray:
    """Generalised diagonal i of tile (p, q):  slot (rho, kappa, c) holds
    W[p*D + kappa, q*D + ((kappa + i + c*M) mod D)], zero outside the matrix."""
    D, tau, M = plan.D, plan.tau, plan.M
    d_out, d_in = W.shape
    s = np.arange(n)
    c = s % tau
    kappa = (s // tau) % D
    row = p * D + kappa
    col = q * D + (kappa + i + c * M) % D
    ok = (row < d_out) & (col < d_in)
    out = np.zeros(n, dtype=np.float64)
    out[ok] = W[row[ok], col[ok]].astype(np.float64)
    return out


def bsgs_plain_slots(W: np.ndarray, plan: Plan, p: int, q: int, j: int, k: int, n: int) -> np.ndarray:
    """Slot vector of Pt[p][q][j][k]: diagonal j*b+k rotated RIGHT by j*b*tau, so that the giant
    rotation applied after the inner sum brings it back into place."""
    d = diagonal_slots(W, plan, p, q, j * plan.b + k, n)
    return np.roll(d, j * plan.b * plan.tau)


def plain_slots(W: np.ndarray, plan: Plan, p: int, q: int, j: int, k: int, n: int) -> np.ndarray:
    """Slot vector of the plaintext Pt[p][q][j][k] that output ciphertext p multiplies into rot(ct_q, k*tau).
    Real packing: the pre-rotated diagonal of row block p.  Complex packing: row block 2p in the real parts
    and row block 2p+1 in the imaginary parts (zero where that block lies outside the matrix)."""
    if plan.pack == "complex":
        return bsgs_plain_slots(W, plan, 2 * p, q, j, k, n) + 1j * bsgs_plain_slots(W, plan, 2 * p + 1, q, j, k, n)
    return bsgs_plain_slots(W, plan, p, q, j, k, n)


def encode_weights(params: Params, plan: Plan, W: np.ndarray, blocks=None) -> dict:
    """Encoded diagonals of a projection W[d_out][d_in] (Sec. 4.2: pre-encoded weight diagonals kept
    as BSGS objects).  Returns {(p, q, j, k): uint64 [r][N] coefficient-domain plaintext} for the
    requested output ciphertexts p (all by default); with double hoisting the plaintexts are reduced
    modulo the special prime too: [r+1][N] over the extended basis."""
    plan.check(params.n)
    d_out, d_in = W.shape
    n_in, n_out = -(-d_in // plan.D), plan.n_out(d_out)
    blocks = range(n_out) if blocks is None else blocks
    idx = [(p, q, j, k) for p in blocks for q in range(n_in) for j in range(plan.g) for k in range(plan.b)]
    out = {}
    step = 256
    for lo in range(0, len(idx), step):
        part = idx[lo:lo + step]
        z = np.stack([plain_slots(W, plan, *t, params.n) for t in part])
        if plan.pack == "complex":
            m = encode_complex_batch(z, params.N, params.scale)
        else:
            m = encode_real_batch(z, params.N, params.scale)
        res = to_residues(m, params.basis if plan.hoist == "double" else params.primes)
        for t, pt in zip(part, res):
            out[t] = pt
    return out


def baby_rotations_ext(params: Params, plan: Plan, ct: np.ndarray, keys: dict, ks=None) -> dict:
    """Double hoisting: X[k] = rot(ct, k*tau) before its division by P, over the extended basis:
    (P * phi_k(c0) + u0, u1) with (u0, u1) = key_switch_ext(c1); for k = 0 simply (P * c0, P * c1), whose
    residue modulo P is zero.  Dividing X[k] by P (mod_down) gives exactly the rotated ciphertext.
    Returns {k: uint64 [2][r+1][N]}, coefficient domain."""
    N, r, basis = params.N, params.r, params.basis
    ks = range(plan.b) if ks is None else ks
    out = {}
    for k in ks:
        steps = k * plan.tau
        X = np.zeros((2, r + 1, N), dtype=np.uint64)
        if steps % params.n == 0:
            parts, u = (ct[0], ct[1]), None
        else:
            g = galois_element(steps, N)
            u = key_switch_ext(params, ct[1], g, keys[g])
            parts = (np.stack([automorphism(ct[0, i], g, qi) for i, qi in enumerate(params.primes)]), None)
        for comp in range(2):
            for i, qi in enumerate(params.primes):
                if parts[comp] is not None:
                    mul_acc(X[comp, i], parts[comp][i], np.full(N, params.P % qi, dtype=np.uint64), [qi], N)
            if u is not None:
                for mi, m in enumerate(basis):
                    X[comp, mi] = _add(X[comp, mi], u[comp, mi], m)
        out[k] = X
    return out


def baby_rotations(params: Params, plan: Plan, ct: np.ndarray, keys: dict, ks=None) -> dict:
    """X[k] = rot(ct, k*tau) for the requested baby steps k (all of 0..b-1 by default)."""
    ks = range(plan.b) if ks is None else ks
    return {k: rotate(params, ct, k * plan.tau, keys) for k in ks}


def inner_sum(params: Params, plan: Plan, Xh: list, encoded: dict, p: int, j: int) -> np.ndarray:
    """A[p][j] = sum_q sum_{k<b} Pt[p][q][j][k] (*) X[q][k], both components, every ciphertext
    prime; Xh[q][k] are the baby-step ciphertexts in the evaluation domain.  Returns the
    coefficient-domain ciphertext [2][r][N].  With double hoisting the sum runs over the extended
    basis (Xh and the plaintexts carry the residue modulo P) and is divided by P once at the end."""
    N, r = params.N, params.r
    moduli = params.basis if plan.hoist == "double" else params.primes
    acc = np.zeros((2, len(moduli), N), dtype=np.uint64)
    for q in range(len(Xh)):
        pts = np.stack([encoded[(p, q, j, k)] for k in range(plan.b)])
        pth = ntt(pts, moduli * plan.b, params)
        for k in range(plan.b):
            for comp in range(2):
                mul_acc(acc[comp], pth[k], Xh[q][k][comp], moduli, N)
    A = intt(acc, moduli * 2, params)
    if plan.hoist == "double":
        A = np.stack([mod_down(A[0], params), mod_down(A[1], params)])
    return A


def linear(params: Params, plan: Plan, cts: list, W: np.ndarray, keys: dict, blocks=None, encoded=None,
           X=None) -> dict:
    """Encrypted matrix-vector product (Sec. 4.2 "BSGS matrix-vector multiply"; Alg. 3 FHE_Linear).

    cts[q] encrypts pack_input(x[q*D:(q+1)*D]).  For output block p:
        Y_p = sum_{j<g} rot( sum_q sum_{k<b} Pt[p][q][j][k] (*) rot(ct_q, k*tau), j*b*tau )
    where (*) multiplies both ciphertext components by the plaintext in R_{q_i}.  Output level is
    unchanged, scale multiplies.  Returns {p: ciphertext}.  X, when given, is the list over q of
    baby_rotations(params, plan, cts[q], keys) computed by an earlier call for the same inputs (several
    projections that read the same ciphertexts need them only once)."""
    N, r, primes, basis = params.N, params.r, params.primes, params.basis
    d_out, d_in = W.shape
    n_in, n_out = -(-d_in // plan.D), plan.n_out(d_out)
    assert len(cts) == n_in
    blocks = list(range(n_out) if blocks is None else blocks)
    if encoded is None:
        encoded = encode_weights(params, plan, W, blocks)
    # baby steps: X[q][k] = rot(ct_q, k*tau) (double hoisting: before its division by P, over the extended
    # basis), then to the evaluation domain for the products
    if X is None:
        rot_fn = baby_rotations_ext if plan.hoist == "double" else baby_rotations
        X = [rot_fn(params, plan, cts[q], keys) for q in range(n_in)]
    assert len(X) == n_in
    x_moduli = basis if plan.hoist == "double" else primes
    Xh = [[ntt(X[q][k], x_moduli * 2, params) for k in range(plan.b)] for q in range(n_in)]
    out = {}
    for p in blocks:
        Y = np.zeros((2, r, N), dtype=np.uint64)
        if plan.moddown == "per_output":
            # giant steps j >= 1: key-switch results summed over j in the extended basis, the rotated c0
            # parts summed beside them; one division by P per component at the end
            U = np.zeros((2, r + 1, N), dtype=np.uint64)
            for j in range(plan.g):
                A = inner_sum(params, plan, Xh, encoded, p, j)
                steps = j * plan.b * plan.tau
                if steps % params.n == 0:
                    rot_c0, u = A[0], None
                    for i, qi in enumerate(primes):
                        Y[1, i] = _add(Y[1, i], A[1, i], qi)
                else:
                    g = galois_element(steps, N)
                    u = key_switch_ext(params, A[1], g, keys[g])
                    rot_c0 = np.stack([automorphism(A[0, i], g, qi) for i, qi in enumerate(primes)])
                    for comp in range(2):
                        for mi, m in enumerate(basis):
                            U[comp, mi] = _add(U[comp, mi], u[comp, mi], m)
                for i, qi in enumerate(primes):
                    Y[0, i] = _add(Y[0, i], rot_c0[i], qi)
            if plan.g > 1:
                v0, v1 = mod_down(U[0], params), mod_down(U[1], params)
                for i, qi in enumerate(primes):
                    Y[0, i] = _add(Y[0, i], v0[i], qi)
                    Y[1, i] = _add(Y[1, i], v1[i], qi)
        else:
            for j in range(plan.g):
                A = inner_sum(params, plan, Xh, encoded, p, j)
                A = rotate(params, A, j * plan.b * plan.tau, keys)
                for comp in range(2):
                    for i, qi in enumerate(primes):
                        Y[comp, i] = _add(Y[comp, i], A[comp, i], qi)
        out[p] = Y
    return out


def rescale(params: Params, ct: np.ndarray) -> np.ndarray:
    """Drop the last prime q_L of a level-L ciphertext: c'_i = (c_i - centred(c_L)) * q_L^{-1} mod q_i,
    which equals round(c / q_L) (Sec. 2.1 rescaling).  [2][L+1][N] -> [2][L][N]."""
    lvl = ct.shape[1]
    primes = params.primes[:lvl]
    qL = primes[-1]
    N = params.N
    out = np.zeros((2, lvl - 1, N), dtype=np.uint64)
    for comp in range(2):
        t = ct[comp, lvl - 1]
        high = t > np.uint64((qL - 1) // 2)
        for i, q in enumerate(primes[:-1]):
            t_q = t % np.uint64(q)
            t_q = np.where(high, _sub(t_q, np.full(N, qL % q, dtype=np.uint64), q), t_q)
            diff = _sub(ct[comp, i], t_q, q)
            inv = int(lib().orc_invmod(qL % q, q))
            acc = np.zeros(N, dtype=np.uint64)
            mul_acc(acc, diff, np.full(N, inv, dtype=np.uint64), [q], N)
            out[comp, i] = acc
    return out


def fold_output(slots: np.ndarray, plan: Plan, p: int, d_out: int) -> np.ndarray:
    """Host-side fold of the tau partial sums of output ciphertext p: y[p*D + kappa] = sum_c slot((0, kappa, c)).
    Complex packing: the real parts give rows 2p*D + kappa, the imaginary parts rows (2p+1)*D + kappa; the
    result is the rows_per_ct rows of ciphertext p in order (cut at d_out)."""
    D, tau = plan.D, plan.tau
    s = np.asarray(slots)[:D * tau]
    part = s.real.reshape(D, tau).sum(axis=1)
    if plan.pack == "complex":
        part = np.concatenate([part, s.imag.reshape(D, tau).sum(axis=1)])
    rows = min(plan.rows_per_ct, d_out - p * plan.rows_per_ct)
    return part[:rows]


def fold_in_ciphertext(params: Params, plan: Plan, ct: np.ndarray, keys: dict) -> np.ndarray:
    """The variant of the output stage that sums the tau partial results inside the ciphertext (the
    packing of Sec. 4.2 leaves slot (rho, kappa, c) with the partial dot product over column class c):
        for i = 0 .. log2(tau) - 1:  ct <- ct + rot(ct, 2^i)
    after which slot (0, kappa, 0) holds the sum over all c, i.e. the complete dot product of row kappa.
    Costs log2(tau) key switches per output ciphertext; level and scale are unchanged.  The default path
    leaves this sum to the host after decryption (fold_output)."""
    assert plan.tau & (plan.tau - 1) == 0, "the fold needs a power-of-two tau"
    q = np.array(params.primes, dtype=np.uint64).reshape(1, -1, 1)
    out = ct.copy()
    for steps in fold_rotations(plan):
        rot = rotate(params, out, steps, keys)
        t = out + rot                       # residues are below 2^60: no wrap-around in 64 bits
        out = np.where(t >= q, t - q, t).astype(np.uint64)
    return out


def folded_output(slots: np.ndarray, plan: Plan, p: int, d_out: int) -> np.ndarray:
    """Reads the complete dot products of a ciphertext folded by fold_in_ciphertext: slot (0, kappa, 0)."""
    D, tau = plan.D, plan.tau
    s = np.asarray(slots)[:D * tau:tau]
    part = np.concatenate([s.real, s.imag]) if plan.pack == "complex" else s.real
    rows = min(plan.rows_per_ct, d_out - p * plan.rows_per_ct)
    return part[:rows]


# --------------------------------------------------------------------------- convenience for tests / smoke

def encrypt_vector(params: Params, plan: Plan, s: np.ndarray, x: np.ndarray, seed: int) -> list:
    """Pack x (length d_in) chunk by chunk and encrypt: one ciphertext per input chunk of D."""
    D = plan.D
    n_in = -(-len(x) // D)
    xp = np.zeros(n_in * D)
    xp[:len(x)] = x
    cts = []
    for q in range(n_in):
        z = pack_input(xp[q * D:(q + 1) * D], plan, params.n)
        m = encode_coeffs(z, params.N, params.scale)
        cts.append(encrypt(params, s, m, seed, q))
    return cts


def decrypt_output(params: Params, plan: Plan, s: np.ndarray, ct: np.ndarray, scale: float, p: int, d_out: int) -> np.ndarray:
    m = decrypt(params, s, ct)
    return fold_output(decode(m, params.N, scale), plan, p, d_out)
