/*
 * CPU oracle for the accelerator-side CKKS linear layer: per-polynomial primitives.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the slow, plain reference that the CUDA library
 * is compared against.  It shares no code, header, table or constant generator with the CUDA
 * path, and the product path never calls it.
 *
 * What is here (each routine cites the passage of the paper, or the standard definition the
 * paper relies on, that it follows):
 *   - modular arithmetic on 64-bit residues through unsigned __int128 and the % operator,
 *   - prime search and primitive roots for the ring R_q = Z_q[X]/(X^N + 1)  (paper Sec. 2.1),
 *   - the negacyclic number-theoretic transform in its textbook form: twist by psi^k, then a
 *     radix-2 cyclic transform with omega = psi^2, output in natural order
 *     (the "NTT kernels" of Sec. 4.2 are a faster route to this same map),
 *   - the ring automorphism a(X) -> a(X^g) in the coefficient domain (rotations, Sec. 2.1),
 *   - the CKKS canonical-embedding encoder as a fixed fp64 arithmetic DAG (Sec. 2.1 slots;
 *     Sec. 4.2 "pre-encodes the weight matrix diagonals").
 *
 * The algorithmic steps of the linear layer (key switching, diagonal matvec, rescale) are
 * composed from these in oracle/ckks.py so they can be read next to the method's description.
 *
 * Build: gcc -O2 -fopenmp -ffp-contract=off -shared -fPIC (see oracle/build.py).
 */
#include <math.h>
#ifdef _OPENMP
#include <omp.h>
#endif
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

typedef uint64_t u64;
typedef int64_t i64;
typedef uint32_t u32;
typedef unsigned __int128 u128;

/* ---------------------------------------------------------------- modular arithmetic */

u64 orc_mulmod(u64 a, u64 b, u64 q) { return (u64)(((u128)a * b) % q); }
u64 orc_addmod(u64 a, u64 b, u64 q) { return (u64)(((u128)a + b) % q); }
u64 orc_submod(u64 a, u64 b, u64 q) { return (u64)(((u128)a + (q - b % q)) % q); }

u64 orc_powmod(u64 a, u64 e, u64 q) {
    u64 result = 1 % q;
    a %= q;
    while (e) {
        if (e & 1) result = orc_mulmod(result, a, q);
        a = orc_mulmod(a, a, q);
        e >>= 1;
    }
    return result;
}

u64 orc_invmod(u64 a, u64 q) { return orc_powmod(a, q - 2, q); } /* q prime (Fermat) */

/* Deterministic Miller-Rabin; the first twelve primes as bases decide every n < 2^64. */
int orc_is_prime(u64 n) {
    static const u64 bases[12] = {2, 3, 5, 7, 11, 13, 17, 19, 23, 29, 31, 37};
    if (n < 2) return 0;
    for (int i = 0; i < 12; i++) {
        if (n == bases[i]) return 1;
        if (n % bases[i] == 0) return 0;
    }
    u64 d = n - 1;
    int s = 0;
    while ((d & 1) == 0) { d >>= 1; s++; }
    for (int i = 0; i < 12; i++) {
        u64 x = orc_powmod(bases[i], d, n);
        if (x == 1 || x == n - 1) continue;
        int witness = 1;
        for (int k = 1; k < s; k++) {
            x = orc_mulmod(x, x, n);
            if (x == n - 1) { witness = 0; break; }
        }
        if (witness) return 0;
    }
    return 1;
}

/* The `count` largest primes p < below with p = 1 (mod two_n), in descending order.
 * These are the NTT-friendly moduli of the RNS chain (Sec. 4.2 "coefficient-modulus primes"). */
int orc_find_primes(u64 below, u64 two_n, int count, u64* out) {
    u64 c = ((below - 2) / two_n) * two_n + 1; /* largest value = 1 mod two_n that is < below */
    int found = 0;
    while (found < count && c > two_n) {
        if (orc_is_prime(c)) out[found++] = c;
        c -= two_n;
    }
    return found;
}

/* A primitive 2N-th root of unity mod q: psi = x^((q-1)/2N) for the smallest x >= 2 that gives
 * psi^N = -1.  Which root is used never shows in a coefficient-form result. */
u64 orc_primitive_root_2n(u64 q, u32 N) {
    u64 e = (q - 1) / (2 * (u64)N);
    for (u64 x = 2; x < q; x++) {
        u64 psi = orc_powmod(x, e, q);
        if (orc_powmod(psi, N, q) == q - 1) return psi;
    }
    return 0;
}

/* ---------------------------------------------------------------- negacyclic NTT */

static u32 bit_reverse(u32 x, int bits) {
    u32 r = 0;
    for (int i = 0; i < bits; i++) { r = (r << 1) | (x & 1); x >>= 1; }
    return r;
}

static int log2_exact(u32 n) {
    int l = 0;
    while ((1u << l) < n) l++;
    return l;
}

/* In-place radix-2 decimation-in-time cyclic transform A_i = sum_k a_k w^{ik}, natural order in
 * and out; wpow[t] = w^t for t < N/2. */
static void cyclic_fft(u64* a, u32 N, u64 q, const u64* wpow) {
    int bits = log2_exact(N);
    for (u32 i = 0; i < N; i++) {
        u32 j = bit_reverse(i, bits);
        if (i < j) { u64 t = a[i]; a[i] = a[j]; a[j] = t; }
    }
    for (u32 len = 2; len <= N; len <<= 1) {
        u32 half = len >> 1, step = N / len;
        for (u32 start = 0; start < N; start += len) {
            for (u32 j = 0; j < half; j++) {
                u64 u = a[start + j];
                u64 v = orc_mulmod(a[start + j + half], wpow[j * step], q);
                a[start + j] = orc_addmod(u, v, q);
                a[start + j + half] = orc_submod(u, v, q);
            }
        }
    }
}

/* Forward negacyclic NTT of `count` polynomials, polynomial b modulo q[b] with 2N-th root psi[b]:
 *   out[i] = a(psi^{2i+1}) = sum_k a_k psi^{(2i+1)k},  i = 0..N-1 (natural order).
 * Evaluating at the odd powers of psi is what turns multiplication modulo X^N + 1 into a
 * pointwise product. */
void orc_ntt_batch(u64* a, u32 count, u32 N, const u64* q, const u64* psi) {
#pragma omp parallel for schedule(dynamic, 1)
    for (u32 b = 0; b < count; b++) {
        u64* p = a + (size_t)b * N;
        u64 qq = q[b];
        u64* wpow = (u64*)malloc(sizeof(u64) * (N / 2 + 1));
        u64 w = orc_mulmod(psi[b], psi[b], qq);
        u64 cur = 1, tw = 1;
        for (u32 k = 0; k < N; k++) { /* twist a_k <- a_k psi^k */
            p[k] = orc_mulmod(p[k] % qq, tw, qq);
            tw = orc_mulmod(tw, psi[b], qq);
        }
        for (u32 t = 0; t < N / 2; t++) { wpow[t] = cur; cur = orc_mulmod(cur, w, qq); }
        cyclic_fft(p, N, qq, wpow);
        free(wpow);
    }
}

/* Inverse of orc_ntt_batch: a_k = N^{-1} psi^{-k} sum_i A_i w^{-ik}. */
void orc_intt_batch(u64* a, u32 count, u32 N, const u64* q, const u64* psi) {
#pragma omp parallel for schedule(dynamic, 1)
    for (u32 b = 0; b < count; b++) {
        u64* p = a + (size_t)b * N;
        u64 qq = q[b];
        u64* wpow = (u64*)malloc(sizeof(u64) * (N / 2 + 1));
        u64 psi_inv = orc_invmod(psi[b], qq);
        u64 w_inv = orc_mulmod(psi_inv, psi_inv, qq);
        u64 cur = 1;
        for (u32 t = 0; t < N / 2; t++) { wpow[t] = cur; cur = orc_mulmod(cur, w_inv, qq); }
        for (u32 k = 0; k < N; k++) p[k] %= qq;
        cyclic_fft(p, N, qq, wpow);
        u64 n_inv = orc_invmod(N % qq, qq);
        u64 tw = n_inv;
        for (u32 k = 0; k < N; k++) {
            p[k] = orc_mulmod(p[k], tw, qq);
            tw = orc_mulmod(tw, psi_inv, qq);
        }
        free(wpow);
    }
}

/* Direct O(N^2) evaluation out[i] = a(psi^{2i+1}); only for pinning the fast transform. */
void orc_ntt_direct(const u64* a, u64* out, u32 N, u64 q, u64 psi) {
    for (u32 i = 0; i < N; i++) {
        u64 x = orc_powmod(psi, 2 * (u64)i + 1, q);
        u64 acc = 0, xp = 1;
        for (u32 k = 0; k < N; k++) {
            acc = orc_addmod(acc, orc_mulmod(a[k] % q, xp, q), q);
            xp = orc_mulmod(xp, x, q);
        }
        out[i] = acc;
    }
}

/* Schoolbook product in Z_q[X]/(X^N + 1): X^N = -1 folds the upper half back with a sign. */
void orc_negacyclic_schoolbook(const u64* a, const u64* b, u64* out, u32 N, u64 q) {
    for (u32 k = 0; k < N; k++) out[k] = 0;
    for (u32 i = 0; i < N; i++) {
        for (u32 j = 0; j < N; j++) {
            u64 prod = orc_mulmod(a[i] % q, b[j] % q, q);
            u32 k = i + j;
            if (k < N) out[k] = orc_addmod(out[k], prod, q);
            else out[k - N] = orc_submod(out[k - N], prod, q);
        }
    }
}

/* ---------------------------------------------------------------- pointwise ring arithmetic */

/* acc[b][i] = (acc[b][i] + x[b][i] * y[b][i]) mod q[b] for `count` polynomials. */
void orc_mul_acc_batch(u64* acc, const u64* x, const u64* y, u32 count, u32 N, const u64* q) {
#pragma omp parallel for schedule(static)
    for (u32 b = 0; b < count; b++) {
        u64 qq = q[b];
        size_t o = (size_t)b * N;
        for (u32 i = 0; i < N; i++)
            acc[o + i] = orc_addmod(acc[o + i], orc_mulmod(x[o + i], y[o + i], qq), qq);
    }
}

/* ---------------------------------------------------------------- automorphism */

/* Coefficient-domain automorphism out(X) = a(X^g) in Z_q[X]/(X^N + 1), g odd:
 * coefficient i moves to i*g mod 2N, and picks up a minus sign when that lands in [N, 2N)
 * because X^N = -1.  With g = 5^r mod 2N this rotates the CKKS slot vector left by r. */
void orc_automorphism(const u64* a, u64* out, u32 N, u64 g, u64 q) {
    u64 two_n = 2 * (u64)N;
    for (u32 i = 0; i < N; i++) {
        u64 k = ((u64)i * (g % two_n)) % two_n;
        u64 v = a[i] % q;
        if (k < N) out[k] = v;
        else out[k - N] = (v == 0) ? 0 : q - v;
    }
}

/* ---------------------------------------------------------------- CKKS encoder (fp64 DAG) */

/*
 * Inverse canonical embedding of a slot vector z in C^n (n = N/2) to integer coefficients
 * (Sec. 2.1: N/2 complex slots per ring element).  Slot j sits at the evaluation point
 * zeta^{5^j}, zeta = exp(i pi / N).  Because zeta_j^n = i, the polynomial splits as
 * m_lo(X) + X^n m_hi(X) with u_k = m_k + i m_{k+n}, and
 *      u_k = (1/n) sum_j z_j zeta^{-5^j k}
 *          = (zeta^{-k} / n) * sum_t v[t] exp(-2 pi i t k / n),     v[(5^j mod 2N - 1)/4] = z_j.
 * m_k = round(scale * Re u_k), m_{k+n} = round(scale * Im u_k).
 *
 * The paper does not fix a floating-point order; this routine fixes one so that results can be
 * compared bit for bit:  (1) place z_j at index (5^j mod 2N - 1)/4;  (2) bit-reverse, then radix-2
 * decimation-in-time stages len = 2, 4, ..., n with butterfly (a, b) -> (a + w b, a - w b),
 * w = T[j n / len], T[t] = (cos(2 pi t / n), -sin(2 pi t / n));  (3) multiply by
 * Z[k] = (cos(pi k / N), -sin(pi k / N));  (4) multiply both parts by scale / n;  (5) round to
 * nearest, ties to even.  Complex products are (br wr - bi wi, br wi + bi wr) with every product
 * and every sum rounded separately (no fused multiply-add: build with -ffp-contract=off).
 * Tables come from this machine's libm at the arguments (double)t * (2 pi / n) and
 * (double)k * (pi / N).
 *
 * Returns 0, or -1 if some |coefficient| >= 2^62.
 */
static const double ORC_PI = 3.141592653589793238462643383279502884;

int orc_encode_slots(const double* zre, const double* zim, u32 N, double scale, i64* m) {
    u32 n = N / 2;
    int bits = log2_exact(n);
    u64 two_n = 2 * (u64)N;
    double* ar = (double*)calloc(n, sizeof(double));
    double* ai = (double*)calloc(n, sizeof(double));
    double* vr = (double*)calloc(n, sizeof(double));
    double* vi = (double*)calloc(n, sizeof(double));
    u32 nt = n / 2 > 0 ? n / 2 : 1;
    double* Tr = (double*)malloc(sizeof(double) * nt);
    double* Ti = (double*)malloc(sizeof(double) * nt);
    const double two_pi_over_n = (2.0 * ORC_PI) / (double)n;
    const double pi_over_N = ORC_PI / (double)N;
    for (u32 t = 0; t < nt; t++) {
        double ang = (double)t * two_pi_over_n;
        Tr[t] = cos(ang);
        Ti[t] = -sin(ang);
    }
    /* (1) slot j -> index (5^j mod 2N - 1)/4 */
    u64 pw = 1;
    for (u32 j = 0; j < n; j++) {
        u32 idx = (u32)((pw - 1) / 4);
        vr[idx] = zre[j];
        vi[idx] = zim ? zim[j] : 0.0;
        pw = (pw * 5) % two_n;
    }
    /* (2) bit reversal, then decimation-in-time stages */
    for (u32 i = 0; i < n; i++) {
        u32 j = bit_reverse(i, bits);
        ar[j] = vr[i];
        ai[j] = vi[i];
    }
    for (u32 len = 2; len <= n; len <<= 1) {
        u32 half = len >> 1, step = n / len;
        for (u32 start = 0; start < n; start += len) {
            for (u32 j = 0; j < half; j++) {
                double wr = Tr[j * step], wi = Ti[j * step];
                double br = ar[start + j + half], bi = ai[start + j + half];
                double p1 = br * wr, p2 = bi * wi, p3 = br * wi, p4 = bi * wr;
                double tr = p1 - p2;
                double ti = p3 + p4;
                double xr = ar[start + j], xi = ai[start + j];
                ar[start + j] = xr + tr;
                ai[start + j] = xi + ti;
                ar[start + j + half] = xr - tr;
                ai[start + j + half] = xi - ti;
            }
        }
    }
    /* (3) twist, (4) scale, (5) round */
    double s = scale / (double)n;
    int status = 0;
    for (u32 k = 0; k < n; k++) {
        double ang = (double)k * pi_over_N;
        double zr = cos(ang), zi = -sin(ang);
        double p1 = ar[k] * zr, p2 = ai[k] * zi, p3 = ar[k] * zi, p4 = ai[k] * zr;
        double ur = p1 - p2;
        double ui = p3 + p4;
        double cr = rint(ur * s); /* default rounding mode: to nearest, ties to even */
        double ci = rint(ui * s);
        if (!(fabs(cr) < 4611686018427387904.0) || !(fabs(ci) < 4611686018427387904.0)) status = -1;
        else { m[k] = (i64)cr; m[k + n] = (i64)ci; }
    }
    free(ar); free(ai); free(vr); free(vi); free(Tr); free(Ti);
    return status;
}

/* Batch of real slot vectors z[count][n] -> coefficients m[count][N]. */
int orc_encode_real_batch(const double* z, u32 count, u32 N, double scale, i64* m) {
    int status = 0;
    u32 n = N / 2;
#pragma omp parallel for schedule(dynamic, 1)
    for (u32 b = 0; b < count; b++) {
        int s = orc_encode_slots(z + (size_t)b * n, NULL, N, scale, m + (size_t)b * N);
        if (s) {
#pragma omp atomic write
            status = s;
        }
    }
    return status;
}

/* Batch of complex slot vectors (zre[count][n], zim[count][n]) -> coefficients m[count][N]. */
int orc_encode_complex_batch(const double* zre, const double* zim, u32 count, u32 N, double scale, i64* m) {
    int status = 0;
    u32 n = N / 2;
#pragma omp parallel for schedule(dynamic, 1)
    for (u32 b = 0; b < count; b++) {
        int s = orc_encode_slots(zre + (size_t)b * n, zim + (size_t)b * n, N, scale, m + (size_t)b * N);
        if (s) {
#pragma omp atomic write
            status = s;
        }
    }
    return status;
}

int orc_num_threads(void) {
    int n = 1;
#ifdef _OPENMP
    n = omp_get_max_threads();
#endif
    return n;
}
