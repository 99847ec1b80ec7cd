// Shared device-side types and modular arithmetic for the CKKS linear-layer kernels (sm_100a).
//
// Residues are 64-bit words modulo primes q < 2^60, so lazily reduced values up to 4q fit a word
// and a sum of up to 2^8 products of two residues fits 128 bits.
#pragma once
#include <cstdint>
#include <cuda_runtime.h>

namespace bf {

typedef uint64_t u64;
typedef int64_t i64;
typedef uint32_t u32;

constexpr int MAX_MODULI = 16;    // ciphertext primes + the special prime
constexpr int MAX_ROT_BATCH = 64; // rotations handled by one key-switch launch

// Per-ring constants handed to every kernel by value (lands in the constant bank).
// Modulus index r is the special prime P; 0..r-1 are the ciphertext primes q_0..q_L.
struct RingDev {
    u32 N, logN, r;
    u64 q[MAX_MODULI];
    u64 mu[MAX_MODULI];          // floor(2^64 / q)
    u64 c64[MAX_MODULI];         // 2^64 mod q
    u64 c64s[MAX_MODULI];        // Shoup companion of c64
    u64 ninv[MAX_MODULI];        // N^{-1} mod q
    u64 ninvs[MAX_MODULI];
    u64 pinv[MAX_MODULI];        // P^{-1} mod q_i (i < r)
    u64 pinvs[MAX_MODULI];
    u64 pmod[MAX_MODULI];        // P mod q_i
    const ulonglong2* tw_fwd;    // [r+1][N]  (psi^brev(k), Shoup companion), merged Cooley-Tukey order
    const ulonglong2* tw_inv;    // [r+1][N]  inverses of the above, for the Gentleman-Sande inverse
};

// floor(x * w / 2^64)-based modular multiplication by a constant w with precomputed
// ws = floor(w * 2^64 / q).  Valid for any 64-bit x; result in [0, 2q).
__device__ __forceinline__ u64 mul_shoup_lazy(u64 x, u64 w, u64 ws, u64 q) {
    u64 hi = __umul64hi(x, ws);
    return x * w - hi * q;
}

__device__ __forceinline__ u64 mul_shoup(u64 x, u64 w, u64 ws, u64 q) {
    u64 v = mul_shoup_lazy(x, w, ws, q);
    return v >= q ? v - q : v;
}

// x mod q for any 64-bit x, mu = floor(2^64 / q).  The quotient estimate is short by at most one.
__device__ __forceinline__ u64 barrett64(u64 x, u64 q, u64 mu) {
    u64 v = x - __umul64hi(x, mu) * q;
    return v >= q ? v - q : v;
}

// (hi * 2^64 + lo) mod q:  hi * (2^64 mod q) by a Shoup product, lo by Barrett, then fold.
__device__ __forceinline__ u64 reduce128(u64 hi, u64 lo, u64 q, u64 mu, u64 c64, u64 c64s) {
    u64 a = mul_shoup_lazy(hi, c64, c64s, q);        // [0, 2q)
    u64 b = lo - __umul64hi(lo, mu) * q;             // [0, 2q)
    u64 v = a + b;                                   // [0, 4q)
    if (v >= 2 * q) v -= 2 * q;
    if (v >= q) v -= q;
    return v;
}

// acc (128-bit, as hi:lo) += a * b
__device__ __forceinline__ void mac128(u64& hi, u64& lo, u64 a, u64 b) {
    u64 pl = a * b;
    u64 ph = __umul64hi(a, b);
    lo += pl;
    hi += ph + (lo < pl ? 1ull : 0ull);
}

__device__ __forceinline__ u64 add_mod(u64 a, u64 b, u64 q) {
    u64 v = a + b;
    return v >= q ? v - q : v;
}

__device__ __forceinline__ u64 sub_mod(u64 a, u64 b, u64 q) {
    return a >= b ? a - b : a + q - b;
}

// How the first pass of a transform reads its input.
enum LoadMode : int {
    LOAD_PLAIN = 0,     // residues already modulo the target prime, in [0, q)
    LOAD_REDUCE = 1,    // any 64-bit non-negative integer (e.g. a residue of another prime): x mod q
    LOAD_I64 = 2,       // signed 64-bit integer coefficient: x mod q in [0, q)
    LOAD_CENTRED = 3,   // residue t in [0, M) of modulus M: centred lift to (-M/2, M/2], then mod q
};

// A batch of equally sized polynomials addressed as (outer index o, slot m):
//   source  = src + o*src_so + m*src_sm      destination = dst + o*dst_so + m*dst_sm
//   modulus index of polynomial (o, m) = mod0 + m*mod_step
// blockIdx.y enumerates o*n_m + m.
struct PolyBatch {
    const void* src;
    u64* dst;
    long long src_so, src_sm, dst_so, dst_sm;
    u32 n_m, mod0, mod_step;
    u64 lift_mod;                 // LOAD_CENTRED: the modulus M the source residues live in
};

}  // namespace bf
