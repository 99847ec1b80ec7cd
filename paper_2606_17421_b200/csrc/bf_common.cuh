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
constexpr int ENC_CONSTS = 5;
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
    u64 qneg[MAX_MODULI];        // -q^{-1} mod 2^64 (Montgomery reduction)
    u64 ninv_m[MAX_MODULI];      // N^{-1} * 2^{-64} mod q: inverse transform that also leaves Montgomery form
    u64 ninv_ms[MAX_MODULI];
    u32 fp_ok[MAX_MODULI];       // modulus below 2^50: its transforms run in fp64 (every value an exact integer below
                                 //   2^53) and its twiddle tables hold the bits of ((double)w, (double)w / q)
    double qd[MAX_MODULI];       // (double)q
    double qinv_d[MAX_MODULI];   // 1.0 / q
    double ninv_d[MAX_MODULI], ninv_q[MAX_MODULI];     // (double)N^{-1} and N^{-1} / q
    double ninvm_d[MAX_MODULI], ninvm_q[MAX_MODULI];   // the same for N^{-1} * 2^{-64} (leaving Montgomery form)
    double c30_d[MAX_MODULI], c30_q[MAX_MODULI];       // (double)(2^30 mod q) and that over q
    double k59_d[MAX_MODULI];    // 2q - (2^59 mod q): undoes the offset of a stored centred lift, keeps it positive
    double pinv_d[MAX_MODULI], pinv_q[MAX_MODULI];     // (double)(P^{-1} mod q_i) and that over q_i (i < r)
    // encoder output (signed 64-bit coefficients) into Montgomery form on the fp64 path: the word is
    // (hi' - 2^31) 2^32 + lo, so times 2^64 it is  hi' (2^96 mod q) + lo (2^64 mod q) - (2^127 mod q).
    // Five doubles per prime, in device memory (kernel parameters stay small): (double)(2^96 mod q), that
    // over q, (double)(2^64 mod q), that over q, and the centred residue of -2^127 (plus 2q for primes of
    // 2^41 or more, whose values stay non-negative)
    const double* enc_consts;    // [r+1][ENC_CONSTS]
    const ulonglong2* tw_fwd;    // [r+1][N]  (psi^brev(k), companion), merged Cooley-Tukey order
    const ulonglong2* tw_inv;    // [r+1][N]  inverses of the above, for the Gentleman-Sande inverse
};

// floor(x * w / 2^64)-based modular multiplication by a constant w with precomputed
// ws = floor(w * 2^64 / q).  Valid for any 64-bit x; result in [0, 2q).
__device__ __forceinline__ u64 mul_shoup_lazy(u64 x, u64 w, u64 ws, u64 q) {
    u64 hi = __umul64hi(x, ws);
    return x * w - hi * q;
}

// First statement of every kernel of a linear-layer call.  Lets the next kernel of the stream be scheduled
// as soon as all blocks of this one have started, then waits until the previous kernel has completed and
// flushed its writes.  A no-op when the launch carries no programmatic dependency.
__device__ __forceinline__ void grid_dependency_enter() {
    asm volatile("griddepcontrol.launch_dependents;");
    asm volatile("griddepcontrol.wait;" ::: "memory");
}

// ---- fp64 arithmetic for primes q < 2^50.  B200 issues fp64 FMAs at the rate of 32-bit integer
// multiply-adds, on a pipe of its own, while a 64x64-bit high product costs about ten integer
// multiply-add slots; and integers below 2^53 are exact in fp64.
__device__ __forceinline__ double u2d(u64 x) {          // exact for x < 2^52
    return __longlong_as_double((long long)(x | 0x4330000000000000ull)) - 4503599627370496.0;
}
__device__ __forceinline__ u64 d2u(double d) {          // d an integer in [0, 2^52)
    return (u64)__double_as_longlong(d + 4503599627370496.0) - 0x4330000000000000ull;
}
// x * w - round(x * w / q) * q for a non-negative integer-valued x and a constant 0 <= w < q given as
// (double)w and wq = (double)w / q.  ph + pl = x*w exactly (FMA); the quotient estimate is within
// 1/2 + x * 2^-52 of x*w/q; ph - qh*q is an integer far below 2^53 and therefore exact, and so is the final
// sum.  For q < 2^41 and x < 2^46 the result lies in (-0.51q, 0.51q); for q < 2^50 and x <= 4q < 2^52 in
// (-0.75q, 0.75q).  Always congruent to x*w.
__device__ __forceinline__ double fp_mul_centred(double x, double w, double wq, double q) {
    const double magic = 4503599627370496.0;             // 2^52
    const double ph = __dmul_rn(x, w);
    const double pl = __fma_rn(x, w, -ph);
    const double qh = __dsub_rn(__fma_rn(x, wq, magic), magic);
    return __dadd_rn(__fma_rn(-qh, q, ph), pl);
}
// The same product for a signed integer-valued |x| < 2^47 and q < 2^41 (rounding constant 1.5 * 2^52, which
// is exact for quotients of either sign): congruent to x*w, |result| <= 0.532 q.
__device__ __forceinline__ double fp_mul_centred_signed(double x, double w, double wq, double q) {
    const double magic = 6755399441055744.0;             // 1.5 * 2^52
    const double ph = __dmul_rn(x, w);
    const double pl = __fma_rn(x, w, -ph);
    const double qh = __dsub_rn(__fma_rn(x, wq, magic), magic);
    return __dadd_rn(__fma_rn(-qh, q, ph), pl);
}
// v - round(v / q) q for a signed integer-valued |v| < 2^50: congruent to v, |result| <= q / 2
__device__ __forceinline__ double fp_centre(double v, double q, double qinv) {
    const double magic = 6755399441055744.0;
    const double qh = __dsub_rn(__fma_rn(v, qinv, magic), magic);
    return __fma_rn(-qh, q, v);
}
// v mod q in [0, q) for an integer-valued 0 <= v < 2^46
__device__ __forceinline__ double fp_reduce(double v, double q, double qinv) {
    const double magic = 4503599627370496.0;
    const double qh = __dsub_rn(__fma_rn(v, qinv, magic), magic);
    double r = __fma_rn(-qh, q, v);
    if (r < 0.0) r = __dadd_rn(r, q);
    return r;
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

// Lazy sum of products of 64-bit words, kept as partial sums of 32-bit limb products so that one
// term costs four 32x32->64 multiplies and no 64-bit high-product sequence:
//   sum a*b = lo + mid * 2^32 + hi * 2^64,   lo = sum a0*b0,  mid = sum (a0*b1 + a1*b0),  hi = sum a1*b1.
// lo and mid carry their overflow into 32-bit counters.  With words below 2^60 and at most 2^8 terms
// hi stays below 2^64 and the total below 2^128.  SMALL drops the carry counter of mid: valid while
// terms * 2 * 2^(bits-32) * 2^32 < 2^64, e.g. words below 2^50 and up to 2^13 terms.
template <bool SMALL>
struct LimbAcc {
    u64 lo = 0, mid = 0, hi = 0;
    u32 lo_c = 0, mid_c = 0;

    __device__ __forceinline__ void mac(u64 a, u64 b) {
        const u32 a0 = (u32)a, a1 = (u32)(a >> 32), b0 = (u32)b, b1 = (u32)(b >> 32);
        if (SMALL) {
            asm("{\n\t.reg .u64 p;\n\t"
                "mul.wide.u32 p, %4, %6;\n\t"
                "add.cc.u64 %0, %0, p;\n\t"
                "addc.u32 %1, %1, 0;\n\t"
                "mad.wide.u32 %2, %4, %7, %2;\n\t"
                "mad.wide.u32 %2, %5, %6, %2;\n\t"
                "mad.wide.u32 %3, %5, %7, %3;\n\t}"
                : "+l"(lo), "+r"(lo_c), "+l"(mid), "+l"(hi)
                : "r"(a0), "r"(a1), "r"(b0), "r"(b1));
        } else {
            asm("{\n\t.reg .u64 p;\n\t"
                "mul.wide.u32 p, %5, %7;\n\t"
                "add.cc.u64 %0, %0, p;\n\t"
                "addc.u32 %1, %1, 0;\n\t"
                "mul.wide.u32 p, %5, %8;\n\t"
                "add.cc.u64 %2, %2, p;\n\t"
                "addc.u32 %3, %3, 0;\n\t"
                "mul.wide.u32 p, %6, %7;\n\t"
                "add.cc.u64 %2, %2, p;\n\t"
                "addc.u32 %3, %3, 0;\n\t"
                "mad.wide.u32 %4, %6, %8, %4;\n\t}"
                : "+l"(lo), "+r"(lo_c), "+l"(mid), "+r"(mid_c), "+l"(hi)
                : "r"(a0), "r"(a1), "r"(b0), "r"(b1));
        }
    }

    // the accumulated integer modulo q, in [0, q)
    __device__ __forceinline__ u64 reduce(u64 q, u64 mu, u64 c64, u64 c64s) const {
        const u64 L = lo + (mid << 32);
        const u64 carry = L < lo ? 1ull : 0ull;
        const u64 H = (u64)lo_c + (mid >> 32) + ((u64)mid_c << 32) + hi + carry;
        return reduce128(H, L, q, mu, c64, c64s);
    }

    // Montgomery reduction of the accumulated integer V: V * 2^{-64} mod q, in [0, q).
    // Requires V < q * 2^64 (number of terms times q below 2^64).  qneg = -q^{-1} mod 2^64.
    __device__ __forceinline__ u64 reduce_mont(u64 q, u64 qneg) const {
        const u64 L = lo + (mid << 32);
        const u64 carry = L < lo ? 1ull : 0ull;
        const u64 H = (u64)lo_c + (mid >> 32) + ((u64)mid_c << 32) + hi + carry;
        const u64 m = L * qneg;
        u64 t = H + __umul64hi(m, q) + (L != 0 ? 1ull : 0ull);   // L + lo(m*q) = 0 mod 2^64, carrying iff L != 0
        return t >= q ? t - q : t;
    }

    // The same by two 32-bit rounds (redc_2x32 below): no 64-bit high product.
    __device__ __forceinline__ u64 reduce_mont32(u64 q, u32 qneg32) const;

    __device__ __forceinline__ void reset_to(u64 v) {
        lo = v; mid = 0; hi = 0; lo_c = 0; mid_c = 0;
    }
};

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
    LOAD_CENTRED = 3,   // centred lift t' in (-M/2, M/2] of a residue of modulus M, stored as t' + 2^59: t' mod q
    LOAD_I64_MONT = 4,  // LOAD_I64, then times 2^64 mod q: the transform's output is in Montgomery form
};

constexpr int MAX_ROT_BATCH = 64; // rotations handled by one key-switch launch

struct RotBatch {                     // one key-switch launch over n rotations
    int n;
    int key[MAX_ROT_BATCH];           // index of the rotation key (and of its permutation table)
    int dig[MAX_ROT_BATCH];           // which digit set the rotation reads
    int c0[MAX_ROT_BATCH];            // which source ciphertext is being rotated (its c0 is added)
    int out[MAX_ROT_BATCH];           // which output ciphertext slot receives the result
    // runs of consecutive rotations that use the same key (filled in by the inner-product launcher): a block of the
    // inner product takes one run, loads the key once and walks the run's digit sets
    int n_groups;
    unsigned char grp_first[MAX_ROT_BATCH], grp_cnt[MAX_ROT_BATCH];
};

// Epilogue of the division by P, fused into the forward transform of the lifted P-residue
// (polynomial (o, m) = (rotation*2 + component, prime i)):  instead of storing t = NTT(lift),
//   v = (u[o][i][n] - t) * P^{-1} + (component == 0 ? c0[c0(rot)][i][n] : 0)
// is scattered to out[out(rot)][component][i][pinv[key(rot)][n]].
//
// Per-output form (n_sum > 0; one division by P per output ciphertext and component): polynomial (o, m) =
// (output p * 2 + component, prime i).  The inner products of the n_sum giant rotations of output p sit in u at
// rotation index jj * n_out + p (jj < n_sum, key rb.key[jj]), un-rotated; they are summed through each
// rotation's permutation (rotated[n] = unrotated[perm[n]]), the inverse transform reads the P-residues that
// way, and the forward transform's last store computes
//   v[n] = (sum_jj u[jj][i][perm_jj[n]] - t[n]) * P^{-1} + (component == 0 ? sum_jj c0[jj][i][perm_jj[n]] : 0)
// into out[p][component][i][n] (no scatter), with c0 of rotation index jj * n_out + p at c0_base + index * c0_stride.
struct ModDownEpilogue {
    const u64* u;                 // [rot][2][r+1][N]
    const u64* c0_base;
    long long c0_stride;
    const u32* pinv;              // [n_keys][N]
    u64* out_base;
    long long out_stride;
    const u32* perm;              // [n_keys][N] (per-output form)
    u32 n_sum, n_out;             // per-output form: giant steps summed per output, number of outputs
    u32 plain;                    // division by P of inner sums kept in the extended basis (double hoisting):
                                  //   polynomial (o, i): out_base[o*out_stride + i*N + n] = (u[o][i][n] - t[n]) * P^{-1},
                                  //   no rotation, nothing added
    // Output assembly in the extended basis (double hoisting with one division per output; inverse transforms only).
    // aext[(j*n_out + p)][comp][r+1][N] are the inner sums, u[((j-1)*n_out + p)*2 + comp][r+1][N] the key-switch
    // results of the giant steps j >= 1; what is rotated (u, and component 0 of the inner sums with j >= 1) was stored
    // through rotation j's permutation by its producer.  Polynomial (o = p, m):
    //   modulus i < r, m = comp*r + i:  aext[p][comp][i] + sum_j u[j][p][comp][i] + (comp == 0) sum_j aext[j*n_out+p][0][i]
    //   modulus P, m = 0, 1:            sum_j u[j][p][comp = m][P]
    //               m = 2, 3:            aext[p][comp = m - 2][P]
    //               m = 3 + j:           aext[j*n_out + p][0][P]
    // (the residues modulo P stay apart because each of those terms is divided by P, i.e. rounded, by itself)
    const u64* aext;
    long long aext_stride;
    u32 assemble;
};

// Double hoisting with one division per output: component 0 of inner sum (j, p), j >= 1, is only ever used rotated
// by giant step j, so the multiply-accumulate stores it through that rotation's permutation (group pj0 + pj has
// j = (pj0 + pj) / n_out; pinv = null: plain stores).
struct MacScatter {
    const u32* pinv;              // [n_keys][N]
    u32 n_out, pj0;
    int key[MAX_ROT_BATCH + 1];   // key (permutation table) of giant step j
};

// Constants of a rescale from `level` primes: q_L^{-1} mod q_i with its Shoup companion, and q_L mod q_i (i < level - 1).
struct RescaleConsts {
    u64 inv[MAX_MODULI], invs[MAX_MODULI], qlmod[MAX_MODULI];
    double inv_d[MAX_MODULI], inv_q[MAX_MODULI], qlmod_d[MAX_MODULI];   // the same as doubles; inv_q = inv / q_i
};

// Tile-major layout of cached plaintexts, chosen so that the multiply-accumulate kernel's blocks
// each stream one contiguous region:  word (group pj, term t, prime i, coefficient n) has index
//   ((pj%PL)*TS + t%TS)*TN + n%TN   inside stage   ((i, n/TN), pj/PL, t/TS)
// with TN = 2^log_tn coefficients per tile, PL = 256/TN group lanes, TS = 8 terms per stage,
// G = ceil(n_pj/PL), C = ceil(n_terms/TS); a stage holds 2048 words.  The stages of one prime are
// contiguous, ordered (tile, pj/PL, t/TS), and every prime stores its words in the narrowest of three
// formats its size allows, because the kernel that reads them is bound by HBM bytes:
//   TILE_W64  8 bytes per word (16 KB per stage)
//   TILE_W40  primes below 2^40: the low 32 bits of all 2048 words, then their high bytes (10 KB per stage)
//   TILE_W32  primes below 2^32: 32-bit words (8 KB per stage)
enum TileFormat : u32 { TILE_W64 = 0, TILE_W40 = 1, TILE_W32 = 2 };
struct TileLayout {
    u32 log_tn, n_terms, n_pj, G, C, ntiles;
    u32 fmt_bits;                           // TileFormat of prime i in bits 2i, 2i+1
    u32 n_primes;                           // primes the plaintexts are held in: r, or r + 1 with double hoisting
                                            //   (the special prime last, always in 8-byte whole words)
};
constexpr u32 TILE_TS = 8;
constexpr u32 TILE_STAGE_WORDS = 2048;

__host__ __device__ __forceinline__ u32 tile_format(const TileLayout& t, u32 i) { return (t.fmt_bits >> (2 * i)) & 3u; }
__host__ __device__ __forceinline__ u32 tile_stage_bytes(u32 fmt) {
    return TILE_STAGE_WORDS * (fmt == TILE_W64 ? 8u : fmt == TILE_W40 ? 5u : 4u);
}
// byte offset of prime i's first stage (i = r: total size): the primes' regions follow one another
__host__ __device__ __forceinline__ size_t tile_prime_base(const TileLayout& t, u32 i) {
    size_t words8 = 0;                      // in units of 2048 bytes: a stage is 8, 5 or 4 of them
    for (u32 k = 0; k < i; ++k) {
        const u32 f = tile_format(t, k);
        words8 += f == TILE_W64 ? 8u : f == TILE_W40 ? 5u : 4u;
    }
    return words8 * TILE_STAGE_WORDS * (size_t)t.ntiles * t.G * t.C;
}
// byte offset of a stage
__host__ __device__ __forceinline__ size_t tile_stage_offset(const TileLayout& t, u32 i, u32 tile, u32 g, u32 ch) {
    return tile_prime_base(t, i) + (((size_t)tile * t.G + g) * t.C + ch) * tile_stage_bytes(tile_format(t, i));
}
// index of a word inside its stage
__host__ __device__ __forceinline__ u32 tile_word_index(const TileLayout& t, u32 pj, u32 term, u32 n) {
    const u32 TN = 1u << t.log_tn, PL = 256u >> t.log_tn;
    return ((pj % PL) * TILE_TS + term % TILE_TS) * TN + (n & (TN - 1));
}
__host__ __device__ __forceinline__ size_t tile_stage_of_word(const TileLayout& t, u32 pj, u32 term, u32 i, u32 n) {
    const u32 PL = 256u >> t.log_tn;
    return tile_stage_offset(t, i, n >> t.log_tn, pj / PL, term / TILE_TS);
}

// A batch of equally sized polynomials addressed as (outer index o, slot m):
//   source  = src + o*src_so + m*src_sm      destination = dst + o*dst_so + m*dst_sm
//   modulus index of polynomial (o, m) = mod0 + m*mod_step
// blockIdx.y enumerates o*n_m + m.
struct PolyBatch {
    const void* src;
    u64* dst;
    long long src_so, src_sm, dst_so, dst_sm;
    u32 n_m, mod0, mod_step;
    u32 mod_wrap;                 // > 0: modulus index = mod0 + (m % mod_wrap) * mod_step (e.g. m = component*r + prime)
    u32 o_div;                    // > 0: source = src + (o / o_div)*src_so2 + (o % o_div)*src_so + m*src_sm
    long long src_so2;
    // inverse only: the input is a sum  src + sum_{t < sum_terms} (sum_src + t*sum_stride)  of residues in [0, q)
    const u64* sum_src;
    long long sum_stride;
    u32 sum_terms;
    u64 lift_mod;                 // LOAD_CENTRED: the modulus M the source residues live in
    u32 src_digits;               // LOAD_REDUCE: the source of outer index o is a residue modulo prime o % r
    u32 store_centred;            // inverse transform: store the centred lift of each coefficient plus 2^59
                                  //   (the form LOAD_CENTRED reads) instead of the residue in [0, q); 2: only for the
                                  //   polynomials modulo the special prime
    u32 from_mont;                // inverse transform only: input is in Montgomery form, output is not
    u64* tile_ptr;                // non-null: the NTT-domain side lives there in the tile-major layout `tile`
    TileLayout tile;              //   (forward writes its final result there, inverse reads its input there);
    u32 tile_pj0, o_base;         //   diagonal o_base + o = pj*n_terms + t; the layout's group 0 is group tile_pj0
    u32 skip_diag;                // forward only: polynomial (o, m) with m < r and o % r == m (a digit in its own prime)
    const u64* diag_src;          //   is not transformed but copied from diag_src + (o / r)*diag_so + m*N, where its
    long long diag_so;            //   transform already exists
    const u32* scatter;           // forward only: final store goes to scatter_dst[scatter[(o / scatter_div) * N + n]]
    u32 scatter_div;              //   instead of dst[n] (same polynomial strides as dst)
    u64* scatter_dst;
    u32 scatter_mont;             //   and the stored value is the result times 2^64 mod q (rotation keys: the inner
                                  //   product ends in a Montgomery reduction)
    u32 split_bits;               // L > 0: the NTT-domain side of the transform is stored as two L-bit-aligned
                                  // limbs per word, (v >> L) << 32 | (v & (2^L - 1)); forward writes, inverse reads it
    u64* lift_ptr;                // forward only, non-null (double hoisting): polynomial (o, m = comp * mod_wrap + i) is also
    long long lift_so;            //   stored times P mod q_i at lift_ptr + o*lift_so + (comp*(r+1) + i)*N, and zeros as the
                                  //   residue modulo P: the un-rotated input lifted to the extended basis
    u64* dtile_ptr;               // forward only, non-null: the final result goes there instead of dst, tile-major in tiles
    u32 dtile_div;                //   of KS_TILE coefficients (see ks_tile_index); with `scatter` the store is permuted
    u32 grid3;                    // set by the launchers: the grid is (x, m, o) and no index has to be divided out
    u32 o_div_magic, dtile_magic; // ceil(2^32 / o_div), ceil(2^32 / dtile_div): o / d = umulhi(o, magic) for o < 2^16
                                  //   (set by the launchers with grid3; 0 = divide)
    const u64* div_t;             // forward from a shared source, non-null (double hoisting): the source of digit
    long long div_so;             //   i = o % o_div of set s = o / o_div is the residue modulo q_i of a polynomial in the
                                  //   extended basis, coefficient domain, and t = div_t + s*div_so holds its residue
                                  //   modulo P as a centred lift plus 2^59: the digit is (source - t) * P^{-1} mod q_i
};

// Operands of the key-switch inner product (digit sets and rotation keys) are kept tile-major, so that what a block
// needs of one (outer index / div, modulus, tile) is contiguous and arrives by one bulk copy:
//   polynomial (o, m), coefficient n  ->  ((((o / div) * n_m + m) * (N / KS_TILE) + n / KS_TILE) * div + o % div) * KS_TILE + n % KS_TILE
// digits: o = set * r + digit, div = r (a block reads the r digit segments of a set, modulus and tile);
// keys: o = (key * r + digit) * 2 + component, div = 2r.
constexpr u32 KS_TILE = 128;
__host__ __device__ __forceinline__ size_t ks_tile_index(u32 N, u32 n_m, u32 div, u32 o, u32 m, u32 n) {
    return ((((size_t)(o / div) * n_m + m) * (N / KS_TILE) + n / KS_TILE) * div + o % div) * KS_TILE + n % KS_TILE;
}

// o / d and o % d with a host-made reciprocal (see PolyBatch::grid3); magic = 0 divides
__device__ __forceinline__ void split_index(u32 o, u32 d, u32 magic, u32& hi, u32& lo) {
    hi = magic ? __umulhi(o, magic) : o / d;
    lo = o - hi * d;
}
// ks_tile_index of coefficient 0 of polynomial (o = o_hi * div + o_lo, m); coefficient n then sits at
// base + (n / KS_TILE) * div * KS_TILE + n % KS_TILE
__device__ __forceinline__ size_t ks_tile_base(u32 N, u32 n_m, u32 div, u32 o_hi, u32 o_lo, u32 m) {
    return (((size_t)o_hi * n_m + m) * (N / KS_TILE) * div + o_lo) * KS_TILE;
}

__device__ __forceinline__ u64 limb_split(u64 v, u32 L) { return ((v >> L) << 32) | (v & ((1ull << L) - 1)); }
__device__ __forceinline__ u64 limb_join(u64 s, u32 L) { return ((s >> 32) << L) | (s & 0xffffffffull); }

// Karatsuba accumulator for products of words given as two L-bit limbs (low limb in the low 32-bit
// half, high limb in the high half), L <= 25:  three 32x32->64 multiply-adds per product and no
// carries.  sum v*x = lo + (mid - lo - hi) * 2^L + hi * 2^(2L), with lo = sum v0*x0, hi = sum v1*x1,
// mid = sum (v0+v1)*(x0+x1); every term of mid is below 2^(2L+2), so 2^(62-2L) terms fit.
struct KaraAcc {
    u64 lo = 0, mid = 0, hi = 0;
    __device__ __forceinline__ void mac(u32 v0, u32 v1, u32 vs, u64 xsplit) {
        const u32 x0 = (u32)xsplit, x1 = (u32)(xsplit >> 32);
        lo += (u64)v0 * x0;
        hi += (u64)v1 * x1;
        mid += (u64)vs * (x0 + x1);
    }
    // the accumulated integer V as (H, L64)
    __device__ __forceinline__ void value(u32 L, u64& H, u64& L64) const {
        const u64 m = mid - lo - hi;
        u64 l = lo, h = 0;
        const u64 a = m << L;
        l += a; h += (l < a) ? 1ull : 0ull;
        h += m >> (64 - L);
        const u64 b = hi << (2 * L);
        l += b; h += (l < b) ? 1ull : 0ull;
        h += hi >> (64 - 2 * L);
        H = h; L64 = l;
    }
};

// Montgomery reduction by two 32-bit rounds: V * 2^{-64} mod q in [0, q), for V = (H, L) < q * 2^64.
// qneg32 = -q^{-1} mod 2^32.  Six 32-bit multiplies instead of a 64x64 high product.
__device__ __forceinline__ u64 redc_2x32(u64 H, u64 L, u64 q, u32 qneg32) {
    u32 l0 = (u32)L, l1 = (u32)(L >> 32), h0 = (u32)H, h1 = (u32)(H >> 32);
    const u32 q0 = (u32)q, q1 = (u32)(q >> 32);
    // first pass: m = l0 * qneg32; (h1 h0 l1 l0) += m * (q1 q0); l0 becomes 0 and is dropped
    // second pass: the same one limb up; the result is (h1 h0)
    asm("{\n\t.reg .u32 m;\n\t"
        "mul.lo.u32 m, %0, %6;\n\t"
        "mad.lo.cc.u32 %0, m, %4, %0;\n\t"
        "madc.hi.cc.u32 %1, m, %4, %1;\n\t"
        "addc.cc.u32 %2, %2, 0;\n\t"
        "addc.u32 %3, %3, 0;\n\t"
        "mad.lo.cc.u32 %1, m, %5, %1;\n\t"
        "madc.hi.cc.u32 %2, m, %5, %2;\n\t"
        "addc.u32 %3, %3, 0;\n\t"
        "mul.lo.u32 m, %1, %6;\n\t"
        "mad.lo.cc.u32 %1, m, %4, %1;\n\t"
        "madc.hi.cc.u32 %2, m, %4, %2;\n\t"
        "addc.u32 %3, %3, 0;\n\t"
        "mad.lo.cc.u32 %2, m, %5, %2;\n\t"
        "madc.hi.u32 %3, m, %5, %3;\n\t}"
        : "+r"(l0), "+r"(l1), "+r"(h0), "+r"(h1)
        : "r"(q0), "r"(q1), "r"(qneg32));
    const u64 t = ((u64)h1 << 32) | h0;
    return t >= q ? t - q : t;
}

template <bool SMALL>
__device__ __forceinline__ u64 LimbAcc<SMALL>::reduce_mont32(u64 q, u32 qneg32) const {
    const u64 L = lo + (mid << 32);
    const u64 carry = L < lo ? 1ull : 0ull;
    const u64 H = (u64)lo_c + (mid >> 32) + ((u64)mid_c << 32) + hi + carry;
    return redc_2x32(H, L, q, qneg32);
}

}  // namespace bf
