// Negacyclic number-theoretic transform over 64-bit RNS residues (the "NTT kernels" the paper's
// FHE backend relies on, Sec. 4.2), batched over polynomials and primes.
//
// Forward: merged-twiddle Cooley-Tukey, natural order in, bit-reversed order out:
//   position i holds a(psi^(2*brev(i)+1)).  Inverse: Gentleman-Sande, bit-reversed in, natural out.
// The internal order never leaves the library: pointwise products do not care, and automorphisms
// are applied as index gathers that account for it.
//
// A transform of N = R*C points runs as two launches.  The strided pass transforms the R rows
// (stride C) of a tile of adjacent columns; the contiguous pass transforms chunks of C adjacent
// points.  Inside a pass every thread keeps a closed set of 4 or 8 points in registers for two or
// three butterfly stages, and sets are exchanged through shared memory between stage groups.
// Butterflies use Harvey's lazy reduction: forward values stay in [0, 4q), inverse in [0, 2q).
#include "bf_host.h"

namespace bf {

cudaEvent_t Profiler::get() {
    if (!pool.empty()) {
        cudaEvent_t e = pool.back();
        pool.pop_back();
        return e;
    }
    cudaEvent_t e = nullptr;
    cudaEventCreate(&e);
    return e;
}

ProfScope::ProfScope(Profiler* prof, int c, cudaStream_t st) : p(prof), cat(c), s(st) {
    if (!p) return;
    p->launches[cat]++;
    if (p->timing && !p->span_open) {
        a = p->get();
        cudaEventRecord(a, s);
    }
}

ProfScope::~ProfScope() {
    if (!p || !a) return;
    cudaEvent_t b = p->get();
    cudaEventRecord(b, s);
    p->recs.push_back({cat, a, b});
}

ProfSpan::ProfSpan(Profiler* prof, int c, cudaStream_t st) : p(prof), cat(c), s(st) {
    if (!p || !p->timing) return;
    a = p->get();
    cudaEventRecord(a, s);
    p->span_open = true;
}

ProfSpan::~ProfSpan() {
    if (!p || !a) return;
    cudaEvent_t b = p->get();
    cudaEventRecord(b, s);
    p->recs.push_back({cat, a, b});
    p->span_open = false;
}

struct LoadConsts {
    u64 q, mu, lift_mod, lift_red;
    double qd, qinv, c30, c30q, k59;      // (LOAD_I64_MONT: c30 = 2^96 mod q, k59 = the offset for -2^127)
    double c64d, c64q;                     // LOAD_I64_MONT: 2^64 mod q
    bool wide;          // target prime of 2^41 or more: values must stay in [0, 4q); otherwise they are signed
    bool src_small;     // LOAD_REDUCE: every source word is below 1.5 q already (block-uniform)
    bool src_fp;        // LOAD_REDUCE: every source word is below 2^51
};

template <int LOAD>
__device__ __forceinline__ u64 load_src(const void* src, size_t idx, const LoadConsts& c) {
    if (LOAD == LOAD_PLAIN) return ((const u64*)src)[idx];
    if (LOAD == LOAD_REDUCE) {
        const u64 t = ((const u64*)src)[idx];
        return c.src_small ? (t >= c.q ? t - c.q : t) : barrett64(t, c.q, c.mu);
    }
    if (LOAD == LOAD_I64 || LOAD == LOAD_I64_MONT) {
        i64 v = ((const i64*)src)[idx];
        u64 a = v < 0 ? (u64)(-v) : (u64)v;
        u64 m = barrett64(a, c.q, c.mu);
        m = (v < 0 && m != 0) ? c.q - m : m;
        if (LOAD == LOAD_I64_MONT) m = mul_shoup(m, c.lift_mod, c.lift_red, c.q);   // (2^64 mod q, its Shoup companion)
        return m;
    }
    // LOAD_CENTRED: the word is t' + 2^59 with t' the centred lift of a residue modulo lift_mod
    const u64 T = ((const u64*)src)[idx];
    const bool neg = T < (1ull << 59);
    const u64 t = neg ? T + c.lift_mod - (1ull << 59) : T - (1ull << 59);      // back to [0, lift_mod)
    u64 m = barrett64(t, c.q, c.mu);
    if (neg) m = sub_mod(m, c.lift_red, c.q);
    return m;
}

// The same loads for a modulus on the fp64 path: the result is an integer-valued double congruent to the
// source, of magnitude below 3.6 q (lazy: the butterflies reduce); non-negative for primes of 2^41 or more.
template <int LOAD>
__device__ __forceinline__ double load_src_fp(const void* src, size_t idx, const LoadConsts& c) {
    if (LOAD == LOAD_REDUCE) {
        const u64 t = ((const u64*)src)[idx];
        if (c.src_small) return u2d(t);
        if (c.src_fp) {                                  // t - round(t / q) q, plus q where values must not be negative
            const double v = fp_centre(u2d(t), c.qd, c.qinv);
            return c.wide ? __dadd_rn(v, c.qd) : v;
        }
        return u2d(barrett64(t, c.q, c.mu));
    }
    if (LOAD == LOAD_CENTRED) {
        // t' + 2^59 = hi 2^30 + lo, so t' = hi (2^30 mod q) + lo - (2^59 mod q)  (mod q); with the product
        // centred in (-0.75 q, 0.75 q), lo < 2^30 and k59 = 2q - (2^59 mod q) the sum is positive
        const u64 T = ((const u64*)src)[idx];
        const double hi = u2d(T >> 30), lo = u2d(T & ((1ull << 30) - 1));
        return __dadd_rn(__dadd_rn(fp_mul_centred(hi, c.c30, c.c30q, c.qd), lo), c.k59);   // (k59: see LoadConsts)
    }
    if (LOAD == LOAD_I64_MONT) {
        // v = (hi' - 2^31) 2^32 + lo with hi' = (v >> 32) + 2^31 in [0, 2^32); two centred products (each
        // within 0.75 q, 0.51 q for primes below 2^41) plus the offset: magnitude below 1.6 q, or within
        // (0, 4q) for the primes whose values must stay non-negative
        const uint2 w = ((const uint2*)src)[idx];
        const double hi = __uint2double_rn(w.y ^ 0x80000000u), lo = __uint2double_rn(w.x);
        return __dadd_rn(__dadd_rn(fp_mul_centred(hi, c.c30, c.c30q, c.qd), fp_mul_centred(lo, c.c64d, c.c64q, c.qd)), c.k59);
    }
    return u2d(load_src<LOAD>(src, idx, c));
}

// Butterflies of one register-resident set of 2^K points over K consecutive stages.
// tw_base = (blocks at the group's first forward stage) * mult, so that stage st, sub-block sub
// uses twiddle (tw_base << st) + (blk << st) + sub.
// Integer version: Harvey's lazy butterflies with Shoup products; forward values stay in [0, 4q),
// inverse values in [0, 2q).
// Twiddle (and companion) number idx: from the global table through the read-only path, or from a copy of
// the table's head that the block staged in shared memory.
template <bool TWSM>
__device__ __forceinline__ ulonglong2 tw_fetch(const ulonglong2* tw, u32 idx) {
    if (TWSM) return tw[idx];
    return __ldg(&tw[idx]);
}

template <int K, bool FWD, bool TWSM = false>
__device__ __forceinline__ void set_butterflies(u64 (&e)[8], const ulonglong2* __restrict__ tw, u32 tw_base, u32 blk,
                                                u64 q, double) {
    const u64 q2 = 2 * q;
#pragma unroll
    for (int s = 0; s < K; ++s) {
        const int st = FWD ? s : (K - 1 - s);
        const int d = (1 << K) >> (st + 1);
#pragma unroll
        for (int sub = 0; sub < (1 << st); ++sub) {
            const ulonglong2 w = tw_fetch<TWSM>(tw, (tw_base << st) + (blk << st) + sub);
#pragma unroll
            for (int off = 0; off < d; ++off) {
                const int i = sub * 2 * d + off;
                if (FWD) {
                    u64 x = e[i];
                    if (x >= q2) x -= q2;
                    u64 t = mul_shoup_lazy(e[i + d], w.x, w.y, q);
                    e[i] = x + t;
                    e[i + d] = x - t + q2;
                } else {
                    u64 a = e[i], b = e[i + d];
                    u64 s2 = a + b;
                    if (s2 >= q2) s2 -= q2;
                    e[i] = s2;
                    e[i + d] = mul_shoup_lazy(a - b + q2, w.x, w.y, q);
                }
            }
        }
    }
}

// fp64 version.  Primes below 2^41: values are signed integer-valued doubles, reduced lazily.
//   Forward: (X, Y) -> (X + s, X - s), s = Y*w centred in (-0.54q, 0.54q): magnitudes grow by at most 0.54q
//   per stage, from at most 3.6q after the load functors to below 13q after log2 N <= 16 stages; one
//   reduction at the very end.
//   Inverse: (a, b) -> (a + b, (a - b)*w centred): the sums double per stage and the product takes
//   |a - b| < 2^47, i.e. magnitudes below 32q going into a stage.  From [0, q) the contiguous pass runs its
//   first two groups (5 stages, sums up to 32q), centres the sums, and leaves at most 4.4q after its last
//   group; the strided pass centres the sums after its first group when more groups follow, which keeps
//   every later stage below 18q going in and the values handed to the final scaling below 35q.
// WIDE (primes from 2^41 up to 2^50): the centred product lies in (-0.75q, 0.75q) and values must stay below
// 4q < 2^52, so the forward butterfly keeps Harvey's invariant [0, 4q) with one conditional subtraction:
// (X, Y) -> (X~ + T, X~ - T + 2q), X~ = X reduced below 2q, T = Y*w + q in (0.25q, 1.75q); the inverse is
// (a, b) -> (a + b reduced below 2q, (a - b + 2q)*w + q in (0.25q, 1.75q)): values in [0, 2q).
template <int K, bool FWD, bool WIDE, bool TWSM>
__device__ __forceinline__ void set_butterflies_fp(double (&e)[8], const ulonglong2* __restrict__ tw, u32 tw_base,
                                                   u32 blk, double q) {
    const double q2 = __dadd_rn(q, q);
#pragma unroll
    for (int s = 0; s < K; ++s) {
        const int st = FWD ? s : (K - 1 - s);
        const int d = (1 << K) >> (st + 1);
#pragma unroll
        for (int sub = 0; sub < (1 << st); ++sub) {
            const ulonglong2 wb = tw_fetch<TWSM>(tw, (tw_base << st) + (blk << st) + sub);
            const double w = __longlong_as_double((long long)wb.x), wq = __longlong_as_double((long long)wb.y);
#pragma unroll
            for (int off = 0; off < d; ++off) {
                const int i = sub * 2 * d + off;
                if (FWD && WIDE) {
                    double x = e[i];
                    if (x >= q2) x = __dsub_rn(x, q2);
                    const double t = __dadd_rn(fp_mul_centred(e[i + d], w, wq, q), q);
                    e[i] = __dadd_rn(x, t);
                    e[i + d] = __dadd_rn(__dsub_rn(x, t), q2);
                } else if (FWD) {
                    const double sv = fp_mul_centred_signed(e[i + d], w, wq, q);
                    const double x = e[i];
                    e[i] = __dadd_rn(x, sv);
                    e[i + d] = __dsub_rn(x, sv);
                } else if (WIDE) {
                    const double a = e[i], b = e[i + d];
                    double s2 = __dadd_rn(a, b);
                    if (s2 >= q2) s2 = __dsub_rn(s2, q2);
                    e[i] = s2;
                    e[i + d] = __dadd_rn(fp_mul_centred(__dadd_rn(__dsub_rn(a, b), q2), w, wq, q), q);
                } else {
                    const double a = e[i], b = e[i + d];
                    e[i] = __dadd_rn(a, b);
                    e[i + d] = fp_mul_centred_signed(__dsub_rn(a, b), w, wq, q);
                }
            }
        }
    }
}

template <int K, bool FWD, bool TWSM = false>
__device__ __forceinline__ void set_butterflies(double (&e)[8], const ulonglong2* __restrict__ tw, u32 tw_base,
                                                u32 blk, u64 q_int, double q) {
    if (q_int >> 41) set_butterflies_fp<K, FWD, true, TWSM>(e, tw, tw_base, blk, q);    // block-uniform
    else set_butterflies_fp<K, FWD, false, TWSM>(e, tw, tw_base, blk, q);
}

// After an inverse group of K stages the first 2^(K-1) values of a set are sums (they doubled per stage),
// the others fresh centred products: bring the sums back to |v| <= q/2.  Signed fp64 path only.
template <int K>
__device__ __forceinline__ void centre_sums(double (&e)[8], u64 q_int, double q, double qinv) {
    if (q_int >> 41) return;
#pragma unroll
    for (int i = 0; i < (1 << K) / 2; ++i) e[i] = fp_centre(e[i], q, qinv);
}
template <int K>
__device__ __forceinline__ void centre_sums(u64 (&)[8], u64, double, double) {}

template <bool FP> struct Elem { typedef u64 T; };
template <> struct Elem<true> { typedef double T; };
__device__ __forceinline__ void from_u64(u64& dst, u64 v) { dst = v; }
__device__ __forceinline__ void from_u64(double& dst, u64 v) { dst = u2d(v); }

// Stage groups of a local transform of 2^LOG_LEN points, in forward order.
__host__ __device__ constexpr int n_groups(int log_len) { return log_len <= 3 ? 1 : (log_len <= 6 ? 2 : 3); }
__host__ __device__ constexpr int group_k(int log_len, int gi) {
    // 1:{1} 2:{2} 3:{3} 4:{2,2} 5:{3,2} 6:{3,3} 7:{3,2,2} 8:{3,3,2}
    return log_len <= 3 ? log_len
         : log_len == 4 ? 2
         : log_len == 5 ? (gi == 0 ? 3 : 2)
         : log_len == 6 ? 3
         : log_len == 7 ? (gi == 0 ? 3 : 2)
         : (gi == 2 ? 2 : 3);
}
// log2 of the point spacing of group gi's sets (forward order index)
__host__ __device__ constexpr int group_log_step(int log_len, int gi) {
    int done = 0;
    for (int i = 0; i <= gi; ++i) done += group_k(log_len, i);
    return log_len - done;
}

// Shared-memory index swizzle for a 256-point chunk of 64-bit words: makes the three access
// patterns of the contiguous pass (spacing 32, spacing 4 and 4 adjacent points per thread) free of
// bank conflicts without padding.
__host__ __device__ constexpr int swz(int i) { return i ^ ((i >> 4) & 3) ^ (((i >> 5) & 3) << 2); }

// The swizzle is linear over GF(2): swz(t ^ k) = swz(t) ^ swz(k).  Every access of the contiguous pass has
// index t ^ k with t depending on the thread and k on the unrolled loop counter, in disjoint bit fields, so
// its byte address is (A ^ 8 * (swz(k) & 15)) + 8 * (swz(k) & ~15) with A = slice base + 8 * swz(t) computed
// once per group: one logic operation and an immediate offset per access.  (The swizzle only changes the low
// four index bits, and t has no bits where swz(k) & ~15 has any.)  The slice base is 128-byte aligned.
template <int K_INDEX>
__device__ __forceinline__ void swz_store(u32 a_thread, u64 v) {
    constexpr int S = swz(K_INDEX);
    asm volatile("st.shared.b64 [%0+%1], %2;" ::"r"(a_thread ^ (u32)(8 * (S & 15))), "n"(8 * (S & ~15)), "l"(v));
}
template <int K_INDEX>
__device__ __forceinline__ void swz_store(u32 a_thread, double v) {
    swz_store<K_INDEX>(a_thread, (u64)__double_as_longlong(v));
}
template <int K_INDEX>
__device__ __forceinline__ void swz_load(u32 a_thread, u64& v) {
    constexpr int S = swz(K_INDEX);
    asm volatile("ld.shared.b64 %0, [%1+%2];" : "=l"(v) : "r"(a_thread ^ (u32)(8 * (S & 15))), "n"(8 * (S & ~15)));
}
template <int K_INDEX>
__device__ __forceinline__ void swz_load(u32 a_thread, double& v) {
    u64 bits;
    swz_load<K_INDEX>(a_thread, bits);
    v = __longlong_as_double((long long)bits);
}
// e[i] <-> slice[swz(t ^ (i << SHIFT))] for i < COUNT
template <int COUNT, int SHIFT, typename T, int I = 0>
__device__ __forceinline__ void swz_store_set(u32 a_thread, const T (&e)[8]) {
    if constexpr (I < COUNT) {
        swz_store<(I << SHIFT)>(a_thread, e[I]);
        swz_store_set<COUNT, SHIFT, T, I + 1>(a_thread, e);
    }
}
template <int COUNT, int SHIFT, typename T, int I = 0>
__device__ __forceinline__ void swz_load_set(u32 a_thread, T (&e)[8]) {
    if constexpr (I < COUNT) {
        swz_load<(I << SHIFT)>(a_thread, e[I]);
        swz_load_set<COUNT, SHIFT, T, I + 1>(a_thread, e);
    }
}

constexpr int LOG_C = 8;              // contiguous pass: chunks of 256 points, one warp each
constexpr int CHUNKS_PER_BLOCK = 4;      // measured: 4 beats 8 by 4 % of the pass, 2 is no better

// Between the two passes of a transform the data sit in dst as lazily reduced values: 64-bit
// integers for the integer path, fp64 bit patterns for the fp64 path (the modulus decides, so both
// passes agree).

// Strided pass: transforms the 2^LOG_R rows (stride 256) of 2^LOG_LANES adjacent columns.
// Forward: first pass (reads the batch source through the load functor).  Inverse: second pass
// (in place, scales by N^{-1}).
// STAGED: the source tile already sits in shared memory (`staged`, [row][lane], raw words) because several
// target primes of the same block read it.
template <bool FWD, int LOAD, int LOG_R, int LOG_LANES, bool FP, bool STAGED = false>
__device__ __forceinline__ void strided_body(const RingDev& R, const PolyBatch& B, u64* sm_raw, ulonglong2* tws, u32 o,
                                             u32 m, u32 mod, const u64* staged = nullptr) {
    typedef typename Elem<FP>::T T;
    constexpr int LEN = 1 << LOG_R, LANES = 1 << LOG_LANES;
    constexpr int NT = (LEN * LANES / 8) < 32 ? 32 : (LEN * LANES / 8);
    constexpr int NG = n_groups(LOG_R);
    T* sm = (T*)sm_raw;
    const u64 q = R.q[mod], mu = R.mu[mod];
    const double qd = R.qd[mod];
    // the strided pass uses the first LEN twiddles of the prime only: the block stages them in shared
    // memory (the load is in flight together with the first data loads)
    const ulonglong2* __restrict__ tw_global = (FWD ? R.tw_fwd : R.tw_inv) + (size_t)mod * R.N;
    const ulonglong2* tw = tws;
    ulonglong2 tw_mine = make_ulonglong2(0, 0);
    if (threadIdx.x < LEN) tw_mine = __ldg(&tw_global[threadIdx.x]);
    u64* dst = B.dst + (size_t)o * B.dst_so + (size_t)m * B.dst_sm;
    const char* src = nullptr;
    if constexpr (!STAGED) {
        u32 o_hi = 0, o_lo = o;
        if (B.o_div) split_index(o, B.o_div, B.o_div_magic, o_hi, o_lo);
        const size_t src_off = B.o_div ? (size_t)o_hi * B.src_so2 + (size_t)o_lo * B.src_so : (size_t)o * B.src_so;
        src = (const char*)B.src + (src_off + (size_t)m * B.src_sm) * 8;
    }
    LoadConsts lc;
    lc.q = q;
    lc.mu = mu;
    lc.lift_red = (LOAD == LOAD_CENTRED) ? barrett64(B.lift_mod, q, mu) : (LOAD == LOAD_I64_MONT) ? R.c64s[mod] : 0;
    lc.lift_mod = (LOAD == LOAD_I64_MONT) ? R.c64[mod] : B.lift_mod;
    lc.qd = qd;
    lc.qinv = R.qinv_d[mod];
    lc.c30 = R.c30_d[mod];
    lc.c30q = R.c30_q[mod];
    lc.c64d = lc.c64q = 0.0;
    lc.wide = (q >> 41) != 0;
    // wide: 2q - (2^59 mod q) keeps the lifted value positive; otherwise the offset is just -(2^59 mod q)
    lc.k59 = lc.wide ? R.k59_d[mod] : __dsub_rn(R.k59_d[mod], __dadd_rn(qd, qd));
    if (LOAD == LOAD_I64_MONT) {
        const double* ec = R.enc_consts + (size_t)mod * ENC_CONSTS;
        lc.c30 = __ldg(ec);
        lc.c30q = __ldg(ec + 1);
        lc.c64d = __ldg(ec + 2);
        lc.c64q = __ldg(ec + 3);
        lc.k59 = __ldg(ec + 4);
    }
    {
        u64 qs = ~(u64)0;
        if (LOAD == LOAD_REDUCE && B.src_digits) {      // the prime the source digit belongs to
            u32 s_hi, s_lo;
            split_index(o, R.r, B.o_div == R.r ? B.o_div_magic : 0u, s_hi, s_lo);
            qs = R.q[s_lo];
        }
        lc.src_small = qs <= q + (q >> 1);
        lc.src_fp = qs < (1ull << 51);
    }
    const int col0 = blockIdx.x * LANES;
    const int tid = threadIdx.x;
#pragma unroll
    for (int gi = 0; gi < NG; ++gi) {
        const int fg = FWD ? gi : NG - 1 - gi;                 // group index in forward order
        const int K = group_k(LOG_R, fg);
        const int log_step = group_log_step(LOG_R, fg);
        const int step = 1 << log_step, t0 = step << (K - 1);
        const int m0 = LEN / (2 * t0);
        const int nsets = (LEN * LANES) >> K;
        const bool g_first = (gi == 0), g_last = (gi == NG - 1);
#pragma unroll
        for (int w0 = 0; w0 < nsets; w0 += NT) {
            const int w = w0 + tid;
            if (NT > nsets && w >= nsets) break;
            const int lane = w & (LANES - 1), u = w >> LOG_LANES;
            const int blk = u >> log_step, off = u & (step - 1);
            const int base = blk * 2 * t0 + off;
            T e[8];
#pragma unroll
            for (int i = 0; i < (1 << K); ++i) {
                const int row = base + i * step;
                if (g_first) {
                    const size_t gidx = ((size_t)row << LOG_C) + col0 + lane;
                    if (FWD) {
                        const void* from = STAGED ? (const void*)staged : (const void*)src;
                        const size_t at = STAGED ? (size_t)(row * LANES + lane) : gidx;
                        if constexpr (FP) e[i] = load_src_fp<LOAD>(from, at, lc);
                        else e[i] = load_src<LOAD>(from, at, lc);
                    } else {
                        e[i] = ((const T*)dst)[gidx];
                    }
                } else {
                    e[i] = sm[row * LANES + lane];
                }
            }
            if (g_first && w0 == 0) {       // (the first sweep of the first group is full for every geometry)
                static_assert(NT <= ((LEN * LANES) >> group_k(LOG_R, FWD ? 0 : NG - 1)), "first sweep must be full");
                if (threadIdx.x < LEN) tws[threadIdx.x] = tw_mine;
                __syncthreads();
            }
            if (K == 3) set_butterflies<3, FWD, true>(e, tw, (u32)m0, (u32)blk, q, qd);
            else if (K == 2) set_butterflies<2, FWD, true>(e, tw, (u32)m0, (u32)blk, q, qd);
            else set_butterflies<1, FWD, true>(e, tw, (u32)m0, (u32)blk, q, qd);
            if (!FWD && g_first && NG > 1) {
                if (K == 3) centre_sums<3>(e, q, qd, R.qinv_d[mod]);
                else if (K == 2) centre_sums<2>(e, q, qd, R.qinv_d[mod]);
                else centre_sums<1>(e, q, qd, R.qinv_d[mod]);
            }
#pragma unroll
            for (int i = 0; i < (1 << K); ++i) {
                const int row = base + i * step;
                if (g_last) {
                    const size_t gidx = ((size_t)row << LOG_C) + col0 + lane;
                    if (FWD) {
                        ((T*)dst)[gidx] = e[i];                 // lazy; the contiguous pass finishes
                    } else {                                    // scale by N^{-1}, to [0, q)
                        const bool mont = B.from_mont != 0;
                        u64 out;
                        if constexpr (FP) {
                            const double nv = mont ? R.ninvm_d[mod] : R.ninv_d[mod];
                            const double nq = mont ? R.ninvm_q[mod] : R.ninv_q[mod];
                            double v;
                            if (q >> 41) {
                                v = __dadd_rn(fp_mul_centred(e[i], nv, nq, qd), qd);
                                if (v >= qd) v = __dsub_rn(v, qd);
                                if (v >= qd) v = __dsub_rn(v, qd);  // (the product can touch 2q for the 50-bit prime)
                            } else {
                                v = fp_mul_centred_signed(e[i], nv, nq, qd);
                                if (v < 0.0) v = __dadd_rn(v, qd);
                            }
                            out = d2u(v);
                        } else {
                            out = mul_shoup(e[i], mont ? R.ninv_m[mod] : R.ninv[mod], mont ? R.ninv_ms[mod] : R.ninvs[mod], q);
                        }
                        if (B.store_centred == 1 || (B.store_centred == 2 && mod == R.r))
                            out = (out > (q - 1) / 2 ? out - q : out) + (1ull << 59);
                        dst[gidx] = out;
                    }
                } else {
                    sm[row * LANES + lane] = e[i];
                }
            }
        }
        if (!g_last) __syncthreads();
    }
}

// Polynomial (o, m) of a block and its modulus: straight from the grid (x, m, o) when the launcher could lay it out
// so, else divided out of blockIdx.y.  (n_m <= 2 * mod_wrap in every batch that wraps.)
__device__ __forceinline__ void block_poly(const PolyBatch& B, u32& o, u32& m, u32& mod) {
    if (B.grid3) {
        m = blockIdx.y;
        o = blockIdx.z;
    } else {
        o = blockIdx.y / B.n_m;
        m = blockIdx.y - o * B.n_m;
    }
    const u32 mm = (B.mod_wrap && m >= B.mod_wrap) ? m - B.mod_wrap : m;
    mod = B.mod0 + mm * B.mod_step;
}
// a digit in its own prime (o = set * r + digit with digit == mod), which ModUp copies instead of transforming
__device__ __forceinline__ bool own_prime(const RingDev& R, const PolyBatch& B, u32 o, u32 mod) {
    if (!B.skip_diag || mod >= R.r) return false;
    u32 hi, lo;
    split_index(o, R.r, B.o_div == R.r ? B.o_div_magic : 0u, hi, lo);
    return lo == mod;
}

template <bool FWD, int LOAD, int LOG_R, int LOG_LANES>
__global__ void __launch_bounds__(((1 << (LOG_R + LOG_LANES)) / 8) < 32 ? 32 : ((1 << (LOG_R + LOG_LANES)) / 8),
                                  ((1 << (LOG_R + LOG_LANES)) / 8) >= 512 ? 2 : ((1 << (LOG_R + LOG_LANES)) / 8) >= 256 ? 4 : 8)
ntt_strided(const RingDev R, const PolyBatch B) {
    __shared__ u64 sm[1 << (LOG_R + LOG_LANES)];
    __shared__ ulonglong2 tws[1 << LOG_R];
    grid_dependency_enter();
    u32 o, m, mod;
    block_poly(B, o, m, mod);
    if (FWD && own_prime(R, B, o, mod)) {
        // this digit's transform in its own prime exists already: copy the tile instead
        const u64* ds = B.diag_src + (size_t)(o / R.r) * B.diag_so + (size_t)mod * R.N;
        u64* dd = B.dst + (size_t)o * B.dst_so + (size_t)m * B.dst_sm;
        size_t tbase = 0;
        if (B.dtile_ptr) {
            u32 t_hi, t_lo;
            split_index(o, B.dtile_div, B.dtile_magic, t_hi, t_lo);
            tbase = ks_tile_base(R.N, B.n_m, B.dtile_div, t_hi, t_lo, m);
        }
        for (int w = threadIdx.x; w < (1 << (LOG_R + LOG_LANES)); w += blockDim.x) {
            const size_t gidx = ((size_t)(w >> LOG_LANES) << LOG_C) + blockIdx.x * (1 << LOG_LANES) + (w & ((1 << LOG_LANES) - 1));
            if (B.dtile_ptr) B.dtile_ptr[tbase + (gidx / KS_TILE) * B.dtile_div * KS_TILE + gidx % KS_TILE] = ds[gidx];
            else dd[gidx] = ds[gidx];
        }
        return;
    }
    if (R.fp_ok[mod]) strided_body<FWD, LOAD, LOG_R, LOG_LANES, true>(R, B, sm, tws, o, m, mod);
    else strided_body<FWD, LOAD, LOG_R, LOG_LANES, false>(R, B, sm, tws, o, m, mod);
}

// Forward strided pass of a batch whose n_m target primes all read the same source polynomial (ModUp digits,
// the P-residues of ModDown): a block stages the source tile in shared memory once and transforms it
// into targets m_begin .. m_begin + m_count - 1, so the source crosses L2 once per block instead of once per
// target.  grid: x = tile, y = outer index o, z = slice of the targets.
template <int LOAD, int LOG_R, int LOG_LANES>
__global__ void __launch_bounds__(((1 << (LOG_R + LOG_LANES)) / 8) < 32 ? 32 : ((1 << (LOG_R + LOG_LANES)) / 8),
                                  ((1 << (LOG_R + LOG_LANES)) / 8) >= 512 ? 2 : ((1 << (LOG_R + LOG_LANES)) / 8) >= 256 ? 4 : 8)
ntt_strided_shared_src(const RingDev R, const PolyBatch B, u32 m_per_block) {
    constexpr int LANES = 1 << LOG_LANES, POINTS = 1 << (LOG_R + LOG_LANES);
    extern __shared__ __align__(16) u64 shared_src_smem[];
    u64* staged = shared_src_smem;                  // [POINTS] raw source words
    u64* sm = shared_src_smem + POINTS;             // [POINTS] exchange between stage groups
    ulonglong2* tws = (ulonglong2*)(shared_src_smem + 2 * POINTS);     // [2^LOG_R] twiddles of the current target
    grid_dependency_enter();
    const u32 o = blockIdx.y;
    const u32 m_begin = blockIdx.z * m_per_block;
    const u32 m_end = min(B.n_m, m_begin + m_per_block);
    {
        u32 o_hi = 0, o_lo = o;
        if (B.o_div) split_index(o, B.o_div, B.o_div_magic, o_hi, o_lo);
        const size_t src_off = B.o_div ? (size_t)o_hi * B.src_so2 + (size_t)o_lo * B.src_so : (size_t)o * B.src_so;
        const u64* src = (const u64*)B.src + src_off;
        if (B.div_t) {
            // the digit is a division by P away: (source - t) * P^{-1} modulo the digit's own prime, t the centred lift
            // of the polynomial's residue modulo P (exact: same value as dividing in the transform domain)
            const u32 i = o_lo;
            LoadConsts dc;
            dc.q = R.q[i];
            dc.mu = R.mu[i];
            dc.lift_mod = R.q[R.r];
            const u64* tp = B.div_t + (size_t)o_hi * B.div_so;
            if (R.fp_ok[i]) {
                // in fp64 (every value an exact integer): t lazily reduced by the load functor, the difference times
                // P^{-1} as a centred product, brought to [0, q) -- the digit must be the canonical residue, since it is
                // reduced into the other primes next
                const double qd = R.qd[i], pv = R.pinv_d[i], pq = R.pinv_q[i];
                dc.qd = qd;
                dc.c30 = R.c30_d[i];
                dc.c30q = R.c30_q[i];
                dc.wide = (dc.q >> 41) != 0;
                dc.k59 = dc.wide ? R.k59_d[i] : __dsub_rn(R.k59_d[i], __dadd_rn(qd, qd));
                const double q3 = __dadd_rn(__dadd_rn(qd, qd), qd);
                for (int w = threadIdx.x; w < POINTS; w += blockDim.x) {
                    const size_t idx = ((size_t)(w >> LOG_LANES) << LOG_C) + blockIdx.x * LANES + (w & (LANES - 1));
                    const double t = load_src_fp<LOAD_CENTRED>(tp, idx, dc);       // (-1.75q, 0.76q), or (0.25q, 2.76q) when wide
                    const double x = __dsub_rn(u2d(src[idx]), t);
                    double s2 = dc.wide ? fp_mul_centred(__dadd_rn(x, q3), pv, pq, qd) : fp_mul_centred_signed(x, pv, pq, qd);
                    if (s2 < 0.0) s2 = __dadd_rn(s2, qd);
                    staged[w] = d2u(s2);
                }
            } else {
                dc.lift_red = barrett64(dc.lift_mod, dc.q, dc.mu);
                const u64 pinv = R.pinv[i], pinvs = R.pinvs[i];
                for (int w = threadIdx.x; w < POINTS; w += blockDim.x) {
                    const size_t idx = ((size_t)(w >> LOG_LANES) << LOG_C) + blockIdx.x * LANES + (w & (LANES - 1));
                    const u64 t = load_src<LOAD_CENTRED>(tp, idx, dc);
                    staged[w] = mul_shoup(sub_mod(src[idx], t, dc.q), pinv, pinvs, dc.q);
                }
            }
        } else {
            for (int w = threadIdx.x; w < POINTS; w += blockDim.x)
                staged[w] = src[((size_t)(w >> LOG_LANES) << LOG_C) + blockIdx.x * LANES + (w & (LANES - 1))];
        }
    }
    __syncthreads();
    for (u32 m = m_begin; m < m_end; ++m) {
        const u32 mod = B.mod0 + ((B.mod_wrap && m >= B.mod_wrap) ? m - B.mod_wrap : m) * B.mod_step;
        if (own_prime(R, B, o, mod)) {
            // this digit's transform in its own prime exists already: copy the tile instead
            const u64* ds = B.diag_src + (size_t)(o / R.r) * B.diag_so + (size_t)mod * R.N;
            u64* dd = B.dst + (size_t)o * B.dst_so + (size_t)m * B.dst_sm;
            size_t tbase = 0;
            if (B.dtile_ptr) {
                u32 t_hi, t_lo;
                split_index(o, B.dtile_div, B.dtile_magic, t_hi, t_lo);
                tbase = ks_tile_base(R.N, B.n_m, B.dtile_div, t_hi, t_lo, m);
            }
            for (int w = threadIdx.x; w < POINTS; w += blockDim.x) {
                const size_t gidx = ((size_t)(w >> LOG_LANES) << LOG_C) + blockIdx.x * LANES + (w & (LANES - 1));
                if (B.dtile_ptr) B.dtile_ptr[tbase + (gidx / KS_TILE) * B.dtile_div * KS_TILE + gidx % KS_TILE] = ds[gidx];
                else dd[gidx] = ds[gidx];
            }
            continue;
        }
        if (R.fp_ok[mod]) strided_body<true, LOAD, LOG_R, LOG_LANES, true, true>(R, B, sm, tws, o, m, mod, staged);
        else strided_body<true, LOAD, LOG_R, LOG_LANES, false, true>(R, B, sm, tws, o, m, mod, staged);
        __syncthreads();            // the exchange buffer is free again
    }
}

// Contiguous pass: every warp transforms one chunk of 256 adjacent points (8 per thread) through
// the groups {3,3,2}; the chunk lives in the warp's own swizzled slice of shared memory between
// groups, so only warp-level synchronisation is needed.
// Forward: second pass (final reduction to [0, q), then the store functors).  Inverse: first pass
// (reads the batch source: plain residues, tiled/limb-split plaintexts, or a sum of arrays).
// TILED: the transform-domain side of the batch lives in the tile-major plaintext cache (B.tile_ptr).
// EPI: 0 = none; 1 = division by P per rotation (scatter through the rotation's permutation); 2 = per output
// (sum over the output's giant rotations, gathered through their permutations); 3 = plain (see ModDownEpilogue).
// DTILE: the forward result goes to the tile-major operand array of the inner product and nowhere else (ModUp: the
// hot case; its index arithmetic is hoisted out of the store loop and none of the other store functors is compiled in).
template <bool FWD, int EPI, bool FP, bool TILED, bool DTILE = false>
__device__ __forceinline__ void contig_body(const RingDev& R, const PolyBatch& B, u64* sm_raw, u32 o, u32 m, u32 mod,
                                            u32 chunk, int lane, const RotBatch& rb, const ModDownEpilogue& epi) {
    typedef typename Elem<FP>::T T;
    constexpr int LEN = 1 << LOG_C;
    T* sm = (T*)sm_raw;
    const u64 q = R.q[mod];
    const double qd = R.qd[mod];
    const ulonglong2* __restrict__ tw = (FWD ? R.tw_fwd : R.tw_inv) + (size_t)mod * R.N;
    u64* dst = B.dst + (size_t)o * B.dst_so + (size_t)m * B.dst_sm;
    const u64* src = FWD ? dst : (const u64*)B.src + (size_t)o * B.src_so + (size_t)m * B.src_sm;
    const u32 mult = (R.N >> LOG_C) + chunk;                   // twiddle index multiplier of this chunk
    const u64* gsrc = src + (size_t)chunk * LEN;
    u64* gdst = dst + (size_t)chunk * LEN;
    // byte addresses (shared window) of the thread's base point in each of the three access patterns
    const u32 slice = (u32)__cvta_generic_to_shared(sm);
    const u32 a_far = slice + 8u * (u32)swz(lane);                                    // points lane + 32 i
    const u32 a_mid = slice + 8u * (u32)swz((lane >> 2) * 32 + (lane & 3));           // points base + 4 i
    const u32 a_near = slice + 8u * (u32)swz(4 * lane);                               // points 4 (lane + 32 it) + i
    T e[8];
    size_t dtile_base = 0;
    if constexpr (DTILE) {
        u32 o_hi, o_lo;
        split_index(o, B.dtile_div, B.dtile_magic, o_hi, o_lo);
        dtile_base = ks_tile_base(R.N, B.n_m, B.dtile_div, o_hi, o_lo, m);
    }
    (void)dtile_base;
    if (FWD) {
        // group 0: K = 3, spacing 32
#pragma unroll
        for (int i = 0; i < 8; ++i) e[i] = ((const T*)gsrc)[lane + 32 * i];
        set_butterflies<3, true>(e, tw, 1u * mult, 0u, q, qd);
        swz_store_set<8, 5>(a_far, e);
        __syncwarp();
        // group 1: K = 3, spacing 4
        {
            const int blk = lane >> 2;
            swz_load_set<8, 2>(a_mid, e);
            set_butterflies<3, true>(e, tw, 8u * mult, (u32)blk, q, qd);
            swz_store_set<8, 2>(a_mid, e);
        }
        __syncwarp();
        // group 2: K = 2, adjacent points; two sets per thread
#pragma unroll
        for (int it = 0; it < 2; ++it) {
            const int s = lane + 32 * it;
            swz_load_set<4, 0>(a_near + (u32)(it * 8 * swz(128)), e);      // (swz(128) = 128: above the bits of 4 * lane)
            // the epilogue's operands do not depend on the transform: ask for them before the last butterflies
            u64 uu[4] = {0, 0, 0, 0}, cc[4] = {0, 0, 0, 0};
            u32 pp[4] = {0, 0, 0, 0};
            if (EPI == 2) {
                const u32 pp_out = o >> 1, comp = o & 1, ip = mod, nb = R.r + 1;
                const size_t n = (size_t)chunk * LEN + 4 * s;
                // three rotations at a time: their permutation entries are requested together, then all the words they
                // point at, so that a group costs two round trips instead of two per rotation
                for (u32 j0 = 0; j0 < epi.n_sum; j0 += 3) {
                    uint4 pv[3];
                    u64 uv[3][4], cv[3][4];
#pragma unroll
                    for (u32 t = 0; t < 3; ++t)
                        if (j0 + t < epi.n_sum) pv[t] = *(const uint4*)(epi.perm + (size_t)rb.key[j0 + t] * R.N + n);
#pragma unroll
                    for (u32 t = 0; t < 3; ++t) {
                        if (j0 + t >= epi.n_sum) continue;
                        const size_t rot = (size_t)(j0 + t) * epi.n_out + pp_out;
                        const u64* up = epi.u + ((rot * 2 + comp) * nb + ip) * R.N;
                        uv[t][0] = __ldg(up + pv[t].x); uv[t][1] = __ldg(up + pv[t].y);
                        uv[t][2] = __ldg(up + pv[t].z); uv[t][3] = __ldg(up + pv[t].w);
                        if (comp == 0) {
                            const u64* cp = epi.c0_base + rot * epi.c0_stride + (size_t)ip * R.N;
                            cv[t][0] = __ldg(cp + pv[t].x); cv[t][1] = __ldg(cp + pv[t].y);
                            cv[t][2] = __ldg(cp + pv[t].z); cv[t][3] = __ldg(cp + pv[t].w);
                        }
                    }
#pragma unroll
                    for (u32 t = 0; t < 3; ++t) {
                        if (j0 + t >= epi.n_sum) continue;
#pragma unroll
                        for (int w = 0; w < 4; ++w) {
                            uu[w] = add_mod(uu[w], uv[t][w], q);
                            if (comp == 0) cc[w] = add_mod(cc[w], cv[t][w], q);
                        }
                    }
                }
            }
            if (EPI == 3) {         // plain division: only the inner sum's residue is needed
                const u64* up = epi.u + ((size_t)o * (R.r + 1) + mod) * R.N + (size_t)chunk * LEN + 4 * s;
                const ulonglong2 u0 = *(const ulonglong2*)up, u1 = *(const ulonglong2*)(up + 2);
                uu[0] = u0.x; uu[1] = u0.y; uu[2] = u1.x; uu[3] = u1.y;
            }
            if (EPI == 1) {
                const u32 rot = o >> 1, comp = o & 1, ip = mod, nb = R.r + 1;
                const size_t n = (size_t)chunk * LEN + 4 * s;
                const u64* up = epi.u + ((size_t)o * nb + ip) * R.N + n;
                const ulonglong2 u0 = *(const ulonglong2*)up, u1 = *(const ulonglong2*)(up + 2);
                uu[0] = u0.x; uu[1] = u0.y; uu[2] = u1.x; uu[3] = u1.y;
                if (comp == 0) {
                    const u64* cp = epi.c0_base + (size_t)rb.c0[rot] * epi.c0_stride + (size_t)ip * R.N + n;
                    const ulonglong2 c0 = *(const ulonglong2*)cp, c1 = *(const ulonglong2*)(cp + 2);
                    cc[0] = c0.x; cc[1] = c0.y; cc[2] = c1.x; cc[3] = c1.y;
                }
                const uint4 pv = *(const uint4*)(epi.pinv + (size_t)rb.key[rot] * R.N + n);
                pp[0] = pv.x; pp[1] = pv.y; pp[2] = pv.z; pp[3] = pv.w;
            }
            set_butterflies<2, true>(e, tw, 64u * mult, (u32)s, q, qd);
            u64 v4[4];
            if (FP && (q >> 41)) {          // final reduction to [0, q)
#pragma unroll
                for (int i = 0; i < 4; ++i) v4[i] = d2u(fp_reduce(*(double*)&e[i], qd, R.qinv_d[mod]));
            } else if (FP) {
                const double qi = R.qinv_d[mod];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    double v = fp_centre(*(double*)&e[i], qd, qi);
                    if (v < 0.0) v = __dadd_rn(v, qd);
                    v4[i] = d2u(v);
                }
            } else {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    u64 v = *(u64*)&e[i];
                    if (v >= 2 * q) v -= 2 * q;
                    if (v >= q) v -= q;
                    v4[i] = v;
                }
            }
            if constexpr (DTILE) {
                // (4 adjacent coefficients never straddle a tile of 128)
                const u32 n = chunk * LEN + 4 * s;
                ulonglong2* gp = (ulonglong2*)(B.dtile_ptr + dtile_base + (size_t)(n / KS_TILE) * B.dtile_div * KS_TILE + n % KS_TILE);
                gp[0] = make_ulonglong2(v4[0], v4[1]);
                gp[1] = make_ulonglong2(v4[2], v4[3]);
                continue;
            }
            if (EPI == 2) {
                const u32 pp_out = o >> 1, comp = o & 1, ip = mod, r = R.r;
                u64* op = epi.out_base + (size_t)pp_out * epi.out_stride + ((size_t)comp * r + ip) * R.N + (size_t)chunk * LEN + 4 * s;
#pragma unroll
                for (int t = 0; t < 4; ++t)
                    v4[t] = add_mod(mul_shoup(sub_mod(uu[t], v4[t], q), R.pinv[ip], R.pinvs[ip], q), cc[t], q);
                ((ulonglong2*)op)[0] = make_ulonglong2(v4[0], v4[1]);
                ((ulonglong2*)op)[1] = make_ulonglong2(v4[2], v4[3]);
                continue;
            }
            if (EPI == 3) {
                u64* op = epi.out_base + (size_t)o * epi.out_stride + (size_t)mod * R.N + (size_t)chunk * LEN + 4 * s;
#pragma unroll
                for (int t = 0; t < 4; ++t) v4[t] = mul_shoup(sub_mod(uu[t], v4[t], q), R.pinv[mod], R.pinvs[mod], q);
                ((ulonglong2*)op)[0] = make_ulonglong2(v4[0], v4[1]);
                ((ulonglong2*)op)[1] = make_ulonglong2(v4[2], v4[3]);
                continue;
            }
            if (EPI == 1) {
                const u32 rot = o >> 1, comp = o & 1, ip = mod, r = R.r;
                u64* op = epi.out_base + (size_t)rb.out[rot] * epi.out_stride + ((size_t)comp * r + ip) * R.N;
#pragma unroll
                for (int t = 0; t < 4; ++t) {
                    u64 v = mul_shoup(sub_mod(uu[t], v4[t], q), R.pinv[ip], R.pinvs[ip], q);
                    v = add_mod(v, cc[t], q);
                    op[pp[t]] = v;
                }
                continue;
            }
            if constexpr (TILED) {   // tile-major plaintext cache; 4 adjacent coefficients never straddle a tile (tiles hold >= 16)
                const u32 pj = (B.o_base + o) / B.tile.n_terms - B.tile_pj0, term = (B.o_base + o) % B.tile.n_terms;
                const u32 n = chunk * LEN + 4 * s;
                unsigned char* stage = (unsigned char*)B.tile_ptr + tile_stage_of_word(B.tile, pj, term, mod, n);
                const u32 at = tile_word_index(B.tile, pj, term, n);
                const u32 fmt = tile_format(B.tile, mod);
                if (fmt == TILE_W64) {
                    if (B.split_bits && !(q >> 50)) {     // (the special prime of double hoisting stays in whole words)
#pragma unroll
                        for (int i = 0; i < 4; ++i) v4[i] = limb_split(v4[i], B.split_bits);
                    }
                    ulonglong2* gp = (ulonglong2*)(stage + (size_t)at * 8);
                    gp[0] = make_ulonglong2(v4[0], v4[1]);
                    gp[1] = make_ulonglong2(v4[2], v4[3]);
                } else {
                    *(uint4*)(stage + (size_t)at * 4) = make_uint4((u32)v4[0], (u32)v4[1], (u32)v4[2], (u32)v4[3]);
                    if (fmt == TILE_W40)
                        *(u32*)(stage + TILE_STAGE_WORDS * 4u + at) = (u32)(v4[0] >> 32) | ((u32)(v4[1] >> 32) << 8) |
                                                                     ((u32)(v4[2] >> 32) << 16) | ((u32)(v4[3] >> 32) << 24);
                }
                continue;
            }
            if (B.lift_ptr) {   // P times the value, into the extended-basis copy of the un-rotated inputs
                const u32 comp = (B.mod_wrap && m >= B.mod_wrap) ? 1u : 0u, nbp = R.r + 1;    // (n_m <= 2 * mod_wrap)
                u64* xp = B.lift_ptr + (size_t)o * B.lift_so + ((size_t)comp * nbp + mod) * R.N + (size_t)chunk * LEN + 4 * s;
                u64 p4[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    u64 hi = 0, lo = 0;
                    mac128(hi, lo, v4[i], R.pmod[mod]);
                    p4[i] = reduce128(hi, lo, q, R.mu[mod], R.c64[mod], R.c64s[mod]);
                }
                ((ulonglong2*)xp)[0] = make_ulonglong2(p4[0], p4[1]);
                ((ulonglong2*)xp)[1] = make_ulonglong2(p4[2], p4[3]);
                if (mod == 0) {     // the residue modulo P of P * ct is zero
                    u64* zp = B.lift_ptr + (size_t)o * B.lift_so + ((size_t)comp * nbp + R.r) * R.N + (size_t)chunk * LEN + 4 * s;
                    ((ulonglong2*)zp)[0] = make_ulonglong2(0, 0);
                    ((ulonglong2*)zp)[1] = make_ulonglong2(0, 0);
                }
            }
            if (B.split_bits) {
#pragma unroll
                for (int i = 0; i < 4; ++i) v4[i] = limb_split(v4[i], B.split_bits);
            }
            if (B.dtile_ptr) {  // operands of the key-switch inner product: tile-major (keys also permuted, times 2^64)
                if (B.scatter) {
                    const u32* sc = B.scatter + (size_t)(o / B.scatter_div) * R.N + chunk * LEN + 4 * s;
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        B.dtile_ptr[ks_tile_index(R.N, B.n_m, B.dtile_div, o, m, sc[i])] =
                            B.scatter_mont ? mul_shoup(v4[i], R.c64[mod], R.c64s[mod], q) : v4[i];
                } else {
                    ulonglong2* gp = (ulonglong2*)(B.dtile_ptr + ks_tile_index(R.N, B.n_m, B.dtile_div, o, m, chunk * LEN + 4 * s));
                    gp[0] = make_ulonglong2(v4[0], v4[1]);
                    gp[1] = make_ulonglong2(v4[2], v4[3]);
                }
                continue;
            }
            if (B.scatter) {    // permuted store (keys are kept pre-permuted by their automorphism)
                const u32* sc = B.scatter + (size_t)(o / B.scatter_div) * R.N + chunk * LEN + 4 * s;
                u64* sd = B.scatter_dst + (size_t)o * B.dst_so + (size_t)m * B.dst_sm;
#pragma unroll
                for (int i = 0; i < 4; ++i) sd[sc[i]] = B.scatter_mont ? mul_shoup(v4[i], R.c64[mod], R.c64s[mod], q) : v4[i];
                continue;
            }
            ulonglong2* gp = (ulonglong2*)(gdst + 4 * s);
            gp[0] = make_ulonglong2(v4[0], v4[1]);
            gp[1] = make_ulonglong2(v4[2], v4[3]);
        }
    } else {
        // inverse: groups in the opposite order
#pragma unroll
        for (int it = 0; it < 2; ++it) {
            const int s = lane + 32 * it;
            u64 v4[4];
            if constexpr (EPI == 2) {   // the residues of this output's giant rotations, each read through its rotation, summed
                const u32 pp_out = o >> 1, comp = o & 1, nb = R.r + 1;
                const size_t n = (size_t)chunk * LEN + 4 * s;
                v4[0] = v4[1] = v4[2] = v4[3] = 0;
                // three rotations at a time: their permutation entries are requested together, then all the words they
                // point at, so that a group costs two round trips instead of two per rotation (these launches are a few
                // polynomials only: latency is all they cost)
                for (u32 j0 = 0; j0 < epi.n_sum; j0 += 3) {
                    uint4 pv[3];
                    u64 uv[3][4];
#pragma unroll
                    for (u32 t = 0; t < 3; ++t)
                        if (j0 + t < epi.n_sum) pv[t] = *(const uint4*)(epi.perm + (size_t)rb.key[j0 + t] * R.N + n);
#pragma unroll
                    for (u32 t = 0; t < 3; ++t) {
                        if (j0 + t >= epi.n_sum) continue;
                        const u64* up = epi.u + ((((size_t)(j0 + t) * epi.n_out + pp_out) * 2 + comp) * nb + mod) * R.N;
                        uv[t][0] = __ldg(up + pv[t].x); uv[t][1] = __ldg(up + pv[t].y);
                        uv[t][2] = __ldg(up + pv[t].z); uv[t][3] = __ldg(up + pv[t].w);
                    }
#pragma unroll
                    for (u32 t = 0; t < 3; ++t) {
                        if (j0 + t >= epi.n_sum) continue;
#pragma unroll
                        for (int w = 0; w < 4; ++w) v4[w] = add_mod(v4[w], uv[t][w], q);
                    }
                }
            } else if constexpr (EPI == 4) {   // output assembly in the extended basis (see ModDownEpilogue::assemble)
                const u32 nb = R.r + 1, g1 = epi.n_sum;
                const size_t n = (size_t)chunk * LEN + 4 * s;
                u32 comp = 0, ju = 0, jc_lo = 1, jc_hi = 0;    // u-terms of giant steps 1..ju, rotated c0 parts of jc_lo..jc_hi
                bool ident = false;
                if (mod < R.r) { comp = m / R.r; ident = true; ju = g1; if (comp == 0) jc_hi = g1; }
                else if (m < 2) { comp = m; ju = g1; }
                else if (m < 4) { comp = m - 2; ident = true; }
                else { jc_lo = jc_hi = m - 3; }
                v4[0] = v4[1] = v4[2] = v4[3] = 0;
                if (ident) {
                    const u64* ap = epi.aext + (size_t)o * epi.aext_stride + ((size_t)comp * nb + mod) * R.N + n;
                    const ulonglong2 a = *(const ulonglong2*)ap, b = *(const ulonglong2*)(ap + 2);
                    v4[0] = a.x; v4[1] = a.y; v4[2] = b.x; v4[3] = b.y;
                }
                // (the producers stored every rotated term through its rotation already: plain loads; the words of
                // three giant steps are requested together)
                const u64* ub = epi.u + (((size_t)o * 2 + comp) * nb + mod) * R.N + n;          // giant step 1
                const size_t u_step = (size_t)epi.n_out * 2 * nb * R.N;
                for (u32 j0 = 1; j0 <= ju; j0 += 3) {
                    ulonglong2 a2[3], b2[3];
#pragma unroll
                    for (u32 t = 0; t < 3; ++t)
                        if (j0 + t <= ju) {
                            const u64* up = ub + (size_t)(j0 + t - 1) * u_step;
                            a2[t] = *(const ulonglong2*)up;
                            b2[t] = *(const ulonglong2*)(up + 2);
                        }
#pragma unroll
                    for (u32 t = 0; t < 3; ++t)
                        if (j0 + t <= ju) {
                            v4[0] = add_mod(v4[0], a2[t].x, q); v4[1] = add_mod(v4[1], a2[t].y, q);
                            v4[2] = add_mod(v4[2], b2[t].x, q); v4[3] = add_mod(v4[3], b2[t].y, q);
                        }
                }
                const u64* cb = epi.aext + (size_t)o * epi.aext_stride + (size_t)mod * R.N + n;  // inner sum (0, p), c0
                const size_t c_step = (size_t)epi.n_out * epi.aext_stride;
                for (u32 j0 = jc_lo; j0 <= jc_hi; j0 += 3) {
                    ulonglong2 a2[3], b2[3];
#pragma unroll
                    for (u32 t = 0; t < 3; ++t)
                        if (j0 + t <= jc_hi) {
                            const u64* cp = cb + (size_t)(j0 + t) * c_step;
                            a2[t] = *(const ulonglong2*)cp;
                            b2[t] = *(const ulonglong2*)(cp + 2);
                        }
#pragma unroll
                    for (u32 t = 0; t < 3; ++t)
                        if (j0 + t <= jc_hi) {
                            v4[0] = add_mod(v4[0], a2[t].x, q); v4[1] = add_mod(v4[1], a2[t].y, q);
                            v4[2] = add_mod(v4[2], b2[t].x, q); v4[3] = add_mod(v4[3], b2[t].y, q);
                        }
                }
            } else if constexpr (TILED) {  // read back from the tile-major plaintext cache
                const u32 pj = (B.o_base + o) / B.tile.n_terms - B.tile_pj0, term = (B.o_base + o) % B.tile.n_terms;
                const u32 n = chunk * LEN + 4 * s;
                const unsigned char* stage = (const unsigned char*)B.tile_ptr + tile_stage_of_word(B.tile, pj, term, mod, n);
                const u32 at = tile_word_index(B.tile, pj, term, n);
                const u32 fmt = tile_format(B.tile, mod);
                if (fmt == TILE_W64) {
                    const ulonglong2* gp = (const ulonglong2*)(stage + (size_t)at * 8);
                    const ulonglong2 a = gp[0], b = gp[1];
                    v4[0] = a.x; v4[1] = a.y; v4[2] = b.x; v4[3] = b.y;
                    if (B.split_bits && !(q >> 50)) {
#pragma unroll
                        for (int i = 0; i < 4; ++i) v4[i] = limb_join(v4[i], B.split_bits);
                    }
                } else {
                    const uint4 lo = *(const uint4*)(stage + (size_t)at * 4);
                    const u32 hi = fmt == TILE_W40 ? *(const u32*)(stage + TILE_STAGE_WORDS * 4u + at) : 0u;
                    v4[0] = lo.x | ((u64)(hi & 255u) << 32);
                    v4[1] = lo.y | ((u64)((hi >> 8) & 255u) << 32);
                    v4[2] = lo.z | ((u64)((hi >> 16) & 255u) << 32);
                    v4[3] = lo.w | ((u64)(hi >> 24) << 32);
                }
            } else {
                const ulonglong2* gp = (const ulonglong2*)(gsrc + 4 * s);
                const ulonglong2 a = gp[0], b = gp[1];
                v4[0] = a.x; v4[1] = a.y; v4[2] = b.x; v4[3] = b.y;
                if (B.split_bits) {
#pragma unroll
                    for (int i = 0; i < 4; ++i) v4[i] = limb_join(v4[i], B.split_bits);
                }
            }
            if (B.sum_terms) {      // the input is a sum of several arrays of the same shape
                const u64* sp = B.sum_src + (size_t)o * B.src_so + (size_t)m * B.src_sm + (size_t)chunk * LEN + 4 * s;
                // three arrays at a time, all their loads in flight together (g - 1 = 3 is the common case)
                u32 t = 0;
                for (; t + 3 <= B.sum_terms; t += 3) {
                    ulonglong2 a2[3], b2[3];
#pragma unroll
                    for (int j = 0; j < 3; ++j) {
                        a2[j] = *(const ulonglong2*)(sp + (size_t)(t + j) * B.sum_stride);
                        b2[j] = *(const ulonglong2*)(sp + (size_t)(t + j) * B.sum_stride + 2);
                    }
#pragma unroll
                    for (int j = 0; j < 3; ++j) {
                        v4[0] = add_mod(v4[0], a2[j].x, q); v4[1] = add_mod(v4[1], a2[j].y, q);
                        v4[2] = add_mod(v4[2], b2[j].x, q); v4[3] = add_mod(v4[3], b2[j].y, q);
                    }
                }
                for (; t < B.sum_terms; ++t) {
                    const ulonglong2 a2 = *(const ulonglong2*)(sp + (size_t)t * B.sum_stride);
                    const ulonglong2 b2 = *(const ulonglong2*)(sp + (size_t)t * B.sum_stride + 2);
                    v4[0] = add_mod(v4[0], a2.x, q); v4[1] = add_mod(v4[1], a2.y, q);
                    v4[2] = add_mod(v4[2], b2.x, q); v4[3] = add_mod(v4[3], b2.y, q);
                }
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) from_u64(e[i], v4[i]);
            set_butterflies<2, false>(e, tw, 64u * mult, (u32)s, q, qd);
            swz_store_set<4, 0>(a_near + (u32)(it * 8 * swz(128)), e);
        }
        __syncwarp();
        {
            const int blk = lane >> 2;
            swz_load_set<8, 2>(a_mid, e);
            set_butterflies<3, false>(e, tw, 8u * mult, (u32)blk, q, qd);
            centre_sums<3>(e, q, qd, R.qinv_d[mod]);
            swz_store_set<8, 2>(a_mid, e);
        }
        __syncwarp();
        swz_load_set<8, 5>(a_far, e);
        set_butterflies<3, false>(e, tw, 1u * mult, 0u, q, qd);
#pragma unroll
        for (int i = 0; i < 8; ++i) ((T*)gdst)[lane + 32 * i] = e[i];      // lazy, below 2q; the strided pass finishes
    }
}

// (the per-output forms run on a few polynomials per launch and hold the operands of three rotations at once: they
// trade resident blocks for registers)
template <bool FWD, int EPI, bool TILED, bool DTILE = false>
__global__ void __launch_bounds__(32 * CHUNKS_PER_BLOCK, (EPI == 2 || EPI == 4) ? 5 : 8) ntt_contig(const RingDev R, const PolyBatch B,
                                                                       u32 chunks_per_block, const RotBatch rb,
                                                                       const ModDownEpilogue epi) {
    __shared__ __align__(128) u64 sm_all[CHUNKS_PER_BLOCK << LOG_C];
    grid_dependency_enter();
    u32 o, m, mod;
    block_poly(B, o, m, mod);
    if (FWD && own_prime(R, B, o, mod)) return;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    if ((u32)warp >= chunks_per_block) return;
    const u32 chunk = blockIdx.x * chunks_per_block + warp;
    u64* sm = sm_all + (warp << LOG_C);
    if (R.fp_ok[mod]) contig_body<FWD, EPI, true, TILED, DTILE>(R, B, sm, o, m, mod, chunk, lane, rb, epi);
    else contig_body<FWD, EPI, false, TILED, DTILE>(R, B, sm, o, m, mod, chunk, lane, rb, epi);
}

NttGeometry ntt_geometry(u32 logN) {
    NttGeometry g;
    g.log_c = LOG_C;
    g.log_r = (int)logN - LOG_C;
    // strided tile: 2048 points (256 threads) unless the row count forces otherwise
    int log_lanes = 11 - g.log_r;
    if (log_lanes < 4) log_lanes = 4;
    if (log_lanes > 8) log_lanes = 8;
    g.strided_lanes = 1 << log_lanes;
    g.strided_threads = ((1 << g.log_r) * g.strided_lanes) / 8 < 32 ? 32 : ((1 << g.log_r) * g.strided_lanes) / 8;
    g.contig_lanes = (1 << g.log_r) < CHUNKS_PER_BLOCK ? (1 << g.log_r) : CHUNKS_PER_BLOCK;
    g.contig_threads = 32 * CHUNKS_PER_BLOCK;
    g.contig_pad = 0;
    return g;
}

// Grid of a batch of n_polys = n_outer * n_m polynomials with x_blocks blocks each: (x, m, o) with the reciprocals
// the kernels use instead of divisions, when the outer count fits the grid's z extent; else (x, o * n_m + m).
static dim3 poly_grid(PolyBatch& B, u32 x_blocks, u32 n_polys) {
    const u32 n_outer = n_polys / B.n_m;
    B.grid3 = 0;
    B.o_div_magic = B.dtile_magic = 0;
    if (n_outer * B.n_m != n_polys || n_outer > 65535u || B.n_m > 65535u) return dim3(x_blocks, n_polys);
    B.grid3 = 1;
    if (B.o_div) B.o_div_magic = (u32)((((u64)1 << 32) + B.o_div - 1) / B.o_div);
    if (B.dtile_div) B.dtile_magic = (u32)((((u64)1 << 32) + B.dtile_div - 1) / B.dtile_div);
    return dim3(x_blocks, B.n_m, n_outer);
}

template <bool FWD, int LOAD, int LOG_R, int LOG_LANES>
static void launch_strided_t(const RingHost& ring, const PolyBatch& B_in, u32 n_polys, cudaStream_t stream) {
    constexpr int NT = ((1 << (LOG_R + LOG_LANES)) / 8) < 32 ? 32 : ((1 << (LOG_R + LOG_LANES)) / 8);
    PolyBatch B = B_in;
    const dim3 grid = poly_grid(B, (1u << LOG_C) >> LOG_LANES, n_polys);
    launch_dependent(ring, ntt_strided<FWD, LOAD, LOG_R, LOG_LANES>, grid, dim3(NT), 0, stream, ring.dev, B);
}

template <int LOAD, int LOG_R, int LOG_LANES>
static void launch_shared_src_t(const RingHost& ring, const PolyBatch& B_in, u32 n_outer, cudaStream_t stream) {
    PolyBatch B = B_in;             // (its grid is (tile, o, slice of the targets): o is never divided out)
    B.grid3 = 0;
    B.dtile_magic = B.dtile_div ? (u32)((((u64)1 << 32) + B.dtile_div - 1) / B.dtile_div) : 0u;
    B.o_div_magic = B.o_div ? (u32)((((u64)1 << 32) + B.o_div - 1) / B.o_div) : 0u;
    constexpr int NT = ((1 << (LOG_R + LOG_LANES)) / 8) < 32 ? 32 : ((1 << (LOG_R + LOG_LANES)) / 8);
    constexpr u32 S = (1u << LOG_C) >> LOG_LANES;
    // targets per block: fewer blocks share the source better but quantise into waves; cost model =
    // waves x (targets per block + half a unit for staging the source)
    const u32 slots = 148u * (NT >= 512 ? 2 : NT >= 256 ? 4 : 8);
    u32 best = 1;
    double best_cost = 1e30;
    for (u32 per = 1; per <= B.n_m; ++per) {
        const u32 slices = (B.n_m + per - 1) / per;
        if ((B.n_m + slices - 1) / slices != per) continue;         // keep the slices balanced
        const u32 blocks = S * n_outer * slices;
        const double cost = (double)((blocks + slots - 1) / slots) * (per + 0.5);
        if (cost <= best_cost) { best_cost = cost; best = per; }
    }
    dim3 grid(S, n_outer, (B.n_m + best - 1) / best);
    constexpr size_t smem = (size_t)2 * 8 * (1u << (LOG_R + LOG_LANES)) + (size_t)16 * (1u << LOG_R);
    static bool attr_set[MAX_DEVICES] = {false};     // opt in once per device to more than 48 KB of dynamic shared memory
    if (smem > 48 * 1024 && !attr_set[device_slot(ring)]) {
        cudaFuncSetAttribute(ntt_strided_shared_src<LOAD, LOG_R, LOG_LANES>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                             (int)smem);
        attr_set[device_slot(ring)] = true;
    }
    launch_dependent(ring, ntt_strided_shared_src<LOAD, LOG_R, LOG_LANES>, grid, dim3(NT), smem, stream, ring.dev, B, best);
}

template <bool FWD, int LOAD>
static cudaError_t launch_strided(const RingHost& ring, const PolyBatch& B, u32 n_polys, cudaStream_t stream) {
    if (n_polys == 0) return cudaSuccess;
    ProfScope prof(ring.prof, FWD ? CAT_NTT_FWD_STRIDED : CAT_NTT_INV_STRIDED, stream);
    if constexpr (FWD && (LOAD == LOAD_REDUCE || LOAD == LOAD_CENTRED)) {
        const u32 n_outer = n_polys / B.n_m;
        if (B.src_sm == 0 && B.n_m > 1 && n_outer <= 65535 && !B.tile_ptr) {
            switch (ring.geom.log_r) {
                case 2: launch_shared_src_t<LOAD, 2, 8>(ring, B, n_outer, stream); break;
                case 3: launch_shared_src_t<LOAD, 3, 8>(ring, B, n_outer, stream); break;
                case 4: launch_shared_src_t<LOAD, 4, 7>(ring, B, n_outer, stream); break;
                case 5: launch_shared_src_t<LOAD, 5, 6>(ring, B, n_outer, stream); break;
                case 6: launch_shared_src_t<LOAD, 6, 5>(ring, B, n_outer, stream); break;
                case 7: launch_shared_src_t<LOAD, 7, 3>(ring, B, n_outer, stream); break;
                case 8: launch_shared_src_t<LOAD, 8, 3>(ring, B, n_outer, stream); break;
                default: return cudaErrorInvalidValue;
            }
            return cudaGetLastError();
        }
    }
    switch (ring.geom.log_r) {
        case 2: launch_strided_t<FWD, LOAD, 2, 8>(ring, B, n_polys, stream); break;
        case 3: launch_strided_t<FWD, LOAD, 3, 8>(ring, B, n_polys, stream); break;
        case 4: launch_strided_t<FWD, LOAD, 4, 7>(ring, B, n_polys, stream); break;
        case 5: launch_strided_t<FWD, LOAD, 5, 6>(ring, B, n_polys, stream); break;
        case 6: launch_strided_t<FWD, LOAD, 6, 5>(ring, B, n_polys, stream); break;
        case 7: launch_strided_t<FWD, LOAD, 7, 4>(ring, B, n_polys, stream); break;
        case 8: launch_strided_t<FWD, LOAD, 8, 4>(ring, B, n_polys, stream); break;
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

template <bool FWD>
static cudaError_t launch_contig(const RingHost& ring, const PolyBatch& B_in, u32 n_polys, cudaStream_t stream,
                                 const RotBatch* rb = nullptr, const ModDownEpilogue* epi = nullptr) {
    if (n_polys == 0) return cudaSuccess;
    ProfScope prof(ring.prof, FWD ? CAT_NTT_FWD_CONTIG : CAT_NTT_INV_CONTIG, stream);
    const u32 chunks = 1u << ring.geom.log_r;
    const u32 cpb = (u32)ring.geom.contig_lanes;
    PolyBatch B = B_in;
    const dim3 grid = poly_grid(B, chunks / cpb, n_polys);
    if (FWD && epi && epi->plain) {
        launch_dependent(ring, ntt_contig<FWD, 3, false>, grid, dim3(32 * CHUNKS_PER_BLOCK), 0, stream, ring.dev, B, cpb, *rb,
                         *epi);
    } else if (!FWD && epi && epi->assemble) {
        launch_dependent(ring, ntt_contig<false, 4, false>, grid, dim3(32 * CHUNKS_PER_BLOCK), 0, stream, ring.dev, B, cpb, *rb,
                         *epi);
    } else if (epi && epi->n_sum) {
        launch_dependent(ring, ntt_contig<FWD, 2, false>, grid, dim3(32 * CHUNKS_PER_BLOCK), 0, stream, ring.dev, B, cpb, *rb,
                         *epi);
    } else if (FWD && epi) {
        launch_dependent(ring, ntt_contig<FWD, 1, false>, grid, dim3(32 * CHUNKS_PER_BLOCK), 0, stream, ring.dev, B, cpb, *rb,
                         *epi);
    } else {
        static const RotBatch no_rb = {};
        static const ModDownEpilogue no_epi = {};
        if (B.tile_ptr)
            launch_dependent(ring, ntt_contig<FWD, 0, true>, grid, dim3(32 * CHUNKS_PER_BLOCK), 0, stream, ring.dev, B, cpb,
                             no_rb, no_epi);
        else if (FWD && B.dtile_ptr && !B.scatter && !B.lift_ptr && !B.split_bits)
            launch_dependent(ring, ntt_contig<true, 0, false, true>, grid, dim3(32 * CHUNKS_PER_BLOCK), 0, stream, ring.dev, B,
                             cpb, no_rb, no_epi);
        else
            launch_dependent(ring, ntt_contig<FWD, 0, false>, grid, dim3(32 * CHUNKS_PER_BLOCK), 0, stream, ring.dev, B, cpb,
                             no_rb, no_epi);
    }
    return cudaGetLastError();
}

cudaError_t ntt_forward(const RingHost& ring, const PolyBatch& B, u32 n_outer, int load, cudaStream_t stream) {
    const u32 n_polys = n_outer * B.n_m;
    cudaError_t e;
    if (load == LOAD_PLAIN) e = launch_strided<true, LOAD_PLAIN>(ring, B, n_polys, stream);
    else if (load == LOAD_REDUCE) e = launch_strided<true, LOAD_REDUCE>(ring, B, n_polys, stream);
    else if (load == LOAD_I64) e = launch_strided<true, LOAD_I64>(ring, B, n_polys, stream);
    else if (load == LOAD_I64_MONT) e = launch_strided<true, LOAD_I64_MONT>(ring, B, n_polys, stream);
    else e = launch_strided<true, LOAD_CENTRED>(ring, B, n_polys, stream);
    if (e != cudaSuccess) return e;
    return launch_contig<true>(ring, B, n_polys, stream);
}

cudaError_t ntt_forward_moddown(const RingHost& ring, const PolyBatch& B, u32 n_outer, const RotBatch& rb,
                                const ModDownEpilogue& epi, cudaStream_t stream) {
    const u32 n_polys = n_outer * B.n_m;
    cudaError_t e = launch_strided<true, LOAD_CENTRED>(ring, B, n_polys, stream);
    if (e != cudaSuccess) return e;
    return launch_contig<true>(ring, B, n_polys, stream, &rb, &epi);
}

// Forward transform whose final store is permuted: polynomial (o, m) ends up at
// final[(o*dst_so + m*dst_sm) + scatter[(o / scatter_div)*N + n]].  B.dst is a staging buffer of the same shape.
cudaError_t ntt_forward_split(const RingHost& ring, const PolyBatch& B0, u32 n_outer, int load, u64* final_dst,
                              const u32* scatter, u32 scatter_div, cudaStream_t stream) {
    PolyBatch B = B0;
    const u32 n_polys = n_outer * B.n_m;
    cudaError_t e;
    if (load == LOAD_PLAIN) e = launch_strided<true, LOAD_PLAIN>(ring, B, n_polys, stream);
    else e = launch_strided<true, LOAD_REDUCE>(ring, B, n_polys, stream);
    if (e != cudaSuccess) return e;
    B.scatter = scatter;
    B.scatter_div = scatter_div;
    B.scatter_dst = final_dst;
    B.scatter_mont = 1;           // (the only permuted store is that of the rotation keys)
    B.dtile_ptr = final_dst;      // tile-major: o = (key * r + digit) * 2 + component
    B.dtile_div = scatter_div;
    return launch_contig<true>(ring, B, n_polys, stream);
}

cudaError_t ntt_inverse_gathersum(const RingHost& ring, const PolyBatch& B, u32 n_outer, const RotBatch& rb,
                                  const ModDownEpilogue& epi, cudaStream_t stream) {
    const u32 n_polys = n_outer * B.n_m;
    cudaError_t e = launch_contig<false>(ring, B, n_polys, stream, &rb, &epi);
    if (e != cudaSuccess) return e;
    return launch_strided<false, LOAD_PLAIN>(ring, B, n_polys, stream);
}

// Last step of the output assembly in the extended basis: the inverse transforms above left, per output p and
// component, the sum of all terms modulo every q_i (in ct) and each separately rounded term's residue modulo P as a
// centred lift plus 2^59 (in T, n_t polynomials per output, indexed as ModDownEpilogue::assemble lists them):
//   ct[p][comp][i][n] = (ct[p][comp][i][n] - sum_terms t_term[n]) * P^{-1}  (mod q_i)
// low non-null: the rescale (Sec. 2.1) follows in the same thread, which holds all residues of its coefficient: the
// result goes to low[p][comp][r-1][N] as c'_i = (c_i - centred(c_{r-1})) * q_{r-1}^{-1} and ct only held the sums.
__global__ void __launch_bounds__(256) finish_division_kernel(const RingDev R, u64* __restrict__ ct, long long ct_stride,
                                                              const u64* __restrict__ T, u32 n_t, const RescaleConsts rc,
                                                              u64* __restrict__ low) {
    grid_dependency_enter();
    const u32 n = blockIdx.x * 256 + threadIdx.x;
    const u32 p = blockIdx.y >> 1, comp = blockIdx.y & 1;
    const u64* tp = T + (size_t)p * n_t * R.N + n;
    u64* cp = ct + (size_t)p * ct_stride + (size_t)comp * R.r * R.N + n;
    u64 v[MAX_MODULI];
#pragma unroll
    for (int i = 0; i < MAX_MODULI; ++i)
        if ((u32)i < R.r) v[i] = cp[(size_t)i * R.N];
    // this component's terms: polynomials comp, comp + 2 and, for component 0, 4 .. n_t - 1.  Their centred values are
    // added as integers, eight at a time (each is below 2^59 in magnitude), and the sum is reduced once per prime
    const u32 nt = comp == 0 ? n_t - 2 : 2u;
    for (u32 k0 = 0; k0 < nt; k0 += 8) {
        i64 S = 0;
        for (u32 k = k0; k < nt && k < k0 + 8; ++k) {
            const u32 m = k < 2 ? comp + 2 * k : k + 2;
            S += (i64)(tp[(size_t)m * R.N] - (1ull << 59));
        }
        const bool neg = S < 0;
        const u64 a = neg ? (u64)(-S) : (u64)S;
#pragma unroll
        for (int i = 0; i < MAX_MODULI; ++i)
            if ((u32)i < R.r) {
                u64 t = barrett64(a, R.q[i], R.mu[i]);
                if (neg && t) t = R.q[i] - t;
                v[i] = sub_mod(v[i], t, R.q[i]);
            }
    }
#pragma unroll
    for (int i = 0; i < MAX_MODULI; ++i)
        if ((u32)i < R.r) v[i] = mul_shoup(v[i], R.pinv[i], R.pinvs[i], R.q[i]);
    if (!low) {
#pragma unroll
        for (int i = 0; i < MAX_MODULI; ++i)
            if ((u32)i < R.r) cp[(size_t)i * R.N] = v[i];
        return;
    }
    u64 t = 0;                      // the residue that is dropped
#pragma unroll
    for (int i = 0; i < MAX_MODULI; ++i) {
        u64 vi = v[i];
        asm volatile("" : "+l"(vi));    // (keeps the selection a chain of moves: as an indexed read it would put v in local memory)
        if ((u32)i == R.r - 1) t = vi;
    }
    const bool high = t > (R.q[R.r - 1] - 1) / 2;
    u64* lp = low + ((size_t)p * 2 + comp) * (R.r - 1) * R.N + n;
#pragma unroll
    for (int i = 0; i < MAX_MODULI; ++i)
        if ((u32)i + 1 < R.r) {
            const u64 q = R.q[i];
            u64 tq = barrett64(t, q, R.mu[i]);
            if (high) tq = sub_mod(tq, rc.qlmod[i], q);
            lp[(size_t)i * R.N] = mul_shoup(sub_mod(v[i], tq, q), rc.inv[i], rc.invs[i], q);
        }
}

// The same in fp64 (every value an exact integer below 2^53), for rings whose ciphertext primes are all on the fp64
// path: a 64-bit modular product costs about twenty integer instructions, an exact fp64 one six on a pipe that is
// otherwise idle here.  Each term sum S = s_hi 2^30 + s_lo is reduced as s_hi (2^30 mod q) + s_lo; products come back
// centred and are brought to [0, q) only where a canonical residue is needed (the stored words, the dropped residue).
__device__ __forceinline__ double fp_times_const(double x, bool wide, double w, double wq, double q, double qinv) {
    // x an integer of magnitude below 2^50 (any sign): x * w mod q in [0, q)
    double s2;
    if (wide) s2 = fp_mul_centred(__dadd_rn(fp_centre(x, q, qinv), q), w, wq, q);     // operand in (0.5q, 1.5q)
    else s2 = fp_mul_centred_signed(x, w, wq, q);
    return s2 < 0.0 ? __dadd_rn(s2, q) : s2;
}

__global__ void __launch_bounds__(256) finish_division_fp_kernel(const RingDev R, u64* __restrict__ ct, long long ct_stride,
                                                                 const u64* __restrict__ T, u32 n_t, const RescaleConsts rc,
                                                                 u64* __restrict__ low) {
    grid_dependency_enter();
    const u32 n = blockIdx.x * 256 + threadIdx.x;
    const u32 p = blockIdx.y >> 1, comp = blockIdx.y & 1;
    const u64* tp = T + (size_t)p * n_t * R.N + n;
    u64* cp = ct + (size_t)p * ct_stride + (size_t)comp * R.r * R.N + n;
    double v[MAX_MODULI];
#pragma unroll
    for (int i = 0; i < MAX_MODULI; ++i)
        if ((u32)i < R.r) v[i] = u2d(cp[(size_t)i * R.N]);
    const u32 nt = comp == 0 ? n_t - 2 : 2u;
    for (u32 k0 = 0; k0 < nt; k0 += 8) {
        i64 S = 0;
        for (u32 k = k0; k < nt && k < k0 + 8; ++k) {
            const u32 m = k < 2 ? comp + 2 * k : k + 2;
            S += (i64)(tp[(size_t)m * R.N] - (1ull << 59));
        }
        const i64 s_hi = S >> 30;                               // |s_hi| < 2^33
        const double lo = u2d((u64)(S & ((1ll << 30) - 1)));
        const bool sneg = s_hi < 0;
        const double ah = u2d((u64)(sneg ? -s_hi : s_hi));
#pragma unroll
        for (int i = 0; i < MAX_MODULI; ++i)
            if ((u32)i < R.r) {
                const double sm = fp_mul_centred(ah, R.c30_d[i], R.c30_q[i], R.qd[i]);      // within 0.75 q
                const double x = __dsub_rn(__dsub_rn(v[i], sneg ? -sm : sm), lo);
                v[i] = fp_centre(x, R.qd[i], R.qinv_d[i]);
            }
    }
#pragma unroll
    for (int i = 0; i < MAX_MODULI; ++i)
        if ((u32)i < R.r) v[i] = fp_times_const(v[i], (R.q[i] >> 41) != 0, R.pinv_d[i], R.pinv_q[i], R.qd[i], R.qinv_d[i]);
    if (!low) {
#pragma unroll
        for (int i = 0; i < MAX_MODULI; ++i)
            if ((u32)i < R.r) cp[(size_t)i * R.N] = d2u(v[i]);
        return;
    }
    double t = 0.0;                 // the residue that is dropped (below 2^46: the launcher checked)
#pragma unroll
    for (int i = 0; i < MAX_MODULI; ++i) {
        double vi = v[i];
        asm volatile("" : "+d"(vi));    // (keeps the selection a chain of moves: as an indexed read it would put v in local memory)
        if ((u32)i == R.r - 1) t = vi;
    }
    const bool high = d2u(t) > (R.q[R.r - 1] - 1) / 2;
    u64* lp = low + ((size_t)p * 2 + comp) * (R.r - 1) * R.N + n;
#pragma unroll
    for (int i = 0; i < MAX_MODULI; ++i)
        if ((u32)i + 1 < R.r) {
            double tq = fp_reduce(t, R.qd[i], R.qinv_d[i]);
            if (high) tq = __dsub_rn(tq, rc.qlmod_d[i]);
            const double y = fp_times_const(__dsub_rn(v[i], tq), (R.q[i] >> 41) != 0, rc.inv_d[i], rc.inv_q[i], R.qd[i],
                                            R.qinv_d[i]);
            lp[(size_t)i * R.N] = d2u(y);
        }
}

cudaError_t finish_division(const RingHost& ring, u64* ct, long long ct_stride, const u64* T, u32 n_t, u32 n_out,
                            cudaStream_t stream, const RescaleConsts* rc, u64* low) {
    ProfScope prof(ring.prof, CAT_DIVIDE, stream);
    RescaleConsts none;
    memset(&none, 0, sizeof(none));
    bool fp = true;
    for (u32 i = 0; i < ring.dev.r; ++i) fp = fp && ring.dev.fp_ok[i];
    if (rc && ring.q[ring.dev.r - 1] >= (1ull << 46)) fp = false;
    if (fp) {
        launch_dependent(ring, finish_division_fp_kernel, dim3(ring.dev.N / 256, n_out * 2), dim3(256), 0, stream, ring.dev,
                         ct, ct_stride, T, n_t, rc ? *rc : none, rc ? low : (u64*)nullptr);
        return cudaGetLastError();
    }
    launch_dependent(ring, finish_division_kernel, dim3(ring.dev.N / 256, n_out * 2), dim3(256), 0, stream, ring.dev, ct,
                     ct_stride, T, n_t, rc ? *rc : none, rc ? low : (u64*)nullptr);
    return cudaGetLastError();
}

cudaError_t ntt_inverse(const RingHost& ring, const PolyBatch& B, u32 n_outer, cudaStream_t stream) {
    const u32 n_polys = n_outer * B.n_m;
    cudaError_t e = launch_contig<false>(ring, B, n_polys, stream);
    if (e != cudaSuccess) return e;
    return launch_strided<false, LOAD_PLAIN>(ring, B, n_polys, stream);
}

}  // namespace bf
