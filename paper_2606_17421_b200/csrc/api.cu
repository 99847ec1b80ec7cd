// C ABI of libbifrost: context and table set-up, key loading, weight encoding, and the launch
// sequence of the encrypted linear layer (Alg. 3: EncodeWeights, FHE_Linear; Sec. 4.2).
#include <cmath>
#include <cstdlib>
#include <cstdio>
#include <cstring>
#include <map>
#include <new>
#include <string>
#include <vector>

#include "../../include/bifrost.h"
#include "bf_host.h"

using namespace bf;

typedef unsigned __int128 u128;

// ------------------------------------------------------------------------------------------------
// host number theory (table set-up only)
static u64 h_mulmod(u64 a, u64 b, u64 q) { return (u64)((u128)a * b % q); }
static u64 h_powmod(u64 a, u64 e, u64 q) {
    u64 r = 1 % q;
    a %= q;
    for (; e; e >>= 1) {
        if (e & 1) r = h_mulmod(r, a, q);
        a = h_mulmod(a, a, q);
    }
    return r;
}
static u64 h_invmod(u64 a, u64 q) { return h_powmod(a % q, q - 2, q); }
static u64 h_shoup(u64 w, u64 q) { return (u64)(((u128)w << 64) / q); }

static bool h_is_prime(u64 n) {
    if (n < 2) return false;
    const u64 small[] = {2, 3, 5, 7, 11, 13, 17, 19, 23, 29, 31, 37};
    for (u64 p : small) {
        if (n % p == 0) return n == p;
    }
    u64 d = n - 1;
    int s = 0;
    while (!(d & 1)) { d >>= 1; ++s; }
    for (u64 a : small) {              // these witnesses are conclusive below 2^64
        u64 x = h_powmod(a, d, n);
        if (x == 1 || x == n - 1) continue;
        bool composite = true;
        for (int i = 1; i < s && composite; ++i) {
            x = h_mulmod(x, x, n);
            if (x == n - 1) composite = false;
        }
        if (composite) return false;
    }
    return true;
}

static u32 h_brev(u32 x, int bits) {
    u32 r = 0;
    for (int i = 0; i < bits; ++i) { r = (r << 1) | (x & 1); x >>= 1; }
    return r;
}

// a primitive 2N-th root of unity modulo q
static u64 h_root_2n(u64 q, u32 N) {
    const u64 e = (q - 1) / (2ull * N);
    for (u64 x = 3; x < q; ++x) {
        u64 psi = h_powmod(x, e, q);
        if (h_powmod(psi, N, q) == q - 1) return psi;
    }
    return 0;
}

// ------------------------------------------------------------------------------------------------
struct DevBuf {
    void* p = nullptr;
    size_t cap = 0;
};

struct bf_weights {
    u32 d_out, d_in, n_in, n_out;
    u32 b, g;           // baby/giant split the diagonals are grouped by (the plan's unless bf_encode_weights_split chose)
    u64* pt;            // groups pj = j*n_out + p of terms t = q*b + k in the tile-major layout `lay`;
                        // NTT domain, Montgomery form (times 2^64 mod q_i), limbs split when the primes allow
    TileLayout lay;
    size_t bytes;
    // coefficient form (bf_set_coefficient_cache): pt is null and the rounded integer coefficients of the diagonals
    // are kept instead, [diagonal][N] in the order [j][p][q][k], 64- or 32-bit; every call transforms them
    void* coef = nullptr;
    u32 coef_bits = 0;
};

struct bf_ctx {
    RingHost ring;
    Profiler prof;
    u32 N, logN, r;
    double scale;
    bf_plan plan;
    cudaStream_t stream;
    int device;
    ulonglong2 *tw_fwd = nullptr, *tw_inv = nullptr;
    u32* slot_of_pos = nullptr;
    double2 *T = nullptr, *Z = nullptr;
    double* enc_consts = nullptr;   // per-prime constants of the encoder's fp64 load
    // fallback path: bound on the scratch that holds just-encoded output groups between the encoder and the
    // multiply-accumulate (at least one group is always held).  Measured on a LLaMA-3-8B layer: 1 GiB 78 ms,
    // 2 GiB 73 ms, 4 GiB 70 ms, 8 GiB 69 ms: the rotated inputs are re-read once per round
    size_t encode_scratch_bytes = (size_t)4 << 30;
    u32 coef_cache_bits = 0;        // 64 / 32: weights encoded from now on are kept as rounded coefficients
    int* overflow_flag = nullptr;   // [0]: encoder range overflow; [1]: a bounded device-side wait gave up
    int* device_error = nullptr;
    // rotation keys
    std::map<u32, int> key_of_steps;
    u64* keys = nullptr;
    u32* perms = nullptr;            // [n_keys][N] pinv: where position n goes under the key's automorphism
    u32* perms_fwd = nullptr;        // [n_keys][N] perm: rotated[n] = unrotated[perm[n]] (per-output division by P)
    u32 n_keys = 0;
    // scratch (grow-only)
    size_t dig_half = 0;            // words from a digit set in Dig to its staging twin
    DevBuf X, X0, Aext, Dig, U, Ubig, Tc, Tn, Cc, A, Rres, Lfull, fft, coef, ptnat, ptjit, stage_in, stage_out, nm_a, nm_b;
    u64 cache_budget = 0, cache_used = 0;
    std::vector<bf_weights*> weights;
    std::string cuda_msg;
    // Captured launch sequences of bf_linear, replayed on later calls with the same arguments.
    struct GraphEntry {
        cudaGraphExec_t exec = nullptr;
        u64 epoch = 0;
        u32 seen = 0;
        bool unusable = false;
        uint64_t launches[CAT_COUNT] = {0};
        uint64_t key_bytes_distinct = 0, key_bytes_per_rotation = 0;
    };
    struct GraphKey {
        const void *ct_in, *weights, *ct_out;
        u32 d_out, d_in;
        bool rescaled;
        bool operator<(const GraphKey& o) const {
            if (rescaled != o.rescaled) return rescaled < o.rescaled;
            if (ct_in != o.ct_in) return ct_in < o.ct_in;
            if (weights != o.weights) return weights < o.weights;
            if (ct_out != o.ct_out) return ct_out < o.ct_out;
            if (d_out != o.d_out) return d_out < o.d_out;
            return d_in < o.d_in;
        }
    };
    std::map<GraphKey, GraphEntry> graphs;
    u64 epoch = 1;                 // bumped whenever memory the graphs point into is replaced
    int use_graphs = 1;
    // Independent key-switch chains of one call (groups of baby rotations; groups of giant rotations) run
    // on side streams between a fork and a join, so that one chain's HBM-bound inner product overlaps
    // another chain's arithmetic-bound transforms.  lane 0 is the context's stream.
    static constexpr int MAX_LANES = 4;
    int n_lanes = 2;                // measured: two chains overlap best (0.651 -> 0.625 ms on the 768 x 2304 layer)
    cudaStream_t side[MAX_LANES - 1] = {nullptr, nullptr, nullptr};
    cudaEvent_t ev_fork = nullptr, ev_join[MAX_LANES - 1] = {nullptr, nullptr, nullptr};
    // stage timing
    int timing = 0;
    cudaEvent_t ev[5] = {nullptr, nullptr, nullptr, nullptr, nullptr};
    bool ev_valid = false;
};

#define CK(call)                                                              \
    do {                                                                      \
        cudaError_t e__ = (call);                                             \
        if (e__ != cudaSuccess) {                                             \
            ctx->cuda_msg = std::string(#call) + ": " + cudaGetErrorString(e__); \
            return BF_ERR_CUDA;                                               \
        }                                                                     \
    } while (0)

static int ensure(bf_ctx* ctx, DevBuf& b, size_t bytes) {
    if (b.cap >= bytes) return BF_OK;
    CK(cudaStreamSynchronize(ctx->stream));
    if (b.p) CK(cudaFree(b.p));
    b.p = nullptr;
    b.cap = 0;
    cudaError_t e = cudaMalloc(&b.p, bytes);
    if (e != cudaSuccess) {
        cudaGetLastError();
        ctx->cuda_msg = std::string("cudaMalloc: ") + cudaGetErrorString(e);
        return BF_ERR_OOM;
    }
    b.cap = bytes;
    ctx->epoch++;                  // captured launch sequences may point into the old buffer
    return BF_OK;
}

#define TRY(call)                     \
    do {                              \
        int s__ = (call);             \
        if (s__ != BF_OK) return s__; \
    } while (0)

static bool is_pow2(u32 x) { return x && !(x & (x - 1)); }

extern "C" const char* bf_strerror(int code) {
    switch (code) {
        case BF_OK: return "ok";
        case BF_ERR_INVALID_ARG: return "invalid argument";
        case BF_ERR_BAD_PRIME: return "bad prime (not prime, not 1 mod 2N, duplicate, or >= 2^60)";
        case BF_ERR_SHAPE: return "shape does not match the plan";
        case BF_ERR_LEVEL: return "bad level";
        case BF_ERR_MISSING_KEY: return "rotation key not loaded";
        case BF_ERR_OOM: return "out of memory or over the cache budget";
        case BF_ERR_CUDA: return "CUDA error";
        case BF_ERR_RANGE: return "encoded coefficient out of range";
        case BF_ERR_TIMEOUT: return "a bounded device-side wait gave up (results of that call are invalid)";
        case BF_ERR_TOO_LARGE: return "request exceeds the fixed capacity of the allocation-free entry point";
        default: return "unknown error";
    }
}

extern "C" const char* bf_last_cuda_error(const bf_ctx* ctx) { return ctx ? ctx->cuda_msg.c_str() : ""; }

// ------------------------------------------------------------------------------------------------
extern "C" int bf_ctx_create(bf_ctx** out, uint32_t N, const uint64_t* primes, uint32_t n_ct_primes, double scale,
                             const bf_plan* plan, void* cuda_stream) {
    if (!out || !primes || !plan) return BF_ERR_INVALID_ARG;
    *out = nullptr;
    if (!is_pow2(N) || N < (1u << 10) || N > (1u << 16)) return BF_ERR_INVALID_ARG;
    if (n_ct_primes < 2 || n_ct_primes + 1 > (u32)MAX_MODULI) return BF_ERR_INVALID_ARG;
    if (!(scale >= 1.0) || !std::isfinite(scale)) return BF_ERR_INVALID_ARG;
    const u32 nb = n_ct_primes + 1;
    for (u32 i = 0; i < nb; ++i) {
        const u64 q = primes[i];
        if (q >= (1ull << 60) || q % (2ull * N) != 1 || !h_is_prime(q)) return BF_ERR_BAD_PRIME;
        for (u32 k = 0; k < i; ++k)
            if (primes[k] == q) return BF_ERR_BAD_PRIME;
    }
    const u32 n = N / 2;
    if (!is_pow2(plan->tile_D) || !is_pow2(plan->tau) || !is_pow2(plan->bsgs_b) || !is_pow2(plan->bsgs_g))
        return BF_ERR_SHAPE;
    if ((u64)plan->tile_D * plan->tau > n || plan->tile_D % plan->tau != 0 ||
        (u64)plan->bsgs_b * plan->bsgs_g != plan->tile_D / plan->tau)
        return BF_ERR_SHAPE;
    if (plan->bsgs_b - 1 > (u32)MAX_ROT_BATCH) return BF_ERR_SHAPE;
    if (plan->flags & ~(u32)(BF_PLAN_COMPLEX_PACK | BF_PLAN_MODDOWN_PER_OUTPUT | BF_PLAN_DOUBLE_HOIST)) return BF_ERR_INVALID_ARG;
    if ((plan->flags & BF_PLAN_MODDOWN_PER_OUTPUT) && plan->bsgs_g - 1 > (u32)MAX_ROT_BATCH) return BF_ERR_SHAPE;

    bf_ctx* ctx = new (std::nothrow) bf_ctx();
    if (!ctx) return BF_ERR_OOM;
    ctx->N = N;
    ctx->logN = 0;
    while ((1u << ctx->logN) < N) ctx->logN++;
    ctx->r = n_ct_primes;
    ctx->scale = scale;
    ctx->plan = *plan;
    ctx->stream = (cudaStream_t)cuda_stream;
    ctx->ring.prof = &ctx->prof;
    int status = BF_OK;
    auto fail = [&](int s) {
        bf_ctx_destroy(ctx);
        return s;
    };
    if (cudaGetDevice(&ctx->device) != cudaSuccess) return fail(BF_ERR_CUDA);
    ctx->ring.device = ctx->device;

    std::vector<double> enc_consts((size_t)MAX_MODULI * ENC_CONSTS, 0.0);
    RingDev& R = ctx->ring.dev;
    memset(&R, 0, sizeof(R));
    R.N = N;
    R.logN = ctx->logN;
    R.r = n_ct_primes;
    ctx->ring.geom = ntt_geometry(ctx->logN);
    ctx->ring.q.assign(primes, primes + nb);
    const u64 P = primes[n_ct_primes];
    std::vector<ulonglong2> twf((size_t)nb * N), twi((size_t)nb * N);
    for (u32 m = 0; m < nb; ++m) {
        const u64 q = primes[m];
        R.q[m] = q;
        R.mu[m] = (u64)((((u128)1) << 64) / q);
        R.c64[m] = (u64)((((u128)1) << 64) % q);
        R.c64s[m] = h_shoup(R.c64[m], q);
        R.ninv[m] = h_invmod(N % q, q);
        R.ninvs[m] = h_shoup(R.ninv[m], q);
        {
            u64 inv = 1;                                   // q^{-1} mod 2^64 by Newton iteration
            for (int it = 0; it < 6; ++it) inv *= 2 - q * inv;
            R.qneg[m] = (u64)0 - inv;
            const u64 two64_inv = h_invmod(R.c64[m], q);
            R.ninv_m[m] = h_mulmod(R.ninv[m], two64_inv, q);
            R.ninv_ms[m] = h_shoup(R.ninv_m[m], q);
        }
        if (m < n_ct_primes) {
            R.pmod[m] = P % q;
            R.pinv[m] = h_invmod(P % q, q);
            R.pinvs[m] = h_shoup(R.pinv[m], q);
        }
        const u64 psi = h_root_2n(q, N);
        if (!psi) return fail(BF_ERR_BAD_PRIME);
        const u64 psi_inv = h_invmod(psi, q);
        std::vector<u64> pw(N), pwi(N);
        pw[0] = 1;
        pwi[0] = 1;
        for (u32 k = 1; k < N; ++k) {
            pw[k] = h_mulmod(pw[k - 1], psi, q);
            pwi[k] = h_mulmod(pwi[k - 1], psi_inv, q);
        }
        R.fp_ok[m] = q < (1ull << 50) ? 1u : 0u;      // below 2^41: lazy fp64 path; up to 2^50: fp64 path in [0, 4q)
        R.qd[m] = (double)q;
        R.qinv_d[m] = 1.0 / (double)q;
        R.ninv_d[m] = (double)R.ninv[m];
        R.ninv_q[m] = (double)R.ninv[m] / (double)q;
        R.ninvm_d[m] = (double)R.ninv_m[m];
        R.ninvm_q[m] = (double)R.ninv_m[m] / (double)q;
        R.c30_d[m] = (double)((1ull << 30) % q);
        R.c30_q[m] = R.c30_d[m] / (double)q;
        R.k59_d[m] = (double)(2 * q - (1ull << 59) % q);
        R.pinv_d[m] = m < n_ct_primes ? (double)R.pinv[m] : 0.0;
        R.pinv_q[m] = m < n_ct_primes ? (double)R.pinv[m] / (double)q : 0.0;
        {   // constants of the encoder's fp64 load (see RingDev::enc_consts)
            const u64 c96 = h_mulmod(R.c64[m], (1ull << 32) % q, q);
            const u64 c127 = h_mulmod(R.c64[m], (1ull << 63) % q, q);
            const u64 neg = c127 ? q - c127 : 0;                         // -2^127 mod q in [0, q)
            double k = neg > q / 2 ? -(double)(q - neg) : (double)neg;    // centred
            if (q >> 41) k += 2.0 * (double)q;
            double* ec = &enc_consts[(size_t)m * ENC_CONSTS];
            ec[0] = (double)c96;
            ec[1] = ec[0] / (double)q;
            ec[2] = (double)R.c64[m];
            ec[3] = ec[2] / (double)q;
            ec[4] = k;
        }
        auto dbits = [](double d) -> u64 {
            u64 bits;
            memcpy(&bits, &d, sizeof(bits));
            return bits;
        };
        // integer path: (w, floor(w * 2^64 / q)); fp64 path: bits of ((double)w, (double)w / q) -- both
        // operands are exact in fp64 and IEEE division rounds correctly
        auto entry = [&](u64 w) -> ulonglong2 {
            if (!R.fp_ok[m]) return make_ulonglong2(w, h_shoup(w, q));
            return make_ulonglong2(dbits((double)w), dbits((double)w / (double)q));
        };
        for (u32 k = 0; k < N; ++k) {
            const u32 e = h_brev(k, (int)ctx->logN);
            twf[(size_t)m * N + k] = entry(pw[e]);
            twi[(size_t)m * N + k] = entry(pwi[e]);
        }
    }
    // encoder tables: twiddles from the host's libm so that results do not depend on the device's
    // own sine and cosine
    const int logn = (int)ctx->logN - 1;
    std::vector<u32> sop(n);
    {
        u64 pw5 = 1;
        for (u32 s = 0; s < n; ++s) {
            const u32 idx = (u32)((pw5 - 1) / 4);
            sop[h_brev(idx, logn)] = s;
            pw5 = (pw5 * 5) % (2ull * N);
        }
    }
    std::vector<double2> T(n / 2), Z(n);
    {
        const double PI = 3.14159265358979323846264338327950288;
        const double two_pi_over_n = (2.0 * PI) / (double)n;
        const double pi_over_N = PI / (double)N;
        for (u32 t = 0; t < n / 2; ++t) {
            const double ang = (double)t * two_pi_over_n;
            T[t] = make_double2(cos(ang), -sin(ang));
        }
        for (u32 k = 0; k < n; ++k) {
            const double ang = (double)k * pi_over_N;
            Z[k] = make_double2(cos(ang), -sin(ang));
        }
    }
#define CKC(call)                                                        \
    do {                                                                 \
        cudaError_t e__ = (call);                                        \
        if (e__ != cudaSuccess) {                                        \
            status = (e__ == cudaErrorMemoryAllocation) ? BF_ERR_OOM : BF_ERR_CUDA; \
            cudaGetLastError();                                          \
            return fail(status);                                         \
        }                                                                \
    } while (0)
    CKC(cudaMalloc(&ctx->tw_fwd, twf.size() * sizeof(ulonglong2)));
    CKC(cudaMalloc(&ctx->tw_inv, twi.size() * sizeof(ulonglong2)));
    CKC(cudaMalloc(&ctx->slot_of_pos, sop.size() * sizeof(u32)));
    CKC(cudaMalloc(&ctx->T, T.size() * sizeof(double2)));
    CKC(cudaMalloc(&ctx->Z, Z.size() * sizeof(double2)));
    CKC(cudaMalloc(&ctx->overflow_flag, 2 * sizeof(int)));
    CKC(cudaMalloc(&ctx->enc_consts, enc_consts.size() * sizeof(double)));
    ctx->device_error = ctx->overflow_flag + 1;
    CKC(cudaMemcpy(ctx->tw_fwd, twf.data(), twf.size() * sizeof(ulonglong2), cudaMemcpyHostToDevice));
    CKC(cudaMemcpy(ctx->tw_inv, twi.data(), twi.size() * sizeof(ulonglong2), cudaMemcpyHostToDevice));
    CKC(cudaMemcpy(ctx->slot_of_pos, sop.data(), sop.size() * sizeof(u32), cudaMemcpyHostToDevice));
    CKC(cudaMemcpy(ctx->T, T.data(), T.size() * sizeof(double2), cudaMemcpyHostToDevice));
    CKC(cudaMemcpy(ctx->Z, Z.data(), Z.size() * sizeof(double2), cudaMemcpyHostToDevice));
    CKC(cudaMemcpy(ctx->enc_consts, enc_consts.data(), enc_consts.size() * sizeof(double), cudaMemcpyHostToDevice));
    CKC(cudaMemset(ctx->overflow_flag, 0, 2 * sizeof(int)));
    CKC(cudaDeviceSynchronize());
#undef CKC
    R.tw_fwd = ctx->tw_fwd;
    R.tw_inv = ctx->tw_inv;
    R.enc_consts = ctx->enc_consts;
    *out = ctx;
    return BF_OK;
}

static void free_buf(DevBuf& b) {
    if (b.p) cudaFree(b.p);
    b.p = nullptr;
    b.cap = 0;
}

static void destroy_graphs(bf_ctx* ctx);

extern "C" void bf_ctx_destroy(bf_ctx* ctx) {
    if (!ctx) return;
    cudaDeviceSynchronize();
    destroy_graphs(ctx);
    for (bf_weights* w : ctx->weights) {
        if (w) {
            cudaFree(w->pt);
            cudaFree(w->coef);
            delete w;
        }
    }
    DevBuf* bufs[] = {&ctx->X, &ctx->X0, &ctx->Aext, &ctx->Dig, &ctx->U, &ctx->Ubig, &ctx->Tc, &ctx->Tn, &ctx->Cc, &ctx->A, &ctx->Rres, &ctx->Lfull,
                      &ctx->fft, &ctx->coef, &ctx->ptnat, &ctx->ptjit, &ctx->stage_in, &ctx->stage_out, &ctx->nm_a, &ctx->nm_b};
    for (DevBuf* b : bufs) free_buf(*b);
    cudaFree(ctx->tw_fwd);
    cudaFree(ctx->tw_inv);
    cudaFree(ctx->slot_of_pos);
    cudaFree(ctx->T);
    cudaFree(ctx->Z);
    cudaFree(ctx->enc_consts);
    for (cudaStream_t& s : ctx->side)
        if (s) { cudaStreamDestroy(s); s = nullptr; }
    for (cudaEvent_t& e : ctx->ev_join)
        if (e) { cudaEventDestroy(e); e = nullptr; }
    if (ctx->ev_fork) { cudaEventDestroy(ctx->ev_fork); ctx->ev_fork = nullptr; }
    cudaFree(ctx->overflow_flag);
    cudaFree(ctx->keys);
    cudaFree(ctx->perms);
    cudaFree(ctx->perms_fwd);
    for (cudaEvent_t& e : ctx->ev)
        if (e) cudaEventDestroy(e);
    for (auto& rec : ctx->prof.recs) { cudaEventDestroy(rec.a); cudaEventDestroy(rec.b); }
    for (cudaEvent_t e : ctx->prof.pool) cudaEventDestroy(e);
    cudaGetLastError();
    delete ctx;
}

// ------------------------------------------------------------------------------------------------
// Drops the resident keys and everything that refers to them: the step -> key map, the permutation tables and
// the captured launch sequences (they hold the addresses of the freed arrays).
static void drop_eval_keys(bf_ctx* ctx) {
    destroy_graphs(ctx);
    ctx->epoch++;
    cudaFree(ctx->keys);
    cudaFree(ctx->perms);
    cudaFree(ctx->perms_fwd);
    ctx->keys = nullptr;
    ctx->perms = nullptr;
    ctx->perms_fwd = nullptr;
    ctx->key_of_steps.clear();
    ctx->n_keys = 0;
}

extern "C" int bf_load_eval_keys(bf_ctx* ctx, const uint32_t* rot_steps, uint32_t n_keys, const uint64_t* keys) {
    if (!ctx || (n_keys && (!rot_steps || !keys))) return BF_ERR_INVALID_ARG;
    const u32 N = ctx->N, r = ctx->r, nb = r + 1, n = N / 2;
    CK(cudaStreamSynchronize(ctx->stream));
    drop_eval_keys(ctx);
    if (n_keys == 0) return BF_OK;
    // every failure below leaves the context without keys (BF_ERR_MISSING_KEY on the next rotation), never
    // with a half-built set
    auto fail = [&](int code) {
        cudaGetLastError();
        drop_eval_keys(ctx);
        return code;
    };
    const size_t key_words = (size_t)r * 2 * nb * N;
    if (cudaMalloc(&ctx->keys, key_words * n_keys * sizeof(u64)) != cudaSuccess) { ctx->keys = nullptr; return fail(BF_ERR_OOM); }
    if (cudaMalloc(&ctx->perms, (size_t)n_keys * N * sizeof(u32)) != cudaSuccess) { ctx->perms = nullptr; return fail(BF_ERR_OOM); }
    // permutation tables: position i of the transform holds the evaluation at psi^(2*brev(i)+1);
    // a(X) -> a(X^g) maps it to the evaluation at exponent (2*brev(i)+1)*g mod 2N, so the rotated
    // polynomial is out[i] = in[perm[i]].  The keys are stored as key'[perm[i]] = key[i], which lets
    // the inner product run in the un-rotated index space; the rotation is applied at the very end
    // as the scatter out[pinv[i]] = v'[i], pinv = perm^{-1}.  Only pinv stays on the device.
    std::vector<u32> perms((size_t)n_keys * N), pinvs((size_t)n_keys * N);
    std::map<u32, int> key_of_steps;
    for (u32 t = 0; t < n_keys; ++t) {
        const u32 steps = rot_steps[t] % n;
        u64 g = 1;
        for (u32 s = 0; s < steps; ++s) g = (g * 5) % (2ull * N);
        for (u32 i = 0; i < N; ++i) {
            const u64 ex = ((2ull * h_brev(i, (int)ctx->logN) + 1) * g) % (2ull * N);
            const u32 pi = h_brev((u32)((ex - 1) / 2), (int)ctx->logN);
            perms[(size_t)t * N + i] = pi;
            pinvs[(size_t)t * N + pi] = i;
        }
        key_of_steps[steps] = (int)t;
    }
    u32* perm_dev = nullptr;
    if (cudaMalloc(&perm_dev, perms.size() * sizeof(u32)) != cudaSuccess) return fail(BF_ERR_OOM);
    if (cudaMemcpy(perm_dev, perms.data(), perms.size() * sizeof(u32), cudaMemcpyHostToDevice) != cudaSuccess ||
        cudaMemcpy(ctx->perms, pinvs.data(), pinvs.size() * sizeof(u32), cudaMemcpyHostToDevice) != cudaSuccess) {
        ctx->cuda_msg = "cudaMemcpy of the permutation tables failed";
        cudaFree(perm_dev);
        return fail(BF_ERR_CUDA);
    }
    PolyBatch B;
    memset(&B, 0, sizeof(B));
    B.src = keys;
    B.src_so = B.dst_so = (long long)nb * N;
    B.src_sm = B.dst_sm = N;
    B.n_m = nb;
    B.mod0 = 0;
    B.mod_step = 1;
    // The first pass of the transform lands in a staging buffer in natural order; the second pass
    // reads it and stores, permuted, into the resident key array (a permuted store in place would
    // overwrite points other blocks have not read yet).
    u64* stage = nullptr;
    if (cudaMalloc(&stage, key_words * n_keys * sizeof(u64)) != cudaSuccess) { cudaFree(perm_dev); return fail(BF_ERR_OOM); }
    B.dst = stage;
    B.scatter = nullptr;
    cudaError_t ne = ntt_forward_split(ctx->ring, B, n_keys * r * 2, LOAD_REDUCE, ctx->keys, perm_dev, 2 * r, ctx->stream);
    cudaError_t se = cudaStreamSynchronize(ctx->stream);
    cudaFree(stage);
    if (ne != cudaSuccess || se != cudaSuccess) {
        cudaFree(perm_dev);
        ctx->cuda_msg = std::string("key transform: ") + cudaGetErrorString(ne != cudaSuccess ? ne : se);
        return fail(BF_ERR_CUDA);
    }
    ctx->perms_fwd = perm_dev;
    ctx->key_of_steps.swap(key_of_steps);
    ctx->n_keys = n_keys;
    ctx->epoch++;
    return BF_OK;
}

extern "C" int bf_set_cache_budget(bf_ctx* ctx, uint64_t bytes) {
    if (!ctx) return BF_ERR_INVALID_ARG;
    ctx->cache_budget = bytes;
    return BF_OK;
}

extern "C" uint64_t bf_cache_bytes_used(const bf_ctx* ctx) { return ctx ? ctx->cache_used : 0; }

static u32 cdiv(u32 a, u32 b) { return (u32)(((u64)a + b - 1) / b); }

// primes the encoded plaintexts are held in: with double hoisting the special prime as well
static u32 mac_primes(const bf_ctx* ctx) { return ctx->r + ((ctx->plan.flags & BF_PLAN_DOUBLE_HOIST) ? 1u : 0u); }

// output ciphertexts of a projection with d_out rows: one per row block of tile_D, or per pair of row blocks
static u32 n_out_cts(const bf_ctx* ctx, u32 d_out) {
    const u32 blocks = cdiv(d_out, ctx->plan.tile_D);
    return (ctx->plan.flags & BF_PLAN_COMPLEX_PACK) ? cdiv(blocks, 2) : blocks;
}

static u64 weights_bytes(const bf_ctx* ctx, u32 d_out, u32 d_in, u32 b, u32 g) {
    const u32 n_in = cdiv(d_in, ctx->plan.tile_D), n_out = n_out_cts(ctx, d_out);
    if (ctx->coef_cache_bits)       // one rounded coefficient per diagonal and ring position, whatever the primes
        return (u64)n_in * n_out * (ctx->plan.tile_D / ctx->plan.tau) * ctx->N * (ctx->coef_cache_bits / 8);
    const TileLayout lay = mac_tile_layout(ctx->ring, n_out * g, n_in * b, mac_primes(ctx));
    return mac_tile_bytes(ctx->ring, lay);
}

extern "C" uint64_t bf_weights_bytes(const bf_ctx* ctx, uint32_t d_out, uint32_t d_in) {
    if (!ctx) return 0;
    return weights_bytes(ctx, d_out, d_in, ctx->plan.bsgs_b, ctx->plan.bsgs_g);
}

// a baby/giant split the context's plan admits
static bool split_ok(const bf_ctx* ctx, u32 b, u32 g) {
    if (!b || !g || (b & (b - 1)) || (g & (g - 1))) return false;
    if ((u64)b * g != ctx->plan.tile_D / ctx->plan.tau || b - 1 > (u32)MAX_ROT_BATCH) return false;
    return !((ctx->plan.flags & BF_PLAN_MODDOWN_PER_OUTPUT) && g - 1 > (u32)MAX_ROT_BATCH);
}

// Encode diagonals [d0, d0 + count) of W (order [j][p][q][k], i.e. group pj = d / n_terms, term d % n_terms)
// into dst in the tile-major layout `lay`, whose group 0 is group pj0 of W.
// The coefficients come from the encoder (W), or from a handle that keeps them (stored; W is then unused); coef_out
// non-null: only encode, leaving the 64-bit coefficients of diagonal d0 + i at coef_out + i*N (no transform).
static int encode_range(bf_ctx* ctx, const float* W, u32 d_out, u32 d_in, u32 d0, u32 count, u64* dst,
                        const TileLayout& lay, u32 pj0, const bf_weights* stored = nullptr, i64* coef_out = nullptr,
                        u32 split_b = 0, u32 split_g = 0) {
    const u32 N = ctx->N, r = lay.n_primes, n = N / 2;       // (r: primes each diagonal is reduced into)
    // diagonals per pass: the encoder and the transforms gain from large batches (measured: 32 -> 128 per
    // pass takes 6 to 8 % off a call that encodes on the fly); the scratch of a pass is held to about 0.5 GB
    u32 chunk = (u32)(((size_t)512 << 20) / ((size_t)r * N * sizeof(u64))) & ~7u;
    if (chunk > 256) chunk = 256;
    if (chunk < 32) chunk = 32;
    if (chunk > count) chunk = count > 0 ? count : 1;
    if (!stored) TRY(ensure(ctx, ctx->fft, (size_t)chunk * n * sizeof(double2)));
    if (!coef_out && !(stored && stored->coef_bits == 64)) TRY(ensure(ctx, ctx->coef, (size_t)chunk * N * sizeof(i64)));
    if (!coef_out) TRY(ensure(ctx, ctx->ptnat, (size_t)chunk * r * N * sizeof(u64)));
    EncodeTables tab;
    tab.slot_of_pos = ctx->slot_of_pos;
    tab.T = ctx->T;
    tab.Z = ctx->Z;
    tab.scale_over_n = ctx->scale / (double)n;
    for (u32 lo = 0; lo < count; lo += chunk) {
        const u32 cnt = (count - lo < chunk) ? count - lo : chunk;
        DiagBatch db;
        db.W = W;
        db.d_out = d_out;
        db.d_in = d_in;
        db.n_in = cdiv(d_in, ctx->plan.tile_D);
        db.n_out = n_out_cts(ctx, d_out);
        db.complex_pack = (ctx->plan.flags & BF_PLAN_COMPLEX_PACK) ? 1u : 0u;
        db.D = ctx->plan.tile_D;
        db.tau = ctx->plan.tau;
        db.b = split_b ? split_b : stored ? stored->b : ctx->plan.bsgs_b;
        db.g = split_g ? split_g : stored ? stored->g : ctx->plan.bsgs_g;
        db.d0 = d0 + lo;
        db.count = cnt;
        const void* coef_src = ctx->coef.p;
        if (stored && stored->coef_bits == 64) {
            coef_src = (const i64*)stored->coef + (size_t)(d0 + lo) * N;
        } else if (stored) {
            CK(launch_widen_i32(ctx->ring, (const int*)stored->coef + (size_t)(d0 + lo) * N, (i64*)ctx->coef.p, (size_t)cnt * N,
                                ctx->stream));
        } else {
            i64* into = coef_out ? coef_out + (size_t)lo * N : (i64*)ctx->coef.p;
            CK(launch_encode(ctx->ring, tab, db, (double2*)ctx->fft.p, into, ctx->overflow_flag, ctx->stream));
            if (coef_out) continue;
        }
        PolyBatch B;
        memset(&B, 0, sizeof(B));
        B.src = coef_src;
        B.dst = (u64*)ctx->ptnat.p;                 // first pass lands here; the second writes the tiles
        B.src_so = N;
        B.src_sm = 0;
        B.dst_so = (long long)r * N;
        B.dst_sm = N;
        B.n_m = r;
        B.mod0 = 0;
        B.mod_step = 1;
        B.split_bits = mac_split_bits(ctx->ring);
        B.tile_ptr = dst;
        B.tile = lay;
        B.tile_pj0 = pj0;
        B.o_base = d0 + lo;
        CK(ntt_forward(ctx->ring, B, cnt, LOAD_I64_MONT, ctx->stream));   // cached form: NTT domain, times 2^64
    }
    return BF_OK;
}

// Reads the two device-side flags (encoder range overflow; a bounded wait that gave up).  Synchronises.
static int check_overflow(bf_ctx* ctx) {
    int flags[2] = {0, 0};
    CK(cudaMemcpyAsync(flags, ctx->overflow_flag, 2 * sizeof(int), cudaMemcpyDeviceToHost, ctx->stream));
    CK(cudaStreamSynchronize(ctx->stream));
    if (flags[0] || flags[1]) {
        CK(cudaMemsetAsync(ctx->overflow_flag, 0, 2 * sizeof(int), ctx->stream));
        return flags[1] ? BF_ERR_TIMEOUT : BF_ERR_RANGE;
    }
    return BF_OK;
}

extern "C" int bf_device_status(bf_ctx* ctx) {
    if (!ctx) return BF_ERR_INVALID_ARG;
    return check_overflow(ctx);
}

extern "C" int bf_encode_weights(bf_ctx* ctx, const float* W, uint32_t d_out, uint32_t d_in, bf_weights** out) {
    if (!ctx) return BF_ERR_INVALID_ARG;
    return bf_encode_weights_split(ctx, W, d_out, d_in, ctx->plan.bsgs_b, ctx->plan.bsgs_g, out);
}

extern "C" int bf_encode_weights_split(bf_ctx* ctx, const float* W, uint32_t d_out, uint32_t d_in, uint32_t bsgs_b,
                                       uint32_t bsgs_g, bf_weights** out) {
    if (!ctx || !W || !out || !d_out || !d_in) return BF_ERR_INVALID_ARG;
    *out = nullptr;
    if (!split_ok(ctx, bsgs_b, bsgs_g)) return BF_ERR_SHAPE;
    const u64 bytes = weights_bytes(ctx, d_out, d_in, bsgs_b, bsgs_g);
    if (ctx->cache_budget && ctx->cache_used + bytes > ctx->cache_budget) return BF_ERR_OOM;
    bf_weights* w = new (std::nothrow) bf_weights();
    if (!w) return BF_ERR_OOM;
    w->d_out = d_out;
    w->d_in = d_in;
    w->n_in = cdiv(d_in, ctx->plan.tile_D);
    w->n_out = n_out_cts(ctx, d_out);
    w->bytes = bytes;
    w->b = bsgs_b;
    w->g = bsgs_g;
    w->lay = mac_tile_layout(ctx->ring, w->n_out * bsgs_g, w->n_in * bsgs_b, mac_primes(ctx));
    const u32 n_diag = w->n_in * w->n_out * (ctx->plan.tile_D / ctx->plan.tau);
    int s = BF_OK;
    if (ctx->coef_cache_bits) {
        // coefficient form: run the encoder only; 32-bit storage goes through a 64-bit staging area in pieces and
        // is refused (BF_ERR_RANGE) when a coefficient does not fit
        w->coef_bits = ctx->coef_cache_bits;
        w->pt = nullptr;
        if (cudaMalloc(&w->coef, bytes) != cudaSuccess) {
            cudaGetLastError();
            delete w;
            return BF_ERR_OOM;
        }
        if (w->coef_bits == 64) {
            s = encode_range(ctx, W, d_out, d_in, 0, n_diag, nullptr, w->lay, 0, nullptr, (i64*)w->coef, bsgs_b, bsgs_g);
        } else {
            const u32 piece = 256;
            s = ensure(ctx, ctx->coef, (size_t)piece * ctx->N * sizeof(i64));
            for (u32 d0 = 0; d0 < n_diag && s == BF_OK; d0 += piece) {
                const u32 cnt = n_diag - d0 < piece ? n_diag - d0 : piece;
                s = encode_range(ctx, W, d_out, d_in, d0, cnt, nullptr, w->lay, 0, nullptr, (i64*)ctx->coef.p, bsgs_b, bsgs_g);
                if (s == BF_OK && launch_narrow_i64(ctx->ring, (const i64*)ctx->coef.p, (int*)w->coef + (size_t)d0 * ctx->N,
                                                    (size_t)cnt * ctx->N, ctx->overflow_flag, ctx->stream) != cudaSuccess)
                    s = BF_ERR_CUDA;
            }
        }
    } else {
        if (cudaMalloc(&w->pt, bytes) != cudaSuccess) {
            cudaGetLastError();
            delete w;
            return BF_ERR_OOM;
        }
        // padding words of the layout are never read, but keep the allocation defined
        if (cudaMemsetAsync(w->pt, 0, bytes, ctx->stream) != cudaSuccess) s = BF_ERR_CUDA;
        if (s == BF_OK) s = encode_range(ctx, W, d_out, d_in, 0, n_diag, w->pt, w->lay, 0, nullptr, nullptr, bsgs_b, bsgs_g);
    }
    if (s == BF_OK) s = check_overflow(ctx);
    if (s != BF_OK) {
        cudaStreamSynchronize(ctx->stream);
        cudaFree(w->pt);
        cudaFree(w->coef);
        cudaGetLastError();
        delete w;
        return s;
    }
    ctx->cache_used += bytes;
    ctx->weights.push_back(w);
    *out = w;
    return BF_OK;
}

extern "C" void bf_weights_free(bf_ctx* ctx, bf_weights* w) {
    if (!ctx || !w) return;
    for (size_t i = 0; i < ctx->weights.size(); ++i) {
        if (ctx->weights[i] == w) {
            cudaStreamSynchronize(ctx->stream);
            cudaFree(w->pt);
            cudaFree(w->coef);
            ctx->cache_used -= w->bytes;
            ctx->epoch++;
            delete w;
            ctx->weights.erase(ctx->weights.begin() + i);
            return;
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Division by the special prime and assembly of rotated ciphertexts for the rotations listed in rb
// (their inner products already sit in U): inverse transform of the P-residues, centred lift into
// every q_i with a forward transform whose last store computes (u - t) * P^{-1} + c0 and scatters
// it through the rotation's permutation.
struct Lane {
    cudaStream_t s;
    u64 *Dig, *U, *Tc, *Tn, *Cc;     // this lane's share of the key-switch scratch
};

static Lane main_lane(bf_ctx* ctx) {
    return Lane{ctx->stream, (u64*)ctx->Dig.p, (u64*)ctx->U.p, (u64*)ctx->Tc.p, (u64*)ctx->Tn.p, (u64*)ctx->Cc.p};
}

static int ensure_lanes(bf_ctx* ctx) {
    if (!ctx->ev_fork) CK(cudaEventCreateWithFlags(&ctx->ev_fork, cudaEventDisableTiming));
    const int n_side = ctx->n_lanes > 2 ? ctx->n_lanes - 1 : 1;       // (one side stream at least: the special prime's MAC)
    for (int i = 0; i < n_side && i + 1 < bf_ctx::MAX_LANES; ++i) {
        if (!ctx->side[i]) CK(cudaStreamCreateWithFlags(&ctx->side[i], cudaStreamNonBlocking));
        if (!ctx->ev_join[i]) CK(cudaEventCreateWithFlags(&ctx->ev_join[i], cudaEventDisableTiming));
    }
    return BF_OK;
}

// side streams wait for everything enqueued on the context's stream so far
static int fork_lanes(bf_ctx* ctx, int used) {
    if (used <= 1) return BF_OK;
    CK(cudaEventRecord(ctx->ev_fork, ctx->stream));
    for (int i = 0; i + 1 < used; ++i) CK(cudaStreamWaitEvent(ctx->side[i], ctx->ev_fork, 0));
    return BF_OK;
}

// the context's stream waits for everything enqueued on the side streams
static int join_lanes(bf_ctx* ctx, int used) {
    for (int i = 0; i + 1 < used; ++i) {
        CK(cudaEventRecord(ctx->ev_join[i], ctx->side[i]));
        CK(cudaStreamWaitEvent(ctx->stream, ctx->ev_join[i], 0));
    }
    return BF_OK;
}

static int moddown_batch(bf_ctx* ctx, const Lane& lane, const RotBatch& rb, const u64* c0_base, long long c0_stride,
                         u64* out_base, long long out_stride) {
    const u32 N = ctx->N, r = ctx->r, nb = r + 1;
    PolyBatch B;
    memset(&B, 0, sizeof(B));
    B.src = (const u64*)lane.U + (size_t)r * N;       // the P-residue of each (rotation, component)
    B.dst = lane.Tc;
    B.src_so = (long long)nb * N;
    B.dst_so = N;
    B.n_m = 1;
    B.mod0 = r;
    B.mod_step = 0;
    B.store_centred = 1;                                // the form the lift below reads
    CK(ntt_inverse(ctx->ring, B, (u32)rb.n * 2, lane.s));
    memset(&B, 0, sizeof(B));
    B.src = lane.Tc;
    B.dst = lane.Tn;                            // staging between the two passes of the transform
    B.src_so = N;
    B.src_sm = 0;
    B.dst_so = (long long)r * N;
    B.dst_sm = N;
    B.n_m = r;
    B.mod0 = 0;
    B.mod_step = 1;
    B.lift_mod = ctx->ring.q[r];
    ModDownEpilogue epi;
    memset(&epi, 0, sizeof(epi));
    epi.u = (const u64*)lane.U;
    epi.c0_base = c0_base;
    epi.c0_stride = c0_stride;
    epi.pinv = ctx->perms;
    epi.out_base = out_base;
    epi.out_stride = out_stride;
    CK(ntt_forward_moddown(ctx->ring, B, (u32)rb.n * 2, rb, epi, lane.s));
    return BF_OK;
}

static int ensure_rot_scratch(bf_ctx* ctx, u32 n_dig_sets, u32 n_rot) {
    const size_t N = ctx->N, r = ctx->r, nb = r + 1;
    // digit sets, tile-major for the inner product, and behind them a staging area of the same size for the
    // intermediate of their transforms (natural order)
    TRY(ensure(ctx, ctx->Dig, (size_t)2 * n_dig_sets * r * nb * N * 8));
    ctx->dig_half = ctx->Dig.cap / 16;
    TRY(ensure(ctx, ctx->U, (size_t)n_rot * 2 * nb * N * 8));
    TRY(ensure(ctx, ctx->Tc, (size_t)n_rot * 2 * N * 8));
    TRY(ensure(ctx, ctx->Tn, (size_t)n_rot * 2 * r * N * 8));
    return BF_OK;
}

static int find_key(bf_ctx* ctx, u32 steps, int* key) {
    auto it = ctx->key_of_steps.find(steps % (ctx->N / 2));
    if (it == ctx->key_of_steps.end()) return BF_ERR_MISSING_KEY;
    *key = it->second;
    return BF_OK;
}

// Digits of c1 (coefficient domain; set s at c1_coeff + s*set_stride, [r][N]) reduced into every prime
// of the extended basis and transformed: dig[set][j][m] = NTT_m( c1_j mod m ).  The digit in its own
// prime is the transform of c1 itself, which the caller already has (c1_ntt + s*c1_ntt_stride, [r][N]):
// it is copied, not recomputed.
// div_t non-null: c1_coeff holds residues of polynomials of the extended basis and div_t + s*set_stride their
// residues modulo P (centred): the digits are those of the polynomial divided by P (then c1_ntt is not used: no
// transform of the quotient exists yet).
static int modup(bf_ctx* ctx, cudaStream_t stream, const u64* c1_coeff, long long set_stride, u32 n_sets, u64* dig,
                 const u64* c1_ntt, long long c1_ntt_stride, const u64* div_t = nullptr) {
    const u32 N = ctx->N, r = ctx->r, nb = r + 1;
    PolyBatch B;
    memset(&B, 0, sizeof(B));
    B.n_m = nb;
    B.mod0 = 0;
    B.mod_step = 1;
    B.src = c1_coeff;
    B.o_div = r;                 // o = set*r + digit
    B.src_so2 = set_stride;
    B.src_so = N;
    B.src_sm = 0;
    B.dst = dig + ctx->dig_half;         // staging between the two passes; the result goes to dig, tile-major
    B.dtile_ptr = dig;
    B.dtile_div = r;
    B.dst_so = (long long)nb * N;
    B.dst_sm = N;
    B.skip_diag = div_t ? 0 : 1;
    B.src_digits = 1;
    B.diag_src = c1_ntt;
    B.diag_so = c1_ntt_stride;
    B.div_t = div_t;
    B.div_so = set_stride;
    CK(ntt_forward(ctx->ring, B, n_sets * r, LOAD_REDUCE, stream));
    return BF_OK;
}

static void stamp(bf_ctx* ctx, int i) {
    if (ctx->timing && ctx->ev[i]) cudaEventRecord(ctx->ev[i], ctx->stream);
}

static u32 giant_batch(const bf_ctx* ctx) {
    // rotations per key-switch launch
    const size_t per_rot = (size_t)ctx->r * (ctx->r + 1) * ctx->N * 8;
    // Measured: fewer, larger launches beat keeping a batch's digits L2-resident.  Cap the digit
    // buffer at 1 GiB.
    size_t nrot = ((size_t)1 << 30) / per_rot;
    if (nrot < 1) nrot = 1;
    if (nrot > (size_t)MAX_ROT_BATCH) nrot = MAX_ROT_BATCH;
    return (u32)nrot;
}

static void rescale_consts(const bf_ctx* ctx, u32 level, RescaleConsts& rc) {
    memset(&rc, 0, sizeof(rc));
    const u64 qL = ctx->ring.q[level - 1];
    for (u32 i = 0; i + 1 < level; ++i) {
        const u64 q = ctx->ring.q[i];
        rc.inv[i] = h_invmod(qL % q, q);
        rc.invs[i] = h_shoup(rc.inv[i], q);
        rc.qlmod[i] = qL % q;
        rc.inv_d[i] = (double)rc.inv[i];
        rc.inv_q[i] = (double)rc.inv[i] / (double)q;
        rc.qlmod_d[i] = (double)rc.qlmod[i];
    }
}

// ct_low non-null: the result is rescaled on the way ([n_out][2][r-1][N] at ct_low; ct_out is not used): fused into the
// last kernel where the plan ends in an element-wise kernel, else as the rescale kernel behind the call.
static int linear_enqueue(bf_ctx* ctx, const uint64_t* ct_in, uint32_t n_in, const bf_weights* pt_weights,
                          const float* W_raw, uint32_t d_out, uint32_t d_in, uint64_t* ct_out, uint32_t n_out,
                          uint64_t* ct_low = nullptr) {
    if (!ctx || !ct_in || (!ct_out && !ct_low) || (!pt_weights && !W_raw) || !d_out || !d_in) return BF_ERR_INVALID_ARG;
    const u32 N = ctx->N, r = ctx->r, nb = r + 1;
    const u32 D = ctx->plan.tile_D, tau = ctx->plan.tau;
    const u32 b = pt_weights ? pt_weights->b : ctx->plan.bsgs_b, g = pt_weights ? pt_weights->g : ctx->plan.bsgs_g;
    if (n_in != cdiv(d_in, D) || n_out != n_out_cts(ctx, d_out)) return BF_ERR_SHAPE;
    if (pt_weights && (pt_weights->d_out != d_out || pt_weights->d_in != d_in)) return BF_ERR_SHAPE;
    const size_t ctw = (size_t)2 * r * N;                 // words per ciphertext
    // rotation keys the plan needs
    std::vector<int> baby_key(b, -1), giant_key(g, -1);
    for (u32 k = 1; k < b; ++k) TRY(find_key(ctx, k * tau, &baby_key[k]));
    for (u32 j = 1; j < g; ++j) TRY(find_key(ctx, j * b * tau, &giant_key[j]));

    const u32 gb = giant_batch(ctx);
    const u32 n_giant = (g - 1) * n_out;
    // input ciphertexts whose baby steps share one hoisted ModUp
    u32 in_batch = b > 1 ? (u32)MAX_ROT_BATCH / (b - 1) : n_in;
    if (in_batch > gb) in_batch = gb;
    if (in_batch > n_in) in_batch = n_in;
    if (in_batch < 1) in_batch = 1;
    // lanes: the rotations of a stage are dealt out to up to n_lanes independent chains
    int lanes = ctx->n_lanes < 1 ? 1 : (ctx->n_lanes > bf_ctx::MAX_LANES ? bf_ctx::MAX_LANES : ctx->n_lanes);
    TRY(ensure_lanes(ctx));
    // per stage: splitting pays when a stage's kernels are too small to fill the GPU by themselves and there is
    // enough to split (measured side by side per layer shape at N = 2^15: with 3 giant rotations, or with 30 and
    // more baby rotations, the stage runs 1 to 2 % faster as one chain; 9 to 18 giant rotations and 15 baby
    // rotations run 1.5 to 3 % faster as two; more than 18 giant rotations were not measured and stay one chain)
    // (rotation counts weighted by the ring size relative to 2^15: at N = 2^16 a LLaMA-3-8B layer ran 0.8 % faster
    // with its 12 giant rotations per call as one chain)
    const u32 ring_weight = N > (1u << 15) ? N >> 15 : 1u;
    const int lanes_giant = (lanes > 1 && n_giant >= 6 && n_giant * ring_weight <= 20) ? lanes : 1;
    const int lanes_baby = (lanes > 1 && in_batch * (b - 1) * ring_weight <= 24) ? lanes : 1;
    const u32 baby_per_lane = b > 1 ? cdiv(b - 1, (u32)lanes) * in_batch : 1u;     // (a lane takes whole keys)
    u32 giant_per_lane = cdiv(n_giant > 0 ? n_giant : 1, (u32)lanes);     // rotations a lane holds at once
    // (rounded down: a single chain uses the buffers of all lanes, giant_per_lane * lanes rotations per launch,
    // and a launch takes at most MAX_ROT_BATCH)
    if (giant_per_lane > gb / (u32)lanes) giant_per_lane = gb / (u32)lanes;
    if (giant_per_lane < 1) giant_per_lane = 1;
    const u32 rot_per_lane = baby_per_lane > giant_per_lane ? baby_per_lane : giant_per_lane;
    u32 n_dig_sets = giant_per_lane * (u32)lanes;       // digit sets alive at once
    if (n_dig_sets < in_batch) n_dig_sets = in_batch;
    // double hoisting: the rotated inputs and the inner sums live in the extended basis {q_i, P}
    const bool dh = (ctx->plan.flags & BF_PLAN_DOUBLE_HOIST) != 0;
    const u32 nmp = mac_primes(ctx);                      // primes of X, of the plaintexts and of the inner sums
    const size_t xw = (size_t)2 * nmp * N;                // words per term of X / per inner sum
    TRY(ensure(ctx, ctx->X, (size_t)n_in * b * xw * 8));
    if (dh) {
        TRY(ensure(ctx, ctx->X0, (size_t)n_in * ctw * 8));
        TRY(ensure(ctx, ctx->Aext, (size_t)n_out * g * xw * 8));
    }
    TRY(ensure(ctx, ctx->A, (size_t)n_out * g * ctw * 8));
    if (ct_low) {                   // the full-level result is an intermediate
        TRY(ensure(ctx, ctx->Lfull, (size_t)n_out * ctw * 8));
        ct_out = (u64*)ctx->Lfull.p;
    }
    RescaleConsts rcs;
    if (ct_low) rescale_consts(ctx, r, rcs);
    // one division by P per output: the inner products of all giant rotations stay alive until every chain is done
    const bool per_output = (ctx->plan.flags & BF_PLAN_MODDOWN_PER_OUTPUT) && n_giant > 0;
    TRY(ensure(ctx, ctx->Rres, (size_t)(per_output ? n_out : n_giant ? n_giant : 1) * ctw * 8));
    // double hoisting with one division per output: the giant steps' inputs are never divided in the transform domain
    // (see below); their coefficient forms keep the residue modulo P
    const bool assemble = dh && per_output;
    const u32 cc_primes = assemble ? nb : r;
    TRY(ensure(ctx, ctx->Cc, (size_t)n_dig_sets * cc_primes * N * 8));
    {
        u32 rot_scratch = rot_per_lane * (u32)lanes;
        if (per_output && rot_scratch < n_out) rot_scratch = n_out;     // Tc, Tn of the per-output division
        if (dh && rot_scratch < n_out * g) rot_scratch = n_out * g;     // Tc, Tn of the division of the inner sums
        if (assemble && rot_scratch * 2 < n_out * (g + 3)) rot_scratch = cdiv(n_out * (g + 3), 2u);   // Tc of the output assembly
        TRY(ensure_rot_scratch(ctx, n_dig_sets, rot_scratch));
    }
    if (per_output) TRY(ensure(ctx, ctx->Ubig, (size_t)n_giant * 2 * nb * N * 8));
    Lane lane[bf_ctx::MAX_LANES];
    for (int c = 0; c < lanes; ++c) {
        lane[c].s = c == 0 ? ctx->stream : ctx->side[c - 1];
        lane[c].Dig = (u64*)ctx->Dig.p + (size_t)c * giant_per_lane * r * nb * N;
        lane[c].U = (u64*)ctx->U.p + (size_t)c * rot_per_lane * 2 * nb * N;
        lane[c].Tc = (u64*)ctx->Tc.p + (size_t)c * rot_per_lane * 2 * N;
        lane[c].Tn = (u64*)ctx->Tn.p + (size_t)c * rot_per_lane * 2 * r * N;
        lane[c].Cc = (u64*)ctx->Cc.p + (size_t)c * giant_per_lane * cc_primes * N;
    }
    u64* X = (u64*)ctx->X.p;
    u64* A = (u64*)ctx->A.p;
    u64* Rres = (u64*)ctx->Rres.p;
    u64* Dig = (u64*)ctx->Dig.p;
    if (ctx->timing) {
        for (cudaEvent_t& e : ctx->ev)
            if (!e) CK(cudaEventCreate(&e));
        ctx->ev_valid = true;
    }
    stamp(ctx, 0);

    // ---- ingest, hoisted ModUp and baby steps, batched over the input ciphertexts
    PolyBatch B;
    memset(&B, 0, sizeof(B));
    // X[q][0] = NTT(ct_q): polynomial (q, component*r + prime).  Double hoisting keeps it apart (X0: the hoisted ModUp
    // copies its c1 part) and puts P * NTT(ct_q), zero modulo P, into X
    u64* X0 = dh ? (u64*)ctx->X0.p : X;
    const long long x0_stride = dh ? (long long)ctw : (long long)b * ctw;
    B.src = ct_in;
    B.dst = X0;
    B.src_so = (long long)ctw;
    B.dst_so = x0_stride;
    B.src_sm = B.dst_sm = N;
    B.n_m = 2 * r;
    B.mod_wrap = r;
    B.mod0 = 0;
    B.mod_step = 1;
    if (dh) {                   // the transform's last store also writes P * NTT(ct_q) as term q*b of X
        B.lift_ptr = X;
        B.lift_so = (long long)b * (long long)xw;
    }
    CK(ntt_forward(ctx->ring, B, n_in, LOAD_PLAIN, ctx->stream));
    if (b > 1) {
        for (u32 q0 = 0; q0 < n_in; q0 += in_batch) {
            const u32 qn = (n_in - q0 < in_batch) ? n_in - q0 : in_batch;
            TRY(modup(ctx, ctx->stream, ct_in + (size_t)q0 * ctw + (size_t)r * N, (long long)ctw, qn, Dig,
                      X0 + (size_t)q0 * x0_stride + (size_t)r * N, x0_stride));
            // the rotations of the batch, key-major (rotation t = (k - 1) * qn + q: those that share a key follow one
            // another, so that an inner-product block loads the key once for all of them), dealt out to the lanes
            // in contiguous runs
            const u32 n_rot = qn * (b - 1);
            const u32 per = cdiv(b - 1, (u32)lanes_baby) * qn;           // whole keys per lane: no key is streamed by two lanes
            const int used = (int)cdiv(n_rot, per);
            TRY(fork_lanes(ctx, used));
            for (int c = 0; c < used; ++c) {
                RotBatch rb;
                memset(&rb, 0, sizeof(rb));
                const u32 t_end = (u32)(c + 1) * per < n_rot ? (u32)(c + 1) * per : n_rot;
                for (u32 t = (u32)c * per; t < t_end; ++t) {
                    const u32 q = t % qn, k = t / qn + 1;
                    const int i = rb.n++;
                    rb.key[i] = baby_key[k];
                    rb.dig[i] = (int)q;
                    rb.c0[i] = (int)((q0 + q) * b);
                    rb.out[i] = (int)((q0 + q) * b + k);
                }
                if (dh) {       // no division by P: the inner product's last step assembles the rotated input in X
                    CK(launch_key_inner_product(ctx->ring, rb, Dig, ctx->keys, nullptr, ctx->device_error, lane[c].s, X,
                                                ctx->perms));
                    continue;
                }
                CK(launch_key_inner_product(ctx->ring, rb, Dig, ctx->keys, lane[c].U, ctx->device_error, lane[c].s));
                TRY(moddown_batch(ctx, lane[c], rb, X, (long long)ctw, X, (long long)ctw));
            }
            TRY(join_lanes(ctx, used));
        }
    }
    stamp(ctx, 1);

    // ---- multiply-accumulate over the encoded diagonals (double hoisting: over the extended basis, into Aext)
    const u32 n_terms = n_in * b, n_pj = n_out * g;
    u64* mac_out = dh ? (u64*)ctx->Aext.p : A;
    MacScatter msc;
    memset(&msc, 0, sizeof(msc));
    if (assemble) {         // component 0 of the inner sums with j >= 1 is stored rotated (only the output assembly reads it)
        msc.pinv = ctx->perms;
        msc.n_out = n_out;
        for (u32 j = 1; j < g; ++j) msc.key[j] = giant_key[j];
    }
    if (pt_weights && pt_weights->pt) {
        // double hoisting: the launch for the special prime (one eighth of the words, on whole-word arithmetic) runs
        // beside the launch for the ciphertext primes
        // (also while single launches are being timed, chains serialised: the pair is then timed as one span, the way
        // it runs)
        const bool beside = dh && (lanes > 1 || ctx->prof.timing);
        ProfSpan span(beside ? &ctx->prof : nullptr, CAT_MAC, ctx->stream);
        if (beside) TRY(fork_lanes(ctx, 2));
        CK(launch_mac(ctx->ring, pt_weights->pt, pt_weights->lay, X, mac_out, n_pj, n_terms, true, ctx->device_error, ctx->stream,
                      beside ? ctx->side[0] : nullptr, &msc));
        if (beside) TRY(join_lanes(ctx, 2));
    } else {
        // fallback: encode groups of (j, p) just in time into a scratch ring, then consume them (weights kept as
        // coefficients: the same without the encoder, only their transforms)
        const size_t group_bytes = (size_t)n_terms * nmp * N * 8;
        const size_t fit = ctx->encode_scratch_bytes / group_bytes;
        const u32 groups = fit < 1 ? 1u : fit > (size_t)n_pj ? n_pj : (u32)fit;
        const TileLayout jl = mac_tile_layout(ctx->ring, groups, n_terms, nmp);
        TRY(ensure(ctx, ctx->ptjit, mac_tile_bytes(ctx->ring, jl)));
        for (u32 pj0 = 0; pj0 < n_pj; pj0 += groups) {
            const u32 cnt = (n_pj - pj0 < groups) ? n_pj - pj0 : groups;
            const TileLayout cl = mac_tile_layout(ctx->ring, cnt, n_terms, nmp);
            TRY(encode_range(ctx, W_raw, d_out, d_in, pj0 * n_terms, cnt * n_terms, (u64*)ctx->ptjit.p, cl, pj0, pt_weights));
            msc.pj0 = pj0;
            CK(launch_mac(ctx->ring, (const u64*)ctx->ptjit.p, cl, X, mac_out + (size_t)pj0 * xw, cnt, n_terms, false,
                          ctx->device_error, ctx->stream, nullptr, &msc));
        }
    }
    if (dh && !assemble) {
        // one division by P per inner sum and component: A[pj][comp][i] = (Aext[pj][comp][i] - t) * P^{-1}, t the
        // centred lift of the residue modulo P
        const u64* Aext = (const u64*)ctx->Aext.p;
        memset(&B, 0, sizeof(B));
        B.src = Aext + (size_t)r * N;
        B.dst = (u64*)ctx->Tc.p;
        B.src_so = (long long)nb * N;
        B.dst_so = N;
        B.n_m = 1;
        B.mod0 = r;
        B.mod_step = 0;
        B.store_centred = 1;
        CK(ntt_inverse(ctx->ring, B, n_pj * 2, ctx->stream));
        memset(&B, 0, sizeof(B));
        B.src = (const u64*)ctx->Tc.p;
        B.dst = (u64*)ctx->Tn.p;
        B.src_so = N;
        B.src_sm = 0;
        B.dst_so = (long long)r * N;
        B.dst_sm = N;
        B.n_m = r;
        B.mod0 = 0;
        B.mod_step = 1;
        B.lift_mod = ctx->ring.q[r];
        RotBatch no_rb;
        memset(&no_rb, 0, sizeof(no_rb));
        ModDownEpilogue epi;
        memset(&epi, 0, sizeof(epi));
        epi.u = Aext;
        epi.out_base = A;
        epi.out_stride = (long long)r * N;
        epi.plain = 1;
        CK(ntt_forward_moddown(ctx->ring, B, n_pj * 2, no_rb, epi, ctx->stream));
    }
    stamp(ctx, 2);

    // ---- giant steps: rotate A[j][p] by j*b*tau (full key switch each), then sum over j
    if (n_giant) {
        const u32 per = cdiv(n_giant, (u32)lanes_giant);
        const int used = (int)cdiv(n_giant, per);
        // a single chain may use the buffers of all lanes (they are contiguous)
        const u32 giant_chunk = lanes_giant == 1 ? giant_per_lane * (u32)lanes : giant_per_lane;
        TRY(fork_lanes(ctx, used));
        for (int c = 0; c < used; ++c) {
            const u32 lane_end = (u32)(c + 1) * per < n_giant ? (u32)(c + 1) * per : n_giant;
            for (u32 rho0 = (u32)c * per; rho0 < lane_end; rho0 += giant_chunk) {
                const u32 cnt = (lane_end - rho0 < giant_chunk) ? lane_end - rho0 : giant_chunk;
                if (cnt > (u32)MAX_ROT_BATCH) return BF_ERR_INVALID_ARG;   // (cannot happen: see giant_per_lane)
                if (assemble) {
                    // The inner sums stay in the extended basis.  A giant step needs the digits of c1 / P: both happen
                    // in the coefficient domain, where the division is element-wise, so one inverse transform over all
                    // r + 1 primes feeds the hoisted ModUp, whose first load divides (no transform of the lift of the
                    // P-residue, none of the quotient back and forth)
                    const u64* Esrc = (const u64*)ctx->Aext.p + (size_t)(n_out + rho0) * xw + (size_t)nmp * N;   // c1 of each
                    memset(&B, 0, sizeof(B));
                    B.src = Esrc;
                    B.dst = lane[c].Cc;
                    B.src_so = (long long)xw;
                    B.src_sm = N;
                    B.dst_so = (long long)nb * N;
                    B.dst_sm = N;
                    B.n_m = nb;
                    B.mod0 = 0;
                    B.mod_step = 1;
                    B.store_centred = 2;
                    CK(ntt_inverse(ctx->ring, B, cnt, lane[c].s));
                    TRY(modup(ctx, lane[c].s, lane[c].Cc, (long long)nb * N, cnt, lane[c].Dig, nullptr, 0,
                              lane[c].Cc + (size_t)r * N));
                    RotBatch rb;
                    memset(&rb, 0, sizeof(rb));
                    rb.n = (int)cnt;
                    for (u32 t = 0; t < cnt; ++t) {
                        rb.key[t] = giant_key[(rho0 + t) / n_out + 1];
                        rb.dig[t] = (int)t;
                        rb.c0[t] = (int)t;
                        rb.out[t] = (int)t;
                    }
                    // (stored through the rotation: the output assembly reads plain sums)
                    CK(launch_key_inner_product(ctx->ring, rb, lane[c].Dig, ctx->keys,
                                                (u64*)ctx->Ubig.p + (size_t)rho0 * 2 * nb * N, ctx->device_error, lane[c].s,
                                                nullptr, ctx->perms));
                    continue;
                }
                const u64* Asrc = A + (size_t)(n_out + rho0) * ctw;      // ciphertexts with j >= 1 are contiguous
                memset(&B, 0, sizeof(B));
                B.src = Asrc + (size_t)r * N;                            // c1 of each
                B.dst = lane[c].Cc;
                B.src_so = (long long)ctw;
                B.src_sm = N;
                B.dst_so = (long long)r * N;
                B.dst_sm = N;
                B.n_m = r;
                B.mod0 = 0;
                B.mod_step = 1;
                CK(ntt_inverse(ctx->ring, B, cnt, lane[c].s));
                TRY(modup(ctx, lane[c].s, lane[c].Cc, (long long)r * N, cnt, lane[c].Dig, Asrc + (size_t)r * N, (long long)ctw));
                RotBatch rb;
                memset(&rb, 0, sizeof(rb));
                rb.n = (int)cnt;
                for (u32 t = 0; t < cnt; ++t) {
                    const u32 j = (rho0 + t) / n_out + 1;
                    rb.key[t] = giant_key[j];
                    rb.dig[t] = (int)t;
                    rb.c0[t] = (int)t;
                    rb.out[t] = (int)t;
                }
                if (per_output) {
                    CK(launch_key_inner_product(ctx->ring, rb, lane[c].Dig, ctx->keys,
                                                (u64*)ctx->Ubig.p + (size_t)rho0 * 2 * nb * N, ctx->device_error, lane[c].s));
                    continue;
                }
                CK(launch_key_inner_product(ctx->ring, rb, lane[c].Dig, ctx->keys, lane[c].U, ctx->device_error, lane[c].s));
                TRY(moddown_batch(ctx, lane[c], rb, Asrc, (long long)ctw, Rres + (size_t)rho0 * ctw, (long long)ctw));
            }
        }
        TRY(join_lanes(ctx, used));
        if (assemble) {
            // Output p, component by component, is a sum of terms of the extended basis, each divided by P by itself
            // (the inner sum of giant step 0, the rotated c0 parts of the other inner sums) or once for their sum (the
            // key-switch results).  The result is wanted in the coefficient domain, where the division is element-
            // wise: so the terms' residues modulo the q_i are summed in the load of one inverse transform, their
            // residues modulo P are transformed apart, and one element-wise kernel divides.  Same values as dividing
            // each term in the transform domain (the transform is linear, the rotation commutes with the centred lift).
            RotBatch rb;
            memset(&rb, 0, sizeof(rb));
            rb.n = (int)(g - 1);
            for (u32 j = 1; j < g; ++j) rb.key[j - 1] = giant_key[j];
            ModDownEpilogue epi;
            memset(&epi, 0, sizeof(epi));
            epi.u = (const u64*)ctx->Ubig.p;
            epi.aext = (const u64*)ctx->Aext.p;
            epi.aext_stride = (long long)xw;
            epi.n_sum = g - 1;
            epi.n_out = n_out;
            epi.assemble = 1;
            const u32 n_t = g + 3;
            const bool beside = lanes > 1;
            if (beside) TRY(fork_lanes(ctx, 2));
            memset(&B, 0, sizeof(B));
            B.src = epi.aext;                                   // (read through epi)
            B.dst = (u64*)ctx->Tc.p;
            B.dst_so = (long long)n_t * N;
            B.dst_sm = N;
            B.n_m = n_t;
            B.mod0 = r;
            B.mod_step = 0;
            B.store_centred = 1;
            CK(ntt_inverse_gathersum(ctx->ring, B, n_out, rb, epi, beside ? ctx->side[0] : ctx->stream));
            memset(&B, 0, sizeof(B));
            B.src = epi.aext;
            B.dst = ct_out;
            B.dst_so = (long long)ctw;
            B.dst_sm = N;
            B.n_m = 2 * r;
            B.mod_wrap = r;
            B.mod0 = 0;
            B.mod_step = 1;
            CK(ntt_inverse_gathersum(ctx->ring, B, n_out, rb, epi, ctx->stream));
            if (beside) TRY(join_lanes(ctx, 2));
            CK(finish_division(ctx->ring, ct_out, (long long)ctw, (const u64*)ctx->Tc.p, n_t, n_out, ctx->stream,
                               ct_low ? &rcs : nullptr, ct_low));
            stamp(ctx, 3);
            stamp(ctx, 4);
            if (!pt_weights) TRY(check_overflow(ctx));
            return BF_OK;
        }
        if (per_output) {
            // sum over the giant steps of each output in the extended basis (each term read through its rotation),
            // then one division by P per output and component; the rotated c0 parts join in the same epilogue
            RotBatch rb;
            memset(&rb, 0, sizeof(rb));
            rb.n = (int)(g - 1);
            for (u32 j = 1; j < g; ++j) rb.key[j - 1] = giant_key[j];
            ModDownEpilogue epi;
            memset(&epi, 0, sizeof(epi));
            epi.u = (const u64*)ctx->Ubig.p;
            epi.c0_base = A + (size_t)n_out * ctw;              // ciphertexts with j >= 1, index (j - 1) * n_out + p
            epi.c0_stride = (long long)ctw;
            epi.pinv = ctx->perms;
            epi.perm = ctx->perms_fwd;
            epi.out_base = Rres;
            epi.out_stride = (long long)ctw;
            epi.n_sum = g - 1;
            epi.n_out = n_out;
            memset(&B, 0, sizeof(B));
            B.src = (const u64*)ctx->Ubig.p;                    // (read through epi)
            B.dst = (u64*)ctx->Tc.p;
            B.dst_so = N;
            B.n_m = 1;
            B.mod0 = r;
            B.mod_step = 0;
            B.store_centred = 1;
            CK(ntt_inverse_gathersum(ctx->ring, B, n_out * 2, rb, epi, ctx->stream));
            memset(&B, 0, sizeof(B));
            B.src = (const u64*)ctx->Tc.p;
            B.dst = (u64*)ctx->Tn.p;
            B.src_so = N;
            B.src_sm = 0;
            B.dst_so = (long long)r * N;
            B.dst_sm = N;
            B.n_m = r;
            B.mod0 = 0;
            B.mod_step = 1;
            B.lift_mod = ctx->ring.q[r];
            CK(ntt_forward_moddown(ctx->ring, B, n_out * 2, rb, epi, ctx->stream));
        }
    }
    stamp(ctx, 3);

    // ---- back to the coefficient domain; the sum over giant steps happens in the transform's load:
    // Y[p] = A[0][p] + sum_{j >= 1} (rotated A[j][p])
    memset(&B, 0, sizeof(B));
    B.src = A;
    B.dst = ct_out;
    B.src_so = B.dst_so = (long long)ctw;
    B.src_sm = B.dst_sm = N;
    B.n_m = 2 * r;
    B.mod_wrap = r;
    B.mod0 = 0;
    B.mod_step = 1;
    B.sum_src = Rres;
    B.sum_terms = per_output ? 1 : g - 1;
    B.sum_stride = (long long)n_out * ctw;
    CK(ntt_inverse(ctx->ring, B, n_out, ctx->stream));
    if (ct_low) CK(launch_rescale(ctx->ring, ct_out, ct_low, n_out, r, rcs.inv, rcs.invs, rcs.qlmod, ctx->stream));
    stamp(ctx, 4);
    if (!pt_weights) TRY(check_overflow(ctx));
    (void)nb;
    return BF_OK;
}

static void destroy_graphs(bf_ctx* ctx) {
    for (auto& kv : ctx->graphs)
        if (kv.second.exec) cudaGraphExecDestroy(kv.second.exec);
    ctx->graphs.clear();
}

// The launch sequence of a call depends only on its arguments and on the context's buffers, so the
// second call with the same arguments is captured into a CUDA graph and later calls replay it: the
// 20-odd dependent launches then cost one submission and lose their launch gaps.  Not used on the
// fallback path (it synchronises to read the encoder's range flag), while per-launch or per-stage
// timing is on, or when the caller's stream is itself being captured.
static int linear_call(bf_ctx* ctx, const uint64_t* ct_in, uint32_t n_in, const bf_weights* pt_weights,
                       const float* W_raw, uint32_t d_out, uint32_t d_in, uint64_t* ct_out, uint32_t n_out, bool rescaled);

extern "C" int bf_linear(bf_ctx* ctx, const uint64_t* ct_in, uint32_t n_in, const bf_weights* pt_weights,
                         const float* W_raw, uint32_t d_out, uint32_t d_in, uint64_t* ct_out, uint32_t n_out) {
    return linear_call(ctx, ct_in, n_in, pt_weights, W_raw, d_out, d_in, ct_out, n_out, false);
}

extern "C" int bf_linear_rescaled(bf_ctx* ctx, const uint64_t* ct_in, uint32_t n_in, const bf_weights* pt_weights,
                                  const float* W_raw, uint32_t d_out, uint32_t d_in, uint64_t* ct_low, uint32_t n_out,
                                  double* scale_inout) {
    if (!ctx) return BF_ERR_INVALID_ARG;
    if (ctx->r < 2) return BF_ERR_LEVEL;
    TRY(linear_call(ctx, ct_in, n_in, pt_weights, W_raw, d_out, d_in, ct_low, n_out, true));
    if (scale_inout) *scale_inout /= (double)ctx->ring.q[ctx->r - 1];
    return BF_OK;
}

// (out: ct_out of bf_linear, or ct_low of bf_linear_rescaled)
static int linear_call(bf_ctx* ctx, const uint64_t* ct_in, uint32_t n_in, const bf_weights* pt_weights,
                       const float* W_raw, uint32_t d_out, uint32_t d_in, uint64_t* ct_out, uint32_t n_out, bool rescaled) {
    if (!ctx) return BF_ERR_INVALID_ARG;
    bool eligible = ctx->use_graphs && pt_weights && !ctx->timing && !ctx->prof.timing && ct_in && ct_out;
    if (eligible) {
        cudaStreamCaptureStatus st = cudaStreamCaptureStatusNone;
        if (cudaStreamIsCapturing(ctx->stream, &st) != cudaSuccess || st != cudaStreamCaptureStatusNone) {
            cudaGetLastError();
            eligible = false;
        }
    }
    if (!eligible) return linear_enqueue(ctx, ct_in, n_in, pt_weights, W_raw, d_out, d_in, rescaled ? nullptr : ct_out, n_out, rescaled ? ct_out : nullptr);
    if (ctx->graphs.size() > 4096) destroy_graphs(ctx);
    bf_ctx::GraphKey key{ct_in, pt_weights, ct_out, d_out, d_in, rescaled};
    bf_ctx::GraphEntry& ge = ctx->graphs[key];
    if (ge.exec && ge.epoch == ctx->epoch) {
        CK(cudaGraphLaunch(ge.exec, ctx->stream));
        for (int c = 0; c < (int)CAT_COUNT; ++c) ctx->prof.launches[c] += ge.launches[c];
        ctx->prof.key_bytes_distinct += ge.key_bytes_distinct;
        ctx->prof.key_bytes_per_rotation += ge.key_bytes_per_rotation;
        return BF_OK;
    }
    if (ge.exec) {                       // stale: buffers, keys or weights changed since the capture
        cudaGraphExecDestroy(ge.exec);
        ge.exec = nullptr;
        ge.seen = 0;
    }
    if (ge.unusable || ge.seen == 0 || ge.epoch != ctx->epoch) {
        // first call with these arguments (or first since a change): run directly, which also grows
        // whatever scratch the shape needs
        const int rc = linear_enqueue(ctx, ct_in, n_in, pt_weights, W_raw, d_out, d_in, rescaled ? nullptr : ct_out, n_out, rescaled ? ct_out : nullptr);
        if (rc == BF_OK) { ge.seen = 1; ge.epoch = ctx->epoch; }
        return rc;
    }
    // second call: capture, instantiate, launch
    uint64_t before[CAT_COUNT];
    for (int c = 0; c < (int)CAT_COUNT; ++c) before[c] = ctx->prof.launches[c];
    const uint64_t kd_before = ctx->prof.key_bytes_distinct, kr_before = ctx->prof.key_bytes_per_rotation;
    if (cudaStreamBeginCapture(ctx->stream, cudaStreamCaptureModeThreadLocal) != cudaSuccess) {
        cudaGetLastError();
        ge.unusable = true;
        return linear_enqueue(ctx, ct_in, n_in, pt_weights, W_raw, d_out, d_in, rescaled ? nullptr : ct_out, n_out, rescaled ? ct_out : nullptr);
    }
    // measured: inside a replayed graph plain edges are as fast as programmatic ones, so capture those
    const bool dependent = ctx->ring.dependent_launch;
    ctx->ring.dependent_launch = false;
    const int rc = linear_enqueue(ctx, ct_in, n_in, pt_weights, W_raw, d_out, d_in, rescaled ? nullptr : ct_out, n_out, rescaled ? ct_out : nullptr);
    ctx->ring.dependent_launch = dependent;
    cudaGraph_t graph = nullptr;
    const cudaError_t ec = cudaStreamEndCapture(ctx->stream, &graph);
    if (rc != BF_OK || ec != cudaSuccess || !graph) {
        cudaGetLastError();
        if (graph) cudaGraphDestroy(graph);
        for (int c = 0; c < (int)CAT_COUNT; ++c) ctx->prof.launches[c] = before[c];
        ctx->prof.key_bytes_distinct = kd_before;
        ctx->prof.key_bytes_per_rotation = kr_before;
        ge.unusable = true;
        if (rc != BF_OK) return rc;      // argument errors are reported as usual
        return linear_enqueue(ctx, ct_in, n_in, pt_weights, W_raw, d_out, d_in, rescaled ? nullptr : ct_out, n_out, rescaled ? ct_out : nullptr);
    }
    cudaGraphExec_t exec = nullptr;
    const cudaError_t ei = cudaGraphInstantiate(&exec, graph, 0);
    cudaGraphDestroy(graph);
    if (ei != cudaSuccess || !exec) {
        cudaGetLastError();
        for (int c = 0; c < (int)CAT_COUNT; ++c) ctx->prof.launches[c] = before[c];
        ctx->prof.key_bytes_distinct = kd_before;
        ctx->prof.key_bytes_per_rotation = kr_before;
        ge.unusable = true;
        return linear_enqueue(ctx, ct_in, n_in, pt_weights, W_raw, d_out, d_in, rescaled ? nullptr : ct_out, n_out, rescaled ? ct_out : nullptr);
    }
    for (int c = 0; c < (int)CAT_COUNT; ++c) ge.launches[c] = ctx->prof.launches[c] - before[c];
    ge.key_bytes_distinct = ctx->prof.key_bytes_distinct - kd_before;
    ge.key_bytes_per_rotation = ctx->prof.key_bytes_per_rotation - kr_before;
    ge.exec = exec;
    ge.epoch = ctx->epoch;
    CK(cudaGraphLaunch(ge.exec, ctx->stream));
    return BF_OK;
}

extern "C" int bf_set_graph_replay(bf_ctx* ctx, int on) {
    if (!ctx) return BF_ERR_INVALID_ARG;
    ctx->use_graphs = on ? 1 : 0;
    if (!on) destroy_graphs(ctx);
    return BF_OK;
}

extern "C" int bf_set_encode_scratch(bf_ctx* ctx, uint64_t bytes) {
    if (!ctx || !bytes) return BF_ERR_INVALID_ARG;
    ctx->encode_scratch_bytes = (size_t)bytes;
    return BF_OK;
}

extern "C" int bf_set_coefficient_cache(bf_ctx* ctx, int bits) {
    if (!ctx || (bits != 0 && bits != 32 && bits != 64)) return BF_ERR_INVALID_ARG;
    ctx->coef_cache_bits = (u32)bits;
    return BF_OK;
}

extern "C" int bf_set_compact_cache(bf_ctx* ctx, int on) {
    if (!ctx) return BF_ERR_INVALID_ARG;
    ctx->ring.compact_cache = on != 0;     // weights encoded from now on (and the fallback path's scratch) use it
    return BF_OK;
}

extern "C" int bf_set_lanes(bf_ctx* ctx, int n_lanes) {
    if (!ctx || n_lanes < 1 || n_lanes > bf_ctx::MAX_LANES) return BF_ERR_INVALID_ARG;
    ctx->n_lanes = n_lanes;
    destroy_graphs(ctx);            // stored graphs have the old shape
    return BF_OK;
}

extern "C" int bf_set_dependent_launch(bf_ctx* ctx, int on) {
    if (!ctx) return BF_ERR_INVALID_ARG;
    ctx->ring.dependent_launch = on != 0;
    destroy_graphs(ctx);            // stored graphs carry the edges of the old setting
    return BF_OK;
}

extern "C" int bf_rescale(bf_ctx* ctx, const uint64_t* ct_in, uint64_t* ct_out, uint32_t n_ct, uint32_t level,
                          double* scale_inout) {
    if (!ctx || !ct_in || !ct_out || !n_ct) return BF_ERR_INVALID_ARG;
    if (level < 2 || level > ctx->r) return BF_ERR_LEVEL;
    const u64 qL = ctx->ring.q[level - 1];
    RescaleConsts rc;
    rescale_consts(ctx, level, rc);
    CK(launch_rescale(ctx->ring, ct_in, ct_out, n_ct, level, rc.inv, rc.invs, rc.qlmod, ctx->stream));
    if (scale_inout) *scale_inout /= (double)qL;
    return BF_OK;
}

extern "C" int bf_linear_host(bf_ctx* ctx, const uint64_t* host_ct_in, uint32_t n_in, const bf_weights* pt_weights,
                              const float* W_raw, uint32_t d_out, uint32_t d_in, uint64_t* host_ct_out,
                              uint32_t n_out) {
    if (!ctx || !host_ct_in || !host_ct_out) return BF_ERR_INVALID_ARG;
    const size_t ctw = (size_t)2 * ctx->r * ctx->N;
    TRY(ensure(ctx, ctx->stage_in, (size_t)n_in * ctw * 8));
    TRY(ensure(ctx, ctx->stage_out, (size_t)n_out * ctw * 8));
    CK(cudaMemcpyAsync(ctx->stage_in.p, host_ct_in, (size_t)n_in * ctw * 8, cudaMemcpyHostToDevice, ctx->stream));
    TRY(bf_linear_rescaled(ctx, (const u64*)ctx->stage_in.p, n_in, pt_weights, W_raw, d_out, d_in, (u64*)ctx->stage_out.p,
                           n_out, nullptr));
    const size_t out_bytes = (size_t)n_out * 2 * (ctx->r - 1) * ctx->N * 8;
    CK(cudaMemcpyAsync(host_ct_out, ctx->stage_out.p, out_bytes, cudaMemcpyDeviceToHost, ctx->stream));
    return check_overflow(ctx);          // synchronises; reports a device-side wait that gave up
}

extern "C" int bf_rotate(bf_ctx* ctx, const uint64_t* ct_in, uint32_t steps, uint64_t* ct_out) {
    if (!ctx || !ct_in || !ct_out) return BF_ERR_INVALID_ARG;
    const u32 N = ctx->N, r = ctx->r;
    const size_t ctw = (size_t)2 * r * N;
    int key = -1;
    TRY(find_key(ctx, steps, &key));
    TRY(ensure(ctx, ctx->X, 2 * ctw * 8));
    TRY(ensure_rot_scratch(ctx, 1, 1));
    u64* X = (u64*)ctx->X.p;
    PolyBatch B;
    memset(&B, 0, sizeof(B));
    B.src = ct_in;
    B.dst = X;
    B.src_so = B.dst_so = (long long)r * N;
    B.src_sm = B.dst_sm = N;
    B.n_m = r;
    B.mod_step = 1;
    CK(ntt_forward(ctx->ring, B, 2, LOAD_PLAIN, ctx->stream));
    TRY(modup(ctx, ctx->stream, ct_in + (size_t)r * N, (long long)r * N, 1, (u64*)ctx->Dig.p, X + (size_t)r * N, 0));
    RotBatch rb;
    memset(&rb, 0, sizeof(rb));
    rb.n = 1;
    rb.key[0] = key;
    rb.out[0] = 1;
    CK(launch_key_inner_product(ctx->ring, rb, (const u64*)ctx->Dig.p, ctx->keys, (u64*)ctx->U.p, ctx->device_error,
                                ctx->stream));
    TRY(moddown_batch(ctx, main_lane(ctx), rb, X, (long long)ctw, X, (long long)ctw));
    memset(&B, 0, sizeof(B));
    B.src = X + ctw;
    B.dst = ct_out;
    B.src_so = B.dst_so = (long long)r * N;
    B.src_sm = B.dst_sm = N;
    B.n_m = r;
    B.mod_step = 1;
    CK(ntt_inverse(ctx->ring, B, 2, ctx->stream));
    return BF_OK;
}

// In-ciphertext fold of the tau partial sums: ct <- ct + rot(ct, 2^i) for i = 0 .. log2(tau) - 1, batched
// over the ciphertexts.  Every round is one key switch per ciphertext: transform, hoisted ModUp of c1, inner
// product with the key of 2^i, division by P with the automorphism as a scatter, then the sum of the
// ciphertext and its rotation goes back to the coefficient domain (the next round decomposes its c1 again).
extern "C" int bf_fold(bf_ctx* ctx, uint64_t* ct, uint32_t n_ct) {
    if (!ctx || !ct || !n_ct) return BF_ERR_INVALID_ARG;
    const u32 N = ctx->N, r = ctx->r, tau = ctx->plan.tau;
    if (tau & (tau - 1)) return BF_ERR_INVALID_ARG;
    const size_t ctw = (size_t)2 * r * N;
    std::vector<int> keys;
    for (u32 steps = 1; steps < tau; steps <<= 1) {
        int key = -1;
        TRY(find_key(ctx, steps, &key));
        keys.push_back(key);
    }
    if (keys.empty()) return BF_OK;
    u32 batch = giant_batch(ctx);
    if (batch > n_ct) batch = n_ct;
    TRY(ensure(ctx, ctx->X, (size_t)batch * 2 * ctw * 8));
    TRY(ensure_rot_scratch(ctx, batch, batch));
    u64* X = (u64*)ctx->X.p;                             // [t][0] = NTT(ct_t), [t][1] = its rotation
    const Lane lane = main_lane(ctx);
    for (u32 t0 = 0; t0 < n_ct; t0 += batch) {
        const u32 cnt = (n_ct - t0 < batch) ? n_ct - t0 : batch;
        u64* cts = ct + (size_t)t0 * ctw;
        for (int key : keys) {
            PolyBatch B;
            memset(&B, 0, sizeof(B));
            B.src = cts;
            B.dst = X;
            B.src_so = (long long)ctw;
            B.dst_so = (long long)2 * ctw;
            B.src_sm = B.dst_sm = N;
            B.n_m = 2 * r;
            B.mod_wrap = r;
            B.mod_step = 1;
            CK(ntt_forward(ctx->ring, B, cnt, LOAD_PLAIN, ctx->stream));
            TRY(modup(ctx, ctx->stream, cts + (size_t)r * N, (long long)ctw, cnt, lane.Dig, X + (size_t)r * N,
                      (long long)2 * ctw));
            RotBatch rb;
            memset(&rb, 0, sizeof(rb));
            rb.n = (int)cnt;
            for (u32 t = 0; t < cnt; ++t) {
                rb.key[t] = key;
                rb.dig[t] = (int)t;
                rb.c0[t] = (int)(2 * t);
                rb.out[t] = (int)(2 * t + 1);
            }
            CK(launch_key_inner_product(ctx->ring, rb, lane.Dig, ctx->keys, lane.U, ctx->device_error, ctx->stream));
            TRY(moddown_batch(ctx, lane, rb, X, (long long)ctw, X, (long long)ctw));
            memset(&B, 0, sizeof(B));
            B.src = X;
            B.dst = cts;
            B.src_so = (long long)2 * ctw;
            B.dst_so = (long long)ctw;
            B.src_sm = B.dst_sm = N;
            B.n_m = 2 * r;
            B.mod_wrap = r;
            B.mod_step = 1;
            B.sum_src = X + ctw;
            B.sum_terms = 1;
            B.sum_stride = 0;
            CK(ntt_inverse(ctx->ring, B, cnt, ctx->stream));
        }
    }
    return BF_OK;
}

extern "C" int bf_negacyclic_mul(bf_ctx* ctx, const uint64_t* a, const uint64_t* b, uint64_t* out, uint32_t n_polys) {
    if (!ctx || !a || !b || !out || !n_polys) return BF_ERR_INVALID_ARG;
    const u32 N = ctx->N, nb = ctx->r + 1;
    const u32 n_outer = cdiv(n_polys, nb);
    // polynomial t uses basis prime t mod (r+1): pad the batch to whole groups of r+1
    TRY(ensure(ctx, ctx->nm_a, (size_t)n_outer * nb * N * 8));
    TRY(ensure(ctx, ctx->nm_b, (size_t)n_outer * nb * N * 8));
    CK(cudaMemsetAsync(ctx->nm_a.p, 0, (size_t)n_outer * nb * N * 8, ctx->stream));
    CK(cudaMemsetAsync(ctx->nm_b.p, 0, (size_t)n_outer * nb * N * 8, ctx->stream));
    CK(cudaMemcpyAsync(ctx->nm_a.p, a, (size_t)n_polys * N * 8, cudaMemcpyDeviceToDevice, ctx->stream));
    CK(cudaMemcpyAsync(ctx->nm_b.p, b, (size_t)n_polys * N * 8, cudaMemcpyDeviceToDevice, ctx->stream));
    PolyBatch B;
    memset(&B, 0, sizeof(B));
    B.src_so = B.dst_so = (long long)nb * N;
    B.src_sm = B.dst_sm = N;
    B.n_m = nb;
    B.mod_step = 1;
    B.src = ctx->nm_a.p;
    B.dst = (u64*)ctx->nm_a.p;
    CK(ntt_forward(ctx->ring, B, n_outer, LOAD_PLAIN, ctx->stream));
    B.src = ctx->nm_b.p;
    B.dst = (u64*)ctx->nm_b.p;
    CK(ntt_forward(ctx->ring, B, n_outer, LOAD_PLAIN, ctx->stream));
    CK(launch_pointwise_mul(ctx->ring, (const u64*)ctx->nm_a.p, (const u64*)ctx->nm_b.p, (u64*)ctx->nm_a.p,
                            n_outer * nb, nb, 0, ctx->stream));
    B.src = ctx->nm_a.p;
    B.dst = (u64*)ctx->nm_a.p;
    CK(ntt_inverse(ctx->ring, B, n_outer, ctx->stream));
    CK(cudaMemcpyAsync(out, ctx->nm_a.p, (size_t)n_polys * N * 8, cudaMemcpyDeviceToDevice, ctx->stream));
    return BF_OK;
}

extern "C" int bf_weights_export(bf_ctx* ctx, const bf_weights* w, uint32_t p, uint32_t q, uint32_t j, uint32_t k,
                                 uint64_t* out) {
    if (!ctx || !w || !out) return BF_ERR_INVALID_ARG;
    if (p >= w->n_out || q >= w->n_in || j >= w->g || k >= w->b) return BF_ERR_SHAPE;
    const u32 N = ctx->N, r = ctx->r;
    const size_t d = (((size_t)j * w->n_out + p) * w->n_in + q) * w->b + k;
    PolyBatch B;
    memset(&B, 0, sizeof(B));
    if (w->coef) {      // coefficient form: reduce the stored integers per prime (through a transform and back)
        const void* src = (const i64*)w->coef + d * N;
        if (w->coef_bits == 32) {
            TRY(ensure(ctx, ctx->coef, (size_t)N * sizeof(i64)));
            CK(launch_widen_i32(ctx->ring, (const int*)w->coef + d * N, (i64*)ctx->coef.p, N, ctx->stream));
            src = ctx->coef.p;
        }
        B.src = src;
        B.dst = out;
        B.src_so = 0;
        B.src_sm = 0;
        B.dst_so = (long long)r * N;
        B.dst_sm = N;
        B.n_m = r;
        B.mod_step = 1;
        CK(ntt_forward(ctx->ring, B, 1, LOAD_I64, ctx->stream));
        B.src = out;
        B.src_so = (long long)r * N;
        B.src_sm = N;
        CK(ntt_inverse(ctx->ring, B, 1, ctx->stream));
        return BF_OK;
    }
    B.src = out;                                 // unused: the first pass reads the tiles
    B.dst = out;
    B.src_so = B.dst_so = (long long)r * N;
    B.src_sm = B.dst_sm = N;
    B.n_m = r;
    B.mod_step = 1;
    B.from_mont = 1;
    B.split_bits = mac_split_bits(ctx->ring);
    B.tile_ptr = w->pt;
    B.tile = w->lay;
    B.tile_pj0 = 0;
    B.o_base = (u32)d;
    CK(ntt_inverse(ctx->ring, B, 1, ctx->stream));
    return BF_OK;
}

extern "C" int bf_set_stage_timing(bf_ctx* ctx, int on) {
    if (!ctx) return BF_ERR_INVALID_ARG;
    ctx->timing = on ? 1 : 0;
    if (!on) ctx->ev_valid = false;
    return BF_OK;
}

extern "C" int bf_get_stage_ms(bf_ctx* ctx, float* ms_out) {
    if (!ctx || !ms_out) return BF_ERR_INVALID_ARG;
    if (!ctx->ev_valid) return BF_ERR_INVALID_ARG;
    CK(cudaStreamSynchronize(ctx->stream));
    for (int i = 0; i < 4; ++i) CK(cudaEventElapsedTime(&ms_out[i], ctx->ev[i], ctx->ev[i + 1]));
    return BF_OK;
}

extern "C" int bf_set_kernel_timing(bf_ctx* ctx, int on) {
    if (!ctx) return BF_ERR_INVALID_ARG;
    ctx->prof.timing = on != 0;
    return BF_OK;
}

extern "C" int bf_kernel_categories(void) { return (int)CAT_COUNT; }

extern "C" const char* bf_kernel_category_name(int cat) {
    static const char* names[CAT_COUNT] = {"ntt_fwd_strided", "ntt_fwd_contig", "ntt_inv_contig", "ntt_inv_strided",
                                           "key_inner_product", "mac", "rescale",
                                           "encode_fft_a", "encode_fft_b", "pointwise_mul", "divide_by_p"};
    return (cat >= 0 && cat < (int)CAT_COUNT) ? names[cat] : "";
}

extern "C" int bf_get_kernel_stats(bf_ctx* ctx, uint64_t* launches_out, float* ms_out) {
    if (!ctx || !launches_out || !ms_out) return BF_ERR_INVALID_ARG;
    CK(cudaStreamSynchronize(ctx->stream));
    for (int c = 0; c < (int)CAT_COUNT; ++c) {
        launches_out[c] = ctx->prof.launches[c];
        ms_out[c] = 0.f;
        ctx->prof.launches[c] = 0;
    }
    for (auto& rec : ctx->prof.recs) {
        float ms = 0.f;
        CK(cudaEventElapsedTime(&ms, rec.a, rec.b));
        ms_out[rec.cat] += ms;
        ctx->prof.pool.push_back(rec.a);
        ctx->prof.pool.push_back(rec.b);
    }
    ctx->prof.recs.clear();
    return BF_OK;
}

extern "C" int bf_get_key_stream_bytes(bf_ctx* ctx, uint64_t* distinct_out, uint64_t* per_rotation_out) {
    if (!ctx || !distinct_out || !per_rotation_out) return BF_ERR_INVALID_ARG;
    *distinct_out = ctx->prof.key_bytes_distinct;
    *per_rotation_out = ctx->prof.key_bytes_per_rotation;
    ctx->prof.key_bytes_distinct = ctx->prof.key_bytes_per_rotation = 0;
    return BF_OK;
}

static int measure_rate(bf_ctx* ctx, bool fp64, double* out) {
    if (!ctx || !out) return BF_ERR_INVALID_ARG;
    TRY(ensure(ctx, ctx->nm_a, 4096));
    cudaDeviceProp prop;
    CK(cudaGetDeviceProperties(&prop, ctx->device));
    const u32 blocks = (u32)prop.multiProcessorCount * 8, iters = 256;
    cudaEvent_t a, b;
    CK(cudaEventCreate(&a));
    CK(cudaEventCreate(&b));
    double best = 0.0;
    for (int rep = 0; rep < 5; ++rep) {
        CK(cudaEventRecord(a, ctx->stream));
        CK(fp64 ? launch_fma64_probe((u64*)ctx->nm_a.p, blocks, iters, ctx->stream)
                : launch_imad_probe((u64*)ctx->nm_a.p, blocks, iters, ctx->stream));
        CK(cudaEventRecord(b, ctx->stream));
        CK(cudaEventSynchronize(b));
        float ms = 0.f;
        CK(cudaEventElapsedTime(&ms, a, b));
        const double rate = (double)blocks * 256.0 * iters * 64.0 / (ms * 1e-3);
        if (rep > 0 && rate > best) best = rate;
    }
    cudaEventDestroy(a);
    cudaEventDestroy(b);
    *out = best;
    return BF_OK;
}

extern "C" int bf_measure_imad_rate(bf_ctx* ctx, double* mad_per_second_out) {
    return measure_rate(ctx, false, mad_per_second_out);
}

extern "C" int bf_measure_fma64_rate(bf_ctx* ctx, double* fma_per_second_out) {
    return measure_rate(ctx, true, fma_per_second_out);
}

// ------------------------------------------------------------------------------------------------
// Allocation-free variant of bf_negacyclic_mul.
//
// bf_negacyclic_mul keeps its two transform-domain operands in scratch memory that the context
// obtains from cudaMalloc on first use.  A caller whose device memory is entirely owned by its own
// pool (a serving engine that reserved the whole GPU up front), or that sits on a latency path
// where the implicit device synchronisation of cudaMalloc is unacceptable, cannot afford that.
// This variant uses a fixed array that lives in the library's device image instead: every GPU that
// loads the library holds BF_NOALLOC_BYTES of it until the process exits.
constexpr size_t BF_NOALLOC_WORDS = (size_t)1 << 19;          // per operand: 4 MiB; 8 MiB in total
static __device__ __align__(256) unsigned long long g_noalloc_scratch[2 * BF_NOALLOC_WORDS];
// The array's name is only a host-side handle.  Its device address is looked up once per device,
// with that device current, and cached here.
static u64* g_noalloc_addr[64] = {nullptr};

extern "C" uint64_t bf_noalloc_max_words(void) { return (uint64_t)BF_NOALLOC_WORDS; }

extern "C" int bf_negacyclic_mul_noalloc(bf_ctx* ctx, const uint64_t* a, const uint64_t* b, uint64_t* out,
                                         uint32_t n_polys) {
    if (!ctx || !a || !b || !out || !n_polys) return BF_ERR_INVALID_ARG;
    const u32 N = ctx->N, nb = ctx->r + 1;
    if ((u64)n_polys * N > BF_NOALLOC_WORDS) return BF_ERR_TOO_LARGE;   // (before any 32-bit rounding of the count)
    const u32 n_outer = cdiv(n_polys, nb);
    const size_t words = (size_t)n_outer * nb * N;               // batch padded to whole groups of r+1 primes
    if (words > BF_NOALLOC_WORDS) return BF_ERR_TOO_LARGE;
    int dev = -1;
    CK(cudaGetDevice(&dev));
    if (dev != ctx->device || dev < 0 || dev >= 64) return BF_ERR_INVALID_ARG;
    if (!g_noalloc_addr[dev]) {                                  // first call on this device: set-up
        void* p = nullptr;
        CK(cudaGetSymbolAddress(&p, g_noalloc_scratch));
        g_noalloc_addr[dev] = (u64*)p;
    }
    u64* sa = g_noalloc_addr[dev];
    u64* sb = sa + BF_NOALLOC_WORDS;
    // The array keeps whatever the previous call left; the padding polynomials of this batch are
    // transformed along with the real ones, so give them defined contents.
    const size_t used = (size_t)n_polys * N;
    if (words > used) {
        CK(cudaMemsetAsync(sa + used, 0, (words - used) * 8, ctx->stream));
        CK(cudaMemsetAsync(sb + used, 0, (words - used) * 8, ctx->stream));
    }
    CK(cudaMemcpyAsync(sa, a, used * 8, cudaMemcpyDeviceToDevice, ctx->stream));
    CK(cudaMemcpyAsync(sb, b, used * 8, cudaMemcpyDeviceToDevice, ctx->stream));
    Profiler* saved = ctx->ring.prof;      // launch timing would create events; keep this path free of that
    ctx->ring.prof = nullptr;
    PolyBatch B;
    memset(&B, 0, sizeof(B));
    B.src_so = B.dst_so = (long long)nb * N;
    B.src_sm = B.dst_sm = N;
    B.n_m = nb;
    B.mod_step = 1;
    cudaError_t e;
    B.src = sa;
    B.dst = sa;
    e = ntt_forward(ctx->ring, B, n_outer, LOAD_PLAIN, ctx->stream);
    if (e == cudaSuccess) {
        B.src = sb;
        B.dst = sb;
        e = ntt_forward(ctx->ring, B, n_outer, LOAD_PLAIN, ctx->stream);
    }
    if (e == cudaSuccess) e = launch_pointwise_mul(ctx->ring, sa, sb, sa, n_outer * nb, nb, 0, ctx->stream);
    if (e == cudaSuccess) {
        B.src = sa;
        B.dst = sa;
        e = ntt_inverse(ctx->ring, B, n_outer, ctx->stream);
    }
    ctx->ring.prof = saved;
    CK(e);
    CK(cudaMemcpyAsync(out, sa, used * 8, cudaMemcpyDeviceToDevice, ctx->stream));
    return BF_OK;
}
