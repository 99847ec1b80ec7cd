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

struct PassCfg {
    int log_len;        // log2 of the local transform length
    int lanes;          // independent local transforms per block (columns, or chunks)
    int n_groups;       // stage groups, in forward order (largest butterfly distance first)
    int K[4];           // stages per group (2 or 3, or 1 for tiny lengths)
    int log_other;      // log2(N / local length): rows for the contiguous pass, columns for the strided
    int first;          // 1: this pass reads the batch source through the load functor; 0: in place on dst
    int pad;            // shared-memory padding per lane in the contiguous pass
};

template <int LOAD>
__device__ __forceinline__ u64 load_src(const void* src, size_t idx, u64 q, u64 mu, u64 lift_mod, u64 lift_red) {
    if (LOAD == LOAD_PLAIN) return ((const u64*)src)[idx];
    if (LOAD == LOAD_REDUCE) return barrett64(((const u64*)src)[idx], q, mu);
    if (LOAD == LOAD_I64) {
        i64 v = ((const i64*)src)[idx];
        u64 a = v < 0 ? (u64)(-v) : (u64)v;
        u64 m = barrett64(a, q, mu);
        return (v < 0 && m != 0) ? q - m : m;
    }
    // LOAD_CENTRED
    u64 t = ((const u64*)src)[idx];
    u64 m = barrett64(t, q, mu);
    if (t > (lift_mod - 1) / 2) m = sub_mod(m, lift_red, q);
    return m;
}

template <int K, bool FWD>
__device__ __forceinline__ void set_butterflies(u64 (&e)[8], const ulonglong2* __restrict__ tw,
                                                u32 m0mult, u32 blk, u64 q) {
    const u64 q2 = 2 * q;
#pragma unroll
    for (int s = 0; s < K; ++s) {
        const int st = FWD ? s : (K - 1 - s);
        const int d = (1 << K) >> (st + 1);
#pragma unroll
        for (int sub = 0; sub < (1 << st); ++sub) {
            const ulonglong2 w = __ldg(&tw[(m0mult << st) + (blk << st) + sub]);
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

// One pass of a batched transform.  FWD/STRIDED pick the direction and which half this is:
//   forward  = strided pass (first), then contiguous pass (in place)
//   inverse  = contiguous pass (first), then strided pass (in place, scales by N^{-1})
template <bool FWD, bool STRIDED, int LOAD>
__global__ void __launch_bounds__(512) ntt_pass(const RingDev R, const PolyBatch B, const PassCfg cfg) {
    extern __shared__ u64 sm[];
    const u32 poly = blockIdx.y;
    const u32 o = poly / B.n_m, m = poly % B.n_m;
    const u32 mod = B.mod0 + m * B.mod_step;
    const u64 q = R.q[mod], mu = R.mu[mod];
    const ulonglong2* __restrict__ tw = (FWD ? R.tw_fwd : R.tw_inv) + (size_t)mod * R.N;
    u64* dst = B.dst + (size_t)o * B.dst_so + (size_t)m * B.dst_sm;
    const char* src = (const char*)B.src + ((size_t)o * B.src_so + (size_t)m * B.src_sm) * 8;
    const u64 lift_red = (LOAD == LOAD_CENTRED) ? barrett64(B.lift_mod, q, mu) : 0;

    const int LEN = 1 << cfg.log_len;
    const int lanes = cfg.lanes;
    const int lane0 = blockIdx.x * lanes;            // first column (strided) or first chunk (contiguous)
    const int other = 1 << cfg.log_other;
    const int pitch = LEN + cfg.pad;                 // contiguous pass: shared-memory pitch per chunk
    const bool from_src = cfg.first != 0;
    const bool last_pass = !from_src;

    // Forward walks the groups from the largest butterfly distance down, inverse the other way.
    int t0 = FWD ? (LEN >> 1) : 0;
    int step_inv = 1;
    for (int gi = 0; gi < cfg.n_groups; ++gi) {
        const int K = FWD ? cfg.K[gi] : cfg.K[cfg.n_groups - 1 - gi];
        if (!FWD) t0 = step_inv << (K - 1);
        const int step = t0 >> (K - 1);              // spacing of a set's points
        const int m0 = LEN / (2 * t0);               // blocks at the group's first forward stage
        const int nsets = (LEN * lanes) >> K;
        const int sets_per_lane = LEN >> K;
        const bool g_first = (gi == 0), g_last = (gi == cfg.n_groups - 1);
        for (int w = threadIdx.x; w < nsets; w += blockDim.x) {
            int lane, u;
            if (STRIDED) { lane = w % lanes; u = w / lanes; }
            else { u = w % sets_per_lane; lane = w / sets_per_lane; }
            const int blk = u / step, off = u % step;
            const int base = blk * 2 * t0 + off;
            const u32 mult = STRIDED ? 1u : (u32)(other + lane0 + lane);
            u64 e[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                if (i < (1 << K)) {
                    const int li = base + i * step;
                    if (g_first) {
                        const size_t gidx = STRIDED ? ((size_t)li * other + lane0 + lane)
                                                    : ((size_t)(lane0 + lane) * LEN + li);
                        e[i] = from_src ? load_src<LOAD>(src, gidx, q, mu, B.lift_mod, lift_red) : dst[gidx];
                    } else {
                        e[i] = STRIDED ? sm[li * lanes + lane] : sm[lane * pitch + li];
                    }
                }
            }
            if (K == 3) set_butterflies<3, FWD>(e, tw, (u32)m0 * mult, (u32)blk, q);
            else if (K == 2) set_butterflies<2, FWD>(e, tw, (u32)m0 * mult, (u32)blk, q);
            else set_butterflies<1, FWD>(e, tw, (u32)m0 * mult, (u32)blk, q);
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                if (i < (1 << K)) {
                    const int li = base + i * step;
                    if (g_last) {
                        const size_t gidx = STRIDED ? ((size_t)li * other + lane0 + lane)
                                                    : ((size_t)(lane0 + lane) * LEN + li);
                        u64 v = e[i];
                        if (last_pass) {
                            if (FWD) {                       // [0, 4q) -> [0, q)
                                if (v >= 2 * q) v -= 2 * q;
                                if (v >= q) v -= q;
                            } else {                         // scale by N^{-1}, [0, 2q) -> [0, q)
                                v = mul_shoup(v, R.ninv[mod], R.ninvs[mod], q);
                            }
                        }
                        dst[gidx] = v;
                    } else {
                        if (STRIDED) sm[li * lanes + lane] = e[i];
                        else sm[lane * pitch + li] = e[i];
                    }
                }
            }
        }
        if (!g_last) __syncthreads();
        if (FWD) t0 >>= K; else step_inv <<= K;
    }
}

static void stage_groups(int s, int* K, int* n) {
    // Split s butterfly stages into register-resident groups of 3 or 2 (1 only when s == 1).
    static const int table[9][4] = {{0, 0, 0, 0}, {1, 0, 0, 0}, {2, 0, 0, 0}, {3, 0, 0, 0}, {2, 2, 0, 0},
                                    {3, 2, 0, 0}, {3, 3, 0, 0}, {3, 2, 2, 0}, {3, 3, 2, 0}};
    *n = 0;
    for (int i = 0; i < 4; ++i) {
        K[i] = table[s][i];
        if (K[i]) (*n)++;
    }
}

NttGeometry ntt_geometry(u32 logN) {
    NttGeometry g;
    g.log_c = 8;                              // contiguous pass: chunks of 256 points
    g.log_r = (int)logN - g.log_c;            // strided pass: 4 .. 256 rows
    const int Rr = 1 << g.log_r;
    int tc = 2048 / Rr;
    if (tc < 16) tc = 16;
    if (tc > 256) tc = 256;
    g.strided_lanes = tc;
    g.strided_threads = (Rr * tc) / 8 < 32 ? 32 : (Rr * tc) / 8;
    g.contig_lanes = Rr < 8 ? Rr : 8;         // up to 8 chunks of 256 points per block
    g.contig_threads = 256;
    g.contig_pad = 8;
    return g;
}

template <bool FWD, bool STRIDED>
static cudaError_t launch_pass(const RingHost& ring, const PolyBatch& B, u32 n_polys, int load, bool first,
                               cudaStream_t stream) {
    const NttGeometry& g = ring.geom;
    PassCfg cfg;
    cfg.log_len = STRIDED ? g.log_r : g.log_c;
    cfg.log_other = STRIDED ? g.log_c : g.log_r;
    cfg.lanes = STRIDED ? g.strided_lanes : g.contig_lanes;
    cfg.first = first ? 1 : 0;
    cfg.pad = STRIDED ? 0 : g.contig_pad;
    stage_groups(cfg.log_len, cfg.K, &cfg.n_groups);
    const int threads = STRIDED ? g.strided_threads : g.contig_threads;
    const int LEN = 1 << cfg.log_len;
    const size_t smem = STRIDED ? (size_t)LEN * cfg.lanes * 8 : (size_t)(LEN + cfg.pad) * cfg.lanes * 8;
    dim3 grid((1u << cfg.log_other) / cfg.lanes, n_polys);
    if (n_polys == 0) return cudaSuccess;
#define BF_LAUNCH(LM) ntt_pass<FWD, STRIDED, LM><<<grid, threads, smem, stream>>>(ring.dev, B, cfg)
    if (!first) BF_LAUNCH(LOAD_PLAIN);
    else if (load == LOAD_PLAIN) BF_LAUNCH(LOAD_PLAIN);
    else if (load == LOAD_REDUCE) BF_LAUNCH(LOAD_REDUCE);
    else if (load == LOAD_I64) BF_LAUNCH(LOAD_I64);
    else BF_LAUNCH(LOAD_CENTRED);
#undef BF_LAUNCH
    return cudaGetLastError();
}

cudaError_t ntt_forward(const RingHost& ring, const PolyBatch& B, u32 n_outer, int load, cudaStream_t stream) {
    const u32 n_polys = n_outer * B.n_m;
    cudaError_t e = launch_pass<true, true>(ring, B, n_polys, load, true, stream);
    if (e != cudaSuccess) return e;
    return launch_pass<true, false>(ring, B, n_polys, LOAD_PLAIN, false, stream);
}

cudaError_t ntt_inverse(const RingHost& ring, const PolyBatch& B, u32 n_outer, cudaStream_t stream) {
    const u32 n_polys = n_outer * B.n_m;
    cudaError_t e = launch_pass<false, false>(ring, B, n_polys, LOAD_PLAIN, true, stream);
    if (e != cudaSuccess) return e;
    return launch_pass<false, true>(ring, B, n_polys, LOAD_PLAIN, false, stream);
}

}  // namespace bf
