// CKKS weight encoding on the device (Sec. 4.2: weight-matrix diagonals are pre-encoded into
// resident BSGS objects, or encoded per call on the fallback path).
//
// For every generalised diagonal of a tile the kernels build the slot vector straight from the
// fp32 weight matrix, apply the inverse canonical embedding as an n-point complex FFT in fp64
// (n = N/2), multiply by the twist exp(-i pi k / N) and by scale/n, and round to 64-bit integer
// coefficients.  The per-prime reduction and the forward NTT happen in the NTT's load stage.
//
// The floating-point arithmetic is a fixed DAG so that results are reproducible bit for bit:
// radix-2 decimation-in-time butterflies (a, b) -> (a + w b, a - w b) over a bit-reversed input,
// the complex product formed as (br wr - bi wi, br wi + bi wr) with each product and each sum
// rounded on its own (the _rn intrinsics are never contracted into fused multiply-adds), twiddles
// taken from host-computed tables, and round-to-nearest-even at the end.  Register blocking only
// regroups butterflies; it does not change any operand.
#include "bf_host.h"

namespace bf {

struct FftCfg {
    int log_len, lanes, n_groups, K[4], log_other, first, pad;
};

__device__ __forceinline__ double2 cmul_rn(double2 b, double2 w) {
    double2 t;
    t.x = __dsub_rn(__dmul_rn(b.x, w.x), __dmul_rn(b.y, w.y));
    t.y = __dadd_rn(__dmul_rn(b.x, w.y), __dmul_rn(b.y, w.x));
    return t;
}

// Slot value of plaintext Pt[p][q][j][k] at slot s: generalised diagonal i = j*b + k of tile (p, q),
// pre-rotated right by j*b*tau.  Slot s' = (rho*D + kappa)*tau + c holds
// W[p*D + kappa][q*D + ((kappa + i + c*M) mod D)], zero outside the matrix.  With complex packing output
// ciphertext p carries two row blocks: W[2p*D + kappa][..] in the real part, W[(2p+1)*D + kappa][..] in
// the imaginary part.
__device__ __forceinline__ double2 diag_value(const DiagBatch& db, u32 dd, u32 s, u32 n) {
    const u32 k = dd % db.b;
    const u32 q = (dd / db.b) % db.n_in;
    const u32 p = (dd / (db.b * db.n_in)) % db.n_out;
    const u32 j = dd / (db.b * db.n_in * db.n_out);
    const u32 sp = (s - j * db.b * db.tau) & (n - 1);
    const u32 c = sp % db.tau;
    const u32 kappa = (sp / db.tau) % db.D;
    const u32 M = db.D / db.tau;
    const u32 row = p * db.D * (db.complex_pack ? 2u : 1u) + kappa;
    const u32 col = q * db.D + ((kappa + j * db.b + k + c * M) % db.D);
    double2 v = make_double2(0.0, 0.0);
    if (col >= db.d_in) return v;
    if (row < db.d_out) v.x = (double)__ldg(&db.W[(size_t)row * db.d_in + col]);
    if (db.complex_pack && row + db.D < db.d_out) v.y = (double)__ldg(&db.W[(size_t)(row + db.D) * db.d_in + col]);
    return v;
}

// One pass of the batched FFT.  CONTIG = the first pass (chunks of adjacent points, small butterfly
// distances, reads the weights); otherwise the strided second pass, which also applies twist,
// scale and rounding.
template <bool CONTIG>
__global__ void __launch_bounds__(256) encode_fft_pass(const EncodeTables tab, const DiagBatch db, const FftCfg cfg,
                                                       u32 logn, double2* __restrict__ scratch,
                                                       i64* __restrict__ coeff, int* __restrict__ overflow) {
    extern __shared__ double2 smc[];
    const u32 n = 1u << logn;
    const u32 diag = blockIdx.y;
    double2* buf = scratch + (size_t)diag * n;
    const int LEN = 1 << cfg.log_len;
    const int lanes = cfg.lanes;
    const int lane0 = blockIdx.x * lanes;
    const int other = 1 << cfg.log_other;
    const int pitch = LEN + cfg.pad;
    const int unit = CONTIG ? 1 : other;              // global index distance of one local index step

    int step = 1;
    for (int gi = 0; gi < cfg.n_groups; ++gi) {
        const int K = cfg.K[cfg.n_groups - 1 - gi];   // smallest distances first
        const int t0 = step << (K - 1);
        const int nsets = (LEN * lanes) >> K;
        const int sets_per_lane = LEN >> K;
        const bool g_first = (gi == 0), g_last = (gi == cfg.n_groups - 1);
        for (int w = threadIdx.x; w < nsets; w += blockDim.x) {
            int lane, u;
            if (CONTIG) { u = w % sets_per_lane; lane = w / sets_per_lane; }
            else { lane = w % lanes; u = w / lanes; }
            const int blk = u / step, off = u % step;
            const int base = blk * 2 * t0 + off;
            double2 e[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                if (i < (1 << K)) {
                    const int li = base + i * step;
                    if (g_first) {
                        const u32 gidx = CONTIG ? (u32)(lane0 + lane) * LEN + li : (u32)li * other + lane0 + lane;
                        if (CONTIG) {
                            e[i] = diag_value(db, db.d0 + diag, __ldg(&tab.slot_of_pos[gidx]), n);
                        } else {
                            e[i] = buf[gidx];
                        }
                    } else {
                        e[i] = CONTIG ? smc[lane * pitch + li] : smc[li * lanes + lane];
                    }
                }
            }
            // stages with set-local distance d = 1, 2, 4 (times `step` in local index units)
#pragma unroll
            for (int s = 0; s < 3; ++s) {
                if (s < K) {
                    const int d = 1 << s;
                    const u32 half_local = (u32)d * step;                  // butterfly distance, local units
                    const u32 tw_stride = n / (2u * half_local * unit);    // n / len
#pragma unroll
                    for (int i = 0; i < 8; ++i) {
                        if (i < (1 << K) && ((i & d) == 0)) {
                            const u32 li = base + i * step;
                            const u32 jj = (li % half_local) * unit + (CONTIG ? 0u : (u32)(lane0 + lane));
                            const double2 wv = __ldg(&tab.T[(size_t)jj * tw_stride]);
                            const double2 t = cmul_rn(e[i + d], wv);
                            const double2 a = e[i];
                            e[i].x = __dadd_rn(a.x, t.x);
                            e[i].y = __dadd_rn(a.y, t.y);
                            e[i + d].x = __dsub_rn(a.x, t.x);
                            e[i + d].y = __dsub_rn(a.y, t.y);
                        }
                    }
                }
            }
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                if (i < (1 << K)) {
                    const int li = base + i * step;
                    if (g_last) {
                        const u32 gidx = CONTIG ? (u32)(lane0 + lane) * LEN + li : (u32)li * other + lane0 + lane;
                        if (CONTIG) {
                            buf[gidx] = e[i];
                        } else {
                            // twist by exp(-i pi k / N), scale by Delta / n, round to nearest even
                            const double2 uu = cmul_rn(e[i], __ldg(&tab.Z[gidx]));
                            const double cr = rint(__dmul_rn(uu.x, tab.scale_over_n));
                            const double ci = rint(__dmul_rn(uu.y, tab.scale_over_n));
                            const double lim = 4611686018427387904.0;      // 2^62
                            if (!(fabs(cr) < lim) || !(fabs(ci) < lim)) {
                                atomicExch(overflow, 1);
                            } else {
                                i64* cp = coeff + (size_t)diag * 2 * n;
                                cp[gidx] = (i64)cr;
                                cp[gidx + n] = (i64)ci;
                            }
                        }
                    } else {
                        if (CONTIG) smc[lane * pitch + li] = e[i];
                        else smc[li * lanes + lane] = e[i];
                    }
                }
            }
        }
        if (!g_last) __syncthreads();
        step <<= K;
    }
}

// ------------------------------------------------------------------------------------------------
// The same two passes with the geometry known at compile time (rings of 2^12 to 2^16, i.e. 8 to 128
// rows in the second pass): index arithmetic becomes shifts and masks, the groups unroll, and the
// position of a diagonal is worked out once per thread.  The floating-point operations, their
// operands and their order are exactly those of the kernel above.
__host__ __device__ constexpr int fft_k(int s, int i) {
    constexpr int t[9][4] = {{0, 0, 0, 0}, {1, 0, 0, 0}, {2, 0, 0, 0}, {3, 0, 0, 0}, {2, 2, 0, 0},
                             {3, 2, 0, 0}, {3, 3, 0, 0}, {3, 2, 2, 0}, {3, 3, 2, 0}};
    return t[s][i];
}
__host__ __device__ constexpr int fft_ng(int s) {
    int n = 0;
    for (int i = 0; i < 4; ++i) n += fft_k(s, i) ? 1 : 0;
    return n;
}
// stages done before group gi (groups run from the last table entry to the first)
__host__ __device__ constexpr int fft_log_step(int s, int gi) {
    int st = 0;
    for (int g = 0; g < gi; ++g) st += fft_k(s, fft_ng(s) - 1 - g);
    return st;
}

struct DiagPos {        // where diagonal dd sits: see diag_value
    u32 rot, row0, col0, ik, log_tau, D, tau, M;
};
__device__ __forceinline__ DiagPos diag_pos(const DiagBatch& db, u32 dd) {
    DiagPos dp;
    const u32 k = dd % db.b;
    const u32 q = (dd / db.b) % db.n_in;
    const u32 p = (dd / (db.b * db.n_in)) % db.n_out;
    const u32 j = dd / (db.b * db.n_in * db.n_out);
    dp.rot = j * db.b * db.tau;
    dp.row0 = p * db.D * (db.complex_pack ? 2u : 1u);
    dp.col0 = q * db.D;
    dp.ik = j * db.b + k;
    dp.log_tau = 31u - (u32)__clz(db.tau);
    dp.D = db.D;
    dp.tau = db.tau;
    dp.M = db.D >> dp.log_tau;
    return dp;
}
__device__ __forceinline__ double2 diag_value_at(const DiagBatch& db, const DiagPos& dp, u32 s, u32 n) {
    const u32 sp = (s - dp.rot) & (n - 1);
    const u32 c = sp & (dp.tau - 1);
    const u32 kappa = (sp >> dp.log_tau) & (dp.D - 1);
    const u32 row = dp.row0 + kappa;
    const u32 col = dp.col0 + ((kappa + dp.ik + c * dp.M) & (dp.D - 1));
    double2 v = make_double2(0.0, 0.0);
    if (col >= db.d_in) return v;
    if (row < db.d_out) v.x = (double)__ldg(&db.W[(size_t)row * db.d_in + col]);
    if (db.complex_pack && row + dp.D < db.d_out) v.y = (double)__ldg(&db.W[(size_t)(row + dp.D) * db.d_in + col]);
    return v;
}

// Shared-memory slot of point li of chunk `lane` in the contiguous pass: 16-byte elements, eight to a row
// of banks; XOR-ing the column with the row number keeps the stride-4 and stride-32 sets of a quarter
// warp on distinct columns (with plain or padded indexing the first two groups conflict 4- and 2-way).
__device__ __forceinline__ int fft_swz(int lane, int li, int log_len) {
    return (lane << log_len) + (li ^ ((li >> 3) & 7));
}

template <bool CONTIG, int LOG_LEN, int LOG_LANES, int LOG_OTHER, int GI>
__device__ __forceinline__ void fft_group(const EncodeTables& tab, const DiagBatch& db, const DiagPos& dp, double2* smc,
                                          double2* __restrict__ buf, i64* __restrict__ cp, int* __restrict__ overflow,
                                          u32 lane0) {
    constexpr int NG = fft_ng(LOG_LEN);
    constexpr int K = fft_k(LOG_LEN, NG - 1 - GI);
    constexpr int LOG_STEP = fft_log_step(LOG_LEN, GI);
    constexpr int LEN = 1 << LOG_LEN, LANES = 1 << LOG_LANES;
    constexpr u32 n = 1u << (LOG_LEN + LOG_OTHER);
    constexpr int STEP = 1 << LOG_STEP;
    constexpr int NSETS = (LEN * LANES) >> K;
    constexpr bool FIRST = GI == 0, LAST = GI == NG - 1;
    constexpr int LOG_UNIT = CONTIG ? 0 : LOG_OTHER;      // global index distance of one local index step
    for (int w = threadIdx.x; w < NSETS; w += blockDim.x) {
        int lane, u;
        if (CONTIG) { u = w & ((LEN >> K) - 1); lane = w >> (LOG_LEN - K); }
        else { lane = w & (LANES - 1); u = w >> LOG_LANES; }
        const int blk = u >> LOG_STEP, off = u & (STEP - 1);
        const int base = (blk << (LOG_STEP + K)) + off;
        double2 e[1 << K];
#pragma unroll
        for (int i = 0; i < (1 << K); ++i) {
            const int li = base + i * STEP;
            if (FIRST) {
                const u32 gidx = CONTIG ? ((u32)(lane0 + lane) << LOG_LEN) + li : ((u32)li << LOG_OTHER) + lane0 + lane;
                if (CONTIG) {
                    e[i] = diag_value_at(db, dp, __ldg(&tab.slot_of_pos[gidx]), n);
                } else {
                    e[i] = buf[gidx];
                }
            } else {
                e[i] = CONTIG ? smc[fft_swz(lane, li, LOG_LEN)] : smc[li * LANES + lane];
            }
        }
#pragma unroll
        for (int s = 0; s < K; ++s) {
            const int d = 1 << s;
            const int log_half = s + LOG_STEP;                        // butterfly distance 2^log_half, local units
            const int log_tw_stride = (LOG_LEN + LOG_OTHER) - 1 - log_half - LOG_UNIT;   // n / len
#pragma unroll
            for (int i = 0; i < (1 << K); ++i) {
                if ((i & d) == 0) {
                    const u32 li = base + i * STEP;
                    const u32 jj = ((li & ((1u << log_half) - 1)) << LOG_UNIT) + (CONTIG ? 0u : (u32)(lane0 + lane));
                    const double2 wv = __ldg(&tab.T[(size_t)jj << log_tw_stride]);
                    const double2 t = cmul_rn(e[i + d], wv);
                    const double2 a = e[i];
                    e[i].x = __dadd_rn(a.x, t.x);
                    e[i].y = __dadd_rn(a.y, t.y);
                    e[i + d].x = __dsub_rn(a.x, t.x);
                    e[i + d].y = __dsub_rn(a.y, t.y);
                }
            }
        }
#pragma unroll
        for (int i = 0; i < (1 << K); ++i) {
            const int li = base + i * STEP;
            if (LAST) {
                const u32 gidx = CONTIG ? ((u32)(lane0 + lane) << LOG_LEN) + li : ((u32)li << LOG_OTHER) + lane0 + lane;
                if (CONTIG) {
                    buf[gidx] = e[i];
                } else {
                    // twist by exp(-i pi k / N), scale by Delta / n, round to nearest even
                    const double2 uu = cmul_rn(e[i], __ldg(&tab.Z[gidx]));
                    const double cr = rint(__dmul_rn(uu.x, tab.scale_over_n));
                    const double ci = rint(__dmul_rn(uu.y, tab.scale_over_n));
                    const double lim = 4611686018427387904.0;      // 2^62
                    if (!(fabs(cr) < lim) || !(fabs(ci) < lim)) {
                        atomicExch(overflow, 1);
                    } else {
                        cp[gidx] = (i64)cr;
                        cp[gidx + n] = (i64)ci;
                    }
                }
            } else {
                if (CONTIG) smc[fft_swz(lane, li, LOG_LEN)] = e[i];
                else smc[li * LANES + lane] = e[i];
            }
        }
    }
    if (!LAST) __syncthreads();
}

template <bool CONTIG, int LOG_LEN, int LOG_LANES, int LOG_OTHER>
__global__ void __launch_bounds__(256) encode_fft_fixed(const EncodeTables tab, const DiagBatch db,
                                                        double2* __restrict__ scratch, i64* __restrict__ coeff,
                                                        int* __restrict__ overflow) {
    extern __shared__ double2 smc[];
    constexpr u32 n = 1u << (LOG_LEN + LOG_OTHER);
    constexpr int NG = fft_ng(LOG_LEN);
    const u32 diag = blockIdx.y;
    double2* buf = scratch + (size_t)diag * n;
    i64* cp = coeff + (size_t)diag * 2 * n;
    const u32 lane0 = blockIdx.x << LOG_LANES;
    DiagPos dp = {};
    if (CONTIG) dp = diag_pos(db, db.d0 + diag);
    fft_group<CONTIG, LOG_LEN, LOG_LANES, LOG_OTHER, 0>(tab, db, dp, smc, buf, cp, overflow, lane0);
    if constexpr (NG > 1) fft_group<CONTIG, LOG_LEN, LOG_LANES, LOG_OTHER, 1>(tab, db, dp, smc, buf, cp, overflow, lane0);
    if constexpr (NG > 2) fft_group<CONTIG, LOG_LEN, LOG_LANES, LOG_OTHER, 2>(tab, db, dp, smc, buf, cp, overflow, lane0);
    if constexpr (NG > 3) fft_group<CONTIG, LOG_LEN, LOG_LANES, LOG_OTHER, 3>(tab, db, dp, smc, buf, cp, overflow, lane0);
}

// log_b rows in the second pass: lanes (columns per block) = 2048 / rows
template <int LOG_B>
static cudaError_t launch_encode_fixed(const RingHost& ring, const EncodeTables& tab, const DiagBatch& db,
                                       double2* fft_scratch, i64* coeff_out, int* overflow_flag, cudaStream_t stream) {
    constexpr int LOG_A = 8, LOG_LANES_A = 3, LOG_LANES_B = 11 - LOG_B;
    {
        dim3 grid((1u << LOG_B) >> LOG_LANES_A, db.count);
        constexpr size_t smem = (size_t)(1 << LOG_A) * (1 << LOG_LANES_A) * sizeof(double2);
        ProfScope prof(ring.prof, CAT_ENCODE_FFT_A, stream);
        encode_fft_fixed<true, LOG_A, LOG_LANES_A, LOG_B><<<grid, 256, smem, stream>>>(tab, db, fft_scratch, coeff_out,
                                                                                      overflow_flag);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    {
        dim3 grid((1u << LOG_A) >> LOG_LANES_B, db.count);
        constexpr size_t smem = (size_t)(1 << LOG_B) * (1 << LOG_LANES_B) * sizeof(double2);
        ProfScope prof(ring.prof, CAT_ENCODE_FFT_B, stream);
        encode_fft_fixed<false, LOG_B, LOG_LANES_B, LOG_A><<<grid, 256, smem, stream>>>(tab, db, fft_scratch, coeff_out,
                                                                                       overflow_flag);
        return cudaGetLastError();
    }
}

static void fft_groups(int s, int* K, int* n) {
    static const int table[9][4] = {{0, 0, 0, 0}, {1, 0, 0, 0}, {2, 0, 0, 0}, {3, 0, 0, 0}, {2, 2, 0, 0},
                                    {3, 2, 0, 0}, {3, 3, 0, 0}, {3, 2, 2, 0}, {3, 3, 2, 0}};
    *n = 0;
    for (int i = 0; i < 4; ++i) {
        K[i] = table[s][i];
        if (K[i]) (*n)++;
    }
}

cudaError_t launch_encode(const RingHost& ring, const EncodeTables& tab, const DiagBatch& db, double2* fft_scratch,
                          i64* coeff_out, int* overflow_flag, cudaStream_t stream) {
    if (db.count == 0) return cudaSuccess;
    const u32 logn = ring.dev.logN - 1;
    switch ((int)logn - 8) {                    // the common ring sizes have kernels of their own
        case 3: return launch_encode_fixed<3>(ring, tab, db, fft_scratch, coeff_out, overflow_flag, stream);
        case 4: return launch_encode_fixed<4>(ring, tab, db, fft_scratch, coeff_out, overflow_flag, stream);
        case 5: return launch_encode_fixed<5>(ring, tab, db, fft_scratch, coeff_out, overflow_flag, stream);
        case 6: return launch_encode_fixed<6>(ring, tab, db, fft_scratch, coeff_out, overflow_flag, stream);
        case 7: return launch_encode_fixed<7>(ring, tab, db, fft_scratch, coeff_out, overflow_flag, stream);
        default: break;
    }
    const int log_a = 8;                        // first pass: chunks of 256 points
    const int log_b = (int)logn - log_a;        // second pass: 2^log_b rows
    FftCfg ca, cb;
    ca.log_len = log_a; ca.log_other = log_b; ca.lanes = 8; ca.first = 1; ca.pad = 1;
    fft_groups(ca.log_len, ca.K, &ca.n_groups);
    cb.log_len = log_b; cb.log_other = log_a; cb.first = 0; cb.pad = 0;
    int tc = 2048 / (1 << log_b);
    if (tc < 16) tc = 16;
    if (tc > 256) tc = 256;
    cb.lanes = tc;
    fft_groups(cb.log_len, cb.K, &cb.n_groups);
    {
        dim3 grid((1u << ca.log_other) / ca.lanes, db.count);
        if ((1u << ca.log_other) < (u32)ca.lanes) { ca.lanes = 1 << ca.log_other; grid.x = 1; }
        const size_t smem = (size_t)((1 << ca.log_len) + ca.pad) * ca.lanes * sizeof(double2);
        ProfScope prof(ring.prof, CAT_ENCODE_FFT_A, stream);
        encode_fft_pass<true><<<grid, 256, smem, stream>>>(tab, db, ca, logn, fft_scratch, coeff_out, overflow_flag);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    {
        dim3 grid((1u << cb.log_other) / cb.lanes, db.count);
        const size_t smem = (size_t)(1 << cb.log_len) * cb.lanes * sizeof(double2);
        int threads = ((1 << cb.log_len) * cb.lanes) / 8;
        if (threads < 32) threads = 32;
        if (threads > 256) threads = 256;
        ProfScope prof(ring.prof, CAT_ENCODE_FFT_B, stream);
        encode_fft_pass<false><<<grid, threads, smem, stream>>>(tab, db, cb, logn, fft_scratch, coeff_out, overflow_flag);
        return cudaGetLastError();
    }
}

}  // namespace bf
