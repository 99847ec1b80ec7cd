// Streaming and element-wise kernels of the encrypted linear layer: the ciphertext x plaintext
// multiply-accumulate that streams encoded weight diagonals from HBM (the "ciphertext-plaintext
// multiplication with pre-encoded weight diagonals" of Sec. 3.5 / Sec. 4.2), the key-switch inner
// product, the division by the special prime, the giant-step sum and the rescale (Sec. 2.1).
#include "bf_host.h"

#include <cstring>

namespace bf {

// ------------------------------------------------------------------------------------------------
// Pointwise product of NTT-domain polynomials (parity helper for the transform).
__global__ void pointwise_mul_kernel(const RingDev R, const u64* __restrict__ a, const u64* __restrict__ b,
                                     u64* __restrict__ out, u32 n_m, u32 mod0) {
    const u32 poly = blockIdx.y;
    const u32 mod = mod0 + poly % n_m;
    const size_t idx = (size_t)poly * R.N + blockIdx.x * blockDim.x + threadIdx.x;
    u64 hi = 0, lo = 0;
    mac128(hi, lo, a[idx], b[idx]);
    out[idx] = reduce128(hi, lo, R.q[mod], R.mu[mod], R.c64[mod], R.c64s[mod]);
}

cudaError_t launch_pointwise_mul(const RingHost& ring, const u64* a, const u64* b, u64* out, u32 n_polys, u32 n_m,
                                 u32 mod0, cudaStream_t stream) {
    if (n_polys == 0) return cudaSuccess;
    dim3 grid(ring.dev.N / 256, n_polys);
    ProfScope prof(ring.prof, CAT_POINTWISE, stream);
    pointwise_mul_kernel<<<grid, 256, 0, stream>>>(ring.dev, a, b, out, n_m, mod0);
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// Asynchronous bulk copies (TMA, untiled form) and transaction barriers.
__device__ __forceinline__ u32 smem_addr(const void* p) { return (u32)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(u64* bar, u32 count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_addr(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(u64* bar, u32 bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_addr(bar)), "r"(bytes) : "memory");
}
// global -> shared copy of `bytes` (multiple of 16, both addresses 16-byte aligned); completion is
// signalled on the barrier as transferred bytes
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, u32 bytes, u64* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_addr(dst)),
                 "l"(src), "r"(bytes), "r"(smem_addr(bar))
                 : "memory");
}
// the same copy, with the lines marked "evict first" in L2: for streams that are read exactly once and must
// not push reused operands (rotated inputs, digits, outputs) out of the cache
__device__ __forceinline__ u64 l2_evict_first_policy() {
    u64 pol;
    asm volatile("createpolicy.fractional.L2::evict_first.b64 %0, 1.0;" : "=l"(pol));
    return pol;
}
__device__ __forceinline__ void bulk_g2s_stream(void* dst, const void* src, u32 bytes, u64* bar, u64 policy) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1], %2, [%3], %4;" ::"r"(
            smem_addr(dst)),
        "l"(src), "r"(bytes), "r"(smem_addr(bar)), "l"(policy)
        : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(u64* bar, u32 parity) {
    u32 ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_addr(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: gives up after a fixed number of polls (each poll may itself suspend for a while),
// records the failure and lets the caller carry on so that the kernel always terminates.
__device__ __forceinline__ void mbar_wait(u64* bar, u32 parity, int* error_flag) {
    for (int it = 0; it < (1 << 22); ++it)
        if (mbar_try_wait(bar, parity)) return;
    atomicExch(error_flag, 1);
}

__device__ __forceinline__ void mbar_arrive(u64* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_addr(bar)) : "memory");
}

// ------------------------------------------------------------------------------------------------
// Multiply-accumulate over encoded diagonals (the ciphertext x plaintext product of Sec. 3.5 / 4.2).
//   A[pj][comp][i][n] = sum_{t < n_terms} Pt[pj][t][i][n] * X[t][comp][i][n]   (mod q_i)
//
// A block owns one prime i and a tile of TN adjacent coefficients.  The rotated inputs X of that
// tile, for every term and both components, are brought into shared memory once and stay there.
// The encoded weights are streamed from HBM through a ring of shared-memory stages filled by bulk
// asynchronous copies that a dedicated producer warp issues; full/empty transaction barriers
// couple it to the eight consumer warps, so no block-wide barrier sits on the stream.  Each
// plaintext word crosses HBM exactly once and is shared by both ciphertext components.  The 256
// consumer threads are arranged as TN coefficients x PL "group lanes": lane l accumulates output
// groups pj = l, l + PL, ...
//
// Arithmetic.  The cached plaintexts are in Montgomery form (times 2^64 mod q_i).  KARA (all
// ciphertext primes below 2^50): they are stored as two 25-bit limbs per word, X is split the same
// way once per block, and products accumulate by Karatsuba (3 multiplies, no carries).  Otherwise
// words are whole and products accumulate as 32-bit limb partial sums with carries.  One Montgomery
// reduction per output word removes the 2^64.
constexpr int MAC_CONSUMERS = 256;
constexpr int MAC_THREADS = MAC_CONSUMERS + 32;   // + one producer warp
constexpr int MAC_TS = (int)TILE_TS;              // terms per stage
constexpr int MAC_STAGES = 2;                             // (measured: three narrower stages in the same ring are slower)
constexpr int MAC_STAGE_WORDS = MAC_TS * MAC_CONSUMERS;   // 2048 words per stage whatever TN is
constexpr int MAC_SLOT_BYTES = MAC_STAGE_WORDS * 8;       // ring slot: room for the widest word format
constexpr int MAC_RING_BYTES = MAC_STAGES * MAC_SLOT_BYTES;
constexpr int MAC_MAX_STAGES = MAC_STAGES;
constexpr u32 KARA_L = 25;

// COMPACT = false: every prime of the layout uses 8-byte words (the default), and the format tests fold away.
template <bool KARA, int LOG_TN, bool COMPACT>
__global__ void __launch_bounds__(MAC_THREADS, 3)
mac_kernel(const RingDev R, const u64* __restrict__ pt, const TileLayout lay, const u64* __restrict__ x,
           u64* __restrict__ a, u32 n_terms, u32 n_pj, u32 pj_per_block, u32 lazy_terms, u32 early_weights,
           u32 n_whole, u32 tail_split, u32 prime0, u32 n_launch_primes, int* __restrict__ error_flag, const MacScatter sc) {
    extern __shared__ __align__(128) unsigned char mac_smem[];
    asm volatile("griddepcontrol.launch_dependents;");
    constexpr u32 TN = 1u << LOG_TN, PL = MAC_CONSUMERS >> LOG_TN;
    unsigned char* ring = mac_smem;                                // [stages][stage bytes of this block's prime]
    u64* xs = (u64*)(mac_smem + MAC_RING_BYTES);                   // [n_terms][2][TN]
    u64* full = xs + (size_t)n_terms * 2 * TN;                     // [MAC_MAX_STAGES]
    u64* empty = full + MAC_MAX_STAGES;                            // [MAC_MAX_STAGES]
    // Work units (tile, prime, slice of the output groups) are numbered tile-fastest.  The first n_whole
    // blocks take one unit each; the units after them (the part that would be a thin last wave) are each
    // cut into tail_split blocks over their output groups, so that the last wave is short instead.
    const u32 N = R.N;
    const u32 r = lay.n_primes;                                    // primes per (term, component) of x and a
    const u32 tid = threadIdx.x;
    u32 unit = blockIdx.x, sub = 0, n_sub = 1;
    if (unit >= n_whole) {
        sub = (unit - n_whole) % tail_split;
        unit = n_whole + (unit - n_whole) / tail_split;
        n_sub = tail_split;
    }
    // (N / TN is a power of two; the remaining quotient by the number of primes of the launch is one division)
    const u32 tiles_log = R.logN - LOG_TN;
    const u32 tile_x = unit & ((1u << tiles_log) - 1u);
    const u32 rest = unit >> tiles_log, slice = rest / n_launch_primes;
    const u32 i = prime0 + (rest - slice * n_launch_primes);          // this launch covers primes prime0 .. + n_launch_primes - 1
    const u32 n0 = tile_x << LOG_TN;
    u32 pj_begin = slice * pj_per_block;
    u32 pj_end = min(n_pj, pj_begin + pj_per_block);
    if (n_sub > 1) {
        const u32 groups = (pj_end - pj_begin + PL - 1) / PL;
        const u32 per = (groups + n_sub - 1) / n_sub * PL;
        pj_begin = min(pj_end, pj_begin + sub * per);
        pj_end = min(pj_end, pj_begin + per);
        if (pj_begin >= pj_end) return;                            // (uniform for the block)
    }
    const u32 fmt = COMPACT ? tile_format(lay, i) : (u32)TILE_W64;          // this prime's word format decides the stage size
    const u32 stage_bytes = tile_stage_bytes(fmt);
    constexpr u32 n_stages = MAC_STAGES;
    const u32 n_groups = (pj_end - pj_begin + PL - 1) / PL;        // rounds of PL output groups
    const u32 n_chunks = (n_terms + MAC_TS - 1) / MAC_TS;
    const u32 n_items = n_groups * n_chunks;

    if (tid == 0) {
        for (int s = 0; s < MAC_MAX_STAGES; ++s) {
            mbar_init(&full[s], 1);                                // the producer's arrive.expect_tx
            mbar_init(&empty[s], MAC_CONSUMERS / 32);              // one arrival per consumer warp
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();

    if (tid >= MAC_CONSUMERS) {
        // ---------------- producer warp
        const u32 lane = tid - MAC_CONSUMERS;
        const u64 stream_policy = l2_evict_first_policy();
        u32 g = 0, ch = 0, slot = 0, phase = 0, k = 0;
        // one stage of the weight stream: a contiguous 16 KB block of the tile-major layout; when its tail
        // is padding (last group round or last term chunk) copy the valid part of every lane only
        const u32 word_lo = fmt == TILE_W64 ? 8u : 4u;                 // bytes per word of the stage's first part
        const unsigned char* prime_base = (const unsigned char*)pt + tile_prime_base(lay, i);
        const u32 hi_at = TILE_STAGE_WORDS * 4u;                       // TILE_W40: where the high bytes start
        auto issue_stage = [&]() {
            const u32 t0 = ch * MAC_TS, cnt = min((u32)MAC_TS, n_terms - t0);
            const u32 first = pj_begin + g * PL;
            const u32 lanes = min((u32)PL, pj_end - first);
            if constexpr (!COMPACT) {
                // the stage is one contiguous 16 KB block of the tile-major layout; when its tail is
                // padding (last group round or last term chunk) copy the valid part of every lane only
                const u64* stage = (const u64*)(prime_base + (((size_t)tile_x * lay.G + first / PL) * lay.C + ch) * (MAC_STAGE_WORDS * 8));
                u64* sdst = (u64*)ring + (size_t)slot * MAC_STAGE_WORDS;
                if (lane == 0) mbar_expect_tx(&full[slot], lanes * cnt * TN * 8);
                __syncwarp();
                if (lanes == PL && cnt == (u32)MAC_TS) {
                    if (lane == 0) bulk_g2s_stream(sdst, stage, MAC_STAGE_WORDS * 8, &full[slot], stream_policy);
                } else if (lane < lanes) {
                    bulk_g2s_stream(sdst + (size_t)lane * MAC_TS * TN, stage + (size_t)lane * MAC_TS * TN, cnt * TN * 8,
                                    &full[slot], stream_policy);
                }
            } else {
                const unsigned char* stage = prime_base + (((size_t)tile_x * lay.G + first / PL) * lay.C + ch) * stage_bytes;
                unsigned char* sdst = ring + (size_t)slot * MAC_SLOT_BYTES;
                const u32 bytes_per_word = fmt == TILE_W64 ? 8u : fmt == TILE_W40 ? 5u : 4u;
                if (lane == 0) mbar_expect_tx(&full[slot], lanes * cnt * TN * bytes_per_word);
                __syncwarp();
                if (lanes == PL && cnt == (u32)MAC_TS) {
                    if (lane == 0) bulk_g2s_stream(sdst, stage, stage_bytes, &full[slot], stream_policy);
                } else if (lane < lanes) {
                    // the valid part of every lane: cnt terms of TN words (and their high bytes)
                    const u32 at = lane * MAC_TS * TN;
                    bulk_g2s_stream(sdst + (size_t)at * word_lo, stage + (size_t)at * word_lo, cnt * TN * word_lo, &full[slot],
                                    stream_policy);
                    if (fmt == TILE_W40)
                        bulk_g2s_stream(sdst + hi_at + at, stage + hi_at + at, cnt * TN, &full[slot], stream_policy);
                }
            }
            if (++ch == n_chunks) { ch = 0; ++g; }
            if (++slot == n_stages) { slot = 0; phase ^= 1; }
            ++k;
        };
        // cached weights do not depend on the previous kernel: fill the ring before waiting for it
        const u32 early = early_weights ? min(n_items, n_stages) : 0u;
        while (k < early) issue_stage();
        asm volatile("griddepcontrol.wait;" ::: "memory");     // weights encoded on the fly come from the previous kernel
        while (k < n_items) {
            if (k >= n_stages) mbar_wait(&empty[slot], phase ^ 1, error_flag);   // consumers left this slot
            issue_stage();
        }
        return;
    }

    // ---------------- consumer warps
    const u32 c = tid & (TN - 1), l = tid >> LOG_TN;
    const u64 q = R.q[i];
    const u32 qneg32 = (u32)R.qneg[i];
    asm volatile("griddepcontrol.wait;" ::: "memory");
    {
        // X tile: [term][component] segments of TN words.  Its latency is exposed at the start of every block
        // (measured: 2 to 4 us of a 17 us block), so all of a thread's words are requested in one batch of
        // plain coalesced loads (one round trip; 32 bulk copies of 1 KB took 3.5 us and a separate split pass
        // 0.9 us), split into limbs on the way, each word exactly once, then made visible to all consumers
        const u64* xg = x + (size_t)i * N + n0 + c;
        const u32 n_seg = n_terms * 2;
        u32 e = l;
        for (; e + 15 * PL < n_seg; e += 16 * PL) {
            u64 v[16];
#pragma unroll
            for (int j = 0; j < 16; ++j) v[j] = __ldg(xg + (size_t)(e + j * PL) * r * N);
#pragma unroll
            for (int j = 0; j < 16; ++j) xs[(size_t)(e + j * PL) * TN + c] = KARA ? limb_split(v[j], KARA_L) : v[j];
        }
        for (; e + 3 * PL < n_seg; e += 4 * PL) {
            u64 v[4];
#pragma unroll
            for (int j = 0; j < 4; ++j) v[j] = __ldg(xg + (size_t)(e + j * PL) * r * N);
#pragma unroll
            for (int j = 0; j < 4; ++j) xs[(size_t)(e + j * PL) * TN + c] = KARA ? limb_split(v[j], KARA_L) : v[j];
        }
        for (; e < n_seg; e += PL) {
            const u64 v = __ldg(xg + (size_t)e * r * N);
            xs[(size_t)e * TN + c] = KARA ? limb_split(v, KARA_L) : v;
        }
        asm volatile("bar.sync 1, %0;" ::"n"(MAC_CONSUMERS) : "memory");
    }
    KaraAcc k0, k1;
    LimbAcc<false> a0, a1;
    u32 since_flush = 0, g = 0, ch = 0, slot = 0, phase = 0;
    for (u32 k = 0; k < n_items; ++k) {
        const u32 pj = pj_begin + g * PL + l;
        const u32 t0 = ch * MAC_TS, cnt = min((u32)MAC_TS, n_terms - t0);
        mbar_wait(&full[slot], phase, error_flag);
        if (pj < pj_end) {
            const u64* xt = xs + (size_t)t0 * 2 * TN + c;
            if constexpr (!COMPACT) {           // whole words; limbs already split when KARA
                const u64* ps = (const u64*)ring + (size_t)slot * MAC_STAGE_WORDS + (size_t)l * MAC_TS * TN + c;
                if (cnt == MAC_TS) {
#pragma unroll
                    for (int ts = 0; ts < MAC_TS; ++ts) {
                        const u64 w = ps[ts * TN];
                        if (KARA) {
                            const u32 w0 = (u32)w, w1 = (u32)(w >> 32), ws = w0 + w1;
                            k0.mac(w0, w1, ws, xt[(ts * 2) * TN]);
                            k1.mac(w0, w1, ws, xt[(ts * 2 + 1) * TN]);
                        } else {
                            a0.mac(w, xt[(ts * 2) * TN]);
                            a1.mac(w, xt[(ts * 2 + 1) * TN]);
                        }
                    }
                } else {
                    for (u32 ts = 0; ts < cnt; ++ts) {
                        const u64 w = ps[ts * TN];
                        if (KARA) {
                            const u32 w0 = (u32)w, w1 = (u32)(w >> 32), ws = w0 + w1;
                            k0.mac(w0, w1, ws, xt[(ts * 2) * TN]);
                            k1.mac(w0, w1, ws, xt[(ts * 2 + 1) * TN]);
                        } else {
                            a0.mac(w, xt[(ts * 2) * TN]);
                            a1.mac(w, xt[(ts * 2 + 1) * TN]);
                        }
                    }
                }
            } else {
                const unsigned char* sbase = ring + (size_t)slot * MAC_SLOT_BYTES;
                const u32 at = l * MAC_TS * TN + c;                    // index of this thread's first word of the stage
                // one streamed word times both components of its X word
                auto mac_word = [&](u64 w, u32 w0, u32 w1, u32 ts) {
                    if (KARA) {
                        const u32 ws = w0 + w1;
                        k0.mac(w0, w1, ws, xt[(ts * 2) * TN]);
                        k1.mac(w0, w1, ws, xt[(ts * 2 + 1) * TN]);
                    } else {
                        a0.mac(w, xt[(ts * 2) * TN]);
                        a1.mac(w, xt[(ts * 2 + 1) * TN]);
                    }
                };
                if (fmt == TILE_W64) {          // whole words; limbs already split when KARA
                    const u64* ps = (const u64*)sbase + at;
                    for (u32 ts = 0; ts < cnt; ++ts) {
                        const u64 w = ps[ts * TN];
                        mac_word(w, (u32)w, (u32)(w >> 32), ts);
                    }
                } else if (fmt == TILE_W40) {   // low 32 bits and high byte, limbs cut here
                    const u32* pl = (const u32*)sbase + at;
                    const unsigned char* ph = sbase + TILE_STAGE_WORDS * 4u + at;
                    if (cnt == MAC_TS) {
#pragma unroll
                        for (int ts = 0; ts < MAC_TS; ++ts) {
                            const u32 lo = pl[ts * TN], hi = ph[ts * TN];
                            mac_word(((u64)hi << 32) | lo, lo & ((1u << KARA_L) - 1), (lo >> KARA_L) | (hi << (32 - KARA_L)), ts);
                        }
                    } else {
                        for (u32 ts = 0; ts < cnt; ++ts) {
                            const u32 lo = pl[ts * TN], hi = ph[ts * TN];
                            mac_word(((u64)hi << 32) | lo, lo & ((1u << KARA_L) - 1), (lo >> KARA_L) | (hi << (32 - KARA_L)), ts);
                        }
                    }
                } else {                        // 32-bit words
                    const u32* pl = (const u32*)sbase + at;
                    for (u32 ts = 0; ts < cnt; ++ts) {
                        const u32 lo = pl[ts * TN];
                        mac_word((u64)lo, lo & ((1u << KARA_L) - 1), lo >> KARA_L, ts);
                    }
                }
            }
        }
        __syncwarp();
        if ((tid & 31) == 0) mbar_arrive(&empty[slot]);              // this warp is done with the slot
        if (pj < pj_end) {
            since_flush += cnt;
            if (ch + 1 == n_chunks) {
                u64* ap = a + ((size_t)pj * 2 * r + i) * N;
                u32 at0 = n0 + c;                                       // where component 0 goes (see MacScatter)
                if (sc.pinv && sc.pj0 + pj >= sc.n_out) at0 = __ldg(sc.pinv + (size_t)sc.key[(sc.pj0 + pj) / sc.n_out] * N + n0 + c);
                if (KARA) {
                    u64 H, L;
                    k0.value(KARA_L, H, L);
                    ap[at0] = redc_2x32(H, L, q, qneg32);
                    k1.value(KARA_L, H, L);
                    ap[(size_t)r * N + n0 + c] = redc_2x32(H, L, q, qneg32);
                    k0 = KaraAcc();
                    k1 = KaraAcc();
                } else {
                    ap[at0] = a0.reduce_mont(q, R.qneg[i]);
                    ap[(size_t)r * N + n0 + c] = a1.reduce_mont(q, R.qneg[i]);
                    a0.reset_to(0);
                    a1.reset_to(0);
                }
                since_flush = 0;
            } else if (!KARA && since_flush + MAC_TS > lazy_terms) {   // keep the partial sums inside their words
                a0.reset_to(a0.reduce(q, R.mu[i], R.c64[i], R.c64s[i]));
                a1.reset_to(a1.reduce(q, R.mu[i], R.c64[i], R.c64s[i]));
                since_flush = 1;
            }
        }
        if (++ch == n_chunks) { ch = 0; ++g; }
        if (++slot == n_stages) { slot = 0; phase ^= 1; }
    }
}

static int bits_of(u64 v) {
    int b = 0;
    while (v) { ++b; v >>= 1; }
    return b;
}

// tile width: the resident X tile (n_terms * 2 * TN words) must stay within 48 KB
static u32 mac_log_tn(u32 n_terms) {
    u32 log_tn = 8;
    while (log_tn > 4 && (size_t)n_terms * 2 * (1u << log_tn) * 8 > 48 * 1024) --log_tn;
    return log_tn;
}

TileLayout mac_tile_layout(const RingHost& ring, u32 n_pj, u32 n_terms, u32 n_primes) {
    TileLayout t;
    memset(&t, 0, sizeof(t));
    t.log_tn = mac_log_tn(n_terms);
    const u32 PL = 256u >> t.log_tn;
    t.n_terms = n_terms;
    t.n_pj = n_pj;
    t.G = (n_pj + PL - 1) / PL;
    t.C = (n_terms + TILE_TS - 1) / TILE_TS;
    t.ntiles = ring.dev.N >> t.log_tn;
    t.n_primes = n_primes ? n_primes : ring.dev.r;
    for (u32 i = 0; i < t.n_primes; ++i) {
        const u32 f = !ring.compact_cache || i >= ring.dev.r ? TILE_W64
                    : ring.q[i] < (1ull << 32) ? TILE_W32 : ring.q[i] < (1ull << 40) ? TILE_W40 : TILE_W64;
        t.fmt_bits |= f << (2 * i);
    }
    return t;
}

size_t mac_tile_bytes(const RingHost& ring, const TileLayout& t) { (void)ring; return tile_prime_base(t, t.n_primes); }

u32 mac_split_bits(const RingHost& ring) {
    u64 qmax = 0;
    for (u32 i = 0; i < ring.dev.r; ++i) qmax = ring.q[i] > qmax ? ring.q[i] : qmax;
    return bits_of(qmax) <= 50 ? KARA_L : 0;
}

template <bool KARA, int LOG_TN, bool COMPACT>
static cudaError_t launch_mac_t(const RingHost& ring, const u64* pt, const TileLayout& lay, const u64* x, u64* a,
                                u32 n_pj, u32 n_terms, u32 lazy, u32 early_weights, u32 prime0, u32 n_launch_primes,
                                int* error_flag, cudaStream_t stream, const MacScatter& sc) {
    constexpr u32 TN = 1u << LOG_TN, PL = MAC_CONSUMERS >> LOG_TN;
    const size_t smem = (size_t)MAC_RING_BYTES + (size_t)n_terms * 2 * TN * 8 + (2 * MAC_MAX_STAGES + 1) * 8;
    if (smem > 200 * 1024) return cudaErrorInvalidValue;
    const int ds = device_slot(ring);
    static bool attr_set[MAX_DEVICES] = {false};     // opt in once per device to the large dynamic shared-memory carve-out
    if (!attr_set[ds]) {
        cudaError_t e = cudaFuncSetAttribute(mac_kernel<KARA, LOG_TN, COMPACT>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             200 * 1024);
        if (e != cudaSuccess) return e;
        attr_set[ds] = true;
    }
    // slices over output groups: enough blocks to fill the machine several times over
    const u32 tiles = (ring.dev.N >> LOG_TN) * n_launch_primes;
    u32 slices = (148u * 2 * 6 + tiles - 1) / tiles;
    const u32 max_slices = (n_pj + PL - 1) / PL;
    if (slices > max_slices) slices = max_slices;
    if (slices < 1) slices = 1;
    u32 pj_per_block = (n_pj + slices - 1) / slices;
    pj_per_block = (pj_per_block + PL - 1) / PL * PL;
    slices = (n_pj + pj_per_block - 1) / pj_per_block;
    // blocks resident at once; when the units leave a thin last wave, cut those units into shorter blocks
    static int sm_counts[MAX_DEVICES] = {0}, per_sms[MAX_DEVICES] = {0};
    static size_t per_sm_smems[MAX_DEVICES] = {0};
    int &sm_count = sm_counts[ds], &per_sm = per_sms[ds];
    if (!sm_count) {
        cudaDeviceGetAttribute(&sm_count, cudaDevAttrMultiProcessorCount, ring.device);
        if (sm_count <= 0) sm_count = 148;
    }
    if (per_sm_smems[ds] != smem) {
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, mac_kernel<KARA, LOG_TN, COMPACT>, MAC_THREADS, smem) != cudaSuccess ||
            per_sm < 1) {
            cudaGetLastError();
            per_sm = 1;
        }
        per_sm_smems[ds] = smem;
    }
    const u32 slots = (u32)sm_count * (u32)per_sm;
    const u32 units = tiles * slices;
    const u32 rem = units % slots;
    u32 tail_split = 1;
    if (units > slots && rem && rem * 2 < slots) {
        tail_split = slots / rem;
        if (tail_split > pj_per_block / PL) tail_split = pj_per_block / PL;
        if (tail_split < 1) tail_split = 1;
    }
    const u32 n_whole = tail_split > 1 ? units - rem : units;
    dim3 grid(n_whole + (units - n_whole) * tail_split);
    return launch_dependent(ring, mac_kernel<KARA, LOG_TN, COMPACT>, grid, dim3(MAC_THREADS), smem, stream, ring.dev, pt, lay, x, a,
                            n_terms, n_pj, pj_per_block, lazy, early_weights, n_whole, tail_split, prime0, n_launch_primes,
                            error_flag, sc);
}

// One launch over primes prime0 .. prime0 + n_launch_primes - 1 of the layout; kara: Karatsuba on 25-bit limbs
// (those primes are all below 2^50), else whole words.
static cudaError_t launch_mac_primes(const RingHost& ring, const u64* pt, const TileLayout& lay, const u64* x, u64* a,
                                     u32 n_pj, u32 n_terms, bool weights_static, u32 prime0, u32 n_launch_primes, bool kara,
                                     int* error_flag, cudaStream_t stream, const MacScatter& sc) {
    ProfScope prof(ring.prof, CAT_MAC, stream);
    u64 qmax = 0;
    for (u32 i = prime0; i < prime0 + n_launch_primes; ++i) qmax = ring.q[i] > qmax ? ring.q[i] : qmax;
    const u32 log_tn = lay.log_tn;
    // terms a lazy sum can take: Karatsuba's middle sum grows by < 2^52 per term; the whole-word
    // path is limited by its high partial sum and by the total staying below q * 2^64
    u32 lazy = 128u;
    const u64 by_q = (~(u64)0) / qmax;
    if ((u64)lazy > by_q - 1) lazy = (u32)(by_q - 1);
    if (kara) {
        if (n_terms > 4000) return cudaErrorInvalidValue;
    } else if (lazy < (u32)MAC_TS) {
        return cudaErrorInvalidValue;
    }
    const u32 early = weights_static ? 1u : 0u;
    bool compact = false;
    for (u32 i = prime0; i < prime0 + n_launch_primes; ++i) compact = compact || tile_format(lay, i) != TILE_W64;
#define BF_MAC(S, L)                                                                                             \
    (compact ? launch_mac_t<S, L, true>(ring, pt, lay, x, a, n_pj, n_terms, lazy, early, prime0, n_launch_primes, error_flag, stream, sc) \
             : launch_mac_t<S, L, false>(ring, pt, lay, x, a, n_pj, n_terms, lazy, early, prime0, n_launch_primes, error_flag, stream, sc))
    if (kara) {
        switch (log_tn) {
            case 8: return BF_MAC(true, 8);
            case 7: return BF_MAC(true, 7);
            case 6: return BF_MAC(true, 6);
            case 5: return BF_MAC(true, 5);
            default: return BF_MAC(true, 4);
        }
    }
    switch (log_tn) {
        case 8: return BF_MAC(false, 8);
        case 7: return BF_MAC(false, 7);
        case 6: return BF_MAC(false, 6);
        case 5: return BF_MAC(false, 5);
        default: return BF_MAC(false, 4);
    }
#undef BF_MAC
}

cudaError_t launch_mac(const RingHost& ring, const u64* pt, const TileLayout& lay, const u64* x, u64* a, u32 n_pj,
                       u32 n_terms, bool weights_static, int* error_flag, cudaStream_t stream, cudaStream_t special_stream,
                       const MacScatter* scatter) {
    if (n_pj == 0) return cudaSuccess;
    if (lay.n_pj != n_pj || lay.n_terms != n_terms) return cudaErrorInvalidValue;
    const u32 r = ring.dev.r;
    const bool kara = mac_split_bits(ring) != 0;
    MacScatter sc;
    if (scatter) sc = *scatter;
    else memset(&sc, 0, sizeof(sc));
    cudaError_t e = launch_mac_primes(ring, pt, lay, x, a, n_pj, n_terms, weights_static, 0, r, kara, error_flag, stream, sc);
    if (e != cudaSuccess || lay.n_primes <= r) return e;
    // double hoisting: the residues modulo the 60-bit special prime, on whole words
    return launch_mac_primes(ring, pt, lay, x, a, n_pj, n_terms, weights_static, r, lay.n_primes - r, false, error_flag,
                             special_stream ? special_stream : stream, sc);
}

// ------------------------------------------------------------------------------------------------
// Key-switch inner product over the extended basis (Sec. 4.2 "key-switching primitives").
// The rotation keys are stored pre-permuted by their automorphism, so the product runs in the
// un-rotated index space with fully coalesced operands:
//   u'[rot][comp][m][n] = sum_j dig[dig(rot)][j][m][n] * key'[key(rot)][j][comp][m][n]
// and the automorphism is applied once, as a scatter, when the rotated ciphertext is assembled.
// Products accumulate as 32-bit limb partial sums (with carry counters where the 60-bit special prime needs
// them), one reduction per output word.
//
// A block owns one (run of rotations that share a key, modulus, tile of 128 coefficients): the baby rotations
// of several input ciphertexts by the same amount, or the giant rotations of several output blocks by the same
// amount.  Keys and digit sets are kept tile-major (see ks_tile_index): the key's 2r segments of the tile are one
// contiguous block, fetched once by one asynchronous bulk copy, and stay in shared memory, so that the key stream
// crosses HBM (and L2) once per run instead of once per rotation; the r digit segments of each rotation of the run
// (one contiguous block as well) follow through two buffers, the next rotation's copy in flight while the current
// one is multiplied.  The keys are resident in Montgomery form (times 2^64 mod q), so the sum
// of the r products ends in the two-round 32-bit Montgomery reduction: r * max digit < 2^64 keeps it below
// q * 2^64.  With double hoisting the block also finishes the rotated input (see launch_key_inner_product).
// grid: x = run, y = tile, z = modulus of the extended basis.
constexpr int KI_TILE = (int)KS_TILE;

// sum over the r digits of digit x key for both key components, reduced (the keys carry a factor 2^64); RC > 0: r == RC
template <bool SMALL, int RC>
__device__ __forceinline__ void ki_products(const u64* sdc, const u64* sk, u32 r, u32 tid, u64 q, u32 qneg32, u64& v0, u64& v1) {
    LimbAcc<SMALL> a0, a1;
    if constexpr (RC > 0) {
#pragma unroll
        for (int j = 0; j < RC; ++j) {
            const u64 d = sdc[j * KI_TILE + tid];
            a0.mac(d, sk[(j * 2) * KI_TILE + tid]);
            a1.mac(d, sk[(j * 2 + 1) * KI_TILE + tid]);
        }
    } else {
        for (u32 j = 0; j < r; ++j) {
            const u64 d = sdc[j * KI_TILE + tid];
            a0.mac(d, sk[(j * 2) * KI_TILE + tid]);
            a1.mac(d, sk[(j * 2 + 1) * KI_TILE + tid]);
        }
    }
    v0 = a0.reduce_mont32(q, qneg32);
    v1 = a1.reduce_mont32(q, qneg32);
}

__global__ void __launch_bounds__(KI_TILE, 8) key_inner_bulk_kernel(const RingDev R, const RotBatch rb,
                                                                   const u64* __restrict__ dig,
                                                                   const u64* __restrict__ keys, u64* __restrict__ u,
                                                                   u32 small_ok, int* __restrict__ error_flag,
                                                                   u64* __restrict__ xext, const u32* __restrict__ pinv) {
    extern __shared__ __align__(128) unsigned char ki_smem[];
    const u32 grp = blockIdx.x, m = blockIdx.z;
    const u32 first = rb.grp_first[grp], cnt = rb.grp_cnt[grp];      // this block's run of rotations: one key
    const u32 N = R.N, r = R.r, nb = r + 1;
    const u32 n0 = blockIdx.y * KI_TILE;
    u64* sk = (u64*)ki_smem;                        // [r][2][KI_TILE] key components
    u64* sd = sk + (size_t)2 * r * KI_TILE;         // [2][r][KI_TILE] digits of the current and the next rotation
    u64* kbar = sd + (size_t)2 * r * KI_TILE;
    u64* dbar = kbar + 1;                           // [2]
    const u32 tid = threadIdx.x;
    asm volatile("griddepcontrol.launch_dependents;");
    if (tid == 0) {
        mbar_init(kbar, 1);
        mbar_init(&dbar[0], 1);
        mbar_init(&dbar[1], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncthreads();
    // digit segments of rotation `first + it` into buffer it & 1
    auto fetch_digits = [&](u32 it) {
        u64* buf = sd + (size_t)(it & 1) * r * KI_TILE;
        if (tid == 0) mbar_expect_tx(&dbar[it & 1], r * KI_TILE * 8);
        __syncwarp();
        // the r digit segments of this set, modulus and tile are contiguous (see ks_tile_index): one copy
        if (tid == 0)
            bulk_g2s(buf, dig + ks_tile_base(N, nb, r, (u32)rb.dig[first + it], 0u, m) + (size_t)blockIdx.y * r * KI_TILE,
                     r * KI_TILE * 8, &dbar[it & 1]);
    };
    if (tid < 32) {
        if (tid == 0) mbar_expect_tx(kbar, 2 * r * KI_TILE * 8);
        __syncwarp();
        // the keys do not depend on the previous kernel: fetch them before waiting for it, the digits after
        const u64 stream_policy = l2_evict_first_policy();      // keys stream through; digits and outputs stay in L2
        if (tid == 0)       // the 2r key segments of this key, modulus and tile: one contiguous block
            bulk_g2s_stream(sk, keys + ks_tile_base(N, nb, 2 * r, (u32)rb.key[first], 0u, m) + (size_t)blockIdx.y * 2 * r * KI_TILE,
                            2 * r * KI_TILE * 8, kbar, stream_policy);
        asm volatile("griddepcontrol.wait;" ::: "memory");
        fetch_digits(0);
        if (cnt > 1) fetch_digits(1);
    } else {
        asm volatile("griddepcontrol.wait;" ::: "memory");
    }
    const u64 q = R.q[m];
    const u32 qneg32 = (u32)R.qneg[m];
    const size_t term_words = (size_t)2 * nb * N;
    // double hoisting: what the last step of a rotation reads from global memory (where the coefficient goes under the
    // rotation, and P*c0) is requested before the wait for the operands, so that it is not a second round trip
    u32 dest = 0;
    u64 pc0 = 0;
    if (pinv) dest = __ldg(&pinv[(size_t)rb.key[first] * N + n0 + tid]);    // (the same for every rotation of the run)
    if (xext) pc0 = xext[(size_t)rb.c0[first] * term_words + (size_t)m * N + n0 + tid];
    mbar_wait(kbar, 0, error_flag);
    for (u32 it = 0; it < cnt; ++it) {
        const u32 rot = first + it;
        const u64* sdc = sd + (size_t)(it & 1) * r * KI_TILE;
        u64 pc0_next = 0;
        if (xext && it + 1 < cnt) pc0_next = xext[(size_t)rb.c0[rot + 1] * term_words + (size_t)m * N + n0 + tid];
        mbar_wait(&dbar[it & 1], (it >> 1) & 1, error_flag);
        u64 v0, v1;
        if (m < r && small_ok) {
            // (digit counts of the shipped parameter sets with the loop unrolled: the launches where several rotations
            // share a key are bound by instruction issue)
            if (r == 7) ki_products<true, 7>(sdc, sk, r, tid, q, qneg32, v0, v1);
            else if (r == 9) ki_products<true, 9>(sdc, sk, r, tid, q, qneg32, v0, v1);
            else ki_products<true, 0>(sdc, sk, r, tid, q, qneg32, v0, v1);
        } else {
            if (r == 7) ki_products<false, 7>(sdc, sk, r, tid, q, qneg32, v0, v1);
            else if (r == 9) ki_products<false, 9>(sdc, sk, r, tid, q, qneg32, v0, v1);
            else ki_products<false, 0>(sdc, sk, r, tid, q, qneg32, v0, v1);
        }
        if (it + 2 < cnt) {                                  // the buffer is free once every thread has read it
            __syncthreads();
            if (tid < 32) fetch_digits(it + 2);
        }
        if (xext) {
            // double hoisting: no division by P; the rotated input in the extended basis is (P*c0 + u0, u1) moved
            // through the rotation's permutation; P*c0 (zero modulo P) was stored as the un-rotated term
            v0 = add_mod(v0, pc0, q);
            u64* xp = xext + (size_t)rb.out[rot] * term_words + (size_t)m * N + dest;
            xp[0] = v0;
            xp[(size_t)nb * N] = v1;
            pc0 = pc0_next;
        } else {
            // (pinv without xext: the plain result, stored through the rotation's permutation)
            u64* up = u + ((size_t)rot * 2 * nb + m) * N + (pinv ? dest : n0 + tid);
            up[0] = v0;
            up[(size_t)nb * N] = v1;
        }
    }
}

cudaError_t launch_key_inner_product(const RingHost& ring, const RotBatch& rb, const u64* dig, const u64* keys, u64* u,
                                     int* error_flag, cudaStream_t stream, u64* xext, const u32* pinv) {
    if (rb.n == 0) return cudaSuccess;
    u64 qmax = 0;
    for (u32 i = 0; i < ring.dev.r; ++i) qmax = ring.q[i] > qmax ? ring.q[i] : qmax;
    // without a carry counter the middle partial sum takes r <= 15 terms below 2^51 each
    const u32 small_ok = (qmax < ((u64)1 << 50)) ? 1u : 0u;
    ProfScope prof(ring.prof, CAT_KEY_INNER, stream);
    const u32 r = ring.dev.r;
    if (ring.prof) {
        const u64 key_bytes = (u64)r * 2 * (r + 1) * ring.dev.N * 8;
        u32 distinct = 0;
        for (int t = 0; t < rb.n; ++t) {
            bool seen = false;
            for (int k = 0; k < t && !seen; ++k) seen = rb.key[k] == rb.key[t];
            distinct += seen ? 0u : 1u;
        }
        ring.prof->key_bytes_distinct += distinct * key_bytes;
        ring.prof->key_bytes_per_rotation += (u64)rb.n * key_bytes;
    }
    const size_t smem = (size_t)4 * r * KI_TILE * 8 + 32;
    // runs of consecutive rotations with the same key: one block per run, tile and modulus
    RotBatch rbg = rb;
    rbg.n_groups = 0;
    for (int t = 0; t < rb.n; ++t) {
        if (t > 0 && rb.key[t] == rb.key[t - 1]) {
            rbg.grp_cnt[rbg.n_groups - 1]++;
        } else {
            rbg.grp_first[rbg.n_groups] = (unsigned char)t;
            rbg.grp_cnt[rbg.n_groups] = 1;
            rbg.n_groups++;
        }
    }
    static bool attr_set[MAX_DEVICES] = {false};     // per device: the attribute belongs to the device's copy of the kernel
    if (!attr_set[device_slot(ring)]) {
        cudaError_t e = cudaFuncSetAttribute(key_inner_bulk_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024);
        if (e != cudaSuccess) return e;
        attr_set[device_slot(ring)] = true;
    }
    dim3 grid(rbg.n_groups, ring.dev.N / KI_TILE, r + 1);
    return launch_dependent(ring, key_inner_bulk_kernel, grid, dim3(KI_TILE), smem, stream, ring.dev, rbg, dig, keys, u,
                            small_ok, error_flag, xext, pinv);
}

// ------------------------------------------------------------------------------------------------
// Rescale (Sec. 2.1): drop the last prime q_L of a level-`level` ciphertext in coefficient form,
//   c'_i = (c_i - centred(c_L)) * q_L^{-1} mod q_i.
// Every address a thread touches is congruent to its coefficient index modulo N, and it reads all
// residues of that coefficient before writing, so one ciphertext can be rescaled in place even
// though the output is packed more tightly ([2][level-1][N]).

// `in` and `out` may alias, hence no __restrict__.  When they do and several ciphertexts are
// rescaled, the launch uses one thread per coefficient that walks the ciphertexts in order
// (n_seq > 1): the packed output of ciphertext t never reaches the input of ciphertext t+1.
__global__ void __launch_bounds__(256) rescale_kernel(const RingDev R, const RescaleConsts rc, const u64* in, u64* out,
                                                      u32 level, u32 n_seq) {
    grid_dependency_enter();
    const u32 N = R.N;
    const u32 n = blockIdx.x * blockDim.x + threadIdx.x;
    const u64 qL = R.q[level - 1];
  for (u32 ct = blockIdx.y; ct < blockIdx.y + n_seq; ++ct) {
    const u64* ip = in + (size_t)ct * 2 * level * N + n;
    u64* op = out + (size_t)ct * 2 * (level - 1) * N + n;
    // In place the packed output of residue (comp, i) lands where residue (comp, i) (component 0) or (comp, i - 1)
    // (component 1) was read, and the dropped residues are read before anything of their component is written: so
    // each residue is read, then its slot (or an earlier one) written, in order, with nothing held back.
#pragma unroll
    for (int comp = 0; comp < 2; ++comp) {
        const u64 t = ip[((size_t)comp * level + (level - 1)) * N];
        const bool high = t > (qL - 1) / 2;
        for (u32 i = 0; i + 1 < level; ++i) {
            const u64 q = R.q[i];
            u64 tq = barrett64(t, q, R.mu[i]);
            if (high) tq = sub_mod(tq, rc.qlmod[i], q);
            const u64 c = ip[((size_t)comp * level + i) * N];
            op[((size_t)comp * (level - 1) + i) * N] = mul_shoup(sub_mod(c, tq, q), rc.inv[i], rc.invs[i], q);
        }
    }
  }
}

// Out-of-place form: one thread per output word (coefficient, ciphertext, component, prime), so the launch is
// wide enough to hide its loads; the dropped prime's residue is read once per output prime (an L2 hit).
// grid: x = coefficients / 256, y = ciphertext, z = component * (level - 1) + prime.
__global__ void __launch_bounds__(256) rescale_wide_kernel(const RingDev R, const RescaleConsts rc, const u64* __restrict__ in,
                                                           u64* __restrict__ out, u32 level) {
    grid_dependency_enter();
    const u32 N = R.N;
    const u32 n = blockIdx.x * blockDim.x + threadIdx.x;
    const u32 ct = blockIdx.y, comp = blockIdx.z / (level - 1), i = blockIdx.z % (level - 1);
    const u64* ip = in + ((size_t)ct * 2 + comp) * level * N + n;
    const u64 qL = R.q[level - 1], q = R.q[i];
    const u64 t = ip[(size_t)(level - 1) * N];
    const u64 c = ip[(size_t)i * N];
    u64 tq = barrett64(t, q, R.mu[i]);
    if (t > (qL - 1) / 2) tq = sub_mod(tq, rc.qlmod[i], q);
    out[(((size_t)ct * 2 + comp) * (level - 1) + i) * N + n] = mul_shoup(sub_mod(c, tq, q), rc.inv[i], rc.invs[i], q);
}

cudaError_t launch_rescale(const RingHost& ring, const u64* in, u64* out, u32 n_ct, u32 level, const u64* inv,
                           const u64* invs, const u64* qlmod, cudaStream_t stream) {
    if (n_ct == 0) return cudaSuccess;
    RescaleConsts rc;
    memset(&rc, 0, sizeof(rc));
    for (u32 i = 0; i + 1 < level; ++i) { rc.inv[i] = inv[i]; rc.invs[i] = invs[i]; rc.qlmod[i] = qlmod[i]; }
    ProfScope prof(ring.prof, CAT_RESCALE, stream);
    if (in == out && n_ct > 1) {
        dim3 grid(ring.dev.N / 64, 1);
        launch_dependent(ring, rescale_kernel, grid, dim3(64), 0, stream, ring.dev, rc, in, out, level, n_ct);
    } else if (in == out || n_ct > 65535) {
        dim3 grid(ring.dev.N / 256, n_ct);
        launch_dependent(ring, rescale_kernel, grid, dim3(256), 0, stream, ring.dev, rc, in, out, level, 1u);
    } else {
        dim3 grid(ring.dev.N / 256, n_ct, 2 * (level - 1));
        launch_dependent(ring, rescale_wide_kernel, grid, dim3(256), 0, stream, ring.dev, rc, in, out, level);
    }
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------------------
// Width changes of the rounded integer coefficients (the coefficient form of cached weights).
__global__ void __launch_bounds__(256) widen_i32_kernel(const int* __restrict__ src, i64* __restrict__ dst, size_t count) {
    grid_dependency_enter();
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (size_t)gridDim.x * blockDim.x)
        dst[i] = (i64)src[i];
}
__global__ void __launch_bounds__(256) narrow_i64_kernel(const i64* __restrict__ src, int* __restrict__ dst, size_t count,
                                                         int* __restrict__ overflow) {
    grid_dependency_enter();
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < count; i += (size_t)gridDim.x * blockDim.x) {
        const i64 v = src[i];
        if (v != (i64)(int)v) atomicExch(overflow, 1);
        dst[i] = (int)v;
    }
}
cudaError_t launch_widen_i32(const RingHost& ring, const int* src, i64* dst, size_t count, cudaStream_t stream) {
    if (!count) return cudaSuccess;
    ProfScope prof(ring.prof, CAT_POINTWISE, stream);
    const u32 blocks = (u32)((count + 1023) / 1024 < 148 * 16 ? (count + 1023) / 1024 : 148 * 16);
    return launch_dependent(ring, widen_i32_kernel, dim3(blocks), dim3(256), 0, stream, src, dst, count);
}
cudaError_t launch_narrow_i64(const RingHost& ring, const i64* src, int* dst, size_t count, int* overflow_flag,
                              cudaStream_t stream) {
    if (!count) return cudaSuccess;
    ProfScope prof(ring.prof, CAT_POINTWISE, stream);
    const u32 blocks = (u32)((count + 1023) / 1024 < 148 * 16 ? (count + 1023) / 1024 : 148 * 16);
    return launch_dependent(ring, narrow_i64_kernel, dim3(blocks), dim3(256), 0, stream, src, dst, count, overflow_flag);
}

// ------------------------------------------------------------------------------------------------
// Throughput probe for the 32x32+64-bit integer multiply-add the modular arithmetic is made of:
// every thread runs 8 independent mad.wide.u32 chains.  Gives the measured denominator for the
// integer-bound kernels (NTT, key switch).
__global__ void __launch_bounds__(256) imad_probe_kernel(u64* __restrict__ sink, u32 iters) {
    const u32 b = threadIdx.x * 2654435761u + blockIdx.x * 40503u + 12345u;
    u64 c[8];
    u32 d[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) { c[k] = b + k; d[k] = b * 3 + k; }
    for (u32 i = 0; i < iters; ++i) {
#pragma unroll
        for (int u = 0; u < 8; ++u) {
#pragma unroll
            for (int k = 0; k < 8; ++k) asm volatile("mad.wide.u32 %0, %1, %2, %0;" : "+l"(c[k]) : "r"(b), "r"(d[(k + 1) & 7]));
        }
    }
    u64 v = 0;
#pragma unroll
    for (int k = 0; k < 8; ++k) v ^= c[k];
    if (v == 0x1234567ull) sink[0] = v;      // practically never true; keeps the chains alive
}

cudaError_t launch_imad_probe(u64* sink, u32 blocks, u32 iters, cudaStream_t stream) {
    imad_probe_kernel<<<blocks, 256, 0, stream>>>(sink, iters);
    return cudaGetLastError();
}

// The same probe for the fp64 fused multiply-add that the transforms of the ciphertext primes are made of:
// every thread runs 8 independent fma.rn.f64 chains.
__global__ void __launch_bounds__(256) fma64_probe_kernel(u64* __restrict__ sink, u32 iters) {
    const double b = 1.0 + (double)(threadIdx.x + blockIdx.x * 256u) * 1e-9;
    double c[8], d[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) { c[k] = b + k; d[k] = 1e-3 * (k + 1); }
    for (u32 i = 0; i < iters; ++i) {
#pragma unroll
        for (int u = 0; u < 8; ++u) {
#pragma unroll
            for (int k = 0; k < 8; ++k) asm volatile("fma.rn.f64 %0, %1, %0, %2;" : "+d"(c[k]) : "d"(b), "d"(d[(k + 1) & 7]));
        }
    }
    double v = 0.0;
#pragma unroll
    for (int k = 0; k < 8; ++k) v += c[k];
    if (v == 0.1234567) sink[0] = (u64)__double_as_longlong(v);      // practically never true; keeps the chains alive
}

cudaError_t launch_fma64_probe(u64* sink, u32 blocks, u32 iters, cudaStream_t stream) {
    fma64_probe_kernel<<<blocks, 256, 0, stream>>>(sink, iters);
    return cudaGetLastError();
}

}  // namespace bf
