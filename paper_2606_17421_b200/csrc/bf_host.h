// Host-side structures and kernel launchers shared by the translation units of libbifrost.
#pragma once
#include <cstddef>
#include <cstdint>
#include <map>
#include <vector>

#include "bf_common.cuh"

namespace bf {

struct NttGeometry {
    int log_r, log_c;                 // N = 2^log_r rows x 2^log_c columns
    int strided_lanes, strided_threads;
    int contig_lanes, contig_threads, contig_pad;
};

// Kernel categories for launch counting and optional per-launch event timing.
enum KernelCat : int {
    CAT_NTT_FWD_STRIDED = 0, CAT_NTT_FWD_CONTIG, CAT_NTT_INV_CONTIG, CAT_NTT_INV_STRIDED,
    CAT_KEY_INNER, CAT_MAC, CAT_RESCALE,
    CAT_ENCODE_FFT_A, CAT_ENCODE_FFT_B, CAT_POINTWISE, CAT_DIVIDE, CAT_COUNT
};

struct Profiler {
    bool timing = false;
    uint64_t launches[CAT_COUNT] = {0};
    // key-switch inner products: bytes of rotation keys counted once per distinct key of a launch (what must come
    // from HBM) and once per rotation (what the launch reads, L2 hits included)
    uint64_t key_bytes_distinct = 0, key_bytes_per_rotation = 0;
    struct Rec { int cat; cudaEvent_t a, b; };
    std::vector<Rec> recs;            // event pairs recorded since the last collection
    std::vector<cudaEvent_t> pool;    // idle events
    bool span_open = false;           // a ProfSpan is timing the launches inside it as one
    cudaEvent_t get();
};

// Counts a launch and, when timing is on, brackets it with two events on the launch stream.
struct ProfScope {
    Profiler* p; int cat; cudaStream_t s; cudaEvent_t a = nullptr;
    ProfScope(Profiler* prof, int c, cudaStream_t st);
    ~ProfScope();
};

// Times a group of launches that run side by side as one span on stream st (from everything before the group to
// everything after its join); the launches inside are still counted by their own ProfScope, but not timed singly.
struct ProfSpan {
    Profiler* p; int cat; cudaStream_t s; cudaEvent_t a = nullptr;
    ProfSpan(Profiler* prof, int c, cudaStream_t st);
    ~ProfSpan();
};

struct RingHost {
    RingDev dev;
    NttGeometry geom;
    std::vector<u64> q;               // q_0..q_L, then P
    Profiler* prof = nullptr;
    bool dependent_launch = true;     // launch the kernels of a call with programmatic stream serialisation
    bool compact_cache = false;       // encode plaintexts in the narrowest word format each prime allows
    int device = 0;                   // the CUDA device of the context (kernel attributes are set once per device)
};
constexpr int MAX_DEVICES = 64;
inline int device_slot(const RingHost& ring) { return ring.device >= 0 && ring.device < MAX_DEVICES ? ring.device : 0; }

// Launch with programmatic stream serialisation: the grid may be scheduled while the previous kernel
// of the stream drains; every kernel launched this way calls grid_dependency_enter() before it touches
// global memory, which waits until that previous kernel has completed and its writes are visible.
template <typename... KArgs, typename... Args>
static inline cudaError_t launch_dependent(const RingHost& ring, void (*kernel)(KArgs...), dim3 grid, dim3 block,
                                           size_t smem, cudaStream_t stream, Args&&... args) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = ring.dependent_launch ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

// ---- ntt.cu
NttGeometry ntt_geometry(u32 logN);
cudaError_t ntt_forward(const RingHost& ring, const PolyBatch& B, u32 n_outer, int load, cudaStream_t stream);
cudaError_t ntt_inverse(const RingHost& ring, const PolyBatch& B, u32 n_outer, cudaStream_t stream);
// Forward transform of the centred lifts of P-residues with the ModDown epilogue fused into its last store.
cudaError_t ntt_forward_moddown(const RingHost& ring, const PolyBatch& B, u32 n_outer, const RotBatch& rb,
                                const ModDownEpilogue& epi, cudaStream_t stream);
// Inverse transform of the P-residues summed over the giant rotations of each output (per-output form of epi).
cudaError_t ntt_inverse_gathersum(const RingHost& ring, const PolyBatch& B, u32 n_outer, const RotBatch& rb,
                                  const ModDownEpilogue& epi, cudaStream_t stream);
// ct[p][comp][i] = (ct[p][comp][i] - sum of the centred P-residues T[p][.]) * P^{-1}: the division that ends the output
// assembly in the extended basis (ModDownEpilogue::assemble names the n_t polynomials of T per output)
// rc, low non-null: the rescale from r primes follows in the same kernel; the result goes to low ([n_out][2][r-1][N])
cudaError_t finish_division(const RingHost& ring, u64* ct, long long ct_stride, const u64* T, u32 n_t, u32 n_out,
                            cudaStream_t stream, const RescaleConsts* rc = nullptr, u64* low = nullptr);
cudaError_t ntt_forward_split(const RingHost& ring, const PolyBatch& B, u32 n_outer, int load, u64* final_dst,
                              const u32* scatter, u32 scatter_div, cudaStream_t stream);

// ---- kernels.cu : element-wise and streaming kernels of the linear layer
// out[t] = a[t] * b[t] pointwise, polynomial t modulo basis prime mod0 + t % n_m
cudaError_t launch_pointwise_mul(const RingHost& ring, const u64* a, const u64* b, u64* out, u32 n_polys, u32 n_m,
                                 u32 mod0, cudaStream_t stream);
// u'[rot][comp][m][n] = sum_j dig[dig(rot)][j][m][n] * key'[key(rot)][j][comp][m][n]  (keys pre-permuted)
// pinv non-null, xext null: u'[rot][comp][m] is stored through the rotation's permutation, at pinv[rb.key[rot]][n].
// xext non-null (double hoisting): rotation `rot` is not stored to u but finished as a rotated input in the
// extended basis: xext[rb.out[rot]][comp][m][pinv[rb.key[rot]][n]] = u'[comp][m][n] + (comp == 0 ?
// xext[rb.c0[rot]][0][m][n] : 0), terms of [2][r+1][N] words (term rb.c0[rot] holds P times the un-rotated input).
cudaError_t launch_key_inner_product(const RingHost& ring, const RotBatch& rb, const u64* dig, const u64* keys, u64* u,
                                     int* error_flag, cudaStream_t stream, u64* xext = nullptr, const u32* pinv = nullptr);
u32 mac_split_bits(const RingHost& ring);   // limb width of the cached plaintext format (0 = whole words)
// layout of n_pj groups of n_terms diagonals held in n_primes primes (0 = the r ciphertext primes)
TileLayout mac_tile_layout(const RingHost& ring, u32 n_pj, u32 n_terms, u32 n_primes = 0);
size_t mac_tile_bytes(const RingHost& ring, const TileLayout& t);           // bytes that layout occupies
// x: [n_terms][2][lay.n_primes][N], a: [n_pj][2][lay.n_primes][N]; every prime of the layout is processed (the special
// prime, when present, by a launch of its own on whole words)
// special_stream non-null: the launch for the special prime goes there (the caller has ordered that stream after
// everything the launch reads and joins it afterwards), beside the launch for the ciphertext primes on `stream`
cudaError_t launch_mac(const RingHost& ring, const u64* pt, const TileLayout& lay, const u64* x, u64* a, u32 n_pj,
                       u32 n_terms, bool weights_static, int* error_flag, cudaStream_t stream,
                       cudaStream_t special_stream = nullptr, const MacScatter* scatter = nullptr);
cudaError_t launch_rescale(const RingHost& ring, const u64* in, u64* out, u32 n_ct, u32 level, const u64* inv,
                           const u64* invs, const u64* qlmod, cudaStream_t stream);

// 32-bit <-> 64-bit signed coefficients (the coefficient form of cached weights); narrowing sets *overflow_flag when a
// value does not fit
cudaError_t launch_widen_i32(const RingHost& ring, const int* src, i64* dst, size_t count, cudaStream_t stream);
cudaError_t launch_narrow_i64(const RingHost& ring, const i64* src, int* dst, size_t count, int* overflow_flag,
                              cudaStream_t stream);
cudaError_t launch_imad_probe(u64* sink, u32 blocks, u32 iters, cudaStream_t stream);   // 64 mad.wide per iteration and thread
cudaError_t launch_fma64_probe(u64* sink, u32 blocks, u32 iters, cudaStream_t stream);  // 64 fma.rn.f64 per iteration and thread

// ---- encode.cu : canonical-embedding encoder (fp64) for weight diagonals
struct EncodeTables {
    const u32* slot_of_pos;           // [n] slot index whose value sits at FFT input position a
    const double2* T;                 // [n/2] (cos, -sin)(2 pi t / n)
    const double2* Z;                 // [n]   (cos, -sin)(pi k / N)
    double scale_over_n;
};
struct DiagBatch {                    // diagonals d0 .. d0+count-1 in [j][p][q][k] order
    const float* W;
    u32 d_out, d_in, n_in, n_out, D, tau, b, g;
    u32 d0, count;
    u32 complex_pack;                 // two row blocks per plaintext: block 2p in the real parts, 2p+1 in the imaginary
};
cudaError_t launch_encode(const RingHost& ring, const EncodeTables& tab, const DiagBatch& db, double2* fft_scratch,
                          i64* coeff_out, int* overflow_flag, cudaStream_t stream);

}  // namespace bf
