/*
 * libbifrost: the accelerator-side CKKS linear layer of a hybrid TEE-FHE serving stack, for one
 * NVIDIA B200 (sm_100a).  The trusted side (key generation, encryption, decryption, non-linear
 * operators) is not here: callers hand in ciphertexts and rotation keys as plain arrays.
 *
 * Conventions shared by all entry points
 *   - Every function returns BF_OK (0) or a negative BF_ERR_* code; nothing throws or aborts.
 *     bf_strerror() names a code; bf_last_cuda_error() gives the CUDA message behind BF_ERR_CUDA.
 *   - A context is bound to the CUDA device that was current at bf_ctx_create() and to one stream.
 *     Calls only enqueue work on that stream (exceptions are stated); the caller synchronises.
 *     Calls on one context must not overlap on the host.
 *   - r = number of ciphertext primes q_0..q_{r-1}; P = special prime; N = ring degree.
 *   - Ciphertext layout at the boundary: uint64 [2][r][N] = component (c0, c1), prime, coefficient,
 *     in the COEFFICIENT domain with every residue in [0, q_i).  Arrays of ciphertexts are stored
 *     back to back.  Decryption is c0 + c1*s.
 *   - Rotation-key layout at the boundary: uint64 [r][2][r+1][N] = digit j, component (b, a),
 *     prime of the extended basis {q_0..q_{r-1}, P}, coefficient; coefficient domain.
 *   - "device" pointers are CUDA device memory owned by the caller; the library keeps no reference
 *     to them after the enqueued work has run.  "host" pointers are ordinary host memory read or
 *     written before the call returns, unless stated.
 */
#ifndef BIFROST_H
#define BIFROST_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
    BF_OK = 0,
    BF_ERR_INVALID_ARG = -1,   /* null pointer, zero size, N not a power of two in [2^10, 2^16], ... */
    BF_ERR_BAD_PRIME = -2,     /* not prime, not 1 mod 2N, duplicate, or not below 2^60 */
    BF_ERR_SHAPE = -3,         /* n_in / n_out do not match d_in / d_out and the plan, or plan inconsistent */
    BF_ERR_LEVEL = -4,         /* level outside [2, r] */
    BF_ERR_MISSING_KEY = -5,   /* the plan needs a rotation whose key was not loaded */
    BF_ERR_OOM = -6,           /* encoded weights exceed the cache budget, or device memory is exhausted */
    BF_ERR_CUDA = -7,          /* a CUDA call failed; see bf_last_cuda_error() */
    BF_ERR_RANGE = -8,         /* an encoded coefficient does not fit 2^62 (scale too large for the data) */
    BF_ERR_TOO_LARGE = -9,     /* more work than the fixed scratch of an allocation-free entry point holds */
    BF_ERR_TIMEOUT = -10       /* a device-side wait on an asynchronous copy hit its poll limit */
};

typedef struct bf_ctx bf_ctx;          /* ring tables, rotation keys, scratch memory */
typedef struct bf_weights bf_weights;  /* device-resident encoded diagonals of one projection */

/* Tiling of a projection (the paper leaves packing open beyond "weight diagonals" kept as
 * baby-step/giant-step objects, Sec. 4.2):  the weight matrix is cut into tile_D x tile_D tiles;
 * slot s = (rho*tile_D + kappa)*tau + c of an input ciphertext holds x[(kappa + c*M) mod tile_D]
 * of its chunk, M = tile_D/tau generalised diagonals per tile, split as M = bsgs_b * bsgs_g.
 * All four are powers of two and tile_D*tau <= N/2.
 * flags select variants of the evaluation that change the output residues (each is mirrored by a mode
 * of the CPU reference the tests compare with); 0 = the plain evaluation:
 *   BF_PLAN_COMPLEX_PACK       two output row blocks share one plaintext, block 2P in the real parts
 *       of the slots and block 2P+1 in the imaginary parts (the input ciphertexts stay real), so
 *       that output ciphertext P decrypts to (rows of block 2P) + i (rows of block 2P+1): half the
 *       diagonals, half the encoded-weight bytes (the memory wall of Sec. 6.1), half the giant
 *       rotations.  n_out = ceil(ceil(d_out / tile_D) / 2) output ciphertexts.
 *   BF_PLAN_MODDOWN_PER_OUTPUT the key-switch results of an output's giant rotations are summed in
 *       the extended basis {q_i, P} and divided by P once per output ciphertext and component
 *       instead of once per rotation (Sec. 4.2 leaves the key-switching primitive open).  Needs
 *       bsgs_g - 1 <= 64.
 *   BF_PLAN_DOUBLE_HOIST       the baby-step rotations are not divided by P: they stay in the extended
 *       basis as (P*phi_k(c0) + u0, u1), the encoded weights are held modulo P as well (one more
 *       60-bit residue per coefficient: (r+1)/r of the cache), the products are summed over the
 *       extended basis, and each inner sum is divided by P once, i.e. n_out * bsgs_g divisions per
 *       call instead of n_in * (bsgs_b - 1). */
enum {
    BF_PLAN_COMPLEX_PACK = 1,
    BF_PLAN_MODDOWN_PER_OUTPUT = 2,
    BF_PLAN_DOUBLE_HOIST = 4
};
typedef struct {
    uint32_t tile_D, tau, bsgs_b, bsgs_g;
    uint32_t flags;                        /* BF_PLAN_* bits */
} bf_plan;

/* Create a context (Sec. 4.2: one CKKS context per projection shape, with its modulus chain and
 * BSGS rotation parameters).
 *   primes       host, n_ct_primes + 1 values: q_0..q_L then the special prime P
 *   scale        Delta used when encoding weights (a power of two keeps the scaling exact)
 *   cuda_stream  a cudaStream_t (0 = default stream)
 * Allocates device tables; synchronises the device once.  Errors: INVALID_ARG, BAD_PRIME, SHAPE,
 * CUDA. */
int bf_ctx_create(bf_ctx** out, uint32_t N, const uint64_t* primes, uint32_t n_ct_primes, double scale,
                  const bf_plan* plan, void* cuda_stream);

/* Frees everything the context owns, including weights not yet freed.  Synchronises. */
void bf_ctx_destroy(bf_ctx* ctx);

/* Load rotation (Galois) keys, replacing any loaded before (Sec. 4.1 "rotation material").
 *   rot_steps  host, n_keys left-rotation amounts; key t switches from s(X^(5^rot_steps[t])) to s
 *   keys       device, [n_keys][r][2][r+1][N] in the boundary layout
 * The keys are transformed into the library's evaluation layout in its own memory.  Required
 * amounts for a plan: k*tau for k = 1..b-1 and j*b*tau for j = 1..g-1.  Synchronises. */
int bf_load_eval_keys(bf_ctx* ctx, const uint32_t* rot_steps, uint32_t n_keys, const uint64_t* keys);

/* Upper bound in bytes on the encoded weights kept resident by this context (Sec. 4.2: persistent
 * cache vs fallback-encode modes).  0 = unlimited (default). */
int bf_set_cache_budget(bf_ctx* ctx, uint64_t bytes);
uint64_t bf_cache_bytes_used(const bf_ctx* ctx);

/* Bytes bf_encode_weights would keep resident for a d_out x d_in projection under the plan. */
uint64_t bf_weights_bytes(const bf_ctx* ctx, uint32_t d_out, uint32_t d_in);

/* EncodeWeights (Alg. 3, offline phase; Sec. 4.2): encode every generalised diagonal of
 * W[d_out][d_in] (device, fp32, row-major) at scale Delta, reduce per prime and transform, keeping
 * the result in device memory owned by the returned handle.  Returns BF_ERR_OOM without
 * allocating when the cache budget would be exceeded: the caller then passes W itself to bf_linear.
 * Synchronises. */
int bf_encode_weights(bf_ctx* ctx, const float* W, uint32_t d_out, uint32_t d_in, bf_weights** out);
/* The same with a baby/giant split of its own for this projection (Sec. 4.2 "BSGS matrix-vector multiply": the
 * split trades hoisted baby rotations of the inputs against full key switches of the outputs, and the best trade
 * depends on n_in and n_out).  bsgs_b * bsgs_g = tile_D / tau as for the plan, both powers of two,
 * bsgs_b - 1 <= 64 (and bsgs_g - 1 <= 64 with BF_PLAN_MODDOWN_PER_OUTPUT), else BF_ERR_SHAPE.  bf_linear with this handle
 * needs the rotation keys of this split: k*tau for k < bsgs_b and j*bsgs_b*tau for j < bsgs_g. */
int bf_encode_weights_split(bf_ctx* ctx, const float* W, uint32_t d_out, uint32_t d_in, uint32_t bsgs_b, uint32_t bsgs_g,
                            bf_weights** out);
void bf_weights_free(bf_ctx* ctx, bf_weights* w);

/* FHE_Linear (Alg. 3, decode loop; Sec. 4.2 "BSGS matrix-vector multiply"):
 *     ct_out[p] = sum_{j<g} rot( sum_q sum_{k<b} Pt[p][q][j][k] * rot(ct_in[q], k*tau), j*b*tau )
 * for p < n_out = ceil(d_out/tile_D) (half of that, rounded up, with BF_PLAN_COMPLEX_PACK),
 * q < n_in = ceil(d_in/tile_D).  Rotations are automorphisms
 * followed by a key switch with one special prime (one prime per digit), each with its own
 * division by P.
 *   ct_in       device, n_in ciphertexts at full level, boundary layout
 *   pt_weights  handle from bf_encode_weights for this (d_out, d_in) (b and g are then the handle's); or NULL, in which case
 *   W_raw       device fp32 [d_out][d_in] is encoded on the fly (fallback path)
 *   ct_out      device, n_out ciphertexts, full level, scale = scale(ct_in) * Delta; must not
 *               overlap ct_in
 * Slot (0, kappa, c) of ct_out[p] decrypts to the partial dot product of row p*tile_D + kappa over
 * column class c (with BF_PLAN_COMPLEX_PACK: rows 2p*tile_D + kappa in the real part and
 * (2p+1)*tile_D + kappa in the imaginary part); the caller adds the tau partial sums.  Asynchronous on the context's stream,
 * except that scratch memory may be grown (which synchronises) the first time a shape is seen.
 * Errors: INVALID_ARG, SHAPE, MISSING_KEY, OOM, RANGE (fallback path only), CUDA. */
int bf_linear(bf_ctx* ctx, const uint64_t* ct_in, uint32_t n_in, const bf_weights* pt_weights,
              const float* W_raw, uint32_t d_out, uint32_t d_in, uint64_t* ct_out, uint32_t n_out);

/* bf_linear followed by bf_rescale from the full level (Sec. 2.1 rescaling; the decode loop of Alg. 3 rescales every
 * product), as one call: ct_low receives n_out ciphertexts of r-1 primes, boundary layout [2][r-1][N], the same residues
 * as the two calls in turn.  Where the plan ends the product in an element-wise kernel (double hoisting with one
 * division per output) the rescale happens inside it; the full-level result then never reaches memory the caller sees.
 * scale_inout (host, may be NULL) is divided by the dropped prime.  Same errors as bf_linear; BF_ERR_LEVEL if r < 2. */
int bf_linear_rescaled(bf_ctx* ctx, const uint64_t* ct_in, uint32_t n_in, const bf_weights* pt_weights,
                       const float* W_raw, uint32_t d_out, uint32_t d_in, uint64_t* ct_low, uint32_t n_out,
                       double* scale_inout);

/* Cache compression (Sec. 6.1 names the encoded-weight cache as the memory wall).  With
 * bf_set_compact_cache(ctx, 1) every weight encoded afterwards, cached or on the fallback path, is
 * held in the narrowest word format its prime allows: 4 bytes per word for primes below 2^32, 5
 * (low 32 bits and high bytes stored apart) below 2^40, 8 otherwise, instead of 8 throughout: with a
 * 50-bit and six 40-bit primes 38 of 56 bytes, i.e. 68 % of the resident size and of the
 * multiply-accumulate's HBM stream.  Results are identical; handles of both kinds can be used side by
 * side.  Default: off (the multiply-accumulate is no faster for it on B200, see the design notes;
 * the gain is capacity).  bf_weights_bytes reports sizes for the current setting. */
int bf_set_compact_cache(bf_ctx* ctx, int on);

/* Coefficient form of the cache (the other answer to the memory wall of Sec. 6.1): with
 * bf_set_coefficient_cache(ctx, 64 or 32) every weight encoded afterwards is kept as the rounded
 * integer coefficients of its diagonals, one 64- or 32-bit word per coefficient whatever the number
 * of primes (1/r or 1/(2r) of the transform-domain cache), and bf_linear reduces them per prime and
 * transforms them on every call: the fallback path without its encoder.  Results are identical.
 * 32 bits hold |coefficient| < 2^31: bf_encode_weights returns BF_ERR_RANGE when the weights and the
 * scale give more.  bits = 0 (default) switches back to transform-domain residues; handles of all
 * kinds can be used side by side.  bf_weights_bytes reports sizes for the current setting. */
int bf_set_coefficient_cache(bf_ctx* ctx, int bits);

/* Fallback path of bf_linear (W_raw given, Sec. 4.2 "fallback encode"): output groups are encoded
 * in rounds into a scratch buffer and consumed by the multiply-accumulate; `bytes` bounds that
 * buffer (default 4 GiB; one output group, n_in * b encoded diagonals, is the minimum whatever the
 * bound).  A larger bound means fewer rounds, and every round re-reads the rotated inputs.  Results
 * do not depend on it.  Takes effect from the next call; the buffer only ever grows.  No counterpart
 * in the paper.  Errors: INVALID_ARG (null context or zero bytes). */
int bf_set_encode_scratch(bf_ctx* ctx, uint64_t bytes);

/* bf_linear replays a captured CUDA graph of its launch sequence from the third call with the same
 * (ct_in, pt_weights, ct_out, d_out, d_in) on: the first call runs directly (and sizes the scratch),
 * the second is captured.  Replay is skipped on the fallback path, while stage or kernel timing is
 * on, and when the context's stream is itself being captured.  bf_set_graph_replay(ctx, 0) turns
 * it off and drops the stored graphs (default: on). */
int bf_set_graph_replay(bf_ctx* ctx, int on);

/* The kernels of a call are launched with programmatic stream serialisation: each may be scheduled
 * while the previous kernel of the stream drains, and waits for that kernel's completion before it
 * touches memory the call writes (the multiply-accumulate and the key-switch inner product fetch
 * their first cached weights and keys before that wait).  Results are unchanged.
 * bf_set_dependent_launch(ctx, 0) falls back to plain stream order (default: on) and drops the
 * stored graphs.  The paper has no counterpart; this is a launch-latency measure. */
int bf_set_dependent_launch(bf_ctx* ctx, int on);

/* The key switches of a call are independent per rotation.  bf_linear deals the baby rotations of a
 * batch, and then the giant rotations, out to n_lanes chains (inner product, then division by the
 * special prime) that run on streams of the library's own between a fork from and a join into the
 * context's stream, so that one chain's HBM-bound inner product overlaps another chain's
 * arithmetic-bound transforms.  n_lanes is an upper bound: a stage is split only where that was
 * measured to pay (at most 24 baby rotations in the batch; 6 to 20 giant rotations; counts weighted
 * by N / 2^15 above that ring size), otherwise it
 * runs as one chain.  Results do not depend on n_lanes.  1 <= n_lanes <= 4 (default 2);
 * bf_set_lanes drops the stored graphs.  The paper has no counterpart. */
int bf_set_lanes(bf_ctx* ctx, int n_lanes);

/* Rescale (Sec. 2.1): drop the last prime of n_ct ciphertexts that have `level` primes each,
 *     c'_i = (c_i - centred(c_{level-1})) * q_{level-1}^{-1} mod q_i ,
 * i.e. round(c / q_{level-1}).  ct_in: device [n_ct][2][level][N]; ct_out: device
 * [n_ct][2][level-1][N]; ct_out may equal ct_in.  *scale_inout is divided by q_{level-1} when not
 * NULL.  Asynchronous.  Errors: INVALID_ARG, LEVEL, CUDA. */
int bf_rescale(bf_ctx* ctx, const uint64_t* ct_in, uint64_t* ct_out, uint32_t n_ct, uint32_t level,
               double* scale_inout);

/* In-ciphertext fold of the tau partial sums (a variant of the output stage; the packing of Sec. 4.2
 * leaves slot (rho, kappa, c) of an output ciphertext with the partial dot product of row kappa over
 * column class c, and by default the caller adds the tau of them after decryption):
 *     for i = 0 .. log2(tau) - 1:  ct <- ct + rot(ct, 2^i)
 * after which slot (0, kappa, 0) holds the complete dot product.  In place on n_ct full-level
 * ciphertexts (device, boundary layout); level and scale are unchanged, so bf_rescale follows as
 * usual.  Needs the rotation keys for 1, 2, ..., tau/2 slots (MISSING_KEY otherwise) and a
 * power-of-two tau (INVALID_ARG otherwise); costs log2(tau) key switches per ciphertext.
 * Asynchronous. */
int bf_fold(bf_ctx* ctx, uint64_t* ct, uint32_t n_ct);

/* bf_linear followed by bf_rescale with HOST buffers: copies n_in ciphertexts from host_ct_in to
 * the device, runs the layer, rescales once and copies the n_out ciphertexts of level r-1 back to
 * host_ct_out ([n_out][2][r-1][N]).  Pinned host memory makes the copies asynchronous; the call
 * returns after the result has arrived (it synchronises the stream). */
int bf_linear_host(bf_ctx* ctx, const uint64_t* host_ct_in, uint32_t n_in, const bf_weights* pt_weights,
                   const float* W_raw, uint32_t d_out, uint32_t d_in, uint64_t* host_ct_out, uint32_t n_out);

/* One key-switched left rotation of a full-level ciphertext by `steps` slots (the primitive the
 * baby and giant steps are made of).  ct_in, ct_out: device, boundary layout.  Asynchronous. */
int bf_rotate(bf_ctx* ctx, const uint64_t* ct_in, uint32_t steps, uint64_t* ct_out);

/* Products in Z_q[X]/(X^N + 1): out[t] = a[t] * b[t] for n_polys polynomials, polynomial t modulo
 * basis prime (t mod (r+1)); all device, [n_polys][N], coefficient domain.  Exercises the forward
 * and inverse transforms.  Asynchronous. */
int bf_negacyclic_mul(bf_ctx* ctx, const uint64_t* a, const uint64_t* b, uint64_t* out, uint32_t n_polys);

/* bf_negacyclic_mul for callers that must not allocate.  (No counterpart in the paper: this is a
 * deployment convenience of the library.)
 * Who needs it: a host program that has handed all device memory to its own pool, or that calls
 * from a latency-critical loop, cannot tolerate the cudaMalloc (and the device-wide
 * synchronisation that comes with it) by which bf_negacyclic_mul grows its scratch on first use.
 * This entry point performs no cudaMalloc, cudaFree or other allocating call.  Its two
 * transform-domain temporaries live in a fixed array inside the library's device image, which
 * every GPU that loads the library holds (8 MiB) until the process exits.
 *   Limit: ceil(n_polys / (r+1)) * (r+1) * N <= bf_noalloc_max_words() (2^19 words); larger
 *   requests return BF_ERR_TOO_LARGE and enqueue nothing.  With N = 2^15 and r = 7 that is two
 *   groups of 8 polynomials; a context with N = 2^16 and r = 9 (10 x 65536 words per group) never
 *   fits, whatever n_polys is.
 *   The first call on a device resolves the array's device address (cudaGetSymbolAddress); make
 *   that call with the context's device current and before starting any stream capture.
 *   All calls, from any context, share the one array, which keeps the previous call's contents;
 *   the part a call uses is overwritten or cleared by that call.  Two calls whose work overlaps on
 *   the GPU (different streams) race on it: serialise them.
 * Arguments, layout, results and asynchrony are those of bf_negacyclic_mul. */
int bf_negacyclic_mul_noalloc(bf_ctx* ctx, const uint64_t* a, const uint64_t* b, uint64_t* out, uint32_t n_polys);
uint64_t bf_noalloc_max_words(void);

/* Coefficient-domain residues [r][N] (device) of the encoded plaintext Pt[p][q][j][k] held by w. */
int bf_weights_export(bf_ctx* ctx, const bf_weights* w, uint32_t p, uint32_t q, uint32_t j, uint32_t k,
                      uint64_t* out);

/* Per-stage device time of the last bf_linear on this context, in milliseconds, when stage timing
 * was switched on with bf_set_stage_timing(ctx, 1) (adds event records; off by default).
 * stages: 0 input transforms + hoisted ModUp + baby steps, 1 multiply-accumulate (on the fallback
 * path: with the on-the-fly encoding), 2 giant steps, 3 output transform.
 * bf_get_stage_ms synchronises the stream. */
int bf_set_stage_timing(bf_ctx* ctx, int on);
int bf_get_stage_ms(bf_ctx* ctx, float* ms_out /* host, 4 values */);

/* Kernels that wait on asynchronous copies poll with a limit; when a wait gives up the kernel
 * records it and still terminates.  bf_device_status synchronises the stream and returns
 * BF_ERR_TIMEOUT if that happened since the last check (the affected call's results are invalid),
 * BF_ERR_RANGE for an encoder overflow on the fallback path, else BF_OK.  bf_linear_host performs
 * this check itself. */
int bf_device_status(bf_ctx* ctx);

/* Launch accounting.  The library counts its kernel launches per category; with
 * bf_set_kernel_timing(ctx, 1) it also brackets every launch with a pair of CUDA events on the
 * context's stream.  bf_get_kernel_stats synchronises the stream, writes for every category the
 * launches since the previous call (launches_out, host, bf_kernel_categories() values) and the
 * summed event time in ms of the timed ones (ms_out, host), and resets both. */
int bf_set_kernel_timing(bf_ctx* ctx, int on);
int bf_kernel_categories(void);
const char* bf_kernel_category_name(int cat);
int bf_get_kernel_stats(bf_ctx* ctx, uint64_t* launches_out, float* ms_out);

/* Measured rate, in operations per second over the whole GPU, of the 32x32+64-bit integer
 * multiply-add (mad.wide.u32) that the 64-bit modular arithmetic of the transforms and the key
 * switch decomposes into: the denominator for the integer-bound kernels' roofline.  Runs a short
 * probe kernel (a few ms) on the context's stream and synchronises. */
int bf_measure_imad_rate(bf_ctx* ctx, double* mad_per_second_out);

/* The same for the fp64 fused multiply-add (fma.rn.f64) that the transforms of the ciphertext primes
 * (below 2^50) are made of: the denominator for their roofline. */
int bf_measure_fma64_rate(bf_ctx* ctx, double* fma_per_second_out);

/* Bytes of rotation keys the key-switch inner products launched since the previous call had to stream:
 * counted once per distinct key of each launch (distinct_out, host: what must come from HBM; Sec. 4.2
 * "key-switching primitives") and once per rotation (per_rotation_out, host: what the launches read,
 * L2 hits included).  Resets both counters.  Does not synchronise. */
int bf_get_key_stream_bytes(bf_ctx* ctx, uint64_t* distinct_out, uint64_t* per_rotation_out);

const char* bf_strerror(int code);
const char* bf_last_cuda_error(const bf_ctx* ctx);

#ifdef __cplusplus
}
#endif
#endif /* BIFROST_H */
