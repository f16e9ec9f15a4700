/*
 * nuq.h -- C ABI of the B200 (sm_100a) NUQSGD codec.
 *
 * The library implements the communication hot path of NUQSGD (arXiv
 * 1908.06077): per-bucket norm, nonuniform stochastic quantization
 * (Definition 1 with the level set (0, 2^-s, ..., 1/2, 1) of Sec. 3.1),
 * ENCODE / DECODE with Elias recursive coding (App. A, Algorithm 2) and the
 * aggregation sum of Algorithm 1, for K simulated workers on one GPU.
 *
 * Conventions
 *   - "device" pointers are CUDA global-memory addresses on the current device;
 *     "host" pointers are ordinary process memory.
 *   - `stream` is a cudaStream_t passed as void* (NULL = legacy default stream).
 *   - Calls only enqueue work and return; argument errors are returned at once,
 *     errors found by the kernels (malformed container, scan time-out) are
 *     latched in a per-stream status word read by nuq_last_status().
 *   - d = vector length, bucket = elements per norm bucket (Sec. 5, "bucket
 *     size"), s = number of internal levels (Sec. 3.1).
 *
 * Limits: 1 <= d < 2^40; bucket a multiple of 256 with 256 <= bucket <= 8192,
 * or bucket in {16384, 32768, 65536}; 1 <= s <= 14 (exponential levels and
 * level tables) or 1 <= s <= 8 (uniform levels) or 1 <= s <= 7 (coded level
 * indices); 1 <= K <= 64.
 *
 * Container written by nuq_encode (all u32 words little endian; bit p of a bit
 * string sits in word p>>5 at bit 31-(p&31)):
 *   words 0..15   header: magic 'NUQ1', version, d (2 words), bucket, s,
 *                 flags (norm | levels<<8 | mode<<16), 256, nblk (2),
 *                 container_bits (2), code_bits (2), nnz (2)
 *   level table   only in streams with NUQ_LEVELS_TABLE: the s interior
 *                 levels l_1 .. l_s as fp32 words, then a zero word if s is
 *                 odd; everything below follows behind it
 *   code lengths  only in streams with NUQ_MODE_CODED: two words whose bytes (in
 *                 memory order) are the code lengths of the level indices
 *                 1 .. s+1, the remaining bytes zero; behind the level table
 *   ERC mode      (nblk+1) u64 bit offsets of the coding blocks, relative to
 *                 the payload that follows the table.  A coding block is up to
 *                 8192 consecutive elements of one bucket: norm (fp32 bits) |
 *                 one u16 token-bit count per 256-element sub-block (padded to
 *                 a word) | the sub-blocks' token strings back to back | zero
 *                 padding to a word.  A token is ERC(gap) sign ERC(level
 *                 index); the gap is counted from the start of the sub-block.
 *   coded mode    as the ERC mode, but the level index of a token is written
 *                 with the canonical prefix code of the lengths above (Sec. 5,
 *                 "efficient encoding": Huffman-coded levels): level indices
 *                 ordered by (length, index), the first word all zeros, each
 *                 next word the previous plus one, extended with zeros.
 *   fixed mode    per bucket: norm word | fields of w bits (sign, level index)
 *                 MSB first | zero padding to a word; no table.
 */
#ifndef NUQ_H_
#define NUQ_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef int nuq_status;
#define NUQ_OK 0
#define NUQ_ERR_INVALID_ARG (-1) /* null / misaligned pointer, size or parameter out of range      */
#define NUQ_ERR_CAPACITY (-2)    /* a fixed capacity is too small (nuq_encode_static: scratch)     */
#define NUQ_ERR_BAD_STREAM (-3)  /* a container failed validation inside nuq_decode_accumulate     */
#define NUQ_ERR_CUDA (-4)        /* a CUDA runtime call failed (allocation, launch)                */
#define NUQ_ERR_TIMEOUT (-5)     /* the encoder's cross-tile scan gave up waiting (bounded spin)   */
#define NUQ_ERR_INTERNAL (-6)    /* an internal capacity check failed (a defect of the library)    */
#define NUQ_WARN_NONFINITE 1     /* status word only: a bucket with a NaN, infinite or vanishing   *
                                  * norm was written unquantized (all symbols zero, norm word kept) */

/* norm_kind argument of nuq_encode: bit fields */
#define NUQ_NORM_L2 0u            /* bits 0-7: Euclidean norm (Sec. 2), the paper's choice        */
#define NUQ_NORM_LINF 1u          /*           max-abs norm (QSGDinf comparison, Sec. 1)          */
#define NUQ_LEVELS_EXP (0u << 8)  /* bits 8-15: levels (0, 2^-s, ..., 1/2, 1)  (Sec. 3.1)         */
#define NUQ_LEVELS_UNIFORM (1u << 8) /*         levels k / 2^s, k = 0..2^s    (QSGD comparison)   */
#define NUQ_LEVELS_TABLE (2u << 8) /*           levels (0, l_1, ..., l_s, 1) set by               *
                                    *           nuq_set_level_table   (Sec. 3.3)                  */
#define NUQ_MODE_ERC (0u << 16)   /* bits 16-23: Elias-recursive token stream (App. A)            */
#define NUQ_MODE_FIXED (1u << 16) /*             fixed-width fields ("4-bit" variant of Sec. 5)   */
#define NUQ_MODE_CODED (2u << 16) /*             as NUQ_MODE_ERC with the level indices written   *
                                   *             in the code of nuq_set_level_code ("encoded       *
                                   *             NUQSGD", Sec. 5); not with uniform levels; s <= 7 */
#define NUQ_TEST_NORMS (1u << 24) /* take bucket norms from nuq_set_test_norms (parity testing)   */
#define NUQ_TEST_SHORT_PATIENCE (1u << 25) /* test hook: the cross-tile scan gives up after two  *
                                   * polls instead of tens of milliseconds, so that a test can    *
                                   * see NUQ_ERR_TIMEOUT without anything being withheld          */

typedef struct nuq_info {
    uint64_t d;
    uint32_t bucket;
    uint32_t s;
    uint32_t flags;          /* norm | levels<<8 | mode<<16 */
    uint32_t sub_block;      /* 256 */
    uint64_t nblk;           /* coding blocks (ERC) or buckets (fixed) */
    uint64_t container_bits; /* what a sender would transmit */
    uint64_t code_bits;      /* token bits only (ERC) or d*w (fixed) */
    uint64_t nnz;            /* coordinates quantized to a nonzero level */
} nuq_info;

/*
 * c <- ENCODE(g)   (Algorithm 1, encode line; App. A; Definition 1).
 *
 * Splits g into buckets of `bucket` elements (the last may be short), takes
 * each bucket's norm, quantizes every coordinate stochastically to the level
 * set and writes the container described above.  Coordinate i (0-based within
 * this call) draws u = (w >> 8) * 2^-24 from word (i & 3) of
 * Philox4x32-10(key = seed, counter = (i >> 2, offset)) and moves to the upper
 * level iff u < p(r_i), so equal (seed, offset) reproduce the stream exactly.
 *
 *   g         device, d floats, 16-byte aligned; read only
 *   out       device, 16-byte aligned, at least nuq_encode_bound() bytes; need
 *             not be zeroed; fully owned by the caller
 *   out_bits  device u64 (may be NULL): receives container_bits
 *   returns   NUQ_ERR_INVALID_ARG for bad arguments, NUQ_ERR_CUDA if the
 *             per-stream workspace cannot be allocated or a launch fails.
 * The call may allocate (and then synchronise the device) when the per-stream
 * workspace has to grow; otherwise it is asynchronous.  Calls on different
 * streams may run at the same time (each stream has its own workspace).
 * The kernel is launched so that its blocks may be set up while the kernel
 * before it in the stream ends; it reads and writes memory only after that
 * kernel has ended, so the order of the stream holds for g, out, out_bits.
 * Once the stream's workspace exists (after a first call of at least this
 * size on the stream), encode calls may be captured into a CUDA graph and
 * replayed: the kernels leave the workspace as they found it.  Decode calls
 * may not: their hand-out counter alternates with the number of the call,
 * which a replay does not advance.
 */
nuq_status nuq_encode(const float* g, uint64_t d, uint32_t bucket, uint32_t s, uint32_t norm_kind, uint64_t seed,
                      uint64_t offset, void* out, uint64_t* out_bits, void* stream);

/*
 * acc <- sum_k DECODE(c_k)   (Algorithm 1, decode and aggregation lines,
 * without the alpha/K factor; App. A decoding).
 *
 *   streams  HOST array of K device pointers to containers written by
 *            nuq_encode with the same (d, bucket, s); each buffer must hold
 *            the container_bits its header declares.  The array is copied at
 *            call time.
 *   acc      device, d floats, 16-byte aligned; OVERWRITTEN with
 *            ((0 + q_0[i]) + q_1[i]) + ... in fp32, k ascending.
 * Each container's header, offsets, lengths and tokens are validated on the
 * device; a violation latches NUQ_ERR_BAD_STREAM (the affected coordinates of
 * acc are then unspecified, nothing outside acc[0..d) is written).
 */
nuq_status nuq_decode_accumulate(const void* const* streams, uint32_t K, uint64_t d, uint32_t bucket, uint32_t s,
                                 float* acc, void* stream);

/*
 * The aggregation line of Algorithm 1 fused into DECODE:
 *     w <- w - (alpha / K) sum_k DECODE(c_k)
 * and, with mu != 0, the momentum rule of Sec. 4 ("NUQSGD with momentum") in its place:
 *     y = w - (alpha / K) G,   y^l = w - l (alpha / K) G,   w <- y + mu (y^l - y^l_prev)
 * with G = sum_k DECODE(c_k); l = 0 is the heavy-ball method, l = 1 Nesterov's.  The
 * sum is applied where the decoder finishes it, so it is not written out and read
 * again by an optimizer kernel.  No projection (Omega = R^d).
 *
 *   streams, K, d, bucket, s   as for nuq_decode_accumulate
 *   acc      device, d floats, 16-byte aligned, or NULL.  If given it receives
 *            the sum as from nuq_decode_accumulate.  With K <= 2 it is REQUIRED
 *            (the library adds the streams up in it).
 *   w        device, d floats, 16-byte aligned: the parameters, updated in place
 *   yl       device, d floats, 16-byte aligned: y^l of the previous step on
 *            entry (the parameters themselves before the first step), y^l of
 *            this step on return; may be NULL when mu == 0 (it is not touched)
 *   alpha    learning rate; mu in [0, 1) momentum; l in [0, 1]
 * Arithmetic: fp32; alpha / K and l alpha / K are formed on the host in double
 * and rounded once, each of the three lines is one fused multiply-add.
 * Errors as for nuq_decode_accumulate; after NUQ_ERR_BAD_STREAM the affected
 * coordinates of w and yl are unspecified.
 */
nuq_status nuq_decode_update(const void* const* streams, uint32_t K, uint64_t d, uint32_t bucket, uint32_t s,
                             float* acc, float* w, float* yl, float alpha, float mu, float l, void* stream);

/*
 * nuq_encode for callers that must not allocate device memory.  (The paper has
 * no counterpart; this entry point exists for deployment reasons only.)
 *
 * Who needs it: code that runs where cudaMalloc is forbidden or would stall --
 * inside a framework that has handed all of the GPU's memory to its own caching
 * allocator, in a latency-critical loop where the implicit device
 * synchronisation of an allocation is not acceptable, or in a process whose
 * memory budget is fixed at start-up.  nuq_encode keeps its cross-tile scan
 * state in a workspace that it allocates (and regrows) on demand; this variant
 * keeps the same state in a fixed array of NUQ_STATIC_SCRATCH_BYTES that is part
 * of the library's device image, so it never calls cudaMalloc, cudaFree or any
 * allocating routine.  Every GPU that loads the library holds that array until
 * the process exits.
 *
 * Arguments, container, random draws and results are exactly those of
 * nuq_encode.  Differences:
 *   - Size limit: with T = ceil(d / tile) tiles (a tile is 8192 elements, or
 *     floor(8192 / bucket) buckets) the scan state needs 64 + 8 * (T + ceil(T / 32))
 *     bytes, plus 4 bytes per bucket when bucket > 8192 and the bucket norms
 *     come from a pass of their own (4-bit fixed-width fields).  If that exceeds
 *     NUQ_STATIC_SCRATCH_BYTES the call returns NUQ_ERR_CAPACITY and enqueues
 *     nothing (d up to about 5.2e8 with bucket = 8192).
 *   - The first call on each device looks up the array's device address (the
 *     device must be current, as for every call here) and uploads a 1 KB code
 *     table.  Make that first call outside any stream capture.
 *   - All calls on one device share the one array, which still holds what the
 *     previous call left; each call clears the part it uses, in stream order,
 *     before its kernel runs.  Two calls whose kernels can overlap on the GPU
 *     (different streams, no dependency between them) race on it and produce
 *     garbage: serialise them.
 *   - Kernel-detected errors (NUQ_ERR_TIMEOUT) are latched in the array and are
 *     reported, and cleared, by nuq_last_status on that device.  nuq_last_status
 *     waits only for the stream it is given: pass the stream the static call ran
 *     on (or synchronise the device first), or a status latched later is missed.
 */
#define NUQ_STATIC_SCRATCH_BYTES (512u * 1024u)
nuq_status nuq_encode_static(const float* g, uint64_t d, uint32_t bucket, uint32_t s, uint32_t norm_kind,
                             uint64_t seed, uint64_t offset, void* out, uint64_t* out_bits, void* stream);

/* Bytes that `out` of nuq_encode must hold for these arguments (0 if they are invalid). */
uint64_t nuq_encode_bound(uint64_t d, uint32_t bucket, uint32_t s, uint32_t norm_kind);

/*
 * General level sequences (Sec. 3.3, e.g. L_p = (0, p^s, ..., p, 1)): sets the s interior
 * levels 0 < l_1 < ... < l_s < 1 (HOST array, copied) that nuq_encode uses from now on when
 * it is called with NUQ_LEVELS_TABLE and this s.  A coordinate with l_j <= r < l_{j+1},
 * r = |v| / norm, moves to l_{j+1} with probability (r - l_j) / (l_{j+1} - l_j) (fp32: r
 * is |v| times the rounded 1 / norm, the quotient a product with the rounded inverse
 * width).  The container carries the levels; nuq_decode_accumulate reads them from there.
 * Returns NUQ_ERR_INVALID_ARG unless the levels increase strictly inside (0, 1) and
 * 1 <= s <= 14.
 */
nuq_status nuq_set_level_table(const float* interior_levels, uint32_t s);

/*
 * Coded level indices (Sec. 5, "efficient encoding": a Huffman code is fitted on an initial
 * sample of gradients and then kept; the paper calls the variant encoded NUQSGD).  Three steps:
 *
 * nuq_level_histogram  quantizes g exactly as nuq_encode would (same arguments, same draws;
 *            norm_kind without a mode, not NUQ_LEVELS_UNIFORM) and counts how often each level
 *            index 0 .. s+1 comes out.  hist: DEVICE array of s + 2 u64 counters, 8-byte
 *            aligned, overwritten in stream order.  Bucket norms are taken in a pass of
 *            their own (fp64 sums), so a coordinate within rounding of a decision threshold
 *            may be counted one level off what nuq_encode sends.
 * nuq_fit_level_code   HOST arrays: from hist[1 .. s+1] (hist[0], the zeros, is not coded)
 *            builds a Huffman tree and returns the s + 1 code lengths, lengths[j-1] for level
 *            index j.  The tree joins, s times, the two nodes of least weight; among equal
 *            weights a leaf goes before a joined node, leaves by index, joined nodes by age.
 *            A level index that never occurred still gets a word.  1 <= s <= 7, so no word is
 *            longer than 7 bits.
 * nuq_set_level_code   HOST array of s + 1 lengths (1 .. 7 each, Kraft sum at most 1; those
 *            of nuq_fit_level_code or any others): the code nuq_encode uses from now on when
 *            called with NUQ_MODE_CODED and this s.  The container carries the lengths;
 *            nuq_decode_accumulate reads them from there.
 * Each returns NUQ_ERR_INVALID_ARG for arguments outside these ranges.
 */
nuq_status nuq_level_histogram(const float* g, uint64_t d, uint32_t bucket, uint32_t s, uint32_t norm_kind, uint64_t seed,
                               uint64_t offset, uint64_t* hist, void* stream);
nuq_status nuq_fit_level_code(const uint64_t* hist, uint32_t s, uint8_t* lengths);
nuq_status nuq_set_level_code(const uint8_t* lengths, uint32_t s);

/* Parity-test hook: device array of ceil(d/bucket) bucket norms that nuq_encode uses in
 * place of its own reduction when NUQ_TEST_NORMS is set; NULL clears it.  The pointer is
 * kept, not copied.                                                                        */
nuq_status nuq_set_test_norms(const float* norms);

/* Synchronises `stream` and returns, then clears, the status latched by the kernels that
 * ran on it since the last call: NUQ_OK, an error (NUQ_ERR_BAD_STREAM, NUQ_ERR_TIMEOUT,
 * NUQ_ERR_INTERNAL; the most negative one wins), or NUQ_WARN_NONFINITE when no error was
 * latched and some bucket was written unquantized.                                         */
nuq_status nuq_last_status(void* stream);

/* Copies the header of a container (device) into *host_out; synchronises `stream`.        */
nuq_status nuq_stream_info(const void* out, nuq_info* host_out, void* stream);

/* Frees every per-stream workspace of the library. */
void nuq_shutdown(void);

const char* nuq_version(void);

#ifdef __cplusplus
}
#endif
#endif /* NUQ_H_ */
