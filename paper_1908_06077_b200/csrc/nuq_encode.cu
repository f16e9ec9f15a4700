// ENCODE of NUQSGD (App. A) for one gradient vector: bucket norm, stochastic
// quantization (Definition 1) and Elias-recursive token packing in one kernel.
//
// ONE WARP owns a tile of up to 8192 consecutive elements (whole buckets, or one
// 8192-element coding block of a wider bucket) and there is no block-level
// barrier anywhere: warps of a CTA only share two read-only code tables.  For
// each bucket of its tile a warp
//   1. reads the bucket once and reduces its norm (fp64 sums of exact squares);
//   2. walks the bucket again in chunks of 512 elements (the second read is
//      served by L2/L1): a lane handles 4 consecutive elements per 128-element
//      row with one 128-bit load and one Philox block;
//   3. keeps only the groups of 4 elements that hold a nonzero symbol (ballot /
//      popc compaction into a shared-memory list), expands those groups to one
//      entry per nonzero symbol (second compaction), and generates the tokens
//      from that dense list, 32 tokens per step, OR-ing them into a small
//      shared-memory bit window behind a running bit cursor;
//   4. flushes the completed words of the window to the warp's scratch slot in
//      global memory, which ends up holding the exact image of the tile
//      (norm word, sub-block lengths, token strings, per bucket).
// The tile's size is then chained to its predecessors by a decoupled look-back
// scan, and the image is copied from the slot (still in L2) to its place in the
// packed stream.  In the fixed-width mode the place is known in advance and the
// window is flushed straight into the stream.
//
// The kernel is bound by instruction issue, not by HBM; the quantizer is branch
// free and all per-symbol work runs on dense lists.
#include "nuq_common.cuh"
#include "nuq_launch.h"

namespace nuq {

// ERC(N) for N = 1..256 (Algorithm 2): bits 0-15 code word (right aligned), bits 16-20 length.
__constant__ uint32_t c_erc_lut[256];

void build_erc_lut(uint32_t* lut) {
    for (uint32_t N = 1; N <= 256; ++N) {
        uint32_t code = 0, len = 1, n = N;           // the trailing 0
        while (n > 1) {
            uint32_t nb = 32 - __builtin_clz(n);     // prepend binary(n)
            code |= n << len;
            len += nb;
            n = nb - 1;
        }
        lut[N - 1] = code | (len << 16);
    }
}

cudaError_t upload_erc_lut() {
    uint32_t lut[256];
    build_erc_lut(lut);
    return cudaMemcpyToSymbol(c_erc_lut, lut, sizeof(lut));
}

// ---------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al. 2011), one block = the draws of 4 consecutive elements.
// ---------------------------------------------------------------------------
// The ten round keys (key + r * Weyl constants) are precomputed on the host and sit in the
// kernel's parameter block, so they cost no instructions here.
__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3,
                                               const uint32_t (&rk)[20]) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ rk[2 * r];
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ rk[2 * r + 1];
        c1 = (uint32_t)p1;
        c3 = (uint32_t)p0;
        c0 = n0;
        c2 = n2;
    }
    return make_uint4(c0, c1, c2, c3);
}

// ---------------------------------------------------------------------------
// Definition 1 for one coordinate.  y = |v| * (2^s / norm), clamped to 2^s; the
// draw is u = m * 2^-24 with m the top 24 bits of `word`; the coordinate moves to
// the upper level iff u < p.
//
// Exponential levels, y >= 1 (r in [2^(e-s), 2^(e+1-s)], e = floor(log2 y)):
//   p = y 2^-e - 1 = mant / 2^23, and u < p  <=>  (word >> 9) < mant.  Adding
//   0x7FFFFF - (word >> 9) to the bit pattern of y carries into the exponent field
//   exactly in that case, so (bits + 0x7FFFFF - (word >> 9)) >> 23 - 126 is the level
//   index e + 1 + [u < p].  For y < 1 the same expression is at most 1, and it is 1
//   only if u < y as well, so the maximum with [u < y] is the index in every case.
// y < 1 (r in [0, 2^-s]): p = y, and u < y  <=>  float(m) - y 2^24 < 0 (both terms
//   exact, the sign of a rounded difference is the sign of the exact one).
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t quantize_exp(float v, float inv, float top, uint32_t word) {
    const float y = fminf(__fmul_rn(fabsf(v), inv), top);
    const int hi = (int)(__float_as_uint(y) + (0x007FFFFFu - 0x3F000000u) - (word >> 9)) >> 23;
    const float diff = __fsub_rn(__uint2float_rn(word >> 8), __fmul_rn(y, 16777216.0f));
    const int up = (int)(__float_as_uint(diff) >> 31);
    return (uint32_t)max(hi, up);
}

// Uniform levels k / 2^s:  p = y - floor(y).
__device__ __forceinline__ uint32_t quantize_uniform(float v, float inv, float top, uint32_t word) {
    const float y = fminf(__fmul_rn(fabsf(v), inv), top);
    const float fl = fminf(floorf(y), top - 1.0f);
    const float p = y - fl;
    return (uint32_t)fl + ((__uint2float_rn(word >> 8) < p * 16777216.0f) ? 1u : 0u);
}

// OR `nbits` (1..64) right-aligned bits of `value` into the MSB-first bit string `dst` at
// `bitpos`.  Up to three words are touched; dst[bitpos/32 + 2] must exist.
__device__ __forceinline__ void or_bits(uint32_t* dst, uint32_t bitpos, uint64_t value, uint32_t nbits) {
    const uint64_t a = value << (64u - nbits);
    const uint32_t hi = (uint32_t)(a >> 32), lo = (uint32_t)a;
    const uint32_t w = bitpos >> 5, sh = bitpos & 31u;
    const uint32_t w0 = hi >> sh;
    const uint32_t w1 = __funnelshift_r(lo, hi, sh);
    const uint32_t w2 = __funnelshift_r(0u, lo, sh);
    if (w0) atomicOr(dst + w, w0);
    if (w1) atomicOr(dst + w + 1, w1);
    if (w2) atomicOr(dst + w + 2, w2);
}

__device__ __forceinline__ uint64_t ld_volatile_u64(const uint64_t* p) {
    return *reinterpret_cast<const volatile uint64_t*>(p);
}
__device__ __forceinline__ void st_volatile_u64(uint64_t* p, uint64_t v) {
    *reinterpret_cast<volatile uint64_t*>(p) = v;
}

// Decoupled look-back over tile payload sizes, run by one warp.  Returns the
// exclusive prefix (words) of `tile`, or sets *failed.  Every wait is bounded.
__device__ uint64_t tile_lookback(Workspace* ws, uint64_t* state, uint64_t tile, uint64_t aggregate, bool* failed) {
    const uint32_t lane = lane_id();
    *failed = false;
    if (tile == 0) {
        if (lane == 0) st_volatile_u64(state, kTilePrefix | aggregate);
        return 0;
    }
    if (lane == 0) st_volatile_u64(state + tile, kTileAggregate | aggregate);
    uint64_t exclusive = 0;
    int64_t idx = (int64_t)tile - 1 - (int64_t)lane;
    for (;;) {
        uint64_t v = idx >= 0 ? ld_volatile_u64(state + idx) : kTilePrefix;   // before tile 0: prefix 0
        uint32_t polls = 0;
        while (__any_sync(0xffffffffu, (v >> 62) == 0)) {
            if (++polls > (1u << 16)) {                    // ~tens of ms: give up, never hang
                if (lane == 0) {
                    latch_status(ws, kErrTimeout);
                    st_volatile_u64(state + tile, kTilePoison);
                }
                *failed = true;
                return 0;
            }
            __nanosleep(polls < 8 ? 200 : 1000);           // a waiting warp should not eat issue slots
            if ((v >> 62) == 0) v = ld_volatile_u64(state + idx);
        }
        if (__any_sync(0xffffffffu, (v >> 62) == 3)) {     // a predecessor gave up
            if (lane == 0) st_volatile_u64(state + tile, kTilePoison);
            *failed = true;
            return 0;
        }
        uint32_t prefix_mask = __ballot_sync(0xffffffffu, (v >> 62) == 2);
        uint32_t first = prefix_mask ? (uint32_t)__ffs(prefix_mask) - 1u : 31u;
        uint64_t contrib = lane <= first ? (v & kTileValueMask) : 0;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) contrib += __shfl_xor_sync(0xffffffffu, contrib, o);
        exclusive += contrib;
        if (prefix_mask) break;
        idx -= 32;
    }
    if (lane == 0) st_volatile_u64(state + tile, kTilePrefix | (exclusive + aggregate));
    return exclusive;
}

constexpr uint32_t kChunk = 512;                 // elements quantized per step of a warp (2 sub-blocks, 4 rows)
constexpr uint32_t kChunkRows = kChunk / 128;

// Symbols travel as small fields: level index in the low bits, sign above it.
template <uint32_t LEVELSET>
struct Sym {
    static constexpr uint32_t kBits = LEVELSET == kLevelsExp ? 7u : 15u;     // index <= 15 resp. <= 256
    static constexpr uint32_t kMask = (1u << kBits) - 1u;
};

// OR `nbits` (1..32) right-aligned bits of `value` into the MSB-first bit string `dst` at `bitpos`.
__device__ __forceinline__ void or_bits32(uint32_t* dst, uint32_t bitpos, uint32_t value, uint32_t nbits) {
    const uint32_t a = value << (32u - nbits);
    const uint32_t w = bitpos >> 5, sh = bitpos & 31u;
    const uint32_t w0 = a >> sh;
    const uint32_t w1 = __funnelshift_r(0u, a, sh);
    if (w0) atomicOr(dst + w, w0);
    if (w1) atomicOr(dst + w + 1, w1);
}

// Shared memory of one warp.
struct WarpMem {
    uint32_t* window;     // bit window behind the cursor
    uint32_t* tokens;     // kChunk entries: position | field << 10
    uint32_t* groups;     // kChunk / 4 entries of 2 (exponential) or 3 (uniform) words
};

template <uint32_t LEVELSET, uint32_t MODE>
__global__ void __launch_bounds__(kEncThreads, kEncMinBlocks) encode_kernel(const __grid_constant__ EncodeParams P) {
    extern __shared__ __align__(16) uint32_t smem[];
    __shared__ uint32_t s_lut[256];                        // ERC(N), N = 1..256: code | len << 16
    __shared__ uint32_t s_lut_signed[256];                 // exponential levels: sign bit + ERC(index) by field

    using S = Sym<LEVELSET>;
    constexpr uint32_t kGroupWords = LEVELSET == kLevelsExp ? 2u : 3u;
    const Geometry& G = P.geo;
    const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    const uint32_t gwarp = blockIdx.x * kEncWarps + warp;
    uint32_t* wmem = smem + warp * P.warp_smem_words;
    WarpMem M;
    M.window = wmem;
    M.tokens = wmem + P.window_words;
    M.groups = M.tokens + kChunk;
    uint64_t* tile_state = reinterpret_cast<uint64_t*>(P.ws + 1);
    uint32_t* slot = P.slots + (uint64_t)gwarp * P.slot_words;
    uint64_t* table = reinterpret_cast<uint64_t*>(P.out + kHeaderWords);
    uint32_t* payload = MODE == kModeErc ? P.out + kHeaderWords + 2 * (G.nblk + 1) : P.out + kHeaderWords;
    const float top = __uint_as_float((127u + G.s) << 23);
    const uint32_t c2 = (uint32_t)P.offset, c3 = (uint32_t)(P.offset >> 32);
    const uint32_t lt_mask = (1u << lane) - 1u;

    {
        const uint32_t e = c_erc_lut[tid];
        s_lut[tid] = e;
        // field = sign << 7 | index: the sign bit followed by ERC(index)
        const uint32_t idx = tid & 0x7Fu;
        uint32_t v = 0;
        if (idx >= 1) {
            const uint32_t l = c_erc_lut[idx - 1u], len = l >> 16;
            v = ((tid >> 7) << len) | (l & 0xffffu) | ((len + 1u) << 16);
        }
        s_lut_signed[tid] = v;
    }
    for (uint32_t i = lane; i < P.window_words; i += 32) M.window[i] = 0;
    __syncthreads();

    for (;;) {
        uint64_t tile = 0;
        if (lane == 0) tile = atomicAdd(reinterpret_cast<unsigned long long*>(&P.ws->ticket), 1ull);
        tile = __shfl_sync(0xffffffffu, tile, 0);
        if (tile >= G.ntiles) break;

        // ---- tile geometry ------------------------------------------------------
        uint64_t elem0, first_block;
        uint32_t tile_len, nblk_tile, blk_elems;
        uint64_t bucket_idx = 0;
        uint32_t bib = 0;                                   // block within a wide bucket
        if (G.bucket <= kBLK) {
            first_block = tile * G.blocks_per_tile;
            elem0 = first_block * G.bucket;
            const uint64_t left = G.d - elem0;
            tile_len = left < G.tile_elems ? (uint32_t)left : G.tile_elems;
            blk_elems = G.bucket;
            nblk_tile = (tile_len + G.bucket - 1) / G.bucket;
        } else {
            bucket_idx = tile / G.blk_per_bucket;
            bib = (uint32_t)(tile % G.blk_per_bucket);
            first_block = tile;
            const uint64_t b0 = bucket_idx * G.bucket;
            const uint64_t blen = G.d - b0 < G.bucket ? G.d - b0 : G.bucket;
            elem0 = b0 + (uint64_t)bib * kBLK;
            const uint64_t left = blen - (uint64_t)bib * kBLK;
            tile_len = left < kBLK ? (uint32_t)left : kBLK;
            blk_elems = kBLK;
            nblk_tile = 1;
        }
        const float* gt = P.g + elem0;

        uint32_t W = 0;                                     // ERC: words of the tile image so far
        uint32_t my_blk_wordoff = 0;                        // ERC: lane bi keeps the word offset of block bi
        uint32_t tile_code_bits = 0, tile_nnz = 0;
        uint64_t fixed_off = 0;                             // fixed mode: word offset of the tile's first record
        if (MODE == kModeFixed)
            fixed_off = G.bucket <= kBLK ? first_block * G.rec_words
                                         : bucket_idx * G.rec_words + 1u + (uint64_t)bib * (kBLK * G.width / 32u);

        for (uint32_t bi = 0; bi < nblk_tile; ++bi) {
            const uint32_t blk_first = bi * blk_elems;
            const uint32_t bl = min(blk_elems, tile_len - blk_first);
            const uint32_t nsb = (bl + kSB - 1) / kSB;
            const uint32_t head_words = 1u + (nsb + 1u) / 2u;
            const float* gb = gt + blk_first;

            // ---- bucket norm: fp64 sum of exact squares (or max |x|), one rounding to fp32 ----
            float norm;
            if (P.norms_in != nullptr) {
                norm = P.norms_in[G.bucket <= kBLK ? first_block + bi : bucket_idx];
            } else {
                double acc = 0.0;
                uint32_t mx = 0;
#pragma unroll 4
                for (uint32_t base = lane * 4u; base < bl; base += 128u) {
                    float4 x;
                    if (base + 4u <= bl) {
                        x = __ldg(reinterpret_cast<const float4*>(gb + base));
                    } else {
                        x.x = __ldg(gb + base);
                        x.y = base + 1u < bl ? __ldg(gb + base + 1u) : 0.0f;
                        x.z = base + 2u < bl ? __ldg(gb + base + 2u) : 0.0f;
                        x.w = 0.0f;
                    }
                    if (G.norm_kind == kNormL2) {
                        acc = fma((double)x.x, (double)x.x, acc);
                        acc = fma((double)x.y, (double)x.y, acc);
                        acc = fma((double)x.z, (double)x.z, acc);
                        acc = fma((double)x.w, (double)x.w, acc);
                    } else {                                // max |x| on the bit patterns: NaN sorts above inf
                        mx = max(max(mx, __float_as_uint(fabsf(x.x))), __float_as_uint(fabsf(x.y)));
                        mx = max(max(mx, __float_as_uint(fabsf(x.z))), __float_as_uint(fabsf(x.w)));
                    }
                }
                if (G.norm_kind == kNormL2) {
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
                    norm = (float)sqrt(acc);
                } else {
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, o));
                    norm = __uint_as_float(mx);
                }
            }
            if (norm != norm) norm = __uint_as_float(0x7fc00000u);     // one NaN pattern in the stream
            float inv = 0.0f;                                           // 0: the bucket is not quantized
            if (norm > 0.0f && norm < __uint_as_float(0x7f800000u)) {
                inv = __fdiv_rn(top, norm);                             // one IEEE division per bucket
                if (!(inv < __uint_as_float(0x7f800000u))) inv = 0.0f;
            }

            // ---- where this block's bits go -----------------------------------------------
            uint32_t* dst;                                  // words of the block's bit string are flushed here
            if (MODE == kModeErc) {
                if (lane == bi) my_blk_wordoff = W;
                dst = slot + W + head_words;
            } else if (G.bucket <= kBLK) {
                dst = payload + fixed_off + (uint64_t)bi * G.rec_words + 1u;
            } else {
                dst = payload + fixed_off;
            }
            uint32_t bits = 0;                              // bits of the block's string so far
            uint32_t flushed = 0;                           // whole words already written to dst
            uint32_t my_len = 0;                            // ERC: lane q keeps the token bits of sub-block q

            for (uint32_t cb = 0; cb < bl; cb += kChunk) {
                const uint32_t win0 = 32u * flushed;        // bit of the block string at window bit 0
                uint32_t ngroups = 0, ntok = 0;

                // ---- quantize (Definition 1), 128 elements per step ---------------------------
                if (inv != 0.0f) {
#pragma unroll 1
                    for (uint32_t r = 0; r < kChunkRows; ++r) {
                        const uint32_t base = cb + r * 128u + lane * 4u;        // element within the block
                        if (cb + r * 128u >= bl) break;
                        float4 x;
                        if (base + 4u <= bl) {
                            x = __ldg(reinterpret_cast<const float4*>(gb + base));
                        } else {
                            x.x = base + 0u < bl ? __ldg(gb + base + 0u) : 0.0f;
                            x.y = base + 1u < bl ? __ldg(gb + base + 1u) : 0.0f;
                            x.z = base + 2u < bl ? __ldg(gb + base + 2u) : 0.0f;
                            x.w = 0.0f;
                        }
                        const uint64_t ctr = (elem0 + blk_first + base) >> 2;
                        const uint4 rnd = philox4x32_10((uint32_t)ctr, (uint32_t)(ctr >> 32), c2, c3, P.round_keys);
                        uint32_t q0, q1, q2, q3;
                        if (LEVELSET == kLevelsExp) {
                            q0 = quantize_exp(x.x, inv, top, rnd.x);
                            q1 = quantize_exp(x.y, inv, top, rnd.y);
                            q2 = quantize_exp(x.z, inv, top, rnd.z);
                            q3 = quantize_exp(x.w, inv, top, rnd.w);
                        } else {
                            q0 = quantize_uniform(x.x, inv, top, rnd.x);
                            q1 = quantize_uniform(x.y, inv, top, rnd.y);
                            q2 = quantize_uniform(x.z, inv, top, rnd.z);
                            q3 = quantize_uniform(x.w, inv, top, rnd.w);
                        }
                        const uint32_t b0 = __float_as_uint(x.x), b1 = __float_as_uint(x.y);
                        const uint32_t b2 = __float_as_uint(x.z), b3 = __float_as_uint(x.w);
                        // fields (index | sign << kBits) of the 4 elements, packed; a zero symbol has no sign
                        uint32_t f01, f23;                   // exponential: f01 holds all four bytes
                        bool any;
                        if (LEVELSET == kLevelsExp) {
                            const uint32_t syms = q0 | (q1 << 8) | (q2 << 16) | (q3 << 24);
                            const uint32_t tops =
                                __byte_perm(__byte_perm(b0, b1, 0x0073), __byte_perm(b2, b3, 0x0073), 0x5410);
                            const uint32_t nzb = (syms + 0x7F7F7F7Fu) & 0x80808080u;   // bit 7 of a byte: symbol != 0
                            f01 = syms | (tops & nzb);
                            f23 = 0;
                            any = syms != 0;
                        } else {
                            f01 = (q0 | (q0 ? (b0 >> 16) & 0x8000u : 0u)) | ((q1 | (q1 ? (b1 >> 16) & 0x8000u : 0u)) << 16);
                            f23 = (q2 | (q2 ? (b2 >> 16) & 0x8000u : 0u)) | ((q3 | (q3 ? (b3 >> 16) & 0x8000u : 0u)) << 16);
                            any = (f01 | f23) != 0;
                        }
                        if (MODE == kModeErc) {
                            // keep the groups that hold a nonzero symbol
                            const uint32_t vote = __ballot_sync(0xffffffffu, any);
                            if (any) {
                                uint32_t* ge = M.groups + (ngroups + __popc(vote & lt_mask)) * kGroupWords;
                                ge[0] = f01;
                                if (LEVELSET == kLevelsExp) {
                                    ge[1] = r * 32u + lane;
                                } else {
                                    ge[1] = f23;
                                    ge[2] = r * 32u + lane;
                                }
                            }
                            ngroups += __popc(vote);
                        } else if (any) {
                            // fixed-width fields, MSB first, straight into the window
                            const uint32_t wbits = G.width;
                            uint32_t f[4];
                            if (LEVELSET == kLevelsExp) {
                                f[0] = f01 & 0xFFu; f[1] = (f01 >> 8) & 0xFFu; f[2] = (f01 >> 16) & 0xFFu; f[3] = f01 >> 24;
                            } else {
                                f[0] = f01 & 0xFFFFu; f[1] = f01 >> 16; f[2] = f23 & 0xFFFFu; f[3] = f23 >> 16;
                            }
                            uint64_t str = 0;
#pragma unroll
                            for (int c = 0; c < 4; ++c) {
                                str = (str << wbits) | ((f[c] & S::kMask) | ((f[c] >> S::kBits) << (wbits - 1u)));
                                tile_nnz += (f[c] & S::kMask) != 0;
                            }
                            or_bits(M.window, base * wbits - win0, str, 4u * wbits);
                        }
                    }
                }

                if (MODE == kModeErc) {
                    __syncwarp();
                    // ---- expand the kept groups to one entry per nonzero symbol ---------------------
                    for (uint32_t g0 = 0; g0 < ngroups; g0 += 32) {
                        const bool valid = g0 + lane < ngroups;
                        uint32_t f01 = 0, f23 = 0, gpos = 0;
                        if (valid) {
                            const uint32_t* ge = M.groups + (g0 + lane) * kGroupWords;
                            f01 = ge[0];
                            if (LEVELSET == kLevelsExp) { gpos = ge[1]; } else { f23 = ge[1]; gpos = ge[2]; }
                        }
                        uint32_t f[4];
                        if (LEVELSET == kLevelsExp) {
                            f[0] = f01 & 0xFFu; f[1] = (f01 >> 8) & 0xFFu; f[2] = (f01 >> 16) & 0xFFu; f[3] = f01 >> 24;
                        } else {
                            f[0] = f01 & 0xFFFFu; f[1] = f01 >> 16; f[2] = f23 & 0xFFFFu; f[3] = f23 >> 16;
                        }
                        const uint32_t cnt = (f[0] != 0) + (f[1] != 0) + (f[2] != 0) + (f[3] != 0);
                        uint32_t incl = cnt;
#pragma unroll
                        for (int o = 1; o < 32; o <<= 1) {
                            const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
                            if (lane >= (uint32_t)o) incl += t;
                        }
                        uint32_t at = ntok + incl - cnt;
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            if (f[c]) M.tokens[at++] = (gpos * 4u + (uint32_t)c) | (f[c] << 10);
                        }
                        ntok += __shfl_sync(0xffffffffu, incl, 31);
                    }
                    __syncwarp();

                    // ---- tokens ERC(gap) sign ERC(index), 32 per step, behind the bit cursor ----------
                    int carry_pos = -1;                     // position (within the chunk) of the last nonzero so far
                    uint32_t my_start = 0xFFFFFFFFu;        // lane q < 2: where sub-block q's string starts
                    for (uint32_t t0 = 0; t0 < ntok; t0 += 32) {
                        const bool valid = t0 + lane < ntok;
                        const uint32_t e = valid ? M.tokens[t0 + lane] : 0u;
                        const int pos = (int)(e & 1023u);
                        const uint32_t field = e >> 10;
                        int prev = __shfl_up_sync(0xffffffffu, pos, 1);
                        if (lane == 0) prev = carry_pos;
                        const bool first_of_sb = (prev >> 8) != (pos >> 8);      // also when there is no predecessor
                        if (first_of_sb) prev = (pos & ~255) - 1;                  // the run restarts: t_0 = 0
                        uint32_t tlen = 0, tokA = 0, lenA = 0, tokB = 0, lenB = 0;
                        if (valid) {
                            const uint32_t gl = s_lut[pos - prev - 1];
                            if (LEVELSET == kLevelsExp) {
                                const uint32_t ll = s_lut_signed[field];
                                lenB = ll >> 16;
                                tokA = ((gl & 0xffffu) << lenB) | (ll & 0xffffu);                  // <= 16 + 8 bits
                                lenA = (gl >> 16) + lenB;
                                tlen = lenA;
                            } else {
                                const uint32_t ll = s_lut[(field & S::kMask) - 1u];
                                tokA = gl & 0xffffu;
                                lenA = gl >> 16;
                                lenB = (ll >> 16) + 1u;                                           // sign + ERC(index) <= 17
                                tokB = ((field >> S::kBits) << (lenB - 1u)) | (ll & 0xffffu);
                                tlen = lenA + lenB;
                            }
                        }
                        uint32_t incl = tlen;
#pragma unroll
                        for (int o = 1; o < 32; o <<= 1) {
                            const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
                            if (lane >= (uint32_t)o) incl += t;
                        }
                        const uint32_t off = bits + incl - tlen;    // bit of the block string where my token starts
                        // the first token of a sub-block marks where that sub-block's string starts
                        uint32_t starts = __ballot_sync(0xffffffffu, valid && first_of_sb);
                        while (starts) {
                            const int src = __ffs(starts) - 1;
                            starts &= starts - 1;
                            const uint32_t q = (uint32_t)__shfl_sync(0xffffffffu, pos, src) >> 8;
                            const uint32_t o = __shfl_sync(0xffffffffu, off, src);
                            if (lane == q) my_start = o;
                        }
                        if (valid) {
                            if (LEVELSET == kLevelsExp) {
                                or_bits32(M.window, off - win0, tokA, lenA);
                            } else {
                                or_bits32(M.window, off - win0, tokA, lenA);
                                or_bits32(M.window, off - win0 + lenA, tokB, lenB);
                            }
                        }
                        bits += __shfl_sync(0xffffffffu, incl, 31);
                        carry_pos = __shfl_sync(0xffffffffu, pos, min(ntok - t0, 32u) - 1u);
                    }
                    tile_nnz += ntok;
                    // sub-block strings follow one another: an empty one starts where the next one does
                    {
                        uint32_t s1 = __shfl_sync(0xffffffffu, my_start, 1);
                        uint32_t s0 = __shfl_sync(0xffffffffu, my_start, 0);
                        if (s1 == 0xFFFFFFFFu) s1 = bits;
                        if (s0 == 0xFFFFFFFFu) s0 = s1;
                        const uint32_t q = cb / kSB;                // first sub-block of this chunk
                        if (lane == q) my_len = s1 - s0;
                        if (lane == q + 1u) my_len = bits - s1;
                    }
                } else {
                    bits = min(cb + kChunk, bl) * G.width;
                }

                // ---- flush the completed words of the window ------------------------------------------
                __syncwarp();
                {
                    const uint32_t full = (bits >> 5) - flushed;
                    for (uint32_t i = lane; i < full; i += 32) dst[flushed + i] = M.window[i];
                    const uint32_t partial = M.window[full];
                    __syncwarp();
                    for (uint32_t i = lane; i < full + 3u; i += 32) M.window[i] = 0;
                    __syncwarp();
                    if (lane == 0) M.window[0] = partial;
                    __syncwarp();
                    flushed += full;
                }
            }

            // ---- end of the block: last partial word, then the block's header ----------------------------
            if (bits & 31u) {
                if (lane == 0) {
                    dst[flushed] = M.window[0];
                    M.window[0] = 0;
                }
                __syncwarp();
            }
            if (MODE == kModeErc) {
                uint32_t* hdr = slot + W;
                if (lane == 0) hdr[0] = __float_as_uint(norm);
                const uint32_t hi = __shfl_down_sync(0xffffffffu, my_len, 1);
                if (!(lane & 1u) && lane < nsb) hdr[1u + lane / 2u] = my_len | (lane + 1u < nsb ? hi << 16 : 0u);
                W += head_words + (bits + 31u) / 32u;
                tile_code_bits += bits;
            } else {
                if (lane == 0 && (G.bucket <= kBLK || bib == 0))
                    payload[G.bucket <= kBLK ? fixed_off + (uint64_t)bi * G.rec_words : bucket_idx * G.rec_words] =
                        __float_as_uint(norm);
            }
        }

        // ---- ERC: chain the tile to its predecessors, then move its image into the stream ---------------
        if (MODE == kModeErc) {
            const uint32_t tile_words = W;
            bool failed;
            const uint64_t tile_off = tile_lookback(P.ws, tile_state, tile, tile_words, &failed);
            __syncwarp();
            if (!failed) {
                for (uint32_t i = lane; i < tile_words; i += 32) payload[tile_off + i] = __ldcg(slot + i);
                if (lane < nblk_tile) table[first_block + lane] = 32ull * (tile_off + my_blk_wordoff);
                if (tile == G.ntiles - 1 && lane == 0) {
                    table[G.nblk] = 32ull * (tile_off + tile_words);
                    P.ws->total_words = tile_off + tile_words;
                }
            }
            if (lane == 0 && tile_code_bits)
                atomicAdd(reinterpret_cast<unsigned long long*>(&P.ws->code_bits), (unsigned long long)tile_code_bits);
        } else {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) tile_nnz += __shfl_xor_sync(0xffffffffu, tile_nnz, o);
        }

        // ---- last tile to finish writes the header -------------------------------------------------------
        __syncwarp();
        if (lane == 0) {
            if (tile_nnz) atomicAdd(reinterpret_cast<unsigned long long*>(&P.ws->nnz), (unsigned long long)tile_nnz);
            __threadfence();
            unsigned long long prev = atomicAdd(reinterpret_cast<unsigned long long*>(&P.ws->done), 1ull);
            if (prev == G.ntiles - 1) {
                __threadfence();
                uint64_t code_bits, words;
                uint64_t nnz = ld_volatile_u64(&P.ws->nnz);
                uint64_t nrec = MODE == kModeErc ? G.nblk : G.nb;
                if (MODE == kModeErc) {
                    code_bits = ld_volatile_u64(&P.ws->code_bits);
                    words = kHeaderWords + 2 * (G.nblk + 1) + ld_volatile_u64(&P.ws->total_words);
                } else {
                    code_bits = G.d * G.width;
                    uint64_t last = G.d - (G.nb - 1) * G.bucket;
                    words = kHeaderWords + (G.nb - 1) * G.rec_words + 1 + (last * G.width + 31) / 32;
                }
                uint64_t container_bits = 32 * words;
                uint32_t* h = P.out;
                h[0] = kMagic; h[1] = kVersion;
                h[2] = (uint32_t)G.d; h[3] = (uint32_t)(G.d >> 32);
                h[4] = G.bucket; h[5] = G.s;
                h[6] = G.norm_kind | (G.levelset << 8) | (G.mode << 16);
                h[7] = kSB;
                h[8] = (uint32_t)nrec; h[9] = (uint32_t)(nrec >> 32);
                h[10] = (uint32_t)container_bits; h[11] = (uint32_t)(container_bits >> 32);
                h[12] = (uint32_t)code_bits; h[13] = (uint32_t)(code_bits >> 32);
                h[14] = (uint32_t)nnz; h[15] = (uint32_t)(nnz >> 32);
                if (P.out_bits) *P.out_bits = container_bits;
            }
        }
    }
}

// ---------------------------------------------------------------------------
// Stand-alone bucket norm, used for buckets wider than one tile: one CTA per
// bucket, fp64 accumulation of exact products, one rounding to fp32.
// ---------------------------------------------------------------------------
__global__ void __launch_bounds__(256) bucket_norm_kernel(const float* __restrict__ g, uint64_t d, uint32_t bucket,
                                                          uint32_t norm_kind, float* __restrict__ norms) {
    __shared__ double s_acc[8];
    __shared__ uint32_t s_max[8];
    const uint64_t b = blockIdx.x;
    const uint64_t lo = b * bucket;
    const uint32_t n = (uint32_t)(d - lo < bucket ? d - lo : bucket);
    const float* v = g + lo;
    double acc = 0.0;
    uint32_t m = 0;
    for (uint32_t i = threadIdx.x * 4u; i < n; i += 1024u) {
        float xs[4];
        if (i + 4u <= n) {
            float4 t = __ldg(reinterpret_cast<const float4*>(v + i));
            xs[0] = t.x; xs[1] = t.y; xs[2] = t.z; xs[3] = t.w;
        } else {
            for (int e = 0; e < 4; ++e) xs[e] = i + e < n ? v[i + e] : 0.0f;
        }
        for (int e = 0; e < 4; ++e) {
            acc = fma((double)xs[e], (double)xs[e], acc);
            m = max(m, __float_as_uint(fabsf(xs[e])));
        }
    }
    for (int o = 16; o > 0; o >>= 1) {
        acc += __shfl_xor_sync(0xffffffffu, acc, o);
        m = max(m, __shfl_xor_sync(0xffffffffu, m, o));
    }
    if ((threadIdx.x & 31) == 0) { s_acc[threadIdx.x >> 5] = acc; s_max[threadIdx.x >> 5] = m; }
    __syncthreads();
    if (threadIdx.x == 0) {
        for (int w = 1; w < 8; ++w) { acc += s_acc[w]; m = max(m, s_max[w]); }
        float norm = norm_kind == kNormL2 ? (float)sqrt(acc) : __uint_as_float(m);
        norms[b] = norm != norm ? __uint_as_float(0x7fc00000u) : norm;
    }
}

// ---------------------------------------------------------------------------
// launchers
// ---------------------------------------------------------------------------
cudaError_t launch_bucket_norms(const float* g, uint64_t d, uint32_t bucket, uint32_t norm_kind, float* norms,
                                uint64_t nb, cudaStream_t stream) {
    bucket_norm_kernel<<<(unsigned)nb, 256, 0, stream>>>(g, d, bucket, norm_kind, norms);
    return cudaGetLastError();
}

int encode_max_blocks(int sms) { return sms * kEncMinBlocks; }

template <uint32_t L, uint32_t M>
static cudaError_t launch_one(const EncodeParams& P, cudaStream_t stream) {
    const size_t smem = (size_t)kEncWarps * P.warp_smem_words * 4u;
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(encode_kernel<L, M>, cudaFuncAttributeMaxDynamicSharedMemorySize, 96 * 1024);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    if (smem > 96 * 1024 || P.grid == 0) return cudaErrorInvalidValue;
    encode_kernel<L, M><<<P.grid, kEncThreads, smem, stream>>>(P);
    return cudaGetLastError();
}

cudaError_t launch_encode(const EncodeParams& P, cudaStream_t stream) {
    const bool uni = P.geo.levelset == kLevelsUniform, fixed = P.geo.mode == kModeFixed;
    if (!uni && !fixed) return launch_one<kLevelsExp, kModeErc>(P, stream);
    if (!uni && fixed) return launch_one<kLevelsExp, kModeFixed>(P, stream);
    if (uni && !fixed) return launch_one<kLevelsUniform, kModeErc>(P, stream);
    return launch_one<kLevelsUniform, kModeFixed>(P, stream);
}

}  // namespace nuq
