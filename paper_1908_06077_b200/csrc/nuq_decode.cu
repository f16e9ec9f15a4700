// DECODE + aggregate (App. A decoding; Algorithm 1, aggregation line): the K
// workers' containers are decoded and summed into one fp32 vector.
//
// Work is handed out by ticket in warp-sized units: S consecutive sub-blocks of a
// tile of up to 8192 output elements (32 coding sub-blocks), for G streams at a
// time (G = 8, or 1 / 2 / 4 when K is smaller; S = 32 / G).  A warp keeps the
// running sums of its S * 256 elements in shared memory and writes them to HBM
// once; warps never wait for one another, and the ticket of the next unit is
// asked for while the current one is decoded.  Per unit and group of streams:
//
//   describe lane (j, q) reads, for stream j and sub-block q of the unit, the block
//            offset, the norm and the sub-block token lengths, range-checks them and
//            so knows where its chain of tokens starts and ends.
//   stage    every lane copies the next 12 words of its chain to shared memory, all
//            loads in flight at once: the walk is a chain of dependent reads, which
//            from global memory would wait for the cache at every step.  A lane that
//            uses its words up stages the next ones and goes on.
//   decode   the lane walks that chain: ERC^-1 gap by table look-up on a 32-bit window
//            (12-bit prefix table), then sign and ERC^-1 level index (one 8-bit
//            look-up for exponential levels, else the 12-bit table again; longer codes
//            take the loop of Algorithm 2).  All 32 chains of a warp advance in lock
//            step; the decoded (position, sign, index) triples go to a per-lane list.
//   add      for j = 0 .. G-1 in order, the warp adds the listed values of
//            stream j into its sums.  Entries of one stream hit distinct elements,
//            so the adds are plain shared-memory updates, and every element receives
//            its terms in ascending stream order: the sum is bit-reproducible and
//            equals ((0 + q_0) + q_1) + ... .
//
// Lists hold 48 entries per chain.  Sparse streams need one decode / add round per
// unit; when the longest chain is expected to hold more tokens, the sub-block is split
// evenly into rounds of positions, and a round whose list runs over is taken again with
// half the positions.  All terms of an element fall into the same round, so the order
// of its adds is unchanged; streams in the fixed-width mode add, in their turn, the
// fields of the positions the round covers.  One CTA per SM holds up to 25 such warps;
// they share only the tables and the validated stream headers.  Nothing spins.
//
// Calls whose streams are all in the fixed-width mode have no chains to walk; they are
// served by a kernel of their own (decode_fixed_kernel below).  A stream whose level indices
// are written in a fitted prefix code (Sec. 5, "efficient encoding") brings the code lengths
// in its header; the CTA builds a small table from them and the stream's lanes look their
// level indices up there instead of in the ERC^-1 table, in the same loop.
#include <type_traits>

#include "nuq_common.cuh"
#include "nuq_launch.h"

namespace nuq {

constexpr uint32_t kLutBits = 12;                       // prefix bits resolved by the ERC^-1 table
constexpr uint32_t kWarpWords = 1152;                   // shared-memory words a warp has for lists and staged tokens
constexpr uint32_t kStageWords = 12;                    // token words per chain copied to shared memory before the walk
constexpr uint32_t kStagedListWords = kWarpWords - 32u * kStageWords;   // what is left for the lists then (48 entries per chain)
constexpr uint32_t kStageSoftBits = 32u * (kStageWords - 2u);   // a lane stops here when its chain goes on behind the staged words
constexpr uint32_t kDecMaxWarps = 25;                   // warps per CTA = per SM (they share the table and the stream heads only)

// One Elias-recursive integer from the top of a 64-bit MSB-first window (Algorithm 2,
// decoding): N = 1; while the next bit is 1, read that bit plus N more as the new N.
__device__ __forceinline__ bool erc_read(uint64_t& win, uint32_t& used, uint32_t& value) {
    uint32_t N = 1;
#pragma unroll 1
    for (int it = 0; it < 6; ++it) {
        if (!(win >> 63)) {
            win <<= 1;
            used += 1;
            value = N;
            return true;
        }
        uint32_t nb = N + 1u;
        if (nb > 32u) return false;
        N = (uint32_t)(win >> (64u - nb));
        win <<= nb;
        used += nb;
    }
    return false;
}

// 64 bits of the MSB-first bit string whose word i is word(i), starting at bit `cur`; word indices are
// clamped to `last`.
template <class Fetch>
__device__ __forceinline__ uint64_t window64(Fetch word, uint32_t cur, uint32_t last) {
    uint32_t wi = cur >> 5, sh = cur & 31u;
    uint32_t w0 = word(min(wi, last));
    uint32_t w1 = word(min(wi + 1u, last));
    uint32_t w2 = word(min(wi + 2u, last));
    uint64_t win = ((uint64_t)w0 << 32 | w1) << sh;
    if (sh) win |= (uint64_t)w2 >> (32u - sh);
    return win;
}

// `hdr`: the container (a level-table stream carries its s interior levels behind the 16 header words)
__device__ __forceinline__ float level_times_norm(float norm, uint32_t levelset, uint32_t s, uint32_t sym, const uint32_t* hdr) {
    // exponential: l_j = 2^(j-1-s) (exact scaling);  uniform: l_k = k / 2^s;  table: l_j as stored, l_{s+1} = 1
    float level;
    if (levelset == kLevelsExp) level = __uint_as_float((126u + sym - s) << 23);
    else if (levelset == kLevelsUniform) level = (float)sym * __uint_as_float((127u - s) << 23);
    else level = sym <= s ? __uint_as_float(__ldg(hdr + kHeaderWords + sym - 1u)) : 1.0f;
    return __fmul_rn(norm, level);
}

// ---------------------------------------------------------------------------
// What happens to the finished sum G = sum_k DECODE(c_k) of an element: it is stored to acc (if there is
// one) and, when the call carries the aggregation step of Algorithm 1, applied to the parameters at once,
// so that the sum is not written out and read again by an optimizer kernel:
//     y = w - (alpha / K) G,   y^l = w - l (alpha / K) G,   w <- y + mu (y^l - y^l_prev)
// (Sec. 4, "NUQSGD with momentum"; mu = 0 is Algorithm 1's own line and leaves y^l alone).  fp32, each line
// one fused multiply-add.
// ---------------------------------------------------------------------------
__device__ __forceinline__ float step_value(const DecodeParams& P, float w, float G, float* yl) {
    const float y = __fmaf_rn(-P.step_c, G, w);
    if (P.mu == 0.0f) return y;
    const float yl_next = __fmaf_rn(-P.step_lc, G, w);
    const float w_next = __fmaf_rn(P.mu, __fsub_rn(yl_next, *yl), y);
    *yl = yl_next;
    return w_next;
}
// element e (a multiple of 4) and the three behind it
__device__ __forceinline__ void finish4(const DecodeParams& P, uint64_t e, float4 G, bool store_sum = true) {
    if (store_sum && P.acc) *reinterpret_cast<float4*>(P.acc + e) = G;
    if (P.w) {
        float4 w = *reinterpret_cast<const float4*>(P.w + e);
        float4 yl = make_float4(0.f, 0.f, 0.f, 0.f);
        if (P.mu != 0.0f) yl = *reinterpret_cast<const float4*>(P.yl + e);
        w.x = step_value(P, w.x, G.x, &yl.x);
        w.y = step_value(P, w.y, G.y, &yl.y);
        w.z = step_value(P, w.z, G.z, &yl.z);
        w.w = step_value(P, w.w, G.w, &yl.w);
        *reinterpret_cast<float4*>(P.w + e) = w;
        if (P.mu != 0.0f) *reinterpret_cast<float4*>(P.yl + e) = yl;
    }
}
__device__ __forceinline__ void finish1(const DecodeParams& P, uint64_t e, float G, bool store_sum = true) {
    if (store_sum && P.acc) P.acc[e] = G;
    if (P.w) {
        float yl = P.mu != 0.0f ? P.yl[e] : 0.0f;
        P.w[e] = step_value(P, P.w[e], G, &yl);
        if (P.mu != 0.0f) P.yl[e] = yl;
    }
}

// ERC^-1 of an nbits-bit prefix: value | length << 8, or 0 when the code is longer than the prefix
// (or is not a code).  Obtained by running Algorithm 2's decoder on the prefix.
__device__ __forceinline__ uint32_t erc_prefix_entry(uint32_t idx, uint32_t nbits) {
    uint32_t N = 1, pos = 0;
    for (int it = 0; it < 6; ++it) {
        if (pos >= nbits) return 0;
        if (!((idx >> (nbits - 1u - pos)) & 1u)) return N | ((pos + 1u) << 8);
        const uint32_t nb = N + 1u;
        if (pos + nb > nbits) return 0;
        N = (idx >> (nbits - pos - nb)) & ((1u << nb) - 1u);
        pos += nb;
    }
    return 0;
}

// Sign and level index of a token from its next 8 bits (sign bit, then ERC(index) of at most 7 bits,
// i.e. index <= 15): the upper byte of the token's list entry, (index - 1) << 9 | sign << 8, and in
// the low byte the bits consumed; 0 when the code is longer.
constexpr uint32_t kSignedBits = 8;
__device__ __forceinline__ uint32_t signed_index_entry(uint32_t idx) {
    const uint32_t r = erc_prefix_entry(idx & 0x7fu, kSignedBits - 1u);
    if (r == 0) return 0;
    return (((r & 0xffu) - 1u) << 9) | ((idx >> 7) << 8) | ((r >> 8) + 1u);
}

// What a lane needs to know to walk sub-block `sb` of one stream.
struct Chain {
    const uint32_t* tok;     // ERC: token words of the sub-block's coding block;  fixed: field words of its bucket
    float norm;
    uint32_t cur, end;       // ERC: first and past-the-end bit of the chain;  fixed: bit of the first field, unused
    uint32_t last;           // last valid word index behind tok
};

// Per stream of the call: what its header says, checked once per CTA.
struct StreamHead {
    const uint32_t* hdr;
    uint64_t cwords;         // container words the header declares
    uint32_t ok, mode, levelset, nlev, width;
    uint32_t hwords;         // header words: 16, plus the level table of a level-table stream
};

// Where a tile lies in the vector and in the containers.
struct TileGeo {
    uint64_t elem0, first_block, bucket_idx;
    uint32_t tile_len, spb, blk_elems, bib, nsb_tile;
};

// Descriptor of sub-block `sb` of the tile in stream `hd` (header already validated): block offsets
// from the table, norm, the chain's place from the sub-block lengths; everything is range-checked.
// Returns false when the container is malformed there.
__device__ bool describe_chain(const Geometry& G, const TileGeo& T, const StreamHead& hd, uint32_t sb, Chain* out) {
    Chain ch;
    ch.tok = hd.hdr;
    ch.norm = 0.0f;
    ch.cur = ch.end = ch.last = 0;
    *out = ch;
    if (sb >= T.nsb_tile) return true;
    const uint32_t bi = sb / T.spb, sb0 = bi * T.spb, sbi = sb - sb0;
    const uint32_t blk_len = min(T.blk_elems, T.tile_len - min(T.tile_len, bi * T.blk_elems));
    const uint32_t nsb_blk = (blk_len + kSB - 1) / kSB;
    if (hd.mode != kModeFixed) {
        const uint64_t head = hd.hwords + 2 * (G.nblk + 1);
        const uint64_t* table = reinterpret_cast<const uint64_t*>(hd.hdr + hd.hwords);
        const uint32_t* payload = hd.hdr + head;
        const uint64_t payload_words = hd.cwords - head;
        const uint64_t off = __ldg(table + T.first_block + bi), end = __ldg(table + T.first_block + bi + 1);
        const uint32_t head_words = 1u + (nsb_blk + 1u) / 2u;
        if (!((off & 31u) == 0 && (end & 31u) == 0 && off < end && (end >> 5) <= payload_words &&
              ((end - off) >> 5) >= head_words && ((end - off) >> 5) <= (1u << 20)))
            return false;
        const uint32_t* rec = payload + (off >> 5);
        const uint32_t tok_words = (uint32_t)((end - off) >> 5) - head_words;
        // start of the chain = sum of the lengths of the earlier sub-blocks of its block
        uint32_t cur = 0, len = 0;
        for (uint32_t w = 0; 2u * w <= sbi; ++w) {
            const uint32_t word = __ldg(rec + 1u + w), lo = word & 0xffffu, hi = word >> 16;
            if (2u * w < sbi) cur += lo; else len = lo;
            if (2u * w + 1u < sbi) cur += hi; else if (2u * w + 1u == sbi) len = hi;
        }
        if (cur + len > 32u * tok_words) return false;
        ch.norm = __uint_as_float(__ldg(rec));
        ch.tok = rec + head_words;
        ch.cur = cur;
        ch.end = cur + len;
        ch.last = tok_words ? tok_words - 1u : 0u;
    } else {
        const uint32_t rec_words = 1u + (G.bucket * hd.width + 31u) / 32u;
        const uint64_t last_len = G.d - (G.nb - 1) * G.bucket;
        const uint32_t* payload = hd.hdr + hd.hwords;
        const uint64_t bucket_of_sb = G.bucket <= kBLK ? T.first_block + bi : T.bucket_idx;
        const uint32_t* rec = payload + bucket_of_sb * rec_words;
        const uint64_t bucket_len = bucket_of_sb == G.nb - 1 ? last_len : G.bucket;
        ch.norm = __uint_as_float(__ldg(rec));
        ch.tok = rec + 1;
        ch.cur = (G.bucket <= kBLK ? sbi * kSB : T.bib * kBLK + sb * kSB) * hd.width;   // bit of the first field
        ch.last = (uint32_t)((bucket_len * hd.width + 31) / 32) - 1u;
    }
    *out = ch;
    return true;
}

// A container's header checked against the call's arguments.
__device__ StreamHead read_head(const Geometry& G, const uint32_t* hdr) {
    const uint32_t flags = __ldg(hdr + 6);
    const uint32_t levelset = (flags >> 8) & 0xffu, mode = (flags >> 16) & 0xffu;
    const uint64_t hd = (uint64_t)__ldg(hdr + 2) | ((uint64_t)__ldg(hdr + 3) << 32);
    const uint64_t hnblk = (uint64_t)__ldg(hdr + 8) | ((uint64_t)__ldg(hdr + 9) << 32);
    const uint64_t cbits = (uint64_t)__ldg(hdr + 10) | ((uint64_t)__ldg(hdr + 11) << 32);
    bool ok = __ldg(hdr) == kMagic && __ldg(hdr + 1) == kVersion && hd == G.d && __ldg(hdr + 4) == G.bucket &&
              __ldg(hdr + 5) == G.s && __ldg(hdr + 7) == kSB && levelset <= 2u && mode <= 2u &&
              (flags & 0xffu) <= 1u && !(levelset == kLevelsUniform && G.s > 8u) && (cbits & 31u) == 0;
    const uint32_t nlev = levelset == kLevelsUniform ? (1u << G.s) + 1u : G.s + 2u;
    const uint32_t hwords = kHeaderWords + (levelset == kLevelsTable ? ((G.s + 1u) & ~1u) : 0u) + (mode == kModeCoded ? 2u : 0u);
    if (ok && mode == kModeCoded) {                         // the lengths must be those of a prefix code of at most 7 bits
        ok = levelset != kLevelsUniform && G.s <= kMaxCodedS;
        uint32_t kraft = 0;
        for (uint32_t j = 0; ok && j <= G.s; ++j) {
            const uint32_t len = (__ldg(hdr + hwords - 2u + (j >> 2)) >> (8u * (j & 3u))) & 0xffu;
            ok = len >= 1u && len <= kMaxCodedS;
            kraft += ok ? 1u << (kMaxCodedS - len) : 0u;
        }
        ok = ok && kraft <= (1u << kMaxCodedS);
    }
    if (ok && levelset == kLevelsTable) {                   // the levels must increase strictly inside (0, 1)
        float below = 0.0f;
        for (uint32_t j = 0; j < G.s; ++j) {
            const float l = __uint_as_float(__ldg(hdr + kHeaderWords + j));
            ok = ok && below < l;
            below = l;
        }
        ok = ok && below < 1.0f;
    }
    const uint32_t width = 1u + (32u - __clz(nlev - 1u));                   // fixed mode: sign bit + ceil(log2(levels))
    const uint64_t cwords = cbits >> 5;
    if (ok && mode != kModeFixed) {
        ok = hnblk == G.nblk && cwords > hwords + 2 * (G.nblk + 1);
    } else if (ok) {
        const uint32_t rec_words = 1u + (G.bucket * width + 31u) / 32u;
        const uint64_t last_len = G.d - (G.nb - 1) * G.bucket;
        ok = hnblk == G.nb &&
             cwords == hwords + (G.nb - 1) * (uint64_t)rec_words + 1 + (last_len * width + 31) / 32;
    }
    StreamHead h;
    h.hdr = hdr; h.cwords = cwords; h.ok = ok ? 1u : 0u; h.mode = mode; h.levelset = levelset;
    h.nlev = nlev; h.width = width; h.hwords = hwords;
    return h;
}

// All streams in the fixed-width mode with the same field width W (sign bit + level index, MSB first):
// no tokens to walk, so a thread takes 32 consecutive elements (W words of every stream, never across a
// bucket: buckets are multiples of 256 elements), adds the K dequantized values of each element in
// stream order in registers and stores the 32 sums.  Same arithmetic and order as the general path.
template <uint32_t W, uint32_t LEVELSET>
__device__ __forceinline__ void decode_all_fixed(const DecodeParams& P, const StreamHead* heads) {
    const Geometry& G = P.geo;
    const uint64_t ngroups = (G.d + 31) / 32;
    const uint32_t nlev = heads[0].nlev;
    const uint32_t exp_bias = (126u - G.s) << 23;           // exponent field of 2^(-1-s)
    const float uni_scale = __uint_as_float((127u - G.s) << 23);
    uint32_t max_sym = 0;
    const uint32_t rec_words = 1u + G.bucket * W / 32u;
    const uint64_t last_len = G.d - (G.nb - 1) * G.bucket;
    constexpr uint32_t fmask = (1u << W) - 1u, smask = (1u << (W - 1u)) - 1u;
    for (uint64_t grp = (uint64_t)blockIdx.x * blockDim.x + threadIdx.x; grp < ngroups; grp += (uint64_t)gridDim.x * blockDim.x) {
        const uint64_t e0 = 32 * grp, b = e0 / G.bucket;
        const uint32_t eb = (uint32_t)(e0 - b * G.bucket);                         // first element within its bucket
        const uint32_t nel = G.d - e0 < 32 ? (uint32_t)(G.d - e0) : 32u;
        const uint32_t bucket_len = b == G.nb - 1 ? (uint32_t)last_len : G.bucket;
        const uint32_t avail = (bucket_len * W + 31u) / 32u - (eb / 32u) * W;      // field words of the record from here on
        float* dst = P.acc + e0;
        // branch free: a zero symbol adds +0 (the sums never are -0, so that changes nothing), the
        // largest symbol seen is checked once at the end; `whole`: all 32 elements exist
        auto body = [&](auto whole) {
#pragma unroll
            for (uint32_t half = 0; half < 2; ++half) {     // 16 elements at a time: the sums stay in few registers
                float acc[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) acc[i] = 0.0f;
                for (uint32_t k = 0; k < P.K; ++k) {
                    const uint32_t* rec = heads[k].hdr + kHeaderWords + b * rec_words;
                    const float norm = __uint_as_float(__ldg(rec));
                    const uint32_t* fw = rec + 1u + (eb / 32u) * W;
                    // the words that hold fields 16 * half .. 16 * half + 15
                    constexpr uint32_t kHalfWords = (16u * W + 31u) / 32u + 1u;
                    const uint32_t w0 = (16u * half * W) >> 5;
                    uint32_t words[kHalfWords + 1];
#pragma unroll
                    for (uint32_t j = 0; j < kHalfWords; ++j) words[j] = w0 + j < avail ? __ldg(fw + w0 + j) : 0u;
                    words[kHalfWords] = 0;
#pragma unroll
                    for (uint32_t i = 0; i < 16; ++i) {
                        const uint32_t bit = (16u * half + i) * W - 32u * w0, a = bit >> 5, sh = bit & 31u;
                        const uint32_t field = sh + W <= 32u ? (words[a] >> (32u - sh - W)) & fmask
                                                             : __funnelshift_l(words[a + 1], words[a], sh) >> (32u - W);
                        const uint32_t sym = field & smask;
                        // exponential: l_j = 2^(j-1-s) (exact scaling);  uniform: l_k = k / 2^s
                        const float level = LEVELSET == kLevelsExp ? __uint_as_float((sym << 23) + exp_bias)
                                                                   : __fmul_rn((float)sym, uni_scale);
                        const float mag = sym ? __fmul_rn(norm, level) : 0.0f;
                        const float v = __uint_as_float(__float_as_uint(mag) ^ ((field << (32u - W)) & 0x80000000u));
                        if (decltype(whole)::value || 16u * half + i < nel) {
                            max_sym = max(max_sym, sym);
                            acc[i] += v;
                        }
                    }
                }
                if (decltype(whole)::value) {
#pragma unroll
                    for (int i = 0; i < 16; i += 4)
                        *reinterpret_cast<float4*>(dst + 16 * half + i) = make_float4(acc[i], acc[i + 1], acc[i + 2], acc[i + 3]);
                } else {
#pragma unroll
                    for (int i = 0; i < 16; ++i)
                        if (16u * half + (uint32_t)i < nel) dst[16 * half + i] = acc[i];
                }
            }
        };
        if (nel == 32u) body(std::true_type());
        else body(std::false_type());
    }
    if (max_sym >= nlev) latch_status(P.ws, kErrBadStream);
}

// The same for the 4-bit fields of the paper's "4-bit" variant (exponential levels with s = 3 .. 6; a
// sign bit and a 3-bit level index) and buckets that are multiples of 2048 elements, where almost all
// the work can be taken out of the inner loop: a CTA takes a tile of up to 8192 elements of one bucket
// by ticket, builds, per stream, the table of the 16 values a field can stand for (+-norm * level, the
// same multiplication as everywhere else, so the sums are bit-identical), and then every thread turns 8
// consecutive elements -- one word of every stream -- into table look-ups and adds, in stream order.
// Symbols that do not exist are found on whole words (a carry out of the index bits).
template <uint32_t LEVELSET>
__device__ __forceinline__ void decode_fixed4_tiles(const DecodeParams& P, const StreamHead* heads) {
    __shared__ float s_tab[kMaxK][16];
    __shared__ unsigned long long s_ticket;
    const Geometry& G = P.geo;
    const uint32_t K = P.K, tid = threadIdx.x;
    const uint32_t nlev = heads[0].nlev;                    // <= 8
    const uint32_t rec_words = 1u + G.bucket / 8u;
    const uint32_t tile_elems = G.bucket < kBLK ? G.bucket : kBLK;
    const uint32_t tiles_per_bucket = G.bucket / tile_elems;
    const uint64_t ntiles = G.nb * tiles_per_bucket;
    const uint64_t last_len = G.d - (G.nb - 1) * G.bucket;
    const uint32_t over = (8u - nlev) * 0x11111111u;        // added to the index bits, a missing symbol carries into bit 3
    uint32_t bad = 0;
    for (;;) {
        __syncthreads();                                    // the tables and the ticket of the previous tile are no longer read
        if (tid == 0) s_ticket = atomicAdd(reinterpret_cast<unsigned long long*>(&P.ws->dec_ticket[P.epoch & 1u]), 1ull);
        __syncthreads();
        const uint64_t tile = s_ticket;
        if (tile >= ntiles) break;
        const uint64_t b = tile / tiles_per_bucket;
        const uint32_t part = (uint32_t)(tile % tiles_per_bucket);
        const uint32_t bucket_len = b == G.nb - 1 ? (uint32_t)last_len : G.bucket;
        const uint32_t first = part * tile_elems;           // first element of the tile within its bucket
        if (first >= bucket_len) continue;
        const uint32_t tile_len = bucket_len - first < tile_elems ? bucket_len - first : tile_elems;
        for (uint32_t t = tid; t < 16u * K; t += blockDim.x) {
            const uint32_t k = t >> 4, f = t & 15u, sym = f & 7u;
            const float norm = __uint_as_float(__ldg(heads[k].hdr + kHeaderWords + b * rec_words));
            const float v = sym && sym < nlev ? level_times_norm(norm, LEVELSET, G.s, sym, heads[k].hdr) : 0.0f;
            s_tab[k][f] = (f & 8u) ? -v : v;
        }
        __syncthreads();
        float* const dst_tile = P.acc + b * G.bucket + first;
        const uint64_t word0 = kHeaderWords + b * rec_words + 1u + first / 8u;     // the tile's first field word in a container
        // Two groups of eight elements per thread and step (el and el + 8 * blockDim.x): the words of both are
        // asked for before either is used, which keeps twice as many loads in flight.
        const uint32_t stride = 8u * blockDim.x;
        for (uint32_t el = 8u * tid; el < tile_len; el += 2u * stride) {
            const bool second = el + stride < tile_len;
            float sum[2][8];
#pragma unroll
            for (int h = 0; h < 2; ++h)
#pragma unroll
                for (int i = 0; i < 8; ++i) sum[h][i] = 0.0f;
            for (uint32_t k0 = 0; k0 < K; k0 += 8u) {
                uint32_t wv[2][8];
#pragma unroll
                for (uint32_t j = 0; j < 8; ++j) {
                    const uint32_t* w = heads[k0 + j < K ? k0 + j : 0u].hdr + word0 + el / 8u;
                    wv[0][j] = k0 + j < K ? __ldg(w) : 0u;
                    wv[1][j] = k0 + j < K && second ? __ldg(w + blockDim.x) : 0u;
                }
#pragma unroll
                for (uint32_t j = 0; j < 8; ++j) {
                    if (k0 + j < K) {
                        const char* tab = reinterpret_cast<const char*>(s_tab[k0 + j]);
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            const uint32_t x = wv[h][j];
                            bad |= ((x & 0x77777777u) + over) & 0x88888888u;
                            // the eight fields times four (byte offsets into the table), four to a register
                            const uint32_t a = (x >> 2) & 0x3C3C3C3Cu, c = (x << 2) & 0x3C3C3C3Cu;   // elements 0 2 4 6 / 1 3 5 7 from the top byte
                            sum[h][0] += *reinterpret_cast<const float*>(tab + __byte_perm(a, 0u, 0x4443));
                            sum[h][1] += *reinterpret_cast<const float*>(tab + __byte_perm(c, 0u, 0x4443));
                            sum[h][2] += *reinterpret_cast<const float*>(tab + __byte_perm(a, 0u, 0x4442));
                            sum[h][3] += *reinterpret_cast<const float*>(tab + __byte_perm(c, 0u, 0x4442));
                            sum[h][4] += *reinterpret_cast<const float*>(tab + __byte_perm(a, 0u, 0x4441));
                            sum[h][5] += *reinterpret_cast<const float*>(tab + __byte_perm(c, 0u, 0x4441));
                            sum[h][6] += *reinterpret_cast<const float*>(tab + __byte_perm(a, 0u, 0x4440));
                            sum[h][7] += *reinterpret_cast<const float*>(tab + __byte_perm(c, 0u, 0x4440));
                        }
                    }
                }
            }
#pragma unroll
            for (int h = 0; h < 2; ++h) {
                const uint32_t e0 = el + h * stride;
                if (h == 1 && !second) break;
                float* dst = dst_tile + e0;
                if (e0 + 8u <= tile_len) {
                    *reinterpret_cast<float4*>(dst) = make_float4(sum[h][0], sum[h][1], sum[h][2], sum[h][3]);
                    *reinterpret_cast<float4*>(dst + 4) = make_float4(sum[h][4], sum[h][5], sum[h][6], sum[h][7]);
                } else {
#pragma unroll
                    for (uint32_t i = 0; i < 8; ++i)
                        if (e0 + i < tile_len) dst[i] = sum[h][i];
                }
            }
        }
    }
    if (bad) latch_status(P.ws, kErrBadStream);
}

// The kernel of that path.  It is launched when the library believes that all streams are in the
// fixed-width mode (it wrote them itself) and the call wants the sums only (a call that carries the
// aggregation step takes the general kernel, which applies it); it checks the headers like the general kernel and, if they
// say otherwise, leaves everything to the general kernel, which is launched behind it in any case and
// returns at once when this one has done the work.
__global__ void __launch_bounds__(256) decode_fixed_kernel(const __grid_constant__ DecodeParams P) {
    __shared__ StreamHead heads[kMaxK];
    __shared__ uint32_t s_width;
    for (uint32_t k = threadIdx.x; k < P.K; k += blockDim.x) heads[k] = read_head(P.geo, P.streams[k]);
    __syncthreads();
    if (threadIdx.x == 0) {
        bool same = true;
        for (uint32_t k = 0; k < P.K; ++k)
            same = same && heads[k].ok && heads[k].mode == kModeFixed && heads[k].levelset == heads[0].levelset &&
                   heads[k].levelset != kLevelsTable;       // (streams with a level table take the general kernel)
        s_width = same ? heads[0].width : 0u;
        if (same && blockIdx.x == 0) *reinterpret_cast<volatile uint32_t*>(&P.ws->dec_done_epoch) = P.epoch;   // tell the general kernel
        if (blockIdx.x == 0) P.ws->dec_ticket[(P.epoch & 1u) ^ 1u] = 0;     // the next call's counter (nobody uses it during this call)
    }
    __syncthreads();
    if (heads[0].levelset == kLevelsExp) {                  // s <= 14: at most 16 levels, 5 bits
        switch (s_width) {
            case 3: decode_all_fixed<3, kLevelsExp>(P, heads); break;
            case 4:
                if (P.geo.bucket % 2048u == 0) decode_fixed4_tiles<kLevelsExp>(P, heads);
                else decode_all_fixed<4, kLevelsExp>(P, heads);
                break;
            case 5: decode_all_fixed<5, kLevelsExp>(P, heads); break;
            default: break;
        }
        return;
    }
    switch (s_width) {
        case 3: decode_all_fixed<3, kLevelsUniform>(P, heads); break;
        case 4: decode_all_fixed<4, kLevelsUniform>(P, heads); break;
        case 5: decode_all_fixed<5, kLevelsUniform>(P, heads); break;
        case 6: decode_all_fixed<6, kLevelsUniform>(P, heads); break;
        case 7: decode_all_fixed<7, kLevelsUniform>(P, heads); break;
        case 8: decode_all_fixed<8, kLevelsUniform>(P, heads); break;
        case 9: decode_all_fixed<9, kLevelsUniform>(P, heads); break;
        case 10: decode_all_fixed<10, kLevelsUniform>(P, heads); break;
        default: break;
    }
}

// A stream with coded level indices brings its own code: per stream a table over the next 7 bits in the
// format of the ERC^-1 table, index | length << 8, or 0 where no code word starts (possible only with
// an incomplete code).  A lane of such a stream looks its level index up there instead.
constexpr uint32_t kCodedEntries = 1u << kMaxCodedS;
__device__ __forceinline__ void build_coded_table(const StreamHead& hd, uint16_t* tab, uint32_t s, uint32_t tid, uint32_t nthreads) {
    const uint32_t w0 = __ldg(hd.hdr + hd.hwords - 2u), w1 = __ldg(hd.hdr + hd.hwords - 1u);   // the lengths, one byte each
    auto len_of = [&](uint32_t j) { return ((j < 4u ? w0 : w1) >> (8u * (j & 3u))) & 0xffu; };
    for (uint32_t i = tid; i < kCodedEntries; i += nthreads) {
        uint32_t e = 0;
        for (uint32_t j = 0; j <= s; ++j) {
            // canonical words: level indices by (length, index), the first word all zeros, each next one the
            // previous plus one; so the word of j counts, in units of its own length, the words before it
            const uint32_t lj = len_of(j);
            uint32_t word = 0;
            for (uint32_t k = 0; k <= s; ++k) {
                const uint32_t lk = len_of(k);
                if (lk < lj || (lk == lj && k < j)) word += 1u << (lj - lk);
            }
            if ((i >> (kMaxCodedS - lj)) == word) e = (j + 1u) | (lj << 8);
        }
        tab[i] = (uint16_t)e;
    }
}

// shared memory: the two ERC^-1 tables, the stream heads, the streams' own code tables, then per warp the running sums of its S sub-blocks
// and kWarpWords for lists and staged tokens
__host__ __device__ inline size_t decode_warp_offset(uint32_t K) {
    return (2u * ((1u << kLutBits) + (1u << kSignedBits)) + (size_t)K * (sizeof(StreamHead) + 2u * kCodedEntries) + 15u) & ~(size_t)15u;
}
// `sums_in_l2`: the running sums of a unit live in the output vector itself (see decode_kernel)
__host__ __device__ inline size_t decode_warp_bytes(uint32_t group, bool sums_in_l2) {
    return 4u * ((sums_in_l2 ? 0u : (32u / group) * kSB) + kWarpWords);
}

// SUMS_IN_L2 = false: a warp keeps the running sums of its S * 256 elements in shared memory and
// stores them once (8 streams side by side: 4 KB per warp).  true: it zeroes its part of the output
// vector and adds into it there, in the L2, with cache-global loads and stores; taken for fewer than
// 8 streams, where the sums of a warp would need 8 to 32 KB of shared memory and only a few warps
// would fit an SM, too few to hide the latency of the walk.  The order of the adds is the same.
// (Taken for one or two streams side by side; with four, 17 warps fit and shared memory is faster.)
template <bool SUMS_IN_L2>
__global__ void __launch_bounds__(32 * (SUMS_IN_L2 ? kDecMaxWarps - 1 : kDecMaxWarps)) decode_kernel(const __grid_constant__ DecodeParams P) {
    extern __shared__ __align__(16) unsigned char dsm[];
    // Behind the fixed-width kernel this one is launched with programmatic stream serialization: its launch is
    // worked off while that kernel still runs, and it waits here until that kernel's writes are visible.
    if (P.after_fixed) asm volatile("griddepcontrol.wait;" ::: "memory");
    if (P.after_fixed && *reinterpret_cast<volatile uint32_t*>(&P.ws->dec_done_epoch) == P.epoch) return;   // the fixed-width kernel did it all
    if (blockIdx.x == 0 && threadIdx.x == 0) P.ws->dec_ticket[(P.epoch & 1u) ^ 1u] = 0;   // the next call's counter (nobody uses it during this call)
    const Geometry& G = P.geo;
    const uint32_t NG = P.group;                            // streams decoded side by side (1, 2, 4 or 8)
    const uint32_t S = 32u / NG;                            // sub-blocks per warp
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5;
    uint16_t* lut = reinterpret_cast<uint16_t*>(dsm);                             // ERC^-1 of 12-bit prefixes
    uint16_t* lut2 = lut + (1u << kLutBits);                                      // sign + ERC^-1 of 7-bit prefixes
    StreamHead* heads = reinterpret_cast<StreamHead*>(lut2 + (1u << kSignedBits));   // [K]
    uint16_t* coded_tabs = reinterpret_cast<uint16_t*>(heads + P.K);                 // [K][128], filled for streams with coded level indices
    float* accw = reinterpret_cast<float*>(dsm + decode_warp_offset(P.K) + warp * decode_warp_bytes(NG, SUMS_IN_L2));   // S * 256 running sums
    uint32_t* list = reinterpret_cast<uint32_t*>(accw + (SUMS_IN_L2 ? 0u : S * kSB));

    for (uint32_t i = threadIdx.x; i < (1u << kLutBits); i += blockDim.x) lut[i] = (uint16_t)erc_prefix_entry(i, kLutBits);
    for (uint32_t i = threadIdx.x; i < (1u << kSignedBits); i += blockDim.x) lut2[i] = (uint16_t)signed_index_entry(i);
    // ---- header validation against the call's arguments, once per stream ----
    for (uint32_t k = threadIdx.x; k < P.K; k += blockDim.x) {
        heads[k] = read_head(G, P.streams[k]);
        if (!heads[k].ok) latch_status(P.ws, kErrBadStream);
    }
    if (!SUMS_IN_L2)
        for (uint32_t i = lane * 4u; i < S * kSB; i += 128u)
            *reinterpret_cast<float4*>(accw + i) = make_float4(0.f, 0.f, 0.f, 0.f);

    __syncthreads();                                        // tables and headers are ready
    {
        bool any = false;
        for (uint32_t k = 0; k < P.K; ++k) {
            if (!(heads[k].ok && heads[k].mode == kModeCoded)) continue;
            build_coded_table(heads[k], coded_tabs + k * kCodedEntries, G.s, threadIdx.x, blockDim.x);
            any = true;
        }
        if (any) __syncthreads();                           // (the same streams in every thread)
    }
    // from here on warps run alone

    // Work is handed out one warp-sized unit at a time (S sub-blocks of one tile, all streams).  The
    // ticket of the next unit is asked for while the current one is decoded, except near the end: a
    // unit reserved by a warp that is busy with a long one would be started late.
    const uint64_t nunits = G.ntiles * NG;
    const uint64_t in_flight = 3ull * gridDim.x * (blockDim.x >> 5);
    const uint64_t reserve_until = nunits > in_flight ? nunits - in_flight : 0;
    unsigned long long next_unit = 0;
    bool have_next = false;
    for (;;) {
        if (!have_next && lane == 0) next_unit = atomicAdd(reinterpret_cast<unsigned long long*>(&P.ws->dec_ticket[P.epoch & 1u]), 1ull);
        const unsigned long long unit = __shfl_sync(0xffffffffu, next_unit, 0);
        if (unit >= nunits) break;
        const uint64_t tile = unit / NG;
        const uint32_t part = (uint32_t)(unit % NG);        // which S sub-blocks of the tile
        have_next = unit < reserve_until;
        if (have_next && lane == 0) next_unit = atomicAdd(reinterpret_cast<unsigned long long*>(&P.ws->dec_ticket[P.epoch & 1u]), 1ull);
        // ---- tile geometry (same tiling as the encoder) ---------------------------
        TileGeo T;
        T.bucket_idx = 0;
        T.bib = 0;
        if (G.bucket <= kBLK) {
            T.first_block = tile * G.blocks_per_tile;
            T.elem0 = T.first_block * G.bucket;
            const uint64_t left = G.d - T.elem0;
            T.tile_len = left < G.tile_elems ? (uint32_t)left : G.tile_elems;
            T.spb = G.sb_per_block;
            T.blk_elems = G.bucket;
        } else {
            T.bucket_idx = tile / G.blk_per_bucket;
            T.bib = (uint32_t)(tile % G.blk_per_bucket);
            T.first_block = tile;
            const uint64_t b0 = T.bucket_idx * G.bucket;
            const uint64_t blen = G.d - b0 < G.bucket ? G.d - b0 : G.bucket;
            T.elem0 = b0 + (uint64_t)T.bib * kBLK;
            const uint64_t left = blen - (uint64_t)T.bib * kBLK;
            T.tile_len = left < kBLK ? (uint32_t)left : kBLK;
            T.spb = 32;
            T.blk_elems = kBLK;
        }
        T.nsb_tile = (T.tile_len + kSB - 1) / kSB;
        const uint32_t tile_len = T.tile_len, nsb_tile = T.nsb_tile;
        const uint64_t elem0 = T.elem0;

        // the unit's part of the output vector and how many of its S * 256 elements exist
        float* const gsum = P.acc + elem0 + part * S * kSB;
        const uint32_t unit_len = tile_len > part * S * kSB ? min(S * kSB, tile_len - part * S * kSB) : 0u;
        if (SUMS_IN_L2) {
            for (uint32_t i = lane * 4u; i < unit_len; i += 128u) {
                if (i + 4u <= unit_len) __stcg(reinterpret_cast<float4*>(gsum + i), make_float4(0.f, 0.f, 0.f, 0.f));
                else for (uint32_t e = i; e < unit_len; ++e) __stcg(gsum + e, 0.0f);
            }
            __syncwarp();
        }
        // sum[idx] += v for element idx of the unit (a malformed chain may name an element that does not exist)
        auto add_to = [&](uint32_t idx, float v) {
            if (SUMS_IN_L2) {
                if (idx < unit_len) __stcg(gsum + idx, __ldcg(gsum + idx) + v);
            } else {
                accw[idx] += v;
            }
        };

        for (uint32_t g0 = 0; g0 < P.K; g0 += NG) {
            const uint32_t gcount = min(NG, P.K - g0);      // streams in this group

            // ================= decode + add, warp-local =================
            // lane (j, q): stream g0 + j, sub-block part * S + q
            const uint32_t lj = lane / S, lq = lane - lj * S;
            const uint32_t my_sb = part * S + lq;
            const uint32_t my_sn = my_sb < nsb_tile ? min(kSB, tile_len - my_sb * kSB) : 0u;   // elements of my sub-block
            bool wide = false;                              // index - 1 does not fit 7 bits (uniform levels, s = 8)
            bool small_index = true;                        // exponential levels, index <= 15: sign and index from one look-up
            for (uint32_t j = 0; j < gcount; ++j) {
                wide = wide || (heads[g0 + j].ok && heads[g0 + j].nlev > 129u);
                small_index = small_index && (!heads[g0 + j].ok || (heads[g0 + j].levelset == kLevelsExp && heads[g0 + j].nlev <= 16u));
            }
            const bool mine = lj < gcount;
            const StreamHead si = heads[g0 + (mine ? lj : 0)];
            Chain ch;                                       // each lane describes the chain it walks
            const bool chain_ok = describe_chain(G, T, si, mine && si.ok ? my_sb : 32u, &ch);
            if (__any_sync(0xffffffffu, !chain_ok) && lane == 0) latch_status(P.ws, kErrBadStream);
            const bool has_chain = mine && si.ok && chain_ok && si.mode != kModeFixed && my_sn > 0 && ch.cur < ch.end;
            // Level indices written with the stream's own code (Sec. 5, "efficient encoding"): such a lane
            // looks the index up in its stream's table (7-bit prefixes) instead of the ERC^-1 table (12-bit).
            // tab2: where the table starts, in entries from `lut`; sh2: 32 - its prefix bits.
            const bool my_coded = mine && si.ok && si.mode == kModeCoded;
            const uint32_t tab2 = my_coded ? (uint32_t)(coded_tabs - lut) + (g0 + lj) * kCodedEntries : 0u;
            const uint32_t sh2 = my_coded ? 32u - kMaxCodedS : 32u - kLutBits;
            small_index = small_index && !__any_sync(0xffffffffu, my_coded);

            // A round decodes, for all 32 chains at once, the tokens whose position lies below a limit,
            // and then adds them stream after stream; every element still receives its terms in ascending
            // stream order because all of its terms fall into the same round.  The walk reads the chain
            // from shared memory: every lane copies the next kStageWords words of its chain there, all
            // loads in flight at once (the walk is a chain of dependent reads, which from global memory
            // would wait for the cache at every step), and again whenever it has used them up.
            // Sparse data takes one round (limit = the whole sub-block).  When the longest chain is
            // expected to hold more tokens than a list (a chain of t tokens in 256 positions takes about
            // t (2 log2(256 / t) + 4) bits, 5 bits per token when it is dense), the sub-block is split
            // evenly into rounds, with a third of slack; a round in which a list runs over is taken again
            // with half the positions.
            const uint32_t cap = (wide ? kStagedListWords : 2u * kStagedListWords) / 32u;   // list entries per chain
            const uint32_t chain_bits = __reduce_max_sync(0xffffffffu, has_chain ? ch.end - ch.cur : 0u);
            uint32_t step = kSB;
            if (chain_bits > 9u * cap) {                    // 9 bits per token is what sparse chains take
                const uint32_t guess = chain_bits <= 512u ? chain_bits / 8u : chain_bits / 5u;
                const uint32_t rounds = max(2u, (guess + guess / 3u + cap - 1u) / cap);
                step = max(cap, (kSB + rounds - 1u) / rounds);
            }
            const uint32_t end = ch.end;
            bool alive = has_chain, bad = false;
            uint32_t cur = ch.cur, pos = 0, max_hi = 0;    // max_hi: the largest entry part (index - 1) << 9 | sign << 8 so far
            uint32_t* st = list + kStagedListWords + lane;   // word i of the staged part of my chain at st[32 i]
            uint16_t* slot16 = reinterpret_cast<uint16_t*>(list) + lane;
            uint32_t* slot32 = list + lane;
            uint32_t n = 0, limit = 0;
            uint32_t rbase = 0, rcur = 0, rlast = 0, rstop = 0;   // first staged bit; cursor, last word and stopping bit relative to it
            bool running = false;
            // One round of the walk over the staged words.
            auto walk = [&](auto wide_entries, auto one_lookup) {
                auto word = [st](uint32_t i) { return st[32u * i]; };
                // Every lane executes every step (a lane that has stopped works on stale but in-bounds
                // data and commits nothing): no divergent branch except the rare long-code path.
                while (__any_sync(0xffffffffu, running)) {
                    const uint32_t wi = rcur >> 5;
                    const uint32_t x0 = word(min(wi, rlast));
                    const uint32_t x1 = word(min(wi + 1u, rlast));
                    const uint32_t win = __funnelshift_l(x1, x0, rcur);                     // 32 bits from the cursor
                    const uint32_t e1 = lut[win >> (32u - kLutBits)];
                    const uint32_t t = win << (e1 >> 8);                                    // the sign bit is on top
                    uint32_t gap = e1 & 0xffu, used, hi;    // hi: (index - 1) << 9 | sign << 8
                    bool good;
                    if (decltype(one_lookup)::value) {
                        const uint32_t e2 = lut2[t >> (32u - kSignedBits)];
                        used = (e1 >> 8) + (e2 & 0xffu);
                        hi = e2 & 0xff00u;
                        good = e1 != 0 && e2 != 0;
                    } else {
                        const uint32_t e2 = lut[tab2 + ((t << 1) >> sh2)];   // the ERC^-1 table, or the stream's own
                        used = (e1 >> 8) + 1u + (e2 >> 8);
                        hi = ((t >> 31) << 8) | (((e2 & 0xffu) - 1u) << 9);
                        good = e1 != 0 && e2 != 0;
                    }
                    if (__any_sync(0xffffffffu, running && !good)) {
                        if (running && !good) {             // a code longer than the table's prefix: Algorithm 2 as a loop
                            uint64_t win64 = window64(word, rcur, rlast);
                            uint32_t sym = 1;
                            used = 0;
                            good = erc_read(win64, used, gap);
                            const uint32_t negative = (uint32_t)(win64 >> 63);
                            win64 <<= 1;
                            used += 1;
                            if (sh2 != 32u - kLutBits) {  // a stream with its own code: every word is in its table
                                const uint32_t c = lut[tab2 + (uint32_t)(win64 >> (64u - kMaxCodedS))];
                                good = good && c != 0;
                                used += c >> 8;
                                sym = c & 0xffu;
                            } else {
                                good = good && erc_read(win64, used, sym);
                            }
                            hi = (negative << 8) | ((min(sym, 0x10000u) - 1u) << 9);
                            if (!good) {                    // not a code at all: the chain is malformed
                                bad = true;
                                alive = false;
                            }
                        }
                    }
                    // Range checks are made once per chain, after the walk (see below): a token of a
                    // malformed chain may be committed, but its position is masked to the sub-block
                    // when it is added, so nothing is written out of bounds.
                    const uint32_t npos = pos + gap;
                    const bool commit = running && good && npos <= limit;   // beyond the limit: a later round's token
                    if (commit) {
                        max_hi = max(max_hi, hi);
                        const uint32_t e = ((npos - 1u) & 0xffu) | hi;
                        const uint32_t at = min(n, cap - 1u) * 32u;     // a list that runs over is noticed after the round
                        if (decltype(wide_entries)::value) slot32[at] = e;
                        else slot16[at] = (uint16_t)e;
                        pos = npos;
                        rcur += used;
                        ++n;
                    }
                    running = commit && rcur < rstop;
                }
            };
            for (;;) {
                const uint32_t done_pos = limit;            // positions below this have been added
                const uint32_t cur_s = cur, pos_s = pos, max_hi_s = max_hi;
                const bool alive_s = alive, bad_s = bad;
                limit = done_pos + step;
                n = 0;
                bool refill = alive;                        // lanes that stage the next words of their chain
                for (;;) {
                    // ---- stage, then walk until every lane has reached the limit, its chain's end or the
                    // end of its staged words; lanes of the last kind stage again and go on alone ----
                    if (refill) {
                        const uint32_t w0 = cur >> 5;
                        const uint32_t nws = min(kStageWords, ((end - 1u) >> 5) - w0 + 1u);     // up to the word that holds the chain's last bit
                        const uint32_t* src = ch.tok + w0;
#pragma unroll
                        for (uint32_t i = 0; i < kStageWords; ++i)
                            if (i < nws) st[i * 32u] = __ldg(src + i);
                        rbase = 32u * w0;
                        rcur = cur - rbase;
                        rlast = nws - 1u;
                        // go on while the cursor is before the chain's end or, when the chain is longer than
                        // the staged words, while two more words lie behind it (the long-code path looks that far)
                        rstop = end - rbase <= 32u * nws ? end - rbase : kStageSoftBits;
                    }
                    __syncwarp();
                    running = refill;
                    if (small_index) walk(std::false_type(), std::true_type());
                    else if (!wide) walk(std::false_type(), std::false_type());
                    else walk(std::true_type(), std::false_type());
                    cur = rbase + rcur;
                    alive = alive && !bad && cur < end;
                    refill = alive && rcur >= rstop && n <= cap;
                    if (!__any_sync(0xffffffffu, refill) || __any_sync(0xffffffffu, n > cap)) break;
                }
                // a list ran over: nothing of this round has been added yet, so take the round again from
                // where it started with half the positions (`cap` positions cannot run over)
                if (__any_sync(0xffffffffu, n > cap)) {
                    if (step <= cap) {                      // cannot happen
                        bad = true;
                        break;
                    }
                    step = max(cap, step / 2u);
                    limit = done_pos;
                    alive = alive_s;
                    bad = bad_s;
                    cur = cur_s;
                    pos = pos_s;
                    max_hi = max_hi_s;
                    continue;
                }
                __syncwarp();

                // ---- add, one stream after the other ----
                // Streams in the fixed-width mode have a term for every element; they add, in their turn,
                // those of the positions this round covers (all the remaining ones when no chain goes on).
                const bool more = __any_sync(0xffffffffu, alive);
                const uint32_t fixed_lo = done_pos, fixed_hi = more ? limit : kSB;
                const uint32_t per_chain = 32u / S;         // lanes that share one chain's list
                const uint32_t c = lane / per_chain, i0 = lane - c * per_chain;
                for (uint32_t j = 0; j < gcount; ++j) {
                    const StreamHead sj = heads[g0 + j];
                    const uint32_t owner = j * S + c;       // the lane that decoded chain (j, c)
                    const uint32_t n_c = __shfl_sync(0xffffffffu, n, owner);
                    const float norm_c = __shfl_sync(0xffffffffu, ch.norm, owner);
                    if (!sj.ok) continue;
                    if (sj.mode != kModeFixed) {
                        const uint32_t part0 = c * kSB;      // first element of chain c's sub-block within the unit
                        if (!wide && sj.levelset == kLevelsExp) {
                            // value = +-norm * 2^(index - 1 - s): the exponent field is built from the entry
                            const uint16_t* src = reinterpret_cast<const uint16_t*>(list) + owner;
                            const uint32_t ebias = 127u - G.s;              // (index - 1) + ebias = biased exponent
                            if (SUMS_IN_L2) {
                                // four entries at a time, loads before stores: the entries of one stream name
                                // distinct elements, and an add in the L2 is a round trip
                                for (uint32_t i = i0; i < n_c; i += 4u * per_chain) {
                                    uint32_t idx[4];
                                    float val[4], old[4];
#pragma unroll
                                    for (uint32_t u = 0; u < 4; ++u) {
                                        const uint32_t ii = i + u * per_chain;
                                        const uint32_t e = ii < n_c ? src[ii * 32u] : 0u;
                                        const float v = __fmul_rn(norm_c, __uint_as_float(((e >> 9) + ebias) << 23));
                                        val[u] = __uint_as_float(__float_as_uint(v) ^ ((e << 23) & 0x80000000u));
                                        idx[u] = ii < n_c ? part0 + (e & 0xffu) : 0xFFFFFFFFu;
                                        old[u] = idx[u] < unit_len ? __ldcg(gsum + idx[u]) : 0.0f;
                                    }
#pragma unroll
                                    for (uint32_t u = 0; u < 4; ++u)
                                        if (idx[u] < unit_len) __stcg(gsum + idx[u], old[u] + val[u]);
                                }
                            } else {
                                for (uint32_t i = i0; i < n_c; i += per_chain) {
                                    const uint32_t e = src[i * 32u];
                                    const float level = __uint_as_float(((e >> 9) + ebias) << 23);
                                    const float v = __fmul_rn(norm_c, level);
                                    add_to(part0 + (e & 0xffu), __uint_as_float(__float_as_uint(v) ^ ((e << 23) & 0x80000000u)));
                                }
                            }
                        } else {
                            for (uint32_t i = i0; i < n_c; i += per_chain) {
                                const uint32_t e = wide ? list[i * 32u + owner]
                                                        : (uint32_t)reinterpret_cast<const uint16_t*>(list)[i * 32u + owner];
                                const float v = level_times_norm(norm_c, sj.levelset, G.s, (e >> 9) + 1u, sj.hdr);
                                add_to(part0 + (e & 0xffu), (e >> 8) & 1u ? -v : v);
                            }
                        }
                    } else {
                        // fixed-width fields: every element of the warp's sub-blocks has one.  A lane
                        // takes 4 consecutive elements at a time: two words hold their 4 * width <= 40 bits
                        bool field_bad = false;
                        const uint32_t wd = sj.width, smask = (1u << (wd - 1u)) - 1u;
                        Chain cf;
                        cf.tok = sj.hdr; cf.norm = 0.0f; cf.cur = cf.end = cf.last = 0;
                        for (uint32_t grp = lane; grp < S * (kSB / 4u); grp += 32) {
                            const uint32_t q = grp >> 6, p = (grp & 63u) * 4u, sb = part * S + q;
                            if ((grp & 32u) == 0) describe_chain(G, T, sj, sb, &cf);   // a sub-block lasts two steps
                            if (sb >= nsb_tile || sb * kSB + p >= tile_len || p + 4u <= fixed_lo || p >= fixed_hi) continue;
                            const uint32_t nel = min(4u, tile_len - (sb * kSB + p));
                            const uint32_t bit = cf.cur + p * wd;
                            const uint32_t wi = bit >> 5;
                            const uint32_t x0 = __ldg(cf.tok + min(wi, cf.last));
                            const uint32_t x1 = __ldg(cf.tok + min(wi + 1u, cf.last));
                            const uint32_t x2 = __ldg(cf.tok + min(wi + 2u, cf.last));
                            // 64 bits from the first field on
                            const uint64_t win = ((uint64_t)__funnelshift_l(x1, x0, bit) << 32) | __funnelshift_l(x2, x1, bit);
#pragma unroll
                            for (uint32_t c = 0; c < 4; ++c) {
                                const uint32_t field = (uint32_t)(win >> (64u - (c + 1u) * wd)) & ((1u << wd) - 1u);
                                const uint32_t sym = field & smask;
                                if (c < nel && p + c >= fixed_lo && p + c < fixed_hi) {
                                    if (sym >= sj.nlev) field_bad = true;
                                    else if (sym) {
                                        const float v = level_times_norm(cf.norm, sj.levelset, G.s, sym, sj.hdr);
                                        add_to(grp * 4u + c, (field >> (wd - 1u)) ? -v : v);
                                    }
                                }
                            }
                        }
                            if (__any_sync(0xffffffffu, field_bad) && lane == 0) latch_status(P.ws, kErrBadStream);
                    }
                    __syncwarp();
                }
                if (!more) break;
            }
            // a well-formed chain ends exactly at its declared length, inside its sub-block, with known indices
            if (has_chain && !bad) bad = cur != end || pos > my_sn || (max_hi >> 9) + 1u >= si.nlev;
            if (__any_sync(0xffffffffu, bad) && lane == 0) latch_status(P.ws, kErrBadStream);
        }

        // ---- write this warp's part of the tile once, and clear it for the next tile ----
        __syncwarp();
        if (!SUMS_IN_L2) {
            const uint32_t first = part * S * kSB;
            for (uint32_t i = lane * 4u; i < S * kSB; i += 128u) {
                if (first + i + 4u <= tile_len) {
                    finish4(P, elem0 + first + i, *reinterpret_cast<const float4*>(accw + i));
                } else {
                    for (uint32_t e = i; e < i + 4u && first + e < tile_len; ++e) finish1(P, elem0 + first + e, accw[e]);
                }
                *reinterpret_cast<float4*>(accw + i) = make_float4(0.f, 0.f, 0.f, 0.f);
            }
        } else if (P.w) {
            // the unit's sums are complete in acc (this instance adds there): apply them to the parameters
            for (uint32_t i = lane * 4u; i < unit_len; i += 128u) {
                const uint64_t e = elem0 + part * S * kSB + i;
                if (i + 4u <= unit_len) {
                    finish4(P, e, __ldcg(reinterpret_cast<const float4*>(gsum + i)), false);
                } else {
                    for (uint32_t k = i; k < unit_len; ++k) finish1(P, e + (k - i), __ldcg(gsum + k), false);
                }
            }
        }
        __syncwarp();
    }
}

static size_t decode_smem_bytes(uint32_t group, uint32_t K, uint32_t warps, bool sums_in_l2) {
    return decode_warp_offset(K) + (size_t)warps * decode_warp_bytes(group, sums_in_l2);
}

cudaError_t launch_decode(const DecodeParams& P, int sms, cudaStream_t stream) {
    constexpr size_t kSmemPerSm = 227u * 1024u, kSmemMaxCta = 227u * 1024u;
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(decode_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemMaxCta);
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(decode_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemMaxCta);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    // One CTA per SM with as many warps as its shared memory holds (25 at most: 80 registers per thread).
    // The warps take equal units of work by ticket, so the kernel lasts ceil(units / warps in flight)
    // rounds, and a round takes about as long as there are warps on the SM (the kernel is bound by
    // instruction issue): among the five largest warp counts take the one with the least rounds * warps,
    // the largest unless a smaller one saves 6 % or more.
    const bool sums_in_l2 = P.group < 4u;                  // 1 or 2 streams side by side
    const size_t fixed = decode_warp_offset(P.K) + 1024u, per_warp = decode_warp_bytes(P.group, sums_in_l2);
    uint32_t wmax = sums_in_l2 ? kDecMaxWarps - 1u : kDecMaxWarps;   // (the instance with the sums in the L2 needs a few registers more)
    while (wmax > 1 && fixed + wmax * per_warp > kSmemPerSm) --wmax;
    const uint64_t units = P.geo.ntiles * P.group;                          // warp-sized units of work
    uint32_t warps = wmax;
    uint64_t best = ~0ull;
    if (units <= (uint64_t)sms * wmax) {                                    // one round: spread it over all SMs
        warps = (uint32_t)((units + sms - 1) / sms);
        best = 0;
    }
    for (uint32_t w = wmax; best && w >= 1 && w + 4 >= wmax; --w) {
        const uint64_t in_flight = (uint64_t)sms * w;
        const uint64_t cost = ((units + in_flight - 1) / in_flight) * w;
        if (w == wmax || cost + cost / 16 < best) {         // fewer warps only for a clear gain: they also hide latency
            best = cost;
            warps = w;
        }
    }
    const uint64_t want = (units + warps - 1) / warps;
    const uint64_t grid = want < (uint64_t)sms ? want : (uint64_t)sms;
    // a CTA of a small call still gets 8 warps: they share the work of building the tables (4096 entries),
    // which one or two warps alone would spend longer on than on decoding; warps without a unit leave at once
    if (warps < 8u && wmax >= 8u) warps = 8u;
    const size_t smem = decode_smem_bytes(P.group, P.K, warps, sums_in_l2);
    if (smem > kSmemMaxCta) return cudaErrorInvalidValue;
    if (P.after_fixed) {
        const uint64_t groups = (P.geo.d + 31) / 32, want_fixed = (groups + 255) / 256, cap_fixed = (uint64_t)sms * 4u;
        decode_fixed_kernel<<<(unsigned)(want_fixed < cap_fixed ? want_fixed : cap_fixed), 256, 0, stream>>>(P);
        if (cudaGetLastError() != cudaSuccess) return cudaErrorUnknown;
    }
    cudaLaunchConfig_t cfg = cudaLaunchConfig_t{};
    cudaLaunchAttribute attr[1];
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3(32u * warps);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 0;
    if (P.after_fixed) {
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.numAttrs = 1;
    }
    if (sums_in_l2) return cudaLaunchKernelEx(&cfg, decode_kernel<true>, P);
    return cudaLaunchKernelEx(&cfg, decode_kernel<false>, P);
}

}  // namespace nuq
