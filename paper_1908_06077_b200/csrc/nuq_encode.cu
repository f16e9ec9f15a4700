// ENCODE of NUQSGD (App. A) for one gradient vector: bucket norm, stochastic
// quantization (Definition 1) and Elias-recursive token packing (Algorithm 2) in one
// kernel that reads the gradient from HBM exactly once.
//
// A persistent CTA takes tiles of up to 8192 consecutive elements (whole buckets, or
// one 8192-element coding block of a wider bucket) by ticket.  The tile's bytes are
// brought into shared memory by bulk asynchronous copies (TMA, completion on an
// mbarrier), one per warp: eight worker warps own 1024 elements (four 256-element
// coding sub-blocks) of the tile each, and a warp starts the copy of its part of the
// next tile as soon as it is done with its part of this one.  Per tile a worker
//   1. adds up the squares of its elements per sub-block (eight per lane in fp32,
//      everything beyond that in fp64); whichever warp is done last turns the partial
//      sums into the tile's bucket norms, once for the whole CTA, before the only CTA
//      barrier of the tile;
//   2. per sub-block: quantizes 8 elements per lane (two Philox blocks), compacts the
//      nonzero symbols into a dense list (one warp scan of per-lane counts; the list
//      lies over the sub-block's own, already consumed, input bytes) and turns the list
//      into tokens ERC(gap) sign ERC(index), 32 per step, appended to the warp's own
//      bit window (two windows per warp, used in turn);
//   3. (ERC mode) shifts its strings of the PREVIOUS tile to their place in a staged
//      image of that tile, which has been laid out in the meantime.
// In the ERC mode a ninth warp, the writer, does everything that concerns a tile as a
// whole: the scan over its 32 sub-block lengths (the layout of its records), the block
// heads, the announcement of its size to the tiles behind it and, once the workers have
// moved their strings, the tile's place in the stream (two-level decoupled look-back
// over tile and group sizes, every wait bounded), the copy of the image to the stream
// and the block offsets.  Workers and writer meet through named barriers on which one
// side only arrives, so the workers never wait for other CTAs.
// In the fixed-width mode there is no writer: a lane packs the fields of its eight
// elements, two lanes exchange halves, and every lane stores one finished word (4-bit
// fields of the exponential level set have a leaner kernel of their own, nuq_encode_fixed4.cu).
// Counters and the container header are written once per CTA, the header by whichever
// CTA finishes last.
// A bucket wider than a tile is encoded by a thread-block cluster, one CTA per tile of the
// bucket: the CTAs send one another their tiles' sums of squares through distributed shared
// memory and agree on the bucket's norm, so the gradient is still read only once.
#include "nuq_encode_common.cuh"
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

// Uniform levels k / 2^s:  p = y - floor(y).
__device__ __forceinline__ uint32_t quantize_uniform(float v, float inv, float top, uint32_t word) {
    const float y = fminf(__fmul_rn(fabsf(v), inv), top);
    const float fl = fminf(floorf(y), top - 1.0f);
    const float p = y - fl;
    return (uint32_t)fl + ((__uint2float_rn(word >> 8) < p * 16777216.0f) ? 1u : 0u);
}

// A general level sequence (0, l_1, ..., l_s, 1) given as a table (Sec. 3.3): r = |v| / norm clamped
// to 1, l_j <= r < l_{j+1}, p = (r - l_j) / (l_{j+1} - l_j) computed as a product with the inverse
// width; the draw is compared as u = m 2^-24.  `lv`, `iw`: the tables in shared memory.
__device__ __forceinline__ uint32_t quantize_table(float v, float inv, uint32_t s, uint32_t word, const float* lv,
                                                   const float* iw) {
    const float r = fminf(__fmul_rn(fabsf(v), inv), 1.0f);
    uint32_t j = 0;
    for (uint32_t k = 1; k <= s + 1u; ++k) j += r >= lv[k] ? 1u : 0u;    // the levels increase: j = index of the last one <= r
    const float p = __fmul_rn(__fsub_rn(r, lv[j]), iw[j]);
    const float u = __fmul_rn(__uint2float_rn(word >> 8), 0x1p-24f);
    return j + (u < p ? 1u : 0u);
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

// OR `nbits` (0..32) right-aligned bits of `value` into the MSB-first bit string `dst` at `bitpos`.
// Two words are touched unconditionally (a zero is OR-ed when there is nothing to add).
__device__ __forceinline__ void or_bits32(uint32_t* dst, uint32_t bitpos, uint32_t value, uint32_t nbits) {
    const uint32_t a = nbits ? value << (32u - nbits) : 0u;
    const uint32_t w = bitpos >> 5, sh = bitpos & 31u;
    atomicOr(dst + w, a >> sh);
    atomicOr(dst + w + 1, __funnelshift_r(0u, a, sh));
}

// OR the left-aligned bits of `a` (zero beyond its last bit) into the MSB-first bit string `dst` at
// `bitpos`.  Two words are touched unconditionally (a zero is OR-ed when there is nothing to add).
__device__ __forceinline__ void or_bits_left(uint32_t* dst, uint32_t bitpos, uint32_t a) {
    const uint32_t w = bitpos >> 5, sh = bitpos & 31u;
    atomicOr(dst + w, a >> sh);
    atomicOr(dst + w + 1, __funnelshift_r(0u, a, sh));
}

// 32 bits of the MSB-first bit string `src` starting at bit `sbit` (>= -31); bits before
// the string read as garbage and must be masked by the caller.
__device__ __forceinline__ uint32_t bits_at(const uint32_t* src, int sbit) {
    if (sbit < 0) return src[0] >> (uint32_t)(-sbit);
    const uint32_t w = (uint32_t)sbit >> 5;
    return __funnelshift_l(src[w + 1], src[w], (uint32_t)sbit);
}

// Inclusive warp scan; the shuffle's own range predicate guards the add.
__device__ __forceinline__ uint32_t warp_incl_scan(uint32_t v) {
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        asm volatile(
            "{\n\t.reg .pred p;\n\t.reg .u32 t;\n\t"
            "shfl.sync.up.b32 t|p, %0, %1, 0, 0xffffffff;\n\t"
            "@p add.u32 %0, %0, t;\n\t}"
            : "+r"(v)
            : "r"(o));
    }
    return v;
}

// ---------------------------------------------------------------------------
// Two-level decoupled look-back over tile payload sizes, run by one warp.  Returns the
// exclusive prefix (words) of `tile`, or sets *failed.  Every wait is bounded.
//
// As many tiles as there are resident CTAs (several hundred) are under way at any time and
// none of them knows its place yet, so a walk over single tiles would have to sum all of
// them.  Sizes are therefore also accumulated per group of 32 consecutive tiles:
//   tile_state[t]   kTileAggregate | words          once tile t has been encoded
//   group_state[g]  count << 48 | words so far      while tiles of the group announce themselves
//                   kTilePrefix | words before the end of the group, written by whoever places
//                   the group's last tile
// A tile sums the sizes of the tiles before it in its own group (one load per lane), then
// walks back over whole groups, 64 per step, to the nearest one that knows its prefix.
// A wait that runs out of patience poisons the tile's own words, so that the tiles behind it
// give up at once instead of spending their own patience one after the other.
// ---------------------------------------------------------------------------
constexpr uint32_t kGroupTiles = 32;
constexpr uint32_t kGroupCountShift = 48;
constexpr uint64_t kGroupSumMask = (1ull << kGroupCountShift) - 1;

__device__ __forceinline__ void announce_tile(uint64_t* tile_state, uint64_t* group_state, uint64_t tile, uint32_t words) {
    st_volatile_u64(tile_state + tile, kTileAggregate | words);
    atomicAdd(reinterpret_cast<unsigned long long*>(group_state + tile / kGroupTiles),
              (1ull << kGroupCountShift) | (unsigned long long)words);
}

// One more poll of a look-back wait; false when the patience is used up.
__device__ __forceinline__ bool lookback_backoff(uint32_t patience, uint32_t& polls) {
    if (++polls > patience) return false;
    __nanosleep(polls < 64 ? 250 : 1000);                   // a waiting warp should not eat issue slots
    return true;
}

__device__ uint64_t tile_lookback(const EncodeParams& P, uint64_t* tile_state, uint64_t* group_state, uint64_t tile,
                                  uint32_t words, bool* failed) {
    const uint32_t lane = lane_id();
    const uint64_t ntiles = P.geo.ntiles;
    const uint64_t grp = tile / kGroupTiles;
    const uint32_t r = (uint32_t)(tile % kGroupTiles);      // tiles of the group before this one
    uint32_t polls = 0;
    uint64_t exclusive = 0;
    bool ok = true;
    // ---- the tiles before this one in its own group ----
    for (;;) {
        const uint64_t v = lane < r ? ld_volatile_u64(tile_state + grp * kGroupTiles + lane) : kTileAggregate;
        if (__any_sync(0xffffffffu, (v >> 62) == 3)) { ok = false; break; }             // a predecessor gave up
        const uint32_t missing = __ballot_sync(0xffffffffu, (v >> 62) != 1);
        if (!missing) {
            exclusive = __reduce_add_sync(0xffffffffu, (uint32_t)v);           // a tile has far fewer than 2^27 words
            break;
        }
        // wait for the first missing one alone, then look at all of them again
        const uint64_t* p = tile_state + grp * kGroupTiles + (__ffs(missing) - 1);
        while (ok && (ld_volatile_u64(p) >> 62) == 0) ok = lookback_backoff(P.patience, polls);
        if (!ok) break;
    }
    // ---- whole groups, nearest first: lane l looks at groups base - l and base - 32 - l ----
    int64_t base = (int64_t)grp - 1;
    while (ok && base >= 0) {
        const int64_t i0 = base - (int64_t)lane, i1 = i0 - 32;
        const uint64_t v0 = i0 >= 0 ? ld_volatile_u64(group_state + i0) : kTilePrefix;    // before group 0: prefix 0
        const uint64_t v1 = i1 >= 0 ? ld_volatile_u64(group_state + i1) : kTilePrefix;
        if (__any_sync(0xffffffffu, (v0 >> 62) == 3 || (v1 >> 62) == 3)) { ok = false; break; }
        const bool p0 = (v0 >> 62) == 2, p1 = (v1 >> 62) == 2;                    // knows its prefix
        const bool n0 = !p0 && (v0 >> kGroupCountShift) != kGroupTiles;           // still collecting (earlier groups are full ones)
        const bool n1 = !p1 && (v1 >> kGroupCountShift) != kGroupTiles;
        const uint64_t pm = (uint64_t)__ballot_sync(0xffffffffu, p0) | ((uint64_t)__ballot_sync(0xffffffffu, p1) << 32);
        const uint64_t nm = (uint64_t)__ballot_sync(0xffffffffu, n0) | ((uint64_t)__ballot_sync(0xffffffffu, n1) << 32);
        const uint32_t first_p = pm ? (uint32_t)__ffsll((long long)pm) - 1u : 64u;
        const uint32_t first_n = nm ? (uint32_t)__ffsll((long long)nm) - 1u : 64u;
        if (first_n < first_p) {
            // a group on the way is not complete yet: wait for it alone, then look at all of them again
            const uint64_t* p = group_state + (base - (int64_t)first_n);
            for (;;) {
                const uint64_t v = ld_volatile_u64(p);
                if ((v >> 62) >= 2 || (v >> kGroupCountShift) == kGroupTiles) break;
                if (!lookback_backoff(P.patience, polls)) { ok = false; break; }
            }
            continue;
        }
        uint64_t c = 0;
        if (lane <= first_p) c += p0 ? v0 & kTileValueMask : v0 & kGroupSumMask;
        if (lane + 32u <= first_p) c += p1 ? v1 & kTileValueMask : v1 & kGroupSumMask;
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
        exclusive += c;
        if (first_p < 64u) break;
        base -= 64;
    }
    // ---- whoever places the last tile of a group tells the later groups where it ends ----
    const bool closes_group = r == kGroupTiles - 1u || tile == ntiles - 1;
    if (ok && closes_group) {
        const uint64_t members = tile == ntiles - 1 ? r + 1u : kGroupTiles;
        for (;;) {                                          // every member's size has been added (they were all seen above)
            const uint64_t v = ld_volatile_u64(group_state + grp);
            if ((v >> kGroupCountShift) == members) break;
            if (!lookback_backoff(P.patience, polls)) { ok = false; break; }
        }
        if (ok && lane == 0) st_volatile_u64(group_state + grp, kTilePrefix | (exclusive + words));
    }
    if (!ok && lane == 0) {
        latch_status(P.ws, kErrTimeout);
        st_volatile_u64(tile_state + tile, kTilePoison);
        if (closes_group) st_volatile_u64(group_state + grp, kTilePoison);
    }
    *failed = !ok;
    return exclusive;
}

// Symbols travel as small fields: level index in the low bits, sign above it.
template <uint32_t LEVELSET>
struct Sym {
    static constexpr uint32_t kBits = LEVELSET != kLevelsUniform ? 7u : 15u;  // index <= 15 resp. <= 256
    static constexpr uint32_t kMask = (1u << kBits) - 1u;
};

constexpr uint32_t kWarpElems = kBLK / kEncWarps;   // 1024 elements of a tile per warp (4 sub-blocks)

// Named CTA barriers.  The 8 worker warps meet at kBarWork once per tile.  In the ERC mode the workers and the writer warp pass
// a tile k from hand to hand through three barriers with index k & 1:
//   kBarDone    the workers arrive when their strings of tile k are complete, the writer waits;
//   kBarLayout  the writer arrives when it has laid the tile out, the workers wait (a tile later);
//   kBarMerged  the workers arrive when they have moved their strings into the image, the writer waits.
constexpr uint32_t kBarWork = 1, kBarDone = 2, kBarLayout = 4, kBarMerged = 6;
constexpr uint32_t kEncAllThreads = kEncThreads + 32;      // ERC mode: workers + the writer warp
template <uint32_t ID, uint32_t COUNT>
__device__ __forceinline__ void bar_sync() {
    asm volatile("bar.sync %0, %1;" ::"n"(ID), "n"(COUNT) : "memory");
}
template <uint32_t ID, uint32_t COUNT>
__device__ __forceinline__ void bar_arrive() {
    __threadfence_block();
    asm volatile("bar.arrive %0, %1;" ::"n"(ID), "n"(COUNT) : "memory");
}
// the barrier BASE + p of tile parity p; immediate barrier numbers, so that the kernel claims only those it uses
template <uint32_t BASE>
__device__ __forceinline__ void pair_sync(uint32_t p) {
    if (p == 0) bar_sync<BASE, kEncAllThreads>();
    else bar_sync<BASE + 1, kEncAllThreads>();
}
template <uint32_t BASE>
__device__ __forceinline__ void pair_arrive(uint32_t p) {
    if (p == 0) bar_arrive<BASE, kEncAllThreads>();
    else bar_arrive<BASE + 1, kEncAllThreads>();
}

// What the workers and the writer tell one another about a tile (ERC mode).
struct TileMeta {
    unsigned long long tile;
    uint32_t nsb, pad;
    uint32_t sb_bits[32];                                  // token bits of each sub-block ...
    uint32_t sb_src[32];                                   // ... and where they start in the owning warp's window
    uint32_t blk_norm[32];                                 // norm word of each coding block of the tile
    uint32_t bitoff[32];                                   // written by the writer: where each sub-block's string goes in the image
    uint32_t wnnz[kEncWarps];                              // nonzero symbols each warp produced
};

// A tile whose records are staged in shared memory and whose place in the stream is not
// yet known.
struct Pending {
    unsigned long long tile;
    uint32_t words, nblk, code_bits, nnz;
    uint32_t blk_wordoff[32];                              // word offset of block bi within the tile
};

// What a CTA has written so far (shared memory; updated by one thread at a time).
struct CtaTotals {
    uint64_t nnz, code_bits;
    uint32_t stop, pad;                                    // stop: tiles the workers encoded (set when they leave)
};

// The writer warp, first half of its work on a tile: the layout of the tile's records from the 32
// sub-block lengths (lane = sub-block), the block heads written into the (zeroed) image, the tile's
// size announced to the tiles behind it, and what the second half needs noted in `pd`.
__device__ void lay_out_tile(const EncodeParams& P, TileMeta& m, Pending& pd, uint32_t* stg, uint64_t* tile_state,
                             uint64_t* group_state, uint32_t lane) {
    const Geometry& G = P.geo;
    const bool narrow = G.bucket <= kBLK;
    const uint32_t spb = narrow ? G.sb_per_block : 32u;
    const uint32_t nsb = m.nsb;
    const uint32_t v = lane < nsb ? m.sb_bits[lane] : 0u;
    const uint32_t incl = warp_incl_scan(v);
    const uint32_t excl = incl - v;
    const uint32_t bi = lane / spb, sb0 = bi * spb;
    const uint32_t sb_last = min(sb0 + spb, nsb) - 1u;                  // meaningful when lane < nsb
    const uint32_t excl0 = __shfl_sync(0xffffffffu, excl, sb0 & 31u);
    const uint32_t incl_last = __shfl_sync(0xffffffffu, incl, sb_last & 31u);
    const uint32_t nsb_blk = sb_last - sb0 + 1u;
    const uint32_t head_words = 1u + (nsb_blk + 1u) / 2u;
    const bool leader = lane < nsb && lane == sb0;
    const uint32_t blk_words = leader ? head_words + (incl_last - excl0 + 31u) / 32u : 0u;
    const uint32_t wincl = warp_incl_scan(blk_words);
    const uint32_t wexcl = wincl - blk_words;
    const uint32_t blk_off = __shfl_sync(0xffffffffu, wexcl, sb0 & 31u);                // words before my block
    m.bitoff[lane] = 32u * (blk_off + head_words) + (excl - excl0);                      // where sub-block `lane` goes
    const uint32_t tile_words = __shfl_sync(0xffffffffu, wincl, 31);
    const uint32_t code_bits = __shfl_sync(0xffffffffu, incl, 31);
    if (lane == 0) announce_tile(tile_state, group_state, m.tile, tile_words);
    // block heads: the norm word, then the u16 lengths of the block's sub-blocks, two per word
    if (leader) stg[blk_off] = m.blk_norm[bi];
    const uint32_t nv = __shfl_down_sync(0xffffffffu, v, 1);
    if (lane < nsb && ((lane - sb0) & 1u) == 0)
        stg[blk_off + 1u + (lane - sb0) / 2u] = v | ((lane + 1u <= sb_last ? nv : 0u) << 16);
    pd.blk_wordoff[lane] = __shfl_sync(0xffffffffu, wexcl, (lane * spb) & 31u);
    uint32_t nnz = lane < (uint32_t)kEncWarps ? m.wnnz[lane] : 0u;
    nnz = __reduce_add_sync(0xffffffffu, nnz);
    if (lane == 0) {
        pd.tile = m.tile;
        pd.words = tile_words;
        pd.nblk = narrow ? (nsb + spb - 1u) / spb : 1u;
        pd.code_bits = code_bits;
        pd.nnz = nnz;
    }
    __syncwarp();
}

// Second half: find the place of the staged tile (its predecessors announced their sizes when they were
// laid out, so the walk rarely waits), copy the image to the stream, clear the image.
__device__ void flush_pending(const EncodeParams& P, Pending& pd, CtaTotals& tot, uint32_t* stg, uint64_t* tile_state,
                              uint64_t* group_state, uint64_t* table, uint32_t* payload, uint32_t lane) {
    const Geometry& G = P.geo;
    const uint64_t tile = pd.tile;
    const uint32_t words = pd.words;
    bool failed;
    const uint64_t off = tile_lookback(P, tile_state, group_state, tile, words, &failed);
    for (uint32_t i = lane; i < words; i += 32) {
        if (!failed) payload[off + i] = stg[i];
        stg[i] = 0;
    }
    if (!failed) {
        const uint64_t first_block = G.bucket <= kBLK ? tile * G.blocks_per_tile : tile;
        if (lane < pd.nblk) table[first_block + lane] = 32ull * (off + pd.blk_wordoff[lane]);
        if (tile == G.ntiles - 1 && lane == 0) {
            table[G.nblk] = 32ull * (off + words);
            P.ws->total_words = off + words;
        }
    }
    __syncwarp();
    if (lane == 0) {
        tot.nnz += pd.nnz;
        tot.code_bits += pd.code_bits;
    }
    __syncwarp();
}

// CLUSTERS: the call's buckets are wider than a tile and each is encoded by a thread-block cluster (see below).
template <uint32_t LEVELSET, uint32_t MODE, bool CLUSTERS>
__global__ void __launch_bounds__(MODE == kModeErc ? kEncAllThreads : kEncThreads, kEncMinBlocks)
encode_kernel(const __grid_constant__ EncodeParams P) {
    extern __shared__ __align__(128) uint32_t smem[];
    __shared__ __align__(8) uint64_t s_full[kEncWarps];    // s_full[w] completes when warp w's part of a tile has landed
    __shared__ uint32_t s_lut[256];                        // ERC(N), N = 1..256: code left aligned | length
    __shared__ uint32_t s_lut_signed[256];                 // exponential levels: sign bit + ERC(index) left aligned | length, by field
    __shared__ double s_partial[32];                       // per sub-block (or per warp) sums of squares
    __shared__ uint32_t s_maxbits[32];                     // ... or max |x| bit patterns
    __shared__ float s_sb_inv[32], s_sb_norm[32];          // per sub-block of the current tile: 2^s / norm (0: not quantized), norm
    __shared__ uint32_t s_sb_bi[32];                       // block (within a tile) of each sub-block
    __shared__ float s_levels[kMaxTableS + 2], s_invw[kMaxTableS + 2];   // level table (level-table streams)
    __shared__ uint32_t s_arrived;                         // warps that have added up their squares (counts on, modulo 8)
    __shared__ TileInfo s_info[4];                         // tiles of the iterations it, it + 1, it + 2
    __shared__ TileMeta s_meta[2];
    __shared__ Pending s_pend[2];
    __shared__ CtaTotals s_tot;
    __shared__ uint32_t s_nnz;                             // fixed-width mode: nonzero symbols of this CTA
    __shared__ uint32_t s_last;                            // this CTA finished last
    // clusters (buckets wider than a tile): what the CTAs of a cluster tell one another
    __shared__ __align__(8) uint64_t s_xbar[2];            // s_xbar[p] completes when every CTA's part of the bucket's norm (iteration parity p) is here
    __shared__ uint64_t s_xchg[2][8];                      // s_xchg[p][r]: CTA r's sum of squares (bits of a double) or max |x| bits
    __shared__ unsigned long long s_bucket[4];             // buckets of the iterations to come, handed out by the cluster's first CTA

    using S = Sym<LEVELSET>;
    const Geometry& G = P.geo;
    const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    float* const data = reinterpret_cast<float*>(smem);                         // kBLK floats: the tile
    uint32_t* const images = smem + kBLK;                                       // [2][stage_words]: staged tile records
    uint32_t* const windows = images + 2u * P.stage_words;                      // [2][kEncWarps][window_words]: token strings
    uint64_t* tile_state = reinterpret_cast<uint64_t*>(P.ws + 1);
    uint64_t* group_state = tile_state + G.ntiles;
    uint64_t* table = reinterpret_cast<uint64_t*>(P.out + G.header_words);
    uint32_t* payload = MODE == kModeErc ? P.out + G.header_words + 2 * (G.nblk + 1) : P.out + G.header_words;
    constexpr bool kSmall = LEVELSET != kLevelsUniform;     // level index <= 15: symbols travel as bytes
    const float top = LEVELSET == kLevelsTable ? 1.0f : __uint_as_float((127u + G.s) << 23);   // the norm is divided into this
    const uint32_t c2 = (uint32_t)P.offset, c3 = (uint32_t)(P.offset >> 32);
    const bool narrow = G.bucket <= kBLK;
    const bool coarse = G.bucket % kWarpElems == 0;         // a warp's four sub-blocks always share one bucket
    const uint32_t spb = narrow ? G.sb_per_block : 32u;     // sub-blocks per coding block

    // Clusters: a bucket wider than a tile is encoded by a cluster of as many CTAs as it has tiles, CTA r
    // taking tile r of the bucket; they add up the bucket's norm among themselves through distributed shared
    // memory, so the gradient is read from HBM once.  The cluster's first CTA takes the tickets (they count
    // buckets then) and writes them into every CTA's s_bucket.
    const uint32_t cl = CLUSTERS ? P.cluster : 1u;
    const uint32_t crank = cl > 1u ? cluster_rank() : 0u;
    auto hand_out_bucket = [&](uint32_t iter) {             // thread 0 of the cluster's first CTA
        const unsigned long long b = atomicAdd(reinterpret_cast<unsigned long long*>(&P.ws->ticket), 1ull);
        for (uint32_t r = 0; r < cl; ++r) st_cluster_u64(cluster_addr(&s_bucket[iter & 3u], r), b);
        asm volatile("fence.acq_rel.cluster;" ::: "memory");
    };
    // thread 0: take a ticket and work out where that tile lies.  Every tile is handed out by ticket, a CTA's
    // first one too: a tile waits (look-back) for the tiles before it, and those must belong to CTAs that are
    // running -- the CTAs of a call need not all be resident at once (another stream's kernel may hold SM
    // slots), and a CTA that is not running must not own a tile that the running ones wait for.
    auto take_ticket = [&](uint32_t iter) {
        TileInfo& ti = s_info[iter & 3u];
        unsigned long long t;
        if (cl > 1u) {
            const unsigned long long b = *reinterpret_cast<volatile unsigned long long*>(&s_bucket[iter & 3u]);
            t = b >= G.nb ? G.ntiles : b * cl + crank;
            if (b < G.nb && t >= G.ntiles) t = G.ntiles + 1u;    // the last bucket is short and has no tile for this CTA
        } else {
            t = atomicAdd(reinterpret_cast<unsigned long long*>(&P.ws->ticket), 1ull);
        }
        describe_tile(G, t, &ti);
    };
    // A warp's part of a tile: elements [1024 w, 1024 (w + 1)) of it.  Whole 16-byte pieces come by a bulk
    // copy that the warp starts itself as soon as it is done with its part of the tile before.
    const uint32_t wbase = warp * kWarpElems;               // first element of the warp within a tile
    auto bulk_elems_of = [&](const TileInfo& ti) {
        const uint32_t n = ti.tile_len > wbase ? min(kWarpElems, ti.tile_len - wbase) : 0u;
        return ti.tile < G.ntiles ? n & ~3u : 0u;
    };
    auto start_copy = [&](uint32_t iter) {                  // one lane of the warp
        const TileInfo& ti = s_info[iter & 3u];
        const uint32_t n = bulk_elems_of(ti);
        if (n) bulk_load(data + wbase, P.g + ti.elem0 + wbase, 4u * n, &s_full[warp]);
    };

    let_next_kernel_start(P);
    if (tid < 256u) {
        const uint32_t e = c_erc_lut[tid], elen = e >> 16;  // at most 16 bits
        s_lut[tid] = ((e & 0xffffu) << (32u - elen)) | elen;
        const uint32_t idx = tid & 0x7Fu;                   // field = sign << 7 | index: sign bit, then ERC(index)
        uint32_t v = 0;
        if (idx >= 1) {
            // the index's code word: ERC(index), or in the coded mode the word of the fitted code
            const bool coded = G.mode == kModeCoded;
            const uint32_t l = coded ? (idx <= kMaxCodedS + 1u ? P.level_code[idx - 1u] : 0u) : c_erc_lut[idx - 1u], len = l >> 16;
            v = ((((tid >> 7) << len) | (l & 0xffffu)) << (31u - len)) | (len + 1u);
        }
        s_lut_signed[tid] = v;
    }
    if (tid < 32u) s_sb_bi[tid] = tid / spb;
    if (tid < kMaxTableS + 2u) {
        s_levels[tid] = P.levels[tid];
        s_invw[tid] = P.inv_width[tid];
    }
    if (MODE == kModeErc)
        for (uint32_t i = tid; i < 2u * P.stage_words + 2u * kEncWarps * P.window_words; i += blockDim.x) images[i] = 0;
    wait_for_previous_kernel(P);                            // nothing above reads or writes global memory
    if (tid == 0) {
        for (int w = 0; w < kEncWarps; ++w) mbar_init(&s_full[w], 1);
        s_nnz = 0;
        s_arrived = 0;
        s_tot.nnz = 0;
        s_tot.code_bits = 0;
        s_tot.stop = 0xFFFFFFFFu;
        s_last = 0;
        if (cl > 1u) {
            mbar_init(&s_xbar[0], cl);
            mbar_init(&s_xbar[1], cl);
        }
        if (cl == 1u) take_ticket(0);
    }
    __syncthreads();
    if (cl > 1u) {
        cluster_sync_all();                                 // every CTA's barriers exist before anyone arrives at them
        if (tid == 0 && crank == 0) {                       // (the first bucket comes by ticket too, like a CTA's first tile)
            hand_out_bucket(0);
            hand_out_bucket(1);
            hand_out_bucket(2);
        }
        cluster_sync_all();                                 // the buckets of the first three iterations are known everywhere
        if (tid == 0) take_ticket(0);
        __syncthreads();
    }
    if (warp < (uint32_t)kEncWarps && lane == 0) start_copy(0);
    if (tid == 0) take_ticket(1);                           // its round trip runs while the first bytes arrive

    const bool writer = MODE == kModeErc && warp == (uint32_t)kEncWarps;
    if (writer) {
        // ---- the writer warp: lays out every tile the workers have encoded, and a tile later, when they
        // have moved their strings into the image, finds the tile's place in the stream and copies it out
        for (uint32_t k = 0;; ++k) {
            const uint32_t p = k & 1u;
            pair_sync<kBarDone>(p);                         // the workers' strings of tile k are complete (or there is no tile k)
            const bool have = k < *reinterpret_cast<volatile uint32_t*>(&s_tot.stop);
            if (have) {
                lay_out_tile(P, s_meta[p], s_pend[p], images + p * P.stage_words, tile_state, group_state, lane);
                pair_arrive<kBarLayout>(p);
            }
            if (k >= 1) {
                pair_sync<kBarMerged>(p ^ 1u);              // the strings of tile k - 1 are in its image
                flush_pending(P, s_pend[p ^ 1u], s_tot, images + (p ^ 1u) * P.stage_words, tile_state, group_state, table,
                              payload, lane);
            }
            if (!have) break;
        }
    }

    // ---- ERC: a worker moves its strings of tile k (window set k & 1, `bits` bits) to their place in
    // the image once the writer has laid the tile out ----
    auto merge_tile = [&](uint32_t k, uint32_t bits) {
        const uint32_t p = k & 1u;
        pair_sync<kBarLayout>(p);
        const TileMeta& m = s_meta[p];
        uint32_t* stg = images + p * P.stage_words;
        uint32_t* win = windows + (p * kEncWarps + warp) * P.window_words;
#pragma unroll 1
        for (uint32_t q = 0; q < 4; q += coarse ? 4u : 1u) {
            // the strings of sub-blocks of one block follow one another in the window and in the
            // tile alike, so a warp whose four sub-blocks share a block moves them in one piece
            const uint32_t sbq = warp * 4u + q;
            if (sbq >= m.nsb) break;
            const uint32_t len = coarse ? bits : m.sb_bits[sbq], src = coarse ? 0u : m.sb_src[sbq];
            const uint32_t dst = m.bitoff[sbq];
            if (len == 0) continue;
            const uint32_t w_first = dst >> 5, w_last = (dst + len - 1u) >> 5;
            for (uint32_t w = w_first + lane; w <= w_last; w += 32) {
                const int sbit = (int)src + (int)(32u * w) - (int)dst;
                uint32_t val = bits_at(win, sbit);
                const uint32_t head = 32u * w < dst ? dst - 32u * w : 0u;     // bits of this word before the string
                const uint32_t tail_end = min(dst + len - 32u * w, 32u);      // bits of this word up to its end
                uint32_t mask = 0xFFFFFFFFu >> head;
                if (tail_end < 32u) mask &= ~(0xFFFFFFFFu >> tail_end);
                val &= mask;
                if (val) atomicOr(stg + w, val);
            }
        }
        __syncwarp();
        for (uint32_t i = lane; i < (bits + 31u) / 32u + 2u; i += 32) win[i] = 0;   // ready for tile k + 2
        __syncwarp();
        pair_arrive<kBarMerged>(p);                        // the writer may take the tile
    };

    uint32_t it = 0;
    uint32_t cta_nnz = 0;                                   // fixed-width mode: this thread's count
    uint32_t prev_bits = 0;                                 // ERC: bits of this warp's strings of the previous tile
    uint32_t parity = 0;                                    // of the next completion of s_full[warp]
    for (; !writer; ++it) {                                 // the 8 worker warps
        const TileInfo& ti = s_info[it & 3u];
        const uint64_t tile = ti.tile;
        if (tile >= G.ntiles) {
            // a CTA without a tile in the cluster's last, short bucket adds nothing to its norm, but says so
            if (cl > 1u && tile == G.ntiles + 1u && warp == 0 && lane < cl) {
                st_cluster_u64(cluster_addr(&s_xchg[it & 1u][crank], lane), 0ull);
                mbar_arrive_cluster(cluster_addr(&s_xbar[it & 1u], lane));
            }
            break;
        }
        const uint64_t elem0 = ti.elem0;
        const uint32_t tile_len = ti.tile_len, nsb_tile = ti.nsb;

        // ---- the warp's part of the tile: wait for the bulk copy, fetch the ragged end, zero the rest ----
        {
            const uint32_t bulk_elems = bulk_elems_of(ti);
            if (bulk_elems) {
                if (!mbar_wait(&s_full[warp], parity) && lane == 0) latch_status(P.ws, kErrTimeout);   // never seen; do not hang
                parity ^= 1u;
            }
            if (bulk_elems < kWarpElems) {
                for (uint32_t i = bulk_elems + lane; i < kWarpElems; i += 32)
                    data[wbase + i] = wbase + i < tile_len ? __ldg(P.g + elem0 + wbase + i) : 0.0f;
                __syncwarp();
            }
        }
        const float4* rows = reinterpret_cast<const float4*>(data + wbase) + lane;   // row j at rows[32 * j]

        // ---- bucket norms.  L2: a lane adds the squares of its 8 elements of a sub-block in fp32 (7 roundings
        // of 2^-24 relative each, of random sign), everything beyond that in fp64: the norm stays within a
        // few 1e-8 of the exactly rounded one.  Linf: max |x|, exact. ----
        if (P.norms_in == nullptr) {
            double acc = 0.0;
            uint32_t mx = 0;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                const float4 x = rows[32 * (2 * q)], y = rows[32 * (2 * q + 1)];
                if (G.norm_kind == kNormL2) {
                    float a = __fmul_rn(x.x, x.x), b = __fmul_rn(x.y, x.y);
                    a = __fmaf_rn(x.z, x.z, a); b = __fmaf_rn(x.w, x.w, b);
                    a = __fmaf_rn(y.x, y.x, a); b = __fmaf_rn(y.y, y.y, b);
                    a = __fmaf_rn(y.z, y.z, a); b = __fmaf_rn(y.w, y.w, b);
                    const float p8 = a + b;
                    // squares that leave the fp32 range (tiny or huge coordinates, NaN): the warp adds this
                    // sub-block up in fp64 instead
                    const bool out_of_range = !(p8 >= 0x1p-60f && p8 < 0x1p120f);
                    if (__any_sync(0xffffffffu, out_of_range)) {
                        double e = 0.0;
                        e = fma((double)x.x, (double)x.x, e); e = fma((double)x.y, (double)x.y, e);
                        e = fma((double)x.z, (double)x.z, e); e = fma((double)x.w, (double)x.w, e);
                        e = fma((double)y.x, (double)y.x, e); e = fma((double)y.y, (double)y.y, e);
                        e = fma((double)y.z, (double)y.z, e); e = fma((double)y.w, (double)y.w, e);
                        acc += e;
                    } else {
                        acc += (double)p8;
                    }
                } else {                                    // on the bit patterns: NaN sorts above inf
                    mx = max(max(mx, __float_as_uint(fabsf(x.x))), __float_as_uint(fabsf(x.y)));
                    mx = max(max(mx, __float_as_uint(fabsf(x.z))), __float_as_uint(fabsf(x.w)));
                    mx = max(max(mx, __float_as_uint(fabsf(y.x))), __float_as_uint(fabsf(y.y)));
                    mx = max(max(mx, __float_as_uint(fabsf(y.z))), __float_as_uint(fabsf(y.w)));
                }
                if (!coarse || q == 3) {                    // one partial per sub-block, or one per warp
                    if (G.norm_kind == kNormL2) {
#pragma unroll
                        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
                    } else {
                        mx = __reduce_max_sync(0xffffffffu, mx);
                    }
                    if (lane == 0) {
                        s_partial[warp * 4 + q] = acc;
                        s_maxbits[warp * 4 + q] = mx;
                    }
                    acc = 0.0;
                    mx = 0;
                }
            }
        }
        // the draws of the warp's first sub-block do not depend on the norms: they are made before the
        // barrier, where the warp would otherwise wait for the slowest one
        const uint64_t ctr_warp = ((elem0 + wbase) >> 2) + lane;               // Philox counter of row 0's block
        uint4 rn0 = philox4x32_10((uint32_t)ctr_warp, (uint32_t)(ctr_warp >> 32), c2, c3, P.round_keys);
        uint4 rn1 = philox4x32_10((uint32_t)(ctr_warp + 32u), (uint32_t)((ctr_warp + 32u) >> 32), c2, c3, P.round_keys);
        // ---- whichever warp gets here last turns the partial sums into norms, once for the whole CTA ----
        {
            uint32_t last = 0;
            __syncwarp();
            if (lane == 0) {
                __threadfence_block();
                last = (atomicAdd(&s_arrived, 1u) & (kEncWarps - 1u)) == kEncWarps - 1u;
            }
            if (__shfl_sync(0xffffffffu, last, 0)) {
                __threadfence_block();
                // lane = sub-block of the tile; the lanes of one bucket all do the same sum, in the same order
                const uint32_t bi = lane / spb, sb0 = bi * spb;
                float norm;
                if (P.norms_in != nullptr) {
                    const uint64_t nb_idx = narrow ? ti.first_block + bi : ti.bucket_idx;
                    norm = nb_idx < G.nb ? P.norms_in[nb_idx] : 0.0f;
                } else if (cl > 1u) {
                    // this CTA's tile is one part of its bucket: every CTA of the cluster sends its sum (or
                    // maximum) to all of them, and all add the parts up in the same order
                    double a = 0.0;
                    uint32_t mxb = 0;
                    for (uint32_t j = 3u; j < 32u; j += 4u) {       // one partial per warp
                        a += s_partial[j];
                        mxb = max(mxb, s_maxbits[j]);
                    }
                    const uint32_t xp = it & 1u;
                    if (lane < cl) {
                        st_cluster_u64(cluster_addr(&s_xchg[xp][crank], lane),
                                       G.norm_kind == kNormL2 ? (uint64_t)__double_as_longlong(a) : (uint64_t)mxb);
                        mbar_arrive_cluster(cluster_addr(&s_xbar[xp], lane));
                    }
                    __syncwarp();
                    norm = 0.0f;
                    if (!mbar_wait_cluster(&s_xbar[xp], (it >> 1) & 1u)) {
                        if (lane == 0) latch_status(P.ws, kErrTimeout);   // never seen; do not hang
                    } else if (G.norm_kind == kNormL2) {
                        a = 0.0;
                        for (uint32_t r = 0; r < cl; ++r) a += __longlong_as_double((long long)s_xchg[xp][r]);
                        norm = (float)sqrt(a);
                    } else {
                        mxb = 0;
                        for (uint32_t r = 0; r < cl; ++r) mxb = max(mxb, (uint32_t)s_xchg[xp][r]);
                        norm = __uint_as_float(mxb);
                    }
                } else if (G.norm_kind == kNormL2) {
                    double a = 0.0;
                    if (coarse) for (uint32_t j = sb0 + 3u; j < sb0 + spb; j += 4u) a += s_partial[j];     // one partial per warp
                    else for (uint32_t j = sb0; j < sb0 + spb; ++j) a += s_partial[j];
                    norm = (float)sqrt(a);
                } else {
                    uint32_t mxb = 0;
                    if (coarse) for (uint32_t j = sb0 + 3u; j < sb0 + spb; j += 4u) mxb = max(mxb, s_maxbits[j]);
                    else for (uint32_t j = sb0; j < sb0 + spb; ++j) mxb = max(mxb, s_maxbits[j]);
                    norm = __uint_as_float(mxb);
                }
                if (norm != norm) norm = __uint_as_float(0x7fc00000u);     // one NaN pattern in the stream
                float inv = 0.0f;                                           // 0: the bucket is not quantized
                if (norm > 0.0f && norm < __uint_as_float(0x7f800000u)) {
                    inv = __fdiv_rn(top, norm);                             // one IEEE division per bucket
                    if (!(inv < __uint_as_float(0x7f800000u))) inv = 0.0f;
                }
                // a bucket that cannot be quantized although it is not all zero: tell the caller
                if (__any_sync(0xffffffffu, inv == 0.0f && norm != 0.0f && lane < nsb_tile) && lane == 0)
                    latch_status(P.ws, kWarnNonfinite);
                s_sb_inv[lane] = inv;
                s_sb_norm[lane] = norm;
                if (MODE == kModeErc && lane == sb0 && lane < nsb_tile) s_meta[it & 1u].blk_norm[bi] = __float_as_uint(norm);
            }
        }
        bar_sync<kBarWork, kEncThreads>();                    // the one barrier of a tile: norms visible,
                                                            // and every warp is done with the previous tile
        // the ticket of the tile after the next is taken now: its round trip ends long before anyone looks
        if (tid == 0) take_ticket(it + 2u);
        if (cl > 1u && tid == 0 && crank == 0) hand_out_bucket(it + 3u);   // seen by the others after the next exchange of norms

        TileMeta* const meta = &s_meta[it & 1u];
        uint32_t* const window = windows + ((it & 1u) * kEncWarps + warp) * P.window_words;   // this warp's token string
        // ---- quantize (Definition 1) and emit, one sub-block (two 128-element rows) at a time ----
        uint32_t bits = 0;                                  // ERC: bits in this warp's window so far
        uint32_t cum = 0;                                   // ERC: nonzero symbols so far (warp uniform)
        // fixed-width mode: where a sub-block's 8 * width words go and how many of them exist
        uint32_t* fx_rec = nullptr;
        uint32_t fx_sb = 0, fx_words = 0;                   // sub-block within its record, valid field words of the record
#pragma unroll 1
        for (uint32_t q = 0; q < 4; ++q) {
            const uint32_t sbq = warp * 4u + q;
            const uint32_t start_bits = bits;
            if (sbq >= nsb_tile) {
                if (MODE == kModeErc && lane == 0) {
                    meta->sb_bits[sbq] = 0;
                    meta->sb_src[sbq] = bits;
                }
                continue;
            }
            const float inv = s_sb_inv[sbq];

            uint32_t* fx_dst = nullptr;
            uint32_t fx_valid = 0;
            if (MODE == kModeFixed) {
                if (q == 0 || !coarse) {
                    const uint32_t bi = s_sb_bi[sbq];
                    uint32_t rec_len;
                    if (narrow) {
                        fx_rec = payload + (ti.first_block + bi) * G.rec_words;
                        fx_sb = sbq - bi * spb;
                        rec_len = min(G.bucket, tile_len - bi * G.bucket);
                    } else {
                        fx_rec = payload + ti.bucket_idx * G.rec_words;
                        fx_sb = ti.bib * 32u + sbq;
                        rec_len = ti.rec_len;
                    }
                    fx_words = (rec_len * G.width + 31u) / 32u;
                } else {
                    fx_sb += 1u;
                }
                const uint32_t sbw = 8u * G.width;          // words of a full sub-block
                if (fx_sb == 0 && lane == 0) fx_rec[0] = __float_as_uint(s_sb_norm[sbq]);
                fx_dst = fx_rec + 1u + fx_sb * sbw;
                fx_valid = min(sbw, fx_words - fx_sb * sbw);
            }

            if (inv != 0.0f) {
                const float4 x0 = rows[32 * (2 * q)], x1 = rows[32 * (2 * q + 1)];
                __syncwarp();                               // the sub-block's bytes are in registers: their place is scratch now
                const uint4 r0 = rn0, r1 = rn1;
                uint32_t qa[8];
                if (LEVELSET == kLevelsTable) {
                    qa[0] = quantize_table(x0.x, inv, G.s, r0.x, s_levels, s_invw); qa[1] = quantize_table(x0.y, inv, G.s, r0.y, s_levels, s_invw);
                    qa[2] = quantize_table(x0.z, inv, G.s, r0.z, s_levels, s_invw); qa[3] = quantize_table(x0.w, inv, G.s, r0.w, s_levels, s_invw);
                    qa[4] = quantize_table(x1.x, inv, G.s, r1.x, s_levels, s_invw); qa[5] = quantize_table(x1.y, inv, G.s, r1.y, s_levels, s_invw);
                    qa[6] = quantize_table(x1.z, inv, G.s, r1.z, s_levels, s_invw); qa[7] = quantize_table(x1.w, inv, G.s, r1.w, s_levels, s_invw);
                } else if (LEVELSET == kLevelsExp) {
                    qa[0] = quantize_exp(x0.x, inv, top, r0.x); qa[1] = quantize_exp(x0.y, inv, top, r0.y);
                    qa[2] = quantize_exp(x0.z, inv, top, r0.z); qa[3] = quantize_exp(x0.w, inv, top, r0.w);
                    qa[4] = quantize_exp(x1.x, inv, top, r1.x); qa[5] = quantize_exp(x1.y, inv, top, r1.y);
                    qa[6] = quantize_exp(x1.z, inv, top, r1.z); qa[7] = quantize_exp(x1.w, inv, top, r1.w);
                } else {
                    qa[0] = quantize_uniform(x0.x, inv, top, r0.x); qa[1] = quantize_uniform(x0.y, inv, top, r0.y);
                    qa[2] = quantize_uniform(x0.z, inv, top, r0.z); qa[3] = quantize_uniform(x0.w, inv, top, r0.w);
                    qa[4] = quantize_uniform(x1.x, inv, top, r1.x); qa[5] = quantize_uniform(x1.y, inv, top, r1.y);
                    qa[6] = quantize_uniform(x1.z, inv, top, r1.z); qa[7] = quantize_uniform(x1.w, inv, top, r1.w);
                }
                const uint32_t xb[8] = {__float_as_uint(x0.x), __float_as_uint(x0.y), __float_as_uint(x0.z), __float_as_uint(x0.w),
                                        __float_as_uint(x1.x), __float_as_uint(x1.y), __float_as_uint(x1.z), __float_as_uint(x1.w)};
                // Exponential levels: the four symbols of a row as bytes, index | sign << 7.
                uint32_t f0 = 0, f1 = 0, nz0 = 0, nz1 = 0;
                if (kSmall) {
                    const uint32_t syms0 = qa[0] | (qa[1] << 8) | (qa[2] << 16) | (qa[3] << 24);
                    const uint32_t syms1 = qa[4] | (qa[5] << 8) | (qa[6] << 16) | (qa[7] << 24);
                    // top bytes of the four inputs: their sign bits at bits 7, 15, 23, 31
                    const uint32_t tops0 = __byte_perm(__byte_perm(xb[0], xb[1], 0x0073), __byte_perm(xb[2], xb[3], 0x0073), 0x5410);
                    const uint32_t tops1 = __byte_perm(__byte_perm(xb[4], xb[5], 0x0073), __byte_perm(xb[6], xb[7], 0x0073), 0x5410);
                    nz0 = (syms0 + 0x7F7F7F7Fu) & 0x80808080u;                  // bit 7 of a byte: symbol != 0
                    nz1 = (syms1 + 0x7F7F7F7Fu) & 0x80808080u;
                    f0 = syms0 | (tops0 & nz0);                                 // a zero symbol carries no sign
                    f1 = syms1 | (tops1 & nz1);
                }

                if (MODE == kModeErc) {
                    // ---- keep the nonzero symbols, in element order: a lane's rank = nonzeros of row 0 in lower
                    // lanes (+ all of row 0 and those of row 1 in lower lanes, for its row-1 elements) ----
                    uint32_t cnt0, cnt1;
                    if (kSmall) {
                        cnt0 = __popc(nz0);
                        cnt1 = __popc(nz1);
                    } else {
                        cnt0 = (qa[0] != 0) + (qa[1] != 0) + (qa[2] != 0) + (qa[3] != 0);
                        cnt1 = (qa[4] != 0) + (qa[5] != 0) + (qa[6] != 0) + (qa[7] != 0);
                    }
                    const uint32_t packed = cnt0 | (cnt1 << 16);
                    const uint32_t incl = warp_incl_scan(packed);
                    const uint32_t totals = __shfl_sync(0xffffffffu, incl, 31);
                    const uint32_t tot0 = totals & 0xffffu;
                    const uint32_t ntok = tot0 + (totals >> 16);
                    uint32_t at0 = (incl & 0xffffu) - cnt0, at1 = tot0 + (incl >> 16) - cnt1;
                    uint32_t* list32 = reinterpret_cast<uint32_t*>(data + wbase + q * kSB);   // over the sub-block's own bytes
                    uint16_t* list16 = reinterpret_cast<uint16_t*>(list32);
                    if (kSmall) {
                        // 16-bit entries position | field << 8, two at a time by byte permutation
                        const uint32_t pb0 = (lane * 4u) * 0x01010101u + 0x03020100u;      // the four positions of row 0, one per byte
                        const uint32_t pb1 = pb0 + 0x80808080u;                            // ... of row 1
                        const uint32_t a01 = __byte_perm(pb0, f0, 0x5140), a23 = __byte_perm(pb0, f0, 0x7362);
                        const uint32_t b01 = __byte_perm(pb1, f1, 0x5140), b23 = __byte_perm(pb1, f1, 0x7362);
                        if (qa[0]) list16[at0++] = (uint16_t)a01;
                        if (qa[1]) list16[at0++] = (uint16_t)(a01 >> 16);
                        if (qa[2]) list16[at0++] = (uint16_t)a23;
                        if (qa[3]) list16[at0++] = (uint16_t)(a23 >> 16);
                        if (qa[4]) list16[at1++] = (uint16_t)b01;
                        if (qa[5]) list16[at1++] = (uint16_t)(b01 >> 16);
                        if (qa[6]) list16[at1++] = (uint16_t)b23;
                        if (qa[7]) list16[at1++] = (uint16_t)(b23 >> 16);
                    } else {
                        // 32-bit entries position | field << 10, field = index | sign << 15
#pragma unroll
                        for (int c = 0; c < 4; ++c) {
                            if (qa[c]) list32[at0++] = (lane * 4u + c) | ((qa[c] | ((xb[c] >> 16) & 0x8000u)) << 10);
                        }
#pragma unroll
                        for (int c = 4; c < 8; ++c) {
                            if (qa[c]) list32[at1++] = (128u + lane * 4u + (c - 4)) | ((qa[c] | ((xb[c] >> 16) & 0x8000u)) << 10);
                        }
                    }
                    __syncwarp();
                    // ---- tokens ERC(gap) sign ERC(index), 32 per step, appended to the warp's window ----
                    int carry_pos = -1;                         // position of the last nonzero so far: the run starts at t_0 = 0
                    for (uint32_t t0 = 0; t0 < ntok; t0 += 32) {
                        const bool valid = t0 + lane < ntok;
                        uint32_t e = 0;
                        if (valid) e = kSmall ? (uint32_t)list16[t0 + lane] : list32[t0 + lane];
                        const int pos = (int)(e & (kSmall ? 255u : 1023u));
                        const uint32_t field = e >> (kSmall ? 8 : 10);
                        int prev = __shfl_up_sync(0xffffffffu, pos, 1);
                        if (lane == 0) prev = carry_pos;
                        uint32_t gl = 0;                        // stays 0 in lanes without a token: no bits, no length
                        if (valid) gl = s_lut[(pos - prev - 1) & 255];
                        uint32_t tlen, tokA, lenA, tokB = 0, lenB = 0;
                        if (kSmall) {
                            // both codes left aligned with their length in the low bits: the token is the gap code
                            // followed by sign and index code, i.e. the second shifted right by the first's length
                            const uint32_t ll = s_lut_signed[field & 255u];
                            lenA = (gl & 31u) + (ll & 31u);
                            tokA = (gl & ~31u) | ((ll & ~31u) >> (gl & 31u));     // <= 16 + 8 bits, left aligned
                            tlen = lenA;
                        } else {
                            const uint32_t ll = s_lut[((field & S::kMask) - 1u) & 255u];
                            lenA = gl & 31u;
                            tokA = gl & ~31u;
                            lenB = valid ? (ll & 31u) + 1u : 0u;                  // sign + ERC(index) <= 17 bits
                            tokB = valid ? ((field >> S::kBits) << 31) | ((ll & ~31u) >> 1) : 0u;
                            tlen = lenA + lenB;
                        }
                        const uint32_t incl_bits = warp_incl_scan(tlen);
                        const uint32_t step_bits = __shfl_sync(0xffffffffu, incl_bits, 31);
                        // the window is sized for the most bits the warp's elements can produce; checked all the same
                        if (bits + step_bits > 32u * (P.window_words - 2u)) {
                            if (lane == 0) latch_status(P.ws, kErrInternal);
                            break;
                        }
                        const uint32_t off = bits + incl_bits - tlen;     // bit of the window where my token starts
                        or_bits_left(window, off, tokA);
                        if (!kSmall) or_bits_left(window, off + lenA, tokB);
                        bits += step_bits;
                        carry_pos = __shfl_sync(0xffffffffu, pos, min(ntok - t0, 32u) - 1u);
                    }
                    cum += ntok;
                    __syncwarp();
                } else {
                    // ---- fixed-width fields (sign bit, then the level index), MSB first ----
                    const uint32_t wbits = G.width;
                    if (kSmall && wbits == 4u) {
                        // nibbles sign << 3 | index of the four elements of a row, first element on top
                        auto pack4 = [](uint32_t f) {
                            const uint32_t t = (f & 0x07070707u) | ((f >> 4) & 0x08080808u);    // one nibble per byte
                            const uint32_t r = __byte_perm(t, 0u, 0x0213);                       // bytes n0 n2 n1 n3 from the top
                            return (r | (r >> 12)) & 0xffffu;                                    // n0 n1 n2 n3
                        };
                        const uint32_t h0 = pack4(f0), h1 = pack4(f1);
                        // even lanes finish a word of row 0, odd lanes one of row 1: the halves trade places
                        const uint32_t got = __shfl_xor_sync(0xffffffffu, (lane & 1u) ? h0 : h1, 1);
                        const uint32_t word = (lane & 1u) ? (got << 16) | h1 : (h0 << 16) | got;
                        const uint32_t wi = (lane & 1u) * 16u + (lane >> 1);
                        if (wi < fx_valid) fx_dst[wi] = word;
                        cta_nnz += __popc(nz0) + __popc(nz1);
                    } else {
                        uint32_t ff[8];
#pragma unroll
                        for (int c = 0; c < 8; ++c) {
                            if (kSmall) ff[c] = ((c < 4 ? f0 : f1) >> (8 * (c & 3))) & 0xffu;
                            else ff[c] = qa[c] | (qa[c] ? (xb[c] >> 16) & 0x8000u : 0u);
                            cta_nnz += qa[c] != 0;
                        }
                        // the sub-block's fields are put together over its own bytes, then copied out
                        uint32_t* stg = reinterpret_cast<uint32_t*>(data + wbase + q * kSB);
                        for (uint32_t i = lane; i < 8u * wbits + 2u; i += 32) stg[i] = 0;
                        __syncwarp();
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            uint64_t str = 0;
#pragma unroll
                            for (int c = 0; c < 4; ++c) {
                                const uint32_t f = ff[4 * h + c];
                                str = (str << wbits) | ((f & S::kMask) | ((f >> S::kBits) << (wbits - 1u)));
                            }
                            if (str) or_bits(stg, (h * 128u + lane * 4u) * wbits, str, 4u * wbits);
                        }
                        __syncwarp();
                        for (uint32_t i = lane; i < fx_valid; i += 32) fx_dst[i] = stg[i];
                    }
                }
            } else if (MODE == kModeFixed) {
                for (uint32_t i = lane; i < fx_valid; i += 32) fx_dst[i] = 0;      // a bucket that is not quantized: all fields zero
            }
            if (MODE == kModeErc && lane == 0) {
                meta->sb_bits[sbq] = bits - start_bits;
                meta->sb_src[sbq] = start_bits;
            }
            if (q < 3u) {                                   // the draws of the next sub-block
                const uint64_t ctr0 = ctr_warp + 64u * (q + 1u), ctr1 = ctr0 + 32u;
                rn0 = philox4x32_10((uint32_t)ctr0, (uint32_t)(ctr0 >> 32), c2, c3, P.round_keys);
                rn1 = philox4x32_10((uint32_t)ctr1, (uint32_t)(ctr1 >> 32), c2, c3, P.round_keys);
            }
        }

        // The warp is done with its part of the tile (and with the lists that lay over it): the bytes of its
        // part of the next tile are asked for now and arrive while the warp finishes this one.
        __syncwarp();
        if (lane == 0) start_copy(it + 1u);
        if (MODE == kModeErc) {
            if (lane == 0) {
                meta->wnnz[warp] = cum;
                if (warp == 0) {
                    meta->tile = tile;
                    meta->nsb = nsb_tile;
                }
            }
            __syncwarp();
            pair_arrive<kBarDone>(it & 1u);                 // the writer may lay the tile out
            if (it > 0) merge_tile(it - 1u, prev_bits);     // the tile before it has been laid out long ago
            prev_bits = bits;
        }
    }

    if (MODE == kModeErc && !writer) {
        // ---- the workers ran `it` iterations: tell the writer that no further tile comes, and move the
        // last tile's strings into its image ----
        if (tid == 0) s_tot.stop = it;
        pair_arrive<kBarDone>(it & 1u);
        if (it > 0) merge_tile(it - 1u, prev_bits);
    }
    if (MODE == kModeFixed) {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) cta_nnz += __shfl_xor_sync(0xffffffffu, cta_nnz, o);
        if (lane == 0 && cta_nnz) atomicAdd(&s_nnz, cta_nnz);
    }
    __syncthreads();                                        // every write of this CTA lies behind this barrier
    if (tid == 0) {
        const bool last = MODE == kModeErc ? finish_cta<MODE>(P, s_tot.nnz, s_tot.code_bits) : finish_cta<MODE>(P, s_nnz, 0);
        if (last) s_last = 1;
    }
    __syncthreads();
    if (s_last) {
        // Every tile of the call has been written: nobody looks at the call's scan state any more.  The CTA
        // that finished last leaves it zeroed, so the next call on this workspace starts without a clearing pass.
        uint64_t* state = reinterpret_cast<uint64_t*>(reinterpret_cast<char*>(P.ws) + kWorkspaceClearFrom);
        const uint64_t n = (sizeof(Workspace) - kWorkspaceClearFrom) / 8 + (MODE == kModeErc ? G.ntiles + (G.ntiles + 31) / 32 : 0);
        for (uint64_t i = tid; i < n; i += blockDim.x) state[i] = 0;    // (only the ERC mode keeps state per tile)
    }
    if (cl > 1u) cluster_sync_all();                        // nobody leaves while another CTA may still write into its shared memory
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

// ---------------------------------------------------------------------------
// Level histogram: how often each level index 0..s+1 comes out of the quantizer (Definition 1) for the
// given vector, seed and offset: the sample on which a code for the level indices is fitted (Sec. 5,
// "efficient encoding").  The quantizer and the draws are the encoder's; the bucket norms are given.
// Not part of the per-step path: a plain grid-stride loop, four elements (one Philox block) per thread.
// ---------------------------------------------------------------------------
template <uint32_t LEVELSET>
__global__ void __launch_bounds__(256) level_histogram_kernel(const __grid_constant__ EncodeParams P,
                                                              unsigned long long* __restrict__ hist) {
    __shared__ unsigned int s_hist[kMaxTableS + 2];
    __shared__ float s_levels[kMaxTableS + 2], s_invw[kMaxTableS + 2];
    const Geometry& G = P.geo;
    const uint32_t tid = threadIdx.x;
    if (tid < kMaxTableS + 2u) {
        s_hist[tid] = 0;
        s_levels[tid] = P.levels[tid];
        s_invw[tid] = P.inv_width[tid];
    }
    __syncthreads();
    const float top = LEVELSET == kLevelsTable ? 1.0f : __uint_as_float((127u + G.s) << 23);
    const float inf = __uint_as_float(0x7f800000u);
    const uint64_t nquads = (G.d + 3) / 4;
    uint32_t zeros = 0;
    for (uint64_t q = blockIdx.x * 256ull + tid; q < nquads; q += gridDim.x * 256ull) {
        const uint64_t i0 = 4 * q;                          // a bucket is a multiple of 4 elements: one norm
        const float norm = __ldg(P.norms_in + i0 / G.bucket);
        float inv = 0.0f;                                   // 0: the bucket is not quantized
        if (norm > 0.0f && norm < inf) {
            inv = __fdiv_rn(top, norm);
            if (!(inv < inf)) inv = 0.0f;
        }
        const uint4 r = philox4x32_10((uint32_t)q, (uint32_t)(q >> 32), (uint32_t)P.offset, (uint32_t)(P.offset >> 32),
                                      P.round_keys);
        const uint32_t w[4] = {r.x, r.y, r.z, r.w};
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            if (i0 + c >= G.d) break;
            const float v = __ldg(P.g + i0 + c);
            const uint32_t sym = LEVELSET == kLevelsTable ? quantize_table(v, inv, G.s, w[c], s_levels, s_invw)
                                                          : quantize_exp(v, inv, top, w[c]);
            if (sym) atomicAdd(&s_hist[sym], 1u);
            else ++zeros;
        }
    }
    zeros = __reduce_add_sync(0xffffffffu, zeros);
    if ((tid & 31u) == 0 && zeros) atomicAdd(&s_hist[0], zeros);
    __syncthreads();
    if (tid < G.s + 2u && s_hist[tid]) atomicAdd(hist + tid, (unsigned long long)s_hist[tid]);
}

cudaError_t launch_level_histogram(const EncodeParams& P, uint64_t* hist, int sms, cudaStream_t stream) {
    const uint64_t nquads = (P.geo.d + 3) / 4;
    const uint64_t want = (nquads + 255) / 256, cap = (uint64_t)sms * 8u;
    const unsigned grid = (unsigned)(want < cap ? want : cap);
    if (P.geo.levelset == kLevelsTable)
        level_histogram_kernel<kLevelsTable><<<grid, 256, 0, stream>>>(P, reinterpret_cast<unsigned long long*>(hist));
    else
        level_histogram_kernel<kLevelsExp><<<grid, 256, 0, stream>>>(P, reinterpret_cast<unsigned long long*>(hist));
    return cudaGetLastError();
}

// shared memory of one CTA: the tile buffers and, in the ERC mode, two staged tile images and two sets of per-warp token windows
size_t encode_smem_bytes(const EncodeParams& P) {
    if (fixed4_applies(P.geo)) return 0;                    // that kernel's tile buffer is static
    size_t words = kBLK;
    if (P.geo.mode != kModeFixed) words += 2u * (size_t)P.stage_words + 2u * (size_t)kEncWarps * P.window_words;
    return 4u * words;
}

constexpr int kEncMaxDynSmem = 112 * 1024;

template <uint32_t L, uint32_t M>
static cudaError_t prepare_kernel() {
    static bool attr_set = false;
    if (attr_set) return cudaSuccess;
    cudaError_t e = cudaFuncSetAttribute(encode_kernel<L, M, false>, cudaFuncAttributeMaxDynamicSharedMemorySize, kEncMaxDynSmem);
    if (e == cudaSuccess)
        e = cudaFuncSetAttribute(encode_kernel<L, M, true>, cudaFuncAttributeMaxDynamicSharedMemorySize, kEncMaxDynSmem);
    if (e == cudaSuccess) attr_set = true;
    return e;
}

template <uint32_t L, uint32_t M>
static int blocks_per_sm(const EncodeParams& P) {
    if (prepare_kernel<L, M>() != cudaSuccess) return 0;
    int n = 0;
    const int threads = M == kModeErc ? (int)kEncAllThreads : kEncThreads;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, encode_kernel<L, M, false>, threads, encode_smem_bytes(P)) != cudaSuccess)
        return 0;
    return n;
}

int encode_blocks_per_sm(const EncodeParams& P) {
    if (fixed4_applies(P.geo)) return fixed4_blocks_per_sm(P);
    const bool uni = P.geo.levelset == kLevelsUniform, fixed = P.geo.mode == kModeFixed;
    if (encode_smem_bytes(P) > (size_t)kEncMaxDynSmem) return 0;
    if (P.geo.levelset == kLevelsTable) return fixed ? blocks_per_sm<kLevelsTable, kModeFixed>(P) : blocks_per_sm<kLevelsTable, kModeErc>(P);
    if (!uni && !fixed) return blocks_per_sm<kLevelsExp, kModeErc>(P);
    if (!uni && fixed) return blocks_per_sm<kLevelsExp, kModeFixed>(P);
    if (uni && !fixed) return blocks_per_sm<kLevelsUniform, kModeErc>(P);
    return blocks_per_sm<kLevelsUniform, kModeFixed>(P);
}

// launch configuration of a call, with the cluster shape when it has one
struct EncodeLaunch {
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[2];
};
template <uint32_t M>
static void fill_launch(EncodeLaunch* L, const EncodeParams& P, unsigned grid, cudaStream_t stream) {
    L->cfg = cudaLaunchConfig_t{};
    L->cfg.gridDim = dim3(grid);
    L->cfg.blockDim = dim3(M == kModeErc ? kEncAllThreads : (uint32_t)kEncThreads);
    L->cfg.dynamicSmemBytes = encode_smem_bytes(P);
    L->cfg.stream = stream;
    L->cfg.attrs = L->attr;
    L->cfg.numAttrs = 0;
    if (P.cluster > 1u) {
        cudaLaunchAttribute& a = L->attr[L->cfg.numAttrs++];
        a.id = cudaLaunchAttributeClusterDimension;
        a.val.clusterDim.x = P.cluster;
        a.val.clusterDim.y = 1;
        a.val.clusterDim.z = 1;
    }
    if (P.overlap) {                                        // may be set up while the kernel before it in the stream ends
        cudaLaunchAttribute& a = L->attr[L->cfg.numAttrs++];
        a.id = cudaLaunchAttributeProgrammaticStreamSerialization;
        a.val.programmaticStreamSerializationAllowed = 1;
    }
}

template <uint32_t L, uint32_t M>
static cudaError_t launch_one(const EncodeParams& P, cudaStream_t stream) {
    const size_t smem = encode_smem_bytes(P);
    cudaError_t e = prepare_kernel<L, M>();
    if (e != cudaSuccess) return e;
    if (smem > (size_t)kEncMaxDynSmem || P.grid == 0 || (P.cluster > 1u && P.grid % P.cluster != 0)) return cudaErrorInvalidValue;
    EncodeLaunch cfg;
    fill_launch<M>(&cfg, P, P.grid, stream);
    if (P.cluster > 1u) return cudaLaunchKernelEx(&cfg.cfg, encode_kernel<L, M, true>, P);
    return cudaLaunchKernelEx(&cfg.cfg, encode_kernel<L, M, false>, P);
}

// clusters of P.cluster CTAs the device holds at once (0 on error)
template <uint32_t L, uint32_t M>
static int max_clusters(const EncodeParams& P) {
    if (prepare_kernel<L, M>() != cudaSuccess) return 0;
    EncodeLaunch cfg;
    fill_launch<M>(&cfg, P, P.cluster, nullptr);
    int n = 0;
    if (cudaOccupancyMaxActiveClusters(&n, encode_kernel<L, M, true>, &cfg.cfg) != cudaSuccess) {
        cudaGetLastError();
        return 0;
    }
    return n;
}

int encode_max_clusters(const EncodeParams& P) {
    const bool uni = P.geo.levelset == kLevelsUniform, fixed = P.geo.mode == kModeFixed;
    if (encode_smem_bytes(P) > (size_t)kEncMaxDynSmem) return 0;
    if (P.geo.levelset == kLevelsTable) return fixed ? max_clusters<kLevelsTable, kModeFixed>(P) : max_clusters<kLevelsTable, kModeErc>(P);
    if (!uni && !fixed) return max_clusters<kLevelsExp, kModeErc>(P);
    if (!uni && fixed) return max_clusters<kLevelsExp, kModeFixed>(P);
    if (uni && !fixed) return max_clusters<kLevelsUniform, kModeErc>(P);
    return max_clusters<kLevelsUniform, kModeFixed>(P);
}

cudaError_t launch_encode(const EncodeParams& P, cudaStream_t stream) {
    if (fixed4_applies(P.geo)) return launch_encode_fixed4(P, stream);
    const bool uni = P.geo.levelset == kLevelsUniform, fixed = P.geo.mode == kModeFixed;
    if (P.geo.levelset == kLevelsTable) return fixed ? launch_one<kLevelsTable, kModeFixed>(P, stream) : launch_one<kLevelsTable, kModeErc>(P, stream);
    if (!uni && !fixed) return launch_one<kLevelsExp, kModeErc>(P, stream);
    if (!uni && fixed) return launch_one<kLevelsExp, kModeFixed>(P, stream);
    if (uni && !fixed) return launch_one<kLevelsUniform, kModeErc>(P, stream);
    return launch_one<kLevelsUniform, kModeFixed>(P, stream);
}

}  // namespace nuq
