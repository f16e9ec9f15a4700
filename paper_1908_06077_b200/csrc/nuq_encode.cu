// ENCODE of NUQSGD (App. A) for one gradient vector: bucket norm, stochastic
// quantization (Definition 1) and Elias-recursive token packing in one kernel
// that reads the gradient from HBM exactly once.
//
// A persistent CTA takes tiles of up to 8192 consecutive elements (whole buckets, or
// one 8192-element coding block of a wider bucket) by ticket.  Eight worker warps
// encode the tile; in the ERC mode a ninth warp, the writer, finds the tile's place
// in the stream and copies it out, so the workers never wait for other CTAs.
// The tile's bytes are brought into shared memory by one bulk asynchronous copy
// (TMA, completion on an mbarrier); the copy of the next tile is started as soon
// as the current tile has been quantized, so HBM latency hides behind the packing
// of the current tile and behind the other CTAs of the SM.  Per tile:
//   1. each warp reduces the squares (fp64) of its 1024 elements per sub-block;
//      after one barrier every warp derives the bucket norms it needs;
//   2. each warp quantizes its elements 256 at a time (one 128-bit shared-memory
//      load and one Philox block per lane and 128-element row), compacts the
//      nonzero symbols with ballots into a dense list, and turns that list into
//      tokens, 32 per step, appended to the warp's own bit string;
//   3. after a second barrier every warp runs the same small scan over the 32
//      sub-block lengths, which gives the layout of the tile's records, and
//      shifts its strings to their place in one of two staged tile images; the
//      tile's size is announced to the tiles behind it at once;
//   4. the writer warp, woken through a named barrier, sums the sizes announced
//      by the tile's predecessors (two-level decoupled look-back: single tiles
//      within a group of 32, whole groups before that; bounded waits), copies the
//      staged image to its place, writes the block offsets and hands the stage
//      back through a second named barrier.  The workers meet the writer again
//      only two tiles later, when they need that stage.
// In the fixed-width mode the fields go straight to their known place and there
// is no writer warp.  Counters and the container header are written once per CTA,
// the header by whichever CTA finishes last.
//
// The kernel is bound by instruction issue, not by HBM: the quantizer is branch
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
//   only if u < y as well.
// y < 1 (r in [0, 2^-s]): p = y, and u < y  <=>  float(m) < y 2^24 (both sides exact).
// With up = [float(m) < y 2^24] (always true for y >= 1) the index is max(hi, 1) if up, else 0.
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t quantize_exp(float v, float inv, float top, uint32_t word) {
    const float y = fminf(__fmul_rn(fabsf(v), inv), top);
    const int hi = (int)(__float_as_uint(y) + (0x007FFFFFu - 0x3F000000u) - (word >> 9)) >> 23;
    const bool up = __uint2float_rn(word >> 8) < __fmul_rn(y, 16777216.0f);
    return up ? (uint32_t)max(hi, 1) : 0u;                  // no round-up: y < 1 and the index is 0
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
constexpr uint32_t kGroupTiles = 32;
constexpr uint32_t kGroupCountShift = 48;
constexpr uint64_t kGroupSumMask = (1ull << kGroupCountShift) - 1;

// The workers' side: tile `tile` takes `words` words.
__device__ __forceinline__ void announce_tile(uint64_t* tile_state, uint64_t* group_state, uint64_t tile, uint32_t words) {
    st_volatile_u64(tile_state + tile, kTileAggregate | words);
    atomicAdd(reinterpret_cast<unsigned long long*>(group_state + tile / kGroupTiles),
              (1ull << kGroupCountShift) | (unsigned long long)words);
}

// One more poll of a look-back wait; false when the patience is used up (tens of ms).
__device__ __forceinline__ bool lookback_backoff(Workspace* ws, uint32_t& polls) {
    if (++polls > (1u << 16)) {
        if (lane_id() == 0) latch_status(ws, kErrTimeout);
        return false;
    }
    __nanosleep(polls < 64 ? 250 : 1000);                   // a waiting warp should not eat issue slots
    return true;
}

__device__ uint64_t tile_lookback(Workspace* ws, const uint64_t* tile_state, uint64_t* group_state, uint64_t tile,
                                  uint64_t ntiles, uint32_t words, bool* failed) {
    const uint32_t lane = lane_id();
    const uint64_t grp = tile / kGroupTiles;
    const uint32_t r = (uint32_t)(tile % kGroupTiles);      // tiles of the group before this one
    uint32_t polls = 0;
    uint64_t exclusive = 0;
    *failed = true;
    // ---- the tiles before this one in its own group ----
    for (;;) {
        const uint64_t v = lane < r ? ld_volatile_u64(tile_state + grp * kGroupTiles + lane) : kTileAggregate;
        const uint32_t missing = __ballot_sync(0xffffffffu, (v >> 62) != 1);
        if (!missing) {
            exclusive = __reduce_add_sync(0xffffffffu, (uint32_t)v);           // a tile has far fewer than 2^27 words
            break;
        }
        // wait for the first missing one alone, then look at all of them again
        const uint64_t* p = tile_state + grp * kGroupTiles + (__ffs(missing) - 1);
        while ((ld_volatile_u64(p) >> 62) != 1)
            if (!lookback_backoff(ws, polls)) return 0;
    }
    // ---- whole groups, nearest first: lane l looks at groups base - l and base - 32 - l ----
    int64_t base = (int64_t)grp - 1;
    while (base >= 0) {
        const int64_t i0 = base - (int64_t)lane, i1 = i0 - 32;
        const uint64_t v0 = i0 >= 0 ? ld_volatile_u64(group_state + i0) : kTilePrefix;    // before group 0: prefix 0
        const uint64_t v1 = i1 >= 0 ? ld_volatile_u64(group_state + i1) : kTilePrefix;
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
                if ((v >> 62) == 2 || (v >> kGroupCountShift) == kGroupTiles) break;
                if (!lookback_backoff(ws, polls)) return 0;
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
    if (r == kGroupTiles - 1u || tile == ntiles - 1) {
        const uint64_t members = tile == ntiles - 1 ? r + 1u : kGroupTiles;
        for (;;) {                                          // every member's size has been added (they were all seen above)
            const uint64_t v = ld_volatile_u64(group_state + grp);
            if ((v >> kGroupCountShift) == members) break;
            if (!lookback_backoff(ws, polls)) return 0;
        }
        if (lane == 0) st_volatile_u64(group_state + grp, kTilePrefix | (exclusive + words));
    }
    *failed = false;
    return exclusive;
}

// ---------------------------------------------------------------------------
// Bulk asynchronous copy (TMA, untiled form) and its mbarrier.  One CTA-local
// barrier, never a cluster multicast.
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}

// Announces `bytes` to the barrier and starts the copy global -> shared.  Both addresses
// 16-byte aligned, `bytes` a positive multiple of 16.
__device__ __forceinline__ void bulk_load(void* dst_smem, const void* src_gmem, uint32_t bytes, uint64_t* bar) {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // earlier generic writes to dst are ordered first
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                     smem_u32(dst_smem)),
                 "l"(src_gmem), "r"(bytes), "r"(smem_u32(bar))
                 : "memory");
}

// Waits until the phase with the given parity has completed.  Bounded: false after ~tens of ms.
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
    const uint32_t addr = smem_u32(bar);
    // the hardware parks the thread for up to the hinted time (ns), so a wait costs a handful of
    // instructions; the number of tries bounds the wait (a fraction of a second at most)
    for (uint32_t polls = 0; polls < (1u << 17); ++polls) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(addr), "r"(parity), "r"(2000u)
            : "memory");
        if (done) return true;
    }
    return false;
}

// Symbols travel as small fields: level index in the low bits, sign above it.
template <uint32_t LEVELSET>
struct Sym {
    static constexpr uint32_t kBits = LEVELSET == kLevelsExp ? 7u : 15u;     // index <= 15 resp. <= 256
    static constexpr uint32_t kMask = (1u << kBits) - 1u;
};

// OR `nbits` (0..32) right-aligned bits of `value` into the MSB-first bit string `dst` at `bitpos`.
// Two words are touched unconditionally (a zero is OR-ed when there is nothing to add).
__device__ __forceinline__ void or_bits32(uint32_t* dst, uint32_t bitpos, uint32_t value, uint32_t nbits) {
    const uint32_t a = nbits ? value << (32u - nbits) : 0u;
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

constexpr uint32_t kWarpElems = kBLK / kEncWarps;   // 1024 elements of a tile per warp (4 sub-blocks)
constexpr uint32_t kChunk = kEncChunk;              // elements quantized before their tokens are generated
constexpr uint32_t kChunkRows = kChunk / 128;

// Named CTA barriers.  The 8 worker warps meet at kBarWork; the writer warp (ERC mode) and the
// workers hand the two staged tiles back and forth through kBarStaged + b (workers arrive, the
// writer waits) and kBarFree + b (the writer arrives, workers wait).
constexpr uint32_t kBarWork = 1, kBarStaged = 2, kBarFree = 5;     // kBarStaged + b, kBarFree + b for stage b < 3
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
// the pair of barriers of stage b (0, 1 or 2); immediate barrier numbers, so that the kernel claims only those it uses
template <uint32_t BASE>
__device__ __forceinline__ void stage_sync(uint32_t b) {
    if (b == 0) bar_sync<BASE, kEncAllThreads>();
    else if (b == 1) bar_sync<BASE + 1, kEncAllThreads>();
    else bar_sync<BASE + 2, kEncAllThreads>();
}
template <uint32_t BASE>
__device__ __forceinline__ void stage_arrive(uint32_t b) {
    if (b == 0) bar_arrive<BASE, kEncAllThreads>();
    else if (b == 1) bar_arrive<BASE + 1, kEncAllThreads>();
    else bar_arrive<BASE + 2, kEncAllThreads>();
}

// A tile whose records are staged in shared memory and whose place in the stream is not
// yet known.
struct Pending {
    unsigned long long tile;
    uint32_t words, nblk, code_bits, nnz, valid, pad;
    uint32_t blk_wordoff[32];                              // word offset of block bi within the tile
};

// What a CTA has written so far (shared memory; updated by one thread at a time, CTA barriers in between).
struct CtaTotals {
    uint64_t nnz, code_bits;
    uint32_t tiles, stop;                                  // stop: iterations the workers ran (set when they leave)
};

// Bookkeeping of a CTA that has written all its tiles: counters, and the container header by
// whichever CTA finishes last.  One thread, after a CTA barrier behind the last write.
template <uint32_t MODE>
__device__ void finish_cta(const EncodeParams& P, uint32_t tiles, uint64_t nnz, uint64_t code_bits) {
    const Geometry& G = P.geo;
    if (tiles == 0) return;
    if (nnz) atomicAdd(reinterpret_cast<unsigned long long*>(&P.ws->nnz), (unsigned long long)nnz);
    if (code_bits) atomicAdd(reinterpret_cast<unsigned long long*>(&P.ws->code_bits), (unsigned long long)code_bits);
    __threadfence();
    const unsigned long long prev = atomicAdd(reinterpret_cast<unsigned long long*>(&P.ws->done), (unsigned long long)tiles);
    if (prev + tiles != G.ntiles) return;
    __threadfence();
    uint64_t code_total, words;
    const uint64_t nnz_total = ld_volatile_u64(&P.ws->nnz);
    const uint64_t nrec = MODE == kModeErc ? G.nblk : G.nb;
    if (MODE == kModeErc) {
        code_total = ld_volatile_u64(&P.ws->code_bits);
        words = kHeaderWords + 2 * (G.nblk + 1) + ld_volatile_u64(&P.ws->total_words);
    } else {
        code_total = G.d * G.width;
        const uint64_t last = G.d - (G.nb - 1) * G.bucket;
        words = kHeaderWords + (G.nb - 1) * G.rec_words + 1 + (last * G.width + 31) / 32;
    }
    const uint64_t container_bits = 32 * words;
    uint32_t* h = P.out;
    h[0] = kMagic; h[1] = kVersion;
    h[2] = (uint32_t)G.d; h[3] = (uint32_t)(G.d >> 32);
    h[4] = G.bucket; h[5] = G.s;
    h[6] = G.norm_kind | (G.levelset << 8) | (G.mode << 16);
    h[7] = kSB;
    h[8] = (uint32_t)nrec; h[9] = (uint32_t)(nrec >> 32);
    h[10] = (uint32_t)container_bits; h[11] = (uint32_t)(container_bits >> 32);
    h[12] = (uint32_t)code_total; h[13] = (uint32_t)(code_total >> 32);
    h[14] = (uint32_t)nnz_total; h[15] = (uint32_t)(nnz_total >> 32);
    if (P.out_bits) *P.out_bits = container_bits;
}

// One warp: find the place of a staged tile (its predecessors announced their sizes an
// iteration ago, so the walk rarely waits), copy the image to the stream, clear the stage.
__device__ void flush_pending(const EncodeParams& P, Pending& pd, CtaTotals& tot, uint32_t* stg, const uint64_t* tile_state,
                              uint64_t* group_state, uint64_t* table, uint32_t* payload, uint32_t lane) {
    const Geometry& G = P.geo;
    const uint64_t tile = pd.tile;
    const uint32_t words = pd.words;
    bool failed;
    const uint64_t off = tile_lookback(P.ws, tile_state, group_state, tile, G.ntiles, words, &failed);
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
        pd.valid = 0;
        tot.tiles += 1;
        tot.nnz += pd.nnz;
        tot.code_bits += pd.code_bits;
    }
    __syncwarp();
}

template <uint32_t LEVELSET, uint32_t MODE>
__global__ void __launch_bounds__(kEncAllThreads, kEncMinBlocks) encode_kernel(const __grid_constant__ EncodeParams P) {
    extern __shared__ __align__(128) uint32_t smem[];
    __shared__ __align__(8) uint64_t s_bar;                // completes when the tile's bytes have landed
    __shared__ uint32_t s_lut[256];                        // ERC(N), N = 1..256: code | len << 16
    __shared__ uint32_t s_lut_signed[256];                 // exponential levels: sign bit + ERC(index), by field
    __shared__ double s_partial[32];                       // per sub-block (or per warp) sums of squares
    __shared__ uint32_t s_maxbits[32];                     // ... or max |x| bit patterns
    __shared__ uint32_t s_sb_bits[32];                     // token bits of each sub-block
    __shared__ uint32_t s_sb_src[32];                      // where they start in the owning warp's window
    __shared__ uint32_t s_start[32];                       // scratch: first token offset of a sub-block (per warp 4)
    __shared__ unsigned long long s_tile[2];
    __shared__ uint32_t s_abort, s_nnz;
    __shared__ Pending s_pend[3];                          // ERC: the staged tiles (current and up to two earlier ones)
    __shared__ CtaTotals s_tot;

    using S = Sym<LEVELSET>;
    const Geometry& G = P.geo;
    const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    float* data = reinterpret_cast<float*>(smem);                               // kBLK floats: the tile
    uint32_t* stage = smem + kBLK;                                              // image of the tile's records
    uint32_t* wmem = stage + P.stages * P.stage_words + warp * P.warp_smem_words;
    uint32_t* window = wmem;                                                    // this warp's token string
    uint32_t* tokens = wmem + P.window_words;               // kChunk entries: position | field << 10 (uniform levels)
    uint16_t* tokens16 = reinterpret_cast<uint16_t*>(tokens);   //                position | field << 8  (exponential levels)
    uint64_t* tile_state = reinterpret_cast<uint64_t*>(P.ws + 1);
    uint64_t* group_state = tile_state + G.ntiles;
    uint64_t* table = reinterpret_cast<uint64_t*>(P.out + kHeaderWords);
    uint32_t* payload = MODE == kModeErc ? P.out + kHeaderWords + 2 * (G.nblk + 1) : P.out + kHeaderWords;
    const float top = __uint_as_float((127u + G.s) << 23);
    const uint32_t c2 = (uint32_t)P.offset, c3 = (uint32_t)(P.offset >> 32);
    const uint32_t lt_mask = (1u << lane) - 1u;
    const bool coarse = G.bucket % kWarpElems == 0;         // a warp's four sub-blocks always share one bucket
    const uint32_t spb = G.bucket <= kBLK ? G.sb_per_block : 32u;       // sub-blocks per coding block
    uint32_t bi_q[4];                                       // block (within a tile) of the warp's four sub-blocks
#pragma unroll
    for (int q = 0; q < 4; ++q) bi_q[q] = (warp * 4u + q) / spb;
    const uint32_t bi_lane = lane / spb;                    // block of sub-block `lane`

    // where tile `t` starts and how long it is
    auto tile_span = [&](uint64_t t, uint64_t& elem0, uint32_t& tile_len) {
        if (G.bucket <= kBLK) {
            elem0 = t * G.blocks_per_tile * G.bucket;
            const uint64_t left = G.d - elem0;
            tile_len = left < G.tile_elems ? (uint32_t)left : G.tile_elems;
        } else {
            const uint64_t bucket_idx = t / G.blk_per_bucket;
            const uint32_t bib = (uint32_t)(t % G.blk_per_bucket);
            const uint64_t b0 = bucket_idx * G.bucket;
            const uint64_t blen = G.d - b0 < G.bucket ? G.d - b0 : G.bucket;
            elem0 = b0 + (uint64_t)bib * kBLK;
            const uint64_t left = blen - (uint64_t)bib * kBLK;
            tile_len = left < kBLK ? (uint32_t)left : kBLK;
        }
    };
    // thread 0: take a ticket ...
    auto take_ticket = [&]() { return atomicAdd(reinterpret_cast<unsigned long long*>(&P.ws->ticket), 1ull); };
    // ... and start the copy of that tile into `data` once nobody reads the previous one
    auto start_copy = [&](uint32_t slot) {
        const uint64_t t = s_tile[slot];
        if (t < G.ntiles) {
            uint64_t elem0;
            uint32_t tile_len;
            tile_span(t, elem0, tile_len);
            const uint32_t bytes = (tile_len * 4u) & ~15u;
            if (bytes) bulk_load(data, P.g + elem0, bytes, &s_bar);
        }
    };

    if (tid < 256u) {
        const uint32_t e = c_erc_lut[tid];
        s_lut[tid] = e;
        const uint32_t idx = tid & 0x7Fu;                   // field = sign << 7 | index: sign bit, then ERC(index)
        uint32_t v = 0;
        if (idx >= 1) {
            const uint32_t l = c_erc_lut[idx - 1u], len = l >> 16;
            v = ((tid >> 7) << len) | (l & 0xffffu) | ((len + 1u) << 16);
        }
        s_lut_signed[tid] = v;
    }
    for (uint32_t i = tid; i < P.stages * P.stage_words; i += blockDim.x) stage[i] = 0;
    if (warp < (uint32_t)kEncWarps)
        for (uint32_t i = lane; i < P.window_words; i += 32) window[i] = 0;
    if (tid == 0) {
        mbar_init(&s_bar, 1);
        s_abort = 0;
        s_nnz = 0;
        s_pend[0].valid = 0;
        s_pend[1].valid = 0;
        s_pend[2].valid = 0;
        s_tot.nnz = 0;
        s_tot.code_bits = 0;
        s_tot.tiles = 0;
        s_tot.stop = 0xFFFFFFFFu;
    }
    __syncthreads();
    if (tid == 0) {
        s_tile[0] = take_ticket();
        start_copy(0);
    }
    __syncthreads();

    const bool writer = MODE == kModeErc && warp == (uint32_t)kEncWarps;
    if (writer) {
        // ---- the writer warp: finds the place of every staged tile (look-back), copies it to the
        // stream and hands the stage back; the workers never wait for it unless it falls two tiles behind
        uint32_t b = 0;                                     // stage of tile k: k mod P.stages
        for (uint32_t k = 0;; ++k) {
            stage_sync<kBarStaged>(b);                      // tile k of this CTA is staged
            if (k >= *reinterpret_cast<volatile uint32_t*>(&s_tot.stop)) break;
            flush_pending(P, s_pend[b], s_tot, stage + b * P.stage_words, tile_state, group_state, table, payload, lane);
            stage_arrive<kBarFree>(b);
            b = b + 1u == P.stages ? 0u : b + 1u;
        }
    }

    uint32_t parity = 0;
    uint32_t it = 0, sg = 0;                                // sg: stage of iteration it, it mod P.stages
    for (; !writer; ++it, sg = sg + 1u == P.stages ? 0u : sg + 1u) {           // the 8 worker warps
        const uint64_t tile = s_tile[it & 1u];
        if (tile >= G.ntiles) break;

        // ---- tile geometry ------------------------------------------------------
        uint64_t elem0, first_block, bucket_idx = 0;
        uint32_t tile_len, nblk_tile, blk_elems, bib = 0;
        tile_span(tile, elem0, tile_len);
        if (G.bucket <= kBLK) {
            first_block = tile * G.blocks_per_tile;
            blk_elems = G.bucket;
            nblk_tile = (tile_len + G.bucket - 1) / G.bucket;
        } else {
            bucket_idx = tile / G.blk_per_bucket;
            bib = (uint32_t)(tile % G.blk_per_bucket);
            first_block = tile;
            blk_elems = kBLK;
            nblk_tile = 1;
        }
        const uint32_t nsb_tile = (tile_len + kSB - 1) / kSB;
        const uint32_t wbase = warp * kWarpElems;           // first element of the warp within the tile

        // ---- the tile's bytes: wait for the bulk copy, fetch the ragged end, zero the rest ----
        {
            const uint32_t bulk_elems = ((tile_len * 4u) & ~15u) / 4u;
            if (bulk_elems) {
                if (!mbar_wait(&s_bar, parity)) {           // never seen in practice; do not hang
                    if (tid == 0) {
                        latch_status(P.ws, kErrTimeout);
                        s_abort = 1;
                    }
                }
                parity ^= 1u;
            }
            if (tile_len < kBLK) {
                for (uint32_t i = bulk_elems + tid; i < kBLK; i += kEncThreads)
                    data[i] = i < tile_len ? __ldg(P.g + elem0 + i) : 0.0f;
                bar_sync<kBarWork, kEncThreads>();
            }
        }
        const float4* rows = reinterpret_cast<const float4*>(data + wbase) + lane;   // row j at rows[32 * j]

        // ---- bucket norms: fp64 sums of exact squares (or max |x|), one rounding to fp32 ----
        if (P.norms_in == nullptr) {
            double acc = 0.0;
            uint32_t mx = 0;
#pragma unroll
            for (int q = 0; q < 4; ++q) {
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    const float4 x = rows[32 * (2 * q + h)];
                    if (G.norm_kind == kNormL2) {
                        acc = fma((double)x.x, (double)x.x, acc);
                        acc = fma((double)x.y, (double)x.y, acc);
                        acc = fma((double)x.z, (double)x.z, acc);
                        acc = fma((double)x.w, (double)x.w, acc);
                    } else {                                // on the bit patterns: NaN sorts above inf
                        mx = max(max(mx, __float_as_uint(fabsf(x.x))), __float_as_uint(fabsf(x.y)));
                        mx = max(max(mx, __float_as_uint(fabsf(x.z))), __float_as_uint(fabsf(x.w)));
                    }
                }
                if (!coarse || q == 3) {                    // one partial per sub-block, or one per warp
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) {
                        acc += __shfl_xor_sync(0xffffffffu, acc, o);
                        mx = max(mx, __shfl_xor_sync(0xffffffffu, mx, o));
                    }
                    if (lane == 0) {
                        s_partial[warp * 4 + q] = acc;
                        s_maxbits[warp * 4 + q] = mx;
                    }
                    acc = 0.0;
                    mx = 0;
                } else if (lane == 0) {
                    s_partial[warp * 4 + q] = 0.0;
                    s_maxbits[warp * 4 + q] = 0;
                }
            }
        }
        bar_sync<kBarWork, kEncThreads>();                    // B1: partials visible
        // the next ticket is asked for now and stored just before the next barrier: the round trip
        // of the atomic is over by then
        unsigned long long next_ticket = 0;
        if (tid == 0) next_ticket = take_ticket();

        // every warp derives the norms of the buckets its own sub-blocks belong to (same
        // reduction tree in every warp, so all agree bit for bit)
        float inv_q[4], norm_q[4];
        {
            const double my_part = s_partial[lane];
            const uint32_t my_max = s_maxbits[lane];
#pragma unroll
            for (int q = 0; q < 4; ++q) {
                if (q > 0 && (coarse || bi_q[q] == bi_q[q - 1])) {            // same bucket as the previous sub-block
                    inv_q[q] = inv_q[q - 1];
                    norm_q[q] = norm_q[q - 1];
                    continue;
                }
                const uint32_t bi = bi_q[q], sb0 = bi * spb;
                float norm;
                if (P.norms_in != nullptr) {
                    const uint64_t nb_idx = G.bucket <= kBLK ? first_block + bi : bucket_idx;
                    norm = nb_idx < G.nb ? P.norms_in[nb_idx] : 0.0f;
                } else {
                    const bool in = lane >= sb0 && lane < sb0 + spb;
                    double a = in ? my_part : 0.0;
                    uint32_t m = in ? my_max : 0u;
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) {
                        a += __shfl_xor_sync(0xffffffffu, a, o);
                        m = max(m, __shfl_xor_sync(0xffffffffu, m, o));
                    }
                    norm = G.norm_kind == kNormL2 ? (float)sqrt(a) : __uint_as_float(m);
                }
                if (norm != norm) norm = __uint_as_float(0x7fc00000u);     // one NaN pattern in the stream
                float inv = 0.0f;                                           // 0: the bucket is not quantized
                if (norm > 0.0f && norm < __uint_as_float(0x7f800000u)) {
                    inv = __fdiv_rn(top, norm);                             // one IEEE division per bucket
                    if (!(inv < __uint_as_float(0x7f800000u))) inv = 0.0f;
                }
                inv_q[q] = inv;
                norm_q[q] = norm;
            }
        }

        // ---- quantize (Definition 1) and generate tokens, one chunk of elements at a time ------
        uint32_t bits = 0;                                  // ERC: bits in this warp's window so far
        uint32_t my_nnz = 0;
        if (MODE == kModeErc && lane < 4) s_start[warp * 4 + lane] = 0xFFFFFFFFu;
        // lane q < 4 keeps 2^s / norm and the block of the warp's sub-block q for the loop below
        const float inv_own = (lane & 3u) == 0 ? inv_q[0] : (lane & 3u) == 1 ? inv_q[1] : (lane & 3u) == 2 ? inv_q[2] : inv_q[3];
        const uint32_t bi_own = (lane & 3u) == 0 ? bi_q[0] : (lane & 3u) == 1 ? bi_q[1] : (lane & 3u) == 2 ? bi_q[2] : bi_q[3];
#pragma unroll 1
        for (uint32_t part = 0; part < kWarpElems / kChunk; ++part) {
            uint32_t ntok = 0;
#pragma unroll
            for (uint32_t r = 0; r < kChunkRows; ++r) {
                const uint32_t j = part * kChunkRows + r;   // row of the warp
                const float inv = __shfl_sync(0xffffffffu, inv_own, j >> 1);
                const uint32_t bi_row = __shfl_sync(0xffffffffu, bi_own, j >> 1);   // block of this row's sub-block
                if (inv == 0.0f) continue;                  // bucket not quantized (warp uniform)
                const float4 x = rows[32 * j];
                const uint32_t base = wbase + j * 128u + lane * 4u;             // element within the tile
                const uint64_t ctr = (elem0 + base) >> 2;
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
                // fields (index | sign << kBits); in the fixed-width mode a zero symbol must carry no sign
                uint32_t f = 0, f0 = 0, f1 = 0, f2 = 0, f3 = 0;
                if (LEVELSET == kLevelsExp) {
                    const uint32_t syms = q0 | (q1 << 8) | (q2 << 16) | (q3 << 24);
                    // top bytes of the four inputs: their sign bits at bits 7, 15, 23, 31
                    uint32_t tops = __byte_perm(__byte_perm(__float_as_uint(x.x), __float_as_uint(x.y), 0x0073),
                                                __byte_perm(__float_as_uint(x.z), __float_as_uint(x.w), 0x0073), 0x5410);
                    if (MODE == kModeFixed) tops &= syms + 0x7F7F7F7Fu;        // bit 7 of a byte: symbol != 0
                    f = syms | (tops & 0x80808080u);
                    if (MODE == kModeFixed) { f0 = f & 0xFFu; f1 = (f >> 8) & 0xFFu; f2 = (f >> 16) & 0xFFu; f3 = f >> 24; }
                } else {
                    f0 = q0 | (q0 ? (__float_as_uint(x.x) >> 16) & 0x8000u : 0u);
                    f1 = q1 | (q1 ? (__float_as_uint(x.y) >> 16) & 0x8000u : 0u);
                    f2 = q2 | (q2 ? (__float_as_uint(x.z) >> 16) & 0x8000u : 0u);
                    f3 = q3 | (q3 ? (__float_as_uint(x.w) >> 16) & 0x8000u : 0u);
                }
                if (MODE == kModeErc) {
                    // keep the nonzero symbols, in element order: rank = nonzeros in lower lanes + own earlier ones
                    const uint32_t v0 = __ballot_sync(0xffffffffu, q0 != 0), v1 = __ballot_sync(0xffffffffu, q1 != 0);
                    const uint32_t v2 = __ballot_sync(0xffffffffu, q2 != 0), v3 = __ballot_sync(0xffffffffu, q3 != 0);
                    uint32_t at = ntok + __popc(v0 & lt_mask) + __popc(v1 & lt_mask) + __popc(v2 & lt_mask) +
                                  __popc(v3 & lt_mask);
                    const uint32_t pos = r * 128u + lane * 4u;                  // position within the 512-element chunk
                    if (LEVELSET == kLevelsExp) {
                        // 16-bit entries position | field << 8, two at a time by byte permutation
                        const uint32_t pb = pos * 0x01010101u + 0x03020100u;    // the four positions, one per byte
                        const uint32_t e01 = __byte_perm(pb, f, 0x5140), e23 = __byte_perm(pb, f, 0x7362);
                        if (q0) tokens16[at++] = (uint16_t)e01;
                        if (q1) tokens16[at++] = (uint16_t)(e01 >> 16);
                        if (q2) tokens16[at++] = (uint16_t)e23;
                        if (q3) tokens16[at++] = (uint16_t)(e23 >> 16);
                    } else {
                        if (q0) tokens[at++] = pos | (f0 << 10);
                        if (q1) tokens[at++] = (pos + 1u) | (f1 << 10);
                        if (q2) tokens[at++] = (pos + 2u) | (f2 << 10);
                        if (q3) tokens[at++] = (pos + 3u) | (f3 << 10);
                    }
                    ntok = __shfl_sync(0xffffffffu, at, 31);                     // lane 31 ends behind the last entry
                } else if (q0 | q1 | q2 | q3) {
                    // fixed-width fields, MSB first, straight into the staged tile
                    const uint32_t wbits = G.width;
                    const uint32_t ff[4] = {f0, f1, f2, f3};
                    uint64_t str = 0;
#pragma unroll
                    for (int c = 0; c < 4; ++c) {
                        str = (str << wbits) | ((ff[c] & S::kMask) | ((ff[c] >> S::kBits) << (wbits - 1u)));
                        my_nnz += (ff[c] & S::kMask) != 0;
                    }
                    uint32_t cursor;
                    if (G.bucket <= kBLK) {
                        const uint32_t bi = bi_row;
                        cursor = 32u * (bi * G.rec_words + 1u) + (base - bi * blk_elems) * wbits;
                    } else {
                        cursor = base * wbits;
                    }
                    or_bits(stage, cursor, str, 4u * wbits);
                }
            }

            if (MODE == kModeErc) {
                __syncwarp();
                // ---- tokens ERC(gap) sign ERC(index), 32 per step, appended to the warp's window ----
                int carry_pos = -1;                         // position (within the chunk) of the last nonzero so far
                for (uint32_t t0 = 0; t0 < ntok; t0 += 32) {
                    const bool valid = t0 + lane < ntok;
                    uint32_t e = 0;
                    if (valid) e = LEVELSET == kLevelsExp ? (uint32_t)tokens16[t0 + lane] : tokens[t0 + lane];
                    const int pos = (int)(e & (LEVELSET == kLevelsExp ? 255u : 1023u));
                    const uint32_t field = e >> (LEVELSET == kLevelsExp ? 8 : 10);
                    int prev = __shfl_up_sync(0xffffffffu, pos, 1);
                    if (lane == 0) prev = carry_pos;
                    const bool first_of_sb = (prev >> 8) != (pos >> 8);      // also when there is no predecessor
                    if (first_of_sb) prev = (pos & ~255) - 1;                  // the run restarts: t_0 = 0
                    const uint32_t gl = s_lut[(pos - prev - 1) & 255];
                    uint32_t tlen, tokA, lenA, tokB = 0, lenB;
                    if (LEVELSET == kLevelsExp) {
                        const uint32_t ll = s_lut_signed[field & 255u];
                        lenB = ll >> 16;
                        tokA = ((gl & 0xffffu) << lenB) | (ll & 0xffffu);     // <= 16 + 8 bits
                        lenA = valid ? (gl >> 16) + lenB : 0u;
                        tlen = lenA;
                    } else {
                        const uint32_t ll = s_lut[((field & S::kMask) - 1u) & 255u];
                        tokA = gl & 0xffffu;
                        lenA = valid ? gl >> 16 : 0u;
                        lenB = valid ? (ll >> 16) + 1u : 0u;                  // sign + ERC(index) <= 17 bits
                        tokB = ((field >> S::kBits) << (ll >> 16)) | (ll & 0xffffu);
                        tlen = lenA + lenB;
                    }
                    uint32_t incl = tlen;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
                        if (lane >= (uint32_t)o) incl += t;
                    }
                    const uint32_t off = bits + incl - tlen;    // bit of the window where my token starts
                    // the first token of a sub-block marks where that sub-block's string starts
                    if (valid && first_of_sb) s_start[warp * 4u + part * (kChunk / kSB) + ((uint32_t)pos >> 8)] = off;
                    or_bits32(window, off, tokA, lenA);
                    if (LEVELSET != kLevelsExp) or_bits32(window, off + lenA, tokB, lenB);
                    bits += __shfl_sync(0xffffffffu, incl, 31);
                    carry_pos = __shfl_sync(0xffffffffu, pos, min(ntok - t0, 32u) - 1u);
                }
                my_nnz += ntok;                             // warp uniform: counted once below
                __syncwarp();
            }
        }
        if (MODE == kModeErc) {
            // sub-block strings follow one another: an empty one starts where the next one does
            uint32_t st = lane < 4 ? s_start[warp * 4u + lane] : 0xFFFFFFFFu;
            uint32_t s3 = __shfl_sync(0xffffffffu, st, 3), s2 = __shfl_sync(0xffffffffu, st, 2);
            uint32_t s1 = __shfl_sync(0xffffffffu, st, 1), s0 = __shfl_sync(0xffffffffu, st, 0);
            if (s3 == 0xFFFFFFFFu) s3 = bits;
            if (s2 == 0xFFFFFFFFu) s2 = s3;
            if (s1 == 0xFFFFFFFFu) s1 = s2;
            if (s0 == 0xFFFFFFFFu) s0 = s1;
            if (lane < 4) {
                const uint32_t begin = lane == 0 ? s0 : lane == 1 ? s1 : lane == 2 ? s2 : s3;
                const uint32_t end = lane == 0 ? s1 : lane == 1 ? s2 : lane == 2 ? s3 : bits;
                s_sb_src[warp * 4u + lane] = begin;
                s_sb_bits[warp * 4u + lane] = end - begin;
            }
            if (lane == 0 && my_nnz) atomicAdd(&s_nnz, my_nnz);
        } else {
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) my_nnz += __shfl_xor_sync(0xffffffffu, my_nnz, o);
            if (lane == 0 && my_nnz) atomicAdd(&s_nnz, my_nnz);
        }
        if (tid == 0) s_tile[(it + 1u) & 1u] = next_ticket;
        bar_sync<kBarWork, kEncThreads>();                    // B2: the tile's data is no longer read; lengths visible
        if (tid == 0) start_copy((it + 1u) & 1u);           // the next tile's bytes arrive while this one is packed

        // ---- layout of the tile's records ---------------------------------------------
        if (MODE == kModeErc) {
            uint32_t* stg = stage + sg * P.stage_words;                      // this tile's image; the others are pending
            // every warp runs the same scan over the 32 sub-block lengths
            const uint32_t sb = lane;
            const uint32_t v = sb < nsb_tile ? s_sb_bits[sb] : 0u;
            uint32_t incl = v;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
                if (lane >= (uint32_t)o) incl += t;
            }
            const uint32_t excl = incl - v;
            const uint32_t bi = bi_lane, sb0 = bi * spb;
            const uint32_t sb_last = min(sb0 + spb, nsb_tile) - 1u;         // meaningful when sb < nsb_tile
            const uint32_t excl0 = __shfl_sync(0xffffffffu, excl, sb0 & 31u);
            const uint32_t incl_last = __shfl_sync(0xffffffffu, incl, sb_last & 31u);
            const uint32_t nsb_blk = sb_last - sb0 + 1u;
            const uint32_t head_words = 1u + (nsb_blk + 1u) / 2u;
            const bool leader = sb < nsb_tile && sb == sb0;
            const uint32_t blk_words = leader ? head_words + (incl_last - excl0 + 31u) / 32u : 0u;
            uint32_t wincl = blk_words;
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const uint32_t t = __shfl_up_sync(0xffffffffu, wincl, o);
                if (lane >= (uint32_t)o) wincl += t;
            }
            const uint32_t wexcl = wincl - blk_words;
            const uint32_t blk_off = __shfl_sync(0xffffffffu, wexcl, sb0 & 31u);    // words before my block
            const uint32_t my_bitoff = 32u * (blk_off + head_words) + (excl - excl0);   // where sub-block `lane` goes
            const uint32_t tile_words = __shfl_sync(0xffffffffu, wincl, 31);
            const uint32_t code_bits = __shfl_sync(0xffffffffu, incl, 31);
            // announce the tile's size to its successors at once; the writer warp looks up its place
            if (tid == 0) announce_tile(tile_state, group_state, tile, tile_words);
            // this stage held the tile of P.stages iterations ago: the writer must be done with it
            if (it >= P.stages) stage_sync<kBarFree>(sg);
            // header words of the blocks: norm, then the u16 lengths two per word.  Lanes 4w .. 4w+3
            // of warp w stand for the warp's own sub-blocks, whose norms it holds.
            if ((lane >> 2) == warp && sb < nsb_tile) {
                const uint32_t q = lane & 3u;
                const float nq = q == 0 ? norm_q[0] : q == 1 ? norm_q[1] : q == 2 ? norm_q[2] : norm_q[3];
                if (leader) stg[blk_off] = __float_as_uint(nq);
                const uint32_t sbi = sb - sb0;
                atomicOr(stg + blk_off + 1u + sbi / 2u, v << (16u * (sbi & 1u)));
            }
            if (warp == 0) {
                Pending& pd = s_pend[sg];
                pd.blk_wordoff[lane] = __shfl_sync(0xffffffffu, wexcl, (lane * spb) & 31u);
                if (lane == 0) {
                    pd.tile = tile;
                    pd.words = tile_words;
                    pd.nblk = nblk_tile;
                    pd.code_bits = code_bits;
                    pd.nnz = s_nnz;
                    pd.valid = 1;
                    s_nnz = 0;
                }
            }

            // ---- every warp moves its sub-block strings to their place in the staged tile ----
            __syncwarp();
#pragma unroll 1
            for (uint32_t q = 0; q < 4; q += coarse ? 4u : 1u) {
                // the strings of sub-blocks of one block follow one another in the window and in the
                // tile alike, so a warp whose four sub-blocks share a block moves them in one piece
                const uint32_t sbq = warp * 4u + q;
                if (sbq >= nsb_tile) break;
                const uint32_t len = coarse ? bits : s_sb_bits[sbq], src = coarse ? 0u : s_sb_src[sbq];
                const uint32_t dst = __shfl_sync(0xffffffffu, my_bitoff, sbq);
                if (len == 0) continue;
                const uint32_t w_first = dst >> 5, w_last = (dst + len - 1u) >> 5;
                for (uint32_t w = w_first + lane; w <= w_last; w += 32) {
                    const int sbit = (int)src + (int)(32u * w) - (int)dst;
                    uint32_t val = bits_at(window, sbit);
                    const uint32_t head = 32u * w < dst ? dst - 32u * w : 0u;     // bits of this word before the string
                    const uint32_t tail_end = min(dst + len - 32u * w, 32u);      // bits of this word up to its end
                    uint32_t mask = 0xFFFFFFFFu >> head;
                    if (tail_end < 32u) mask &= ~(0xFFFFFFFFu >> tail_end);
                    val &= mask;
                    if (val) atomicOr(stg + w, val);
                }
            }
            __syncwarp();
            for (uint32_t i = lane; i < (bits + 31u) / 32u + 2u; i += 32) window[i] = 0;   // ready for the next tile
            stage_arrive<kBarStaged>(sg);                  // the writer may take the tile
        } else {
            uint64_t tile_off;
            uint32_t tile_words;
            if (G.bucket <= kBLK) {
                tile_off = first_block * G.rec_words;
                tile_words = (nblk_tile - 1u) * G.rec_words + 1u +
                             ((tile_len - (nblk_tile - 1u) * G.bucket) * G.width + 31u) / 32u;
                // norm words: lanes 4w .. 4w+3 of warp w stand for the warp's own sub-blocks
                if ((lane >> 2) == warp && lane < nsb_tile && lane == bi_lane * spb) {
                    const uint32_t q = lane & 3u;
                    const float nq = q == 0 ? norm_q[0] : q == 1 ? norm_q[1] : q == 2 ? norm_q[2] : norm_q[3];
                    stage[bi_lane * G.rec_words] = __float_as_uint(nq);
                }
            } else {
                tile_off = bucket_idx * G.rec_words + 1u + (uint64_t)bib * (kBLK * G.width / 32u);
                tile_words = (tile_len * G.width + 31u) / 32u;
                if (bib == 0 && tid == 0) payload[bucket_idx * G.rec_words] = __float_as_uint(norm_q[0]);
            }
            bar_sync<kBarWork, kEncThreads>();                // the staged fields are complete
            for (uint32_t i = tid; i < tile_words; i += kEncThreads) {
                payload[tile_off + i] = stage[i];
                stage[i] = 0;
            }
            if (tid == 0) {
                s_tot.nnz += s_nnz;
                s_tot.tiles += 1;
                s_nnz = 0;
            }
        }
    }

    if (MODE == kModeErc && !writer) {
        // ---- the workers ran `it` iterations (the next one would use stage sg): wait until the writer
        // has written the last tiles, telling it in between that no further one comes ----
        if (it >= P.stages) stage_sync<kBarFree>(sg);       // tile it - stages: its barriers are used again below
        if (tid == 0) s_tot.stop = it;
        stage_arrive<kBarStaged>(sg);
        for (uint32_t back = P.stages - 1u; back >= 1u; --back) {   // tiles it - stages + 1 .. it - 1
            if (it >= back) {
                const uint32_t bb = (sg + P.stages - back) % P.stages;
                stage_sync<kBarFree>(bb);
            }
        }
    }
    __syncthreads();                                        // every write of this CTA lies behind this barrier
    if (tid == 0) finish_cta<MODE>(P, s_tot.tiles, s_tot.nnz, s_tot.code_bits);
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

// shared memory of one CTA: the tile, its staged image, and per warp a bit window and a token list
size_t encode_smem_bytes(const EncodeParams& P) {
    return 4u * ((size_t)kBLK + (size_t)P.stages * P.stage_words + (size_t)kEncWarps * P.warp_smem_words);
}

constexpr int kEncMaxDynSmem = 112 * 1024;

template <uint32_t L, uint32_t M>
static cudaError_t prepare_kernel() {
    static bool attr_set = false;
    if (attr_set) return cudaSuccess;
    cudaError_t e = cudaFuncSetAttribute(encode_kernel<L, M>, cudaFuncAttributeMaxDynamicSharedMemorySize, kEncMaxDynSmem);
    if (e == cudaSuccess) attr_set = true;
    return e;
}

template <uint32_t L, uint32_t M>
static int blocks_per_sm(const EncodeParams& P) {
    if (prepare_kernel<L, M>() != cudaSuccess) return 0;
    int n = 0;
    const int threads = M == kModeErc ? (int)kEncAllThreads : kEncThreads;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, encode_kernel<L, M>, threads, encode_smem_bytes(P)) != cudaSuccess)
        return 0;
    return n < kEncMinBlocks ? n : kEncMinBlocks;
}

int encode_blocks_per_sm(const EncodeParams& P) {
    const bool uni = P.geo.levelset == kLevelsUniform, fixed = P.geo.mode == kModeFixed;
    if (encode_smem_bytes(P) > (size_t)kEncMaxDynSmem) return 0;
    if (!uni && !fixed) return blocks_per_sm<kLevelsExp, kModeErc>(P);
    if (!uni && fixed) return blocks_per_sm<kLevelsExp, kModeFixed>(P);
    if (uni && !fixed) return blocks_per_sm<kLevelsUniform, kModeErc>(P);
    return blocks_per_sm<kLevelsUniform, kModeFixed>(P);
}

template <uint32_t L, uint32_t M>
static cudaError_t launch_one(const EncodeParams& P, cudaStream_t stream) {
    const size_t smem = encode_smem_bytes(P);
    cudaError_t e = prepare_kernel<L, M>();
    if (e != cudaSuccess) return e;
    if (smem > (size_t)kEncMaxDynSmem || P.grid == 0) return cudaErrorInvalidValue;
    encode_kernel<L, M><<<P.grid, M == kModeErc ? kEncAllThreads : (uint32_t)kEncThreads, smem, stream>>>(P);
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
