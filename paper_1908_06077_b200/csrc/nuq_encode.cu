// ENCODE of NUQSGD (App. A) for one gradient vector: bucket norm, stochastic
// quantization (Definition 1) and Elias-recursive token packing in ONE pass over
// the input.  A CTA owns a tile of up to 8192 consecutive elements (32 coding
// sub-blocks of 256); every lane keeps its 4 x 8 consecutive elements in
// registers between the norm reduction and the quantizer, so the gradient is
// read from HBM exactly once.  Tiles are chained by a decoupled look-back scan
// over their payload sizes, which gives each tile its place in the packed
// stream without a second kernel.
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
__device__ __forceinline__ uint4 philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0,
                                               uint32_t k1) {
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        c1 = (uint32_t)p1;
        c3 = (uint32_t)p0;
        c0 = n0;
        c2 = n2;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    return make_uint4(c0, c1, c2, c3);
}

// ---------------------------------------------------------------------------
// Definition 1 for one coordinate.  y = |v| * (2^s / norm), clamped to 2^s.
// The draw is u = m * 2^-24 with m the top 24 bits of `word`; the coordinate moves
// to the upper level iff u < p.  Both sides of that comparison are scaled by 2^24
// (exact), and for y >= 1 the 23 mantissa bits of y ARE p * 2^23, so the test
// becomes an integer comparison.
// ---------------------------------------------------------------------------
template <uint32_t LEVELSET>
__device__ __forceinline__ uint32_t quantize_one(float v, float inv, float top, uint32_t s, uint32_t word) {
    float y = fminf(__fmul_rn(fabsf(v), inv), top);
    uint32_t m24 = word >> 8;
    if (LEVELSET == kLevelsExp) {
        if (y < 1.0f) {                                    // r in [0, 2^-s]:  p_1 = 2^s r
            return (__uint2float_rn(m24) < y * 16777216.0f) ? 1u : 0u;
        }
        uint32_t yb = __float_as_uint(y);
        uint32_t e = (yb >> 23) - 127u;                    // r in [2^(e-s), 2^(e+1-s)]:  p_2 = 2^(s-e) r - 1
        if (e >= s) return s + 1u;                         // y == 2^s: p = 1
        return e + 1u + (((m24 >> 1) < (yb & 0x7FFFFFu)) ? 1u : 0u);
    } else {                                               // levels k / 2^s:  p = y - floor(y)
        float fl = fminf(floorf(y), top - 1.0f);
        float p = y - fl;
        return (uint32_t)fl + ((__uint2float_rn(m24) < p * 16777216.0f) ? 1u : 0u);
    }
}

// OR `nbits` (<= 33) right-aligned bits of `value` into the MSB-first bit string `stage` at `bitpos`.
__device__ __forceinline__ void stage_or(uint32_t* stage, uint32_t bitpos, uint64_t value, uint32_t nbits) {
    uint32_t w = bitpos >> 5, sh = bitpos & 31u;
    uint64_t placed = (value << (64u - nbits)) >> sh;      // nbits + sh <= 64
    uint32_t hi = (uint32_t)(placed >> 32), lo = (uint32_t)placed;
    atomicOr(stage + w, hi);
    if (lo) atomicOr(stage + w + 1, lo);
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
            if (++polls > (1u << 18)) {                    // ~tens of ms: give up, never hang
                if (lane == 0) {
                    latch_status(ws, kErrTimeout);
                    st_volatile_u64(state + tile, kTilePoison);
                }
                *failed = true;
                return 0;
            }
            __nanosleep(64);
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

// symbols of the 8 consecutive elements one lane owns in one sub-block
struct LaneSyms {
    uint32_t masks;   // bits 0-7 nonzero mask, bits 8-15 sign mask
    uint32_t lo, hi;  // (sym-1) of elements 0-3 / 4-7, one byte each
};

__device__ __forceinline__ uint32_t sym_of(const LaneSyms& q, uint32_t e) {
    return (((e < 4 ? q.lo : q.hi) >> (8u * (e & 3u))) & 0xffu) + 1u;
}

template <uint32_t LEVELSET, uint32_t MODE>
__global__ void __launch_bounds__(kEncThreads, 2) encode_kernel(const __grid_constant__ EncodeParams P) {
    extern __shared__ __align__(16) uint32_t stage[];      // staged payload of the tile
    __shared__ uint32_t s_lut[256];
    __shared__ double s_sb_partial[32];
    __shared__ uint32_t s_sb_maxbits[32];
    __shared__ float s_blk_norm[32];
    __shared__ float s_blk_inv[32];                        // 2^s / norm, or 0 for a bucket that is not quantized
    __shared__ uint32_t s_sb_bits[32];
    __shared__ uint32_t s_sb_bitoff[32];
    __shared__ uint32_t s_blk_wordoff[33];
    __shared__ unsigned long long s_tile, s_tile_off;
    __shared__ uint32_t s_tile_words, s_abort, s_nnz;

    const Geometry& G = P.geo;
    const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    uint64_t* tile_state = reinterpret_cast<uint64_t*>(P.ws + 1);
    uint64_t* table = reinterpret_cast<uint64_t*>(P.out + kHeaderWords);
    uint32_t* payload = MODE == kModeErc ? P.out + kHeaderWords + 2 * (G.nblk + 1) : P.out + kHeaderWords;
    const float top = __uint_as_float((127u + G.s) << 23);
    const uint32_t k0 = (uint32_t)P.seed, k1 = (uint32_t)(P.seed >> 32);
    const uint32_t c2 = (uint32_t)P.offset, c3 = (uint32_t)(P.offset >> 32);

    s_lut[tid] = c_erc_lut[tid];
    for (uint32_t i = tid; i < P.stage_words; i += kEncThreads) stage[i] = 0;

    for (;;) {
        __syncthreads();
        if (tid == 0) {
            s_tile = atomicAdd(reinterpret_cast<unsigned long long*>(&P.ws->ticket), 1ull);
            s_abort = 0;
            s_nnz = 0;
        }
        __syncthreads();
        const uint64_t tile = s_tile;
        if (tile >= G.ntiles) break;

        // ---- tile geometry ------------------------------------------------------
        uint64_t elem0, first_block;
        uint32_t tile_len, nblk_tile, spb, blk_elems;
        uint64_t bucket_idx = 0;
        uint32_t bib = 0;                                   // block within a wide bucket
        if (G.bucket <= kBLK) {
            first_block = tile * G.blocks_per_tile;
            elem0 = first_block * G.bucket;
            uint64_t left = G.d - elem0;
            tile_len = left < G.tile_elems ? (uint32_t)left : G.tile_elems;
            blk_elems = G.bucket;
            nblk_tile = (tile_len + G.bucket - 1) / G.bucket;
            spb = G.sb_per_block;
        } else {
            bucket_idx = tile / G.blk_per_bucket;
            bib = (uint32_t)(tile % G.blk_per_bucket);
            first_block = tile;
            uint64_t b0 = bucket_idx * G.bucket;
            uint64_t blen = G.d - b0 < G.bucket ? G.d - b0 : G.bucket;
            elem0 = b0 + (uint64_t)bib * kBLK;
            uint64_t left = blen - (uint64_t)bib * kBLK;
            tile_len = left < kBLK ? (uint32_t)left : kBLK;
            blk_elems = kBLK;
            nblk_tile = 1;
            spb = 32;
        }
        const uint32_t nsb_tile = (tile_len + kSB - 1) / kSB;

        // ---- load: 4 sub-blocks per warp, 8 consecutive elements per lane --------
        float x[kSbPerWarp][8];
#pragma unroll
        for (int j = 0; j < kSbPerWarp; ++j) {
            uint32_t base = (warp * kSbPerWarp + j) * kSB + lane * 8u;
            if (base + 8u <= tile_len) {
                const float4* src = reinterpret_cast<const float4*>(P.g + elem0 + base);
                float4 a = __ldg(src), b = __ldg(src + 1);
                x[j][0] = a.x; x[j][1] = a.y; x[j][2] = a.z; x[j][3] = a.w;
                x[j][4] = b.x; x[j][5] = b.y; x[j][6] = b.z; x[j][7] = b.w;
            } else {
#pragma unroll
                for (int e = 0; e < 8; ++e) x[j][e] = base + e < tile_len ? __ldg(P.g + elem0 + base + e) : 0.0f;
            }
        }

        // ---- bucket norms ----------------------------------------------------------
        if (P.norms_in == nullptr) {
#pragma unroll
            for (int j = 0; j < kSbPerWarp; ++j) {
                if (G.norm_kind == kNormL2) {
                    double acc = 0.0;
#pragma unroll
                    for (int e = 0; e < 8; ++e) acc = fma((double)x[j][e], (double)x[j][e], acc);
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
                    if (lane == 0) s_sb_partial[warp * kSbPerWarp + j] = acc;
                } else {                                    // max |x| on the bit patterns: NaN sorts above inf
                    uint32_t m = 0;
#pragma unroll
                    for (int e = 0; e < 8; ++e) m = max(m, __float_as_uint(fabsf(x[j][e])));
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) m = max(m, __shfl_xor_sync(0xffffffffu, m, o));
                    if (lane == 0) s_sb_maxbits[warp * kSbPerWarp + j] = m;
                }
            }
            __syncthreads();
        }
        if (tid < nblk_tile) {
            float norm;
            if (P.norms_in != nullptr) {
                norm = P.norms_in[G.bucket <= kBLK ? first_block + tid : bucket_idx];
            } else if (G.norm_kind == kNormL2) {
                double acc = 0.0;
                uint32_t sb0 = tid * spb, sb1 = min(sb0 + spb, nsb_tile);
                for (uint32_t sb = sb0; sb < sb1; ++sb) acc += s_sb_partial[sb];
                norm = (float)sqrt(acc);
            } else {
                uint32_t m = 0;
                uint32_t sb0 = tid * spb, sb1 = min(sb0 + spb, nsb_tile);
                for (uint32_t sb = sb0; sb < sb1; ++sb) m = max(m, s_sb_maxbits[sb]);
                norm = __uint_as_float(m);
            }
            if (norm != norm) norm = __uint_as_float(0x7fc00000u);     // one NaN pattern in the stream
            float inv = 0.0f;
            if (norm > 0.0f && norm < __uint_as_float(0x7f800000u)) {
                inv = __fdiv_rn(top, norm);                 // one IEEE division per bucket
                if (!(inv < __uint_as_float(0x7f800000u))) inv = 0.0f;
            }
            s_blk_norm[tid] = norm;
            s_blk_inv[tid] = inv;
        }
        __syncthreads();

        // ---- quantize (Definition 1) ------------------------------------------------
        LaneSyms q[kSbPerWarp];
        uint32_t lane_off[kSbPerWarp];
        uint32_t my_nnz = 0;
#pragma unroll
        for (int j = 0; j < kSbPerWarp; ++j) {
            const uint32_t sb = warp * kSbPerWarp + j;
            q[j].masks = 0; q[j].lo = 0; q[j].hi = 0;
            lane_off[j] = 0;
            if (sb >= nsb_tile) continue;
            const float inv = s_blk_inv[sb / spb];
            if (inv != 0.0f) {
                uint64_t ctr = (elem0 + (uint64_t)sb * kSB + lane * 8u) >> 2;
                uint4 r0 = philox4x32_10((uint32_t)ctr, (uint32_t)(ctr >> 32), c2, c3, k0, k1);
                ++ctr;
                uint4 r1 = philox4x32_10((uint32_t)ctr, (uint32_t)(ctr >> 32), c2, c3, k0, k1);
                const uint32_t rw[8] = {r0.x, r0.y, r0.z, r0.w, r1.x, r1.y, r1.z, r1.w};
#pragma unroll
                for (int e = 0; e < 8; ++e) {
                    uint32_t sym = quantize_one<LEVELSET>(x[j][e], inv, top, G.s, rw[e]);
                    if (sym) {
                        uint32_t neg = __float_as_uint(x[j][e]) >> 31;
                        q[j].masks |= (1u << e) | (neg << (8 + e));
                        if (e < 4) q[j].lo |= (sym - 1u) << (8 * e);
                        else q[j].hi |= (sym - 1u) << (8 * (e - 4));
                    }
                }
            }
            my_nnz += __popc(q[j].masks & 0xffu);

            if (MODE == kModeErc) {
                // token lengths: gap to the previous nonzero of the sub-block (1-based positions)
                uint32_t nz = q[j].masks & 0xffu;
                uint32_t last_pos = nz ? lane * 8u + (31u - __clz(nz)) + 1u : 0u;
                uint32_t any = __ballot_sync(0xffffffffu, nz != 0);
                uint32_t lower = any & ((1u << lane) - 1u);
                uint32_t prev = __shfl_sync(0xffffffffu, last_pos, lower ? 31 - __clz(lower) : 0);
                if (!lower) prev = 0;
                uint32_t bits = 0;
                while (nz) {
                    uint32_t e = __ffs(nz) - 1u;
                    nz &= nz - 1u;
                    uint32_t pos = lane * 8u + e + 1u;
                    bits += (s_lut[pos - prev - 1u] >> 16) + 1u + (s_lut[sym_of(q[j], e) - 1u] >> 16);
                    prev = pos;
                }
                uint32_t incl = bits;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
                    if (lane >= (uint32_t)o) incl += t;
                }
                lane_off[j] = incl - bits;
                if (lane == 31) s_sb_bits[sb] = incl;
            }
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) my_nnz += __shfl_xor_sync(0xffffffffu, my_nnz, o);
        if (lane == 0 && my_nnz) atomicAdd(&s_nnz, my_nnz);
        __syncthreads();

        // ---- layout of the tile's records -------------------------------------------
        uint64_t tile_off = 0;
        uint32_t tile_words = 0;
        if (MODE == kModeErc) {
            if (warp == 0) {
                const uint32_t sb = lane;
                uint32_t v = sb < nsb_tile ? s_sb_bits[sb] : 0u;
                uint32_t incl = v;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
                    if (lane >= (uint32_t)o) incl += t;
                }
                const uint32_t excl = incl - v;
                const uint32_t bi = sb / spb, sb0 = bi * spb;
                const uint32_t sb_last = min(sb0 + spb, nsb_tile) - 1u;     // meaningful when sb < nsb_tile
                const uint32_t excl0 = __shfl_sync(0xffffffffu, excl, sb0 & 31u);
                const uint32_t incl_last = __shfl_sync(0xffffffffu, incl, sb_last & 31u);
                const uint32_t nsb_blk = sb_last - sb0 + 1u;
                const uint32_t head_words = 1u + (nsb_blk + 1u) / 2u;
                const bool leader = sb < nsb_tile && sb == sb0;
                uint32_t blk_words = leader ? head_words + (incl_last - excl0 + 31u) / 32u : 0u;
                uint32_t wincl = blk_words;
#pragma unroll
                for (int o = 1; o < 32; o <<= 1) {
                    uint32_t t = __shfl_up_sync(0xffffffffu, wincl, o);
                    if (lane >= (uint32_t)o) wincl += t;
                }
                const uint32_t wexcl = wincl - blk_words;
                if (leader) s_blk_wordoff[bi] = wexcl;
                const uint32_t blk_off = __shfl_sync(0xffffffffu, wexcl, sb0 & 31u);
                if (sb < nsb_tile) s_sb_bitoff[sb] = 32u * (blk_off + head_words) + (excl - excl0);
                tile_words = __shfl_sync(0xffffffffu, wincl, 31);
                uint32_t code_bits = __shfl_sync(0xffffffffu, incl, 31);
                if (lane == 0) {
                    s_tile_words = tile_words;
                    s_blk_wordoff[nblk_tile] = tile_words;
                    atomicAdd(reinterpret_cast<unsigned long long*>(&P.ws->code_bits), (unsigned long long)code_bits);
                }
            }
            __syncthreads();
            tile_words = s_tile_words;
            if (warp == 0) {                                // chain the tiles while the others emit tokens
                bool failed;
                uint64_t off = tile_lookback(P.ws, tile_state, tile, tile_words, &failed);
                if (lane == 0) {
                    s_tile_off = off;
                    if (failed) s_abort = 1;
                }
            }
        } else {
            if (G.bucket <= kBLK) {
                tile_off = first_block * G.rec_words;
                tile_words = (nblk_tile - 1u) * G.rec_words + 1u +
                             ((tile_len - (nblk_tile - 1u) * G.bucket) * G.width + 31u) / 32u;
            } else {
                tile_off = bucket_idx * G.rec_words + 1u + (uint64_t)bib * (kBLK * G.width / 32u);
                tile_words = (tile_len * G.width + 31u) / 32u;
            }
        }

        // ---- emit into the staging buffer -------------------------------------------
        if (MODE == kModeErc) {
            if (tid < nblk_tile) stage[s_blk_wordoff[tid]] = __float_as_uint(s_blk_norm[tid]);
            if (tid < nsb_tile) {
                uint32_t bi = tid / spb, sbi = tid - bi * spb;
                atomicOr(stage + s_blk_wordoff[bi] + 1u + sbi / 2u, s_sb_bits[tid] << (16u * (sbi & 1u)));
            }
#pragma unroll
            for (int j = 0; j < kSbPerWarp; ++j) {
                const uint32_t sb = warp * kSbPerWarp + j;
                uint32_t nz = q[j].masks & 0xffu;
                // the previous nonzero position is needed again; recompute it (cheap)
                uint32_t last_pos = nz ? lane * 8u + (31u - __clz(nz)) + 1u : 0u;
                uint32_t any = __ballot_sync(0xffffffffu, nz != 0);
                uint32_t lower = any & ((1u << lane) - 1u);
                uint32_t prev = __shfl_sync(0xffffffffu, last_pos, lower ? 31 - __clz(lower) : 0);
                if (!lower) prev = 0;
                if (sb >= nsb_tile) continue;
                uint32_t cursor = s_sb_bitoff[sb] + lane_off[j];
                while (nz) {
                    uint32_t e = __ffs(nz) - 1u;
                    nz &= nz - 1u;
                    uint32_t pos = lane * 8u + e + 1u;
                    uint32_t gl = s_lut[pos - prev - 1u], ll = s_lut[sym_of(q[j], e) - 1u];
                    uint32_t glen = gl >> 16, llen = ll >> 16;
                    uint64_t sign = (q[j].masks >> (8u + e)) & 1u;
                    uint64_t token = ((uint64_t)(gl & 0xffffu) << (1u + llen)) | (sign << llen) | (ll & 0xffffu);
                    uint32_t tlen = glen + 1u + llen;
                    stage_or(stage, cursor, token, tlen);
                    cursor += tlen;
                    prev = pos;
                }
            }
        } else {
            if (G.bucket <= kBLK) {
                if (tid < nblk_tile) stage[tid * G.rec_words] = __float_as_uint(s_blk_norm[tid]);
            } else if (bib == 0 && tid == 0) {
                payload[bucket_idx * G.rec_words] = __float_as_uint(s_blk_norm[0]);
            }
            const uint32_t wbits = G.width;
#pragma unroll
            for (int j = 0; j < kSbPerWarp; ++j) {
                const uint32_t sb = warp * kSbPerWarp + j;
                const uint32_t base = sb * kSB + lane * 8u;
                if (base >= tile_len) continue;
                uint32_t bi = G.bucket <= kBLK ? sb / spb : 0u;
                uint32_t in_blk = base - bi * blk_elems;
                uint32_t cursor = G.bucket <= kBLK ? 32u * (bi * G.rec_words + 1u) + in_blk * wbits : base * wbits;
#pragma unroll
                for (uint32_t e = 0; e < 8; ++e) {
                    if (base + e >= tile_len) break;
                    uint32_t field = 0;
                    if ((q[j].masks >> e) & 1u) field = (((q[j].masks >> (8u + e)) & 1u) << (wbits - 1u)) | sym_of(q[j], e);
                    if (field) stage_or(stage, cursor, field, wbits);
                    cursor += wbits;
                }
            }
        }
        __syncthreads();

        // ---- copy the tile out -------------------------------------------------------
        if (MODE == kModeErc) tile_off = s_tile_off;
        const bool aborted = s_abort != 0;
        for (uint32_t i = tid; i < tile_words; i += kEncThreads) {
            if (!aborted) payload[tile_off + i] = stage[i];
            stage[i] = 0;
        }
        if (MODE == kModeErc && !aborted) {
            if (tid < nblk_tile) table[first_block + tid] = 32ull * (tile_off + s_blk_wordoff[tid]);
            if (tile == G.ntiles - 1 && tid == 0) {
                table[G.nblk] = 32ull * (tile_off + tile_words);
                P.ws->total_words = tile_off + tile_words;
            }
        }
        __syncthreads();

        // ---- last tile to finish writes the header ------------------------------------
        if (tid == 0) {
            if (s_nnz) atomicAdd(reinterpret_cast<unsigned long long*>(&P.ws->nnz), (unsigned long long)s_nnz);
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

template <uint32_t L, uint32_t M>
static cudaError_t launch_one(const EncodeParams& P, int sms, cudaStream_t stream) {
    size_t smem = (size_t)P.stage_words * 4;
    static bool attr_set = false;
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(encode_kernel<L, M>, cudaFuncAttributeMaxDynamicSharedMemorySize, 64 * 1024);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    uint64_t grid = P.geo.ntiles < (uint64_t)(2 * sms) ? P.geo.ntiles : (uint64_t)(2 * sms);
    encode_kernel<L, M><<<(unsigned)grid, kEncThreads, smem, stream>>>(P);
    return cudaGetLastError();
}

cudaError_t launch_encode(const EncodeParams& P, int sms, cudaStream_t stream) {
    const bool uni = P.geo.levelset == kLevelsUniform, fixed = P.geo.mode == kModeFixed;
    if (!uni && !fixed) return launch_one<kLevelsExp, kModeErc>(P, sms, stream);
    if (!uni && fixed) return launch_one<kLevelsExp, kModeFixed>(P, sms, stream);
    if (uni && !fixed) return launch_one<kLevelsUniform, kModeErc>(P, sms, stream);
    return launch_one<kLevelsUniform, kModeFixed>(P, sms, stream);
}

}  // namespace nuq
