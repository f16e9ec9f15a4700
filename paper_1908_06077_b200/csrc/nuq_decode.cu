// DECODE + aggregate (App. A decoding; Algorithm 1, aggregation line): the K
// workers' containers are decoded and summed into one fp32 vector.  A warp owns
// a tile of up to 8192 output elements held in shared memory; lane l walks the
// token chain of sub-block l of the tile, stream after stream in ascending k, so
// every output element receives its terms in the order k = 0, 1, ... and the
// result is bit-reproducible.  The tile is written to HBM once.
#include "nuq_common.cuh"
#include "nuq_launch.h"

namespace nuq {

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

// 64 bits of the MSB-first bit string `words` starting at bit `cur`; word indices are clamped to `last`.
__device__ __forceinline__ uint64_t window64(const uint32_t* __restrict__ words, uint32_t cur, uint32_t last) {
    uint32_t wi = cur >> 5, sh = cur & 31u;
    uint32_t w0 = __ldg(words + min(wi, last));
    uint32_t w1 = __ldg(words + min(wi + 1u, last));
    uint32_t w2 = __ldg(words + min(wi + 2u, last));
    uint64_t win = ((uint64_t)w0 << 32 | w1) << sh;
    if (sh) win |= (uint64_t)w2 >> (32u - sh);
    return win;
}

__device__ __forceinline__ float level_times_norm(float norm, uint32_t levelset, uint32_t s, uint32_t sym) {
    // exponential: l_j = 2^(j-1-s) (exact scaling);  uniform: l_k = k / 2^s
    float level = levelset == kLevelsExp ? __uint_as_float((126u + sym - s) << 23)
                                         : (float)sym * __uint_as_float((127u - s) << 23);
    return __fmul_rn(norm, level);
}

__global__ void __launch_bounds__(32) decode_kernel(const __grid_constant__ DecodeParams P) {
    extern __shared__ __align__(16) float tile_acc[];       // kBLK floats
    const Geometry& G = P.geo;
    const uint32_t lane = threadIdx.x;

    for (uint64_t tile = blockIdx.x; tile < G.ntiles; tile += gridDim.x) {
        // ---- tile geometry (same tiling as the encoder) ---------------------------
        uint64_t elem0, first_block, bucket_idx = 0;
        uint32_t tile_len, spb, blk_elems, bib = 0;
        if (G.bucket <= kBLK) {
            first_block = tile * G.blocks_per_tile;
            elem0 = first_block * G.bucket;
            uint64_t left = G.d - elem0;
            tile_len = left < G.tile_elems ? (uint32_t)left : G.tile_elems;
            spb = G.sb_per_block;
            blk_elems = G.bucket;
        } else {
            bucket_idx = tile / G.blk_per_bucket;
            bib = (uint32_t)(tile % G.blk_per_bucket);
            first_block = tile;
            uint64_t b0 = bucket_idx * G.bucket;
            uint64_t blen = G.d - b0 < G.bucket ? G.d - b0 : G.bucket;
            elem0 = b0 + (uint64_t)bib * kBLK;
            uint64_t left = blen - (uint64_t)bib * kBLK;
            tile_len = left < kBLK ? (uint32_t)left : kBLK;
            spb = 32;
            blk_elems = kBLK;
        }
        const uint32_t nsb_tile = (tile_len + kSB - 1) / kSB;
        const uint32_t sb = lane;
        const uint32_t bi = sb / spb, sb0 = bi * spb, sbi = sb - sb0;
        const uint32_t blk_len = min(blk_elems, tile_len - min(tile_len, bi * blk_elems));   // elements of my block
        const uint32_t nsb_blk = (blk_len + kSB - 1) / kSB;
        const uint32_t sn = sb < nsb_tile ? min(kSB, tile_len - sb * kSB) : 0u;              // elements of my sub-block
        float* mine = tile_acc + sb * kSB;

        for (uint32_t i = lane * 4u; i < kBLK; i += 128u)
            *reinterpret_cast<float4*>(tile_acc + i) = make_float4(0.f, 0.f, 0.f, 0.f);
        __syncwarp();

        for (uint32_t k = 0; k < P.K; ++k) {
            const uint32_t* hdr = P.streams[k];
            // ---- header validation against the call's arguments ---------------------
            const uint32_t flags = __ldg(hdr + 6);
            const uint32_t levelset = (flags >> 8) & 0xffu, mode = (flags >> 16) & 0xffu;
            const uint64_t hd = (uint64_t)__ldg(hdr + 2) | ((uint64_t)__ldg(hdr + 3) << 32);
            const uint64_t hnblk = (uint64_t)__ldg(hdr + 8) | ((uint64_t)__ldg(hdr + 9) << 32);
            const uint64_t cbits = (uint64_t)__ldg(hdr + 10) | ((uint64_t)__ldg(hdr + 11) << 32);
            bool ok = __ldg(hdr) == kMagic && __ldg(hdr + 1) == kVersion && hd == G.d && __ldg(hdr + 4) == G.bucket &&
                      __ldg(hdr + 5) == G.s && __ldg(hdr + 7) == kSB && levelset <= 1u && mode <= 1u &&
                      (flags & 0xffu) <= 1u && !(levelset == kLevelsUniform && G.s > 8u) && (cbits & 31u) == 0;
            const uint32_t nlev = levelset == kLevelsExp ? G.s + 2u : (1u << G.s) + 1u;
            const uint64_t cwords = cbits >> 5;

            if (ok && mode == kModeErc) {
                const uint64_t head = kHeaderWords + 2 * (G.nblk + 1);
                ok = hnblk == G.nblk && cwords > head;
                bool lane_ok = true;
                uint32_t cur = 0, endb = 0, last = 0;
                const uint32_t* tok = hdr;
                float norm = 0.0f;
                if (ok) {
                    const uint64_t* table = reinterpret_cast<const uint64_t*>(hdr + kHeaderWords);
                    const uint32_t* payload = hdr + head;
                    const uint64_t payload_words = cwords - head;
                    uint32_t len = 0, head_words = 0, rec_words = 0;
                    if (sb < nsb_tile) {
                        uint64_t off = __ldg(table + first_block + bi), end = __ldg(table + first_block + bi + 1);
                        head_words = 1u + (nsb_blk + 1u) / 2u;
                        lane_ok = (off & 31u) == 0 && (end & 31u) == 0 && off < end && (end >> 5) <= payload_words &&
                                  ((end - off) >> 5) >= head_words && ((end - off) >> 5) <= (1u << 20);
                        if (lane_ok) {
                            const uint32_t* rec = payload + (off >> 5);
                            rec_words = (uint32_t)((end - off) >> 5);
                            norm = __uint_as_float(__ldg(rec));
                            len = (__ldg(rec + 1u + sbi / 2u) >> (16u * (sbi & 1u))) & 0xffffu;
                            tok = rec + head_words;
                        }
                    }
                    // start of my chain = sum of the lengths of the earlier sub-blocks of my block
                    uint32_t incl = len;
#pragma unroll
                    for (int o = 1; o < 32; o <<= 1) {
                        uint32_t t = __shfl_up_sync(0xffffffffu, incl, o);
                        if (lane >= (uint32_t)o) incl += t;
                    }
                    const uint32_t excl0 = __shfl_sync(0xffffffffu, incl - len, sb0 & 31u);
                    cur = incl - len - excl0;
                    endb = cur + len;
                    if (sb < nsb_tile && lane_ok) {
                        uint32_t tok_words = rec_words - head_words;
                        lane_ok = endb <= 32u * tok_words;
                        last = tok_words ? tok_words - 1u : 0u;
                    }
                }
                if (!__all_sync(0xffffffffu, ok && lane_ok)) ok = false;
                if (ok && sb < nsb_tile) {
                    // ---- the token walk: ERC^-1 gap, sign bit, ERC^-1 level index ----------
                    uint32_t pos = 0;
                    while (cur < endb) {
                        uint64_t win = window64(tok, cur, last);
                        uint32_t used = 0, gap, sym;
                        bool good = erc_read(win, used, gap);
                        uint32_t negative = (uint32_t)(win >> 63);
                        win <<= 1;
                        used += 1;
                        good = good && erc_read(win, used, sym);
                        pos += gap;
                        if (!good || used > endb - cur || pos > sn || sym == 0 || sym >= nlev) {
                            ok = false;
                            break;
                        }
                        float v = level_times_norm(norm, levelset, G.s, sym);
                        mine[pos - 1u] += negative ? -v : v;
                        cur += used;
                    }
                }
            } else if (ok) {
                // ---- fixed-width fields ------------------------------------------------------
                const uint32_t w = 1u + (32u - __clz(nlev - 1u));           // sign bit + ceil(log2(levels))
                const uint32_t rec_words = 1u + (G.bucket * w + 31u) / 32u;
                const uint64_t last_len = G.d - (G.nb - 1) * G.bucket;
                ok = hnblk == G.nb &&
                     cwords == kHeaderWords + (G.nb - 1) * (uint64_t)rec_words + 1 + (last_len * w + 31) / 32;
                if (ok && sb < nsb_tile) {
                    const uint32_t* payload = hdr + kHeaderWords;
                    uint64_t bucket_of_sb = G.bucket <= kBLK ? first_block + bi : bucket_idx;
                    const uint32_t* rec = payload + bucket_of_sb * rec_words;
                    uint32_t in_bucket = G.bucket <= kBLK ? sbi * kSB : bib * kBLK + sb * kSB;
                    float norm = __uint_as_float(__ldg(rec));
                    uint64_t bucket_len = bucket_of_sb == G.nb - 1 ? last_len : G.bucket;
                    uint32_t lastw = (uint32_t)((bucket_len * w + 31) / 32) - 1u;
                    const uint32_t* fields = rec + 1;
                    for (uint32_t e = 0; e < sn; ++e) {
                        uint32_t cur = (in_bucket + e) * w;
                        uint32_t wi = cur >> 5, sh = cur & 31u;
                        uint64_t two = (uint64_t)__ldg(fields + wi) << 32 | __ldg(fields + min(wi + 1u, lastw));
                        uint32_t field = (uint32_t)((two << sh) >> (64u - w));
                        uint32_t sym = field & ((1u << (w - 1u)) - 1u);
                        if (sym >= nlev) { ok = false; break; }
                        if (sym) {
                            float v = level_times_norm(norm, levelset, G.s, sym);
                            mine[e] += (field >> (w - 1u)) ? -v : v;
                        }
                    }
                }
            }
            if (!__all_sync(0xffffffffu, ok)) {
                if (lane == 0) latch_status(P.ws, kErrBadStream);
            }
        }
        __syncwarp();

        // ---- write the tile once ----------------------------------------------------------
        float* dst = P.acc + elem0;
        for (uint32_t i = lane * 4u; i < tile_len; i += 128u) {
            if (i + 4u <= tile_len) {
                *reinterpret_cast<float4*>(dst + i) = *reinterpret_cast<const float4*>(tile_acc + i);
            } else {
                for (uint32_t e = i; e < tile_len; ++e) dst[e] = tile_acc[e];
            }
        }
        __syncwarp();
    }
}

cudaError_t launch_decode(const DecodeParams& P, int sms, cudaStream_t stream) {
    static bool attr_set = false;
    const size_t smem = kBLK * sizeof(float);
    if (!attr_set) {
        cudaError_t e = cudaFuncSetAttribute(decode_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        attr_set = true;
    }
    uint64_t cap = (uint64_t)sms * 6 * 4;
    uint64_t grid = P.geo.ntiles < cap ? P.geo.ntiles : cap;
    decode_kernel<<<(unsigned)grid, 32, smem, stream>>>(P);
    return cudaGetLastError();
}

}  // namespace nuq
