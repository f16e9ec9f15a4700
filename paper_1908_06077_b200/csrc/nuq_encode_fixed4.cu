// ENCODE in the fixed-width mode with 4-bit fields (the paper's "4-bit" variant, Sec. 5: a sign bit and
// a 3-bit level index of the exponential level set, s = 3 .. 6): bucket norm, stochastic quantization
// (Definition 1) and packing in one kernel that reads the gradient from HBM once.
//
// Fixed-width records have a known place in the stream, so nothing is scanned, staged or handed from
// warp to warp: a kernel of its own, without the token machinery of the general encoder.  A persistent
// CTA of 8 warps takes tiles of up to 8192 elements (whole buckets, or one 8192-element block of a wider
// bucket) by ticket.  A warp owns 1024 consecutive elements (four sub-blocks of 256) of the tile, brought
// into shared memory by a bulk asynchronous copy (TMA, completion on the warp's own mbarrier) that the
// warp starts as soon as it is done with its part of the tile before.  Per tile a warp
//   1. adds up the squares of its elements (a lane's 8 or 32 in fp32, pairwise; everything beyond that in
//      fp64); the warp that is done last turns the partial sums into the tile's norms and 2^s / norm;
//      one CTA barrier;
//   2. per sub-block, a lane quantizes 8 consecutive elements (two Philox blocks), which are exactly one
//      32-bit word of eight fields, and stores that word to its place: 128 contiguous bytes per warp.
#include "nuq_encode_common.cuh"
#include "nuq_launch.h"

namespace nuq {

constexpr uint32_t kFx4WarpElems = kBLK / kEncWarps;    // 1024 elements of a tile per warp

bool fixed4_applies(const Geometry& G) {
    return G.mode == kModeFixed && G.levelset == kLevelsExp && G.width == 4u;
}

// Eight elements -> eight fields sign << 3 | index, first element in the top nibble.
__device__ __forceinline__ uint32_t quantize8_fixed4(const float4& a, const float4& b, float inv, float top, const uint4& ra,
                                                     const uint4& rb) {
    const float x[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
    const uint32_t r[8] = {ra.x, ra.y, ra.z, ra.w, rb.x, rb.y, rb.z, rb.w};
    uint32_t word = 0;
#pragma unroll
    for (int k = 0; k < 8; ++k) {
        const float y = fminf(__fmul_rn(fabsf(x[k]), inv), top);
        // see quantize_exp: the round-up is the carry into the exponent field; below the lowest level an exact comparison
        const uint32_t hi = (__float_as_uint(fmaxf(y, 1.0f)) + (0x007FFFFFu - 0x3F000000u) - (r[k] >> 9)) >> 23;
        const bool up = __uint2float_rn(r[k] >> 8) < __fmul_rn(y, 16777216.0f);
        const uint32_t field = hi | ((__float_as_uint(x[k]) >> 28) & 8u);      // a zero symbol carries no sign
        word = (word << 4) | (up ? field : 0u);
    }
    return word;
}

// COARSE: the bucket is a multiple of 1024 elements, so a warp's four sub-blocks share one bucket.
template <bool COARSE>
__global__ void __launch_bounds__(kEncThreads, kEncMinBlocks) encode_fixed4_kernel(const __grid_constant__ EncodeParams P) {
    __shared__ __align__(128) float data[kBLK];            // the tile
    __shared__ __align__(8) uint64_t s_full[kEncWarps];    // s_full[w] completes when warp w's part of a tile has landed
    __shared__ double s_partial[32];                       // sums of squares: per sub-block, or per warp at [4 w]
    __shared__ uint32_t s_maxbits[32];                     // ... or max |x| bit patterns
    __shared__ float s_sb_inv[32], s_sb_norm[32];          // per sub-block of the current tile: 2^s / norm (0: not quantized), norm
    __shared__ uint32_t s_arrived;                         // warps that have added up their squares (counts on, modulo 8)
    __shared__ TileInfo s_info[4];                         // tiles of the iterations it, it + 1, it + 2
    __shared__ uint32_t s_nnz;                             // nonzero symbols of this CTA
    __shared__ uint32_t s_last;                            // this CTA finished last

    const Geometry& G = P.geo;
    const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    uint32_t* const payload = P.out + G.header_words;
    const float top = __uint_as_float((127u + G.s) << 23); // 2^s: the norm is divided into this
    const uint32_t c2 = (uint32_t)P.offset, c3 = (uint32_t)(P.offset >> 32);
    const bool narrow = G.bucket <= kBLK;
    const uint32_t spb = narrow ? G.sb_per_block : 32u;     // sub-blocks per bucket (of the part of it a tile holds)
    const uint32_t wbase = warp * kFx4WarpElems;            // first element of the warp within a tile

    auto take_ticket = [&](uint32_t iter) {                 // thread 0: a CTA's first tile is the one with its own number
        const unsigned long long t =
            iter == 0 ? blockIdx.x : gridDim.x + atomicAdd(reinterpret_cast<unsigned long long*>(&P.ws->ticket), 1ull);
        describe_tile(G, t, &s_info[iter & 3u]);
    };
    auto bulk_elems_of = [&](const TileInfo& ti) {          // whole 16-byte pieces of the warp's part
        const uint32_t n = ti.tile_len > wbase ? min(kFx4WarpElems, ti.tile_len - wbase) : 0u;
        return ti.tile < G.ntiles ? n & ~3u : 0u;
    };
    auto start_copy = [&](uint32_t iter) {                  // one lane of the warp
        const TileInfo& ti = s_info[iter & 3u];
        const uint32_t n = bulk_elems_of(ti);
        if (n) bulk_load(data + wbase, P.g + ti.elem0 + wbase, 4u * n, &s_full[warp]);
    };

    let_next_kernel_start(P);
    wait_for_previous_kernel(P);                            // (this kernel has next to no set-up to do meanwhile)
    if (tid == 0) {
        for (int w = 0; w < kEncWarps; ++w) mbar_init(&s_full[w], 1);
        s_nnz = 0;
        s_arrived = 0;
        s_last = 0;
        take_ticket(0);
    }
    __syncthreads();
    if (lane == 0) start_copy(0);
    if (tid == 0) take_ticket(1);                           // its round trip runs while the first bytes arrive

    uint32_t it = 0;
    uint32_t my_nnz = 0;
    uint32_t parity = 0;                                    // of the next completion of s_full[warp]
    for (;; ++it) {
        const TileInfo& ti = s_info[it & 3u];
        if (ti.tile >= G.ntiles) break;
        const uint64_t elem0 = ti.elem0;
        const uint32_t tile_len = ti.tile_len, nsb_tile = ti.nsb;

        // ---- the warp's part of the tile: wait for the bulk copy, fetch the ragged end, zero the rest ----
        {
            const uint32_t bulk_elems = bulk_elems_of(ti);
            if (bulk_elems) {
                if (!mbar_wait(&s_full[warp], parity) && lane == 0) latch_status(P.ws, kErrTimeout);   // never seen; do not hang
                parity ^= 1u;
            }
            if (bulk_elems < kFx4WarpElems) {
                for (uint32_t i = bulk_elems + lane; i < kFx4WarpElems; i += 32)
                    data[wbase + i] = wbase + i < tile_len ? __ldg(P.g + elem0 + wbase + i) : 0.0f;
                __syncwarp();
            }
        }
        // a lane's eight consecutive elements of sub-block q: rows[64 q] and rows[64 q + 1]
        const float4* rows = reinterpret_cast<const float4*>(data + wbase) + 2u * lane;

        // ---- bucket norms.  L2: a lane adds the squares of its elements in fp32, pairwise (at most 5 roundings
        // of 2^-24 relative each), everything beyond that in fp64.  Linf: max |x| on the bit patterns, exact. ----
        if (P.norms_in == nullptr) {
            if (G.norm_kind == kNormL2) {
                float p8[4];
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const float4 x = rows[64 * q], y = rows[64 * q + 1];
                    float a = __fmul_rn(x.x, x.x), b = __fmul_rn(x.y, x.y);
                    a = __fmaf_rn(x.z, x.z, a); b = __fmaf_rn(x.w, x.w, b);
                    a = __fmaf_rn(y.x, y.x, a); b = __fmaf_rn(y.y, y.y, b);
                    a = __fmaf_rn(y.z, y.z, a); b = __fmaf_rn(y.w, y.w, b);
                    p8[q] = a + b;
                }
                auto exact8 = [&](int q) {                  // the same eight squares in fp64
                    const float4 x = rows[64 * q], y = rows[64 * q + 1];
                    double e = 0.0;
                    e = fma((double)x.x, (double)x.x, e); e = fma((double)x.y, (double)x.y, e);
                    e = fma((double)x.z, (double)x.z, e); e = fma((double)x.w, (double)x.w, e);
                    e = fma((double)y.x, (double)y.x, e); e = fma((double)y.y, (double)y.y, e);
                    e = fma((double)y.z, (double)y.z, e); e = fma((double)y.w, (double)y.w, e);
                    return e;
                };
                auto warp_sum = [&](double acc) {
#pragma unroll
                    for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
                    return acc;
                };
                if (COARSE) {
                    const float p32 = (p8[0] + p8[1]) + (p8[2] + p8[3]);
                    // sums that leave the fp32 range (tiny or huge coordinates, NaN): the warp adds up in fp64 instead
                    const bool out_of_range = !(p32 >= 0x1p-60f && p32 < 0x1p120f);
                    double acc = (double)p32;
                    if (__any_sync(0xffffffffu, out_of_range)) acc = (exact8(0) + exact8(1)) + (exact8(2) + exact8(3));
                    acc = warp_sum(acc);
                    if (lane == 0) s_partial[4u * warp] = acc;
                } else {
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const bool out_of_range = !(p8[q] >= 0x1p-60f && p8[q] < 0x1p120f);
                        double acc = (double)p8[q];
                        if (__any_sync(0xffffffffu, out_of_range)) acc = exact8(q);
                        acc = warp_sum(acc);
                        if (lane == 0) s_partial[4u * warp + q] = acc;
                    }
                }
            } else {
                uint32_t mx = 0;
#pragma unroll
                for (int q = 0; q < 4; ++q) {
                    const float4 x = rows[64 * q], y = rows[64 * q + 1];
                    mx = max(max(mx, __float_as_uint(fabsf(x.x))), __float_as_uint(fabsf(x.y)));    // NaN sorts above inf
                    mx = max(max(mx, __float_as_uint(fabsf(x.z))), __float_as_uint(fabsf(x.w)));
                    mx = max(max(mx, __float_as_uint(fabsf(y.x))), __float_as_uint(fabsf(y.y)));
                    mx = max(max(mx, __float_as_uint(fabsf(y.z))), __float_as_uint(fabsf(y.w)));
                    if (!COARSE || q == 3) {
                        mx = __reduce_max_sync(0xffffffffu, mx);
                        if (lane == 0) s_maxbits[4u * warp + (COARSE ? 0 : q)] = mx;
                        mx = 0;
                    }
                }
            }
        }
        // the draws of the warp's first sub-block do not depend on the norms: they are made before the
        // barrier, where the warp would otherwise wait for the slowest one
        const uint64_t ctr_lane = ((elem0 + wbase) >> 2) + 2u * lane;          // Philox counter of the lane's first block
        uint4 rn0 = philox4x32_10((uint32_t)ctr_lane, (uint32_t)(ctr_lane >> 32), c2, c3, P.round_keys);
        uint4 rn1 = philox4x32_10((uint32_t)(ctr_lane + 1u), (uint32_t)((ctr_lane + 1u) >> 32), c2, c3, P.round_keys);
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
                } else if (G.norm_kind == kNormL2) {
                    double a = 0.0;
                    for (uint32_t j = sb0; j < sb0 + spb; j += COARSE ? 4u : 1u) a += s_partial[j];
                    norm = (float)sqrt(a);
                } else {
                    uint32_t mxb = 0;
                    for (uint32_t j = sb0; j < sb0 + spb; j += COARSE ? 4u : 1u) mxb = max(mxb, s_maxbits[j]);
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
            }
        }
        __syncthreads();                                    // the one barrier of a tile: norms visible, and every warp is
                                                            // done with the previous tile's norms
        // the ticket of the tile after the next is taken now: its round trip ends long before anyone looks
        if (tid == 0) take_ticket(it + 2u);

        // ---- where the warp's words go: sub-block sbq of the tile is words [32 fx_sb, 32 fx_sb + 32) of its
        // bucket's record, behind the norm word ----
        const uint32_t sbq0 = 4u * warp;
        uint32_t* rec = nullptr;                            // the record of the bucket that holds sub-block `sbq0 + q` ...
        uint32_t fx_sb = 0, fx_words = 0;                   // ... the sub-block's number within it, field words the record has
        auto locate = [&](uint32_t sbq) {
            const uint32_t bi = sbq / spb;
            uint32_t rec_len;
            if (narrow) {
                rec = payload + (ti.first_block + bi) * G.rec_words;
                fx_sb = sbq - bi * spb;
                rec_len = min(G.bucket, tile_len - bi * G.bucket);
            } else {
                rec = payload + ti.bucket_idx * G.rec_words;
                fx_sb = ti.bib * 32u + sbq;
                rec_len = ti.rec_len;
            }
            fx_words = (rec_len + 7u) / 8u;
        };
        if (COARSE && sbq0 < nsb_tile) locate(sbq0);
        const float inv_coarse = s_sb_inv[sbq0];

#pragma unroll
        for (uint32_t q = 0; q < 4; ++q) {
            const uint32_t sbq = sbq0 + q;
            if (sbq >= nsb_tile) break;
            if (!COARSE) locate(sbq);
            else if (q) fx_sb += 1u;
            const float inv = COARSE ? inv_coarse : s_sb_inv[sbq];
            const uint32_t valid = min(32u, fx_words - 32u * fx_sb);
            if (fx_sb == 0 && lane == 0) rec[0] = __float_as_uint(s_sb_norm[sbq]);
            uint32_t word = 0;                              // a bucket that is not quantized: all fields zero
            if (inv != 0.0f) {
                word = quantize8_fixed4(rows[64 * q], rows[64 * q + 1], inv, top, rn0, rn1);
                // a field is nonzero iff its index is: adding 7 to the index carries into the field's top bit
                my_nnz += __popc(((word & 0x77777777u) + 0x77777777u) & 0x88888888u);
            }
            if (lane < valid) rec[1u + 32u * fx_sb + lane] = word;
            if (q < 3u) {                                   // the draws of the next sub-block
                const uint64_t ctr = ctr_lane + 64u * (q + 1u);
                rn0 = philox4x32_10((uint32_t)ctr, (uint32_t)(ctr >> 32), c2, c3, P.round_keys);
                rn1 = philox4x32_10((uint32_t)(ctr + 1u), (uint32_t)((ctr + 1u) >> 32), c2, c3, P.round_keys);
            }
        }

        // The warp is done with its part of the tile: the bytes of its part of the next tile are asked for now
        // and arrive while the other warps finish this one.
        __syncwarp();
        if (lane == 0) start_copy(it + 1u);
    }

#pragma unroll
    for (int o = 16; o > 0; o >>= 1) my_nnz += __shfl_xor_sync(0xffffffffu, my_nnz, o);
    if (lane == 0 && my_nnz) atomicAdd(&s_nnz, my_nnz);
    __syncthreads();                                        // every write of this CTA lies behind this barrier
    if (tid == 0 && finish_cta<kModeFixed>(P, s_nnz, 0)) s_last = 1;
    __syncthreads();
    if (s_last) {
        // Every tile of the call has been written.  The CTA that finished last leaves the call's counters zeroed,
        // so the next call on this workspace starts without a clearing pass (this kernel keeps no state per tile).
        uint64_t* state = reinterpret_cast<uint64_t*>(reinterpret_cast<char*>(P.ws) + kWorkspaceClearFrom);
        const uint64_t n = (sizeof(Workspace) - kWorkspaceClearFrom) / 8;
        for (uint64_t i = tid; i < n; i += blockDim.x) state[i] = 0;
    }
}

int fixed4_blocks_per_sm(const EncodeParams& P) {
    int n = 0;
    const bool coarse = P.geo.bucket % kFx4WarpElems == 0;
    const cudaError_t e = coarse ? cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, encode_fixed4_kernel<true>, kEncThreads, 0)
                                 : cudaOccupancyMaxActiveBlocksPerMultiprocessor(&n, encode_fixed4_kernel<false>, kEncThreads, 0);
    return e == cudaSuccess ? n : 0;
}

cudaError_t launch_encode_fixed4(const EncodeParams& P, cudaStream_t stream) {
    if (P.grid == 0) return cudaErrorInvalidValue;
    cudaLaunchConfig_t cfg = cudaLaunchConfig_t{};
    cudaLaunchAttribute attr[1];
    cfg.gridDim = dim3(P.grid);
    cfg.blockDim = dim3(kEncThreads);
    cfg.stream = stream;
    cfg.attrs = attr;
    cfg.numAttrs = 0;
    if (P.overlap) {                                        // may be set up while the kernel before it in the stream ends
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.numAttrs = 1;
    }
    if (P.geo.bucket % kFx4WarpElems == 0) return cudaLaunchKernelEx(&cfg, encode_fixed4_kernel<true>, P);
    return cudaLaunchKernelEx(&cfg, encode_fixed4_kernel<false>, P);
}

}  // namespace nuq
