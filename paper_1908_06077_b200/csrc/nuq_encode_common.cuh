// Device helpers shared by the encode kernels: Philox4x32-10, the quantizer of Definition 1 for the
// exponential level set, the bulk asynchronous copy with its mbarrier, tile geometry, and the end-of-CTA
// bookkeeping that writes the container header.
#pragma once
#include "nuq_common.cuh"

namespace nuq {

__device__ __forceinline__ uint64_t ld_volatile_u64(const uint64_t* p) {
    return *reinterpret_cast<const volatile uint64_t*>(p);
}
__device__ __forceinline__ void st_volatile_u64(uint64_t* p, uint64_t v) {
    *reinterpret_cast<volatile uint64_t*>(p) = v;
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
// With up = [float(m) < y 2^24] (always true for y >= 1) the index is max(hi, 1) if up, else 0; the
// maximum is taken on y itself (max(y, 1) has index 1 and no carry), where it is a cheap float operation.
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t quantize_exp(float v, float inv, float top, uint32_t word) {
    const float y = fminf(__fmul_rn(fabsf(v), inv), top);
    const uint32_t hi = (__float_as_uint(fmaxf(y, 1.0f)) + (0x007FFFFFu - 0x3F000000u) - (word >> 9)) >> 23;
    const bool up = __uint2float_rn(word >> 8) < __fmul_rn(y, 16777216.0f);
    return up ? hi : 0u;                                    // no round-up: y < 1 and the index is 0
}

// ---------------------------------------------------------------------------
// Bulk asynchronous copy (TMA, untiled form) and its mbarrier.  CTA-local barriers only.
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

// ---------------------------------------------------------------------------
// Thread-block clusters: shared memory of the other CTAs of the cluster (distributed shared memory).
// ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t cluster_rank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// the address, in the cluster's shared window, of this CTA's shared-memory object `p` in CTA `rank`
__device__ __forceinline__ uint32_t cluster_addr(const void* p, uint32_t rank) {
    uint32_t a;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(a) : "r"(smem_u32(p)), "r"(rank));
    return a;
}
__device__ __forceinline__ void st_cluster_u64(uint32_t addr, uint64_t v) {
    asm volatile("st.shared::cluster.u64 [%0], %1;" ::"r"(addr), "l"(v) : "memory");
}
// arrival at an mbarrier of another CTA of the cluster; the thread's earlier writes are visible to whoever
// sees the phase complete with mbar_wait_cluster
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(addr) : "memory");
}
// like mbar_wait, for a barrier at which other CTAs of the cluster arrive.  Bounded.
__device__ __forceinline__ bool mbar_wait_cluster(uint64_t* bar, uint32_t parity) {
    const uint32_t addr = smem_u32(bar);
    for (uint32_t polls = 0; polls < (1u << 17); ++polls) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\tmbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2, %3;\n\tselp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(addr), "r"(parity), "r"(2000u)
            : "memory");
        if (done) return true;
    }
    return false;
}
// every thread of every CTA of the cluster
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}

// Geometry of a tile, worked out once by the thread that took its ticket.
struct TileInfo {
    unsigned long long tile;                               // >= ntiles: there is no such tile
    unsigned long long elem0;                              // first element
    unsigned long long first_block;                        // first coding block (ERC) / bucket (narrow buckets)
    unsigned long long bucket_idx;                         // wide buckets: the bucket the tile lies in
    uint32_t tile_len, nsb;                                // elements, sub-blocks
    uint32_t bib;                                          // wide buckets: which 8192-element block of its bucket
    uint32_t rec_len;                                      // wide buckets: elements of that bucket
};

// Where tile `t` lies: whole buckets of at most 8192 elements, or one 8192-element block of a wider bucket.
__device__ __forceinline__ void describe_tile(const Geometry& G, unsigned long long t, TileInfo* out) {
    TileInfo& ti = *out;
    ti.tile = t;
    if (t >= G.ntiles) return;
    if (G.bucket <= kBLK) {
        ti.first_block = t * G.blocks_per_tile;
        ti.elem0 = ti.first_block * G.bucket;
        const uint64_t left = G.d - ti.elem0;
        ti.tile_len = left < G.tile_elems ? (uint32_t)left : G.tile_elems;
        ti.bucket_idx = 0;
        ti.bib = 0;
        ti.rec_len = 0;
    } else {
        ti.bucket_idx = t / G.blk_per_bucket;
        ti.bib = (uint32_t)(t % G.blk_per_bucket);
        ti.first_block = t;
        const uint64_t b0 = ti.bucket_idx * G.bucket;
        const uint64_t blen = G.d - b0 < G.bucket ? G.d - b0 : G.bucket;
        ti.rec_len = (uint32_t)blen;
        ti.elem0 = b0 + (uint64_t)ti.bib * kBLK;
        const uint64_t left = blen - (uint64_t)ti.bib * kBLK;
        ti.tile_len = left < kBLK ? (uint32_t)left : kBLK;
    }
    ti.nsb = (ti.tile_len + kSB - 1) / kSB;
}

// Kernels that follow one another in a stream (programmatic dependent launch).  An encode kernel says at once,
// as each CTA starts, that the kernel behind it may be launched: that kernel's CTAs then take the SM slots as
// this one's leave them and do their set-up (tables in shared memory, barriers) while the last CTAs here still
// work.  A kernel launched that way must not touch global memory before the kernel in front of it has ended
// and its writes are visible: every thread waits for that ahead of its first access (the input may have been
// written by that very kernel).  Without the launch attribute both instructions do nothing.
__device__ __forceinline__ void let_next_kernel_start(const EncodeParams& P) {
    if (P.overlap) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}
__device__ __forceinline__ void wait_for_previous_kernel(const EncodeParams& P) {
    if (P.overlap) asm volatile("griddepcontrol.wait;" ::: "memory");
}

// Bookkeeping of a CTA that has written all its tiles and takes no further ticket: counters, and the
// container header by whichever CTA finishes last (returns true there; that CTA then zeroes the call's
// state).  One thread, after a CTA barrier behind the last write.  CTAs are counted, not tiles: a CTA
// that started late and found no tile left has taken tickets all the same, and the ticket counter must
// not be zeroed before it has (the next call would start counting above zero and skip its first tiles).
template <uint32_t MODE>
__device__ bool finish_cta(const EncodeParams& P, uint64_t nnz, uint64_t code_bits) {
    const Geometry& G = P.geo;
    if (nnz) atomicAdd(reinterpret_cast<unsigned long long*>(&P.ws->nnz), (unsigned long long)nnz);
    if (code_bits) atomicAdd(reinterpret_cast<unsigned long long*>(&P.ws->code_bits), (unsigned long long)code_bits);
    __threadfence();
    const unsigned long long prev = atomicAdd(reinterpret_cast<unsigned long long*>(&P.ws->done), 1ull);
    if (prev + 1ull != (unsigned long long)gridDim.x) return false;
    __threadfence();
    uint64_t code_total, words;
    const uint64_t nnz_total = ld_volatile_u64(&P.ws->nnz);
    const uint64_t nrec = MODE == kModeErc ? G.nblk : G.nb;
    if (MODE == kModeErc) {
        code_total = ld_volatile_u64(&P.ws->code_bits);
        words = G.header_words + 2 * (G.nblk + 1) + ld_volatile_u64(&P.ws->total_words);
    } else {
        code_total = G.d * G.width;
        const uint64_t last = G.d - (G.nb - 1) * G.bucket;
        words = G.header_words + (G.nb - 1) * G.rec_words + 1 + (last * G.width + 31) / 32;
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
    if (G.levelset == kLevelsTable)                         // the interior levels, then zero padding
        for (uint32_t j = 0; j < ((G.s + 1u) & ~1u); ++j) h[kHeaderWords + j] = j < G.s ? __float_as_uint(P.levels[j + 1]) : 0u;
    if (G.mode == kModeCoded) {                             // the code lengths, one byte per level index
        uint32_t w0 = 0, w1 = 0;
        for (uint32_t j = 0; j <= G.s; ++j) {
            const uint32_t len = P.level_code[j] >> 16;
            if (j < 4u) w0 |= len << (8u * j); else w1 |= len << (8u * (j - 4u));
        }
        h[G.header_words - 2u] = w0;
        h[G.header_words - 1u] = w1;
    }
    if (P.out_bits) *P.out_bits = container_bits;
    return true;
}

}  // namespace nuq
