// C ABI of the library (see include/nuq.h): argument validation, geometry,
// per-stream workspace, kernel launches.  No torch types, no CPU fallback: every
// step of the path runs in the kernels of nuq_encode.cu / nuq_decode.cu.
#include <map>
#include <mutex>
#include <set>
#include <utility>

#include "../../include/nuq.h"
#include "nuq_common.cuh"
#include "nuq_launch.h"

namespace nuq {
namespace {

// Scratch of nuq_encode_static: lives in the library's device image, so every
// GPU that loads the library holds these bytes until the process exits.  In host
// code this name is only a handle for cudaGetSymbolAddress, never an address.
constexpr size_t kStaticScratchBytes = NUQ_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

struct WsEntry {
    Workspace* ptr = nullptr;
    size_t bytes = 0;
    // Bytes from the start that may hold something else than zeros where an encode call keeps its scan state
    // (0: none).  The allocation is zeroed and every encode kernel leaves its scan state zeroed, but the bucket
    // norms of a wide-bucket call or of a histogram call stay behind, at a place that depends on that call's size.
    size_t dirty_to = 0;
    uint32_t dec_epoch = 0;  // decode calls made on this workspace (see DecodeParams::epoch)
};

// One mutex guards the host-side bookkeeping below (maps, tables); it is held for the microseconds a
// call spends on the host, never across a wait for the device, except where a workspace has to grow.
std::mutex g_mu;
std::map<std::pair<int, cudaStream_t>, WsEntry> g_ws;
std::map<int, int> g_sms;                 // device -> SM count
std::set<int> g_lut_ready;                // devices whose constant LUT is uploaded
std::map<int, const float*> g_test_norms;   // device -> bucket norms of nuq_set_test_norms
float g_levels[kMaxTableS + 2], g_inv_width[kMaxTableS + 2];   // the level table of nuq_set_level_table ...
uint32_t g_levels_s = 0;                                       // ... and its number of interior levels (0: none set)
uint32_t g_level_code[kMaxCodedS + 1];                         // the code of nuq_set_level_code: word | length << 16 ...
uint32_t g_level_code_n = 0;                                   // ... and how many level indices it covers (0: none set)
std::map<int, Workspace*> g_static_ws;   // device -> address of g_static_scratch on that device
uint32_t g_erc_len[256];
bool g_erc_len_ready = false;

uint32_t erc_len(uint32_t n) {            // |ERC(n)|, 1 <= n <= 256
    if (!g_erc_len_ready) {
        uint32_t lut[256];
        build_erc_lut(lut);
        for (int i = 0; i < 256; ++i) g_erc_len[i] = lut[i] >> 16;
        g_erc_len_ready = true;
    }
    return g_erc_len[n - 1];
}

bool bucket_ok(uint32_t bucket) {
    if (bucket >= kSB && bucket <= kBLK) return bucket % kSB == 0;
    return bucket == 16384u || bucket == 32768u || bucket == 65536u;
}

bool make_geometry(uint64_t d, uint32_t bucket, uint32_t s, uint32_t flags, Geometry* G) {
    const uint32_t norm_kind = flags & 0xffu, levelset = (flags >> 8) & 0xffu, mode = (flags >> 16) & 0xffu;
    if (d == 0 || d >= (1ull << 40) || !bucket_ok(bucket) || s < 1) return false;
    if (norm_kind > 1 || levelset > 2 || mode > 2) return false;
    if (mode == kModeCoded && (levelset == kLevelsUniform || s > kMaxCodedS)) return false;
    if (s > (levelset == kLevelsUniform ? 8u : 14u)) return false;
    if (flags & ~(0x00ffffffu | NUQ_TEST_NORMS | NUQ_TEST_SHORT_PATIENCE)) return false;
    G->d = d;
    G->bucket = bucket;
    G->s = s;
    G->norm_kind = norm_kind;
    G->levelset = levelset;
    G->mode = mode;
    G->nb = (d + bucket - 1) / bucket;
    G->nlev = levelset == kLevelsUniform ? (1u << s) + 1u : s + 2u;
    G->header_words = kHeaderWords + (levelset == kLevelsTable ? ((s + 1u) & ~1u) : 0u) + (mode == kModeCoded ? 2u : 0u);
    G->pad = 0;
    uint32_t b = 0;
    while ((1u << b) < G->nlev) ++b;
    G->width = b + 1u;
    G->rec_words = 1u + (uint32_t)(((uint64_t)bucket * G->width + 31) / 32);
    const uint64_t last = d - (G->nb - 1) * bucket;
    if (bucket <= kBLK) {
        G->blocks_per_tile = kBLK / bucket;
        G->tile_elems = G->blocks_per_tile * bucket;
        G->sb_per_block = bucket / kSB;
        G->blk_per_bucket = 1;
        G->nblk = G->nb;
        G->ntiles = (G->nb + G->blocks_per_tile - 1) / G->blocks_per_tile;
    } else {
        G->blocks_per_tile = 1;
        G->tile_elems = kBLK;
        G->sb_per_block = 32;
        G->blk_per_bucket = bucket / kBLK;
        G->nblk = (G->nb - 1) * G->blk_per_bucket + (last + kBLK - 1) / kBLK;
        G->ntiles = G->nblk;
    }
    return true;
}

uint32_t max_level_code_bits(const Geometry& G) {
    if (G.mode == kModeCoded) return kMaxCodedS;            // whatever code is set
    uint32_t best = 0;
    for (uint32_t sym = 1; sym < G.nlev; ++sym) best = erc_len(sym) > best ? erc_len(sym) : best;
    return best;
}

// Most token bits that `elems` consecutive elements lying in at most `buckets` buckets can produce.
// Always true: a token has at most |ERC(1)| + 1 + L bits per position it consumes (L = longest
// level code), i.e. 2 + L bits per element.  With the Euclidean norm computed by the encoder
// itself a much smaller bound holds: a symbol above the lowest level needs r > 2^-s, and at most
// 4^s coordinates of a bucket can have that (the counting step of the paper's sparsity lemma,
// Lemma 10); all others cost at most |ERC(1)| + 1 + |ERC(1)| = 3 bits per consumed position.
// In the coded mode the same holds with the lengths of the code in use: a lowest-level token costs
// at most 2 + len(1) bits per consumed position (|ERC(gap)| + 1 + len(1) <= gap (2 + len(1))), the
// others at most the longest of the remaining words more.
uint32_t token_bits_bound(const Geometry& G, uint32_t elems, uint32_t buckets, bool norms_are_ours) {
    uint32_t L = max_level_code_bits(G), low = 1u, rest = L;    // longest code, code of index 1, longest of the others
    if (G.mode == kModeCoded) {
        L = rest = 0;
        low = g_level_code[0] >> 16;
        for (uint32_t j = 0; j <= G.s; ++j) {
            const uint32_t len = g_level_code[j] >> 16;
            L = len > L ? len : L;
            if (j >= 1) rest = len > rest ? len : rest;
        }
    }
    const uint32_t safe = elems * (2u + L);
    if (!norms_are_ours || G.norm_kind != kNormL2 || G.levelset != kLevelsExp || G.s > 7u) return safe;
    const uint64_t high = (uint64_t)buckets * ((1ull << (2u * G.s)) + 8u);      // + slack for the rounding of the norm
    const uint32_t nhigh = high < elems ? (uint32_t)high : elems;
    const uint32_t tight = (2u + low) * elems + nhigh * (rest > low ? rest - low : 0u);
    return tight < safe ? tight : safe;
}

// words of shared-memory staging the records of one ERC tile can need
uint32_t stage_words_for(const Geometry& G, bool norms_are_ours) {
    uint32_t head = 1u + (G.sb_per_block + 1u) / 2u + 1u;          // norm, lengths, padding
    return G.blocks_per_tile * head + (token_bits_bound(G, kBLK, G.blocks_per_tile, norms_are_ours) + 31u) / 32u;
}

uint64_t bound_bytes(const Geometry& G) {
    if (G.mode == kModeFixed) return 4ull * (G.header_words + G.nb * G.rec_words);
    uint64_t head = 1u + (G.sb_per_block + 1u) / 2u + 1u;
    uint64_t token_words = (G.d * (2ull + max_level_code_bits(G)) + 31) / 32;
    return 4ull * (G.header_words + 2 * (G.nblk + 1) + G.nblk * head + token_words);
}

int device_sms(int dev) {
    auto it = g_sms.find(dev);
    if (it != g_sms.end()) return it->second;
    int sms = 0;
    if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0) sms = 148;
    g_sms[dev] = sms;
    return sms;
}

// Workspace of (current device, stream), grown to `bytes`.  Growing synchronises the stream.
nuq_status get_workspace(cudaStream_t stream, size_t bytes, Workspace** out, int* dev_out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return NUQ_ERR_CUDA;
    *dev_out = dev;
    WsEntry& e = g_ws[std::make_pair(dev, stream)];
    if (e.bytes < bytes) {
        int carried = 0;
        if (e.ptr) {
            if (cudaStreamSynchronize(stream) != cudaSuccess) return NUQ_ERR_CUDA;
            if (cudaMemcpy(&carried, &e.ptr->status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return NUQ_ERR_CUDA;
            cudaFree(e.ptr);
            e.ptr = nullptr;
            e.bytes = 0;
        }
        size_t want = bytes + bytes / 2;
        void* p = nullptr;
        if (cudaMalloc(&p, want) != cudaSuccess) { cudaGetLastError(); return NUQ_ERR_CUDA; }
        // (in the call's own stream: a clearing pass on the default stream is not ordered before kernels of a
        // non-blocking stream, which would then run on a workspace that is still being cleared)
        if (cudaMemsetAsync(p, 0, want, stream) != cudaSuccess) return NUQ_ERR_CUDA;
        e.ptr = static_cast<Workspace*>(p);
        e.bytes = want;
        e.dirty_to = 0;
        if (carried && (cudaMemcpyAsync(&e.ptr->status, &carried, sizeof(int), cudaMemcpyHostToDevice, stream) != cudaSuccess ||
                        cudaStreamSynchronize(stream) != cudaSuccess))
            return NUQ_ERR_CUDA;
    }
    *out = e.ptr;
    return NUQ_OK;
}

}  // namespace
}  // namespace nuq

using namespace nuq;

// Mode of the containers this process has encoded, by device and address (see enqueue_encode): a hint
// for the decoder's choice of kernels, which check it against the containers' headers on the device.
// Guarded by g_mu.
static std::map<std::pair<int, const void*>, uint32_t> g_container_mode;

// What one encode call needs from its workspace and from shared memory.
struct EncodePlan {
    size_t state_bytes;      // control block + one look-back word per tile and per group of 32 tiles
    size_t norms_bytes;      // bucket norms for buckets wider than a tile
    uint32_t want_grid;      // CTAs that give every SM its full share
};

static EncodePlan plan_encode(EncodeParams& P, int sms, uint32_t flags) {
    const Geometry& G = P.geo;
    const bool norms_are_ours = (flags & NUQ_TEST_NORMS) == 0;
    EncodePlan pl;
    pl.state_bytes = sizeof(Workspace) + 8 * (G.ntiles + (G.ntiles + 31) / 32);
    pl.norms_bytes = G.bucket > kBLK ? 4 * G.nb : 0;
    // a look-back wait polls this often (with a pause in between: tens of ms in all) before it gives up
    P.patience = (flags & NUQ_TEST_SHORT_PATIENCE) ? 2u : 1u << 16;
    P.window_words = 0;
    P.stage_words = 0;
    if (G.mode != kModeFixed) {
        P.stage_words = (stage_words_for(G, norms_are_ours) + 3u) & ~3u;
        // a warp's 1024 elements lie in at most this many buckets
        const uint32_t warp_elems = kBLK / kEncWarps;
        // (tiles start at bucket boundaries and a warp's part at a multiple of 1024 elements)
        const uint32_t warp_buckets = G.bucket >= warp_elems ? (G.bucket % warp_elems == 0 ? 1u : 2u)
                                                             : (warp_elems % G.bucket == 0 ? warp_elems / G.bucket : warp_elems / G.bucket + 1u);
        P.window_words = (token_bits_bound(G, warp_elems, warp_buckets, norms_are_ours) + 31u) / 32u + 4u;
    }
    int best = encode_blocks_per_sm(P);                     // resident CTAs per SM: what shared memory and registers allow
    if (best > kEncMaxBlocks) best = kEncMaxBlocks;
    const int per_sm = best < 1 ? 1 : best;
    const uint64_t cap = (uint64_t)sms * (uint64_t)per_sm;
    pl.want_grid = (uint32_t)(G.ntiles < cap ? G.ntiles : cap);
    // A bucket wider than a tile: a thread-block cluster of as many CTAs as the bucket has tiles encodes it and adds
    // up its norm through distributed shared memory, so there is no separate pass over the gradient for the norms.
    // (Not with norms supplied by the caller, and not in the 4-bit fixed-width encoder.)
    P.cluster = 0;
    P.overlap = 0;
    if (G.bucket > kBLK && norms_are_ours && !fixed4_applies(G)) {
        P.cluster = G.blk_per_bucket;
        int clusters = encode_max_clusters(P);
        const int cap_clusters = sms * per_sm / (int)P.cluster;
        if (clusters > cap_clusters) clusters = cap_clusters;
        if (clusters >= 1) {
            pl.norms_bytes = 0;
            pl.want_grid = (uint32_t)(G.nb < (uint64_t)clusters ? G.nb : (uint64_t)clusters) * P.cluster;
        } else {
            P.cluster = 0;                                  // no room for a cluster: the separate norm pass
        }
    }
    return pl;
}

// Shared tail of the two encode entry points: clears the call's scan state in `ws` and
// enqueues the kernels.  `ws` must hold pl.state_bytes + pl.norms_bytes.
static nuq_status enqueue_encode(EncodeParams& P, const EncodePlan& pl, const float* g, uint32_t norm_kind,
                                 uint64_t seed, uint64_t offset, void* out, uint64_t* out_bits, Workspace* ws,
                                 WsEntry* entry, int dev, cudaStream_t stream) {
    Geometry& G = P.geo;
    const bool test_norms = (norm_kind & NUQ_TEST_NORMS) != 0;
    if (!g_lut_ready.count(dev)) {
        if (upload_erc_lut() != cudaSuccess) return NUQ_ERR_CUDA;
        g_lut_ready.insert(dev);
    }
    // The encode kernel leaves its scan state zeroed when it ends, so a clearing pass is needed only where
    // that cannot be relied on: entry == nullptr (the shared static array: always), or something was left
    // behind in the workspace (then all of that is cleared, not only what this call will use: a later, longer
    // call keeps scan state further up).
    if (entry == nullptr || entry->dirty_to > kWorkspaceClearFrom) {
        size_t upto = pl.state_bytes;
        if (entry && entry->dirty_to > upto) upto = entry->dirty_to < entry->bytes ? entry->dirty_to : entry->bytes;
        if (cudaMemsetAsync(reinterpret_cast<char*>(ws) + kWorkspaceClearFrom, 0, upto - kWorkspaceClearFrom, stream) !=
            cudaSuccess)
            return NUQ_ERR_CUDA;
        if (entry) entry->dirty_to = 0;
    }

    P.g = g;
    P.norms_in = nullptr;
    if (test_norms) {
        P.norms_in = g_test_norms[dev];
    } else if (pl.norms_bytes) {
        float* norms = reinterpret_cast<float*>(reinterpret_cast<char*>(ws) + pl.state_bytes);
        if (launch_bucket_norms(g, G.d, G.bucket, G.norm_kind, norms, G.nb, stream) != cudaSuccess) return NUQ_ERR_CUDA;
        P.norms_in = norms;
    }
    P.out = static_cast<uint32_t*>(out);
    P.out_bits = out_bits;
    P.ws = ws;
    // The kernel may be set up (its CTAs started, their tables built) while the kernel before it in the stream
    // ends; it touches global memory only when that kernel has ended.  Not on the static array, which is
    // cleared before every call, and not for calls with hundreds of tiles per CTA, which gain nothing from it
    // (the 2^30-element workload in clusters measured 2 % slower).
    P.overlap = entry && G.ntiles <= 32ull * P.grid ? 1u : 0u;
    P.seed = seed;
    P.offset = offset;
    for (uint32_t j = 0; j < kMaxTableS + 2u; ++j) {
        P.levels[j] = G.levelset == kLevelsTable ? g_levels[j] : 0.0f;
        P.inv_width[j] = G.levelset == kLevelsTable ? g_inv_width[j] : 0.0f;
    }
    for (uint32_t j = 0; j <= kMaxCodedS; ++j) P.level_code[j] = G.mode == kModeCoded ? g_level_code[j] : 0u;
    for (uint32_t r = 0; r < 10; ++r) {               // Philox key schedule (Weyl sequence)
        P.round_keys[2 * r] = (uint32_t)seed + r * 0x9E3779B9u;
        P.round_keys[2 * r + 1] = (uint32_t)(seed >> 32) + r * 0xBB67AE85u;
    }
    // the bucket norms of a wide-bucket call lie behind its scan state, where a later call with more tiles
    // keeps scan state: the next call has to clear first
    if (pl.norms_bytes && entry && !test_norms) entry->dirty_to = pl.state_bytes + pl.norms_bytes;
    if (launch_encode(P, stream) != cudaSuccess) {
        if (entry) entry->dirty_to = entry->bytes;          // whatever state the failed launch left
        return NUQ_ERR_CUDA;
    }
    // remember the mode of the container at this address: a hint for the decoder's choice of kernels,
    // checked against the header on the device
    if (g_container_mode.size() > 4096) g_container_mode.clear();
    g_container_mode[std::make_pair(dev, static_cast<const void*>(out))] = G.mode;
    return NUQ_OK;
}

static bool encode_args_ok(const float* g, uint64_t d, uint32_t bucket, uint32_t s, uint32_t norm_kind, void* out,
                           uint64_t* out_bits, Geometry* G) {
    if (!g || !out || !make_geometry(d, bucket, s, norm_kind, G)) return false;
    if ((reinterpret_cast<uintptr_t>(g) & 15u) || (reinterpret_cast<uintptr_t>(out) & 15u) ||
        (reinterpret_cast<uintptr_t>(out_bits) & 7u))
        return false;
    if (norm_kind & NUQ_TEST_NORMS) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess || !g_test_norms.count(dev) || !g_test_norms[dev]) return false;
    }
    if (G->levelset == kLevelsTable && g_levels_s != s) return false;   // no level table of this length has been set
    if (G->mode == kModeCoded && g_level_code_n != s + 1) return false; // no code for s + 1 level indices has been set
    return true;
}

extern "C" {

uint64_t nuq_encode_bound(uint64_t d, uint32_t bucket, uint32_t s, uint32_t norm_kind) {
    std::lock_guard<std::mutex> lock(g_mu);
    Geometry G;
    if (!make_geometry(d, bucket, s, norm_kind, &G)) return 0;
    return (bound_bytes(G) + 15) & ~15ull;
}

nuq_status nuq_set_level_table(const float* interior_levels, uint32_t s) {
    std::lock_guard<std::mutex> lock(g_mu);
    if (!interior_levels || s < 1 || s > kMaxTableS) return NUQ_ERR_INVALID_ARG;
    float lv[kMaxTableS + 2], iw[kMaxTableS + 2];
    lv[0] = 0.0f;
    for (uint32_t j = 1; j <= s; ++j) lv[j] = interior_levels[j - 1];
    lv[s + 1] = 1.0f;
    for (uint32_t j = 0; j <= s; ++j) {
        if (!(lv[j] < lv[j + 1])) return NUQ_ERR_INVALID_ARG;              // strictly increasing inside (0, 1), no NaN
        iw[j] = 1.0f / (lv[j + 1] - lv[j]);                                 // one IEEE division per level
        if (!(iw[j] < __builtin_huge_valf())) return NUQ_ERR_INVALID_ARG;
    }
    iw[s + 1] = 0.0f;
    for (uint32_t j = 0; j < kMaxTableS + 2u; ++j) {
        g_levels[j] = j <= s + 1 ? lv[j] : 1.0f;
        g_inv_width[j] = j <= s + 1 ? iw[j] : 0.0f;
    }
    g_levels_s = s;
    return NUQ_OK;
}

// Canonical code words for the given lengths: level indices ordered by (length, index); the first
// word is all zeros, each next one is the previous plus one, extended with zeros to its length.
static bool canonical_code(const uint8_t* lengths, uint32_t n, uint32_t* code) {
    uint32_t kraft = 0;                                      // in units of 2^-7
    for (uint32_t j = 0; j < n; ++j) {
        if (lengths[j] < 1 || lengths[j] > kMaxCodedS) return false;
        kraft += 1u << (kMaxCodedS - lengths[j]);
    }
    if (kraft > (1u << kMaxCodedS)) return false;           // no prefix code has these lengths
    uint32_t word = 0, have = 0;
    for (uint32_t len = 1; len <= kMaxCodedS; ++len) {
        word <<= 1;
        for (uint32_t j = 0; j < n; ++j)
            if (lengths[j] == len) { code[j] = word | (len << 16); ++word; ++have; }
    }
    return have == n;
}

nuq_status nuq_set_level_code(const uint8_t* lengths, uint32_t s) {
    std::lock_guard<std::mutex> lock(g_mu);
    if (!lengths || s < 1 || s > kMaxCodedS) return NUQ_ERR_INVALID_ARG;
    uint32_t code[kMaxCodedS + 1] = {0};
    if (!canonical_code(lengths, s + 1, code)) return NUQ_ERR_INVALID_ARG;
    for (uint32_t j = 0; j <= kMaxCodedS; ++j) g_level_code[j] = j <= s ? code[j] : 0u;
    g_level_code_n = s + 1;
    return NUQ_OK;
}

nuq_status nuq_fit_level_code(const uint64_t* hist, uint32_t s, uint8_t* lengths) {
    if (!hist || !lengths || s < 1 || s > kMaxCodedS) return NUQ_ERR_INVALID_ARG;
    // Huffman's construction with two queues: the leaves sorted by (count, index) and the joined nodes in
    // the order they were made (their weights never decrease).  The lighter front is taken, a leaf
    // before a joined node of the same weight.
    const uint32_t n = s + 1;
    uint32_t order[kMaxCodedS + 1];
    for (uint32_t i = 0; i < n; ++i) order[i] = i;
    for (uint32_t i = 1; i < n; ++i)                        // insertion sort, stable: equal counts stay in index order
        for (uint32_t k = i; k > 0 && hist[1 + order[k]] < hist[1 + order[k - 1]]; --k) {
            const uint32_t t = order[k]; order[k] = order[k - 1]; order[k - 1] = t;
        }
    uint64_t weight[2 * (kMaxCodedS + 1)];
    int parent[2 * (kMaxCodedS + 1)];
    for (uint32_t i = 0; i < n; ++i) { weight[i] = hist[1 + i]; parent[i] = -1; }
    uint32_t leaf = 0, joined = n, made = n;                // fronts of the two queues, next node to make
    for (uint32_t step = 0; step + 1 < n; ++step) {
        int pick[2];
        for (int k = 0; k < 2; ++k) {
            const bool leaf_left = leaf < n, joined_left = joined < made;
            if (leaf_left && (!joined_left || weight[order[leaf]] <= weight[joined])) pick[k] = (int)order[leaf++];
            else pick[k] = (int)joined++;
        }
        weight[made] = weight[pick[0]] + weight[pick[1]];
        parent[made] = -1;
        parent[pick[0]] = parent[pick[1]] = (int)made;
        ++made;
    }
    for (uint32_t i = 0; i < n; ++i) {
        uint32_t depth = 0;
        for (int at = (int)i; parent[at] >= 0; at = parent[at]) ++depth;
        lengths[i] = (uint8_t)depth;
    }
    return NUQ_OK;
}

nuq_status nuq_level_histogram(const float* g, uint64_t d, uint32_t bucket, uint32_t s, uint32_t norm_kind, uint64_t seed,
                               uint64_t offset, uint64_t* hist, void* stream_) {
    std::lock_guard<std::mutex> lock(g_mu);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    EncodeParams P;
    Geometry& G = P.geo;
    if (!g || !hist || (reinterpret_cast<uintptr_t>(hist) & 7u) || (reinterpret_cast<uintptr_t>(g) & 15u)) return NUQ_ERR_INVALID_ARG;
    if ((norm_kind >> 16) & 0xffu) return NUQ_ERR_INVALID_ARG;                      // no mode: nothing is coded here
    if (!make_geometry(d, bucket, s, norm_kind, &G) || G.levelset == kLevelsUniform) return NUQ_ERR_INVALID_ARG;
    if (G.levelset == kLevelsTable && g_levels_s != s) return NUQ_ERR_INVALID_ARG;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return NUQ_ERR_CUDA;
    P.g = g;
    P.norms_in = nullptr;
    if (norm_kind & NUQ_TEST_NORMS) {
        if (!g_test_norms.count(dev) || !g_test_norms[dev]) return NUQ_ERR_INVALID_ARG;
        P.norms_in = g_test_norms[dev];
    } else {
        Workspace* ws = nullptr;
        nuq_status st = get_workspace(stream, sizeof(Workspace) + 4 * G.nb, &ws, &dev);
        if (st != NUQ_OK) return st;
        WsEntry& e = g_ws[std::make_pair(dev, stream)];     // the norms lie where an encode call keeps its scan state
        if (e.dirty_to < sizeof(Workspace) + 4 * G.nb) e.dirty_to = sizeof(Workspace) + 4 * G.nb;
        float* norms = reinterpret_cast<float*>(reinterpret_cast<char*>(ws) + sizeof(Workspace));
        if (launch_bucket_norms(g, G.d, G.bucket, G.norm_kind, norms, G.nb, stream) != cudaSuccess) return NUQ_ERR_CUDA;
        P.norms_in = norms;
    }
    P.out = nullptr; P.out_bits = nullptr; P.ws = nullptr;
    P.seed = seed;
    P.offset = offset;
    for (uint32_t j = 0; j < kMaxTableS + 2u; ++j) {
        P.levels[j] = G.levelset == kLevelsTable ? g_levels[j] : 0.0f;
        P.inv_width[j] = G.levelset == kLevelsTable ? g_inv_width[j] : 0.0f;
    }
    for (uint32_t j = 0; j <= kMaxCodedS; ++j) P.level_code[j] = 0;
    for (uint32_t r = 0; r < 10; ++r) {
        P.round_keys[2 * r] = (uint32_t)seed + r * 0x9E3779B9u;
        P.round_keys[2 * r + 1] = (uint32_t)(seed >> 32) + r * 0xBB67AE85u;
    }
    P.stage_words = P.window_words = P.patience = P.grid = P.cluster = P.overlap = 0;
    if (cudaMemsetAsync(hist, 0, 8 * (s + 2), stream) != cudaSuccess) return NUQ_ERR_CUDA;
    if (launch_level_histogram(P, hist, device_sms(dev), stream) != cudaSuccess) return NUQ_ERR_CUDA;
    return NUQ_OK;
}

nuq_status nuq_set_test_norms(const float* norms) {
    std::lock_guard<std::mutex> lock(g_mu);
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return NUQ_ERR_CUDA;
    g_test_norms[dev] = norms;
    return NUQ_OK;
}

nuq_status nuq_encode(const float* g, uint64_t d, uint32_t bucket, uint32_t s, uint32_t norm_kind, uint64_t seed,
                      uint64_t offset, void* out, uint64_t* out_bits, void* stream_) {
    std::lock_guard<std::mutex> lock(g_mu);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    EncodeParams P;
    Geometry& G = P.geo;
    if (!encode_args_ok(g, d, bucket, s, norm_kind, out, out_bits, &G)) return NUQ_ERR_INVALID_ARG;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return NUQ_ERR_CUDA;
    const EncodePlan pl = plan_encode(P, device_sms(dev), norm_kind);
    P.grid = pl.want_grid;
    Workspace* ws = nullptr;
    nuq_status st = get_workspace(stream, pl.state_bytes + pl.norms_bytes, &ws, &dev);
    if (st != NUQ_OK) return st;
    return enqueue_encode(P, pl, g, norm_kind, seed, offset, out, out_bits, ws, &g_ws[std::make_pair(dev, stream)],
                          dev, stream);
}

nuq_status nuq_encode_static(const float* g, uint64_t d, uint32_t bucket, uint32_t s, uint32_t norm_kind,
                             uint64_t seed, uint64_t offset, void* out, uint64_t* out_bits, void* stream_) {
    std::lock_guard<std::mutex> lock(g_mu);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    EncodeParams P;
    Geometry& G = P.geo;
    if (!encode_args_ok(g, d, bucket, s, norm_kind, out, out_bits, &G)) return NUQ_ERR_INVALID_ARG;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return NUQ_ERR_CUDA;
    const EncodePlan pl = plan_encode(P, device_sms(dev), norm_kind);
    if (pl.state_bytes + pl.norms_bytes > kStaticScratchBytes) return NUQ_ERR_CAPACITY;   // vector too long for the array
    P.grid = pl.want_grid;
    auto it = g_static_ws.find(dev);
    if (it == g_static_ws.end()) {
        // first call on this device: ask the runtime where this device keeps the array
        void* p = nullptr;
        if (cudaGetSymbolAddress(&p, g_static_scratch) != cudaSuccess || !p) {
            cudaGetLastError();
            return NUQ_ERR_CUDA;
        }
        it = g_static_ws.emplace(dev, static_cast<Workspace*>(p)).first;
    }
    // the array is shared by every stream of the device: it is cleared before every call
    return enqueue_encode(P, pl, g, norm_kind, seed, offset, out, out_bits, it->second, nullptr, dev, stream);
}

// Shared by the two decode entry points.  `w` == nullptr: the sums only.
static nuq_status enqueue_decode(const void* const* streams, uint32_t K, uint64_t d, uint32_t bucket, uint32_t s, float* acc,
                                 float* w, float* yl, float alpha, float mu, float l, void* stream_) {
    std::lock_guard<std::mutex> lock(g_mu);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    DecodeParams P;
    if (!streams || K < 1 || K > kMaxK) return NUQ_ERR_INVALID_ARG;
    // with one or two streams the sums are added up in acc itself, so it is needed even when only w is wanted
    if (!acc && (!w || K < 3)) return NUQ_ERR_INVALID_ARG;
    if (w && mu != 0.0f && !yl) return NUQ_ERR_INVALID_ARG;
    if (w && !(alpha == alpha && mu >= 0.0f && mu < 1.0f && l >= 0.0f && l <= 1.0f)) return NUQ_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(acc) & 15u) || (reinterpret_cast<uintptr_t>(w) & 15u) ||
        (reinterpret_cast<uintptr_t>(yl) & 15u))
        return NUQ_ERR_INVALID_ARG;
    // the level set and mode come from each container's header; geometry only needs (d, bucket, s)
    if (!make_geometry(d, bucket, s, 0, &P.geo)) return NUQ_ERR_INVALID_ARG;
    for (uint32_t k = 0; k < K; ++k) {
        if (!streams[k] || (reinterpret_cast<uintptr_t>(streams[k]) & 15u)) return NUQ_ERR_INVALID_ARG;
        P.streams[k] = static_cast<const uint32_t*>(streams[k]);
    }
    for (uint32_t k = K; k < kMaxK; ++k) P.streams[k] = nullptr;
    P.K = K;
    P.group = K >= 8 ? 8u : K >= 3 ? 4u : K;            // 1, 2, 4 or 8 streams side by side
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return NUQ_ERR_CUDA;
    // A small call with the widest units (32 / group sub-blocks per warp) gives only a few warps of the whole
    // GPU something to do, and a warp's walk is a chain of dependent steps: narrower units (lanes left idle)
    // put more warps to work.
    while (P.group < 8u && 2u * P.geo.ntiles * P.group <= 8u * (uint64_t)device_sms(dev)) P.group *= 2u;
    P.after_fixed = w ? 0u : 1u;                        // all streams believed to be in the fixed-width mode? (sums only)
    for (uint32_t k = 0; k < K; ++k) {
        auto it = g_container_mode.find(std::make_pair(dev, streams[k]));
        if (it == g_container_mode.end() || it->second != kModeFixed) P.after_fixed = 0;
    }
    P.acc = acc;
    P.w = w;
    P.yl = w && mu != 0.0f ? yl : nullptr;
    P.step_c = w ? (float)((double)alpha / (double)K) : 0.0f;          // one rounding each
    P.step_lc = w ? (float)((double)l * (double)alpha / (double)K) : 0.0f;
    P.mu = w ? mu : 0.0f;
    P.pad2 = 0;
    Workspace* ws = nullptr;
    nuq_status st = get_workspace(stream, sizeof(Workspace), &ws, &dev);
    if (st != NUQ_OK) return st;
    P.ws = ws;
    // The ticket counter a decode call uses has been zeroed by the call before it (or by the allocation, or by an
    // encode call, which leaves both zeroed): calls take the two counters in turn and each zeroes the other one.
    WsEntry& entry = g_ws[std::make_pair(dev, stream)];
    if (++entry.dec_epoch == 0) entry.dec_epoch = 2;        // never 0, parity kept
    P.epoch = entry.dec_epoch;
    P.pad = 0;
    if (launch_decode(P, device_sms(dev), stream) != cudaSuccess) return NUQ_ERR_CUDA;
    return NUQ_OK;
}

nuq_status nuq_decode_accumulate(const void* const* streams, uint32_t K, uint64_t d, uint32_t bucket, uint32_t s,
                                 float* acc, void* stream) {
    if (!acc) return NUQ_ERR_INVALID_ARG;
    return enqueue_decode(streams, K, d, bucket, s, acc, nullptr, nullptr, 0.0f, 0.0f, 0.0f, stream);
}

nuq_status nuq_decode_update(const void* const* streams, uint32_t K, uint64_t d, uint32_t bucket, uint32_t s, float* acc,
                             float* w, float* yl, float alpha, float mu, float l, void* stream) {
    if (!w) return NUQ_ERR_INVALID_ARG;
    return enqueue_decode(streams, K, d, bucket, s, acc, w, yl, alpha, mu, l, stream);
}

nuq_status nuq_last_status(void* stream_) {
    std::lock_guard<std::mutex> lock(g_mu);
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return NUQ_ERR_CUDA;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return NUQ_ERR_CUDA;
    int status = 0;
    auto it = g_ws.find(std::make_pair(dev, stream));
    if (it != g_ws.end() && it->second.ptr) {
        if (cudaMemcpy(&status, &it->second.ptr->status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return NUQ_ERR_CUDA;
        if (status != 0 && cudaMemset(&it->second.ptr->status, 0, sizeof(int)) != cudaSuccess) return NUQ_ERR_CUDA;
    }
    auto st = g_static_ws.find(dev);               // kernels of nuq_encode_static latch into the static scratch
    if (st != g_static_ws.end()) {
        int s2 = 0;
        if (cudaMemcpy(&s2, &st->second->status, sizeof(int), cudaMemcpyDeviceToHost) != cudaSuccess) return NUQ_ERR_CUDA;
        if (s2 != 0 && cudaMemset(&st->second->status, 0, sizeof(int)) != cudaSuccess) return NUQ_ERR_CUDA;
        if (s2 < status) status = s2;
    }
    return status;
}

nuq_status nuq_stream_info(const void* out, nuq_info* host_out, void* stream_) {
    if (!out || !host_out) return NUQ_ERR_INVALID_ARG;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_);
    uint32_t h[kHeaderWords];
    if (cudaMemcpyAsync(h, out, sizeof(h), cudaMemcpyDeviceToHost, stream) != cudaSuccess) return NUQ_ERR_CUDA;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return NUQ_ERR_CUDA;
    if (h[0] != kMagic || h[1] != kVersion) return NUQ_ERR_BAD_STREAM;
    auto u64 = [&](int i) { return (uint64_t)h[i] | ((uint64_t)h[i + 1] << 32); };
    host_out->d = u64(2);
    host_out->bucket = h[4];
    host_out->s = h[5];
    host_out->flags = h[6];
    host_out->sub_block = h[7];
    host_out->nblk = u64(8);
    host_out->container_bits = u64(10);
    host_out->code_bits = u64(12);
    host_out->nnz = u64(14);
    return NUQ_OK;
}

void nuq_shutdown(void) {
    std::lock_guard<std::mutex> lock(g_mu);
    int cur = 0;
    cudaGetDevice(&cur);
    for (auto& kv : g_ws) {
        if (kv.second.ptr) {
            cudaSetDevice(kv.first.first);
            cudaFree(kv.second.ptr);
        }
    }
    g_ws.clear();
    cudaSetDevice(cur);
}

const char* nuq_version(void) { return "nuq-b200 0.1 (sm_100a)"; }

}  // extern "C"
