// Shared definitions of the CUDA side: container constants, kernel parameter
// blocks, small device helpers.  Nothing here is used by the CPU oracle.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace nuq {

constexpr uint32_t kMagic = 0x3151554Eu;  // 'N','U','Q','1'
constexpr uint32_t kVersion = 1u;
constexpr uint32_t kSB = 256;             // elements per coding sub-block (one warp pass, 8 per lane)
constexpr uint32_t kBLK = 32 * kSB;       // elements per coding block / per tile
constexpr uint32_t kHeaderWords = 16;
constexpr uint32_t kMaxK = 64;

constexpr int kEncThreads = 256;          // 8 warps share a tile, 1024 elements each
constexpr int kEncWarps = kEncThreads / 32;
constexpr int kEncMinBlocks = 4;          // resident CTAs per SM the encoder is compiled for (register cap) ...
constexpr int kEncMaxBlocks = 4;          // ... and the most it is launched with

enum : uint32_t { kNormL2 = 0, kNormLinf = 1 };
enum : uint32_t { kLevelsExp = 0, kLevelsUniform = 1, kLevelsTable = 2 };
constexpr uint32_t kMaxTableS = 14;       // interior levels of a level table
enum : uint32_t { kModeErc = 0, kModeFixed = 1, kModeCoded = 2 };   // coded: as ERC, the level index written with a fitted prefix code
constexpr uint32_t kMaxCodedS = 7;        // coded level indices: at most 8 of them, code words of at most 7 bits

// status latched by kernels (most negative wins; the warning only when nothing else is latched)
enum : int { kOk = 0, kWarnNonfinite = 1, kErrBadStream = -3, kErrTimeout = -5, kErrInternal = -6 };

// look-back tile states, kept in the two top bits of a 64-bit word
constexpr uint64_t kTileAggregate = 1ull << 62;
constexpr uint64_t kTilePrefix = 2ull << 62;
constexpr uint64_t kTilePoison = 3ull << 62;
constexpr uint64_t kTileValueMask = (1ull << 62) - 1;

// per-stream scratch owned by the library
struct Workspace {
    int status;             // latched kernel status; survives calls until nuq_last_status reads it
    uint32_t dec_done_epoch; // decoder: the call (DecodeParams::epoch) whose fixed-width kernel did all the work
    // everything below is cleared at the start of every encode call
    uint64_t ticket;        // next tile to hand out
    uint64_t done;          // CTAs that have finished (they take no further ticket)
    uint64_t code_bits;     // token bits of the whole call
    uint64_t nnz;           // nonzero symbols of the whole call
    uint64_t total_words;   // payload words of the whole call
    uint64_t dec_ticket[2]; // decoder: next unit to hand out; a call uses the counter of its epoch's parity and zeroes the other one
    // followed by: uint64_t tile_state[ntiles], group_state[ceil(ntiles / 32)], then float norms[nb] for wide buckets
};
constexpr size_t kWorkspaceClearFrom = 8;

struct Geometry {
    uint64_t d;
    uint64_t nb;             // buckets
    uint64_t nblk;           // coding blocks (ERC) == table entries - 1
    uint64_t ntiles;         // CTAs' work items (<= 8192 elements each)
    uint32_t bucket;
    uint32_t s;
    uint32_t norm_kind, levelset, mode;
    uint32_t tile_elems;     // elements a full tile covers
    uint32_t blocks_per_tile;// buckets per tile when bucket <= 8192, else 1
    uint32_t sb_per_block;   // sub-blocks of a full coding block
    uint32_t blk_per_bucket; // coding blocks of a full bucket (1 when bucket <= 8192)
    uint32_t nlev;           // number of levels including zero
    uint32_t width;          // fixed-mode bits per element
    uint32_t rec_words;      // fixed mode: words per full bucket record
    uint32_t header_words;   // 16, plus the level table (padded to an even count) of a level-table stream,
                             // plus two words of code lengths in the coded mode (the last two)
    uint32_t pad;
};

struct EncodeParams {
    Geometry geo;
    const float* g;
    const float* norms_in;   // bucket norms to use, or nullptr
    uint32_t* out;
    uint64_t* out_bits;
    Workspace* ws;
    uint64_t seed, offset;
    uint32_t round_keys[20]; // Philox4x32-10 key schedule of `seed`: (k0, k1) of round 0, 1, ..., 9
    float levels[kMaxTableS + 2];    // level table: l_0 = 0, l_1 .. l_s, l_{s+1} = 1 ...
    float inv_width[kMaxTableS + 2]; // ... and 1 / (l_{j+1} - l_j), 0 for the last
    uint32_t level_code[kMaxCodedS + 1];   // coded mode: word | length << 16 of level index j at [j - 1]
    uint32_t stage_words;    // ERC: shared-memory image of a tile's records (multiple of 4); a CTA holds two
    uint32_t window_words;   // ERC: shared-memory token string of one warp and tile; a warp holds two
    uint32_t patience;       // polls a look-back wait may take before it gives up
    uint32_t grid;           // CTAs to launch
    uint32_t cluster;        // CTAs per thread-block cluster: the blocks of one wide bucket (0: no clusters)
    uint32_t overlap;        // launched so that its CTAs are set up while the kernel before it in the stream ends
};

struct DecodeParams {
    Geometry geo;
    const uint32_t* streams[kMaxK];
    uint32_t K;
    uint32_t group;          // streams decoded side by side (1, 2, 4 or 8)
    uint32_t after_fixed;    // the fixed-width kernel runs first; the general kernel returns if it did the work
    uint32_t epoch;          // number of this decode call on its workspace (never 0)
    uint32_t pad;
    // the aggregation step fused into the decoder (w == nullptr: none): see step_value in nuq_decode.cu
    float* w;                // parameters, updated in place
    float* yl;               // the momentum rule's y^l, updated in place (not touched when mu == 0)
    float step_c, step_lc;   // alpha / K and l alpha / K
    float mu;
    uint32_t pad2;
    float* acc;
    Workspace* ws;
};

__device__ __forceinline__ void latch_status(Workspace* ws, int code) {
    if (code > 0) atomicCAS(&ws->status, 0, code);          // a warning never hides an error
    else atomicMin(&ws->status, code);
}

__device__ __forceinline__ uint32_t lane_id() { return threadIdx.x & 31u; }

}  // namespace nuq
