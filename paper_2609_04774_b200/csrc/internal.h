// Internal declarations shared by the translation units of libcpattn (not part of the ABI).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include <vector>

#include "cpattn.h"

namespace cpattn {

// One query tile of the persistent scheduler: up to 128 consecutive new tokens of one request, processed
// once per pair of query heads; with an odd number of query heads per KV head, up to 256 tokens (two
// consecutive tiles), processed once per head.
struct TileItem {
    int32_t q_row0;     // first row in the packed q / out tensors
    int32_t n_rows;     // 1..128 (1..256 for tile pairs)
    int32_t kv_len0;    // keys visible to the first row: P + r0 + 1 (row i sees kv_len0 + i)
    int32_t pt_base;    // offset of the request's page table in the packed page table
    int32_t n_pages;    // entries of that page table
    int32_t n_kv_tiles; // KV tiles the unit walks: 128-key tiles from kv_lo / 128 up to its last visible key
    int32_t kv_lo;      // keys the unit may attend: absolute positions [kv_lo, kv_hi), cut by the causal
    int32_t kv_hi;      // limit; [0, INT32_MAX) for the ordinary calls
};
static_assert(sizeof(TileItem) == 32, "TileItem layout");

// One entry of a CTA's work list: KV tiles [t_begin, t_end) of query tile `item` for head pair `pair`.
// slot < 0: the piece covers the whole KV range of the unit and writes the final rows; otherwise it
// writes a normalised fp32 partial (+ LSE) into partial slot `slot`, merged afterwards.
struct PieceEntry {
    int32_t item;
    int16_t pair;
    int16_t slot;
    int32_t t_begin;
    int32_t t_end;
};
static_assert(sizeof(PieceEntry) == 16, "PieceEntry layout");

// A (query tile, head pair) unit whose KV range was split over several CTAs: its partial slots.
struct MergeEntry {
    int32_t item;
    int32_t pair;
    int32_t n_slots;
    int32_t slot_off;   // into the flat slot list
};

// Host-side schedule of one launch.
struct Schedule {
    std::vector<TileItem> items;        // query tiles, longest first
    std::vector<int32_t> cta_off;       // grid + 1 offsets into pieces
    std::vector<PieceEntry> pieces;
    std::vector<MergeEntry> merges;
    std::vector<int32_t> merge_slots;
    int32_t grid = 0;
    int32_t n_slots = 0;
};

// Device layout of a schedule inside the workspace (byte offsets from the workspace base).
struct WorkspaceLayout {
    size_t items, cta_off, pieces, merges, merge_slots, partial_o, partial_lse, total;
};

constexpr int kDefaultPageTokens = 64;   // page size assumed where no cache is at hand (schedule inspection)
constexpr int kMaxGrid = 192;                          // upper bound on CTAs (SMs) a schedule may use
constexpr int kMaxSlots = 2 * kMaxGrid + 32;           // partial slots a schedule may use
constexpr int kMinShareTiles = 8;                      // smallest per-CTA share worth spreading work for
constexpr int kMinPieceTiles = 4;                      // never cut a unit into pieces shorter than this
constexpr int kMergeLaunchCostTiles = 6;                // the merge launch behind a schedule with cut units, in KV tile steps
constexpr int kLptMaxShareTiles = 256;                 // per-CTA share up to which the least-loaded-first schedules are tried
constexpr int kLptMaxUnitsPerCta = 16;                 // ... and units per CTA (more than that balance by their number)
constexpr int kPieceCostTiles = 2;                     // fixed cost of a piece of work (prologue, epilogue, ramp) in KV tile steps
constexpr size_t kPartialRowFloats = 128;              // fp32 values of one partial row
constexpr size_t kPartialSlotRows = 2 * 128;           // two heads x 128 query rows per slot

constexpr size_t kWorkspaceHeader = 256;
constexpr int kTileRows = 128;
constexpr int kStatusWords = 4;
constexpr int kStageBuffers = 4;
constexpr size_t kStatusBytes = kStatusWords * sizeof(int32_t);
// A schedule whose work lists fit in this many bytes travels inside the kernel's launch parameters instead of
// being copied into the workspace first (one launch less for small problems).
constexpr size_t kInlineSchedBytes = 24576;
struct InlineSched {
    alignas(16) unsigned char bytes[kInlineSchedBytes];
};
constexpr int kMaxFillRanges = 4;        // row ranges a partial-result call fills with zeros / -inf inside the kernel

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

int set_error(int code, const char* fmt, ...);
int check_cuda(cudaError_t e, const char* what);

// Host planner pieces (plan.cpp)
int64_t max_tiles(int32_t B, const int64_t* new_len, const int32_t* C);
// Builds the tile list of a batch, cut at the chunk boundaries of every request's zigzag plan and
// sorted longest first.  only_shard < 0 keeps all shards; only_chunk >= 0 (B == 1) keeps that one zigzag
// chunk and numbers its rows from the chunk's first row (q, out and lse then hold the chunk alone).
// [kv_lo, kv_hi) restricts the keys (absolute positions); tiles that see none of them are left out.
// tile_rows: 128, or 256 when the units are single heads over tile pairs.
int validate_kv_cache(const cp_kv_cache* c, const char* who);
int validate_kv_cache_fp8(const cp_kv_cache_fp8* c, const char* who);
int build_tiles(int32_t B, const int64_t* cu_new, const int64_t* prefix_len, const int32_t* C,
                const int64_t* cu_pages, int32_t page_size, int32_t only_shard, int32_t only_chunk, int64_t kv_lo,
                int64_t kv_hi, int32_t tile_rows, std::vector<TileItem>& out);
// Distributes the (tile, head pair) units of s.items over `grid_max` CTAs (pairs_per_kv = units of one KV
// head per tile): whole units, KV head by KV head and longest first within a head,
// onto the least loaded CTA while they fit under the per-CTA share, the rest cut into KV ranges that
// fill every CTA to the same number of KV tiles.  Fills cta_off / pieces / merges / merge_slots.
int build_schedule(int32_t pairs_per_tile, int32_t pairs_per_kv, int32_t grid_max, Schedule& s);
// pairs_per_kv to pass to build_schedule: the real value when the batch's K/V is large, else 0 (one group)
int32_t kv_major_pairs(int32_t B, const int64_t* cu_new, const int64_t* prefix_len, int32_t Hkv, int32_t pairs_per_kv);
WorkspaceLayout workspace_layout(size_t n_items, size_t n_pieces, size_t n_merges, size_t n_merge_slots, size_t grid,
                                 size_t n_slots, size_t align = 256);
// Row ranges [begin, end) of [0, total_rows) that no tile covers, ascending; returns their number and writes
// at most max_gaps of them (pairs of int64).
int uncovered_rows(const std::vector<TileItem>& items, int64_t total_rows, int64_t* gaps, int max_gaps);

}  // namespace cpattn

struct cp_ctx {
    int device;
    int num_sms;
    int32_t* d_status;                 // kStatusWords int32 on the device
    int32_t* h_status;                 // pinned mirror
    void* h_stage[cpattn::kStageBuffers];       // pinned (device-visible) staging buffers for schedules
    size_t stage_bytes;
    cudaEvent_t stage_event[cpattn::kStageBuffers];
    bool stage_used[cpattn::kStageBuffers];
    int stage_next;
    cpattn::EncodeTiledFn encode_tiled;
    bool attn_attr_set;
    // schedule reuse (cp_ctx_cache_schedule): what the last attention call left in its workspace
    bool cache_on;
    bool cache_valid;
    std::vector<int64_t> cache_args;   // every argument the schedule depends on, compared element by element
    const void* cache_ws;              // workspace the cached schedule lives in
    cpattn::WorkspaceLayout cache_lay;
    int32_t cache_grid, cache_items, cache_merges;
    int64_t cache_rows;
    // the tensor maps of the last attention call, reused while the buffers and shapes they describe stay the same
    // (the layers of a model call with the same q / cache buffers over and over)
    bool maps_valid;
    int64_t maps_key[12];
    CUtensorMap maps[3];
    bool cache_inline;                 // the remembered work lists travel in the launch parameters
    cpattn::InlineSched cache_inl;
    int32_t cache_n_fill;
    bool cache_fill_all;
    int32_t cache_fill[2 * cpattn::kMaxFillRanges];
};
