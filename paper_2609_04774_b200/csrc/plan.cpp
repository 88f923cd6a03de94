// Host-side integer work: the zigzag shard plan and the q-tile list of the persistent scheduler.
#include <algorithm>

#include "internal.h"

namespace cpattn {

// Chunk j of the right-padded zigzag split of R tokens into 2C chunks (Section 2.1).
static inline void chunk_range(int64_t R, int32_t C, int64_t j, int64_t& b, int64_t& e) {
    const int64_t cl = (R + 2 * (int64_t)C - 1) / (2 * (int64_t)C);
    b = std::min(j * cl, R);
    e = std::min((j + 1) * cl, R);
}

// Visible (query, key) pairs of rows [b, e): sum over r of (P + r + 1).
static inline uint64_t pairs_of(int64_t P, int64_t b, int64_t e) {
    const uint64_t n = (uint64_t)(e - b);
    // sum_{r=b}^{e-1} (r + 1) = (b + 1 + e) * n / 2
    return n * (uint64_t)P + ((uint64_t)(b + 1 + e) * n) / 2;
}

int64_t max_tiles(int32_t B, const int64_t* new_len, const int32_t* C) {
    int64_t total = 0;
    for (int32_t b = 0; b < B; ++b) {
        if (new_len[b] < 1 || C[b] < 1) return -1;
        total += (new_len[b] + kTileRows - 1) / kTileRows + 2 * (int64_t)C[b];
    }
    return total;
}

int build_tiles(int32_t B, const int64_t* cu_new, const int64_t* prefix_len, const int32_t* C,
                const int64_t* cu_pages, int32_t only_shard, std::vector<TileItem>& out) {
    out.clear();
    for (int32_t b = 0; b < B; ++b) {
        const int64_t R = cu_new[b + 1] - cu_new[b];
        const int64_t P = prefix_len[b];
        const int32_t Cb = C[b];
        for (int64_t j = 0; j < 2 * (int64_t)Cb; ++j) {
            const int32_t shard = (int32_t)(j < Cb ? j : 2 * (int64_t)Cb - 1 - j);
            if (only_shard >= 0 && shard != only_shard) continue;
            int64_t cb, ce;
            chunk_range(R, Cb, j, cb, ce);
            for (int64_t r0 = cb; r0 < ce; r0 += kTileRows) {
                TileItem t;
                t.q_row0 = (int32_t)(cu_new[b] + r0);
                t.n_rows = (int32_t)std::min<int64_t>(kTileRows, ce - r0);
                t.kv_len0 = (int32_t)(P + r0 + 1);
                t.pt_base = (int32_t)cu_pages[b];
                t.n_pages = (int32_t)((P + R + 63) / 64);   // entries the request really uses
                t.n_kv_tiles = (int32_t)((t.kv_len0 + t.n_rows - 1 + kTileRows - 1) / kTileRows);
                t.request = b;
                t.shard = shard;
                out.push_back(t);
            }
        }
    }
    // Longest first; ties keep (request, row) order so the schedule is deterministic.
    std::stable_sort(out.begin(), out.end(),
                     [](const TileItem& a, const TileItem& b) { return a.n_kv_tiles > b.n_kv_tiles; });
    return CP_OK;
}

}  // namespace cpattn

using namespace cpattn;

extern "C" int cp_plan(int64_t new_len, int64_t prefix_len, int32_t C, cp_shard_plan* out) {
    if (new_len < 1 || prefix_len < 0 || C < 1 || !out)
        return set_error(CP_ERR_INVALID_ARG, "cp_plan: new_len=%lld prefix_len=%lld C=%d out=%p", (long long)new_len,
                         (long long)prefix_len, C, (void*)out);
    for (int32_t k = 0; k < C; ++k) {
        cp_shard_plan& s = out[k];
        s.pairs = 0;
        const int64_t js[2] = {k, 2 * (int64_t)C - 1 - k};
        for (int i = 0; i < 2; ++i) {
            chunk_range(new_len, C, js[i], s.q_begin[i], s.q_end[i]);
            s.kv_end[i] = prefix_len + s.q_end[i];
            s.pairs += pairs_of(prefix_len, s.q_begin[i], s.q_end[i]);
        }
    }
    return CP_OK;
}

extern "C" size_t cp_workspace_bytes(int32_t B, const int64_t* new_len, const int32_t* C) {
    if (B < 1 || !new_len || !C) return 0;
    const int64_t n = max_tiles(B, new_len, C);
    if (n < 0) return 0;
    return kWorkspaceHeader + (size_t)n * sizeof(TileItem);
}
