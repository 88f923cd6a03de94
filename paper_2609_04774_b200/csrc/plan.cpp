// Host-side integer work: the zigzag shard plan and the q-tile list of the persistent scheduler.
#include <algorithm>
#include <climits>
#include <cstdint>
#include <queue>
#include <utility>
#include <vector>

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
                const int64_t* cu_pages, int32_t page_size, int32_t only_shard, int32_t only_chunk, int64_t kv_lo,
                int64_t kv_hi, int32_t tile_rows, std::vector<TileItem>& out) {
    out.clear();
    // A launch over ALL shards of a request walks its rows as one run: adjacent zigzag chunks are adjacent rows
    // with consecutive causal limits, which the per-row limit kv_len0 + row already expresses, so a query tile may
    // span a chunk boundary (never a request).  The shard stays the accounting unit of cp_plan; only the calls
    // that compute one shard or one chunk cut their tiles at its chunk boundaries.
    const bool all_shards = only_shard < 0 && only_chunk < 0;
    for (int32_t b = 0; b < B; ++b) {
        const int64_t R = cu_new[b + 1] - cu_new[b];
        const int64_t P = prefix_len[b];
        const int32_t Cb = C[b];
        const int64_t n_runs = all_shards ? 1 : 2 * (int64_t)Cb;
        for (int64_t j = 0; j < n_runs; ++j) {
            int64_t cb = 0, ce = R;
            if (!all_shards) {
                const int32_t shard = (int32_t)(j < Cb ? j : 2 * (int64_t)Cb - 1 - j);
                if (only_shard >= 0 && shard != only_shard) continue;
                if (only_chunk >= 0 && j != only_chunk) continue;
                chunk_range(R, Cb, j, cb, ce);
            }
            // a single-chunk list addresses q / out / lse rows relative to the chunk's first row
            const int64_t row_base = only_chunk >= 0 ? cb : 0;
            for (int64_t r0 = cb; r0 < ce; r0 += tile_rows) {
                TileItem t;
                t.q_row0 = (int32_t)(cu_new[b] + r0 - row_base);
                t.n_rows = (int32_t)std::min<int64_t>(tile_rows, ce - r0);
                t.kv_len0 = (int32_t)(P + r0 + 1);
                t.pt_base = (int32_t)cu_pages[b];
                // entries the request really uses; a single chunk reads none behind its last key
                t.n_pages = (int32_t)((P + (only_chunk >= 0 ? ce : R) + page_size - 1) / page_size);
                // keys the tile's last row sees, cut to the allowed range; tiles that see none are left out
                const int64_t hi = std::min<int64_t>(kv_hi, (int64_t)t.kv_len0 + t.n_rows - 1);
                const int64_t t_lo = kv_lo / kTileRows, t_hi = (hi + kTileRows - 1) / kTileRows;
                if (t_hi <= t_lo) continue;
                t.n_kv_tiles = (int32_t)(t_hi - t_lo);
                t.kv_lo = (int32_t)kv_lo;
                t.kv_hi = (int32_t)std::min<int64_t>(kv_hi, INT32_MAX);
                out.push_back(t);
            }
        }
    }
    // Longest first; ties keep (request, row) order so the schedule is deterministic.
    std::stable_sort(out.begin(), out.end(),
                     [](const TileItem& a, const TileItem& b) { return a.n_kv_tiles > b.n_kv_tiles; });
    return CP_OK;
}

// Row ranges [begin, end) of [0, total_rows) that no tile of `items` covers (rows of other shards, rows that see
// no key of a key range), in ascending order.  Returns how many there are; at most max_gaps are written.
int uncovered_rows(const std::vector<TileItem>& items, int64_t total_rows, int64_t* gaps, int max_gaps) {
    std::vector<std::pair<int64_t, int64_t>> iv;
    iv.reserve(items.size());
    for (const TileItem& t : items) iv.emplace_back((int64_t)t.q_row0, (int64_t)t.q_row0 + t.n_rows);
    std::sort(iv.begin(), iv.end());
    int n = 0;
    int64_t at = 0;
    auto emit = [&](int64_t b, int64_t e) {
        if (e <= b) return;
        if (n > 0 && n <= max_gaps && gaps[2 * (n - 1) + 1] == b) { gaps[2 * (n - 1) + 1] = e; return; }
        if (n < max_gaps) { gaps[2 * n] = b; gaps[2 * n + 1] = e; }
        ++n;
    };
    for (const auto& x : iv) {
        emit(at, x.first);
        at = std::max(at, x.second);
    }
    emit(at, total_rows);
    return n;
}

static inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

WorkspaceLayout workspace_layout(size_t n_items, size_t n_pieces, size_t n_merges, size_t n_merge_slots, size_t grid,
                                 size_t n_slots, size_t align) {
    WorkspaceLayout w;
    size_t off = kWorkspaceHeader;
    w.items = off;        off = align_up(off + n_items * sizeof(TileItem), align);
    w.cta_off = off;      off = align_up(off + (grid + 1) * sizeof(int32_t), align);
    w.pieces = off;       off = align_up(off + n_pieces * sizeof(PieceEntry), align);
    w.merges = off;       off = align_up(off + n_merges * sizeof(MergeEntry), align);
    w.merge_slots = off;  off = align_up(off + n_merge_slots * sizeof(int32_t), align);
    w.partial_o = off;    off = align_up(off + n_slots * kPartialSlotRows * kPartialRowFloats * sizeof(float), align);
    w.partial_lse = off;  off = align_up(off + n_slots * kPartialSlotRows * sizeof(float), align);
    w.total = off;
    return w;
}

// Estimated time of a schedule in KV tile steps: the slowest CTA's tiles plus kPieceCostTiles per piece of work,
// plus the merge launch when any unit is cut.
static int64_t schedule_cost(const Schedule& s) {
    int64_t worst = 0;
    for (int32_t g = 0; g < s.grid; ++g) {
        int64_t cost = 0;
        for (int32_t k = s.cta_off[g]; k < s.cta_off[g + 1]; ++k) cost += s.pieces[k].t_end - s.pieces[k].t_begin + kPieceCostTiles;
        worst = std::max(worst, cost);
    }
    // a schedule with cut units is followed by the merge launch (about ten microseconds: six tile steps)
    return worst + (s.merges.empty() ? 0 : kMergeLaunchCostTiles);
}

// Schedule for batches whose K/V is small enough that the order of the units does not matter for L2 (one group).
// A piece of work costs its KV tile steps plus kPieceCostTiles (prologue, epilogue and the pipeline's ramp: about two
// tile steps, measured), so a CTA with many short pieces gets fewer tiles.  Whole units go, longest first, to the CTA
// with the smallest cost so far while they fit under the share; the rest are cut into KV ranges that fill the
// least-loaded CTAs up to the share (raised one step at a time when nothing fits any more).
// With cuts = false nothing is cut (plain longest-first dealing to the least-loaded CTA): no partial results and no
// merge launch, which wins for small batches of many short units.
// Returns false when the cuts need more partial slots than there are (the caller then uses the dealing scheme).
static bool build_schedule_lpt(int32_t HP, int32_t PK, int32_t grid_max, int64_t W, int32_t longest, bool cuts, Schedule& s) {
    const int64_t n_items = (int64_t)s.items.size();
    const int64_t n_units = n_items * HP;
    const int64_t c = kPieceCostTiles;
    const int64_t Wc = W + c * n_units;
    int64_t T = std::max<int64_t>((Wc + grid_max - 1) / grid_max, std::min<int32_t>(longest, kMinShareTiles) + c);
    const int32_t G = (int32_t)std::max<int64_t>(1, std::min<int64_t>(grid_max, (Wc + T - 1) / T));
    struct Piece { int32_t item; int32_t pair; int32_t t_begin; int32_t t_end; int32_t slot; int32_t cta; };
    std::vector<Piece> ps;
    ps.reserve((size_t)n_units + 2 * (size_t)G);
    // least-loaded CTA first; equal costs: lowest CTA index (the schedule is a pure function of its inputs).
    // Heap keys are cost * 256 + CTA index in one integer (kMaxGrid < 256): one comparison per step.
    struct Slot { int64_t first; int32_t second; };
    struct Heap {
        std::priority_queue<int64_t, std::vector<int64_t>, std::greater<int64_t>> q;
        void push(Slot v) { q.push(v.first * 256 + v.second); }
        Slot top() const { return {q.top() >> 8, (int32_t)(q.top() & 255)}; }
        void pop() { q.pop(); }
    } heap;
    static_assert(kMaxGrid <= 256, "CTA index must fit the key's low byte");
    for (int32_t g = 0; g < G; ++g) heap.push({0, g});
    // items are sorted longest first (build_tiles), so walking them in order is longest first
    struct TailUnit { int32_t item; int32_t pair; int32_t n; };
    std::vector<TailUnit> tail;
    // PK < HP: KV head by KV head (all CTAs then read one head's K/V at a time), longest first within a head
    for (int32_t g0 = 0; g0 < HP; g0 += PK)
    for (int64_t i = 0; i < n_items; ++i) {
        const int32_t n = s.items[i].n_kv_tiles;
        for (int32_t pr = g0; pr < g0 + PK; ++pr) {
            const Slot top = heap.top();
            if (!cuts || top.first + n + c <= T) {      // without cuts: every unit whole, to the least-loaded CTA
                heap.pop();
                ps.push_back({(int32_t)i, pr, 0, n, -1, top.second});
                heap.push({top.first + n + c, top.second});
            } else {
                tail.push_back({(int32_t)i, pr, n});
            }
        }
    }
    s.merges.clear();
    s.merge_slots.clear();
    int32_t n_slots = 0;
    const int64_t minp = kMinPieceTiles;
    for (const TailUnit& tu : tail) {
        int32_t t = 0;
        const size_t first = ps.size();
        while (t < tu.n) {
            Slot top = heap.top();
            const int64_t left = tu.n - t;
            int64_t room = T - top.first - c;
            if (room < std::min<int64_t>(minp, left)) {      // even the emptiest CTA is full: raise the share a little
                ++T;
                continue;
            }
            int64_t len = std::min<int64_t>(left, room);
            if (left - len > 0 && left - len < minp) len = (left - minp >= minp) ? left - minp : left;   // no tiny remainder
            heap.pop();
            ps.push_back({tu.item, tu.pair, t, (int32_t)(t + len), -1, top.second});
            heap.push({top.first + len + c, top.second});
            t += (int32_t)len;
        }
        if (ps.size() - first > 1) {
            s.merges.push_back({tu.item, tu.pair, (int32_t)(ps.size() - first), (int32_t)s.merge_slots.size()});
            for (size_t k = first; k < ps.size(); ++k) {
                ps[k].slot = n_slots++;
                s.merge_slots.push_back(ps[k].slot);
            }
        }
    }
    if (n_slots > kMaxSlots) return false;
    std::vector<int32_t> count(G, 0);
    for (const Piece& q : ps) ++count[q.cta];
    s.grid = G;
    s.n_slots = n_slots;
    s.cta_off.assign(G + 1, 0);
    for (int32_t g = 0; g < G; ++g) s.cta_off[g + 1] = s.cta_off[g] + count[g];
    s.pieces.resize(ps.size());
    std::vector<int32_t> fill(s.cta_off.begin(), s.cta_off.end() - 1);
    for (const Piece& q : ps)        // a CTA's pieces in the order they were dealt: whole units longest first, then its KV ranges
        s.pieces[(size_t)fill[q.cta]++] = {q.item, (int16_t)q.pair, (int16_t)q.slot, q.t_begin, q.t_end};
    return true;
}

static int build_schedule_impl(int32_t pairs_per_tile, int32_t pairs_per_kv, int32_t grid_max, bool allow_split,
                               Schedule& s) {
    const int32_t HP = pairs_per_tile;
    // units of one KV head per tile; 0 (or anything that does not divide HP): one group, longest first overall
    const int32_t PK = (pairs_per_kv >= 1 && HP % pairs_per_kv == 0) ? pairs_per_kv : HP;
    const int64_t n_items = (int64_t)s.items.size();
    const int64_t n_units = n_items * HP;
    int64_t W = 0;
    int32_t longest = 0;
    for (const TileItem& t : s.items) {
        W += (int64_t)t.n_kv_tiles * HP;
        longest = std::max(longest, t.n_kv_tiles);
    }
    if (W <= 0 || W > 0x7fffffffll || n_units > 0x7fffffffll)
        return set_error(CP_ERR_UNSUPPORTED, "schedule: %lld KV tile steps", (long long)W);
    grid_max = std::min(grid_max, kMaxGrid);
    // per-CTA share of KV tile steps; never below a short unit's length (cutting those only adds
    // prologues and merges), which also shrinks the grid for tiny problems
    const int64_t T = std::max<int64_t>((W + grid_max - 1) / grid_max, std::min<int32_t>(longest, kMinShareTiles));
    // When there are no more units than CTAs and none is longer than the share, every unit gets a CTA of its own:
    // the same critical path as packing them, and nothing is cut, so no partial results and no merge launch.
    const bool one_each = n_units <= grid_max && longest <= T;
    // Small shares (a CTA gets at most kLptMaxShareTiles KV tile steps, so the fixed cost of a piece of work is
    // felt) and few units per CTA (many short units balance by their number alone): two more schedules are built, least-loaded-first with and without cuts, and the cheapest of the three
    // by estimate is kept (the others must lose by at least 3 %).  Larger batches are balanced within a per cent
    // by the dealing scheme below, and three schedules would only cost host time.
    Schedule alt, whole;
    bool have_alt = false, have_whole = false;
    if (!one_each && allow_split && T <= kLptMaxShareTiles && n_units <= (int64_t)kLptMaxUnitsPerCta * grid_max) {
        alt.items = s.items;
        have_alt = build_schedule_lpt(HP, PK, grid_max, W, longest, true, alt);
        whole.items = s.items;
        have_whole = build_schedule_lpt(HP, PK, grid_max, W, longest, false, whole);
    }
    const int32_t G = one_each ? (int32_t)n_units
                               : (int32_t)std::max<int64_t>(1, std::min<int64_t>(grid_max, (W + T - 1) / T));
    s.grid = G;

    // 1. whole units dealt to the CTAs in serpentine order (0..G-1, G-1..0, ...) while they fit under the
    //    share; what does not fit goes to the tail.  Order: longest first, either over all units or (PK < HP)
    //    KV head by KV head.  In the second order all CTAs read the K/V of one KV head at a time (an eighth
    //    of the cache for 8 KV heads), which keeps a long context's K/V in L2 instead of streaming it from
    //    HBM for every query tile; the caller asks for it when the K/V of the batch is large.
    std::vector<int64_t> load(G, 0);
    std::vector<int32_t> count(G, 0);                  // pieces per CTA
    std::vector<int16_t> cta_of((size_t)n_units);      // CTA of a whole unit, -1 = tail
    struct TailUnit { int32_t item; int32_t pair; int32_t n; };
    std::vector<TailUnit> tail;
    {
        int64_t k = 0;   // running index over the units that were dealt
        for (int32_t g0 = 0; g0 < HP; g0 += PK)
        for (int64_t i = 0; i < n_items; ++i) {
            const int32_t n = s.items[i].n_kv_tiles;
            for (int32_t pr = g0; pr < g0 + PK; ++pr) {
                const int64_t r = k / G;
                const int32_t pos = (int32_t)(k - r * G);
                const int32_t c = (r & 1) ? G - 1 - pos : pos;
                if (load[c] + n <= T) {
                    load[c] += n;
                    ++count[c];
                    cta_of[(size_t)(i * HP + pr)] = (int16_t)c;
                    ++k;
                } else {
                    cta_of[(size_t)(i * HP + pr)] = -1;
                    tail.push_back({(int32_t)i, pr, n});
                }
            }
        }
    }

    // 2. the tail, cut into KV ranges that fill every CTA up to the share
    const int64_t minp = std::min<int64_t>(kMinPieceTiles, std::max<int64_t>(1, T));   // shortest piece worth a cut
    struct Cut { int32_t unit; int32_t cta; int32_t t_begin; int32_t t_end; int32_t slot; };
    std::vector<Cut> cuts;
    s.merges.clear();
    s.merge_slots.clear();
    int32_t n_slots = 0;
    int32_t c = 0;
    int64_t tail_left = 0;
    for (const TailUnit& tu : tail) tail_left += tu.n;
    int64_t T_cur = T;       // raised when every CTA is full and work is still left (shares are rounded)
    for (size_t u = 0; u < tail.size(); ++u) {
        int32_t t = 0;
        const int32_t n = tail[u].n;
        const size_t first = cuts.size();
        while (t < n) {
            int32_t scanned = 0;
            while (T_cur - load[c] < std::min<int64_t>(minp, n - t)) {                     // CTA is full
                c = (c + 1 == G) ? 0 : c + 1;
                if (++scanned >= G) {
                    T_cur += std::max<int64_t>(minp, (tail_left + G - 1) / G);
                    scanned = 0;
                }
            }
            int64_t len = std::min<int64_t>(n - t, T_cur - load[c]);
            if (!allow_split) len = n - t;
            if (n - t - len > 0 && n - t - len < minp) len = n - t;                           // no tiny remainder
            cuts.push_back({(int32_t)u, c, t, (int32_t)(t + len), -1});
            load[c] += len;
            ++count[c];
            t += (int32_t)len;
            tail_left -= len;
        }
        if (cuts.size() - first > 1) {
            s.merges.push_back({tail[u].item, tail[u].pair, (int32_t)(cuts.size() - first), (int32_t)s.merge_slots.size()});
            for (size_t k = first; k < cuts.size(); ++k) {
                cuts[k].slot = n_slots++;
                s.merge_slots.push_back(cuts[k].slot);
            }
        }
    }
    if (n_slots > kMaxSlots) {
        // cannot happen with one cut per CTA boundary; if it ever does, fall back to whole units only
        if (allow_split) return build_schedule_impl(pairs_per_tile, pairs_per_kv, grid_max, false, s);
        return set_error(CP_ERR_UNSUPPORTED, "schedule: %d partial slots", n_slots);
    }
    s.n_slots = n_slots;

    // 3. per-CTA lists: whole units in dealing order, then the CTA's KV ranges
    s.cta_off.assign(G + 1, 0);
    for (int32_t k = 0; k < G; ++k) s.cta_off[k + 1] = s.cta_off[k] + count[k];
    s.pieces.resize((size_t)s.cta_off[G]);
    std::vector<int32_t> fill(s.cta_off.begin(), s.cta_off.end() - 1);
    for (int32_t g0 = 0; g0 < HP; g0 += PK)
    for (int64_t i = 0; i < n_items; ++i) {
        const int32_t n = s.items[i].n_kv_tiles;
        for (int32_t pr = g0; pr < g0 + PK; ++pr) {
            const int16_t k = cta_of[(size_t)(i * HP + pr)];
            if (k >= 0) s.pieces[(size_t)fill[k]++] = {(int32_t)i, (int16_t)pr, (int16_t)-1, 0, n};
        }
    }
    for (const Cut& k : cuts)
        s.pieces[(size_t)fill[k.cta]++] = {tail[k.unit].item, (int16_t)tail[k.unit].pair, (int16_t)k.slot, k.t_begin, k.t_end};
    auto take = [&s](Schedule& o) {
        s.pieces.swap(o.pieces);
        s.cta_off.swap(o.cta_off);
        s.merges.swap(o.merges);
        s.merge_slots.swap(o.merge_slots);
        s.grid = o.grid;
        s.n_slots = o.n_slots;
    };
    if (have_alt && schedule_cost(alt) * 100 < schedule_cost(s) * 97) take(alt);     // by a margin: the estimate is coarse
    if (have_whole && schedule_cost(whole) * 100 < schedule_cost(s) * 97) take(whole);
    return CP_OK;
}

int build_schedule(int32_t pairs_per_tile, int32_t pairs_per_kv, int32_t grid_max, Schedule& s) {
    return build_schedule_impl(pairs_per_tile, pairs_per_kv, grid_max, true, s);
}

// KV head by KV head once the batch's K and V (bf16, D = 128) exceed a quarter of a 126 MB L2.
int32_t kv_major_pairs(int32_t B, const int64_t* cu_new, const int64_t* prefix_len, int32_t Hkv, int32_t pairs_per_kv) {
    int64_t tokens = 0;
    for (int32_t b = 0; b < B; ++b) tokens += prefix_len[b] + (cu_new[b + 1] - cu_new[b]);
    return tokens * Hkv * 128 * 4 > (32ll << 20) ? pairs_per_kv : 0;
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

extern "C" size_t cp_workspace_bytes(int32_t B, const int64_t* new_len, const int32_t* C, int32_t Hq) {
    if (B < 1 || !new_len || !C || Hq < 1) return 0;
    const int64_t n = max_tiles(B, new_len, C);
    if (n < 0) return 0;
    const size_t pairs = (size_t)Hq;          // one unit per head in the worst case (odd group size)
    // every unit is one piece, plus at most one extra piece per cut; the partial slots are bounded
    return workspace_layout((size_t)n, (size_t)n * pairs + kMaxSlots, kMaxSlots, kMaxSlots, kMaxGrid, kMaxSlots).total;
}

extern "C" size_t cp_workspace_bytes_fp8(int32_t B, const int64_t* new_len, const int32_t* C, int32_t Hq) {
    const size_t base = cp_workspace_bytes(B, new_len, C, Hq);
    if (base == 0) return 0;
    int64_t rows = 0;
    for (int32_t b = 0; b < B; ++b) rows += new_len[b];
    // quantised queries (one byte per element) and one fp32 scale per (token, head) row
    return base + align_up((size_t)rows * Hq * (128 + sizeof(float)), 256);
}

extern "C" int cp_schedule_inspect(int32_t B, const int64_t* cu_new, const int64_t* prefix_len, const int32_t* C,
                                   int32_t Hq, int32_t Hkv, int32_t num_sms, int64_t* summary, int32_t* pieces,
                                   int64_t max_pieces, int32_t* items, int64_t max_items) {
    if (B < 1 || !cu_new || !prefix_len || !C || Hq < 1 || Hkv < 1 || Hq % Hkv != 0 || num_sms < 1 || !summary)
        return set_error(CP_ERR_INVALID_ARG, "cp_schedule_inspect: bad arguments");
    const int32_t heads_per_unit = ((Hq / Hkv) % 2 == 0) ? 2 : 1;
    std::vector<int64_t> cu_pages(B + 1, 0);
    for (int32_t b = 0; b < B; ++b) {
        const int64_t R = cu_new[b + 1] - cu_new[b];
        if (R < 1 || prefix_len[b] < 0 || C[b] < 1) return set_error(CP_ERR_INVALID_ARG, "cp_schedule_inspect: request %d", b);
        cu_pages[b + 1] = cu_pages[b] + (prefix_len[b] + R + kDefaultPageTokens - 1) / kDefaultPageTokens;
    }
    Schedule sch;
    build_tiles(B, cu_new, prefix_len, C, cu_pages.data(), kDefaultPageTokens, -1, -1, 0, INT32_MAX,
                heads_per_unit == 2 ? kTileRows : 2 * kTileRows, sch.items);
    if (int rc = build_schedule(Hq / heads_per_unit, kv_major_pairs(B, cu_new, prefix_len, Hkv, (Hq / Hkv) / heads_per_unit),
                                num_sms, sch)) return rc;
    int64_t max_load = 0, min_load = INT64_MAX, total = 0;
    for (int32_t c = 0; c < sch.grid; ++c) {
        int64_t load = 0;
        for (int32_t k = sch.cta_off[c]; k < sch.cta_off[c + 1]; ++k) load += sch.pieces[k].t_end - sch.pieces[k].t_begin;
        max_load = std::max(max_load, load);
        min_load = std::min(min_load, load);
        total += load;
    }
    summary[0] = sch.grid;
    summary[1] = (int64_t)sch.items.size();
    summary[2] = (int64_t)sch.pieces.size();
    summary[3] = (int64_t)sch.merges.size();
    summary[4] = sch.n_slots;
    summary[5] = max_load;
    summary[6] = min_load;
    summary[7] = total;
    // does the block of work lists fit the launch parameters, and how many launches the call then makes
    const WorkspaceLayout il = workspace_layout(sch.items.size(), sch.pieces.size(), sch.merges.size(), sch.merge_slots.size(),
                                                sch.grid, 0, 16);
    summary[8] = (il.partial_o - il.items <= kInlineSchedBytes) ? 1 : 0;
    summary[9] = (summary[8] ? 0 : 1) + 1 + (sch.merges.empty() ? 0 : 1);
    if (pieces) {
        if ((int64_t)sch.pieces.size() > max_pieces) return set_error(CP_ERR_WORKSPACE, "cp_schedule_inspect: %zu pieces", sch.pieces.size());
        for (int32_t c = 0; c < sch.grid; ++c)
            for (int32_t k = sch.cta_off[c]; k < sch.cta_off[c + 1]; ++k) {
                const PieceEntry& e = sch.pieces[k];
                int32_t* o = pieces + (int64_t)k * 6;
                o[0] = c; o[1] = e.item; o[2] = e.pair; o[3] = e.t_begin; o[4] = e.t_end; o[5] = e.slot;
            }
    }
    if (items) {
        if ((int64_t)sch.items.size() > max_items) return set_error(CP_ERR_WORKSPACE, "cp_schedule_inspect: %zu items", sch.items.size());
        for (size_t i = 0; i < sch.items.size(); ++i) {
            int32_t* o = items + (int64_t)i * 4;
            o[0] = sch.items[i].q_row0; o[1] = sch.items[i].n_rows; o[2] = sch.items[i].kv_len0; o[3] = sch.items[i].n_kv_tiles;
        }
    }
    return CP_OK;
}
