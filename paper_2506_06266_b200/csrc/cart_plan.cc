// Host-side work planner: see include/cart_plan.h for the contract.
#include <algorithm>
#include <cstdint>
#include <tuple>
#include <vector>

#include "cart_plan.h"

namespace {

// One (shared segment, M-tile, KV head) run of full shared tiles.
struct Combo {
    int32_t cls;           // shared segment class
    uint32_t reader_begin; // first reader entry of the M-tile
    uint32_t n_readers;
    uint32_t kv_head;
    uint64_t n_tiles;
    uint32_t n_chunks;     // filled by the partition
};

struct SharedClass {
    cart_plan_seg seg;      // the stored segment (row of token 0, KV head 0, layer 0)
    uint32_t reader_begin;  // entries of this class are contiguous in readers[]
    uint32_t n_readers;
    uint32_t first_combo;   // combos of this class: (m * n_kv_heads + g) from here
};

// Hands out tiles of consecutive groups (row groups of the stream, tile runs of the shared part) to
// `C` blocks in order.  A tile weighs 1, every part of a group that a block takes ("unit") weighs
// `A` on top.  When a block is opened it is given an equal share of the weight that is left, counting
// one unit per group still to come and one more per block boundary still to come (a boundary is
// assumed to cut a group); the share is recomputed for every block, so an error in that assumption
// does not pile up on the last block.  With A = 0 the blocks' tile counts differ by at most one.
struct Balancer {
    uint64_t C, A;
    uint64_t tiles_left;   // tiles not handed out yet
    uint64_t groups_left;  // groups of which nothing has been handed out yet
    uint64_t c = 0;        // block being filled
    uint64_t acc = 0;      // weight block c holds
    uint64_t budget = 0;
    bool whole = false;    // every block takes exactly one whole group (small batches: see the stream part)

    Balancer(uint64_t blocks, uint64_t unit_cost, uint64_t tiles, uint64_t groups)
        : C(blocks), A(unit_cost), tiles_left(tiles), groups_left(groups) { open(false); }

    void open(bool mid_group)
    {
        const uint64_t blocks = C > c ? C - c : 1;
        const uint64_t wt = tiles_left + A * (groups_left + (mid_group ? 1 : 0) + (blocks - 1));
        budget = (wt + blocks - 1) / blocks;
        acc = 0;
    }
    // Tiles the current block takes from a group with `rem` tiles left (>= 1); moves on to the next block
    // first if the current one cannot pay for another unit.  `fresh`: nothing of the group was taken yet.
    uint64_t take(uint64_t rem, bool fresh)
    {
        if (whole) {
            if (acc > 0 && c + 1 < C) { ++c; open(false); }
            return rem;
        }
        for (;;) {
            const uint64_t paid = acc + A;
            uint64_t room = budget > paid ? budget - paid : 0;
            if (room == 0 && acc > 0 && c + 1 < C) { ++c; open(!fresh); continue; }
            if (room == 0) room = 1;
            if (c + 1 >= C) room = rem;  // the last block takes what is left
            return rem < room ? rem : room;
        }
    }
    // Books `t` tiles of a group on block c; `more`: the group still has tiles after them.
    void commit(uint64_t t, bool fresh, bool more)
    {
        acc += A + t;
        tiles_left -= t;
        if (fresh) --groups_left;
        if (whole) return;
        if (acc >= budget && c + 1 < C) { ++c; open(more); }
    }
    bool block_has_work() const { return acc > 0; }
};

bool same_storage(const cart_plan_seg &a, const cart_plan_seg &b)
{
    return a.k_row == b.k_row && a.v_row == b.v_row && a.n_tok == b.n_tok && a.head_stride == b.head_stride &&
           a.layer_stride == b.layer_stride && (a.flags & CART_SEG_PAGED) == (b.flags & CART_SEG_PAGED);
}

}  // namespace

extern "C" cart_status cart_plan_build_shared(const cart_plan_seg *segs, const int32_t *seg_begin, int32_t n_reqs,
                                              int32_t n_kv_heads, int32_t group, int32_t n_cta,
                                              int32_t tile_tokens, int32_t share_min_readers,
                                              int32_t share_tile_tokens, cart_plan_out *o)
{
    if (!segs || !seg_begin || !o || !o->items || !o->cta_begin || !o->merges) return CART_ERR_INVALID_ARG;
    if (n_reqs < 1 || n_kv_heads < 1 || n_cta < 1 || tile_tokens < 1 || group < 1 || group > 128 ||
        share_min_readers < 0)
        return CART_ERR_INVALID_ARG;
    const bool want_share = share_min_readers > 0;
    if (want_share && (share_tile_tokens < tile_tokens || share_tile_tokens % tile_tokens != 0 || !o->units ||
                       !o->unit_cta_begin || !o->readers || !o->reader_slot || !o->reader_merge))
        return CART_ERR_INVALID_ARG;

    const uint64_t T = (uint64_t)tile_tokens;
    const uint64_t TS = want_share ? (uint64_t)share_tile_tokens : 0;
    const int32_t n_segs = seg_begin[n_reqs];
    for (int32_t i = 0; i < n_reqs; ++i) {
        uint64_t toks = 0;
        for (int32_t s = seg_begin[i]; s < seg_begin[i + 1]; ++s) {
            if (segs[s].n_tok == 0) return CART_ERR_INVALID_ARG;
            toks += segs[s].n_tok;
        }
        if (toks == 0) return CART_ERR_EMPTY;
    }

    // ---- 1. which segments are shared, and by whom ------------------------------------------------
    std::vector<int32_t> seg_entry((size_t)n_segs, -1);  // reader entry of a shared segment occurrence
    std::vector<int32_t> seg_cls((size_t)n_segs, -1);
    std::vector<SharedClass> classes;
    std::vector<Combo> combos;
    int32_t n_entries = 0;
    const uint32_t R = (uint32_t)(128 / group);  // readers per M-tile
    if (want_share) {
        // order the candidate occurrences by storage, then by position in the batch
        std::vector<int32_t> order;
        for (int32_t s = 0; s < n_segs; ++s)
            if (segs[s].n_tok >= TS) order.push_back(s);
        auto key = [&](int32_t s) {
            return std::make_tuple(segs[s].k_row, segs[s].v_row, segs[s].n_tok, segs[s].head_stride,
                                   segs[s].layer_stride, s);
        };
        std::sort(order.begin(), order.end(), [&](int32_t a, int32_t b) { return key(a) < key(b); });
        std::vector<std::pair<int32_t, int32_t>> groups;  // (first index in order, count), shared ones only
        for (size_t a = 0; a < order.size();) {
            size_t b = a + 1;
            while (b < order.size() && same_storage(segs[order[a]], segs[order[b]])) ++b;
            if ((int64_t)(b - a) >= share_min_readers) groups.emplace_back((int32_t)a, (int32_t)(b - a));
            a = b;
        }
        // classes in order of first appearance in the batch (a deterministic, input-order layout)
        std::sort(groups.begin(), groups.end(), [&](const std::pair<int32_t, int32_t> &x,
                                                    const std::pair<int32_t, int32_t> &y) {
            return order[(size_t)x.first] < order[(size_t)y.first];
        });
        for (const auto &gr : groups) {
            if (n_entries + gr.second > o->readers_cap) return CART_ERR_CAPACITY;
            SharedClass c;
            c.seg = segs[order[(size_t)gr.first]];
            c.reader_begin = (uint32_t)n_entries;
            c.n_readers = (uint32_t)gr.second;
            c.first_combo = (uint32_t)combos.size();
            for (int32_t j = 0; j < gr.second; ++j) {
                const int32_t s = order[(size_t)(gr.first + j)];
                seg_entry[(size_t)s] = n_entries;
                seg_cls[(size_t)s] = (int32_t)classes.size();
                // batch index of the request that owns occurrence s
                const int32_t req = (int32_t)(std::upper_bound(seg_begin, seg_begin + n_reqs + 1, s) - seg_begin) - 1;
                o->readers[n_entries++] = (uint32_t)req;
            }
            const uint32_t m_tiles = (c.n_readers + R - 1) / R;
            for (uint32_t m = 0; m < m_tiles; ++m)
                for (int32_t g = 0; g < n_kv_heads; ++g) {
                    Combo cb;
                    cb.cls = (int32_t)classes.size();
                    cb.reader_begin = c.reader_begin + m * R;
                    cb.n_readers = std::min(R, c.n_readers - m * R);
                    cb.kv_head = (uint32_t)g;
                    cb.n_tiles = c.seg.n_tok / TS;
                    cb.n_chunks = 0;
                    combos.push_back(cb);
                }
            classes.push_back(c);
        }
    }

    // ---- 2. divide the shared runs over blocks; shrink the block count until the partials fit ------
    // Blocks are balanced by weight: a tile weighs 1, a unit weighs unit_cost on top (its queries are
    // loaded, its partials written).
    uint64_t W_sh = 0;
    for (const Combo &cb : combos) W_sh += cb.n_tiles;
    const uint64_t Au = o->unit_cost > 0 ? (uint64_t)o->unit_cost : 0;
    // walks the runs; calls emit(combo index, tiles done before, tiles taken, chunk, block) per unit and
    // returns the number of blocks that received work
    auto walk = [&](uint64_t C, auto &&emit) -> uint64_t {
        Balancer bal(C, Au, W_sh, (uint64_t)combos.size());
        for (size_t ci = 0; ci < combos.size(); ++ci) {
            uint64_t rem = combos[ci].n_tiles, done = 0;
            uint32_t chunk = 0;
            while (rem > 0) {
                const bool fresh = done == 0;
                const uint64_t t = bal.take(rem, fresh);
                emit(ci, done, t, chunk++, bal.c);
                rem -= t;
                done += t;
                bal.commit(t, fresh, rem > 0);
            }
        }
        return bal.block_has_work() ? bal.c + 1 : bal.c;
    };
    // Side by side: how many of the n_cta blocks the shared kernel gets.  Estimated times in nanoseconds,
    // fitted to measurements on B200 (launch lists of the two kernels at several divisions of the SMs):
    //   shared kernel on s blocks   3000 + (1200 per 128-token tile + 4000 per unit) of its heaviest block
    //   stream kernel on c blocks   3000 + max((510 per 64-token tile + 1500 per row-group piece) / c,
    //                                          5.1 per tile)      -- the second term is the HBM bound
    // One after the other costs the sum of the two on all blocks; side by side the larger of the two on their shares.  The division with the smallest estimate is taken if it beats one-after-the-other by 5 %.
    uint64_t n_cta_stream = (uint64_t)n_cta, n_cta_shared = (uint64_t)n_cta;
    o->n_shared_ctas = 0;
    if (W_sh > 0 && o->side_by_side > 0 && n_cta >= 2) {
        uint64_t st_tiles = 0, st_rgs = 0;
        for (int32_t i = 0; i < n_reqs; ++i) {
            uint64_t t = 0;
            for (int32_t sgi = seg_begin[i]; sgi < seg_begin[i + 1]; ++sgi) {
                const uint64_t nt = seg_cls[(size_t)sgi] < 0 ? segs[sgi].n_tok : segs[sgi].n_tok % TS;
                t += (nt + T - 1) / T;
            }
            st_tiles += t * (uint64_t)n_kv_heads;
            if (t > 0) st_rgs += (uint64_t)n_kv_heads;
        }
        if (st_tiles > 0) {
            // The heaviest block of the division that step 3 would make of the runs (runs of unequal length do not
            // divide evenly: a block that holds a long run whole sets the time).  With very many runs the walk per
            // candidate is not worth its host time and the even share stands in for it.
            auto est_shared = [&](uint64_t blocks) -> uint64_t {
                blocks = std::min<uint64_t>(blocks, std::max<uint64_t>(1, W_sh / 2));
                if (combos.size() > 256) {
                    const uint64_t cuts = combos.size() % blocks == 0 ? 0 : blocks - 1;
                    return 3000 + (W_sh * 1200 + (combos.size() + cuts) * 4000) / blocks;
                }
                uint64_t at = 0, w = 0, worst = 0;
                walk(blocks, [&](size_t, uint64_t, uint64_t take, uint32_t, uint64_t c) {
                    if (c != at) { worst = std::max(worst, w); w = 0; at = c; }
                    w += take * 1200 + 4000;
                });
                return 3000 + std::max(worst, w);
            };
            auto est_stream = [&](uint64_t blocks) {
                return 3000 + std::max<uint64_t>((st_tiles * 510 + (st_rgs + blocks) * 1500) / blocks, (st_tiles * 51) / 10);
            };
            uint64_t S = 0;
            if (o->side_by_side > 1) {
                S = std::min<uint64_t>((uint64_t)o->side_by_side, (uint64_t)n_cta - 1);
            } else {
                uint64_t best = UINT64_MAX;
                for (uint64_t s2 = 1; s2 < (uint64_t)n_cta; ++s2) {
                    // (a division that leaves the runs whole is preferred: measured on one shared Cartridge of 32 runs, 28 blocks
                    //  for the tensor-core kernel took 8 us longer per layer than 32)
                    const uint64_t est = std::max(est_shared(s2), est_stream((uint64_t)n_cta - s2)) +
                                         (combos.size() % s2 == 0 ? 0 : 6000);
                    if (est < best) { best = est; S = s2; }
                }
                const uint64_t serial = est_shared((uint64_t)n_cta) + est_stream((uint64_t)n_cta);
                if (best * 100 >= serial * 95) S = 0;  // not worth it: each kernel gets all blocks in turn
            }
            if (S > 0) {
                n_cta_shared = S;
                n_cta_stream = (uint64_t)n_cta - S;
                o->n_shared_ctas = (int32_t)S;
            }
        }
    }
    uint64_t C_sh = 0;
    if (W_sh > 0) {
        // a block should get at least two tiles
        C_sh = std::min<uint64_t>(n_cta_shared, std::max<uint64_t>(1, W_sh / 2));
        // every stream piece of a row group with a shared part takes a slot, and so does every split
        const int64_t stream_reserve = (int64_t)n_reqs * n_kv_heads + 2 * (int64_t)n_cta;
        for (;;) {
            int64_t need = 0;
            for (Combo &cb : combos) cb.n_chunks = 0;
            walk(C_sh, [&](size_t ci, uint64_t, uint64_t, uint32_t, uint64_t) {
                ++combos[ci].n_chunks;
                need += combos[ci].n_readers;
            });
            if (need + stream_reserve <= (int64_t)o->slots_cap) break;
            C_sh /= 2;
            if (C_sh == 0) break;
        }
        if (C_sh == 0) {  // cannot fit: share nothing
            combos.clear();
            classes.clear();
            std::fill(seg_entry.begin(), seg_entry.end(), -1);
            std::fill(seg_cls.begin(), seg_cls.end(), -1);
            n_entries = 0;
            W_sh = 0;
            n_cta_stream = (uint64_t)n_cta;
            o->n_shared_ctas = 0;
        }
    }

    // ---- 3. emit the shared units ------------------------------------------------------------------
    int32_t nu = 0;
    uint64_t used_sh = 0;
    if (want_share) {
        o->unit_cta_begin[0] = 0;
        uint64_t cur = 0;  // block whose units are being written
        bool overflow = false;
        if (C_sh > 0)
            used_sh = walk(C_sh, [&](size_t ci, uint64_t done, uint64_t take, uint32_t chunk, uint64_t c) {
                if (nu >= o->units_cap) { overflow = true; return; }
                while (cur < c) o->unit_cta_begin[++cur] = (uint32_t)nu;
                const Combo &cb = combos[ci];
                const cart_plan_seg &sg = classes[(size_t)cb.cls].seg;
                cart_shared_unit &u = o->units[nu++];
                const uint32_t tok0 = (uint32_t)(done * TS);
                u.flags = (sg.flags & CART_SEG_SUFFIX) ? (uint16_t)CART_UNIT_SUFFIX : (uint16_t)0;
                if (sg.flags & CART_SEG_PAGED) {
                    u.k_row = sg.k_row + (uint32_t)(tok0 / T);
                    u.v_row = cb.kv_head * sg.head_stride;
                    u.flags |= (uint16_t)CART_UNIT_PAGED;
                } else {
                    u.k_row = sg.k_row + cb.kv_head * sg.head_stride + tok0;
                    u.v_row = sg.v_row + cb.kv_head * sg.head_stride + tok0;
                }
                u.layer_stride = sg.layer_stride;
                u.n_tiles = (uint32_t)take;
                u.reader_begin = cb.reader_begin;
                u.n_readers = cb.n_readers;
                u.kv_head = (uint16_t)cb.kv_head;
                u.chunk = chunk;
                u.lim_base = 0;
                u.lim_cap = 0;
                u.tr_hi = 0;
                u.reserved = 0;
            });
        if (overflow) return CART_ERR_CAPACITY;
        for (uint64_t b = cur; b < (uint64_t)n_cta; ++b) o->unit_cta_begin[b + 1] = (uint32_t)nu;
    }
    o->n_units = nu;
    o->n_unit_cta_used = (int32_t)used_sh;
    o->n_readers = n_entries;
    o->shared_tiles = (int64_t)W_sh;

    // ---- 4. the stream: what is left of every request, laid end to end -------------------------------
    // A shared segment leaves its ragged tail (n_tok mod TS tokens) in its readers' streams.
    auto stream_part = [&](int32_t s, uint32_t *tok0, uint32_t *ntok) {
        if (seg_cls[(size_t)s] < 0) { *tok0 = 0; *ntok = segs[s].n_tok; return; }
        const uint32_t full = (uint32_t)((segs[s].n_tok / TS) * TS);
        *tok0 = full;
        *ntok = segs[s].n_tok - full;
    };
    uint64_t tiles_per_head = 0;
    for (int32_t s = 0; s < n_segs; ++s) {
        uint32_t t0, nt;
        stream_part(s, &t0, &nt);
        tiles_per_head += (nt + T - 1) / T;
    }
    const uint64_t W = tiles_per_head * (uint64_t)n_kv_heads;
    const uint64_t C = std::min<uint64_t>(n_cta_stream, W);

    int32_t ni = 0, nm = 0;
    uint32_t next_slot = 0;
    uint64_t pos = 0;  // tiles handed out so far
    uint64_t c = 0;    // block being filled
    // Blocks are balanced by weight: a tile weighs 1, starting a piece weighs piece_cost (what its
    // epilogue costs a block, in tile times).
    const uint64_t A = o->piece_cost > 0 ? (uint64_t)o->piece_cost : 0;
    uint64_t rgs_with_tiles = 0;
    for (int32_t i = 0; i < n_reqs; ++i) {
        bool any = false;
        for (int32_t s = seg_begin[i]; s < seg_begin[i + 1] && !any; ++s) {
            uint32_t t0, nt;
            stream_part(s, &t0, &nt);
            any = nt > 0;
        }
        if (any) rgs_with_tiles += (uint64_t)n_kv_heads;
    }
    // Small batches are bound by latencies, not by bandwidth: when every row group can have a block of its own and
    // an even split would leave a block only a few tiles, a row group is not cut at all -- a block streams it whole
    // and writes the result itself (or one partial, if part of the cache is shared), which saves the partials,
    // the arrival tickets and the merge, a chain of dependent memory round trips longer than the tiles it spares.
    uint64_t longest_rg = 0;
    for (int32_t i = 0; i < n_reqs; ++i) {
        uint64_t t = 0;
        for (int32_t sgi = seg_begin[i]; sgi < seg_begin[i + 1]; ++sgi) {
            uint32_t t0, nt;
            stream_part(sgi, &t0, &nt);
            t += (nt + T - 1) / T;
        }
        longest_rg = std::max(longest_rg, t);
    }
    const bool whole = A > 0 && rgs_with_tiles > 0 && rgs_with_tiles <= n_cta_stream && W <= 4 * n_cta_stream &&
                       longest_rg <= 24;
    Balancer bal(whole ? rgs_with_tiles : (C ? C : 1), A, W, rgs_with_tiles);
    bal.whole = whole;
    o->cta_begin[0] = 0;

    for (int32_t i = 0; i < n_reqs; ++i) {
        const int32_t s0 = seg_begin[i], s1 = seg_begin[i + 1];
        uint64_t rg_tiles = 0;
        bool has_shared = false;
        for (int32_t s = s0; s < s1; ++s) {
            uint32_t t0, nt;
            stream_part(s, &t0, &nt);
            rg_tiles += (nt + T - 1) / T;
            has_shared = has_shared || seg_cls[(size_t)s] >= 0;
        }
        for (int32_t g = 0; g < n_kv_heads; ++g) {
            const uint32_t rg = (uint32_t)i * (uint32_t)n_kv_heads + (uint32_t)g;
            const uint64_t rg_start = pos, rg_end = pos + rg_tiles;
            const uint32_t slot_first = next_slot;
            bool split = false;
            int32_t my_merge = -1;
            if (has_shared) {
                if (nm >= o->merges_cap) return CART_ERR_CAPACITY;
                my_merge = nm++;
                split = true;
                for (int32_t s = s0; s < s1; ++s) {
                    if (seg_cls[(size_t)s] < 0) continue;
                    const SharedClass &cl = classes[(size_t)seg_cls[(size_t)s]];
                    const uint32_t e = (uint32_t)seg_entry[(size_t)s];
                    const uint32_t m = (e - cl.reader_begin) / R;
                    const Combo &cb = combos[cl.first_combo + m * (uint32_t)n_kv_heads + (uint32_t)g];
                    o->reader_slot[(size_t)e * n_kv_heads + g] = next_slot;
                    o->reader_merge[(size_t)e * n_kv_heads + g] = (uint32_t)my_merge;
                    next_slot += cb.n_chunks;
                }
            }
            // skip segments that leave nothing in the stream
            int32_t s = s0;
            uint32_t seg_tok0 = 0, seg_ntok = 0;
            auto settle = [&]() {
                while (s < s1) {
                    stream_part(s, &seg_tok0, &seg_ntok);
                    if (seg_ntok > 0) break;
                    ++s;
                }
            };
            settle();
            uint64_t seg_tile = 0;  // tiles of segment s already handed out
            while (pos < rg_end) {
                // tiles of this row group that the block takes (the balancer may close the block first)
                const bool fresh = pos == rg_start;
                const uint64_t piece_tiles = bal.take(rg_end - pos, fresh);
                while (c < bal.c) o->cta_begin[++c] = (uint32_t)ni;
                const uint64_t piece_end = pos + piece_tiles;
                const bool direct = !has_shared && pos == rg_start && piece_end == rg_end;
                uint64_t want = piece_end - pos;
                bool first = true;
                while (want > 0) {
                    const uint64_t seg_tiles = (seg_ntok + T - 1) / T;
                    const uint64_t take = std::min(want, seg_tiles - seg_tile);
                    if (ni >= o->items_cap) return CART_ERR_CAPACITY;
                    cart_work_item &it = o->items[ni++];
                    const uint64_t tok0 = seg_tile * T;
                    const uint64_t tok1 = std::min<uint64_t>(seg_ntok, (seg_tile + take) * T);
                    it.flags = first ? CART_ITEM_BEGIN : 0u;
                    if (segs[s].flags & CART_SEG_PAGED) {
                        // a page holds one tile: the run starts (seg_tok0 + tok0) / T pages into the segment
                        it.k_row = segs[s].k_row + (uint32_t)((seg_tok0 + tok0) / T);
                        it.v_row = (uint32_t)g * segs[s].head_stride;
                        it.flags |= CART_ITEM_PAGED;
                    } else {
                        it.k_row = segs[s].k_row + (uint32_t)g * segs[s].head_stride + seg_tok0 + (uint32_t)tok0;
                        it.v_row = segs[s].v_row + (uint32_t)g * segs[s].head_stride + seg_tok0 + (uint32_t)tok0;
                    }
                    it.layer_stride = segs[s].layer_stride;
                    it.n_tok = (uint32_t)(tok1 - tok0);
                    it.row_group = rg;
                    if (s == s1 - 1 && tok1 == seg_ntok) it.flags |= CART_ITEM_TAIL;
                    if (segs[s].flags & CART_SEG_SUFFIX) it.flags |= CART_ITEM_SUFFIX;
                    it.slot = 0;
                    it.merge = 0;
                    first = false;
                    want -= take;
                    seg_tile += take;
                    if (seg_tile == seg_tiles) { ++s; seg_tile = 0; settle(); }
                }
                cart_work_item &last = o->items[ni - 1];
                last.flags |= CART_ITEM_END;
                if (direct) {
                    last.flags |= CART_ITEM_DIRECT;
                } else {
                    if (!split) {
                        if (nm >= o->merges_cap) return CART_ERR_CAPACITY;
                        my_merge = nm++;
                        split = true;
                    }
                    last.slot = next_slot++;
                    last.merge = (uint32_t)my_merge;
                }
                pos = piece_end;
                bal.commit(piece_tiles, fresh, pos < rg_end);
                while (c < bal.c) o->cta_begin[++c] = (uint32_t)ni;
            }
            if (split) {
                o->merges[my_merge].row_group = rg;
                o->merges[my_merge].slot_begin = slot_first;
                o->merges[my_merge].slot_end = next_slot;
                o->merges[my_merge].reserved = 0;
            }
        }
    }
    const uint64_t used = C ? (bal.block_has_work() ? bal.c + 1 : bal.c) : 0;
    for (uint64_t b = c; b < (uint64_t)n_cta; ++b) o->cta_begin[b + 1] = (uint32_t)ni;
    if ((int64_t)next_slot > (int64_t)o->slots_cap) return CART_ERR_CAPACITY;
    o->n_items = ni;
    o->n_merges = nm;
    o->n_cta_used = (int32_t)used;
    o->n_slots = (int32_t)next_slot;
    o->total_tiles = (int64_t)W;
    return CART_OK;
}

extern "C" cart_status cart_plan_build(const cart_plan_seg *segs, const int32_t *seg_begin,
                                       int32_t n_reqs, int32_t n_kv_heads, int32_t n_cta,
                                       int32_t tile_tokens, cart_work_item *items, int32_t items_cap,
                                       int32_t *n_items, uint32_t *cta_begin, cart_merge_item *merges,
                                       int32_t merges_cap, int32_t *n_merges, int32_t *n_cta_used,
                                       int32_t *n_slots, int64_t *total_tiles)
{
    if (!n_items || !n_merges || !n_cta_used || !n_slots || !total_tiles) return CART_ERR_INVALID_ARG;
    cart_plan_out o{};
    o.items = items;
    o.items_cap = items_cap;
    o.cta_begin = cta_begin;
    o.merges = merges;
    o.merges_cap = merges_cap;
    o.slots_cap = INT32_MAX;
    const cart_status st = cart_plan_build_shared(segs, seg_begin, n_reqs, n_kv_heads, 1, n_cta, tile_tokens, 0, 0, &o);
    if (st != CART_OK) return st;
    *n_items = o.n_items;
    *n_merges = o.n_merges;
    *n_cta_used = o.n_cta_used;
    *n_slots = o.n_slots;
    *total_tiles = o.total_tiles;
    return CART_OK;
}

extern "C" int32_t cart_plan_reusable(const int32_t *plan_len, const int32_t *cur_len, int32_t n_reqs,
                                      int32_t max_grow, int32_t *grow)
{
    if (!plan_len || !cur_len || !grow || n_reqs < 1 || max_grow < 0) return 0;
    const int64_t d = (int64_t)cur_len[0] - plan_len[0];
    if (d < 0 || d > max_grow) return 0;
    for (int32_t i = 0; i < n_reqs; ++i) {
        if ((int64_t)cur_len[i] - plan_len[i] != d) return 0;
        if (d > 0 && plan_len[i] < 1) return 0;
    }
    *grow = (int32_t)d;
    return 1;
}
