// Host-side work planner: see include/cart_plan.h for the contract.
#include <algorithm>
#include <cstdint>
#include <vector>

#include "cart_plan.h"

extern "C" cart_status cart_plan_build(const cart_plan_seg *segs, const int32_t *seg_begin,
                                       int32_t n_reqs, int32_t n_kv_heads, int32_t n_cta,
                                       int32_t tile_tokens, cart_work_item *items, int32_t items_cap,
                                       int32_t *n_items, uint32_t *cta_begin, cart_merge_item *merges,
                                       int32_t merges_cap, int32_t *n_merges, int32_t *n_cta_used,
                                       int32_t *n_slots, int64_t *total_tiles)
{
    if (!segs || !seg_begin || !items || !n_items || !cta_begin || !merges || !n_merges ||
        !n_cta_used || !n_slots || !total_tiles)
        return CART_ERR_INVALID_ARG;
    if (n_reqs < 1 || n_kv_heads < 1 || n_cta < 1 || tile_tokens < 1) return CART_ERR_INVALID_ARG;

    const uint64_t T = (uint64_t)tile_tokens;
    uint64_t tiles_per_head = 0; // tiles of one KV head summed over the batch
    for (int32_t i = 0; i < n_reqs; ++i) {
        uint64_t toks = 0;
        for (int32_t s = seg_begin[i]; s < seg_begin[i + 1]; ++s) {
            if (segs[s].n_tok == 0) return CART_ERR_INVALID_ARG;
            toks += segs[s].n_tok;
            tiles_per_head += (segs[s].n_tok + T - 1) / T;
        }
        if (toks == 0) return CART_ERR_EMPTY;
    }
    const uint64_t W = tiles_per_head * (uint64_t)n_kv_heads;
    const uint64_t C = std::min<uint64_t>((uint64_t)n_cta, W);

    int32_t ni = 0, nm = 0;
    uint32_t next_slot = 0;
    uint64_t pos = 0; // tiles handed out so far
    uint64_t c = 0;   // block being filled
    auto range_end = [&](uint64_t blk) { return ((blk + 1) * W) / C; };
    cta_begin[0] = 0;

    for (int32_t i = 0; i < n_reqs; ++i) {
        const int32_t s0 = seg_begin[i], s1 = seg_begin[i + 1];
        uint64_t rg_tiles = 0;
        for (int32_t s = s0; s < s1; ++s) rg_tiles += (segs[s].n_tok + T - 1) / T;
        for (int32_t g = 0; g < n_kv_heads; ++g) {
            const uint32_t rg = (uint32_t)i * (uint32_t)n_kv_heads + (uint32_t)g;
            const uint64_t rg_start = pos, rg_end = pos + rg_tiles;
            int32_t s = s0;        // segment under the cursor
            uint64_t seg_tile = 0; // tiles of segment s already handed out
            const uint32_t slot_first = next_slot;
            bool split = false;
            int32_t my_merge = -1;
            while (pos < rg_end) {
                const uint64_t piece_end = std::min(rg_end, range_end(c));
                const bool direct = (pos == rg_start && piece_end == rg_end);
                uint64_t want = piece_end - pos;
                bool first = true;
                while (want > 0) {
                    const uint64_t seg_tiles = (segs[s].n_tok + T - 1) / T;
                    const uint64_t take = std::min(want, seg_tiles - seg_tile);
                    if (ni >= items_cap) return CART_ERR_CAPACITY;
                    cart_work_item &it = items[ni++];
                    const uint64_t tok0 = seg_tile * T;
                    const uint64_t tok1 = std::min<uint64_t>(segs[s].n_tok, (seg_tile + take) * T);
                    it.k_row = segs[s].k_row + (uint32_t)g * segs[s].head_stride + (uint32_t)tok0;
                    it.v_row = segs[s].v_row + (uint32_t)g * segs[s].head_stride + (uint32_t)tok0;
                    it.layer_stride = segs[s].layer_stride;
                    it.n_tok = (uint32_t)(tok1 - tok0);
                    it.row_group = rg;
                    it.flags = first ? CART_ITEM_BEGIN : 0u;
                    it.slot = 0;
                    it.merge = 0;
                    first = false;
                    want -= take;
                    seg_tile += take;
                    if (seg_tile == seg_tiles) { ++s; seg_tile = 0; }
                }
                cart_work_item &last = items[ni - 1];
                last.flags |= CART_ITEM_END;
                if (direct) {
                    last.flags |= CART_ITEM_DIRECT;
                } else {
                    if (!split) {
                        if (nm >= merges_cap) return CART_ERR_CAPACITY;
                        my_merge = nm++;
                        split = true;
                    }
                    last.slot = next_slot++;
                    last.merge = (uint32_t)my_merge;
                }
                pos = piece_end;
                if (pos == range_end(c)) { ++c; cta_begin[c] = (uint32_t)ni; }
            }
            if (split) {
                merges[my_merge].row_group = rg;
                merges[my_merge].slot_begin = slot_first;
                merges[my_merge].slot_end = next_slot;
                merges[my_merge].reserved = 0;
            }
        }
    }
    for (uint64_t b = c; b < (uint64_t)n_cta; ++b) cta_begin[b + 1] = (uint32_t)ni;
    *n_items = ni;
    *n_merges = nm;
    *n_cta_used = (int32_t)C;
    *n_slots = (int32_t)next_slot;
    *total_tiles = (int64_t)W;
    return CART_OK;
}
