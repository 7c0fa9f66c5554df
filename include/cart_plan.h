/*
 * cart_plan.h -- the host-side work planner of libcart.so, exported so that it can be tested
 * without a device.  cart_decode_attention calls it once per (batch, lengths) and reuses the result
 * for every layer of a decode step.
 *
 * The paper gives no schedule (Sec. 3.3 only says a Cartridge is served like a cached prefix of
 * length p); this split is the library's own.  The KV cache of a (request, KV head) pair -- a "row
 * group": the G = Hq/Hkv query heads that read the same K/V (GQA) -- is the concatenation of its
 * segments (Cartridge parts in composition order, then the suffix; Sec. 3.2 layout).  Each segment
 * is cut into tiles of `tile_tokens` tokens (the last one ragged).  The tiles of all row groups,
 * laid end to end in batch order, are divided into `n_cta` contiguous, equal (+-1 tile) ranges, one
 * per persistent thread block.  Where a range boundary falls inside a row group, that row group is
 * "split": each block holding a piece writes a partial (o, lse) into its own slot and the block
 * that finishes last merges the pieces by log-sum-exp (softmax over a union of token sets, from
 * Eq. 1).  A row
 * group held entirely by one block is written directly.
 */
#ifndef CART_PLAN_H_
#define CART_PLAN_H_

#include <stdint.h>
#include "cart.h"

#ifdef __cplusplus
extern "C" {
#endif

/* One KV segment of a request, as rows of 128 bf16 (256 bytes) counted from the arena base. */
typedef struct {
    uint32_t k_row;        /* row of token 0, KV head 0, layer 0 (keys) */
    uint32_t v_row;        /* same for values */
    uint32_t head_stride;  /* rows between consecutive KV heads (p, or the suffix capacity) */
    uint32_t layer_stride; /* rows between consecutive layers (n_kv_heads * head_stride) */
    uint32_t n_tok;        /* tokens in the segment (> 0) */
    uint32_t flags;        /* CART_SEG_* */
} cart_plan_seg;

#define CART_SEG_SUFFIX 1u  /* the segment lies in a request's suffix buffer, which kernels write (append, extend,
                               fused decode step); a stored Cartridge is only ever written by copies */
#define CART_SEG_PAGED 2u   /* the segment is stored in pages of tile_tokens tokens (a paged suffix): k_row is the index
                               of the page that holds the segment's first token in the batch's page list (a device
                               array of page base rows), v_row is unused, head_stride = rows between consecutive KV
                               heads inside a page (2 * tile_tokens: the head's K rows, then its V rows), layer_stride =
                               rows between consecutive layers inside a page.  The segment starts on a page boundary. */

#define CART_ITEM_BEGIN 1u  /* first item of a row-group piece in this block: load q, reset state */
#define CART_ITEM_END 2u    /* last item of the piece: combine the warps' states and write */
#define CART_ITEM_DIRECT 4u /* the piece is the whole row group: write out / lse, not a partial */
#define CART_ITEM_TAIL 8u   /* the item ends with the last token of the request's cache (the token a fused
                               append + decode call writes before it attends) */
#define CART_ITEM_SUFFIX 16u /* the item's tiles lie in suffix storage (CART_SEG_SUFFIX): a kernel earlier on the
                               stream may have written them, so they are fetched only once those kernels are
                               known to be complete; Cartridge tiles may be fetched ahead of that */
#define CART_ITEM_PAGED 32u  /* the item's tiles are pages (CART_SEG_PAGED): k_row is the index of the first tile's
                               entry in the page list, v_row the row of the KV head's K block inside a page (its V
                               block follows tile_tokens rows later); tile j of the item lies in page k_row + j */

/* A run of consecutive tiles of one segment of one row group, processed by one block. */
typedef struct {
    uint32_t k_row;        /* first row of the run for layer 0 (KV head already applied) */
    uint32_t v_row;
    uint32_t layer_stride; /* add layer * layer_stride to both rows */
    uint32_t n_tok;        /* tokens in the run (> 0); only the last tile may be ragged */
    uint32_t row_group;    /* batch index * n_kv_heads + KV head */
    uint32_t flags;        /* CART_ITEM_* */
    uint32_t slot;         /* partial slot (meaningful with END and without DIRECT) */
    uint32_t merge;        /* index of the row group's cart_merge_item (same condition) */
} cart_work_item;

/* A split row group: its partials are slots slot_begin .. slot_end-1. */
typedef struct {
    uint32_t row_group;
    uint32_t slot_begin;
    uint32_t slot_end;
    uint32_t reserved;
} cart_merge_item;

/*
 * Builds the plan.  All pointers are host memory.
 *   segs, seg_begin   request i of the batch owns segs[seg_begin[i] .. seg_begin[i+1]-1], in cache
 *                     order; every request must own at least one token
 *   n_cta             persistent blocks available (>= 1)
 *   tile_tokens       tokens per tile (>= 1)
 *   items / items_cap work items, grouped by block; block c owns items[cta_begin[c] .. cta_begin[c+1]-1]
 *   cta_begin         [n_cta + 1]
 *   merges / merges_cap  one entry per split row group
 *   n_cta_used        blocks that received work (<= n_cta); blocks beyond it own no item
 *   n_slots           partial slots used
 *   total_tiles       tiles in the whole batch
 * Errors: INVALID_ARG, EMPTY (a request without tokens), CAPACITY (items_cap / merges_cap too small).
 */
CART_API cart_status cart_plan_build(const cart_plan_seg *segs, const int32_t *seg_begin, int32_t n_reqs,
                            int32_t n_kv_heads, int32_t n_cta, int32_t tile_tokens,
                            cart_work_item *items, int32_t items_cap, int32_t *n_items,
                            uint32_t *cta_begin, cart_merge_item *merges, int32_t merges_cap,
                            int32_t *n_merges, int32_t *n_cta_used, int32_t *n_slots,
                            int64_t *total_tiles);

/*
 * Shared segments.  When several requests of a batch attend to the same stored Cartridge (one
 * Cartridge serving many users, Sec. 1 and Sec. 3.3; members of a pool composed by many requests,
 * Sec. 5.4), its K/V tiles need not be streamed once per request: the query heads of all its readers
 * form the rows of one dense product per tile.  cart_plan_build_shared takes such segments out of the
 * per-request stream and describes them as "shared units" for a tensor-core kernel:
 *   - a segment is shared when at least share_min_readers requests of the batch hold it (same k_row,
 *     v_row and length) and it has at least one full tile of share_tile_tokens tokens;
 *   - its readers, in batch order, are cut into M-tiles of at most 128 / group requests (128 query
 *     rows: row i * group + h is head h of the M-tile's i-th reader);
 *   - only the full share_tile_tokens-token tiles are shared; the ragged tail (fewer tokens than one
 *     tile) stays in each reader's stream as a short segment;
 *   - the (segment, M-tile, KV head) tile runs, laid end to end, are divided into contiguous ranges,
 *     one per block, as the stream is; a range boundary inside a run cuts it into "chunks".
 * Every unit writes one partial (o, lse) per reader row group; the partial slots of a row group are
 * contiguous: first its shared chunks (segments in cache order, chunks in order), then its stream
 * pieces.  A row group with a shared part is never written directly: its cart_merge_item counts all
 * of its partials and whichever block delivers the last one merges them.
 */
typedef struct {
    uint32_t k_row;        /* first row of the run for layer 0 (KV head and token offset applied) */
    uint32_t v_row;
    uint32_t layer_stride; /* add layer * layer_stride to both rows */
    uint32_t n_tiles;      /* full tiles of share_tile_tokens tokens in the run (> 0) */
    uint32_t reader_begin; /* first entry of the M-tile in readers[] */
    uint32_t n_readers;    /* entries of the M-tile (1 .. 128 / group) */
    uint16_t kv_head;
    uint16_t flags;        /* CART_UNIT_*: CART_UNIT_SUFFIX = the run lies in suffix storage (see CART_ITEM_SUFFIX) */
    uint32_t chunk;        /* ordinal of the run among the runs of its (segment, M-tile, KV head) */
    /* Masked runs (CART_UNIT_MASKED; the planner does not emit them, the training forward builds them): row r of the
     * M-tile (token offset tr = r / group) sees the run's keys 0 .. limit with
     *     limit = tr < tr_hi ? min(lim_base + tr, lim_cap) : -1        (negative: the row sees nothing of the run)
     * so a causal run has lim_base = first row's token - run's first token, and a run every row sees whole but that
     * ends inside a tile has lim_base = lim_cap = its last key.  n_tiles then counts the ragged last tile too. */
    int32_t lim_base;
    int32_t lim_cap;
    uint32_t tr_hi;
    uint32_t reserved;     /* plans with chains: on a chain's first unit, how many units on the next chain begins (0: none follows
                              in the block); else 0 */
} cart_shared_unit;

#define CART_UNIT_SUFFIX 1u
#define CART_UNIT_MASKED 4u   /* see lim_base */
#define CART_UNIT_CONT 8u     /* the unit continues the M-tile of the unit before it in the same block: the softmax state
                                 and the accumulator carry over (same readers, same KV head) */
#define CART_UNIT_HOLD 16u    /* nothing is written at the unit's end: the next unit (CART_UNIT_CONT) goes on */
#define CART_UNIT_DIRECT 32u  /* the unit's end writes the rows' final bf16 output and lse (row i of reader j goes to
                                 query row readers[reader_begin + j]), not a partial: the chain covers the rows' whole
                                 caches */
#define CART_UNIT_PAGED 2u    /* the run lies in pages: k_row = index of its first page in the page list (a shared
                                 tile of share_tile_tokens tokens spans share_tile_tokens / tile_tokens consecutive
                                 entries), v_row = row of the KV head's K block inside a page, layer_stride as in
                                 CART_SEG_PAGED */

/* Capacities (in) and results (out) of cart_plan_build_shared; all arrays are host memory. */
typedef struct {
    /* stream part, as in cart_plan_build */
    cart_work_item *items;     int32_t items_cap;    int32_t n_items;
    uint32_t *cta_begin;       /* [n_cta + 1] */
    cart_merge_item *merges;   int32_t merges_cap;   int32_t n_merges;
    int32_t n_cta_used;        /* blocks of the stream kernel that received work (may be 0) */
    int32_t slots_cap;         /* partial slots available */
    int32_t n_slots;           /* partial slots used (shared + stream) */
    int64_t total_tiles;       /* stream tiles */
    int32_t piece_cost;        /* in: what starting a row-group piece costs a block, in tile times; the stream
                                  blocks are balanced by tiles + piece_cost * pieces (0: by tiles alone) */
    /* shared part */
    cart_shared_unit *units;   int32_t units_cap;    int32_t n_units;
    uint32_t *unit_cta_begin;  /* [n_cta + 1]: block c of the shared kernel owns units[unit_cta_begin[c] ..] */
    int32_t n_unit_cta_used;   /* blocks of the shared kernel that received work (0 = nothing shared) */
    uint32_t *readers;         int32_t readers_cap;  int32_t n_readers;  /* batch index per reader entry */
    uint32_t *reader_slot;     /* [readers_cap * n_kv_heads]: first slot of (entry, KV head); + unit.chunk */
    uint32_t *reader_merge;    /* [readers_cap * n_kv_heads]: merge item of (entry, KV head) */
    int64_t shared_tiles;      /* tile runs handed to the shared kernel, in share_tile_tokens tiles */
    int32_t unit_cost;         /* in: what a shared unit costs a block on top of its tiles, in tile times; the
                                  shared blocks are balanced by tiles + unit_cost * units (0: by tiles alone) */
    int32_t side_by_side;      /* in: 0 = the shared kernel and the stream kernel each get all n_cta blocks (they run
                                  one after the other); 1 = the n_cta blocks are divided between them so that both
                                  are resident at once (chosen from the two parts' estimated times); > 1 = the
                                  same with exactly this many blocks for the shared kernel (< n_cta) */
    int32_t n_shared_ctas;     /* out: blocks set aside for the shared kernel when running side by side (else 0) */
} cart_plan_out;

/*
 * Builds the stream plan and the shared units.  segs / seg_begin / n_reqs / n_kv_heads / n_cta /
 * tile_tokens as in cart_plan_build; group = query heads per KV head (1..8);
 * share_min_readers = 0 disables sharing (the result then equals cart_plan_build's);
 * share_tile_tokens is a multiple of tile_tokens.
 * Side by side (out->side_by_side): the tensor-core kernel is bound by latencies and barely touches HBM,
 * the stream kernel is bound by HBM bandwidth and loses little of it on three quarters of the SMs, so a
 * batch with both parts finishes sooner when the two kernels share the SMs than when each has all of
 * them in turn.  The division is chosen by minimising the larger of the two parts' estimated times.
 * If the partial slots the shared chunks need exceed slots_cap, the shared ranges are made longer
 * (fewer blocks, fewer chunks) until they fit; if they cannot fit, nothing is shared.
 * Errors: INVALID_ARG, EMPTY, CAPACITY (an output array is too small).
 */
CART_API cart_status cart_plan_build_shared(const cart_plan_seg *segs, const int32_t *seg_begin, int32_t n_reqs,
                                            int32_t n_kv_heads, int32_t group, int32_t n_cta, int32_t tile_tokens,
                                            int32_t share_min_readers, int32_t share_tile_tokens,
                                            cart_plan_out *out);

/*
 * Plan reuse across decode steps.  A plan built for a batch whose requests had suffix lengths
 * plan_len[i] stays usable while every request of the same batch has grown by the same number of
 * tokens d (each fused decode step appends one token to every request, Sec. 2.3): the kernels then
 * add d to the token count of every item marked CART_ITEM_TAIL, which only lengthens the last run of
 * every row group.  Returns 1 and writes d to *grow when cur_len[i] - plan_len[i] == d for all i with
 * 0 <= d <= max_grow, and, if d > 0, every plan_len[i] >= 1 (the tail item then lies in the suffix);
 * returns 0 otherwise (re-plan).  max_grow bounds how far the blocks' shares may drift apart.
 */
CART_API int32_t cart_plan_reusable(const int32_t *plan_len, const int32_t *cur_len, int32_t n_reqs,
                                    int32_t max_grow, int32_t *grow);

#ifdef __cplusplus
}
#endif
#endif /* CART_PLAN_H_ */
