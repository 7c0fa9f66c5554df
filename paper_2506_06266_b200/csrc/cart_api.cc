// Host side of libcart.so: handle tables, the arena allocator, plan caching and kernel launches.
// The contract of every entry point is stated in include/cart.h.
#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>
#include <string>
#include <vector>

#include "cart.h"
#include "cart_internal.h"

namespace {

using namespace cart;

constexpr int kMaxCta = 1024;   // upper bound on persistent blocks (device independent)
constexpr int kPlanSlots = 4;   // ring of uploaded plans
constexpr uint64_t kAlign = 256;
constexpr size_t kMaxTimedLaunches = 8192;

uint64_t round_up(uint64_t x, uint64_t a) { return (x + a - 1) / a * a; }

// A Cartridge is handed to the shared-segment kernel when at least this many requests of the batch
// hold it (and it has at least one full 128-token tile); below that its readers stream it one by one.
constexpr int kShareMinReaders = 4;
// What the planner charges a stream block for starting a row-group piece, in 64-token tile times.
constexpr int kPieceCostTiles = 3;
// What the planner charges a shared-segment block per unit on top of its tiles, in 128-token tile times.
constexpr int kUnitCostTiles = 4;
// A decode plan is kept while every request of the batch has grown by the same number of tokens, up to this
// many (the blocks' shares drift apart by one tile per 64 tokens of growth and tail item).
constexpr int kMaxGrowTokens = 192;

struct ScratchLayout {
    uint64_t status_off, tickets_off, plan_off, plan_slot_bytes, cta_begin_off, merges_off, items_off;
    // shared-segment part of a plan slot
    uint64_t shared_off, unit_cta_begin_off, readers_off, reader_slot_off, reader_merge_off, units_off;
    uint64_t pages_off;  // page list of the batch's paged suffixes (base row per page)
    uint64_t part_o_off, part_lse_off, total;
    int items_cap, slots_cap, merges_cap, units_cap, readers_cap, pages_cap;
};

ScratchLayout scratch_layout(const cart_config &c)
{
    ScratchLayout s{};
    const int parts = c.max_parts > 0 ? c.max_parts : 8;
    const int group = c.n_q_heads / c.n_kv_heads;
    const int row_groups = c.max_requests * c.n_kv_heads;
    // a row group owns at most parts + 2 segments (Cartridge parts, during prefill the shared head of the
    // suffix, and the suffix), and every block boundary cuts one item in two
    s.items_cap = row_groups * (parts + 2) + kMaxCta;
    // a row group with a shared part is always merged; the others only when a block boundary splits them
    s.merges_cap = row_groups + kMaxCta;
    // partial slots: stream pieces (one per row group with a shared part, two per block boundary) plus
    // the chunks of shared segments (the planner keeps them within what is left)
    s.slots_cap = 10 * row_groups + 2 * kMaxCta;
    s.readers_cap = c.max_requests * (parts + 1);  // + 1: the shared head of a suffix during prefill
    s.units_cap = s.readers_cap * c.n_kv_heads + kMaxCta;
    s.status_off = 0;          // the status word; the side-by-side flag sits 128 bytes behind it
    s.tickets_off = kAlign;  // one arrival counter per merge item, zero between launches
    s.plan_off = s.tickets_off + round_up((uint64_t)s.merges_cap * 4, kAlign);
    // one plan slot: [cta_begin][merges][items] [unit_cta_begin][readers][reader_slot][reader_merge][units]
    s.cta_begin_off = 0;
    s.merges_off = round_up((uint64_t)(kMaxCta + 1) * 4, kAlign);
    s.items_off = s.merges_off + round_up((uint64_t)s.merges_cap * sizeof(cart_merge_item), kAlign);
    s.shared_off = s.items_off + round_up((uint64_t)s.items_cap * sizeof(cart_work_item), kAlign);
    s.unit_cta_begin_off = s.shared_off;
    s.readers_off = s.unit_cta_begin_off + round_up((uint64_t)(kMaxCta + 1) * 4, kAlign);
    s.reader_slot_off = s.readers_off + round_up((uint64_t)s.readers_cap * 4, kAlign);
    s.reader_merge_off = s.reader_slot_off + round_up((uint64_t)s.readers_cap * c.n_kv_heads * 4, kAlign);
    s.units_off = s.reader_merge_off + round_up((uint64_t)s.readers_cap * c.n_kv_heads * 4, kAlign);
    s.pages_off = s.units_off + round_up((uint64_t)s.units_cap * sizeof(cart_shared_unit), kAlign);
    // (a function of the table sizes alone, like the rest of the layout: 16 k tokens of paged suffix per request
    //  on average, and room for a few very long ones)
    s.pages_cap = 256 * c.max_requests + 8192;
    s.plan_slot_bytes = s.pages_off + round_up((uint64_t)s.pages_cap * 4, kAlign);
    s.part_o_off = s.plan_off + (uint64_t)kPlanSlots * s.plan_slot_bytes;
    s.part_lse_off = s.part_o_off + round_up((uint64_t)s.slots_cap * group * kHeadDim * 4, kAlign);
    s.total = s.part_lse_off + round_up((uint64_t)s.slots_cap * kMaxGroup * 4, kAlign);
    return s;
}

cart_status check_config(const cart_config *c)
{
    if (!c) return CART_ERR_INVALID_ARG;
    if (c->n_layers < 1 || c->n_q_heads < 1 || c->n_kv_heads < 1 || c->max_requests < 1 ||
        c->max_cartridges < 1 || c->max_parts < 0 || !(c->softmax_scale >= 0.f))
        return CART_ERR_INVALID_ARG;
    if (c->head_dim != kHeadDim || c->n_q_heads % c->n_kv_heads != 0 ||
        c->n_q_heads / c->n_kv_heads > kMaxGroup)
        return CART_ERR_SHAPE;
    return CART_OK;
}

struct FreeBlock { uint64_t start, len; };  // in rows of 256 bytes

struct Cartridge {
    bool live = false;
    bool composed = false;
    int32_t p = 0;                 // tokens (sum over parts for a composition)
    uint64_t k_row = 0, v_row = 0; // registered only
    uint64_t alloc_start = 0, alloc_rows = 0;
    std::vector<int32_t> parts;    // composed: registered ids, flattened, in order
    int32_t refs = 0;              // open requests + compositions that hold it
    bool evicted = false;          // registered only: the arena space has been given back
};

struct Request {
    bool live = false;
    int32_t cart = CART_NONE;
    int32_t cap = 0;
    uint64_t k_row = 0, v_row = 0;
    uint64_t alloc_start = 0, alloc_rows = 0;
    std::vector<int32_t> len;  // per layer
    uint64_t stamp = 0;
    bool paged = false;            // the suffix lives in pages (base rows in `pages`); k_row / v_row / alloc_* unused
    std::vector<uint32_t> pages;
    bool evicted = false;          // the suffix is swapped out: no storage, lengths kept
    uint64_t list_stamp = 0;       // plan building: the request's pages are in the page list at list_base
    uint32_t list_base = 0;
};

struct PlanSlot {
    uint8_t *host = nullptr;   // pinned
    uint8_t *dev = nullptr;    // inside the arena scratch
    cudaEvent_t ev = nullptr;
    bool ev_recorded = false;
    bool valid = false;
    cudaStream_t last_stream = nullptr;
    std::vector<uint32_t> key;   // prefill plans: (request, suffix length, new tokens)
    std::vector<int32_t> reqs;   // decode plans: the batch and its suffix lengths when the plan was built
    std::vector<int32_t> lens;
    bool prefill = false;
    uint64_t epoch = 0;
    int32_t n_items = 0, n_merges = 0, n_cta_used = 0, n_slots = 0;
    int32_t n_units = 0, n_unit_cta_used = 0;
    // a plan of chains (prefill of a message, training forward): what it was built from and where its tables are
    bool chain = false;
    std::vector<uint64_t> chain_key;
    uint32_t chain_blocks = 0, chain_merges = 0;
    uint64_t chain_off[6] = {0, 0, 0, 0, 0, 0};
};

}  // namespace

struct cart_ctx {
    cart_config cfg{};
    ScratchLayout lay{};
    int group = 1;
    float scale = 0.f;
    int n_cta = 0;
    int share_min_readers = kShareMinReaders;
    int piece_cost = kPieceCostTiles;
    int max_grow = kMaxGrowTokens;
    int side_by_side = 1;        // shared and stream kernel share the SMs (0: one after the other; > 1: blocks for the shared kernel)
    int prefill_split = -1;      // pieces a short message's chains are cut into along the keys (-1: chosen per call; 0: never)
    bool plan_only = false;      // decode_impl stops after the plan (cart_graph_begin)
    // a recorded decode loop (cart_graph_begin .. cart_graph_end): its batch, the ring buffer of its plan, its steps
    bool graph_active = false;
    std::vector<int32_t> graph_reqs;
    int graph_slot = -1;
    int32_t graph_max_steps = 0;
    uint64_t plans_built = 0;
    uint64_t n_rows = 0;
    alignas(64) CUtensorMap tmap;
    alignas(64) CUtensorMap tmap_edge;
    void *encode_fn = nullptr;  // cuTensorMapEncodeTiled
    std::vector<FreeBlock> free_list;
    std::vector<Cartridge> carts;
    std::vector<Request> reqs;
    PlanSlot slots[kPlanSlots];
    int cur_slot = -1;
    uint64_t epoch = 1;
    uint64_t stamp = 0;
    uint64_t list_stamp = 0;
    uint64_t launches = 0;
    std::vector<cart_plan_seg> seg_tmp;
    std::vector<int32_t> head_tmp;
    std::vector<int32_t> seg_begin_tmp;
    std::vector<uint32_t> key_tmp;
    std::vector<int32_t> len_tmp;
    std::vector<uint64_t> chain_key_tmp;
    std::vector<cart_shared_unit> unit_tmp;
    std::vector<uint32_t> piece_tmp;
    bool timing = false;
    std::vector<cudaEvent_t> ev_pool;  // pairs: start, stop
    size_t ev_used = 0;
    char err[256] = {0};
};

namespace {

struct ChainPart { uint64_t k_row, v_row; uint32_t p; };
struct ChainStrand { uint64_t k_row, v_row; uint32_t cap, len, row_begin, n_rows, key_first; };
cart_status launch_chains(cart_ctx *ctx, int32_t layer, const std::vector<ChainPart> &parts, const std::vector<ChainStrand> &strands,
                          uint32_t T, const void *q, void *out, float *lse, cudaStream_t s, uint32_t n_split = 1);

cart_status fail(cart_ctx *ctx, cart_status st, const char *fmt, ...)
{
    if (ctx) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(ctx->err, sizeof ctx->err, fmt, ap);
        va_end(ap);
    }
    return st;
}

#define CART_CUDA(ctx, call)                                                                        \
    do {                                                                                            \
        cudaError_t e_ = (call);                                                                    \
        if (e_ != cudaSuccess)                                                                      \
            return fail(ctx, CART_ERR_CUDA, "%s failed: %s", #call, cudaGetErrorString(e_));        \
    } while (0)

bool arena_alloc(cart_ctx *ctx, uint64_t rows, uint64_t *start)
{
    for (size_t i = 0; i < ctx->free_list.size(); ++i) {
        FreeBlock &b = ctx->free_list[i];
        if (b.len >= rows) {
            *start = b.start;
            b.start += rows;
            b.len -= rows;
            if (b.len == 0) ctx->free_list.erase(ctx->free_list.begin() + (long)i);
            return true;
        }
    }
    return false;
}

void arena_free(cart_ctx *ctx, uint64_t start, uint64_t rows)
{
    if (rows == 0) return;
    auto &fl = ctx->free_list;
    size_t i = 0;
    while (i < fl.size() && fl[i].start < start) ++i;
    fl.insert(fl.begin() + (long)i, FreeBlock{start, rows});
    if (i + 1 < fl.size() && fl[i].start + fl[i].len == fl[i + 1].start) {
        fl[i].len += fl[i + 1].len;
        fl.erase(fl.begin() + (long)i + 1);
    }
    if (i > 0 && fl[i - 1].start + fl[i - 1].len == fl[i].start) {
        fl[i - 1].len += fl[i].len;
        fl.erase(fl.begin() + (long)i);
    }
}

bool aligned16(const void *p) { return p && (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

Cartridge *get_cart(cart_ctx *ctx, cart_id id)
{
    if (id < 0 || (size_t)id >= ctx->carts.size() || !ctx->carts[(size_t)id].live) return nullptr;
    return &ctx->carts[(size_t)id];
}

Request *get_req(cart_ctx *ctx, cart_req r)
{
    if (r < 0 || (size_t)r >= ctx->reqs.size() || !ctx->reqs[(size_t)r].live) return nullptr;
    return &ctx->reqs[(size_t)r];
}

uint8_t *arena_ptr(cart_ctx *ctx, uint64_t row) { return static_cast<uint8_t *>(ctx->cfg.arena) + row * kRowBytes; }

// A page holds kTileTokens tokens of a request for every layer and KV head: [layer][KV head][K rows, V rows].
uint64_t page_rows(const cart_ctx *ctx) { return (uint64_t)ctx->cfg.n_layers * ctx->cfg.n_kv_heads * 2 * kTileTokens; }
// Row of token `pos` of (layer, KV head 0) in a paged suffix: K rows; the V rows are kTileTokens further on, the
// next KV head 2 * kTileTokens.
uint64_t paged_row(const cart_ctx *ctx, const Request &r, int32_t layer, int32_t pos)
{
    return (uint64_t)r.pages[(size_t)(pos / kTileTokens)] + (uint64_t)layer * ctx->cfg.n_kv_heads * 2 * kTileTokens +
           (uint64_t)(pos % kTileTokens);
}
// Takes pages until the paged request holds at least `tokens` tokens.  False: the arena is full (pages taken so
// far are kept).  A new page changes the page list, so cached plans are dropped.
bool grow_pages(cart_ctx *ctx, Request &r, int64_t tokens)
{
    while ((int64_t)r.cap < tokens) {
        uint64_t start = 0;
        if (!arena_alloc(ctx, page_rows(ctx), &start)) return false;
        r.pages.push_back((uint32_t)start);
        r.cap += kTileTokens;
        ++ctx->epoch;
    }
    return true;
}
void drop_storage(cart_ctx *ctx, Request &r)
{
    if (r.paged) {
        for (uint32_t pg : r.pages) arena_free(ctx, pg, page_rows(ctx));
        r.pages.clear();
    } else if (r.alloc_rows > 0) {
        arena_free(ctx, r.alloc_start, r.alloc_rows);
    }
    r.alloc_rows = 0;
}
// Does a request that is resident attend to registered Cartridge `id`?
bool cartridge_has_active_reader(const cart_ctx *ctx, int32_t id)
{
    for (const Request &r : ctx->reqs) {
        if (!r.live || r.evicted || r.cart == CART_NONE) continue;
        const Cartridge &c = ctx->carts[(size_t)r.cart];
        if (r.cart == id) return true;
        if (c.composed)
            for (int32_t b : c.parts)
                if (b == id) return true;
    }
    return false;
}
// The first evicted registered Cartridge a request attends to, or -1.
int32_t evicted_part(const cart_ctx *ctx, const Request &r)
{
    if (r.cart == CART_NONE) return -1;
    const Cartridge &c = ctx->carts[(size_t)r.cart];
    if (!c.composed) return c.evicted ? r.cart : -1;
    for (int32_t b : c.parts)
        if (ctx->carts[(size_t)b].evicted) return b;
    return -1;
}

typedef CUresult (*EncodeFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                             const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                             CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

cart_status encode_tensor_map(cart_ctx *ctx)
{
    void *fn = nullptr;
    cudaDriverEntryPointQueryResult qres;
    CART_CUDA(ctx, cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
    if (!fn || qres != cudaDriverEntryPointSuccess)
        return fail(ctx, CART_ERR_CUDA, "the driver does not provide cuTensorMapEncodeTiled");
    ctx->encode_fn = fn;
    // The whole arena as a matrix of rows of 128 bf16; a KV tile is 64 consecutive rows, fetched as
    // two boxes of 64 rows x 64 elements (128 bytes, the widest row a 128-byte swizzle allows).
    const cuuint64_t gdim[2] = {(cuuint64_t)kHeadDim, (cuuint64_t)ctx->n_rows};
    const cuuint64_t gstride[1] = {(cuuint64_t)kRowBytes};
    const cuuint32_t box[2] = {64u, (cuuint32_t)kTileTokens};
    const cuuint32_t estride[2] = {1u, 1u};
    CUresult r = reinterpret_cast<EncodeFn>(fn)(&ctx->tmap, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, ctx->cfg.arena,
                                                gdim, gstride, box, estride, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                                CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                                CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(ctx, CART_ERR_CUDA, "cuTensorMapEncodeTiled failed with code %d", (int)r);
    // The same matrix in smaller boxes: a ragged last tile of a segment is fetched only as far as it has tokens.
    const cuuint32_t edge_box[2] = {64u, (cuuint32_t)kEdgeBoxRows};
    r = reinterpret_cast<EncodeFn>(fn)(&ctx->tmap_edge, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, ctx->cfg.arena, gdim,
                                       gstride, edge_box, estride, CU_TENSOR_MAP_INTERLEAVE_NONE,
                                       CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                                       CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(ctx, CART_ERR_CUDA, "cuTensorMapEncodeTiled (edge) failed with code %d", (int)r);
    return CART_OK;
}

}  // namespace

extern "C" {

const char *cart_status_string(cart_status s)
{
    switch (s) {
    case CART_OK: return "CART_OK";
    case CART_ERR_INVALID_ARG: return "CART_ERR_INVALID_ARG";
    case CART_ERR_SHAPE: return "CART_ERR_SHAPE";
    case CART_ERR_BAD_HANDLE: return "CART_ERR_BAD_HANDLE";
    case CART_ERR_CAPACITY: return "CART_ERR_CAPACITY";
    case CART_ERR_OOM: return "CART_ERR_OOM";
    case CART_ERR_EMPTY: return "CART_ERR_EMPTY";
    case CART_ERR_IN_USE: return "CART_ERR_IN_USE";
    case CART_ERR_CUDA: return "CART_ERR_CUDA";
    case CART_ERR_TIMEOUT: return "CART_ERR_TIMEOUT";
    case CART_ERR_EVICTED: return "CART_ERR_EVICTED";
    }
    return "CART_ERR_UNKNOWN";
}

const char *cart_last_error(const cart_ctx *ctx) { return ctx ? ctx->err : "no context"; }

uint64_t cart_launch_count(const cart_ctx *ctx) { return ctx ? ctx->launches : 0; }

uint64_t cart_plan_count(const cart_ctx *ctx) { return ctx ? ctx->plans_built : 0; }

cart_status cart_scratch_bytes(const cart_config *cfg, uint64_t *out_bytes)
{
    if (!out_bytes) return CART_ERR_INVALID_ARG;
    cart_status st = check_config(cfg);
    if (st != CART_OK) return st;
    *out_bytes = scratch_layout(*cfg).total;
    return CART_OK;
}

cart_status cart_create(const cart_config *cfg, cart_ctx **out)
{
    if (!out) return CART_ERR_INVALID_ARG;
    cart_status st = check_config(cfg);
    if (st != CART_OK) return st;
    if (!cfg->arena || (reinterpret_cast<uintptr_t>(cfg->arena) & (kAlign - 1)) != 0 || cfg->device < 0)
        return CART_ERR_INVALID_ARG;
    const ScratchLayout lay = scratch_layout(*cfg);
    if (cfg->arena_bytes < lay.total + kRowBytes) return CART_ERR_OOM;
    if (cfg->arena_bytes / kRowBytes >= (1ull << 31)) return CART_ERR_INVALID_ARG;

    cart_ctx *ctx = new (std::nothrow) cart_ctx();
    if (!ctx) return CART_ERR_OOM;
    ctx->cfg = *cfg;
    if (ctx->cfg.max_parts == 0) ctx->cfg.max_parts = 8;
    ctx->lay = lay;
    ctx->group = cfg->n_q_heads / cfg->n_kv_heads;
    ctx->scale = cfg->softmax_scale > 0.f ? cfg->softmax_scale : 1.0f / std::sqrt((float)cfg->head_dim);
    ctx->n_rows = cfg->arena_bytes / kRowBytes;

    auto bail = [&](cart_status s) {
        for (auto &sl : ctx->slots) {
            if (sl.host) cudaFreeHost(sl.host);
            if (sl.ev) cudaEventDestroy(sl.ev);
        }
        delete ctx;
        return s;
    };
    cudaError_t e = cudaSetDevice(cfg->device);
    if (e != cudaSuccess) return bail(CART_ERR_CUDA);
    int sms = 0;
    e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, cfg->device);
    if (e != cudaSuccess || sms < 1) return bail(CART_ERR_CUDA);
    ctx->n_cta = std::min(sms, kMaxCta);
    if (prepare_kernels() != cudaSuccess || prepare_shared_kernel() != cudaSuccess ||
        prepare_train_kernels() != cudaSuccess)
        return bail(CART_ERR_CUDA);
    if (encode_tensor_map(ctx) != CART_OK) return bail(CART_ERR_CUDA);
    for (int i = 0; i < kPlanSlots; ++i) {
        PlanSlot &sl = ctx->slots[i];
        if (cudaHostAlloc(reinterpret_cast<void **>(&sl.host), lay.plan_slot_bytes, cudaHostAllocDefault) != cudaSuccess)
            return bail(CART_ERR_CUDA);
        if (cudaEventCreateWithFlags(&sl.ev, cudaEventDisableTiming) != cudaSuccess) return bail(CART_ERR_CUDA);
        sl.dev = static_cast<uint8_t *>(cfg->arena) + lay.plan_off + (uint64_t)i * lay.plan_slot_bytes;
    }
    if (cudaMemset(static_cast<uint8_t *>(cfg->arena) + lay.status_off, 0, lay.plan_off) != cudaSuccess)
        return bail(CART_ERR_CUDA);

    const uint64_t first_row = lay.total / kRowBytes;
    ctx->free_list.push_back(FreeBlock{first_row, ctx->n_rows - first_row});
    ctx->carts.resize((size_t)cfg->max_cartridges);
    ctx->reqs.resize((size_t)cfg->max_requests);
    *out = ctx;
    return CART_OK;
}

cart_status cart_destroy(cart_ctx *ctx)
{
    if (!ctx) return CART_OK;
    cudaSetDevice(ctx->cfg.device);
    cudaDeviceSynchronize();
    for (auto &sl : ctx->slots) {
        if (sl.host) cudaFreeHost(sl.host);
        if (sl.ev) cudaEventDestroy(sl.ev);
    }
    for (cudaEvent_t e : ctx->ev_pool) cudaEventDestroy(e);
    delete ctx;
    return CART_OK;
}

cart_status cart_set_timing(cart_ctx *ctx, int32_t enable)
{
    if (!ctx) return CART_ERR_INVALID_ARG;
    ctx->timing = enable != 0;
    return CART_OK;
}

cart_status cart_set_share_min_readers(cart_ctx *ctx, int32_t min_readers)
{
    if (!ctx) return CART_ERR_INVALID_ARG;
    if (min_readers < 0) return fail(ctx, CART_ERR_INVALID_ARG, "share_min_readers: negative");
    ctx->share_min_readers = min_readers;
    ++ctx->epoch;  // cached plans were built under the old policy
    return CART_OK;
}

cart_status cart_set_piece_cost(cart_ctx *ctx, int32_t tiles)
{
    if (!ctx) return CART_ERR_INVALID_ARG;
    if (tiles < 0 || tiles > 64) return fail(ctx, CART_ERR_INVALID_ARG, "piece_cost: out of range");
    ctx->piece_cost = tiles;
    ++ctx->epoch;
    return CART_OK;
}

cart_status cart_set_side_by_side(cart_ctx *ctx, int32_t mode)
{
    if (!ctx) return CART_ERR_INVALID_ARG;
    if (mode < 0 || mode >= ctx->n_cta) return fail(ctx, CART_ERR_INVALID_ARG, "side_by_side: out of range");
    ctx->side_by_side = mode;
    ++ctx->epoch;
    return CART_OK;
}

cart_status cart_set_prefill_split(cart_ctx *ctx, int32_t pieces)
{
    if (!ctx) return CART_ERR_INVALID_ARG;
    if (pieces < -1 || pieces > 64) return fail(ctx, CART_ERR_INVALID_ARG, "prefill_split: out of range");
    ctx->prefill_split = pieces;
    return CART_OK;
}

cart_status cart_set_plan_reuse(cart_ctx *ctx, int32_t max_grow_tokens)
{
    if (!ctx) return CART_ERR_INVALID_ARG;
    if (max_grow_tokens < 0 || max_grow_tokens > (1 << 20))
        return fail(ctx, CART_ERR_INVALID_ARG, "plan_reuse: out of range");
    ctx->max_grow = max_grow_tokens;
    return CART_OK;
}

cart_status cart_get_timing(cart_ctx *ctx, double *total_ms, uint64_t *n_launches)
{
    if (!ctx) return CART_ERR_INVALID_ARG;
    if (!total_ms || !n_launches) return fail(ctx, CART_ERR_INVALID_ARG, "get_timing: null out");
    double sum = 0.0;
    for (size_t i = 0; i + 1 < ctx->ev_used; i += 2) {
        CART_CUDA(ctx, cudaEventSynchronize(ctx->ev_pool[i + 1]));
        float ms = 0.f;
        CART_CUDA(ctx, cudaEventElapsedTime(&ms, ctx->ev_pool[i], ctx->ev_pool[i + 1]));
        sum += (double)ms;
    }
    *total_ms = sum;
    *n_launches = ctx->ev_used / 2;
    ctx->ev_used = 0;
    return CART_OK;
}

cart_status cart_register_cartridge(cart_ctx *ctx, const void *k, const void *v, int32_t p, void *stream,
                                    cart_id *out)
{
    if (!ctx) return CART_ERR_INVALID_ARG;
    if (!out || !aligned16(k) || !aligned16(v) || p < 1)
        return fail(ctx, CART_ERR_INVALID_ARG, "register: null/misaligned pointer or p < 1");
    int32_t id = -1;
    for (size_t i = 0; i < ctx->carts.size(); ++i)
        if (!ctx->carts[i].live) { id = (int32_t)i; break; }
    if (id < 0) return fail(ctx, CART_ERR_CAPACITY, "register: Cartridge table full (%d)", ctx->cfg.max_cartridges);
    const uint64_t rows_one = (uint64_t)ctx->cfg.n_layers * ctx->cfg.n_kv_heads * (uint64_t)p;
    uint64_t start = 0;
    if (!arena_alloc(ctx, 2 * rows_one, &start))
        return fail(ctx, CART_ERR_OOM, "register: arena has no room for %llu bytes",
                    (unsigned long long)(2 * rows_one * kRowBytes));
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemcpyAsync(arena_ptr(ctx, start), k, rows_one * kRowBytes, cudaMemcpyDefault, s);
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(arena_ptr(ctx, start + rows_one), v, rows_one * kRowBytes, cudaMemcpyDefault, s);
    if (e != cudaSuccess) {
        arena_free(ctx, start, 2 * rows_one);
        return fail(ctx, CART_ERR_CUDA, "register: copy failed: %s", cudaGetErrorString(e));
    }
    Cartridge &c = ctx->carts[(size_t)id];
    c = Cartridge();
    c.live = true;
    c.p = p;
    c.k_row = start;
    c.v_row = start + rows_one;
    c.alloc_start = start;
    c.alloc_rows = 2 * rows_one;
    ++ctx->epoch;
    *out = id;
    return CART_OK;
}

cart_status cart_compose(cart_ctx *ctx, const cart_id *parts, int32_t n_parts, cart_id *out)
{
    if (!ctx) return CART_ERR_INVALID_ARG;
    if (!parts || !out || n_parts < 1) return fail(ctx, CART_ERR_INVALID_ARG, "compose: no parts");
    std::vector<int32_t> flat;
    int64_t total = 0;
    for (int32_t i = 0; i < n_parts; ++i) {
        Cartridge *c = get_cart(ctx, parts[i]);
        if (!c) return fail(ctx, CART_ERR_BAD_HANDLE, "compose: part %d is not a live Cartridge", i);
        if (c->composed) flat.insert(flat.end(), c->parts.begin(), c->parts.end());
        else flat.push_back(parts[i]);
        total += c->p;
    }
    if ((int32_t)flat.size() > ctx->cfg.max_parts)
        return fail(ctx, CART_ERR_CAPACITY, "compose: %d parts exceed max_parts = %d", (int)flat.size(), ctx->cfg.max_parts);
    if (total > INT32_MAX) return fail(ctx, CART_ERR_CAPACITY, "compose: too many tokens");
    int32_t id = -1;
    for (size_t i = 0; i < ctx->carts.size(); ++i)
        if (!ctx->carts[i].live) { id = (int32_t)i; break; }
    if (id < 0) return fail(ctx, CART_ERR_CAPACITY, "compose: Cartridge table full");
    for (int32_t b : flat) ++ctx->carts[(size_t)b].refs;
    Cartridge &c = ctx->carts[(size_t)id];
    c = Cartridge();
    c.live = true;
    c.composed = true;
    c.p = (int32_t)total;
    c.parts = flat;
    ++ctx->epoch;
    *out = id;
    return CART_OK;
}

cart_status cart_release_cartridge(cart_ctx *ctx, cart_id id)
{
    if (!ctx) return CART_ERR_INVALID_ARG;
    Cartridge *c = get_cart(ctx, id);
    if (!c) return fail(ctx, CART_ERR_BAD_HANDLE, "release: not a live Cartridge");
    if (c->refs > 0) return fail(ctx, CART_ERR_IN_USE, "release: %d users still hold the Cartridge", c->refs);
    if (c->composed) {
        for (int32_t b : c->parts) --ctx->carts[(size_t)b].refs;
    } else if (!c->evicted) {
        arena_free(ctx, c->alloc_start, c->alloc_rows);
    }
    *c = Cartridge();
    ++ctx->epoch;
    return CART_OK;
}

}  // extern "C"

namespace {
cart_status open_impl(cart_ctx *ctx, cart_id cartridge, int32_t suffix_capacity, bool paged, cart_req *out)
{
    if (!ctx) return CART_ERR_INVALID_ARG;
    if (!out || suffix_capacity < 0) return fail(ctx, CART_ERR_INVALID_ARG, "open: bad argument");
    if (cartridge != CART_NONE && !get_cart(ctx, cartridge))
        return fail(ctx, CART_ERR_BAD_HANDLE, "open: not a live Cartridge");
    int32_t id = -1;
    for (size_t i = 0; i < ctx->reqs.size(); ++i)
        if (!ctx->reqs[i].live) { id = (int32_t)i; break; }
    if (id < 0) return fail(ctx, CART_ERR_CAPACITY, "open: request table full (%d)", ctx->cfg.max_requests);
    const int64_t cap = ((int64_t)suffix_capacity + kTileTokens - 1) / kTileTokens * kTileTokens;
    Request &r = ctx->reqs[(size_t)id];
    if (paged) {
        r = Request();
        r.paged = true;
        if (!grow_pages(ctx, r, cap)) {
            drop_storage(ctx, r);
            r = Request();
            return fail(ctx, CART_ERR_OOM, "open: arena has no room for %lld tokens of pages", (long long)cap);
        }
    } else {
        const uint64_t rows_one = (uint64_t)ctx->cfg.n_layers * ctx->cfg.n_kv_heads * (uint64_t)cap;
        uint64_t start = 0;
        if (rows_one > 0 && !arena_alloc(ctx, 2 * rows_one, &start))
            return fail(ctx, CART_ERR_OOM, "open: arena has no room for a suffix of %lld tokens", (long long)cap);
        r = Request();
        r.cap = (int32_t)cap;
        r.k_row = start;
        r.v_row = start + rows_one;
        r.alloc_start = start;
        r.alloc_rows = 2 * rows_one;
    }
    r.live = true;
    r.cart = cartridge;
    r.len.assign((size_t)ctx->cfg.n_layers, 0);
    if (cartridge != CART_NONE) ++ctx->carts[(size_t)cartridge].refs;
    ++ctx->epoch;
    *out = id;
    return CART_OK;
}
}  // namespace

extern "C" {

cart_status cart_request_open(cart_ctx *ctx, cart_id cartridge, int32_t suffix_capacity, cart_req *out)
{
    return open_impl(ctx, cartridge, suffix_capacity, false, out);
}

cart_status cart_request_open_paged(cart_ctx *ctx, cart_id cartridge, int32_t initial_capacity, cart_req *out)
{
    return open_impl(ctx, cartridge, initial_capacity, true, out);
}

cart_status cart_request_reserve(cart_ctx *ctx, cart_req req, int32_t suffix_capacity, void *stream)
{
    if (!ctx) return CART_ERR_INVALID_ARG;
    Request *r = get_req(ctx, req);
    if (!r) return fail(ctx, CART_ERR_BAD_HANDLE, "reserve: not an open request");
    if (suffix_capacity < 0) return fail(ctx, CART_ERR_INVALID_ARG, "reserve: negative capacity");
    if (r->evicted) return fail(ctx, CART_ERR_EVICTED, "reserve: the request is swapped out");
    const int64_t cap = ((int64_t)suffix_capacity + kTileTokens - 1) / kTileTokens * kTileTokens;
    if (cap <= r->cap) return CART_OK;  // a buffer never shrinks
    if (r->paged) {
        // pages instead of a copy; on failure the pages taken by this call go back
        const size_t had = r->pages.size();
        if (!grow_pages(ctx, *r, cap)) {
            while (r->pages.size() > had) {
                arena_free(ctx, r->pages.back(), page_rows(ctx));
                r->pages.pop_back();
                r->cap -= kTileTokens;
            }
            return fail(ctx, CART_ERR_OOM, "reserve: arena has no room for %lld tokens of pages", (long long)cap);
        }
        return CART_OK;
    }
    const uint64_t heads = (uint64_t)ctx->cfg.n_layers * ctx->cfg.n_kv_heads;
    const uint64_t rows_one = heads * (uint64_t)cap;
    uint64_t start = 0;
    if (!arena_alloc(ctx, 2 * rows_one, &start))
        return fail(ctx, CART_ERR_OOM, "reserve: arena has no room for a suffix of %lld tokens", (long long)cap);
    int32_t longest = 0;
    for (int32_t l : r->len) longest = std::max(longest, l);
    if (longest > 0) {
        // every (layer, KV head) keeps its tokens in one run: old runs are r->cap rows apart, new ones cap rows
        cudaStream_t s = static_cast<cudaStream_t>(stream);
        cudaError_t e = cudaMemcpy2DAsync(arena_ptr(ctx, start), (size_t)cap * kRowBytes, arena_ptr(ctx, r->k_row),
                                          (size_t)r->cap * kRowBytes, (size_t)longest * kRowBytes, heads,
                                          cudaMemcpyDeviceToDevice, s);
        if (e == cudaSuccess)
            e = cudaMemcpy2DAsync(arena_ptr(ctx, start + rows_one), (size_t)cap * kRowBytes, arena_ptr(ctx, r->v_row),
                                  (size_t)r->cap * kRowBytes, (size_t)longest * kRowBytes, heads,
                                  cudaMemcpyDeviceToDevice, s);
        if (e != cudaSuccess) {
            arena_free(ctx, start, 2 * rows_one);
            return fail(ctx, CART_ERR_CUDA, "reserve: copy failed: %s", cudaGetErrorString(e));
        }
    }
    if (r->alloc_rows > 0) arena_free(ctx, r->alloc_start, r->alloc_rows);
    r->cap = (int32_t)cap;
    r->k_row = start;
    r->v_row = start + rows_one;
    r->alloc_start = start;
    r->alloc_rows = 2 * rows_one;
    ++ctx->epoch;  // cached plans address the old buffer
    return CART_OK;
}

cart_status cart_request_close(cart_ctx *ctx, cart_req req)
{
    if (!ctx) return CART_ERR_INVALID_ARG;
    Request *r = get_req(ctx, req);
    if (!r) return fail(ctx, CART_ERR_BAD_HANDLE, "close: not an open request");
    if (r->cart != CART_NONE) --ctx->carts[(size_t)r->cart].refs;
    drop_storage(ctx, *r);
    *r = Request();
    ++ctx->epoch;
    return CART_OK;
}

}  // extern "C"

namespace {
// Copies the first n tokens of every (layer, KV head) run of a request's suffix to (out = true) or from a dense
// [L][Hkv][n][128] pair of buffers.  A paged suffix moves page by page: inside a page the (layer, KV head) blocks of
// K (and of V) are 2 * kTileTokens rows apart.
cart_status swap_copy(cart_ctx *ctx, const Request &r, void *k_buf, void *v_buf, int32_t n, bool out, cudaStream_t s)
{
    const uint64_t heads = (uint64_t)ctx->cfg.n_layers * ctx->cfg.n_kv_heads;
    const size_t dense_pitch = (size_t)n * kRowBytes;
    auto copy2d = [&](void *dense, size_t dense_off, uint64_t arena_row, size_t arena_pitch, size_t width) -> cudaError_t {
        uint8_t *d = static_cast<uint8_t *>(dense) + dense_off;
        uint8_t *a = arena_ptr(ctx, arena_row);
        return out ? cudaMemcpy2DAsync(d, dense_pitch, a, arena_pitch, width, heads, cudaMemcpyDefault, s)
                   : cudaMemcpy2DAsync(a, arena_pitch, d, dense_pitch, width, heads, cudaMemcpyDefault, s);
    };
    if (r.paged) {
        for (int32_t t0 = 0; t0 < n; t0 += kTileTokens) {
            const size_t width = (size_t)std::min(kTileTokens, n - t0) * kRowBytes;
            const uint64_t pg = r.pages[(size_t)(t0 / kTileTokens)];
            CART_CUDA(ctx, copy2d(k_buf, (size_t)t0 * kRowBytes, pg, 2 * kTileTokens * kRowBytes, width));
            CART_CUDA(ctx, copy2d(v_buf, (size_t)t0 * kRowBytes, pg + kTileTokens, 2 * kTileTokens * kRowBytes, width));
        }
    } else {
        CART_CUDA(ctx, copy2d(k_buf, 0, r.k_row, (size_t)r.cap * kRowBytes, dense_pitch));
        CART_CUDA(ctx, copy2d(v_buf, 0, r.v_row, (size_t)r.cap * kRowBytes, dense_pitch));
    }
    return CART_OK;
}
}  // namespace

extern "C" {

cart_status cart_evict_request(cart_ctx *ctx, cart_req req, void *k_out, void *v_out, int32_t *n_tokens_out, void *stream)
{
    if (!ctx) return CART_ERR_INVALID_ARG;
    Request *r = get_req(ctx, req);
    if (!r) return fail(ctx, CART_ERR_BAD_HANDLE, "evict: not an open request");
    if (!n_tokens_out) return fail(ctx, CART_ERR_INVALID_ARG, "evict: null n_tokens_out");
    if (r->evicted) return fail(ctx, CART_ERR_EVICTED, "evict: the request is already swapped out");
    int32_t n = 0;
    for (int32_t l : r->len) n = std::max(n, l);
    if (n > 0 && (!k_out || !v_out)) return fail(ctx, CART_ERR_INVALID_ARG, "evict: null buffer for %d tokens", n);
    if (n > 0) {
        const cart_status st = swap_copy(ctx, *r, k_out, v_out, n, true, static_cast<cudaStream_t>(stream));
        if (st != CART_OK) return st;
    }
    drop_storage(ctx, *r);
    r->evicted = true;
    ++ctx->epoch;
    *n_tokens_out = n;
    return CART_OK;
}

cart_status cart_restore_request(cart_ctx *ctx, cart_req req, const void *k_in, const void *v_in, void *stream)
{
    if (!ctx) return CART_ERR_INVALID_ARG;
    Request *r = get_req(ctx, req);
    if (!r) return fail(ctx, CART_ERR_BAD_HANDLE, "restore: not an open request");
    if (!r->evicted) return fail(ctx, CART_ERR_EVICTED, "restore: the request is not swapped out");
    int32_t n = 0;
    for (int32_t l : r->len) n = std::max(n, l);
    if (n > 0 && (!k_in || !v_in)) return fail(ctx, CART_ERR_INVALID_ARG, "restore: null buffer for %d tokens", n);
    if (r->paged) {
        r->cap = 0;
        if (!grow_pages(ctx, *r, n)) {
            drop_storage(ctx, *r);
            return fail(ctx, CART_ERR_OOM, "restore: arena has no room for %d tokens of pages", n);
        }
    } else {
        const uint64_t rows_one = (uint64_t)ctx->cfg.n_layers * ctx->cfg.n_kv_heads * (uint64_t)r->cap;
        uint64_t start = 0;
        if (rows_one > 0 && !arena_alloc(ctx, 2 * rows_one, &start))
            return fail(ctx, CART_ERR_OOM, "restore: arena has no room for a suffix of %d tokens", r->cap);
        r->k_row = start;
        r->v_row = start + rows_one;
        r->alloc_start = start;
        r->alloc_rows = 2 * rows_one;
    }
    if (n > 0) {
        const cart_status st = swap_copy(ctx, *r, const_cast<void *>(k_in), const_cast<void *>(v_in), n, false,
                                         static_cast<cudaStream_t>(stream));
        if (st != CART_OK) {
            drop_storage(ctx, *r);
            return st;
        }
    }
    r->evicted = false;
    ++ctx->epoch;
    return CART_OK;
}

cart_status cart_evict_cartridge(cart_ctx *ctx, cart_id id)
{
    if (!ctx) return CART_ERR_INVALID_ARG;
    Cartridge *c = get_cart(ctx, id);
    if (!c || c->composed) return fail(ctx, CART_ERR_BAD_HANDLE, "evict: not a registered Cartridge");
    if (c->evicted) return fail(ctx, CART_ERR_EVICTED, "evict: the Cartridge is already swapped out");
    if (cartridge_has_active_reader(ctx, id))
        return fail(ctx, CART_ERR_IN_USE, "evict: a resident request attends to the Cartridge");
    arena_free(ctx, c->alloc_start, c->alloc_rows);
    c->alloc_rows = 0;
    c->evicted = true;
    ++ctx->epoch;
    return CART_OK;
}

cart_status cart_restore_cartridge(cart_ctx *ctx, cart_id id, const void *k, const void *v, void *stream)
{
    if (!ctx) return CART_ERR_INVALID_ARG;
    Cartridge *c = get_cart(ctx, id);
    if (!c || c->composed) return fail(ctx, CART_ERR_BAD_HANDLE, "restore: not a registered Cartridge");
    if (!c->evicted) return fail(ctx, CART_ERR_EVICTED, "restore: the Cartridge is not swapped out");
    if (!aligned16(k) || !aligned16(v)) return fail(ctx, CART_ERR_INVALID_ARG, "restore: null/misaligned pointer");
    const uint64_t rows_one = (uint64_t)ctx->cfg.n_layers * ctx->cfg.n_kv_heads * (uint64_t)c->p;
    uint64_t start = 0;
    if (!arena_alloc(ctx, 2 * rows_one, &start))
        return fail(ctx, CART_ERR_OOM, "restore: arena has no room for %llu bytes", (unsigned long long)(2 * rows_one * kRowBytes));
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemcpyAsync(arena_ptr(ctx, start), k, rows_one * kRowBytes, cudaMemcpyDefault, s);
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(arena_ptr(ctx, start + rows_one), v, rows_one * kRowBytes, cudaMemcpyDefault, s);
    if (e != cudaSuccess) {
        arena_free(ctx, start, 2 * rows_one);
        return fail(ctx, CART_ERR_CUDA, "restore: copy failed: %s", cudaGetErrorString(e));
    }
    c->k_row = start;
    c->v_row = start + rows_one;
    c->alloc_start = start;
    c->alloc_rows = 2 * rows_one;
    c->evicted = false;
    ++ctx->epoch;
    return CART_OK;
}

cart_status cart_append_kv(cart_ctx *ctx, int32_t layer, const cart_req *reqs, int32_t n_reqs, const void *k_new,
                           const void *v_new, void *stream)
{
    if (!ctx) return CART_ERR_INVALID_ARG;
    if (!reqs || n_reqs < 1 || !aligned16(k_new) || !aligned16(v_new))
        return fail(ctx, CART_ERR_INVALID_ARG, "append: null/misaligned pointer or empty batch");
    if (layer < 0 || layer >= ctx->cfg.n_layers) return fail(ctx, CART_ERR_BAD_HANDLE, "append: layer out of range");
    const uint64_t stamp = ++ctx->stamp;
    for (int32_t i = 0; i < n_reqs; ++i) {
        Request *r = get_req(ctx, reqs[i]);
        if (!r) return fail(ctx, CART_ERR_BAD_HANDLE, "append: reqs[%d] is not an open request", i);
        if (r->stamp == stamp) return fail(ctx, CART_ERR_INVALID_ARG, "append: reqs[%d] appears twice", i);
        r->stamp = stamp;
        if (r->evicted) return fail(ctx, CART_ERR_EVICTED, "append: reqs[%d] is swapped out", i);
        if (!r->paged && r->len[(size_t)layer] >= r->cap)
            return fail(ctx, CART_ERR_CAPACITY, "append: suffix of reqs[%d] is full (%d tokens)", i, r->cap);
    }
    for (int32_t i = 0; i < n_reqs; ++i) {  // paged suffixes take a page when the token opens one
        Request &r = ctx->reqs[(size_t)reqs[i]];
        if (r.paged && !grow_pages(ctx, r, (int64_t)r.len[(size_t)layer] + 1))
            return fail(ctx, CART_ERR_OOM, "append: arena has no page left for reqs[%d]", i);
    }
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int Hkv = ctx->cfg.n_kv_heads;
    static_assert(sizeof(AppendParams) <= 4096, "append parameters must fit the kernel parameter space");
    AppendParams ap;
    for (int32_t b0 = 0; b0 < n_reqs; b0 += kAppendBatch) {
        const int32_t n = std::min(kAppendBatch, n_reqs - b0);
        for (int32_t i = 0; i < n; ++i) {
            const Request &r = ctx->reqs[(size_t)reqs[b0 + i]];
            if (r.paged) {
                const uint64_t row = paged_row(ctx, r, layer, r.len[(size_t)layer]);
                ap.e[i].k_row = (uint32_t)row;
                ap.e[i].v_row = (uint32_t)(row + kTileTokens);
                ap.e[i].head_stride = 2u * kTileTokens;
                continue;
            }
            const uint64_t off = (uint64_t)layer * Hkv * (uint64_t)r.cap + (uint64_t)r.len[(size_t)layer];
            ap.e[i].k_row = (uint32_t)(r.k_row + off);
            ap.e[i].v_row = (uint32_t)(r.v_row + off);
            ap.e[i].head_stride = (uint32_t)r.cap;
        }
        ap.arena = ctx->cfg.arena;
        ap.k_new = static_cast<const uint8_t *>(k_new) + (uint64_t)b0 * Hkv * kRowBytes;
        ap.v_new = static_cast<const uint8_t *>(v_new) + (uint64_t)b0 * Hkv * kRowBytes;
        ap.n = n;
        ap.n_kv_heads = Hkv;
        CART_CUDA(ctx, launch_append(ap, s));
        ++ctx->launches;
    }
    for (int32_t i = 0; i < n_reqs; ++i) ++ctx->reqs[(size_t)reqs[i]].len[(size_t)layer];
    return CART_OK;
}

cart_status cart_extend_kv(cart_ctx *ctx, int32_t layer, cart_req req, const void *k, const void *v,
                           int32_t n_tokens, void *stream)
{
    if (!ctx) return CART_ERR_INVALID_ARG;
    if (!aligned16(k) || !aligned16(v) || n_tokens < 1)
        return fail(ctx, CART_ERR_INVALID_ARG, "extend: null/misaligned pointer or n_tokens < 1");
    if (layer < 0 || layer >= ctx->cfg.n_layers) return fail(ctx, CART_ERR_BAD_HANDLE, "extend: layer out of range");
    Request *r = get_req(ctx, req);
    if (!r) return fail(ctx, CART_ERR_BAD_HANDLE, "extend: not an open request");
    if (r->evicted) return fail(ctx, CART_ERR_EVICTED, "extend: the request is swapped out");
    if (r->paged) {
        if (!grow_pages(ctx, *r, (int64_t)r->len[(size_t)layer] + n_tokens))
            return fail(ctx, CART_ERR_OOM, "extend: arena has no pages left for %d more tokens", n_tokens);
        // one scatter per page touched
        const int Hkv = ctx->cfg.n_kv_heads;
        int32_t done = 0;
        while (done < n_tokens) {
            const int32_t pos = r->len[(size_t)layer] + done;
            const int32_t n = std::min(n_tokens - done, kTileTokens - pos % kTileTokens);
            ExtendParams ep;
            const uint64_t row = paged_row(ctx, *r, layer, pos);
            ep.arena = ctx->cfg.arena;
            ep.k = static_cast<const uint8_t *>(k) + (uint64_t)done * Hkv * kRowBytes;
            ep.v = static_cast<const uint8_t *>(v) + (uint64_t)done * Hkv * kRowBytes;
            ep.k_row = (uint32_t)row;
            ep.v_row = (uint32_t)(row + kTileTokens);
            ep.head_stride = 2u * kTileTokens;
            ep.n_tokens = n;
            ep.n_kv_heads = Hkv;
            CART_CUDA(ctx, launch_extend(ep, static_cast<cudaStream_t>(stream)));
            ++ctx->launches;
            done += n;
        }
        r->len[(size_t)layer] += n_tokens;
        return CART_OK;
    }
    if ((int64_t)r->len[(size_t)layer] + n_tokens > r->cap)
        return fail(ctx, CART_ERR_CAPACITY, "extend: %d + %d tokens exceed the capacity %d", r->len[(size_t)layer],
                    n_tokens, r->cap);
    ExtendParams ep;
    const uint64_t off = (uint64_t)layer * ctx->cfg.n_kv_heads * (uint64_t)r->cap + (uint64_t)r->len[(size_t)layer];
    ep.arena = ctx->cfg.arena;
    ep.k = k;
    ep.v = v;
    ep.k_row = (uint32_t)(r->k_row + off);
    ep.v_row = (uint32_t)(r->v_row + off);
    ep.head_stride = (uint32_t)r->cap;
    ep.n_tokens = n_tokens;
    ep.n_kv_heads = ctx->cfg.n_kv_heads;
    CART_CUDA(ctx, launch_extend(ep, static_cast<cudaStream_t>(stream)));
    ++ctx->launches;
    r->len[(size_t)layer] += n_tokens;
    return CART_OK;
}

}  // extern "C"

namespace {

// Decode attention for a batch; with k_new / v_new non-null the stream kernel first writes each
// request's new token at position len - 1 of its suffix (the host lengths already count it).
// Prefill mode (n_pre > 0): reqs[0 .. n_pre) are requests, and the batch is, request after request, the last
// n_new_list[c] suffix tokens of request c as query rows; a row attends over the Cartridge(s) and the suffix up
// to and including its own token (Eq. 1 for the rows of the new block).  The rows are planned like requests
// that share the Cartridge(s) and, group by group, the part of the suffix before the group's first token, so
// those go through the shared-segment kernel.  (One request: prefill of a user's message.  Many requests
// that are whole conversations over one Cartridge: the forward of training-time attention.)
// Launches the kernels of a plan for one layer: the stream kernel, the tensor-core kernel for the shared part and the
// merge kernel, as the plan needs them.  grow: tokens every request has appended since the plan was built, or, with
// grow_ctr set, the device word that holds that count (a launch recorded in a CUDA graph).
cart_status launch_plan(cart_ctx *ctx, PlanSlot *sl, int32_t layer, const void *q, void *out, float *lse, const void *k_new,
                        const void *v_new, int32_t grow, const uint32_t *grow_ctr, cudaStream_t s)
{
    const int Hkv = ctx->cfg.n_kv_heads;
    sl->last_stream = s;

    uint8_t *arena = static_cast<uint8_t *>(ctx->cfg.arena);
    DecodeParams dp;
    dp.cta_begin = reinterpret_cast<const uint32_t *>(sl->dev + ctx->lay.cta_begin_off);
    dp.items = reinterpret_cast<const cart_work_item *>(sl->dev + ctx->lay.items_off);
    dp.q = q;
    dp.k_new = k_new;
    dp.v_new = v_new;
    dp.arena = ctx->cfg.arena;
    dp.out = out;
    dp.lse = lse;
    dp.part_o = reinterpret_cast<float *>(arena + ctx->lay.part_o_off);
    dp.part_lse2 = reinterpret_cast<float *>(arena + ctx->lay.part_lse_off);
    dp.merges = reinterpret_cast<const cart_merge_item *>(sl->dev + ctx->lay.merges_off);
    // Few split row groups: the block that delivers the last partial merges (arrival tickets, no extra
    // launch).  Many (every reader of a shared Cartridge is one): a merge kernel over all of them.
    const bool merge_after = sl->n_merges > ctx->n_cta;
    dp.tickets = merge_after ? nullptr : reinterpret_cast<uint32_t *>(arena + ctx->lay.tickets_off);
    dp.status = reinterpret_cast<uint32_t *>(arena + ctx->lay.status_off);
    dp.layer = layer;
    dp.group = ctx->group;
    dp.scale_log2 = ctx->scale * 1.4426950408889634f;
    dp.grow = (uint32_t)grow;
    dp.grow_ctr = grow_ctr;
    dp.edge_boxes = 1u;
    dp.pages = reinterpret_cast<const uint32_t *>(sl->dev + ctx->lay.pages_off);
    const bool timed = ctx->timing && grow_ctr == nullptr && ctx->ev_used + 2 <= kMaxTimedLaunches * 2;
    if (timed) {
        while (ctx->ev_pool.size() < ctx->ev_used + 2) {
            cudaEvent_t e;
            CART_CUDA(ctx, cudaEventCreate(&e));
            ctx->ev_pool.push_back(e);
        }
        CART_CUDA(ctx, cudaEventRecord(ctx->ev_pool[ctx->ev_used], s));
    }
    // A batch with a shared part and a stream part runs the two kernels side by side: the stream kernel
    // is launched first on its share of the SMs, the shared kernel right behind it on the rest (a dependent
    // launch starts as soon as every block of the kernel before has started).
    const bool pair = sl->n_units > 0 && sl->n_items > 0 && ctx->side_by_side > 0;
    if (pair) {
        dp.ready_flag = reinterpret_cast<uint32_t *>(arena + ctx->lay.status_off + 128);
    }
    if (pair) {
        CART_CUDA(ctx, launch_decode(ctx->tmap, ctx->tmap_edge, dp, sl->n_cta_used, s));
        ++ctx->launches;
    }
    if (sl->n_units > 0) {
        SharedParams sp;
        sp.unit_cta_begin = reinterpret_cast<const uint32_t *>(sl->dev + ctx->lay.unit_cta_begin_off);
        sp.units = reinterpret_cast<const cart_shared_unit *>(sl->dev + ctx->lay.units_off);
        sp.readers = reinterpret_cast<const uint32_t *>(sl->dev + ctx->lay.readers_off);
        sp.reader_slot = reinterpret_cast<const uint32_t *>(sl->dev + ctx->lay.reader_slot_off);
        sp.reader_merge = reinterpret_cast<const uint32_t *>(sl->dev + ctx->lay.reader_merge_off);
        sp.merges = dp.merges;
        sp.q = q;
        sp.out = out;
        sp.lse = lse;
        sp.part_o = dp.part_o;
        sp.part_lse2 = dp.part_lse2;
        sp.tickets = dp.tickets;
        sp.status = dp.status;
        sp.layer = layer;
        sp.group = ctx->group;
        sp.n_kv_heads = Hkv;
        sp.n_q_heads = ctx->cfg.n_q_heads;
        sp.scale_log2 = dp.scale_log2;
        sp.ready_flag = dp.ready_flag;
        sp.pages = dp.pages;
        CART_CUDA(ctx, launch_shared(ctx->tmap, sp, sl->n_unit_cta_used, s));
        ++ctx->launches;
    }
    if (sl->n_items > 0 && !pair) {
        CART_CUDA(ctx, launch_decode(ctx->tmap, ctx->tmap_edge, dp, sl->n_cta_used, s));
        ++ctx->launches;
    }
    if (merge_after) {
        MergeParams mp;
        mp.merges = dp.merges;
        mp.part_o = dp.part_o;
        mp.part_lse2 = dp.part_lse2;
        mp.out = out;
        mp.lse = lse;
        mp.group = ctx->group;
        CART_CUDA(ctx, launch_merge(mp, sl->n_merges, s));
        ++ctx->launches;
    }
    if (timed) {
        CART_CUDA(ctx, cudaEventRecord(ctx->ev_pool[ctx->ev_used + 1], s));
        ctx->ev_used += 2;
    }
    return CART_OK;
}

cart_status decode_impl(cart_ctx *ctx, int32_t layer, const cart_req *reqs, int32_t n_reqs, const void *q,
                        void *out, float *lse, const void *k_new, const void *v_new, void *stream,
                        const int32_t *n_new_list = nullptr, int32_t n_pre = 0)
{
    const bool prefill = n_pre > 0;
    if (prefill) {
        int64_t rows = 0;
        for (int32_t c = 0; c < n_pre; ++c) {
            if (n_new_list[c] < 1) return fail(ctx, CART_ERR_INVALID_ARG, "prefill: n_new < 1");
            rows += n_new_list[c];
        }
        if (rows > ctx->cfg.max_requests)
            return fail(ctx, CART_ERR_CAPACITY, "prefill: %lld rows exceed max_requests %d", (long long)rows,
                        ctx->cfg.max_requests);
        n_reqs = (int32_t)rows;
    }
    if (!reqs || n_reqs < 1 || !aligned16(q) || !aligned16(out) || (lse && (reinterpret_cast<uintptr_t>(lse) & 3u)))
        return fail(ctx, CART_ERR_INVALID_ARG, "decode: null/misaligned pointer or empty batch");
    if (layer < 0 || layer >= ctx->cfg.n_layers) return fail(ctx, CART_ERR_BAD_HANDLE, "decode: layer out of range");
    if (n_reqs > ctx->cfg.max_requests)
        return fail(ctx, CART_ERR_CAPACITY, "decode: batch %d exceeds max_requests %d", n_reqs, ctx->cfg.max_requests);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int Hkv = ctx->cfg.n_kv_heads;

    // The plan depends on which requests are in the batch and on their lengths in this layer.  A decode
    // plan stays good while every request has grown by the same number of tokens since it was built (one
    // per fused decode step): the kernels add that number to the tail items.
    std::vector<uint32_t> &key = ctx->key_tmp;
    std::vector<int32_t> &cur_len = ctx->len_tmp;
    key.clear();
    cur_len.clear();
    for (int32_t c = 0; c < n_pre; ++c) {
        Request *r = get_req(ctx, reqs[c]);
        if (!r) return fail(ctx, CART_ERR_BAD_HANDLE, "prefill: not an open request");
        if (r->evicted) return fail(ctx, CART_ERR_EVICTED, "prefill: the request is swapped out");
        if (evicted_part(ctx, *r) >= 0)
            return fail(ctx, CART_ERR_EVICTED, "prefill: Cartridge %d is swapped out", evicted_part(ctx, *r));
        if (r->len[(size_t)layer] < n_new_list[c])
            return fail(ctx, CART_ERR_INVALID_ARG, "prefill: the suffix holds %d tokens, fewer than n_new = %d",
                        r->len[(size_t)layer], n_new_list[c]);
        key.push_back((uint32_t)reqs[c]);
        key.push_back((uint32_t)r->len[(size_t)layer]);
        key.push_back((uint32_t)n_new_list[c]);
    }
    for (int32_t i = 0; i < n_reqs && !prefill; ++i) {
        Request *r = get_req(ctx, reqs[i]);
        if (!r) return fail(ctx, CART_ERR_BAD_HANDLE, "decode: reqs[%d] is not an open request", i);
        if (r->evicted) return fail(ctx, CART_ERR_EVICTED, "decode: reqs[%d] is swapped out", i);
        if (evicted_part(ctx, *r) >= 0)
            return fail(ctx, CART_ERR_EVICTED, "decode: reqs[%d] attends to Cartridge %d, which is swapped out", i,
                        evicted_part(ctx, *r));
        const int32_t len = r->len[(size_t)layer];
        if (len == 0 && r->cart == CART_NONE)
            return fail(ctx, CART_ERR_EMPTY, "decode: reqs[%d] has no KV token in layer %d", i, layer);
        cur_len.push_back(len);
    }

    PlanSlot *sl = ctx->cur_slot >= 0 ? &ctx->slots[ctx->cur_slot] : nullptr;
    int32_t grow = 0;
    bool reuse = sl && sl->valid && sl->epoch == ctx->epoch && sl->prefill == prefill && !ctx->plan_only;
    if (reuse && prefill) reuse = sl->key == key;
    if (reuse && !prefill)
        reuse = sl->reqs.size() == (size_t)n_reqs && std::memcmp(sl->reqs.data(), reqs, (size_t)n_reqs * sizeof(int32_t)) == 0 &&
                cart_plan_reusable(sl->lens.data(), cur_len.data(), n_reqs, ctx->max_grow, &grow) != 0;
    if (!reuse) {
        grow = 0;
        // Build a new plan in the next ring slot.
        if (sl && sl->valid) {
            CART_CUDA(ctx, cudaEventRecord(sl->ev, sl->last_stream));
            sl->ev_recorded = true;
        }
        const int next = (ctx->cur_slot + 1) % kPlanSlots;
        PlanSlot &ns = ctx->slots[next];
        if (ns.ev_recorded) {
            CART_CUDA(ctx, cudaEventSynchronize(ns.ev));
            ns.ev_recorded = false;
        }
        ns.valid = false;
        ns.chain = false;
        // Paged suffixes.  In a fused decode loop every request takes a new page once per 64 steps, each at a step
        // of its own, and a new page means a new plan; so when a plan is built anyway, requests with less than a
        // page of room are given their next page now (if the arena has one), and the plan lasts 64 steps or more.
        if (k_new != nullptr)
            for (int32_t i = 0; i < n_reqs; ++i) {
                Request &r = ctx->reqs[(size_t)reqs[i]];
                if (r.paged) (void)grow_pages(ctx, r, (int64_t)r.len[(size_t)layer] + kTileTokens);
            }
        // the batch's page list: every page of every paged request, request by request
        uint32_t *page_list = reinterpret_cast<uint32_t *>(ns.host + ctx->lay.pages_off);
        uint32_t n_listed = 0;
        const uint64_t list_stamp = ++ctx->list_stamp;
        auto &segs = ctx->seg_tmp;
        auto &sb = ctx->seg_begin_tmp;
        segs.clear();
        sb.clear();
        sb.push_back(0);
        // Prefill: the rows are cut into groups of 128 / G consecutive tokens (the rows one tensor-core
        // tile holds per KV head).  Everything before a group's first token, rounded down to whole shared
        // tiles, is visible to all of its rows: that is the group's shared head of the suffix, a
        // staircase that follows the causal diagonal, so a row streams fewer than 128 + 128 / G tokens
        // by itself.  A step is only taken if enough rows stand on it to be shared.
        // row_of[i] = (request of row i, its index among the request's new tokens, its group's shared head)
        struct RowOf { int32_t c, i, head; };
        std::vector<RowOf> row_of;
        const int32_t rows_per_tile = 128 / ctx->group;
        for (int32_t c = 0; c < n_pre; ++c) {
            const int32_t n_new = n_new_list[c];
            std::vector<int32_t> &head_of_group = ctx->head_tmp;
            head_of_group.clear();
            if (ctx->share_min_readers > 0 && n_new >= ctx->share_min_readers) {
                const int32_t s_old = ctx->reqs[(size_t)reqs[c]].len[(size_t)layer] - n_new;
                const int32_t n_groups = (n_new + rows_per_tile - 1) / rows_per_tile;
                auto natural = [&](int32_t g) { return (s_old + g * rows_per_tile) / kShareTileTokens * kShareTileTokens; };
                int32_t cur = natural(0);
                for (int32_t g = 0; g < n_groups; ++g) {
                    const int32_t nat = natural(g);
                    if (nat != cur) {
                        int32_t g2 = g;
                        while (g2 < n_groups && natural(g2) == nat) ++g2;
                        const int32_t rows = std::min(n_new, g2 * rows_per_tile) - g * rows_per_tile;
                        if (rows >= ctx->share_min_readers) cur = nat;
                    }
                    head_of_group.push_back(cur);
                }
            }
            for (int32_t i = 0; i < n_new; ++i)
                row_of.push_back(RowOf{c, i, head_of_group.empty() ? 0 : head_of_group[(size_t)(i / rows_per_tile)]});
        }
        bool list_full = false;
        // describes the part of a paged suffix that starts at token `first` (a multiple of the page size)
        auto paged_seg = [&](Request &r, uint32_t first, cart_plan_seg *sg) {
            if (r.list_stamp != list_stamp) {
                if (n_listed + r.pages.size() > (size_t)ctx->lay.pages_cap) { list_full = true; return; }
                r.list_stamp = list_stamp;
                r.list_base = n_listed;
                for (uint32_t pg : r.pages) page_list[n_listed++] = pg;
            }
            sg->k_row = r.list_base + first / (uint32_t)kTileTokens;
            sg->v_row = 0;
            sg->head_stride = 2u * kTileTokens;
            sg->layer_stride = (uint32_t)Hkv * 2u * kTileTokens;
            sg->flags |= CART_SEG_PAGED;
        };
        for (int32_t i = 0; i < n_reqs; ++i) {
            Request &r = ctx->reqs[(size_t)reqs[prefill ? row_of[(size_t)i].c : i]];
            auto push_cart = [&](const Cartridge &c) {
                cart_plan_seg sg;
                sg.k_row = (uint32_t)c.k_row;
                sg.v_row = (uint32_t)c.v_row;
                sg.head_stride = (uint32_t)c.p;
                sg.layer_stride = (uint32_t)((uint64_t)Hkv * c.p);
                sg.n_tok = (uint32_t)c.p;
                sg.flags = 0;
                segs.push_back(sg);
            };
            if (r.cart != CART_NONE) {
                const Cartridge &c = ctx->carts[(size_t)r.cart];
                if (c.composed) for (int32_t b : c.parts) push_cart(ctx->carts[(size_t)b]);
                else push_cart(c);
            }
            int32_t len = r.len[(size_t)layer];
            uint32_t first = 0;  // first suffix token of the segment
            if (prefill) {
                // row i sees the suffix up to its own token; its group's shared head is a segment of its own
                const int32_t s_old = len - n_new_list[row_of[(size_t)i].c];
                len = s_old + row_of[(size_t)i].i + 1;
                const int32_t head = row_of[(size_t)i].head;
                if (head > 0) {
                    cart_plan_seg sg;
                    sg.k_row = (uint32_t)r.k_row;
                    sg.v_row = (uint32_t)r.v_row;
                    sg.head_stride = (uint32_t)r.cap;
                    sg.layer_stride = (uint32_t)((uint64_t)Hkv * r.cap);
                    sg.n_tok = (uint32_t)head;
                    sg.flags = CART_SEG_SUFFIX;
                    if (r.paged) paged_seg(r, 0u, &sg);
                    segs.push_back(sg);
                    first = (uint32_t)head;
                }
            }
            if (len > (int32_t)first) {
                cart_plan_seg sg;
                sg.k_row = (uint32_t)r.k_row + first;
                sg.v_row = (uint32_t)r.v_row + first;
                sg.head_stride = (uint32_t)r.cap;
                sg.layer_stride = (uint32_t)((uint64_t)Hkv * r.cap);
                sg.n_tok = (uint32_t)len - first;
                sg.flags = CART_SEG_SUFFIX;
                if (r.paged) paged_seg(r, first, &sg);
                segs.push_back(sg);
            }
            sb.push_back((int32_t)segs.size());
        }
        if (list_full) return fail(ctx, CART_ERR_CAPACITY, "decode: the batch names more than %d pages", ctx->lay.pages_cap);
        const ScratchLayout &lay = ctx->lay;
        cart_plan_out po{};
        po.items = reinterpret_cast<cart_work_item *>(ns.host + lay.items_off);
        po.items_cap = lay.items_cap;
        po.cta_begin = reinterpret_cast<uint32_t *>(ns.host + lay.cta_begin_off);
        po.merges = reinterpret_cast<cart_merge_item *>(ns.host + lay.merges_off);
        po.merges_cap = lay.merges_cap;
        po.slots_cap = lay.slots_cap;
        po.piece_cost = ctx->piece_cost;
        po.unit_cost = kUnitCostTiles;
        po.side_by_side = ctx->side_by_side;
        po.units = reinterpret_cast<cart_shared_unit *>(ns.host + lay.units_off);
        po.units_cap = lay.units_cap;
        po.unit_cta_begin = reinterpret_cast<uint32_t *>(ns.host + lay.unit_cta_begin_off);
        po.readers = reinterpret_cast<uint32_t *>(ns.host + lay.readers_off);
        po.readers_cap = lay.readers_cap;
        po.reader_slot = reinterpret_cast<uint32_t *>(ns.host + lay.reader_slot_off);
        po.reader_merge = reinterpret_cast<uint32_t *>(ns.host + lay.reader_merge_off);
        cart_status st = cart_plan_build_shared(segs.data(), sb.data(), n_reqs, Hkv, ctx->group, ctx->n_cta,
                                                kTileTokens, ctx->share_min_readers, kShareTileTokens, &po);
        if (st != CART_OK) return fail(ctx, st, "decode: planning failed (%s)", cart_status_string(st));
        ns.n_items = po.n_items;
        ns.n_merges = po.n_merges;
        ns.n_cta_used = po.n_cta_used;
        ns.n_slots = po.n_slots;
        ns.n_units = po.n_units;
        ns.n_unit_cta_used = po.n_unit_cta_used;
        const uint64_t bytes = lay.items_off + (uint64_t)ns.n_items * sizeof(cart_work_item);
        CART_CUDA(ctx, cudaMemcpyAsync(ns.dev, ns.host, bytes, cudaMemcpyHostToDevice, s));
        if (ns.n_units > 0) {
            const uint64_t sh_bytes = lay.units_off + (uint64_t)ns.n_units * sizeof(cart_shared_unit) - lay.shared_off;
            CART_CUDA(ctx, cudaMemcpyAsync(ns.dev + lay.shared_off, ns.host + lay.shared_off, sh_bytes,
                                           cudaMemcpyHostToDevice, s));
        }
        if (n_listed > 0)
            CART_CUDA(ctx, cudaMemcpyAsync(ns.dev + lay.pages_off, ns.host + lay.pages_off, (uint64_t)n_listed * 4,
                                           cudaMemcpyHostToDevice, s));
        ns.key = key;
        ns.prefill = prefill;
        ns.reqs.assign(reqs, reqs + (prefill ? n_pre : n_reqs));
        ns.lens = cur_len;
        ns.epoch = ctx->epoch;
        ns.valid = true;
        ++ctx->plans_built;
        ctx->cur_slot = next;
        sl = &ns;
    }
    if (ctx->plan_only) return CART_OK;   // (a recorded decode loop launches from the plan later)
    return launch_plan(ctx, sl, layer, q, out, lse, k_new, v_new, grow, nullptr, s);
}

}  // namespace

extern "C" {

cart_status cart_decode_attention(cart_ctx *ctx, int32_t layer, const cart_req *reqs, int32_t n_reqs, const void *q,
                                  void *out, float *lse, void *stream)
{
    if (!ctx) return CART_ERR_INVALID_ARG;
    return decode_impl(ctx, layer, reqs, n_reqs, q, out, lse, nullptr, nullptr, stream);
}

cart_status cart_prefill_attention(cart_ctx *ctx, int32_t layer, cart_req req, const void *q, int32_t n_new, void *out,
                                   float *lse, void *stream)
{
    if (!ctx) return CART_ERR_INVALID_ARG;
    if (n_new < 1) return fail(ctx, CART_ERR_INVALID_ARG, "prefill: n_new < 1");
    // A message goes through chains of masked tiles on the tensor-core kernel, the diagonal too: a chain is an M-tile
    // of 128 / G tokens times a KV head, over the Cartridge(s) and the suffix up to the M-tile's last token.  With a
    // chain or more per SM, or at least half as many, every chain writes its rows' output itself (1024 tokens over a
    // 2048-token Cartridge: 194 us per layer against 256 through the decode kernels; 512 tokens: 75 against 122).
    // A shorter message has too few chains to fill the device, so each chain is cut along its keys into pieces of at
    // least two tiles, as many as give every SM one, and the merge kernel combines the pieces' partials (64 tokens:
    // 25 us against 34; 256: 40 against 67).  Paged suffixes, messages of fewer than four tokens (decode in all but
    // name: 2 tokens take 20 us there, 25 as chains) and suffixes beyond 16 k tokens -- where every chain re-reads the
    // whole suffix while the decode kernels' shared steps read it once per group of steps (1024 tokens behind 30 k:
    // 775 us against 680) -- go through the decode kernels.
    Request *r = get_req(ctx, req);
    const int32_t tpt = 128 / ctx->group;
    if (r && !r->paged && !r->evicted && ctx->share_min_readers > 0 && n_new <= ctx->cfg.max_requests &&
        r->len[(size_t)std::max(0, std::min(layer, ctx->cfg.n_layers - 1))] <= 16384 &&
        layer >= 0 && layer < ctx->cfg.n_layers && r->len[(size_t)layer] >= n_new && evicted_part(ctx, *r) < 0 && aligned16(q) &&
        aligned16(out)) {
        std::vector<ChainPart> parts;
        uint32_t chain_tiles = 0;
        if (r->cart != CART_NONE) {
            const Cartridge &c = ctx->carts[(size_t)r->cart];
            if (c.composed) for (int32_t b : c.parts) parts.push_back(ChainPart{ctx->carts[(size_t)b].k_row, ctx->carts[(size_t)b].v_row, (uint32_t)ctx->carts[(size_t)b].p});
            else parts.push_back(ChainPart{c.k_row, c.v_row, (uint32_t)c.p});
        }
        for (const ChainPart &pt : parts) chain_tiles += (pt.p + 127u) / 128u;
        const uint32_t len = (uint32_t)r->len[(size_t)layer];
        chain_tiles += (len + 127u) / 128u;
        const int64_t chains = (int64_t)((n_new + tpt - 1) / tpt) * ctx->cfg.n_kv_heads;
        uint32_t n_split = 1;
        if (chains < ctx->n_cta) {
            const bool chosen = ctx->prefill_split >= 0;
            n_split = chosen ? (uint32_t)ctx->prefill_split
                             : (n_new >= 4 ? (uint32_t)std::max<int64_t>(1, std::min<int64_t>(ctx->n_cta / chains, chain_tiles / 2u)) : 0u);
            // no more pieces than the chain has tiles or the partial slots hold
            const int64_t rgs = (int64_t)n_new * ctx->cfg.n_kv_heads;
            n_split = std::min(n_split, std::max(chain_tiles, 1u));
            while (n_split > 1u && rgs * n_split > ctx->lay.slots_cap) --n_split;
        }
        if (n_split >= 1u) {
            std::vector<ChainStrand> strands{ChainStrand{r->k_row, r->v_row, (uint32_t)r->cap, len, 0u, (uint32_t)n_new, len - (uint32_t)n_new}};
            return launch_chains(ctx, layer, parts, strands, (uint32_t)n_new, q, out, lse, static_cast<cudaStream_t>(stream), n_split);
        }
    }
    return decode_impl(ctx, layer, &req, 1, q, out, lse, nullptr, nullptr, stream, &n_new, 1);
}

cart_status cart_decode_step(cart_ctx *ctx, int32_t layer, const cart_req *reqs, int32_t n_reqs, const void *k_new,
                             const void *v_new, const void *q, void *out, float *lse, void *stream)
{
    if (!ctx) return CART_ERR_INVALID_ARG;
    if (!reqs || n_reqs < 1 || !aligned16(k_new) || !aligned16(v_new))
        return fail(ctx, CART_ERR_INVALID_ARG, "decode_step: null/misaligned pointer or empty batch");
    if (layer < 0 || layer >= ctx->cfg.n_layers) return fail(ctx, CART_ERR_BAD_HANDLE, "decode_step: layer out of range");
    const uint64_t stamp = ++ctx->stamp;
    for (int32_t i = 0; i < n_reqs; ++i) {
        Request *r = get_req(ctx, reqs[i]);
        if (!r) return fail(ctx, CART_ERR_BAD_HANDLE, "decode_step: reqs[%d] is not an open request", i);
        if (r->stamp == stamp) return fail(ctx, CART_ERR_INVALID_ARG, "decode_step: reqs[%d] appears twice", i);
        r->stamp = stamp;
        if (r->evicted) return fail(ctx, CART_ERR_EVICTED, "decode_step: reqs[%d] is swapped out", i);
        if (!r->paged && r->len[(size_t)layer] >= r->cap)
            return fail(ctx, CART_ERR_CAPACITY, "decode_step: suffix of reqs[%d] is full (%d tokens)", i, r->cap);
    }
    for (int32_t i = 0; i < n_reqs; ++i) {  // paged suffixes take a page when the new token opens one
        Request &r = ctx->reqs[(size_t)reqs[i]];
        if (r.paged && !grow_pages(ctx, r, (int64_t)r.len[(size_t)layer] + 1))
            return fail(ctx, CART_ERR_OOM, "decode_step: arena has no page left for reqs[%d]", i);
    }
    // The plan must see the new token: count it first, take it back if nothing was launched.
    for (int32_t i = 0; i < n_reqs; ++i) ++ctx->reqs[(size_t)reqs[i]].len[(size_t)layer];
    const uint64_t launches_before = ctx->launches;
    const cart_status st = decode_impl(ctx, layer, reqs, n_reqs, q, out, lse, k_new, v_new, stream);
    if (st != CART_OK && ctx->launches == launches_before)
        for (int32_t i = 0; i < n_reqs; ++i) --ctx->reqs[(size_t)reqs[i]].len[(size_t)layer];
    return st;
}

// ---- a decode loop that can be recorded into a CUDA graph ----------------------------------------------------------
// cart_graph_begin plans the batch once, for the step that appends the first token, and clears a device word that
// counts the steps since; cart_graph_step launches a layer's kernels from that plan, reading the count from the
// word, and after the last layer a one-thread kernel advances it: no host work depends on the step, so the launches
// of one step can be recorded once and replayed.  cart_graph_end tells the host-side mirror how many steps ran.

static uint32_t *graph_counter(cart_ctx *ctx)
{
    return reinterpret_cast<uint32_t *>(static_cast<uint8_t *>(ctx->cfg.arena) + ctx->lay.status_off + 192);
}

cart_status cart_graph_begin(cart_ctx *ctx, const cart_req *reqs, int32_t n_reqs, int32_t max_steps, void *stream)
{
    if (!ctx) return CART_ERR_INVALID_ARG;
    if (ctx->graph_active) return fail(ctx, CART_ERR_IN_USE, "graph_begin: a recorded loop is already open");
    if (!reqs || n_reqs < 1 || max_steps < 1)
        return fail(ctx, CART_ERR_INVALID_ARG, "graph_begin: empty batch or max_steps < 1");
    if (max_steps > ctx->max_grow + 1)
        return fail(ctx, CART_ERR_CAPACITY, "graph_begin: max_steps %d exceeds what a kept plan covers (%d)", max_steps,
                    ctx->max_grow + 1);
    const int L = ctx->cfg.n_layers;
    const uint64_t stamp = ++ctx->stamp;
    for (int32_t i = 0; i < n_reqs; ++i) {
        Request *r = get_req(ctx, reqs[i]);
        if (!r) return fail(ctx, CART_ERR_BAD_HANDLE, "graph_begin: reqs[%d] is not an open request", i);
        if (r->stamp == stamp) return fail(ctx, CART_ERR_INVALID_ARG, "graph_begin: reqs[%d] appears twice", i);
        r->stamp = stamp;
        if (r->evicted) return fail(ctx, CART_ERR_EVICTED, "graph_begin: reqs[%d] is swapped out", i);
        for (int l = 1; l < L; ++l)
            if (r->len[(size_t)l] != r->len[0])
                return fail(ctx, CART_ERR_INVALID_ARG, "graph_begin: reqs[%d] holds %d tokens in layer %d and %d in layer 0", i,
                            r->len[(size_t)l], l, r->len[0]);
        if (!r->paged && r->len[0] + max_steps > r->cap)
            return fail(ctx, CART_ERR_CAPACITY, "graph_begin: reqs[%d] has room for %d more tokens, fewer than max_steps", i,
                        r->cap - r->len[0]);
    }
    for (int32_t i = 0; i < n_reqs; ++i) {  // paged suffixes take the pages of all the steps now
        Request &r = ctx->reqs[(size_t)reqs[i]];
        if (r.paged && !grow_pages(ctx, r, (int64_t)r.len[0] + max_steps))
            return fail(ctx, CART_ERR_OOM, "graph_begin: arena has no pages left for reqs[%d]", i);
    }
    // the plan of the first step: every request one token longer (the fused append writes that token)
    for (int32_t i = 0; i < n_reqs; ++i) ++ctx->reqs[(size_t)reqs[i]].len[0];
    ctx->plan_only = true;
    alignas(16) static const unsigned char dummy[16] = {0};   // (plan only: no pointer is used, they only have to pass the checks)
    alignas(16) static unsigned char sink[16];
    const cart_status st = decode_impl(ctx, 0, reqs, n_reqs, dummy, sink, nullptr, dummy, dummy, stream);
    ctx->plan_only = false;
    for (int32_t i = 0; i < n_reqs; ++i) --ctx->reqs[(size_t)reqs[i]].len[0];
    if (st != CART_OK) return st;
    CART_CUDA(ctx, cudaMemsetAsync(graph_counter(ctx), 0, 4, static_cast<cudaStream_t>(stream)));
    ctx->graph_active = true;
    ctx->graph_reqs.assign(reqs, reqs + n_reqs);
    ctx->graph_slot = ctx->cur_slot;
    ctx->graph_max_steps = max_steps;
    return CART_OK;
}

cart_status cart_graph_step(cart_ctx *ctx, int32_t layer, const void *k_new, const void *v_new, const void *q, void *out,
                            float *lse, void *stream)
{
    if (!ctx) return CART_ERR_INVALID_ARG;
    if (!ctx->graph_active) return fail(ctx, CART_ERR_INVALID_ARG, "graph_step: no recorded loop is open");
    if (layer < 0 || layer >= ctx->cfg.n_layers) return fail(ctx, CART_ERR_BAD_HANDLE, "graph_step: layer out of range");
    if (!aligned16(k_new) || !aligned16(v_new) || !aligned16(q) || !aligned16(out) || (lse && (reinterpret_cast<uintptr_t>(lse) & 3u)))
        return fail(ctx, CART_ERR_INVALID_ARG, "graph_step: null/misaligned pointer");
    if (ctx->cur_slot != ctx->graph_slot || !ctx->slots[ctx->graph_slot].valid)
        return fail(ctx, CART_ERR_INVALID_ARG, "graph_step: another attention call has taken the loop's plan");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    PlanSlot *sl = &ctx->slots[ctx->graph_slot];
    const cart_status st = launch_plan(ctx, sl, layer, q, out, lse, k_new, v_new, 0, graph_counter(ctx), s);
    if (st != CART_OK) return st;
    if (layer == ctx->cfg.n_layers - 1) {
        CART_CUDA(ctx, launch_advance(graph_counter(ctx), s));
        ++ctx->launches;
    }
    return CART_OK;
}

cart_status cart_graph_end(cart_ctx *ctx, int32_t steps_run)
{
    if (!ctx) return CART_ERR_INVALID_ARG;
    if (!ctx->graph_active) return fail(ctx, CART_ERR_INVALID_ARG, "graph_end: no recorded loop is open");
    if (steps_run < 0 || steps_run > ctx->graph_max_steps)
        return fail(ctx, CART_ERR_INVALID_ARG, "graph_end: %d steps, the loop was opened for at most %d", steps_run,
                    ctx->graph_max_steps);
    for (int32_t r : ctx->graph_reqs)
        for (int l = 0; l < ctx->cfg.n_layers; ++l) ctx->reqs[(size_t)r].len[(size_t)l] += steps_run;
    ctx->graph_active = false;
    ctx->graph_slot = -1;
    ++ctx->epoch;   // the kept plan describes the lengths before the loop
    return CART_OK;
}

}  // extern "C"

namespace {

// What the two training calls share: the conversations' lengths in `layer`, their common Cartridge (or none).
struct TrainBatch {
    std::vector<int32_t> len;   // tokens per conversation
    std::vector<int32_t> cu;    // running sum, n_convs + 1 entries
    int32_t T = 0;
    const Cartridge *z = nullptr;
};

cart_status train_batch(cart_ctx *ctx, int32_t layer, const cart_req *convs, int32_t n_convs, TrainBatch *tb)
{
    if (!convs || n_convs < 1) return fail(ctx, CART_ERR_INVALID_ARG, "train: no conversations");
    if (layer < 0 || layer >= ctx->cfg.n_layers) return fail(ctx, CART_ERR_BAD_HANDLE, "train: layer out of range");
    tb->cu.assign(1, 0);
    int32_t cart = CART_NONE;
    const uint64_t stamp = ++ctx->stamp;
    for (int32_t c = 0; c < n_convs; ++c) {
        Request *r = get_req(ctx, convs[c]);
        if (!r) return fail(ctx, CART_ERR_BAD_HANDLE, "train: convs[%d] is not an open request", c);
        if (r->stamp == stamp) return fail(ctx, CART_ERR_INVALID_ARG, "train: convs[%d] appears twice", c);
        r->stamp = stamp;
        if (r->evicted) return fail(ctx, CART_ERR_EVICTED, "train: convs[%d] is swapped out", c);
        if (r->paged) return fail(ctx, CART_ERR_INVALID_ARG, "train: convs[%d] has a paged suffix", c);
        if (c == 0) cart = r->cart;
        if (r->cart != cart) return fail(ctx, CART_ERR_INVALID_ARG, "train: the conversations attend to different Cartridges");
        const int32_t n = r->len[(size_t)layer];
        if (n < 1) return fail(ctx, CART_ERR_EMPTY, "train: convs[%d] has no token in layer %d", c, layer);
        tb->len.push_back(n);
        tb->cu.push_back(tb->cu.back() + n);
    }
    tb->T = tb->cu.back();
    if (tb->T > ctx->cfg.max_requests)
        return fail(ctx, CART_ERR_CAPACITY, "train: %d tokens exceed max_requests %d", tb->T, ctx->cfg.max_requests);
    if (cart != CART_NONE) {
        const Cartridge &z = ctx->carts[(size_t)cart];
        if (z.composed) return fail(ctx, CART_ERR_INVALID_ARG, "train: the Cartridge is a composition");
        if (z.evicted) return fail(ctx, CART_ERR_EVICTED, "train: the Cartridge is swapped out");
        tb->z = &z;
    }
    return CART_OK;
}

}  // namespace

extern "C" {

}  // extern "C"

namespace {

// Rows that attend causally, as chains of units on the tensor-core kernel (prefill of a message; the forward of
// training attention).  The rows are numbered 0 .. T - 1 (row t = query row t of q / out / lse); every row sees
// all of `parts` (Cartridge blocks, in order) and then its own "strand": strand c owns the rows row_begin ..
// row_begin + n_rows - 1, its keys are the first key_first + i + 1 tokens of a contiguous suffix buffer for its row i.
//
// One chain of units per (M-tile of 128 / G consecutive rows' tokens, KV head): the parts' tiles (every row sees all
// of them), then, strand by strand, the tiles of the strands the M-tile's rows belong to, masked causally.  With
// n_split = 1 the chain's last unit writes out and lse directly -- no partials, no merge, and no row streams its
// diagonal by itself.  With n_split > 1 (one strand only: a message too short to give every SM a chain) a chain is cut
// along its keys into up to n_split pieces, each a chain of its own that ends in a partial, and the merge kernel
// combines a row's partials; a piece starts no later than the tile that holds the first key which the M-tile's first
// row sees last, so every row sees at least one key of every piece.
//
// The plan is laid out back to back in a buffer of the plan ring -- [block -> first unit][reader -> query row]
// [reader slots][reader merges][merge items][units] -- so that one copy of just those bytes uploads it, and it is
// kept: a call with the same parts, strands and split (the next layer of the same step) launches from the buffer as
// it is.
cart_status launch_chains(cart_ctx *ctx, int32_t layer, const std::vector<ChainPart> &parts, const std::vector<ChainStrand> &strands,
                          uint32_t T, const void *q, void *out, float *lse, cudaStream_t s, uint32_t n_split)
{
    const int Hkv = ctx->cfg.n_kv_heads, G = ctx->group;
    const uint32_t tpt = 128u / (uint32_t)G;   // tokens (readers) per M-tile
    const uint32_t n_rt = (T + tpt - 1) / tpt;
    const int32_t n_strands = (int32_t)strands.size();
    const ScratchLayout &lay = ctx->lay;
    if (n_split < 1u || (n_split > 1u && n_strands != 1)) return fail(ctx, CART_ERR_INVALID_ARG, "chains: bad split");

    std::vector<uint64_t> &key = ctx->chain_key_tmp;
    key.clear();
    key.push_back(((uint64_t)T << 32) | n_split);
    for (const ChainPart &pt : parts) { key.push_back(pt.k_row); key.push_back(pt.v_row); key.push_back(pt.p); }
    key.push_back(~0ull);
    for (const ChainStrand &st : strands) {
        key.push_back(st.k_row); key.push_back(st.v_row);
        key.push_back(((uint64_t)st.cap << 32) | st.len);
        key.push_back(((uint64_t)st.row_begin << 32) | st.n_rows);
        key.push_back(st.key_first);
    }
    PlanSlot *cur = ctx->cur_slot >= 0 ? &ctx->slots[ctx->cur_slot] : nullptr;
    PlanSlot *sl = nullptr;
    if (cur && cur->chain && cur->chain_key == key) {
        sl = cur;
    } else {
        if (cur && (cur->valid || cur->chain)) {
            CART_CUDA(ctx, cudaEventRecord(cur->ev, cur->last_stream));
            cur->ev_recorded = true;
        }
        const int next = (ctx->cur_slot + 1) % kPlanSlots;
        PlanSlot &ns = ctx->slots[next];
        if (ns.ev_recorded) {
            CART_CUDA(ctx, cudaEventSynchronize(ns.ev));
            ns.ev_recorded = false;
        }
        ns.valid = false;
        ns.chain = false;
        ns.epoch = 0;

        uint32_t part_tiles = 0;
        for (const ChainPart &pt : parts) part_tiles += (pt.p + 127u) / 128u;
        // keys of strand c that the rows of [a, b) need: up to the last of its rows in the tile
        auto needed = [&](const ChainStrand &st, uint32_t b) {
            const uint32_t last_row = std::min(b, st.row_begin + st.n_rows) - 1u;
            return st.key_first + (last_row - st.row_begin) + 1u;
        };
        std::vector<cart_shared_unit> &units = ctx->unit_tmp;
        std::vector<uint32_t> &piece_of_rt = ctx->piece_tmp;   // pieces of M-tile rt's chains (the same for every KV head)
        std::vector<uint32_t> chain_start;                     // index in `units` of every chain's (piece's) first unit
        units.clear();
        piece_of_rt.assign(n_rt, 1u);
        std::vector<cart_shared_unit> cu;   // the units of one chain before it is cut
        std::vector<uint32_t> cuts;
        int32_t c0 = 0;
        for (int g = 0; g < Hkv; ++g) {
            c0 = 0;
            for (uint32_t rt = 0; rt < n_rt; ++rt) {
                const uint32_t a = rt * tpt, b = std::min(T, a + tpt);
                while (strands[(size_t)c0].row_begin + strands[(size_t)c0].n_rows <= a) ++c0;
                int32_t c_last = c0;
                while (c_last + 1 < n_strands && strands[(size_t)c_last + 1].row_begin < b) ++c_last;
                cu.clear();
                for (const ChainPart &pt : parts) {
                    cart_shared_unit u{};
                    u.k_row = (uint32_t)(pt.k_row + (uint64_t)g * pt.p);
                    u.v_row = (uint32_t)(pt.v_row + (uint64_t)g * pt.p);
                    u.layer_stride = (uint32_t)Hkv * pt.p;
                    u.n_tiles = (pt.p + 127u) / 128u;
                    u.flags = (pt.p % 128u) ? CART_UNIT_MASKED : 0;
                    u.lim_base = (int32_t)pt.p - 1;
                    u.lim_cap = (int32_t)pt.p - 1;
                    u.tr_hi = tpt;
                    cu.push_back(u);
                }
                for (int32_t c = c0; c <= c_last; ++c) {
                    const ChainStrand &st = strands[(size_t)c];
                    cart_shared_unit u{};
                    u.k_row = (uint32_t)(st.k_row + (uint64_t)g * st.cap);
                    u.v_row = (uint32_t)(st.v_row + (uint64_t)g * st.cap);
                    u.layer_stride = (uint32_t)((uint64_t)Hkv * st.cap);
                    u.n_tiles = (needed(st, b) + 127u) / 128u;
                    u.flags = CART_UNIT_MASKED | CART_UNIT_SUFFIX;
                    // token offset 0 of the M-tile is the strand's row a - row_begin (negative: the strand starts inside the tile)
                    u.lim_base = (int32_t)st.key_first + ((int32_t)a - (int32_t)st.row_begin);
                    u.lim_cap = (int32_t)st.len - 1;                   // the strand's last stored key
                    u.tr_hi = st.row_begin + st.n_rows - a;            // tokens from here on belong to later strands
                    cu.push_back(u);
                }
                uint32_t total = 0;
                for (const cart_shared_unit &u : cu) total += u.n_tiles;
                // where the chain is cut: piece k starts at tile cuts[k] of the chain
                cuts.assign(1, 0u);
                if (n_split > 1u) {
                    const uint32_t safe = part_tiles + (uint32_t)std::max(cu.back().lim_base, 0) / 128u;
                    for (uint32_t k = 1; k < n_split; ++k) {
                        const uint32_t at = std::min((uint32_t)((uint64_t)k * total / n_split), safe);
                        if (at > cuts.back() && at < total) cuts.push_back(at);
                    }
                }
                piece_of_rt[rt] = (uint32_t)cuts.size();
                cuts.push_back(total);
                for (size_t k = 0; k + 1 < cuts.size(); ++k) {
                    const uint32_t lo = cuts[k], hi = cuts[k + 1];
                    chain_start.push_back((uint32_t)units.size());
                    uint32_t u0 = 0;
                    bool first = true;
                    for (const cart_shared_unit &src : cu) {
                        const uint32_t u1 = u0 + src.n_tiles;
                        const uint32_t x = std::max(lo, u0), y = std::min(hi, u1);
                        if (x < y) {
                            cart_shared_unit u = src;
                            const uint32_t skip = (x - u0) * 128u;   // keys of the unit that earlier pieces hold
                            u.k_row += skip;
                            u.v_row += skip;
                            u.lim_base -= (int32_t)skip;
                            u.lim_cap -= (int32_t)skip;
                            u.n_tiles = y - x;
                            u.reader_begin = a;
                            u.n_readers = b - a;
                            u.kv_head = (uint16_t)g;
                            u.chunk = (uint32_t)k;
                            u.reserved = 0;
                            if (!first) u.flags |= CART_UNIT_CONT;
                            if (y < hi) u.flags |= CART_UNIT_HOLD;
                            else if (n_split == 1u) u.flags |= CART_UNIT_DIRECT;
                            first = false;
                            units.push_back(u);
                        }
                        u0 = u1;
                    }
                }
            }
        }
        const size_t nu = units.size();
        // a chain's first unit names the distance to the next chain (the kernel fetches that chain's query rows ahead)
        for (size_t i = 0; i < chain_start.size(); ++i)
            units[chain_start[i]].reserved = i + 1 < chain_start.size() ? chain_start[i + 1] - chain_start[i] : 0u;
        // a chain goes to the block whose share of the tiles it starts in (chains of unequal length, no more of them
        // than blocks, would leave some blocks with two and others with none that way: then every chain gets a block)
        uint64_t total_tiles = 0;
        for (const cart_shared_unit &u : units) total_tiles += u.n_tiles;
        const uint32_t n_blocks = (uint32_t)std::min<uint64_t>((uint64_t)ctx->n_cta, (uint64_t)chain_start.size());
        const uint32_t n_merges = n_split > 1u ? T * (uint32_t)Hkv : 0u;
        // the buffer's layout
        auto up = [](uint64_t x) { return (x + 63u) & ~63ull; };
        const uint64_t off_ucb = lay.shared_off;
        const uint64_t off_readers = up(off_ucb + (uint64_t)(n_blocks + 1u) * 4u);
        const uint64_t off_rslot = up(off_readers + (uint64_t)T * 4u);
        const uint64_t off_rmerge = up(off_rslot + (uint64_t)n_merges * 4u);
        const uint64_t off_merges = up(off_rmerge + (uint64_t)n_merges * 4u);
        const uint64_t off_units = up(off_merges + (uint64_t)n_merges * sizeof(cart_merge_item));
        const uint64_t end = off_units + (uint64_t)nu * sizeof(cart_shared_unit);
        if (end > lay.plan_slot_bytes) return fail(ctx, CART_ERR_CAPACITY, "chains: the plan of %u rows does not fit its buffer", T);
        if ((uint64_t)n_merges * n_split > (uint64_t)lay.slots_cap)
            return fail(ctx, CART_ERR_CAPACITY, "chains: %u rows in %u pieces exceed the partial slots", T, n_split);
        uint32_t *unit_cta_begin = reinterpret_cast<uint32_t *>(ns.host + off_ucb);
        uint32_t *readers = reinterpret_cast<uint32_t *>(ns.host + off_readers);
        uint32_t blk = 0;
        uint64_t given = 0;
        unit_cta_begin[0] = 0;
        const bool one_each = chain_start.size() <= (size_t)n_blocks;   // no more chains than blocks: a block each
        for (size_t i = 0; i < chain_start.size(); ++i) {
            while (blk + 1 < n_blocks && (one_each ? (size_t)blk < i : given * n_blocks >= (uint64_t)(blk + 1) * total_tiles))
                unit_cta_begin[++blk] = chain_start[i];
            const size_t e = i + 1 < chain_start.size() ? chain_start[i + 1] : nu;
            for (size_t j = chain_start[i]; j < e; ++j) given += units[j].n_tiles;
        }
        while (blk < n_blocks) unit_cta_begin[++blk] = (uint32_t)nu;
        for (uint32_t t = 0; t < T; ++t) readers[t] = t;   // reader entry t = query row t
        if (n_split > 1u) {
            uint32_t *rslot = reinterpret_cast<uint32_t *>(ns.host + off_rslot);
            uint32_t *rmerge = reinterpret_cast<uint32_t *>(ns.host + off_rmerge);
            cart_merge_item *merges = reinterpret_cast<cart_merge_item *>(ns.host + off_merges);
            for (uint32_t t = 0; t < T; ++t)
                for (uint32_t g = 0; g < (uint32_t)Hkv; ++g) {
                    const uint32_t rg = t * (uint32_t)Hkv + g;
                    rslot[rg] = rg * n_split;
                    rmerge[rg] = rg;
                    merges[rg] = cart_merge_item{rg, rg * n_split, rg * n_split + piece_of_rt[t / tpt], 0u};
                }
        }
        std::memcpy(ns.host + off_units, units.data(), nu * sizeof(cart_shared_unit));
        CART_CUDA(ctx, cudaMemcpyAsync(ns.dev + off_ucb, ns.host + off_ucb, end - off_ucb, cudaMemcpyHostToDevice, s));
        ns.chain = true;
        ns.chain_key = key;
        ns.chain_blocks = n_blocks;
        ns.chain_merges = n_merges;
        ns.chain_off[0] = off_ucb; ns.chain_off[1] = off_readers; ns.chain_off[2] = off_rslot;
        ns.chain_off[3] = off_rmerge; ns.chain_off[4] = off_merges; ns.chain_off[5] = off_units;
        ++ctx->plans_built;
        ctx->cur_slot = next;
        sl = &ns;
    }
    sl->last_stream = s;

    uint8_t *arena = static_cast<uint8_t *>(ctx->cfg.arena);
    SharedParams sp;
    sp.unit_cta_begin = reinterpret_cast<const uint32_t *>(sl->dev + sl->chain_off[0]);
    sp.readers = reinterpret_cast<const uint32_t *>(sl->dev + sl->chain_off[1]);
    sp.reader_slot = reinterpret_cast<const uint32_t *>(sl->dev + sl->chain_off[2]);
    sp.reader_merge = reinterpret_cast<const uint32_t *>(sl->dev + sl->chain_off[3]);
    sp.merges = reinterpret_cast<const cart_merge_item *>(sl->dev + sl->chain_off[4]);
    sp.units = reinterpret_cast<const cart_shared_unit *>(sl->dev + sl->chain_off[5]);
    sp.q = q;
    sp.out = out;
    sp.lse = lse;
    sp.part_o = reinterpret_cast<float *>(arena + lay.part_o_off);
    sp.part_lse2 = reinterpret_cast<float *>(arena + lay.part_lse_off);
    sp.tickets = nullptr;
    sp.status = reinterpret_cast<uint32_t *>(arena + lay.status_off);
    sp.layer = layer;
    sp.group = G;
    sp.n_kv_heads = Hkv;
    sp.n_q_heads = ctx->cfg.n_q_heads;
    sp.scale_log2 = ctx->scale * 1.4426950408889634f;
    sp.pages = nullptr;
    CART_CUDA(ctx, launch_shared(ctx->tmap, sp, (int)sl->chain_blocks, s, true));
    ++ctx->launches;
    if (sl->chain_merges > 0) {
        MergeParams mp;
        mp.merges = sp.merges;
        mp.part_o = sp.part_o;
        mp.part_lse2 = sp.part_lse2;
        mp.out = out;
        mp.lse = lse;
        mp.group = G;
        CART_CUDA(ctx, launch_merge(mp, (int)sl->chain_merges, s));
        ++ctx->launches;
    }
    CART_CUDA(ctx, cudaEventRecord(sl->ev, s));   // whoever takes this buffer next waits for these launches
    sl->ev_recorded = true;
    return CART_OK;
}

}  // namespace

extern "C" {

cart_status cart_train_attention_fwd(cart_ctx *ctx, int32_t layer, const cart_req *convs, int32_t n_convs, const void *q,
                                     void *out, float *lse, void *stream)
{
    if (!ctx) return CART_ERR_INVALID_ARG;
    if (!lse) return fail(ctx, CART_ERR_INVALID_ARG, "train: the forward must write lse");
    TrainBatch tb;
    const cart_status st = train_batch(ctx, layer, convs, n_convs, &tb);
    if (st != CART_OK) return st;
    if (!aligned16(q) || !aligned16(out)) return fail(ctx, CART_ERR_INVALID_ARG, "train: null/misaligned pointer");
    std::vector<ChainPart> parts;
    if (tb.z) parts.push_back(ChainPart{tb.z->k_row, tb.z->v_row, (uint32_t)tb.z->p});
    std::vector<ChainStrand> strands;
    for (int32_t c = 0; c < n_convs; ++c) {
        const Request &r = ctx->reqs[(size_t)convs[c]];
        strands.push_back(ChainStrand{r.k_row, r.v_row, (uint32_t)r.cap, (uint32_t)tb.len[(size_t)c],
                                      (uint32_t)tb.cu[(size_t)c], (uint32_t)tb.len[(size_t)c], 0u});
    }
    return launch_chains(ctx, layer, parts, strands, (uint32_t)tb.T, q, out, lse, static_cast<cudaStream_t>(stream));
}

cart_status cart_train_attention_bwd(cart_ctx *ctx, int32_t layer, const cart_req *convs, int32_t n_convs, const void *q,
                                     const void *out, const float *lse, const void *dout, float *delta, float *dq, float *dk,
                                     float *dv, float *dzk, float *dzv, void *stream)
{
    if (!ctx) return CART_ERR_INVALID_ARG;
    TrainBatch tb;
    cart_status st = train_batch(ctx, layer, convs, n_convs, &tb);
    if (st != CART_OK) return st;
    if (!aligned16(q) || !aligned16(out) || !aligned16(dout) || !aligned16(dq) || !aligned16(dk) || !aligned16(dv) || !lse ||
        !delta || (tb.z && (!aligned16(dzk) || !aligned16(dzv))))
        return fail(ctx, CART_ERR_INVALID_ARG, "train: null/misaligned pointer");
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int Hkv = ctx->cfg.n_kv_heads, Hq = ctx->cfg.n_q_heads, G = ctx->group;
    const uint32_t tpt = 128u / (uint32_t)G;
    const uint32_t T = (uint32_t)tb.T;
    const uint32_t n_rt = (T + tpt - 1) / tpt;
    const uint32_t p = tb.z ? (uint32_t)tb.z->p : 0u;

    // ---- work items: Cartridge tiles first (long), then the conversations' own key tiles ------------
    // They go through the next buffer of the plan ring (a decode plan kept there is dropped).
    PlanSlot *cur = ctx->cur_slot >= 0 ? &ctx->slots[ctx->cur_slot] : nullptr;
    if (cur && cur->valid) {
        CART_CUDA(ctx, cudaEventRecord(cur->ev, cur->last_stream));
        cur->ev_recorded = true;
    }
    const int next = (ctx->cur_slot + 1) % kPlanSlots;
    PlanSlot &ns = ctx->slots[next];
    if (ns.ev_recorded) {
        CART_CUDA(ctx, cudaEventSynchronize(ns.ev));
        ns.ev_recorded = false;
    }
    ns.valid = false;
    ns.chain = false;
    TrainItem *items = reinterpret_cast<TrainItem *>(ns.host + ctx->lay.items_off);
    const size_t items_cap = (size_t)ctx->lay.items_cap * sizeof(cart_work_item) / sizeof(TrainItem);
    size_t n_items = 0;
    const uint32_t z_tiles = (p + 127u) / 128u;
    // a Cartridge tile's rows are divided among several blocks when there are fewer tiles than SMs
    uint32_t nsplit = 1;
    if (z_tiles > 0) nsplit = std::max<uint32_t>(1u, std::min<uint32_t>(n_rt, (uint32_t)ctx->n_cta / (z_tiles * (uint32_t)Hkv)));
    bool full = false;
    auto push = [&](const TrainItem &ti) {
        if (n_items >= items_cap) { full = true; return; }
        items[n_items++] = ti;
    };
    for (uint32_t zt = 0; zt < z_tiles; ++zt)
        for (int g = 0; g < Hkv; ++g)
            for (uint32_t sp = 0; sp < nsplit; ++sp) {
                TrainItem ti{};
                ti.k_row = (uint32_t)(tb.z->k_row + (uint64_t)g * p + zt * 128u);
                ti.v_row = (uint32_t)(tb.z->v_row + (uint64_t)g * p + zt * 128u);
                ti.layer_stride = (uint32_t)Hkv * p;
                ti.n_keys = std::min(128u, p - zt * 128u);
                ti.kv_head = (uint32_t)g;
                ti.rt_begin = (uint32_t)((uint64_t)n_rt * sp / nsplit);
                ti.rt_end = (uint32_t)((uint64_t)n_rt * (sp + 1) / nsplit);
                if (ti.rt_end == ti.rt_begin) continue;
                // blocks that add into the same rows of dq (the tiles of one KV head) start at different row tiles
                ti.rt_first = ti.rt_begin + (zt * 5u) % (ti.rt_end - ti.rt_begin);
                ti.key_tok0 = 0;
                ti.tok_end = T;
                ti.causal = 0;
                ti.dst_row = (uint32_t)g * p + zt * 128u;
                ti.dst_stride = 1;
                ti.is_z = 1;
                push(ti);
            }
    for (int32_t c = 0; c < n_convs; ++c) {
        const Request &r = ctx->reqs[(size_t)convs[c]];
        const uint32_t n = (uint32_t)tb.len[(size_t)c], t0 = (uint32_t)tb.cu[(size_t)c], t1 = (uint32_t)tb.cu[(size_t)c + 1];
        for (uint32_t kc = 0; kc * 128u < n; ++kc)
            for (int g = 0; g < Hkv; ++g) {
                TrainItem ti{};
                ti.k_row = (uint32_t)(r.k_row + (uint64_t)g * r.cap + kc * 128u);
                ti.v_row = (uint32_t)(r.v_row + (uint64_t)g * r.cap + kc * 128u);
                ti.layer_stride = (uint32_t)((uint64_t)Hkv * r.cap);
                ti.n_keys = std::min(128u, n - kc * 128u);
                ti.kv_head = (uint32_t)g;
                ti.key_tok0 = t0 + kc * 128u;
                ti.tok_end = t1;
                ti.rt_begin = ti.key_tok0 / tpt;
                ti.rt_end = (t1 + tpt - 1) / tpt;
                ti.rt_first = ti.rt_begin;
                ti.causal = 1;
                ti.dst_row = ti.key_tok0 * (uint32_t)Hkv + (uint32_t)g;
                ti.dst_stride = (uint32_t)Hkv;
                ti.is_z = 0;
                push(ti);
            }
    }
    if (full) return fail(ctx, CART_ERR_CAPACITY, "train: more than %zu work items", items_cap);
    uint8_t *dev_items = ns.dev + ctx->lay.items_off;
    CART_CUDA(ctx, cudaMemcpyAsync(dev_items, items, n_items * sizeof(TrainItem), cudaMemcpyHostToDevice, s));
    ns.last_stream = s;
    ns.epoch = 0;
    ctx->cur_slot = next;
    CART_CUDA(ctx, cudaEventRecord(ns.ev, s));  // (recorded again below, after the kernels)
    ns.ev_recorded = true;

    // ---- q and dout as [T][Hq][128], fetched in boxes of 128 / G tokens x G heads x 64 dims -----------
    alignas(64) CUtensorMap tmap_q, tmap_do, tmap_dq;
    {
        const cuuint64_t gdim[3] = {(cuuint64_t)kHeadDim, (cuuint64_t)Hq, (cuuint64_t)T};
        const cuuint64_t gstride[2] = {(cuuint64_t)kRowBytes, (cuuint64_t)Hq * kRowBytes};
        const cuuint32_t box[3] = {64u, (cuuint32_t)G, (cuuint32_t)tpt};
        const cuuint32_t estride[3] = {1u, 1u, 1u};
        EncodeFn enc = reinterpret_cast<EncodeFn>(ctx->encode_fn);
        CUresult r1 = enc(&tmap_q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(q), gdim, gstride, box, estride,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        CUresult r2 = enc(&tmap_do, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(dout), gdim, gstride, box, estride,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        // dq as fp32 [T][Hq][128]: boxes of 128 / G tokens x G heads x 32 dims (128 bytes, the swizzle's span)
        const cuuint64_t dstride[2] = {(cuuint64_t)kHeadDim * 4, (cuuint64_t)Hq * kHeadDim * 4};
        const cuuint32_t dbox[3] = {32u, (cuuint32_t)G, (cuuint32_t)tpt};
        CUresult r3 = enc(&tmap_dq, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 3, dq, gdim, dstride, dbox, estride,
                          CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                          CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r1 != CUDA_SUCCESS || r2 != CUDA_SUCCESS || r3 != CUDA_SUCCESS)
            return fail(ctx, CART_ERR_CUDA, "train: cuTensorMapEncodeTiled failed with code %d",
                        (int)(r1 != CUDA_SUCCESS ? r1 : r2 != CUDA_SUCCESS ? r2 : r3));
    }
    // ---- zero the outputs (they are accumulated into), D, then the kernel ----------------------------
    CART_CUDA(ctx, cudaMemsetAsync(dq, 0, (size_t)T * Hq * kHeadDim * 4, s));
    CART_CUDA(ctx, cudaMemsetAsync(dk, 0, (size_t)T * Hkv * kHeadDim * 4, s));
    CART_CUDA(ctx, cudaMemsetAsync(dv, 0, (size_t)T * Hkv * kHeadDim * 4, s));
    if (tb.z) {
        CART_CUDA(ctx, cudaMemsetAsync(dzk, 0, (size_t)Hkv * p * kHeadDim * 4, s));
        CART_CUDA(ctx, cudaMemsetAsync(dzv, 0, (size_t)Hkv * p * kHeadDim * 4, s));
    }
    TrainDeltaParams dpm;
    dpm.out = out;
    dpm.dout = dout;
    dpm.delta = delta;
    dpm.n_rows = (int32_t)(T * (uint32_t)Hq);
    CART_CUDA(ctx, launch_train_delta(dpm, s));
    ++ctx->launches;
    TrainBwdParams bp;
    bp.items = reinterpret_cast<const TrainItem *>(dev_items);
    bp.lse = lse;
    bp.delta = delta;
    bp.dq = dq;
    bp.dk = dk;
    bp.dv = dv;
    bp.dzk = dzk;
    bp.dzv = dzv;
    bp.status = reinterpret_cast<uint32_t *>(static_cast<uint8_t *>(ctx->cfg.arena) + ctx->lay.status_off);
    bp.layer = layer;
    bp.group = G;
    bp.n_q_heads = Hq;
    bp.n_tokens = (int32_t)T;
    bp.scale = ctx->scale;
    CART_CUDA(ctx, launch_train_bwd(ctx->tmap, tmap_q, tmap_do, tmap_dq, bp, (int)n_items, s));
    ++ctx->launches;
    CART_CUDA(ctx, cudaEventRecord(ns.ev, s));
    ns.ev_recorded = true;
    return CART_OK;
}

cart_status cart_suffix_len(cart_ctx *ctx, cart_req req, int32_t layer, int32_t *out_len)
{
    if (!ctx) return CART_ERR_INVALID_ARG;
    if (!out_len) return fail(ctx, CART_ERR_INVALID_ARG, "suffix_len: null out");
    Request *r = get_req(ctx, req);
    if (!r || layer < 0 || layer >= ctx->cfg.n_layers) return fail(ctx, CART_ERR_BAD_HANDLE, "suffix_len: bad handle");
    *out_len = r->len[(size_t)layer];
    return CART_OK;
}

cart_status cart_kv_bytes(cart_ctx *ctx, cart_req req, uint64_t *logical, uint64_t *unique_private)
{
    if (!ctx) return CART_ERR_INVALID_ARG;
    if (!logical || !unique_private) return fail(ctx, CART_ERR_INVALID_ARG, "kv_bytes: null out");
    Request *r = get_req(ctx, req);
    if (!r) return fail(ctx, CART_ERR_BAD_HANDLE, "kv_bytes: not an open request");
    const uint64_t per_token = 2ull * ctx->cfg.n_kv_heads * kRowBytes;  // K and V, all KV heads, one layer
    uint64_t suffix = 0;
    for (int32_t l : r->len) suffix += (uint64_t)l;
    const uint64_t cart_tokens = r->cart == CART_NONE ? 0ull : (uint64_t)ctx->carts[(size_t)r->cart].p;
    *unique_private = suffix * per_token;
    *logical = (cart_tokens * (uint64_t)ctx->cfg.n_layers + suffix) * per_token;
    return CART_OK;
}

cart_status cart_sync_status(cart_ctx *ctx, void *stream)
{
    if (!ctx) return CART_ERR_INVALID_ARG;
    CART_CUDA(ctx, cudaStreamSynchronize(static_cast<cudaStream_t>(stream)));
    uint32_t word = 0;
    uint8_t *st = static_cast<uint8_t *>(ctx->cfg.arena) + ctx->lay.status_off;
    CART_CUDA(ctx, cudaMemcpy(&word, st, 4, cudaMemcpyDeviceToHost));
    if (word != 0) {
        // a block that gave up may have left arrival tickets behind: clear them with the word
        CART_CUDA(ctx, cudaMemset(st, 0, ctx->lay.plan_off));
        return fail(ctx, CART_ERR_TIMEOUT, "a device-side wait ran out (status word 0x%x)", word);
    }
    return CART_OK;
}

}  // extern "C"
