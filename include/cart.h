/*
 * cart.h -- C ABI of the B200 Cartridge decode-attention library (libcart.so).
 *
 * The library serves the attention part of decoding with Cartridges (arXiv 2506.06266): every
 * request attends over a trained, compact KV cache (a Cartridge of p key/value tokens per layer,
 * Sec. 3.2; possibly several Cartridges concatenated, Sec. 3.1 / Sec. 5.4; possibly shared by many
 * requests and stored once) followed by the request's own growing suffix KV (Sec. 2.3): a Cartridge is
 * served like a cached prefix of p tokens (Sec. 3.3).
 *
 * Conventions that hold for every entry point
 *   - Returns a cart_status.  Out-parameters are written only on CART_OK.  Nothing throws, aborts
 *     or exits.  cart_last_error(ctx) gives a one-line reason for the last failure on that context.
 *   - Arguments are validated on the host before anything is launched; a failing call changes no
 *     state.
 *   - "device" pointers are CUDA device pointers on the context's device; "host" pointers are
 *     ordinary host memory.  Each parameter says which.
 *   - All device memory comes from the caller: the arena handed to cart_create and the q / k / v /
 *     out tensors passed per call.  The library itself never allocates device memory.  The arena
 *     stays owned by the caller and must outlive the context.
 *   - Calls that take a stream enqueue work on it and return without synchronising the stream or the
 *     device, with one bounded exception: the attention calls keep their work lists (plans) in a ring of
 *     four device buffers, and a call that has to build a new plan first waits on the host until the
 *     kernels that used the buffer three plans back have finished (back-pressure; in a decode loop a
 *     plan is kept for many steps, so this wait is rare and normally already satisfied).  A context is
 *     meant to be driven from one host thread on one stream at a time; to switch streams the caller
 *     orders them (event or synchronise).  Capturing calls into a CUDA graph is not supported: lengths and
 *     plans live on the host and change from call to call.
 *   - Tensors are bf16 (upper half of IEEE binary32), head_dim = 128, dense row-major in the stated
 *     index order.  Device tensor pointers must be 16-byte aligned.
 *   - Query head h reads KV head h / (n_q_heads / n_kv_heads) (contiguous groups).
 *   - Keys are stored as given (already position-encoded by the caller); the library applies no
 *     positional transform and no causal mask: the single decode query of a request sees its whole
 *     cache [Cartridge(s) ; suffix].
 */
#ifndef CART_H_
#define CART_H_

#include <stdint.h>

#if defined(__GNUC__)
#define CART_API __attribute__((visibility("default")))
#else
#define CART_API
#endif

#ifdef __cplusplus
extern "C" {
#endif

typedef struct cart_ctx cart_ctx; /* opaque */
typedef int32_t cart_id;          /* Cartridge handle (registered or composed) */
typedef int32_t cart_req;         /* request handle (owns one suffix KV buffer) */
#define CART_NONE (-1)            /* "no Cartridge": the request attends to its suffix only */

typedef enum {
    CART_OK = 0,
    CART_ERR_INVALID_ARG = 1, /* NULL / misaligned pointer, negative size, bad flag */
    CART_ERR_SHAPE = 2,       /* head_dim != 128, n_q_heads not a multiple of n_kv_heads, group > 8 */
    CART_ERR_BAD_HANDLE = 3,  /* unknown, closed or released handle; layer out of range */
    CART_ERR_CAPACITY = 4,    /* suffix buffer full, handle table full, too many parts */
    CART_ERR_OOM = 5,         /* the arena has no room left */
    CART_ERR_EMPTY = 6,       /* a request has no KV token at all in the layer asked for */
    CART_ERR_IN_USE = 7,      /* releasing a Cartridge that an open request or composition uses */
    CART_ERR_CUDA = 8,        /* a CUDA runtime / driver call failed (see cart_last_error) */
    CART_ERR_TIMEOUT = 9,     /* a bounded device-side wait ran out (reported by cart_sync_status) */
    CART_ERR_EVICTED = 10     /* the request, or a Cartridge it attends to, is swapped out of the arena */
} cart_status;

typedef struct {
    int32_t n_layers;       /* L >= 1 */
    int32_t n_q_heads;      /* Hq */
    int32_t n_kv_heads;     /* Hkv; Hq % Hkv == 0 and Hq / Hkv <= 8 */
    int32_t head_dim;       /* must be 128 */
    int32_t max_requests;   /* size of the request table (>= 1) */
    int32_t max_cartridges; /* size of the Cartridge table, compositions included (>= 1) */
    int32_t max_parts;      /* most registered Cartridges one composition may hold; 0 => 8 */
    float softmax_scale;    /* multiplies q.k before the softmax; 0 => 1/sqrt(head_dim) (Eq. 1) */
    void *arena;            /* device; 256-byte aligned; holds every Cartridge, suffix and scratch */
    uint64_t arena_bytes;
    int32_t device;         /* CUDA device ordinal the arena lives on */
} cart_config;

/* Bytes of the arena the library reserves for its own scratch (work lists, split partials) under
 * this configuration; the rest is available to Cartridges and suffix buffers.  Pure host
 * arithmetic, needs no device.  *out_bytes is a multiple of 256. */
CART_API cart_status cart_scratch_bytes(const cart_config *cfg /*host*/, uint64_t *out_bytes /*host*/);

/* Creates a context on cfg->device over the caller's arena.  Makes cfg->device current, builds the
 * tensor map the kernels use to fetch KV tiles from the arena, allocates small pinned host staging
 * buffers.  Errors: INVALID_ARG, SHAPE, OOM (arena smaller than the scratch), CUDA. */
CART_API cart_status cart_create(const cart_config *cfg /*host*/, cart_ctx **out /*host*/);

/* Synchronises the device, frees host-side state.  The arena is untouched.  NULL is accepted. */
CART_API cart_status cart_destroy(cart_ctx *ctx);

/* Sec. 3.2 / Sec. 3.3: make a trained Cartridge resident in the KV cache and addressable by handle.  k and v are bf16 [n_layers][n_kv_heads][p][128], in device memory or in host
 * memory (a Cartridge loaded from disk and swapped in while other requests decode: page-locked host
 * memory makes the copy asynchronous); they are copied into the arena on `stream` (the caller may free
 * or reuse them once the stream has passed this point).  p >= 1, the same in every layer.  A Cartridge
 * is stored once however many requests open on it; cart_release_cartridge gives its space back.
 * The Cartridge is always copied: every tile of the arena is fetched through one tensor map, and a block left in
 * the caller's memory would need a map of its own in every kernel, so borrowing a caller's buffer is not offered (a
 * cache too large to hold twice is registered from host memory, or in parts that are then composed).
 * Errors: INVALID_ARG, CAPACITY (table full), OOM, CUDA. */
CART_API cart_status cart_register_cartridge(cart_ctx *ctx, const void *k /*device or host*/, const void *v /*device or host*/,
                                    int32_t p, void *stream /*cudaStream_t*/, cart_id *out /*host*/);

/* Composition (Sec. 3.1, Sec. 5.4): the handle returned stands for the concatenation
 * [Z_1, Z_2, ...] of the parts along the token axis, in list order, with no retraining, no copy and
 * no re-encoding of positions.  Parts may themselves be compositions (flattened).  The parts stay
 * referenced until the composition is released.  parts is a host array.
 * Errors: INVALID_ARG (n_parts < 1), BAD_HANDLE, CAPACITY (more than max_parts registered parts
 * after flattening, or table full). */
CART_API cart_status cart_compose(cart_ctx *ctx, const cart_id *parts /*host*/, int32_t n_parts,
                         cart_id *out /*host*/);

/* Drops a Cartridge or composition.  Its arena space becomes reusable for later registrations; the
 * caller makes sure no enqueued decode still reads it.  Errors: BAD_HANDLE, IN_USE. */
CART_API cart_status cart_release_cartridge(cart_ctx *ctx, cart_id id);

/* Opens a request that attends to `cartridge` (or CART_NONE) followed by its own suffix, and
 * reserves a suffix buffer of suffix_capacity tokens per layer in the arena (Sec. 3.3: per-user KV
 * caches next to the shared prefix).  suffix_capacity >= 0; it is rounded up to a multiple of 64.
 * Errors: BAD_HANDLE, CAPACITY (table full), OOM. */
CART_API cart_status cart_request_open(cart_ctx *ctx, cart_id cartridge, int32_t suffix_capacity,
                              cart_req *out /*host*/);

/* The same with the suffix stored in pages (Sec. 3.3: a Cartridge is served by the mechanisms that handle cached
 * prefixes and per-user KV caches; paging is how such caches grow without being moved).  A page holds CART_PAGE_TOKENS
 * tokens of the request for every layer and KV head -- per (layer, KV head) the K rows, then the V rows -- and may lie
 * anywhere in the arena; the attention kernels find a tile through the request's page list.  initial_capacity tokens
 * (rounded up to whole pages, may be 0) are reserved now; cart_append_kv, cart_extend_kv and cart_decode_step take
 * further pages from the arena as the suffix grows (CART_ERR_OOM when none is left; nothing is appended then), and
 * cart_request_reserve takes pages instead of copying.  Pages return to the arena with cart_request_close or
 * cart_evict_request.  Everything else is as for cart_request_open; results are bitwise those of a request with a
 * contiguous suffix.  One attention call may name at most 256 * max_requests + 8192 pages over its whole batch
 * (CART_ERR_CAPACITY beyond).  Errors: BAD_HANDLE, CAPACITY (table full), OOM. */
#define CART_PAGE_TOKENS 64
CART_API cart_status cart_request_open_paged(cart_ctx *ctx, cart_id cartridge, int32_t initial_capacity,
                                             cart_req *out /*host*/);

/* Grows the suffix buffer of an open request to at least suffix_capacity tokens per layer (rounded up
 * to a multiple of 64), for conversations that outlive the capacity they were opened with (Sec. 3.3:
 * per-user KV caches of any length next to the shared prefix).  A new buffer is taken from the arena,
 * the tokens stored so far are copied into it on `stream` (device to device, one strided copy for K and
 * one for V), and the old buffer returns to the arena; decode calls enqueued on the same stream before
 * the call still read the old buffer, later ones the new.  A capacity not above the current one
 * changes nothing.  The arena must have room for the new buffer while the old one is still held.
 * Errors: BAD_HANDLE, INVALID_ARG, OOM (nothing has changed), CUDA. */
CART_API cart_status cart_request_reserve(cart_ctx *ctx, cart_req req, int32_t suffix_capacity, void *stream);

/* Eviction (Sec. 3.3: many users' caches share one GPU; a scheduler keeps the active ones resident).
 *
 * cart_evict_request swaps a paused request's suffix out: the tokens stored so far are copied on `stream` to k_out /
 * v_out (host memory -- page-locked makes the copy asynchronous -- or device memory outside the arena), each laid out
 * bf16 [n_layers][n_kv_heads][n][128] with n = *n_tokens_out = the longest layer's length, and the request's pages or
 * buffer return to the arena at once (later calls on the same stream may reuse them; the caller orders other
 * streams).  The handle stays open and keeps its lengths; until it is restored, every call that would read or write
 * its suffix returns CART_ERR_EVICTED.  With n = 0 nothing is copied and k_out / v_out may be NULL.
 * cart_restore_request takes storage for n tokens again (pages for a paged request, else a buffer of the old
 * capacity) and copies k_in / v_in back (same layout and n as evict returned).
 * Errors: BAD_HANDLE, INVALID_ARG, EVICTED (evict: already out; restore: not out), OOM (restore; nothing changed), CUDA. */
CART_API cart_status cart_evict_request(cart_ctx *ctx, cart_req req, void *k_out /*host or device*/,
                                        void *v_out /*host or device*/, int32_t *n_tokens_out /*host*/, void *stream);
CART_API cart_status cart_restore_request(cart_ctx *ctx, cart_req req, const void *k_in /*host or device*/,
                                          const void *v_in /*host or device*/, void *stream);

/* cart_evict_cartridge returns a registered Cartridge's arena space while its handle, the compositions that contain
 * it and the requests opened on it stay valid.  A Cartridge is never written after registration, so nothing is copied
 * out: the caller restores it from wherever it keeps trained Cartridges.  Refused with CART_ERR_IN_USE while a request
 * that is not itself evicted attends to it (directly or through a composition): evict those requests first.  While
 * it is out, decode and prefill calls on requests that attend to it return CART_ERR_EVICTED.
 * cart_restore_cartridge takes space again and copies k / v in (as cart_register_cartridge; same p).
 * Errors: BAD_HANDLE (also: a composition), IN_USE, EVICTED (as above), OOM, INVALID_ARG, CUDA. */
CART_API cart_status cart_evict_cartridge(cart_ctx *ctx, cart_id id);
CART_API cart_status cart_restore_cartridge(cart_ctx *ctx, cart_id id, const void *k /*device or host*/,
                                            const void *v /*device or host*/, void *stream);

/* Closes a request and returns its suffix buffer to the arena.  Errors: BAD_HANDLE. */
CART_API cart_status cart_request_close(cart_ctx *ctx, cart_req req);

/* Sec. 2.3, decode phase (the new token's key and value join the KV cache): for i < n_reqs, writes token i of k_new / v_new
 * (device bf16 [n_reqs][n_kv_heads][128]) at the end of request reqs[i]'s suffix in `layer`, and
 * advances that length by one.  reqs is a host array; a handle may appear at most once.
 * Errors: INVALID_ARG, BAD_HANDLE, CAPACITY (some suffix is full; nothing is appended), CUDA. */
CART_API cart_status cart_append_kv(cart_ctx *ctx, int32_t layer, const cart_req *reqs /*host*/, int32_t n_reqs,
                           const void *k_new /*device*/, const void *v_new /*device*/, void *stream);

/* Sec. 2.3, prefill of the user's message: appends n_tokens consecutive tokens to one request's
 * suffix in `layer`.  k and v are device bf16 [n_tokens][n_kv_heads][128] (token-major, as a
 * projection over the message's tokens produces them).
 * Errors: INVALID_ARG, BAD_HANDLE, CAPACITY, CUDA. */
CART_API cart_status cart_extend_kv(cart_ctx *ctx, int32_t layer, cart_req req, const void *k /*device*/,
                           const void *v /*device*/, int32_t n_tokens, void *stream);

/* Eq. 1 (Sec. 2.3) at the last position, for a batch: for i < n_reqs and every query head h,
 *     out[i][h] = sum_j softmax_j(scale * <q[i][h], K*_j>) V*_j,   lse[i][h] = ln sum_j exp(scale * <q[i][h], K*_j>)
 * where K*, V* are KV head h / G of request reqs[i]'s cache in `layer`: its Cartridge(s) in
 * composition order, then its suffix (layout of Sec. 3.2).  q and out are device bf16
 * [n_reqs][n_q_heads][128]; lse is device fp32 [n_reqs][n_q_heads] or NULL.  Products and sums are
 * accumulated in fp32; out is rounded to nearest-even bf16.  reqs is a host array (duplicates
 * allowed).  The result does not depend on how the library splits the cache across thread blocks
 * beyond fp32 rounding, and is bitwise reproducible for the same sequence of calls (the split is a
 * function of the batch, its lengths and the plan that was kept, see cart_set_plan_reuse).
 * Errors: INVALID_ARG, BAD_HANDLE, EMPTY, CAPACITY (batch larger than max_requests), CUDA. */
CART_API cart_status cart_decode_attention(cart_ctx *ctx, int32_t layer, const cart_req *reqs /*host*/,
                                  int32_t n_reqs, const void *q /*device*/, void *out /*device*/,
                                  float *lse /*device or NULL*/, void *stream);

/* Sec. 2.3, one decode step of a layer in one call: what cart_append_kv followed by
 * cart_decode_attention computes, with the append done inside the attention kernel (the block that
 * reads the last tile of a request's suffix first writes the new token's K and V rows there), so a
 * step costs one kernel launch less per layer.  k_new / v_new: device bf16 [n_reqs][n_kv_heads][128];
 * q, out, lse as in cart_decode_attention.  A handle may appear at most once in reqs.  On success every
 * request's suffix in `layer` is one token longer and that token has been attended to (Eq. 1 sums
 * over j <= i: the query sees its own position).
 * Errors: those of cart_append_kv and cart_decode_attention; on an error nothing is appended. */
CART_API cart_status cart_decode_step(cart_ctx *ctx, int32_t layer, const cart_req *reqs /*host*/, int32_t n_reqs,
                             const void *k_new /*device*/, const void *v_new /*device*/, const void *q /*device*/,
                             void *out /*device*/, float *lse /*device or NULL*/, void *stream);

/* Sec. 2.3, the decode loop as launches that can be recorded into a CUDA graph.  cart_decode_step does host work
 * every step (it advances the lengths it mirrors and passes the tokens appended since the plan was built as a
 * kernel parameter), so its launches cannot be replayed.  These three calls move that count to device memory:
 *
 *   cart_graph_begin(ctx, reqs, n_reqs, max_steps, stream)
 *       plans the batch once and uploads the plan (not capturable: call it before the capture), clears the device
 *       word that counts the steps, and reserves room for max_steps more tokens per request (paged suffixes take
 *       their pages now).  Every request must hold the same number of tokens in all layers; a handle may appear
 *       once; max_steps <= the plan-reuse limit + 1 (cart_set_plan_reuse; 193 by default).
 *   cart_graph_step(ctx, layer, k_new, v_new, q, out, lse, stream)
 *       what cart_decode_step computes for `layer` of the batch given to cart_graph_begin, in its order; only
 *       kernel launches, so the calls for layers 0 .. n_layers - 1 of ONE step can be captured (stream capture or
 *       explicit nodes) and replayed; after the last layer's kernels a one-thread kernel advances the count.  The
 *       pointers are recorded: refill the same buffers between replays.
 *   cart_graph_end(ctx, steps_run)
 *       host only: the step ran steps_run times (<= max_steps), every request is that much longer in every layer.
 *
 * Between begin and end no other attention, prefill or training call may be made on ctx (it would take the loop's
 * plan: cart_graph_step then returns INVALID_ARG; replays of a recorded step cannot notice), and the requests
 * must not be closed, reserved or evicted.  Running more than max_steps steps writes past the reserved room.
 * Errors: begin: INVALID_ARG, BAD_HANDLE, CAPACITY (room, max_steps), OOM, EVICTED, IN_USE (a loop is open), CUDA;
 * step: INVALID_ARG (no loop open, plan taken, pointers), BAD_HANDLE (layer), CUDA; end: INVALID_ARG. */
CART_API cart_status cart_graph_begin(cart_ctx *ctx, const cart_req *reqs /*host*/, int32_t n_reqs, int32_t max_steps,
                                      void *stream);
CART_API cart_status cart_graph_step(cart_ctx *ctx, int32_t layer, const void *k_new /*device*/, const void *v_new /*device*/,
                                     const void *q /*device*/, void *out /*device*/, float *lse /*device or NULL*/,
                                     void *stream);
CART_API cart_status cart_graph_end(cart_ctx *ctx, int32_t steps_run);

/* Sec. 2.3, prefill of the user's message over a Cartridge: attention for the LAST n_new tokens of
 * request req's suffix in `layer` (append them first with cart_extend_kv).  Row i of q (device bf16
 * [n_new][n_q_heads][128], token-major as the projection produces it) is the query of the i-th new
 * token and attends, per Eq. 1 with its causal sum over j <= i, to the request's Cartridge(s), the
 * suffix tokens before the new ones and the new tokens 0 .. i.  out, lse as in cart_decode_attention,
 * with n_new rows.  A message of 4 tokens or more behind a contiguous suffix of at most 16 k tokens runs on the
 * tensor cores throughout: per group of 128 / (n_q_heads / n_kv_heads) consecutive new tokens and KV head, the
 * Cartridge(s) and the suffix up to the group's last token are read once, the tiles on the causal diagonal masked
 * per row (see cart_set_prefill_split for short messages).  Otherwise, when n_new reaches the sharing threshold,
 * the Cartridge(s) are read once for all rows and the suffix before each group once for that group, and a row
 * reads by itself only the fewer than 128 + 128 / G tokens around the causal diagonal.  n_new <= max_requests.
 * Errors: INVALID_ARG (also: the suffix holds fewer than n_new tokens), BAD_HANDLE, CAPACITY, CUDA. */
CART_API cart_status cart_prefill_attention(cart_ctx *ctx, int32_t layer, cart_req req, const void *q /*device*/,
                                   int32_t n_new, void *out /*device*/, float *lse /*device or NULL*/,
                                   void *stream);

/* Training-time attention over a shared trainable Cartridge.  Self-Study (Sec. 4.2) trains the key and value vectors
 * of a Cartridge (Sec. 3.2: Z holds p trainable key and value vectors per layer and KV head) by back-propagating
 * through attention of many short conversations that all attend to Z; Sec. 6 names shared-prefix attention kernels as
 * the way to make that cheaper.  These two calls are that attention layer, forward and backward.
 *
 * convs: n_convs open requests, all on the same registered Cartridge Z (or all on CART_NONE), with contiguous (not
 * paged) suffix storage; request c's suffix in `layer` holds conversation c's keys and values (cart_extend_kv).  The
 * conversations are packed back to back on one token axis: conversation c owns tokens cu[c] .. cu[c+1] - 1 with cu the
 * running sum of the suffix lengths, T = cu[n_convs] <= max_requests.  Token i of a conversation attends, per Eq. 1
 * (Sec. 2.3) with its causal sum over j <= i, to all of Z and to the conversation's tokens 0 .. i.
 *
 * cart_train_attention_fwd: q device bf16 [T][n_q_heads][128] -> out device bf16 [T][n_q_heads][128] and lse device
 * fp32 [T][n_q_heads] (natural log; required, the backward reads it).  Z is read once per 128 query rows by the
 * tensor-core kernel, whichever conversations the rows belong to.
 *
 * cart_train_attention_bwd: given q, out, lse of the forward and dout (device bf16 [T][n_q_heads][128], the gradient
 * of the loss with respect to out), writes the gradients with respect to q (dq, device fp32 [T][n_q_heads][128]), to
 * the conversations' keys and values (dk, dv, device fp32 [T][n_kv_heads][128], token-major like the tensors
 * cart_extend_kv took) and to the Cartridge (dzk, dzv, device fp32 [n_kv_heads][p][128], summed over all
 * conversations; may be NULL without a Cartridge).  delta is device scratch, fp32 [T][n_q_heads].  All outputs are
 * overwritten.  Products run on the tensor cores in bf16 with fp32 accumulation; sums over blocks use fp32 atomic
 * adds, so the last bits depend on the order of arrival.
 * Errors: INVALID_ARG (also: requests on different Cartridges, a composition, a paged request), BAD_HANDLE, EVICTED,
 * EMPTY (a conversation without tokens), CAPACITY (T > max_requests, or more work items than the scratch holds), CUDA. */
CART_API cart_status cart_train_attention_fwd(cart_ctx *ctx, int32_t layer, const cart_req *convs /*host*/, int32_t n_convs,
                                              const void *q /*device*/, void *out /*device*/, float *lse /*device*/,
                                              void *stream);
CART_API cart_status cart_train_attention_bwd(cart_ctx *ctx, int32_t layer, const cart_req *convs /*host*/, int32_t n_convs,
                                              const void *q /*device*/, const void *out /*device*/,
                                              const float *lse /*device*/, const void *dout /*device*/,
                                              float *delta /*device scratch*/, float *dq /*device*/, float *dk /*device*/,
                                              float *dv /*device*/, float *dzk /*device or NULL*/,
                                              float *dzv /*device or NULL*/, void *stream);

/* Sharing policy.  When at least min_readers requests of a decode batch attend to the same stored
 * Cartridge (one Cartridge serving many users, Sec. 1 and Sec. 3.3; pool members composed by many
 * requests, Sec. 5.4), cart_decode_attention reads each of its K/V tiles once for up to 128 query
 * rows (all heads of up to 128 / G readers) and multiplies them on the tensor cores, instead of once
 * per request; the result is the same up to fp32 rounding.  Default 4; 0 switches sharing off (every
 * request streams its whole cache).  Errors: INVALID_ARG. */
CART_API cart_status cart_set_share_min_readers(cart_ctx *ctx, int32_t min_readers);

/* How a batch with a shared part is run.  1 (default): the tensor-core kernel for the shared Cartridges and
 * the stream kernel for the requests' own tokens are resident at the same time, each on its share of the
 * SMs (the first is bound by latencies, the second by HBM bandwidth, which three quarters of the SMs nearly
 * saturate); the planner chooses the division.  0: one after the other, each on all SMs.  2 .. SMs - 1:
 * side by side with exactly this many blocks for the tensor-core kernel.  Results are the same up to fp32
 * rounding.  Errors: INVALID_ARG. */
CART_API cart_status cart_set_side_by_side(cart_ctx *ctx, int32_t mode);

/* Planner tuning.  The stream kernel's blocks are given equal shares of tiles + tiles_per_piece * pieces,
 * a piece being the part of a (request, KV head) cache that one block handles; the constant stands
 * for what finishing a piece (combining the warps' states, writing the result) costs a block, in
 * units of the time a 64-token tile takes.  Default 3; 0 balances by tiles alone; at most 64.  The
 * results do not depend on it beyond fp32 rounding.  Errors: INVALID_ARG. */
CART_API cart_status cart_set_piece_cost(cart_ctx *ctx, int32_t tiles_per_piece);

/* How cart_prefill_attention runs a message that is too short to give every SM a chain of tensor-core tiles (a
 * chain: 128 / G consecutive new tokens times a KV head, over the Cartridge(s) and the suffix up to the causal
 * diagonal).  -1 (default): with fewer chains than half the SMs, every chain is cut along its keys into as many
 * pieces of two tiles or more as give every SM one, and a merge kernel combines the pieces' partial results;
 * messages of fewer than 4 tokens go through the decode kernels.  0: short messages go through the decode kernels
 * (the shared tiles on the tensor cores, each row's stretch of the causal diagonal streamed by itself).  1 .. 64:
 * cut into this many pieces (1: whole chains, however few).  Results are the same up to fp32 rounding.
 * Errors: INVALID_ARG. */
CART_API cart_status cart_set_prefill_split(cart_ctx *ctx, int32_t pieces);

/* Plan reuse.  The attention calls split the batch's KV tokens over the thread blocks on the host (a
 * "plan") and upload the result.  In a decode loop (Sec. 2.3) every request grows by one token per step, so
 * a plan is kept while the batch is the same and every request has grown by the same number of tokens, at
 * most max_grow_tokens, since the plan was built; the kernels add that number to the last run of every
 * request.  Default 192; 0 builds a new plan whenever a length has changed.  Results are the same up to
 * fp32 rounding.  Errors: INVALID_ARG. */
CART_API cart_status cart_set_plan_reuse(cart_ctx *ctx, int32_t max_grow_tokens);

/* Number of plans this context has built and uploaded so far (a decode loop that keeps its plan does
 * not advance it). */
CART_API uint64_t cart_plan_count(const cart_ctx *ctx);

/* Current suffix length of a request in a layer (host-side mirror). */
CART_API cart_status cart_suffix_len(cart_ctx *ctx, cart_req req, int32_t layer, int32_t *out_len /*host*/);

/* KV bytes a request attends to, summed over layers (Sec. 3.2: a Cartridge costs what a p-token
 * prompt costs).  logical counts every Cartridge token as if private; unique_private counts only
 * the request's own suffix tokens (what is not shared with other requests). */
CART_API cart_status cart_kv_bytes(cart_ctx *ctx, cart_req req, uint64_t *logical /*host*/,
                          uint64_t *unique_private /*host*/);

/* Synchronises `stream` and reports the device-side status word: CART_OK, or CART_ERR_TIMEOUT if a
 * kernel gave up on a bounded wait since the last call (the word is then cleared). */
CART_API cart_status cart_sync_status(cart_ctx *ctx, void *stream);

/* Kernel timing for the benchmark's roofline line.  With timing enabled, every decode-attention
 * call's kernels (the shared-segment kernel, if the batch shares a Cartridge, and the stream kernel; not
 * the append) are bracketed by one pair of CUDA events on their stream.  cart_get_timing synchronises the recorded events, returns the summed kernel time in
 * milliseconds and the number of launches since the last call, and forgets them.  At most 8192
 * launches are remembered between two reads; later ones go untimed.  Errors: INVALID_ARG, CUDA. */
CART_API cart_status cart_set_timing(cart_ctx *ctx, int32_t enable);
CART_API cart_status cart_get_timing(cart_ctx *ctx, double *total_ms /*host*/, uint64_t *n_launches /*host*/);

/* Decode attention for callers that cannot allocate.  (The paper has no counterpart; this is a
 * convenience of the library.)  The entry points above need an arena from the caller and pinned
 * staging memory from cart_create.  Callers that may call neither cudaMalloc nor a framework's
 * allocator -- code running while a memory pool is frozen, a plug-in that is only handed tensors,
 * an early health check -- can use this one call instead: it needs no context, and the kernels'
 * scratch (work list, split partials; CART_STATIC_SCRATCH_BYTES) lives in a fixed device array inside
 * the library image, which every GPU that loads the library holds until the process exits.
 *
 * Computes the same result as cart_decode_attention for n_reqs requests that each attend over their
 * own n_tokens KV tokens: q and out are device bf16 [n_reqs][n_q_heads][128]; kv is ONE device
 * buffer, 256-byte aligned, bf16 [2][n_reqs][n_kv_heads][n_tokens][128] (all keys, then all values);
 * lse is device fp32 [n_reqs][n_q_heads] or NULL; softmax_scale 0 => 1/sqrt(128).  `device` must be
 * the current CUDA device and the one the buffers live on.
 *
 * Limits: n_reqs * n_kv_heads <= CART_STATIC_MAX_ROW_GROUPS, 2 * n_reqs * n_kv_heads * n_tokens < 2^31,
 * n_q_heads / n_kv_heads <= 8, device < 64; anything larger returns CART_ERR_CAPACITY and launches
 * nothing.  The call runs no cudaMalloc, cudaFree, cudaHostAlloc or other allocating routine.
 *
 * The first call on a device also does that device's one-time set-up (it looks up the scratch
 * array's device address and raises the kernel's shared-memory limit); make that first call before
 * any stream capture begins.  The work list is copied from ordinary (pageable) host memory, so the
 * call may wait for earlier work on `stream` before it returns.  All calls share the one scratch
 * array, which keeps the previous call's contents (the call clears what it needs zeroed): calls
 * whose GPU work may overlap -- different streams, different host threads -- race and must be
 * ordered by the caller.  The host copy of the work list is one fixed array too, so calls from different
 * host threads must not overlap either.  A device-side wait that ran out is not reported by this entry
 * point.  A CART_ERR_CUDA return may leave the clearing of the scratch or the copy of the work list
 * enqueued on `stream` (harmless: the next call redoes both).
 * Errors: INVALID_ARG, SHAPE, CAPACITY, CUDA. */
#define CART_STATIC_MAX_ROW_GROUPS 2048
#define CART_STATIC_SCRATCH_BYTES 2228224
CART_API cart_status cart_decode_attention_static(const void *q /*device*/, const void *kv /*device*/,
                                                  int32_t n_reqs, int32_t n_q_heads, int32_t n_kv_heads,
                                                  int32_t n_tokens, float softmax_scale, void *out /*device*/,
                                                  float *lse /*device or NULL*/, int32_t device, void *stream);

/* Number of kernels this context has launched so far (for the benchmark's launch count). */
CART_API uint64_t cart_launch_count(const cart_ctx *ctx);

CART_API const char *cart_status_string(cart_status s);
CART_API const char *cart_last_error(const cart_ctx *ctx);

#ifdef __cplusplus
}
#endif
#endif /* CART_H_ */
