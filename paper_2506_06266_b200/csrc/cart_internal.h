// Internal declarations shared by the host API (cart_api.cc) and the kernels (cart_kernels.cu).
#ifndef CART_INTERNAL_H_
#define CART_INTERNAL_H_

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "cart_plan.h"

namespace cart {

constexpr int kHeadDim = 128;
constexpr int kRowBytes = kHeadDim * 2;  // one token of one KV head: 128 bf16
constexpr int kTileTokens = 64;          // tokens per shared-memory stage
constexpr int kEdgeBoxRows = 32;         // tokens per box when a ragged last tile is fetched piecewise
constexpr int kMaxGroup = 8;             // query heads per KV head the kernels support
constexpr int kShareTileTokens = 128;    // tokens per tile of the shared-segment kernel
constexpr int kAppendBatch = 256;        // requests one append launch takes (kernel-parameter budget)

// bits of the device status word
constexpr uint32_t kStatusTimeoutProducer = 1u;
constexpr uint32_t kStatusTimeoutConsumer = 2u;
constexpr uint32_t kStatusTimeoutMma = 4u;

struct DecodeParams {
    const uint32_t *cta_begin;   // [grid + 1]
    const cart_work_item *items;
    const void *q;               // bf16 [n_reqs][Hq][128]
    const void *k_new = nullptr; // fused append: bf16 [n_reqs][Hkv][128] written to the suffix ends; else null
    const void *v_new = nullptr;
    void *arena = nullptr;                 // base of the row heap (row r is at arena + 256 r)
    void *out;                   // bf16 [n_reqs][Hq][128]
    float *lse;                  // fp32 [n_reqs][Hq] or null
    float *part_o;               // fp32 [slot][G][128], normalised partial outputs
    float *part_lse2;            // fp32 [slot][kMaxGroup], base-2 log-sum-exp of a partial
    const cart_merge_item *merges;  // split row groups (which slots belong together)
    uint32_t *tickets;           // one arrival counter per merge item, zero between launches; null: the
                                 // merge kernel runs afterwards and nobody takes tickets
    uint32_t *status;
    int32_t layer;
    int32_t group;               // G
    float scale_log2;            // softmax scale * log2(e)
    // Side by side with the shared-segment kernel (launched right after this one, resident at the same
    // time): once this kernel knows that the kernels before it are complete, block 0 stores 1 here and
    // the shared kernel, which cannot learn it from griddepcontrol.wait without waiting for this kernel
    // too, reads it; the shared kernel's last block clears it on its way out.  Null otherwise.
    uint32_t *ready_flag = nullptr;
    uint32_t grow = 0;           // tokens every request has appended since the plan was built: added to the token
                                 // count of every item marked CART_ITEM_TAIL
    const uint32_t *grow_ctr = nullptr;  // if set, that number is read from here instead (a launch recorded in a CUDA
                                         // graph cannot carry it as a parameter); a kernel earlier on the stream
                                         // advances it, so it is read only after griddepcontrol.wait
    uint32_t edge_boxes = 0;     // 1: ragged last tiles are fetched in boxes of kEdgeBoxRows rows through the second
                                 // tensor map; 0: every tile is fetched whole
    const uint32_t *pages = nullptr;  // page list of the batch (base row of every page of every paged suffix), read by
                                      // items marked CART_ITEM_PAGED
};

// Parameters of the shared-segment kernel (units and reader tables as the planner lays them out).
struct SharedParams {
    const uint32_t *unit_cta_begin;  // [grid + 1]
    const cart_shared_unit *units;
    const uint32_t *readers;         // batch index per reader entry
    const uint32_t *reader_slot;     // [entry * Hkv + KV head]: first partial slot; + unit.chunk
    const uint32_t *reader_merge;    // [entry * Hkv + KV head]: merge item
    const cart_merge_item *merges;
    const void *q;                   // bf16 [n_reqs][Hq][128]
    void *out;
    float *lse;
    float *part_o;
    float *part_lse2;
    uint32_t *tickets;
    uint32_t *status;
    int32_t layer;
    int32_t group;
    int32_t n_kv_heads;
    int32_t n_q_heads;
    float scale_log2;
    // Side by side with the stream kernel (launched right before this one): "the kernels before the pair
    // are complete" is read from this flag (1 once they are) instead of griddepcontrol.wait, which this kernel
    // then only executes on its way out, so that it never completes before the stream kernel; the block that
    // leaves last (counted in the word behind the flag) clears the flag for the next pair.  No launch number is
    // involved, so the pair can be recorded into a CUDA graph.  Null: alone.
    uint32_t *ready_flag = nullptr;
    const uint32_t *pages = nullptr;  // page list (units marked CART_UNIT_PAGED)
};

struct MergeParams {
    const cart_merge_item *merges;
    const float *part_o;
    const float *part_lse2;
    void *out;
    float *lse;
    int32_t group;
};

struct AppendEntry {
    uint32_t k_row;        // destination row of KV head 0 (layer and position applied)
    uint32_t v_row;
    uint32_t head_stride;  // rows between KV heads
};

struct AppendParams {
    AppendEntry e[kAppendBatch];
    void *arena;
    const void *k_new;  // bf16 [n][Hkv][128], already offset to the first request of this launch
    const void *v_new;
    int32_t n;
    int32_t n_kv_heads;
};

struct ExtendParams {
    void *arena;
    const void *k;  // bf16 [T][Hkv][128]
    const void *v;
    uint32_t k_row; // destination row of KV head 0, first new token
    uint32_t v_row;
    uint32_t head_stride;
    int32_t n_tokens;
    int32_t n_kv_heads;
};

// ---- training-time attention (backward) ---------------------------------------------------------
// One unit of the backward kernel's work: a tile of up to 128 keys of one KV head -- of the shared Cartridge
// or of a conversation -- against a range of row tiles.  Rows are (token, head of the group) pairs in
// token-major order; a row tile holds the 128 / G tokens [rt * tpt, (rt + 1) * tpt) of the packed batch.
struct TrainItem {
    uint32_t k_row;       // arena row of the tile's first key in layer 0 (KV head applied); values at v_row
    uint32_t v_row;
    uint32_t layer_stride;
    uint32_t n_keys;      // valid keys in the tile (1 .. 128)
    uint32_t kv_head;
    uint32_t rt_begin;    // row tiles [rt_begin, rt_end)
    uint32_t rt_end;
    uint32_t rt_first;    // the tile the loop starts with (it wraps around): items that share rows start apart
    uint32_t key_tok0;    // conversation tile: packed token index of key 0; Cartridge tile: 0
    uint32_t tok_end;     // conversation tile: one past the conversation's last token; Cartridge tile: T
    uint32_t causal;      // 1: key j is seen by rows of tokens >= key_tok0 + j only (conversation tile)
    uint32_t dst_row;     // row of key 0 in the gradient tensors: Cartridge [Hkv][p] -> kv_head * p + key;
                          // conversation [T][Hkv] -> token * Hkv + kv_head (dst_stride = Hkv rows between keys)
    uint32_t dst_stride;
    uint32_t is_z;        // 1: gradients go to dzk / dzv, else to dk / dv
    uint32_t pad[2];
};

struct TrainBwdParams {
    const TrainItem *items;
    const float *lse;     // fp32 [T][Hq], natural log (forward)
    const float *delta;   // fp32 [T][Hq]: <dout, out> per row
    float *dq;            // fp32 [T][Hq][128]
    float *dk, *dv;       // fp32 [T][Hkv][128]
    float *dzk, *dzv;     // fp32 [Hkv][p][128]
    uint32_t *status;
    int32_t layer;
    int32_t group;        // G
    int32_t n_q_heads;
    int32_t n_tokens;     // T
    float scale;          // softmax scale
};

struct TrainDeltaParams {
    const void *out;      // bf16 [T][Hq][128]
    const void *dout;     // bf16 [T][Hq][128]
    float *delta;         // fp32 [T][Hq]
    int32_t n_rows;       // T * Hq
};

// Launch configuration shared by the decode kernels: the kernel may start (become resident, run its
// prologue) before the kernel before it on the stream has finished; it orders itself with
// griddepcontrol.wait.
inline cudaLaunchConfig_t pdl_config(int grid, int block, size_t smem, cudaStream_t s, cudaLaunchAttribute *attr)
{
    attr->id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr->val.programmaticStreamSerializationAllowed = 1;
    cudaLaunchConfig_t c{};
    c.gridDim = dim3((unsigned)grid);
    c.blockDim = dim3((unsigned)block);
    c.dynamicSmemBytes = smem;
    c.stream = s;
    c.attrs = attr;
    c.numAttrs = 1;
    return c;
}

// Launchers (defined in cart_kernels.cu).  Each returns the cudaError_t of the launch.
size_t decode_smem_bytes();
int decode_threads();
cudaError_t prepare_kernels();  // sets the dynamic shared-memory attribute; call once per device
// tmap: boxes of kTileTokens rows x 64 elements; tmap_edge: the same matrix in boxes of kEdgeBoxRows rows (only read
// when p.edge_boxes is set; otherwise pass tmap twice)
cudaError_t launch_decode(const CUtensorMap &tmap, const CUtensorMap &tmap_edge, const DecodeParams &p, int grid,
                          cudaStream_t s);
cudaError_t prepare_shared_kernel();
// chains: the plan holds chained / masked / directly written units (see CART_UNIT_CONT in cart_plan.h)
cudaError_t launch_shared(const CUtensorMap &tmap, const SharedParams &p, int grid, cudaStream_t s, bool chains = false);
cudaError_t launch_merge(const MergeParams &p, int n_merges, cudaStream_t s);
cudaError_t launch_advance(uint32_t *ctr, cudaStream_t s);
cudaError_t launch_append(const AppendParams &p, cudaStream_t s);
cudaError_t launch_extend(const ExtendParams &p, cudaStream_t s);
cudaError_t prepare_train_kernels();
cudaError_t launch_train_delta(const TrainDeltaParams &p, cudaStream_t s);
// tmap: the arena (boxes of 64 rows x 64 elements); tmap_q / tmap_do: q and dout as [T][Hq][128] in boxes of
// 128 / G tokens x G heads x 64 elements
// tmap_dq: dq as fp32 [T][Hq][128] in boxes of 128 / G tokens x G heads x 32 elements (written by bulk reductions)
cudaError_t launch_train_bwd(const CUtensorMap &tmap, const CUtensorMap &tmap_q, const CUtensorMap &tmap_do,
                             const CUtensorMap &tmap_dq, const TrainBwdParams &p, int n_items, cudaStream_t s);

}  // namespace cart
#endif
